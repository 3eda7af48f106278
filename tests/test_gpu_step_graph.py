"""talon_step replays a captured graph from the second call with the same arguments: the replays
must give what the plain launch sequence gives, read their inputs afresh, and count their launches."""
import numpy as np
import pytest
import torch

from paper_2601_07353_b200 import synth
from tests import test_gpu_parity as GP

pytestmark = pytest.mark.gpu


def _snapshot(wl):
    tr = wl.tree
    return [x.clone() for x in (tr.n_nodes, tr.token, tr.parent, tr.depth, tr.position, tr.layer_off, tr.score, tr.mask,
                                wl.out, wl.accept_len, wl.accept_nodes, wl.bonus_tok, wl.target_tok)]


def test_replayed_steps_equal_plain_steps_and_read_fresh_inputs():
    from paper_2601_07353_b200 import talon, workload
    cfg = synth.CONFIGS["tiny"].scaled(batch=3, prefix_min=50, prefix_max=400)
    t = workload.make_talon(cfg)
    wl = workload.build_workload(cfg, t, GP.SEED)
    workload.run_step(t, wl)                        # entry by entry: the reference result
    torch.cuda.synchronize()
    want = _snapshot(wl)
    per_step = None
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        for call in range(5):                       # 1: plain, 2: capture + replay, 3..: replay
            for x in (wl.tree.token, wl.out, wl.accept_len, wl.bonus_tok):
                x.zero_()
            before = t.launch_count()
            workload.run_step_fused(t, wl)
            side.synchronize()
            assert t.poll_status() == talon.OK
            n = t.launch_count() - before
            per_step = n if per_step is None else per_step
            assert n == per_step and n > 0          # replays count the kernels they launch
            assert t.layers_run() == cfg.max_depth
            for a, b in zip(want, _snapshot(wl)):
                assert torch.equal(a, b), f"call {call}"
        # same pointers, new contents: a replay must pick them up
        wl.root_tok[0] = (int(wl.root_tok[0]) + 1) % cfg.vocab
        workload.run_step_fused(t, wl)
        side.synchronize()
        assert int(wl.tree.token[0, 0]) == int(wl.root_tok[0])
    GP.check_verify(cfg, wl, [1, 2])                # untouched sequences still match the oracle
    t.close()


def test_timed_and_default_stream_steps_take_the_plain_path():
    from paper_2601_07353_b200 import talon, workload
    cfg = synth.CONFIGS["tiny"]
    t = workload.make_talon(cfg)
    wl = workload.build_workload(cfg, t, GP.SEED)
    for _ in range(3):                              # legacy default stream: never captured
        workload.run_step_fused(t, wl)
    torch.cuda.synchronize()
    assert t.poll_status() == talon.OK
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        for _ in range(3):
            workload.run_step_fused(t, wl)
        t.timing_enable(64)
        workload.run_step_fused(t, wl)              # bracketed by events: launched one by one
        kt = t.timing_read()
        assert kt["expand_rows"][1] == cfg.max_depth and kt["tree_attention"][1] == 1
        t.timing_enable(0)
        workload.run_step_fused(t, wl)
        side.synchronize()
    assert t.poll_status() == talon.OK
    GP.check_expansion(cfg, wl, [0])
    GP.check_verify(cfg, wl, [0])
    t.close()


@pytest.mark.parametrize("name,seqs,heads", [("llama8b", None, None), ("llama8b_batched", [0, 9, 15], [0, 31])])
def test_full_size_replayed_step_matches_the_oracle(name, seqs, heads):
    """The launch configuration the benchmark times (talon_step on its own stream, replaying its
    captured graph) against the oracle at full size."""
    from paper_2601_07353_b200 import talon, workload
    cfg = synth.CONFIGS[name]
    t = workload.make_talon(cfg)
    wl = workload.build_workload(cfg, t, GP.SEED)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        for _ in range(4):
            workload.run_step_fused(t, wl)
        side.synchronize()
    assert t.poll_status() == talon.OK
    check = list(range(wl.B)) if seqs is None else seqs
    GP.check_expansion(cfg, wl, check)
    GP.check_verify(cfg, wl, check, heads)
    t.close()


def test_more_argument_sets_than_graph_slots():
    """The library keeps 64 captured steps; with 70 argument sets in rotation the least recently used
    ones are dropped and re-captured, and every step still gives the same result."""
    from paper_2601_07353_b200 import talon, workload
    cfg = synth.CONFIGS["tiny"].scaled(vocab=4096, batch=2, prefix_min=30, prefix_max=60)
    t = workload.make_talon(cfg)
    wl = workload.build_workload(cfg, t, GP.SEED)
    workload.run_step(t, wl)
    torch.cuda.synchronize()
    want = wl.out.clone()
    want_tok = wl.tree.token.clone()
    outs = [torch.zeros_like(wl.out) for _ in range(70)]
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        for rnd in range(3):
            for o in outs:
                wl.out = o                      # a different output pointer is a different argument set
                workload.run_step_fused(t, wl)
        side.synchronize()
    assert t.poll_status() == talon.OK
    for o in outs:
        assert torch.equal(o, want)
    assert torch.equal(wl.tree.token, want_tok)
    t.close()


@pytest.mark.parametrize("batch,layers", [(1, None), (3, 2), (24, None), (24, 1)])
def test_close_and_accept_equals_build_then_accept(batch, layers):
    """The tail of a step in one call: the accept walk's warp writes what talon_build_tree writes
    (positions, sentinel slots, the unused tail of the layer offsets) before it walks.  Small batches
    take the route where the argmax kernel's last CTA walks, large ones the separate walk kernel;
    fewer layers than D_max leave layer offsets for the closing pass to fill."""
    from paper_2601_07353_b200 import talon, workload
    cfg = synth.CONFIGS["tiny"].scaled(batch=batch, prefix_min=20, prefix_max=300, vocab=8000)
    t = workload.make_talon(cfg)
    wl = workload.build_workload(cfg, t, GP.SEED)
    n_layers = cfg.max_depth if layers is None else layers
    tr = wl.tree

    def head():
        for x in (tr.token, tr.parent, tr.depth, tr.position, tr.layer_off, tr.mask, wl.accept_len, wl.accept_nodes,
                  wl.bonus_tok, wl.target_tok):
            x.fill_(77)                              # stale contents everywhere the tail must write
        tr.score.fill_(7.0)
        t.reset(tr, wl.root_tok, wl.prefix_len)
        for _ in range(n_layers):
            t.expand_layer(tr, wl.draft)

    head()
    t.build_tree(tr)
    t.accept(tr, wl.target, wl.accept_len, wl.accept_nodes, wl.bonus_tok, wl.target_tok)
    torch.cuda.synchronize()
    assert t.poll_status() == talon.OK
    want = _snapshot(wl)
    head()
    before = t.launch_count()
    t.close_and_accept(tr, wl.target, wl.accept_len, wl.accept_nodes, wl.bonus_tok, wl.target_tok)
    torch.cuda.synchronize()
    assert t.poll_status() == talon.OK
    assert t.launch_count() - before in (1, 2)       # argmax (+ walk): no closing launch
    names = ("n_nodes", "token", "parent", "depth", "position", "layer_off", "score", "mask", "out", "accept_len",
             "accept_nodes", "bonus_tok", "target_tok")
    for name, a, b in zip(names, want, _snapshot(wl)):
        if name == "score":
            assert torch.equal(a.view(torch.int64), b.view(torch.int64)), name     # -inf sentinels included
        else:
            assert torch.equal(a, b), name
    t.close()
