"""GPU parity on the layouts and shapes the other tests do not reach: vocabularies that are not a
multiple of four, row strides wider than the vocabulary (NaN between the rows), a sequence with an
empty prefix inside a batch, and query-group sizes that take the warp-MMA attention kernel."""
import math

import numpy as np
import pytest
import torch

from oracle import talon_oracle as O
from paper_2601_07353_b200 import synth
from tests import parity_util as PU

pytestmark = pytest.mark.gpu
SEED = 4711
ATT_MAX_ABS, ATT_MEAN_ABS = 1e-2, 1e-3


def _mods():
    from paper_2601_07353_b200 import talon, workload
    return talon, workload


def _check_all(cfg, t, wl, talon, temperature=None):
    """Expansion, attention and greedy acceptance of every sequence of ``wl`` against the oracle
    (prefix lengths taken from the workload, so overrides are honoured)."""
    p = PU.oracle_params(cfg)
    plens = wl.prefix_len.cpu().numpy()
    starts = wl.kv_start.cpu().numpy()
    f32 = lambda x: x.to(torch.float32).cpu().numpy()
    for bi, s in enumerate(wl.seq_ids):
        g = PU.tree_to_host(wl.tree, bi)
        fn = lambda path: synth.draft_logits_row(cfg, wl.seed, s, path)
        tr, _ = PU.follow_tree(cfg, p, synth.root_token(cfg, wl.seed, s), fn, g["token"], g["parent"], g["n_nodes"],
                               g["layer_off"], f"{cfg.name}[seq {s}]")
        PU.compare_tree_arrays(O.finalize(tr, int(plens[bi])), g, f"{cfg.name}[seq {s}]")
        a, L = int(starts[bi]), int(plens[bi])
        want = O.tree_attention(f32(wl.q[bi]), f32(wl.k_prefix[a:a + L]), f32(wl.v_prefix[a:a + L]), f32(wl.k_tree[bi]),
                                f32(wl.v_tree[bi]), tr, 1.0 / math.sqrt(cfg.head_dim))
        err = np.abs(wl.out[bi].to(torch.float64).cpu().numpy() - want)
        assert err.max() <= ATT_MAX_ABS and err.mean() <= ATT_MEAN_ABS, f"attention [{bi}] {err.max()} {err.mean()}"
        assert (wl.out[bi][g["n_nodes"]:] == 0).all()
        tt = O.target_argmax(wl.target[bi].cpu().numpy(), g["n_nodes"])
        alen, path, bonus = O.accept(tr, tt)
        assert (wl.target_tok[bi].cpu().numpy() == tt).all()
        assert int(wl.accept_len[bi]) == alen and int(wl.bonus_tok[bi]) == bonus
        assert list(wl.accept_nodes[bi].cpu().numpy()[: alen + 1]) == path
        if temperature is not None:
            n = g["n_nodes"]
            rows = [wl.target[bi, i].cpu().numpy() for i in range(n)]
            ua, us = synth.verify_uniforms(wl.seed, s, cfg.budget, 0)
            yield bi, tr, rows, ua, us


@pytest.mark.parametrize("vocab,row_pad", [(1001, 0), (1001, 8), (32001, 0), (32002, 4), (4099, 12), (32000, 8)])
def test_odd_vocabulary_and_padded_rows(vocab, row_pad):
    """V % 4 != 0 and row_stride > V with NaN in the padding: expansion, target argmax, the softmax
    statistics of the sampling verification and the walk all have to stay inside the rows."""
    talon, workload = _mods()
    cfg = synth.CONFIGS["tiny"].scaled(vocab=vocab, batch=3, prefix_min=40, prefix_max=200)
    t = workload.make_talon(cfg)
    wl = workload.build_workload(cfg, t, SEED, row_pad=row_pad)
    assert wl.draft.stride(-2) % 4 == 0 and wl.draft.stride(-2) >= vocab
    workload.run_step(t, wl)
    assert t.poll_status() == talon.OK
    T = 0.8
    todo = list(_check_all(cfg, t, wl, talon, temperature=T))
    ua = torch.from_numpy(np.stack([x[3] for x in todo])).cuda()
    us = torch.tensor([x[4] for x in todo], dtype=torch.float64, device="cuda")
    s_tok = torch.zeros(len(todo), dtype=torch.int32, device="cuda")
    t.accept_sample(wl.tree, wl.target, T, ua, us, wl.accept_len, wl.accept_nodes, s_tok)
    assert t.poll_status() == talon.OK
    for bi, tr, rows, u_a, u_s in todo:
        PU.follow_sampling(tr, rows, u_a, u_s, T, int(wl.accept_len[bi]), wl.accept_nodes[bi].cpu().numpy(), int(s_tok[bi]),
                           f"V={vocab} pad={row_pad} [{bi}]")
    t.close()


def test_empty_prefix_inside_a_batch():
    """A sequence with L_b = 0 between two sequences with a prefix: it attends to tree keys only."""
    talon, workload = _mods()
    cfg = synth.CONFIGS["tiny"].scaled(batch=3, prefix_min=0, prefix_max=300)
    t = workload.make_talon(cfg)
    wl = workload.build_workload(cfg, t, SEED, prefix_lens=[130, 0, 257])
    assert wl.prefix_len.cpu().tolist() == [130, 0, 257]
    workload.run_step(t, wl)
    assert t.poll_status() == talon.OK
    list(_check_all(cfg, t, wl, talon))
    t.close()


def test_all_prefixes_empty():
    talon, workload = _mods()
    cfg = synth.CONFIGS["tiny"].scaled(batch=2, prefix_min=0, prefix_max=0)
    t = workload.make_talon(cfg)
    wl = workload.build_workload(cfg, t, SEED)
    workload.run_step(t, wl)
    assert t.poll_status() == talon.OK
    list(_check_all(cfg, t, wl, talon))
    t.close()


@pytest.mark.parametrize("hq,hkv,batch", [(24, 8, 1), (24, 8, 24), (28, 4, 2), (12, 2, 40), (40, 8, 3)])
def test_group_sizes_that_do_not_divide_128(hq, hkv, batch):
    """g = 3, 5, 6, 7: packed query rows do not tile 128-row blocks by whole nodes, so the warp-MMA
    kernel runs, with split-KV (few CTAs) and without (many sequences)."""
    talon, workload = _mods()
    cfg = synth.CONFIGS["tiny"].scaled(n_q_heads=hq, n_kv_heads=hkv, batch=batch, prefix_min=100, prefix_max=700,
                                       vocab=8000)
    assert 128 % cfg.group != 0
    t = workload.make_talon(cfg)
    wl = workload.build_workload(cfg, t, SEED)
    workload.run_step(t, wl)
    assert t.poll_status() == talon.OK
    launches = t.launch_count()
    workload.run_step(t, wl)
    per_step = t.launch_count() - launches
    # reset + D expansions + build + attention (+ combine when the keys are split) + argmax (+ walk, unless folded)
    assert per_step in (cfg.max_depth + 4, cfg.max_depth + 5, cfg.max_depth + 6)
    list(_check_all(cfg, t, wl, talon))
    t.close()


@pytest.mark.parametrize("mode", ["0", "2"])
@pytest.mark.parametrize("batch,prefix", [(1, 700), (1, 2900), (3, 1500)])
def test_key_ranges_merged_in_a_cluster_or_by_the_second_kernel(mode, batch, prefix, monkeypatch):
    """Few sequences: a (sequence, head) is cut into key ranges.  Their partial results are merged
    either through the distributed shared memory of a thread-block cluster (forced here for every
    size: 2 to 8 ranges per cluster, ragged last range, unused query tile) or by a second kernel;
    both against the oracle, and against each other within the rounding of the final division."""
    talon, workload = _mods()
    monkeypatch.setenv("TALON_ATTN_CLUSTER", mode)                   # read when the context is made
    cfg = synth.CONFIGS["tiny"].scaled(batch=batch, prefix_min=prefix, prefix_max=prefix + 130, vocab=8000)
    t = workload.make_talon(cfg)
    wl = workload.build_workload(cfg, t, SEED)
    launches = t.launch_count()
    workload.run_step(t, wl)
    per_step = t.launch_count() - launches
    assert t.poll_status() == talon.OK
    list(_check_all(cfg, t, wl, talon))
    if mode == "2":
        assert per_step <= cfg.max_depth + 4         # reset, layers, build, attention (merged in the kernel), arg-max
    t.close()
