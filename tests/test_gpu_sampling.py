"""Sampling verification (Appendix B steps 1-3) on the GPU against the oracle, decision by decision,
on the seeded workloads: every sequence of the small cases, sampled sequences of the full-size ones,
several independent draws of the uniforms each, plus the degenerate inputs."""
import numpy as np
import pytest
import torch

from oracle import talon_oracle as O
from paper_2601_07353_b200 import synth
from tests import parity_util as PU

pytestmark = pytest.mark.gpu
SEED = synth.DEFAULT_SEED


def _mods():
    from paper_2601_07353_b200 import talon, workload
    return talon, workload


def sample_and_check(cfg, seqs=None, check=None, temperatures=(1.0,), draws=3):
    talon, workload = _mods()
    t = workload.make_talon(cfg, batch_max=len(seqs) if seqs else cfg.batch)
    wl = workload.build_workload(cfg, t, SEED, seqs)
    B, N = wl.B, cfg.budget
    dev = wl.target.device
    alen = torch.zeros(B, dtype=torch.int32, device=dev)
    nodes = torch.zeros(B, cfg.max_depth + 1, dtype=torch.int32, device=dev)
    tok = torch.zeros(B, dtype=torch.int32, device=dev)
    check = list(range(B)) if check is None else check
    tolerated = 0
    lens = []
    for T in temperatures:
        for draw in range(draws):
            us = [synth.verify_uniforms(SEED, wl.seq_ids[bi], N, draw) for bi in range(B)]
            ua = torch.from_numpy(np.stack([u for u, _ in us])).to(dev)
            usamp = torch.tensor([s for _, s in us], dtype=torch.float64, device=dev)
            t.accept_sample(wl.tree, wl.target, T, ua, usamp, alen, nodes, tok)
            assert t.poll_status() == talon.OK
            for bi in check:
                g = PU.tree_to_host(wl.tree, bi)
                tree = PU.oracle_tree_from_arrays(g, N, cfg.max_depth)
                rows = wl.target[bi].cpu().numpy()
                gl = int(alen[bi])
                gp = nodes[bi].cpu().numpy()
                assert (gp[gl + 1:] == -1).all()
                tolerated += PU.follow_sampling(tree, rows, us[bi][0], us[bi][1], T, gl, gp, int(tok[bi]),
                                                f"{cfg.name}[seq {wl.seq_ids[bi]}] T={T} draw {draw}")
                lens.append(gl)
    print(f"{cfg.name}: sampling verification, tolerated decisions {tolerated}, accepted lengths {lens}")
    t.close()
    return tolerated


def test_tiny_all_sequences_three_temperatures():
    cfg = synth.CONFIGS["tiny"]
    sample_and_check(cfg, seqs=list(range(8)), temperatures=(1.0, 0.6, 0.2, 2.0), draws=4)


def test_llama8b_full():
    sample_and_check(synth.CONFIGS["llama8b"], temperatures=(1.0, 0.3, 0.15), draws=4)


def test_llama8b_batched_full_sampled():
    sample_and_check(synth.CONFIGS["llama8b_batched"], check=[0, 7, 15], temperatures=(1.0, 0.25), draws=2)


def test_qwen32b_full_sampled():
    sample_and_check(synth.CONFIGS["qwen32b"], check=[0, 5], temperatures=(1.0, 0.25), draws=2)


def test_longctx_full_sampled():
    sample_and_check(synth.CONFIGS["longctx"], check=[3, 31], temperatures=(1.0, 0.2), draws=1)


@pytest.mark.parametrize("vocab", [8, 100, 1028, 4100, 33000])
def test_odd_vocabulary_sizes(vocab):
    cfg = synth.CONFIGS["tiny"].scaled(vocab=vocab, batch=3, prefix_min=5, prefix_max=130)
    sample_and_check(cfg, temperatures=(1.0, 0.3), draws=3)


def _one_tree(cfg, seqs):
    talon, workload = _mods()
    t = workload.make_talon(cfg, batch_max=len(seqs))
    wl = workload.build_workload(cfg, t, SEED, seqs)
    dev = wl.target.device
    B = wl.B
    out = dict(alen=torch.zeros(B, dtype=torch.int32, device=dev),
               nodes=torch.zeros(B, cfg.max_depth + 1, dtype=torch.int32, device=dev),
               tok=torch.zeros(B, dtype=torch.int32, device=dev))
    return talon, t, wl, out


def test_extreme_uniforms_and_masked_tokens():
    cfg = synth.CONFIGS["tiny"]
    talon, t, wl, o = _one_tree(cfg, [0, 1])
    N, dev = cfg.budget, wl.target.device
    target = wl.target.clone()
    target[0, 0, 100:200] = -float("inf")                 # masked vocabulary entries have no mass
    g = [PU.tree_to_host(wl.tree, bi) for bi in range(2)]
    trees = [PU.oracle_tree_from_arrays(x, N, cfg.max_depth) for x in g]
    kids0 = [int(trees[0].token[c]) for c in O.children_of(trees[0], 0)]
    for ua_val, us_val in [(0.0, 0.0), (1.0 - 2.0 ** -53, 1.0 - 2.0 ** -53), (1.0 - 2.0 ** -53, 0.0)]:
        ua = torch.full((2, N), ua_val, dtype=torch.float64, device=dev)
        us = torch.full((2,), us_val, dtype=torch.float64, device=dev)
        t.accept_sample(wl.tree, target, 1.0, ua, us, o["alen"], o["nodes"], o["tok"])
        assert t.poll_status() == talon.OK
        for bi in range(2):
            PU.follow_sampling(trees[bi], target[bi].cpu().numpy(), np.full(N, ua_val), us_val, 1.0,
                               int(o["alen"][bi]), o["nodes"][bi].cpu().numpy(), int(o["tok"][bi]), f"extreme[{bi}]")
        if ua_val > 0.5:                                   # everything rejected at the root
            assert int(o["alen"][0]) == 0
            tok0 = int(o["tok"][0])
            assert tok0 not in kids0 and not (100 <= tok0 < 200)
    t.close()


def test_non_finite_row_and_bad_arguments():
    cfg = synth.CONFIGS["tiny"]
    talon, t, wl, o = _one_tree(cfg, [0, 1])
    N, dev = cfg.budget, wl.target.device
    ua = torch.full((2, N), 0.5, dtype=torch.float64, device=dev)
    us = torch.full((2,), 0.5, dtype=torch.float64, device=dev)
    for bad in (0.0, -1.0, float("nan"), float("inf")):
        with pytest.raises(talon.TalonError) as e:
            t.accept_sample(wl.tree, wl.target, bad, ua, us, o["alen"], o["nodes"], o["tok"])
        assert e.value.code == talon.ERR_INVALID_ARG
    target = wl.target.clone()
    target[1, 0, 7] = float("nan")
    t.accept_sample(wl.tree, target, 1.0, ua, us, o["alen"], o["nodes"], o["tok"])
    assert t.poll_status() == talon.ERR_NONFINITE
    assert int(o["alen"][1]) == 0 and int(o["tok"][1]) == -1
    # the healthy sequence is unaffected
    g = PU.tree_to_host(wl.tree, 0)
    PU.follow_sampling(PU.oracle_tree_from_arrays(g, N, cfg.max_depth), target[0].cpu().numpy(), np.full(N, 0.5), 0.5,
                       1.0, int(o["alen"][0]), o["nodes"][0].cpu().numpy(), int(o["tok"][0]), "healthy")
    t.close()


def test_one_hot_targets_give_the_greedy_result():
    """With a dominant target logit per row the sampling walk must equal talon_accept's."""
    cfg = synth.CONFIGS["tiny"]
    talon, t, wl, o = _one_tree(cfg, [0, 1, 2])
    N, dev = cfg.budget, wl.target.device
    target = wl.target.clone()
    top = target.argmax(dim=-1, keepdim=True)
    target.scatter_add_(-1, top, torch.full_like(top, 90.0, dtype=torch.float32))
    t.accept(wl.tree, target, wl.accept_len, wl.accept_nodes, wl.bonus_tok, wl.target_tok)
    us = [synth.verify_uniforms(SEED, s, N, 9) for s in wl.seq_ids]
    ua = torch.from_numpy(np.stack([u for u, _ in us])).to(dev)
    usamp = torch.tensor([s for _, s in us], dtype=torch.float64, device=dev)
    t.accept_sample(wl.tree, target, 1.0, ua, usamp, o["alen"], o["nodes"], o["tok"])
    assert t.poll_status() == talon.OK
    assert torch.equal(o["alen"], wl.accept_len) and torch.equal(o["nodes"], wl.accept_nodes)
    assert torch.equal(o["tok"], wl.bonus_tok)
    t.close()


def test_more_than_32_sequences():
    cfg = synth.CONFIGS["tiny"].scaled(vocab=4096, batch=40, prefix_min=3, prefix_max=200)
    sample_and_check(cfg, temperatures=(1.0, 0.3), draws=1)


def test_many_struck_children_in_the_full_pool_mode():
    """With the paper's whole-vocabulary pool a parent can hold dozens of children: walk to the node
    with the most children (uniform 0 along the way), reject them all there (uniform just below 1) and
    draw from what is left."""
    talon, workload = _mods()
    cfg = synth.CONFIGS["llama8b"].scaled(vocab=2048, batch=4, prefix_min=10, prefix_max=90, budget=100, mu=1e-4,
                                          spike="none")
    t = workload.make_talon(cfg, cand_topk=0)
    wl = workload.build_workload(cfg, t, SEED)
    N, dev, B = cfg.budget, wl.target.device, wl.B
    trees = [PU.oracle_tree_from_arrays(PU.tree_to_host(wl.tree, bi), N, cfg.max_depth) for bi in range(B)]
    ua = np.full((B, N), 1.0 - 2.0 ** -53)
    most = []
    for bi, tr in enumerate(trees):
        kids = [len(O.children_of(tr, v)) for v in range(tr.n_nodes)]
        end = int(np.argmax(kids))
        most.append(kids[end])
        v = end
        while v > 0:                      # accept everything on the way down to `end`
            ua[bi, v] = 0.0
            v = int(tr.parent[v])
    assert max(most) > 32, most
    alen = torch.zeros(B, dtype=torch.int32, device=dev)
    nodes = torch.zeros(B, cfg.max_depth + 1, dtype=torch.int32, device=dev)
    tok = torch.zeros(B, dtype=torch.int32, device=dev)
    us = np.array([0.1, 0.5, 0.9, 0.999])
    t.accept_sample(wl.tree, wl.target, 1.0, torch.from_numpy(ua).to(dev), torch.from_numpy(us).to(dev), alen, nodes, tok)
    assert t.poll_status() == talon.OK
    for bi in range(B):
        PU.follow_sampling(trees[bi], wl.target[bi].cpu().numpy(), ua[bi], float(us[bi]), 1.0, int(alen[bi]),
                           nodes[bi].cpu().numpy(), int(tok[bi]), f"full pool [{bi}]")
    t.close()
