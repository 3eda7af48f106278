"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle on the same seeded inputs.

Integer outputs (token ids, topology, positions, masks, accepted paths) must match bit for bit,
except for selection differences between candidates whose fp64 oracle scores lie within 1e-5,
which are logged and counted.  Attention must match within max-abs 1e-2 and mean-abs 1e-3 of the
fp64 oracle evaluated on the same bf16-rounded inputs."""
import math

import numpy as np
import pytest
import torch

from oracle import talon_oracle as O
from paper_2601_07353_b200 import synth
from tests import parity_util as PU

pytestmark = pytest.mark.gpu

ATT_MAX_ABS, ATT_MEAN_ABS = 1e-2, 1e-3
SEED = synth.DEFAULT_SEED


def _mods():
    from paper_2601_07353_b200 import talon, workload
    return talon, workload


def check_expansion(cfg, wl, seqs, cand_topk=None, init_layers=1, seed=SEED):
    p = PU.oracle_params(cfg, cand_topk, init_layers)
    tolerated = 0
    for bi in seqs:
        s = wl.seq_ids[bi]
        g = PU.tree_to_host(wl.tree, bi)
        fn = lambda path: synth.draft_logits_row(cfg, seed, s, path)
        t, tol = PU.follow_tree(cfg, p, synth.root_token(cfg, seed, s), fn, g["token"], g["parent"], g["n_nodes"],
                                g["layer_off"], f"{cfg.name}[seq {s}]")
        tolerated += tol
        fin = O.finalize(t, synth.prefix_len(cfg, seed, s))
        PU.compare_tree_arrays(fin, g, f"{cfg.name}[seq {s}]")
    return tolerated


def check_verify(cfg, wl, seqs, heads=None, seed=SEED):
    """Tree attention and greedy acceptance of sequences `seqs` against the oracle."""
    Hq, Hkv, Dh, N = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.budget
    starts = wl.kv_start.cpu().numpy()
    plens = wl.prefix_len.cpu().numpy()
    worst_max = worst_mean = 0.0
    for bi in seqs:
        g = PU.tree_to_host(wl.tree, bi)
        t = PU.oracle_tree_from_arrays(g, N, cfg.max_depth)
        f32 = lambda x: x.to(torch.float32).cpu().numpy()
        a, L = int(starts[bi]), int(plens[bi])
        hs = list(range(Hq)) if heads is None else heads
        kvs = sorted({h // cfg.group for h in hs})
        q = f32(wl.q[bi])[:, hs]
        # oracle call on the selected heads only: rebuild a dense sub-problem with matching grouping
        outs = []
        for h in hs:
            kv = h // cfg.group
            o = O.tree_attention(f32(wl.q[bi][:, h:h + 1]), f32(wl.k_prefix[a:a + L, kv:kv + 1]),
                                 f32(wl.v_prefix[a:a + L, kv:kv + 1]), f32(wl.k_tree[bi][:, kv:kv + 1]),
                                 f32(wl.v_tree[bi][:, kv:kv + 1]), t, 1.0 / math.sqrt(Dh))
            outs.append(o[:, 0])
        want = np.stack(outs, axis=1)
        got = wl.out[bi].to(torch.float64).cpu().numpy()[:, hs]
        err = np.abs(got - want)
        worst_max, worst_mean = max(worst_max, err.max()), max(worst_mean, err.mean())
        assert err.max() <= ATT_MAX_ABS and err.mean() <= ATT_MEAN_ABS, f"{cfg.name}[{bi}] attention {err.max()} {err.mean()}"
        assert (got[g["n_nodes"]:] == 0).all()
        # acceptance
        y = wl.target[bi].cpu().numpy()
        tt = O.target_argmax(y, g["n_nodes"])
        alen, path, bonus = O.accept(t, tt)
        assert (wl.target_tok[bi].cpu().numpy() == tt).all()
        assert int(wl.accept_len[bi]) == alen and int(wl.bonus_tok[bi]) == bonus
        nodes = wl.accept_nodes[bi].cpu().numpy()
        assert list(nodes[: alen + 1]) == path and (nodes[alen + 1:] == -1).all()
    return worst_max, worst_mean


def run_config(cfg, seqs=None, check_seqs=None, heads=None, cand_topk=None, init_layers=1):
    talon, workload = _mods()
    t = workload.make_talon(cfg, batch_max=len(seqs) if seqs else cfg.batch, cand_topk=cand_topk, init_layers=init_layers)
    wl = workload.build_workload(cfg, t, SEED, seqs)
    workload.run_step(t, wl)           # the whole step again on the cached inputs (what bench.py times)
    assert t.poll_status() == talon.OK
    check = list(range(wl.B)) if check_seqs is None else check_seqs
    tol = check_expansion(cfg, wl, check, cand_topk, init_layers)
    mx, mean = check_verify(cfg, wl, check, heads)
    print(f"{cfg.name}: tolerated selection differences {tol}; attention max-abs {mx:.2e} mean-abs {mean:.2e}; "
          f"n_nodes {wl.tree.n_nodes.cpu().tolist()} accept {wl.accept_len.cpu().tolist()}")
    t.close()
    return wl


def test_generator_matches_between_numpy_and_cuda():
    cfg = synth.CONFIGS["tiny"]
    a = synth.draft_logits_row(cfg, 3, 1, [4, 5, 6])
    b = synth.draft_logits_row(cfg, 3, 1, [4, 5, 6], device="cuda").cpu().numpy()
    assert (a.view(np.int32) == b.view(np.int32)).all()
    a = synth.target_logits_row(cfg, 3, 1, [4, 5, 6])
    b = synth.target_logits_row(cfg, 3, 1, [4, 5, 6], device="cuda").cpu().numpy()
    assert (a.view(np.int32) == b.view(np.int32)).all()
    a = synth.qkv_block(3, synth.STREAM_K, 2, 5000, None, 128)
    b = synth.qkv_block(3, synth.STREAM_K, 2, 5000, "cuda", 128).cpu().numpy()
    assert (a == b).all()


def test_tiny_full():
    run_config(synth.CONFIGS["tiny"])


@pytest.mark.parametrize("seq", [1, 2, 3, 4, 5])
def test_tiny_other_sequences(seq):
    run_config(synth.CONFIGS["tiny"], seqs=[seq])


def test_llama8b_full():
    run_config(synth.CONFIGS["llama8b"], heads=[0, 5, 13, 31])


def test_llama8b_batched_full_sampled():
    run_config(synth.CONFIGS["llama8b_batched"], check_seqs=[0, 7, 15], heads=[1, 30])


def test_llama8b_batched_small_vocab_all_sequences():
    run_config(synth.CONFIGS["llama8b_batched"].scaled(vocab=5000, prefix_min=0, prefix_max=300), heads=[0, 9, 31])


def test_qwen32b_full_sampled():
    run_config(synth.CONFIGS["qwen32b"], check_seqs=[0, 5], heads=[3, 60])


def test_longctx_full_sampled():
    run_config(synth.CONFIGS["longctx"], check_seqs=[4, 29], heads=[2, 17])


def test_longctx_small_all_sequences():
    run_config(synth.CONFIGS["longctx"].scaled(vocab=3000, batch=8, prefix_min=1, prefix_max=700), heads=[0, 31])


@pytest.mark.parametrize("vocab", [8, 100, 1000, 1028, 4100, 33000])
def test_odd_vocabulary_sizes(vocab):
    cfg = synth.CONFIGS["tiny"].scaled(vocab=vocab, batch=3, prefix_min=5, prefix_max=130)
    run_config(cfg, heads=[0, 31])


def test_paper_exact_pool_mode():
    """cand_topk = 0 keeps N-1 candidates per parent, which equals Eq. 3's whole-vocabulary pool."""
    cfg = synth.CONFIGS["llama8b"].scaled(vocab=2048, batch=4, prefix_min=10, prefix_max=90, budget=40)
    talon, workload = _mods()
    t = workload.make_talon(cfg, cand_topk=0)
    wl = workload.build_workload(cfg, t, SEED)
    assert t.poll_status() == talon.OK
    assert check_expansion(cfg, wl, range(4), cand_topk=cfg.vocab) == 0
    t.close()
    cfg = synth.CONFIGS["longctx"].scaled(vocab=1024, batch=2, prefix_min=10, prefix_max=20)
    t = workload.make_talon(cfg, cand_topk=0)
    wl = workload.build_workload(cfg, t, SEED, with_verify=False)
    check_expansion(cfg, wl, range(2), cand_topk=cfg.vocab)
    t.close()


@pytest.mark.parametrize("init_layers", [0, 2, 3])
def test_init_layer_variants(init_layers):
    cfg = synth.CONFIGS["llama8b"].scaled(vocab=4096, batch=4, prefix_min=64, prefix_max=64)
    run_config(cfg, heads=[7], init_layers=init_layers)


@pytest.mark.parametrize("mu", [1.0, 0.5, 1e-6])
def test_threshold_extremes(mu):
    cfg = synth.CONFIGS["tiny"].scaled(vocab=2000, batch=4, mu=mu, budget=40, max_depth=30)
    run_config(cfg, heads=[0])


def test_depth_stop_leaves_sentinels():
    cfg = synth.CONFIGS["llama8b"].scaled(vocab=3000, spike="all8", max_depth=5, batch=2)
    wl = run_config(cfg, heads=[0, 1])
    assert (wl.tree.n_nodes.cpu().numpy() < cfg.budget).all()


def test_repeatable_bits():
    talon, workload = _mods()
    cfg = synth.CONFIGS["llama8b"].scaled(vocab=16384, batch=3, prefix_min=100, prefix_max=900)
    t = workload.make_talon(cfg)
    wl = workload.build_workload(cfg, t, SEED)
    snaps = []
    for _ in range(3):
        workload.run_step(t, wl)
        torch.cuda.synchronize()
        snaps.append([x.clone() for x in (wl.tree.token, wl.tree.parent, wl.tree.score, wl.tree.mask, wl.out,
                                          wl.accept_nodes, wl.bonus_tok)])
    for s in snaps[1:]:
        for a, b in zip(snaps[0], s):
            assert torch.equal(a, b)
    t.close()


def test_more_than_32_sequences():
    """Above 32 sequences the frontier geometry goes through shared memory instead of registers."""
    cfg = synth.CONFIGS["tiny"].scaled(vocab=4096, batch=40, prefix_min=3, prefix_max=200)
    run_config(cfg, heads=[0, 17])


@pytest.mark.parametrize("k,budget", [(16, 64), (32, 100), (12, 128)])
def test_wide_candidate_lists_on_the_fused_kernel(k, budget):
    """Per-parent caps up to 32 stay on the fused kernel (different lane-group sizes for the bound)."""
    cfg = synth.CONFIGS["tiny"].scaled(vocab=8192, batch=3, topk=k, budget=budget, max_depth=10, prefix_min=20,
                                      prefix_max=90)
    run_config(cfg, heads=[3])
    cfg = synth.CONFIGS["llama8b"].scaled(batch=2, topk=k, budget=budget, prefix_min=64, prefix_max=64)
    run_config(cfg, heads=[3])


@pytest.mark.parametrize("alpha", [0.7, 1.35, 5.0])
def test_zipf_rows_of_the_papers_micro_benchmark(alpha):
    """Expansion on the appendix's Zipf rows (P(rank r) ~ r^-alpha): the same tree as the oracle's.
    Each row is generated once on the host and handed to both sides."""
    talon, workload = _mods()
    V, N, K, D = 32000, 60, 10, 8
    t = talon.Talon(batch_max=1, vocab=V, budget=N, root_topk=K, cand_topk=K, max_depth=D, mu=0.03, n_q_heads=32,
                    n_kv_heads=8, head_dim=128)
    rows = {}

    def row(path):                                    # a node's row depends on its token path only
        key = tuple(path)
        if key not in rows:
            rows[key] = synth.zipf_logits_row(V, alpha, 5, len(rows))
        return rows[key]

    p = O.Params(N, K, K, 0.03, D)
    want = O.expand(7, row, p)
    tree = t.alloc_tree(1)
    dev = tree.token.device
    draft = torch.zeros(1, N, V, dtype=torch.float32, device=dev)
    t.reset(tree, torch.tensor([7], dtype=torch.int32, device=dev), torch.zeros(1, dtype=torch.int32, device=dev))
    for d in range(D):
        n = int(tree.n_nodes[0])
        tok, par = tree.token[0].cpu().numpy(), tree.parent[0].cpu().numpy()
        paths = workload.node_paths(tok, par, n)
        for i in range(n):
            draft[0, i] = torch.from_numpy(row(paths[i])).to(dev)
        t.expand_layer(tree, draft)
    t.build_tree(tree)
    assert t.poll_status() == talon.OK
    g = PU.tree_to_host(tree, 0)
    # every row is a permutation of the same values, so path scores of different parents tie exactly
    # in exact arithmetic: the comparison goes through the tolerated-tie rule
    followed, tolerated = PU.follow_tree(None, p, 7, row, g["token"], g["parent"], g["n_nodes"], g["layer_off"],
                                         f"zipf alpha {alpha}")
    PU.compare_tree_arrays(O.finalize(followed, 0), g, f"zipf alpha {alpha}")
    assert want.n_nodes == g["n_nodes"]
    print(f"zipf alpha {alpha}: n_nodes {g['n_nodes']}, tolerated ties {tolerated}")
    t.close()
