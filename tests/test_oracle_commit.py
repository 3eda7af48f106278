"""Pins for the generation-loop bookkeeping of Section 5.3: the committed cache is the prefix
followed by the accepted path's rows, the counts follow Algorithm 2's loop, and delta, tau and R
satisfy the wall-time identity they are derived from."""
import numpy as np

from oracle import talon_oracle as O
from paper_2601_07353_b200 import synth
from tests.test_oracle_verify import make_tree


def test_commit_appends_the_accepted_path_in_order():
    rng = np.random.default_rng(1)
    tree = make_tree(parents=[-1, 0, 0, 1, 1, 3], tokens=[9, 4, 7, 2, 8, 5])
    tree.layers_run = 3
    L, hkv, dh = 5, 2, 4
    kp, vp = rng.standard_normal((L, hkv, dh)), rng.standard_normal((L, hkv, dh))
    kt, vt = rng.standard_normal((6, hkv, dh)), rng.standard_normal((6, hkv, dh))
    k2, v2, root, counts = O.commit(tree, 3, [0, 1, 3, 5, -1], 11, kt, vt, kp, vp)
    assert k2.shape == (L + 4, hkv, dh) and root == 11 and counts == (1, 3, 4)
    # written out: the old rows are untouched, then node 0, 1, 3, 5 one by one
    for t in range(L):
        assert (k2[t] == kp[t]).all() and (v2[t] == vp[t]).all()
    for j, node in enumerate([0, 1, 3, 5]):
        assert (k2[L + j] == kt[node]).all() and (v2[L + j] == vt[node]).all()
    # nothing accepted: only the root joins, one token (the correction) is produced
    k3, v3, root, counts = O.commit(tree, 0, [0, -1, -1], 2, kt, vt, kp, vp)
    assert k3.shape[0] == L + 1 and (k3[L] == kt[0]).all() and counts == (1, 3, 1)


def test_draft_passes_are_the_layers_algorithm_2_expands():
    cfg = synth.CONFIGS["tiny"]
    p = O.Params(cfg.budget, cfg.topk, cfg.topk, cfg.mu, cfg.max_depth)
    for seq in range(4):
        t = O.expand(synth.root_token(cfg, 7, seq), lambda path: synth.draft_logits_row(cfg, 7, seq, path), p)
        # one pass per layer that had a frontier and budget left: all layers but the deepest,
        # unless the depth stop ended the loop first
        depth = int(t.depth[: t.n_nodes].max())
        assert t.layers_run == depth
        assert t.layers_run == len(t.layer_off) - 2


def test_speedup_formula_is_the_wall_time_ratio():
    """R = L T_p / (N_p T_p + N_q T_q) (the definition) must equal tau / (1 + c delta)."""
    rng = np.random.default_rng(2)
    for _ in range(50):
        L, n_p, n_q = int(rng.integers(50, 2000)), int(rng.integers(10, 400)), int(rng.integers(10, 3000))
        t_p, t_q = float(rng.uniform(5, 50)), float(rng.uniform(0.1, 5))
        direct = (L * t_p) / (n_p * t_p + n_q * t_q)
        tau, delta = O.mean_accepted_tokens(L, n_p), O.draft_efficiency(n_q, n_p)
        assert abs(O.speedup(tau, delta, t_q / t_p) - direct) < 1e-12 * direct
    # a static tree of depth D spends D + 1 draft passes per verification: delta = D + 1
    D, steps = 8, 37
    assert O.draft_efficiency((D + 1) * steps, steps) == D + 1
    # free drafting (c = 0) gives R = tau; drafting as costly as verifying gives tau / (1 + delta)
    assert O.speedup(4.0, 9.0, 0.0) == 4.0 and O.speedup(4.0, 9.0, 1.0) == 0.4


def test_binding_loop_metrics_agree_with_the_oracle():
    import torch
    from paper_2601_07353_b200 import talon
    counters = torch.tensor([[3, 20, 11], [3, 31, 7], [2, 9, 9]], dtype=torch.int64)
    m = talon.loop_metrics(counters, 0.05)
    n_p, n_q, L = 8, 60, 27
    assert (m["n_p"], m["n_q"], m["tokens"]) == (n_p, n_q, L)
    assert abs(m["delta"] - O.draft_efficiency(n_q, n_p)) < 1e-15
    assert abs(m["tau"] - O.mean_accepted_tokens(L, n_p)) < 1e-15
    assert abs(m["speedup"] - O.speedup(L / n_p, n_q / n_p, 0.05)) < 1e-15
