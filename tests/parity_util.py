"""Helpers shared by the GPU parity tests: run the oracle beside the CUDA path on the same
seeded inputs and compare, with the one tolerated exception (a selection difference between
candidates whose fp64 oracle scores differ by less than 1e-5), which is logged and counted."""
from __future__ import annotations

import math
from typing import Callable, List

import numpy as np

from oracle import talon_oracle as O
from paper_2601_07353_b200 import synth

TIE_EPS = 1e-5
tie_log: List[str] = []          # every tolerated selection difference, for the test report


def oracle_params(cfg, cand_topk=None, init_layers=1) -> O.Params:
    return O.Params(cfg.budget, cfg.topk, cfg.topk if cand_topk is None else cand_topk, cfg.mu, cfg.max_depth,
                    init_layers)


def follow_tree(cfg, p: O.Params, root_token: int, logits_fn: Callable, g_token, g_parent, g_nnodes: int,
                g_layer_off, label: str):
    """Re-run Algorithm 2 with the oracle, layer by layer, beside a tree the GPU produced.

    Returns (oracle tree, number of tolerated differences).  A layer where the two selections
    differ is accepted only if every candidate on either side of the difference lies within
    TIE_EPS (fp64 log-score) of the decision boundary; the oracle is then forced onto the GPU's
    choice so that later layers stay comparable.  Anything else raises AssertionError."""
    tree = O.new_tree(root_token, p.budget, p.max_depth)
    tolerated = 0
    while O.is_active(tree):
        d = tree.layers_run
        rows = [logits_fn(O.path_tokens(tree, v)) for v in tree.frontier]
        pool = O.layer_pool(tree, rows, p)
        remaining = tree.budget - tree.n_nodes
        chosen = O.select_layer(pool, d, remaining, p)
        want = sorted((v, w) for _, v, w in chosen)
        lo, hi = int(g_layer_off[d + 1]), int(g_layer_off[d + 2])
        got = [(int(g_parent[i]), int(g_token[i])) for i in range(lo, hi)]
        if got != want:
            scores = {(v, w): s for s, v, w in pool}
            assert len(got) == len(want) and got == sorted(got), f"{label}: layer {d} size/order differs"
            diff = set(got) ^ set(want)
            assert all(u in scores for u in diff), f"{label}: layer {d}: GPU chose a non-candidate"
            # decision boundary: the worst selected score, or the gate threshold
            bounds = [min(s for s, _, _ in chosen)]
            if d >= p.init_layers:
                bounds.append(math.log(p.mu) + max(s for s, _, _ in pool))
            for u in diff:
                assert min(abs(scores[u] - b) for b in bounds) < TIE_EPS, \
                    f"{label}: layer {d}: selection differs beyond the tie tolerance at {u}"
            tolerated += 1
            tie_log.append(f"{label} layer {d}: {sorted(diff)}")
            chosen = [(scores[u], u[0], u[1]) for u in got]
        # append (same statements as the oracle's expand_layer, on the agreed selection)
        chosen = sorted(chosen, key=lambda u: (u[1], u[2]))
        for s, v, w in chosen:
            i = tree.n_nodes
            tree.token[i], tree.parent[i], tree.depth[i], tree.score[i] = w, v, tree.depth[v] + 1, s
            tree.mask[i] = tree.mask[v]
            tree.mask[i, i // 64] |= np.uint64(1) << np.uint64(i % 64)
            tree.n_nodes += 1
        tree.layer_off.append(tree.n_nodes)
        tree.layers_run += 1
    assert tree.n_nodes == g_nnodes, f"{label}: n_nodes {g_nnodes} != oracle {tree.n_nodes}"
    return tree, tolerated


def compare_tree_arrays(fin: dict, g: dict, label: str, score_tol=2e-5):
    """Bit-exact comparison of every integer output; scores within score_tol (absolute, log)."""
    n = fin["n_nodes"]
    assert g["n_nodes"] == n, label
    for name in ("token", "parent", "depth", "position"):
        assert (np.asarray(g[name]) == fin[name]).all(), f"{label}: {name} differs"
    assert (np.asarray(g["mask"]).astype(np.uint64) == fin["mask"]).all(), f"{label}: mask differs"
    assert (np.asarray(g["layer_off"]) == fin["layer_off"]).all(), f"{label}: layer_off differs"
    gs, os_ = np.asarray(g["score"]), fin["score"]
    assert np.isneginf(gs[n:]).all() and np.abs(gs[:n] - os_[:n]).max() <= score_tol, f"{label}: score differs"


def tree_to_host(tree, b: int) -> dict:
    return dict(n_nodes=int(tree.n_nodes[b].item()), token=tree.token[b].cpu().numpy(),
                parent=tree.parent[b].cpu().numpy(), depth=tree.depth[b].cpu().numpy(),
                position=tree.position[b].cpu().numpy(), layer_off=tree.layer_off[b].cpu().numpy(),
                score=tree.score[b].cpu().numpy(), mask=tree.mask[b].cpu().numpy().view(np.uint64))


def oracle_tree_from_arrays(g: dict, budget: int, max_depth: int) -> O.Tree:
    """An oracle Tree object holding a given topology (used to feed attention/accept oracles)."""
    t = O.new_tree(int(g["token"][0]), budget, max_depth)
    n = g["n_nodes"]
    t.token[:n], t.parent[:n], t.depth[:n] = g["token"][:n], g["parent"][:n], g["depth"][:n]
    for i in range(1, n):
        t.mask[i] = t.mask[t.parent[i]]
        t.mask[i, i // 64] |= np.uint64(1) << np.uint64(i % 64)
    t.n_nodes = n
    return t


SAMPLE_EPS = 1e-6
sample_log: List[str] = []       # every tolerated sampling decision, for the test report


def follow_sampling(tree: O.Tree, rows, u_accept, u_sample: float, temperature: float, g_len: int, g_path,
                    g_tok: int, label: str) -> int:
    """Checks a sampling verification the GPU produced against the oracle's procedure, decision by
    decision along the GPU's path.  The GPU decides in fp64 from fp32 row statistics, so a decision
    whose two sides differ by less than SAMPLE_EPS (relative) may fall either way: such a decision is
    logged and counted, anything else must agree.  Returns the number of tolerated decisions; when it
    is 0 the GPU result equals ``O.accept_stochastic`` outright (checked too)."""
    tolerated = 0
    cur = 0
    assert int(g_path[0]) == 0, f"{label}: path does not start at the root"
    step = 0
    while True:
        p = O.target_posterior(rows[cur], temperature)
        mass = 1.0
        nxt = -1
        g_next = int(g_path[step + 1]) if step < g_len else -1
        for c in O.children_of(tree, cur):
            w = int(tree.token[c])
            lhs = float(u_accept[c]) * mass
            take = lhs < p[w]
            g_take = (c == g_next)
            if take != g_take:
                assert abs(lhs - p[w]) <= SAMPLE_EPS * max(p[w], lhs), \
                    f"{label}: node {cur} child {c}: accept decision differs (u*mass {lhs}, p {p[w]})"
                tolerated += 1
                sample_log.append(f"{label}: accept decision at child {c}")
                take = g_take
            if take:
                nxt = c
                break
            mass -= p[w]
            p[w] = 0.0
        assert nxt == g_next, f"{label}: after node {cur} the GPU went to {g_next}, the procedure to {nxt}"
        if nxt < 0:
            break
        cur = nxt
        step += 1
    assert step == g_len, f"{label}: accepted length {g_len} vs {step}"
    cdf = np.cumsum(p)
    total = cdf[-1]
    target = float(u_sample) * total
    want = min(int(np.searchsorted(cdf, target, side="right")), int(np.nonzero(p > 0.0)[0][-1]))
    if g_tok != want:
        assert 0 <= g_tok < len(p) and p[g_tok] > 0.0, f"{label}: correction token {g_tok} has no mass"
        lo, hi = cdf[g_tok] - p[g_tok], cdf[g_tok]
        tol = SAMPLE_EPS * total
        assert lo - tol <= target <= hi + tol, f"{label}: correction token {g_tok} vs {want} beyond tolerance"
        tolerated += 1
        sample_log.append(f"{label}: correction token {g_tok} vs {want}")
    if tolerated == 0:
        alen, path, tok = O.accept_stochastic(tree, rows, u_accept, u_sample, temperature)
        assert (alen, path, tok) == (g_len, [int(x) for x in g_path[: g_len + 1]], g_tok), label
    return tolerated
