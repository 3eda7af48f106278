"""Pins for the oracle's tree expansion (Algorithm 2, Eq. 2-5) against things other than itself:
a hand-worked example, brute-force enumeration in probability space, closed forms, invariants."""
import itertools
import math
import os
import random

import numpy as np
import pytest

from oracle import talon_oracle as O
from paper_2601_07353_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------- hand-worked
def test_handworked_example():
    """Algorithm 2 / Eq. 3-5 worked by hand (tests/golden/handworked_expand.txt)."""
    dist = {
        (2,): [0.50, 0.30, 0.15, 0.05],
        (2, 0): [0.90, 0.05, 0.03, 0.02],
        (2, 1): [0.40, 0.35, 0.15, 0.10],
        (2, 0, 0): [0.25, 0.25, 0.25, 0.25],
        (2, 1, 0): [0.70, 0.10, 0.10, 0.10],
        (2, 1, 1): [0.05, 0.05, 0.10, 0.80],
    }
    rows = [l.split() for l in open(os.path.join(GOLDEN, "handworked_expand.txt")) if not l.startswith("#")]
    want = [(int(a), int(b), int(c), int(d), float(e)) for a, b, c, d, e in rows]

    def logits_fn(path):
        # a shifted log-probability row: softmax undoes the shift
        return (np.log(np.asarray(dist[tuple(path)], np.float64)) + 1.5).astype(np.float32)

    p = O.Params(budget=7, root_topk=2, cand_topk=4, mu=0.25, max_depth=10)
    t = O.expand(2, logits_fn, p)
    assert t.n_nodes == 7
    for node, par, tok, dep, prob in want:
        assert t.parent[node] == par and t.token[node] == tok and t.depth[node] == dep
        assert math.exp(t.score[node]) == pytest.approx(prob, rel=1e-6)
    assert t.layer_off == [0, 1, 3, 5, 7]


# ----------------------------------------------------------------------------- brute force
def brute_force_tree(root, row_of, V, N, K, mu, max_depth):
    """Eq. 3-5 + budget truncation with every candidate materialised, in probability space.
    Returns the set of root-to-node token paths and the list of layer sizes."""
    nodes = [((root,), 1.0)]            # (path, p)
    frontier = [0]
    layers = []
    d = 0
    while len(nodes) < N and d < max_depth and frontier:
        pool = []
        for v in frontier:
            path, pv = nodes[v]
            z = [float(x) for x in row_of(path)]
            zmax = max(z)
            e = [math.exp(x - zmax) for x in z]
            tot = sum(e)
            for w in range(V):
                pool.append((pv * e[w] / tot, v, w))
        pool.sort(key=lambda u: (-u[0], u[1], u[2]))
        if d == 0:
            keep = pool[:K]
        else:
            m = pool[0][0]
            keep = [u for u in pool if u[0] >= mu * m]
        keep = keep[: N - len(nodes)]
        keep.sort(key=lambda u: (u[1], u[2]))
        frontier = []
        for pu, v, w in keep:
            frontier.append(len(nodes))
            nodes.append((nodes[v][0] + (w,), pu))
        layers.append(len(keep))
        d += 1
    return nodes, layers


@pytest.mark.parametrize("trial", range(60))
def test_bruteforce_probability_space(trial):
    rng = random.Random(1000 + trial)
    V = rng.randint(2, 8)
    N = rng.randint(2, 10)
    K = rng.randint(1, 4)
    mu = rng.choice([0.03, 0.1, 0.3, 0.6, 1.0])
    max_depth = rng.randint(1, 3)
    scale = rng.choice([0.5, 1.5, 4.0])
    cache = {}

    def row_of(path):
        path = tuple(path)
        if path not in cache:
            r = np.random.default_rng(abs(hash((trial,) + path)) % (2 ** 32))
            cache[path] = (r.standard_normal(V) * scale).astype(np.float32)
        return cache[path]

    p = O.Params(budget=N, root_topk=K, cand_topk=V, mu=mu, max_depth=max_depth)
    t = O.expand(3, row_of, p)
    nodes, layers = brute_force_tree(3, row_of, V, N, K, mu, max_depth)
    assert t.n_nodes == len(nodes)
    for i in range(t.n_nodes):
        assert tuple(O.path_tokens(t, i)) == nodes[i][0]
        assert math.exp(t.score[i]) == pytest.approx(nodes[i][1], rel=1e-9)
    assert [t.layer_off[i + 2] - t.layer_off[i + 1] for i in range(len(layers))] == layers


def test_candidate_cap_at_least_remaining_is_exact():
    """A parent can never place more than N-|T| children, so a cap k >= N-1 equals the full pool."""
    cfg = synth.CONFIGS["tiny"].scaled(vocab=500, budget=12)
    for seq in range(6):
        fn = lambda path: synth.draft_logits_row(cfg, 7, seq, path)
        full = O.expand(1, fn, O.Params(12, 4, 500, 0.03, 8))
        capped = O.expand(1, fn, O.Params(12, 4, 11, 0.03, 8))
        assert full.n_nodes == capped.n_nodes
        assert (full.token == capped.token).all() and (full.parent == capped.parent).all()


# ----------------------------------------------------------------------------- closed forms
def test_all_equal_logits_is_pure_tiebreak():
    V, N, K, k = 50, 14, 3, 3
    t = O.expand(0, lambda path: np.zeros(V, np.float32), O.Params(N, K, k, 0.03, 8))
    assert t.n_nodes == N
    assert list(t.token[1:4]) == [0, 1, 2] and list(t.parent[1:4]) == [0, 0, 0]
    # layer 1: every candidate ties; parents 1,2,3 each offer tokens 0..2 and all 9 fit
    assert list(t.parent[4:13]) == [1, 1, 1, 2, 2, 2, 3, 3, 3]
    assert list(t.token[4:13]) == [0, 1, 2] * 3
    # layer 2: one slot left; lowest parent index, lowest token id
    assert t.parent[13] == 4 and t.token[13] == 0


def test_dominant_spike_gives_topk_plus_chain():
    V, K, k, Dmax = 300, 4, 4, 9
    rng = np.random.default_rng(5)

    def row(path):
        z = rng.standard_normal(V).astype(np.float32) * 0.1
        z[(sum(path) * 7 + 1) % V] += 20.0
        return z

    for N in (8, 12, 40):
        t = O.expand(0, row, O.Params(N, K, k, 0.03, Dmax))
        assert t.n_nodes == min(N, 1 + K + (Dmax - 1))
        assert t.depth[: t.n_nodes].max() == min(N - K, Dmax)
        # below the root layer every layer holds exactly one node
        sizes = [t.layer_off[i + 1] - t.layer_off[i] for i in range(len(t.layer_off) - 1)]
        assert sizes[0] == 1 and sizes[1] == K and all(s == 1 for s in sizes[2:])


def test_mu_one_keeps_only_the_anchor():
    cfg = synth.CONFIGS["tiny"].scaled(vocab=400, spike="none")
    t = O.expand(5, lambda path: synth.draft_logits_row(cfg, 3, 0, path), O.Params(12, 4, 4, 1.0, 20))
    sizes = [t.layer_off[i + 1] - t.layer_off[i] for i in range(len(t.layer_off) - 1)]
    assert sizes[1] == 4 and all(s == 1 for s in sizes[2:]) and t.n_nodes == 12


def test_tiny_mu_makes_each_layer_a_pure_top_r():
    V = 64
    cfg = synth.CONFIGS["tiny"].scaled(vocab=V, spike="none")
    fn = lambda path: synth.draft_logits_row(cfg, 11, 0, path)
    N, K = 20, 3
    t = O.expand(5, fn, O.Params(N, K, V, 1e-300, 20))
    # layer 1 must be the top (N-1-K) of all 3*V candidates by score
    pool = []
    for v in (1, 2, 3):
        z = fn(O.path_tokens(t, v)).astype(np.float64)
        lp = z - (z.max() + math.log(np.exp(z - z.max()).sum()))
        pool += [(t.score[v] + lp[w], v, w) for w in range(V)]
    pool.sort(key=lambda u: (-u[0], u[1], u[2]))
    want = sorted((v, w) for _, v, w in pool[: N - 1 - K])
    got = [(int(t.parent[i]), int(t.token[i])) for i in range(1 + K, N)]
    assert got == want


def test_root_layer_is_plain_topk():
    cfg = synth.CONFIGS["tiny"]
    z = synth.draft_logits_row(cfg, 1, 0, [17])
    t = O.new_tree(17, 16, 8)
    O.expand_layer(t, [z], O.Params(16, 4, 4, 0.03, 8))
    want = sorted(sorted(range(cfg.vocab), key=lambda w: (-float(z[w]), w))[:4])
    assert list(t.token[1:5]) == want
    lse = math.log(sum(math.exp(float(x)) for x in z))
    for i in range(1, 5):
        assert t.score[i] == pytest.approx(float(z[t.token[i]]) - lse, abs=1e-9)


def test_minus_inf_tokens_are_never_selected_and_nonfinite_rows_raise():
    V = 10
    z = np.full(V, -np.inf, np.float32)
    z[3] = 1.0
    z[7] = 0.5
    t = O.new_tree(0, 8, 4)
    assert O.expand_layer(t, [z], O.Params(8, 4, 4, 0.03, 4)) == 2      # only two tokens have p > 0
    assert list(t.token[1:3]) == [3, 7]
    for bad in (np.nan, np.inf):
        zz = np.zeros(V, np.float32)
        zz[2] = bad
        with pytest.raises(O.NonFiniteLogits):
            O.expand_layer(O.new_tree(0, 8, 4), [zz], O.Params(8, 4, 4, 0.03, 4))
    with pytest.raises(O.NonFiniteLogits):
        O.expand_layer(O.new_tree(0, 8, 4), [np.full(V, -np.inf, np.float32)], O.Params(8, 4, 4, 0.03, 4))


# ----------------------------------------------------------------------------- invariants
def closure_by_brute_force(parent, n, cap):
    m = np.zeros((cap, cap), bool)
    for i in range(n):
        j = i
        while j >= 0:
            m[i, j] = True
            j = parent[j]
    return m


@pytest.mark.parametrize("name,vocab,seq", [("tiny", 32000, 0), ("tiny", 32000, 1), ("llama8b", 4096, 0),
                                            ("llama8b", 4096, 3), ("longctx", 2048, 2), ("qwen32b", 3000, 1)])
def test_structural_invariants(name, vocab, seq):
    cfg = synth.CONFIGS[name].scaled(vocab=vocab)
    p = O.Params(cfg.budget, cfg.topk, cfg.topk, cfg.mu, cfg.max_depth)
    root = synth.root_token(cfg, 9, seq)
    t = O.expand(root, lambda path: synth.draft_logits_row(cfg, 9, seq, path), p)
    n = t.n_nodes
    if t.layers_run < cfg.max_depth:
        assert n == cfg.budget                      # the budget is met exactly unless the depth stop binds
    assert n <= cfg.budget
    for i in range(1, n):
        par = t.parent[i]
        assert 0 <= par < i
        assert t.depth[i] == t.depth[par] + 1
    for d in range(t.layers_run + 1):
        lo, hi = t.layer_off[d], t.layer_off[d + 1]
        assert all(t.depth[i] == d for i in range(lo, hi))
        keys = [(t.parent[i], t.token[i]) for i in range(lo, hi)]
        assert keys == sorted(keys) and len(set(keys)) == len(keys)
    fin = O.finalize(t, 100)
    dm = O.dense_mask(t)
    want = closure_by_brute_force(t.parent, n, cfg.budget)
    assert (dm[:n] == want[:n]).all()
    for i in range(n):
        assert bin(int(fin["mask"][i, 0]) | (int(fin["mask"][i, 1]) << 64 if fin["mask"].shape[1] > 1 else 0)).count("1") == t.depth[i] + 1
        assert fin["position"][i] == 100 + t.depth[i]
    for i in range(n, cfg.budget):
        assert fin["token"][i] == -1 and fin["parent"][i] == -1 and fin["position"][i] == -1
    # every node's score is the sum of its path's log-probabilities (Eq. 2)
    for i in range(1, n):
        path = O.path_tokens(t, i)
        s = 0.0
        for j in range(1, len(path)):
            z = synth.draft_logits_row(cfg, 9, seq, path[:j]).astype(np.float64)
            s += z[path[j]] - (z.max() + math.log(np.exp(z - z.max()).sum()))
        assert t.score[i] == pytest.approx(s, abs=1e-9)


def test_tree_shapes_follow_confidence():
    """Confident rows give deep-and-narrow trees, flat rows shallow-and-wide ones (Section 5.2)."""
    base = synth.CONFIGS["llama8b"].scaled(vocab=8192, max_depth=64)
    p = O.Params(base.budget, base.topk, base.topk, base.mu, base.max_depth)
    deep = O.expand(1, lambda path: synth.draft_logits_row(base.scaled(spike="all8"), 2, 0, path), p)
    wide = O.expand(1, lambda path: synth.draft_logits_row(base.scaled(spike="none"), 2, 0, path), p)
    assert deep.n_nodes == wide.n_nodes == base.budget
    assert deep.depth.max() > 3 * wide.depth.max()
    assert wide.layers_run <= 3


def test_zipf_rows_shape_the_tree():
    """Micro-benchmark rows: alpha=5 is near-deterministic (chain), alpha=0.7 is wide."""
    V = 32000
    p = O.Params(60, 10, 10, 0.03, 64)
    chain = O.expand(1, lambda path: synth.zipf_logits_row(V, 5.0, 1, len(path)), p)
    wide = O.expand(1, lambda path: synth.zipf_logits_row(V, 0.7, 1, len(path)), p)
    # rank 2 has relative probability 2^-5 = 0.03125 >= mu at alpha = 5, so layer d holds the d+1
    # paths with at most one rank-2 step: narrow and deep; alpha = 0.7 spends the budget in two layers
    assert chain.depth.max() >= 3 * wide.depth.max()
    assert wide.layers_run == 2
