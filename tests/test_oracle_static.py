"""Pins of the oracle's Algorithm 1 (static tree construction): a hand-worked example, the layer
structure the algorithm fixes, path probabilities recomputed with a library softmax, Top-K of a
sorted pool, and the pruning step as 'the N most probable nodes, which form a tree'."""
import math
import os

import numpy as np
import scipy.special

from oracle import talon_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "handworked_static.txt")


def _golden(section):
    rows, on = [], False
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line in ("unpruned", "pruned"):
            on = line == section
            continue
        if on:
            f = line.split()
            rows.append((int(f[1]), int(f[2]), int(f[3]), float(f[4])))
    return rows


def _handworked_rows(path):
    table = {(9,): [0.5, 0.3, 0.2], (9, 0): [0.1, 0.5, 0.4], (9, 1): [0.7, 0.2, 0.1]}
    p = table.get(tuple(path), [1 / 3, 1 / 3, 1 / 3])
    return np.log(np.asarray(p, np.float64)).astype(np.float32)


def test_handworked_example_of_algorithm_1():
    t = O.expand_static(9, _handworked_rows, width=2, depth=1)
    want = _golden("unpruned")
    assert t.n_nodes == len(want) == 5
    for i, (tok, par, dep, p) in enumerate(want):
        assert (t.token[i], t.parent[i], t.depth[i]) == (tok, par, dep)
        assert abs(math.exp(t.score[i]) - p) < 1e-6
    pr = O.prune_static(t, 4)
    want = _golden("pruned")
    assert pr.n_nodes == len(want) == 4
    for i, (tok, par, dep, p) in enumerate(want):
        assert (pr.token[i], pr.parent[i], pr.depth[i]) == (tok, par, dep)
        assert abs(math.exp(pr.score[i]) - p) < 1e-6


def _random_rows(seed, vocab):
    def fn(path):
        r = np.random.default_rng(abs(hash((seed,) + tuple(path))) % (1 << 32))
        z = r.normal(size=vocab) * 2.0
        z[r.integers(vocab)] += r.choice([0.0, 3.0, 8.0])
        return z.astype(np.float32)
    cache = {}
    return lambda path: cache.setdefault(tuple(path), fn(path))


def test_layers_have_width_k_and_scores_are_path_probabilities():
    for seed in range(12):
        V, K, D = 40, 4, 3
        fn = _random_rows(seed, V)
        t = O.expand_static(5, fn, K, D)
        assert t.n_nodes == 1 + K * (D + 1) and t.layer_off == [0, 1] + [1 + K * (d + 1) for d in range(D + 1)]
        for i in range(1, t.n_nodes):
            v = int(t.parent[i])
            assert t.depth[i] == t.depth[v] + 1 and v < i
            d = int(t.depth[i])
            assert t.layer_off[d] <= i < t.layer_off[d + 1] and t.layer_off[d - 1] <= v < t.layer_off[d]
            # p(u) = p(v) * P(u | v), the conditional from a library softmax of the parent's row
            logp = scipy.special.log_softmax(fn(O.path_tokens(t, v)).astype(np.float64))
            assert abs(t.score[i] - (t.score[v] + logp[t.token[i]])) < 1e-9
            # the token is among the parent's K most probable
            assert t.token[i] in np.argsort(-logp, kind="stable")[:K]
        # first layer: the root row's Top-K by a plain sort
        root = scipy.special.log_softmax(fn([5]).astype(np.float64))
        assert sorted(t.token[1:1 + K]) == sorted(np.argsort(-root, kind="stable")[:K])


def test_every_layer_is_the_top_k_of_its_pool():
    V, K, D = 25, 3, 2
    fn = _random_rows(77, V)
    t = O.expand_static(1, fn, K, D)
    for d in range(D + 1):
        parents = range(t.layer_off[d], t.layer_off[d + 1])
        pool = []
        for v in parents:
            logp = scipy.special.log_softmax(fn(O.path_tokens(t, v)).astype(np.float64))
            for w in np.argsort(-logp, kind="stable")[:K]:
                pool.append((t.score[v] + logp[w], v, int(w)))
        assert len(pool) == len(parents) * K                   # the K x K pool (K at the root)
        best = sorted(pool, key=lambda u: -u[0])[:K]
        got = [(int(t.parent[i]), int(t.token[i])) for i in range(t.layer_off[d + 1], t.layer_off[d + 2])]
        assert sorted((v, w) for _, v, w in best) == sorted(got)


def test_pruning_keeps_the_n_most_probable_nodes_and_they_form_a_tree():
    for seed in range(10):
        fn = _random_rows(100 + seed, 30)
        t = O.expand_static(2, fn, 4, 4)
        for keep in (1, 5, 9, 16, 21, 40):
            pr = O.prune_static(t, keep)
            n = min(keep, t.n_nodes)
            assert pr.n_nodes == n
            kept_scores = sorted(pr.score[:n], reverse=True)
            assert kept_scores == sorted(t.score[:t.n_nodes], reverse=True)[:n]
            closure = O.dense_mask(pr)
            for i in range(1, n):
                v = int(pr.parent[i])
                assert 0 <= v < i and pr.depth[i] == pr.depth[v] + 1
                assert closure[i, i] and closure[i, v] and (closure[i] >= closure[v]).all()
                assert bin(int(pr.mask[i, 0]) | (int(pr.mask[i, 1]) << 64 if pr.mask.shape[1] > 1 else 0)).count("1") == pr.depth[i] + 1
            assert pr.layer_off[-1] == n
