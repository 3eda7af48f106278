"""Pins for the oracle's verification side (Appendix B): tree attention and greedy acceptance."""
import math
import random

import numpy as np
import pytest
import torch

from oracle import talon_oracle as O
from paper_2601_07353_b200 import synth


def make_tree(parents, tokens=None, cap=None):
    """Tree with given parent links (node order must be topological, layer by layer)."""
    n = len(parents)
    cap = cap or n
    t = O.new_tree(tokens[0] if tokens else 0, cap, 64)
    for i in range(1, n):
        v = parents[i]
        t.token[i] = tokens[i] if tokens else i
        t.parent[i] = v
        t.depth[i] = t.depth[v] + 1
        t.score[i] = 0.0
        t.mask[i] = t.mask[v]
        t.mask[i, i // 64] |= np.uint64(1) << np.uint64(i % 64)
    t.n_nodes = n
    return t


def rand_qkv(seed, n, L, hq, hkv, dh=16):
    r = np.random.default_rng(seed)
    f = lambda *s: synth.round_to_bf16(r.standard_normal(s).astype(np.float32))
    return f(n, hq, dh), f(L, hkv, dh), f(L, hkv, dh), f(n, hkv, dh), f(n, hkv, dh)


def test_chain_tree_is_causal_attention():
    """A chain-shaped tree must reduce to causal attention of the last n positions (Appendix B)."""
    n, L, hq, hkv, dh = 9, 37, 4, 2, 16
    q, kp, vp, kt, vt = rand_qkv(1, n, L, hq, hkv, dh)
    t = make_tree([-1] + list(range(n - 1)))
    scale = 1.0 / math.sqrt(dh)
    got = O.tree_attention(q, kp, vp, kt, vt, t, scale)
    K = torch.from_numpy(np.concatenate([kp, kt]).astype(np.float64)).permute(1, 0, 2)
    V = torch.from_numpy(np.concatenate([vp, vt]).astype(np.float64)).permute(1, 0, 2)
    K = K.repeat_interleave(hq // hkv, dim=0)
    V = V.repeat_interleave(hq // hkv, dim=0)
    Qfull = torch.zeros(hq, L + n, dh, dtype=torch.float64)
    Qfull[:, L:] = torch.from_numpy(q.astype(np.float64)).permute(1, 0, 2)
    ref = torch.nn.functional.scaled_dot_product_attention(Qfull, K, V, is_causal=True, scale=scale)
    ref = ref[:, L:].permute(1, 0, 2).numpy()
    assert np.abs(got - ref).max() < 1e-12


def test_star_tree_sees_prefix_root_and_self_only():
    n, L, hq, hkv, dh = 6, 11, 2, 1, 16
    q, kp, vp, kt, vt = rand_qkv(2, n, L, hq, hkv, dh)
    t = make_tree([-1, 0, 0, 0, 0, 0])
    got = O.tree_attention(q, kp, vp, kt, vt, t, 0.25)
    for i in range(n):
        keys = list(range(L)) + ([L] if i else []) + [L + i]
        K = np.concatenate([kp, kt]).astype(np.float64)[keys, 0]
        V = np.concatenate([vp, vt]).astype(np.float64)[keys, 0]
        for h in range(hq):
            s = K @ q[i, h].astype(np.float64) * 0.25
            p = np.exp(s - s.max())
            p /= p.sum()
            assert np.abs(got[i, h] - p @ V).max() < 1e-12


def test_attention_weights_sum_to_one_and_unused_rows_are_zero():
    n, cap, L, hq, hkv, dh = 5, 8, 20, 4, 4, 16
    q, kp, vp, kt, vt = rand_qkv(3, cap, L, hq, hkv, dh)
    vp[:] = 1.0
    vt[:] = 1.0
    t = make_tree([-1, 0, 1, 1, 0], cap=cap)
    out = O.tree_attention(q, kp, vp, kt, vt, t, 0.3)
    assert np.abs(out[:n] - 1.0).max() < 1e-12
    assert (out[n:] == 0).all()


def test_sibling_relabelling_permutes_outputs():
    """Swapping two sibling subtrees (with their q/k/v rows) permutes the outputs accordingly."""
    n, L, hq, hkv, dh = 7, 13, 2, 2, 16
    q, kp, vp, kt, vt = rand_qkv(4, n, L, hq, hkv, dh)
    # tree A: 0 -> {1, 2}; 1 -> {3, 4}; 2 -> {5, 6}.  tree B: same shape with 1<->2 and {3,4}<->{5,6}
    t = make_tree([-1, 0, 0, 1, 1, 2, 2])
    perm = [0, 2, 1, 5, 6, 3, 4]
    a = O.tree_attention(q, kp, vp, kt, vt, t, 0.2)
    b = O.tree_attention(q[perm], kp, vp, kt[perm], vt[perm], t, 0.2)
    assert np.abs(a[perm] - b).max() < 1e-12


def test_mask_excludes_non_ancestors():
    """Moving a non-ancestor's key/value must not change a node's output; moving an ancestor's must."""
    n, L, hq, hkv, dh = 5, 6, 1, 1, 16
    q, kp, vp, kt, vt = rand_qkv(5, n, L, hq, hkv, dh)
    t = make_tree([-1, 0, 0, 1, 2])
    base = O.tree_attention(q, kp, vp, kt, vt, t, 0.2)
    vt2 = vt.copy()
    vt2[2] += 1.0                                    # node 2 is not on node 3's path, but is on node 4's
    out = O.tree_attention(q, kp, vp, kt, vt2, t, 0.2)
    assert np.abs(out[3] - base[3]).max() == 0
    assert np.abs(out[4] - base[4]).max() > 1e-3


# ----------------------------------------------------------------------------- acceptance
def longest_matching_path(tree, t):
    """EAGLE's formulation: enumerate root-to-leaf paths, take the longest accepted prefix."""
    n = tree.n_nodes
    children = {i: [c for c in range(n) if tree.parent[c] == i] for i in range(n)}
    leaves = [i for i in range(n) if not children[i]]
    best = [0]
    for leaf in leaves:
        path = []
        j = leaf
        while j >= 0:
            path.append(j)
            j = int(tree.parent[j])
        path = path[::-1]
        ok = [0]
        for a, b in zip(path[:-1], path[1:]):
            if tree.token[b] == t[a]:
                ok.append(b)
            else:
                break
        if len(ok) > len(best):
            best = ok
    return best


@pytest.mark.parametrize("trial", range(40))
def test_accept_walk_equals_longest_matching_prefix(trial):
    rng = random.Random(trial)
    n = rng.randint(1, 24)
    V = 5
    parents, tokens = [-1], [rng.randrange(V)]
    layer, i = [0], 1
    while i < n:
        new = []
        for v in layer:
            for w in sorted(rng.sample(range(V), rng.randint(0, 3))):
                if i < n:
                    parents.append(v)
                    tokens.append(w)
                    new.append(i)
                    i += 1
        if not new:
            new = [i]
            parents.append(layer[0])
            tokens.append(0)
            i += 1
        layer = new
    tree = make_tree(parents, tokens)
    t = np.array([rng.randrange(V) for _ in range(n)], np.int32)
    alen, path, bonus = O.accept(tree, t)
    want = longest_matching_path(tree, t)
    assert path == want and alen == len(want) - 1 and bonus == t[want[-1]]


def test_accept_all_on_a_matching_chain_and_none_when_absent():
    tree = make_tree([-1, 0, 1, 2, 3], [7, 1, 2, 3, 4])
    t = np.array([1, 2, 3, 4, 9], np.int32)
    assert O.accept(tree, t) == (4, [0, 1, 2, 3, 4], 9)
    t = np.array([5, 2, 3, 4, 9], np.int32)
    assert O.accept(tree, t) == (0, [0], 5)


def test_target_argmax_lowest_index_on_ties():
    y = np.zeros((4, 9), np.float32)
    y[0, 3] = y[0, 5] = 2.0
    y[1, 8] = 1.0
    y[2, :] = -np.inf
    y[2, 4] = -5.0
    t = O.target_argmax(y, 3)
    assert list(t) == [3, 8, 4, -1]


def test_synthetic_target_accepts_confident_spikes():
    """With the synthetic generator a confident draft row's spike is also the target's choice."""
    cfg = synth.CONFIGS["tiny"].scaled(vocab=4096, spike="all8")
    p = O.Params(cfg.budget, cfg.topk, cfg.topk, cfg.mu, cfg.max_depth)
    tree = O.expand(3, lambda path: synth.draft_logits_row(cfg, 1, 0, path), p)
    y = np.stack([synth.target_logits_row(cfg, 1, 0, O.path_tokens(tree, i)) for i in range(tree.n_nodes)])
    alen, path, bonus = O.accept(tree, O.target_argmax(y, tree.n_nodes))
    assert alen == tree.depth[: tree.n_nodes].max()
