"""Pins for the oracle's sampling verification (Appendix B steps 1-3).

The appendix fixes the property, not the procedure: what is emitted must be distributed exactly as
the target model's own samples.  The tests below hold the oracle to that property (exactly, on
dyadic tables where a midpoint grid over the uniforms integrates without error; statistically, on
random tables), to the greedy walk in the limit of a one-hot posterior, and to a library softmax.
"""
import itertools
import math

import numpy as np
import pytest
import scipy.special

from oracle import talon_oracle as O
from tests.test_oracle_verify import make_tree


def logits_of(p):
    with np.errstate(divide="ignore"):
        return np.log(np.asarray(p, dtype=np.float64)).astype(np.float32)


def emitted(tree, rows, u_accept, u_sample, temperature=1.0):
    alen, path, tok = O.accept_stochastic(tree, rows, u_accept, u_sample, temperature)
    assert alen == len(path) - 1 and path[0] == 0
    for a, b in zip(path, path[1:]):
        assert tree.parent[b] == a
    return tuple(int(tree.token[c]) for c in path[1:]) + (tok,)


def target_law(tree, P):
    """Law of the emitted sequence if the tokens were drawn from the target itself, one after the
    other, and emission stopped at the first drawn token that no child of the current node
    carries: probabilities multiply along the tree."""
    law = {}

    def rec(node, prefix, pr):
        kids = {int(tree.token[c]): c for c in O.children_of(tree, node)}
        for w, pw in enumerate(P[node]):
            if pw == 0.0:
                continue
            if w in kids:
                rec(kids[w], prefix + (w,), pr * pw)
            else:
                law[prefix + (w,)] = law.get(prefix + (w,), 0.0) + pr * pw

    rec(0, (), 1.0)
    return law


DYADIC_TREE = dict(parents=[-1, 0, 0, 1], tokens=[3, 0, 1, 2])
DYADIC_P = np.array([
    [1 / 2, 1 / 4, 1 / 8, 1 / 8],      # after the root: children carry tokens 0 and 1
    [1 / 4, 1 / 4, 1 / 2, 0.0],        # after node 1 (token 0): its child carries token 2
    [1 / 8, 1 / 8, 1 / 4, 1 / 2],      # after node 2 (token 1): a leaf
    [1 / 2, 1 / 2, 0.0, 0.0],          # after node 3 (token 2): a leaf
])


def test_emitted_sequences_follow_the_target_exactly_on_dyadic_tables():
    """Every acceptance threshold and every CDF step of this example is a multiple of 1/8, so the
    midpoints of an 8-cell grid per uniform integrate the procedure exactly: the frequency of each
    emitted sequence must equal the product of target probabilities along it."""
    tree = make_tree(**DYADIC_TREE)
    rows = logits_of(DYADIC_P)
    G = 8
    mid = (np.arange(G) + 0.5) / G
    freq = {}
    for u1, u2, u3, us in itertools.product(mid, repeat=4):
        seq = emitted(tree, rows, np.array([0.0, u1, u2, u3]), us)
        freq[seq] = freq.get(seq, 0.0) + 1.0 / G ** 4
    law = target_law(tree, DYADIC_P)
    assert set(freq) == set(law)
    for seq, pr in law.items():
        assert abs(freq[seq] - pr) < 1e-12, (seq, freq[seq], pr)
    assert abs(sum(law.values()) - 1.0) < 1e-12
    # spot values worked by hand: accept token 0 then token 2, then a leaf sample of token 1
    assert abs(law[(0, 2, 1)] - 0.5 * 0.5 * 0.5) < 1e-15
    # both children of the root rejected, correction token 3
    assert abs(law[(3,)] - 1 / 8) < 1e-15


def test_first_emitted_token_follows_the_target_on_random_tables():
    """Monte-Carlo version of the same property on a table that is not dyadic (seeded)."""
    V = 7
    rng = np.random.default_rng(11)
    tree = make_tree(parents=[-1, 0, 0, 0, 1, 1, 2], tokens=[5, 1, 4, 6, 0, 3, 2])
    rows = (1.5 * rng.standard_normal((7, V))).astype(np.float32)
    P = np.stack([O.target_posterior(r) for r in rows])
    law = target_law(tree, P)
    n = 40000
    cnt = {}
    U = rng.random((n, 8))
    for i in range(n):
        seq = emitted(tree, rows, U[i, :7], U[i, 7])
        cnt[seq] = cnt.get(seq, 0) + 1
    assert set(cnt) <= set(law)
    chi2 = sum((cnt.get(s, 0) - n * pr) ** 2 / (n * pr) for s, pr in law.items() if n * pr >= 5)
    dof = sum(1 for pr in law.values() if n * pr >= 5) - 1
    assert chi2 < dof + 5 * math.sqrt(2 * dof), (chi2, dof)


def test_one_hot_posterior_reduces_to_the_greedy_walk():
    rng = np.random.default_rng(3)
    V = 50
    tree = make_tree(parents=[-1, 0, 0, 1, 1, 3], tokens=[9, 4, 7, 2, 8, 5])
    rows = rng.standard_normal((6, V)).astype(np.float32)
    for node, tok in [(0, 4), (1, 2), (3, 5), (5, 11), (2, 1), (4, 0)]:
        rows[node, tok] += 80.0
    t = O.target_argmax(rows, 6)
    want = O.accept(tree, t)
    for trial in range(20):
        u = 0.001 + 0.998 * rng.random(7)
        got = O.accept_stochastic(tree, rows, u[:6], u[6])
        assert got == want
    assert want[0] == 3 and want[1] == [0, 1, 3, 5] and want[2] == 11


def test_correction_token_is_never_a_rejected_child():
    rng = np.random.default_rng(5)
    V = 12
    tree = make_tree(parents=[-1, 0, 0, 0], tokens=[0, 3, 6, 9])
    rows = rng.standard_normal((4, V)).astype(np.float32)
    for _ in range(300):
        u = rng.random(5)
        u[1:4] = 0.999999        # (almost) certainly reject all three children
        alen, path, tok = O.accept_stochastic(tree, rows, u[:4], u[4])
        if alen == 0:
            assert tok not in (3, 6, 9)


def test_zero_uniform_accepts_the_first_child_with_mass_and_masked_tokens_never_win():
    tree = make_tree(parents=[-1, 0, 0], tokens=[0, 1, 2])
    rows = logits_of([[0.0, 0.0, 0.25, 0.75], [0.5, 0.5, 0.0, 0.0], [0.0, 1.0, 0.0, 0.0]])
    alen, path, tok = O.accept_stochastic(tree, rows, np.zeros(3), 0.0)
    assert path == [0, 2] and tok == 1          # child with token 1 has no mass; token 2 is taken at u = 0
    alen, path, tok = O.accept_stochastic(tree, rows, np.array([0.0, 0.9, 0.9]), 0.999999)
    assert path == [0] and tok == 3             # token 2 rejected and struck; only token 3 is left


def test_posterior_is_the_library_softmax_at_any_temperature():
    rng = np.random.default_rng(9)
    z = (3 * rng.standard_normal(1000)).astype(np.float32)
    z[17] = -np.inf
    for T in (1.0, 0.7, 2.5):
        want = scipy.special.softmax(z.astype(np.float64) / T)
        assert np.abs(O.target_posterior(z, T) - want).max() < 1e-15
    with pytest.raises(O.NonFiniteLogits):
        O.target_posterior(np.array([0.0, np.nan], np.float32))
    with pytest.raises(O.NonFiniteLogits):
        O.target_posterior(np.array([-np.inf, -np.inf], np.float32))


def test_planted_mistakes_break_the_exact_pin():
    """The exact pin notices the plausible slips: forgetting to renormalise by the unclaimed mass,
    and drawing the correction token from the full posterior instead of the struck one."""
    tree = make_tree(**DYADIC_TREE)
    rows = logits_of(DYADIC_P)
    law = target_law(tree, DYADIC_P)
    mid = (np.arange(8) + 0.5) / 8

    def wrong_no_renorm(u, us):
        p = DYADIC_P[0].copy()
        for c in (1, 2):
            w = int(tree.token[c])
            if u[c] < p[w]:                      # should be u * mass < p[w]
                return (w,)
            p[w] = 0.0
        cdf = np.cumsum(p)
        return (int(np.searchsorted(cdf, us * cdf[-1], side="right")),)

    def wrong_full_posterior(u, us):
        p = DYADIC_P[0].copy()
        mass = 1.0
        for c in (1, 2):
            w = int(tree.token[c])
            if u[c] * mass < p[w]:
                return (w,)
            mass -= p[w]
        cdf = np.cumsum(p)                        # rejected tokens not struck
        return (int(np.searchsorted(cdf, us * cdf[-1], side="right")),)

    first = {}
    for s, pr in law.items():
        first[s[0]] = first.get(s[0], 0.0) + pr
    for wrong in (wrong_no_renorm, wrong_full_posterior):
        freq = {}
        for u1, u2, us in itertools.product(mid, repeat=3):
            w = wrong(np.array([0.0, u1, u2]), us)[0]
            freq[w] = freq.get(w, 0.0) + 1.0 / 8 ** 3
        assert max(abs(freq.get(w, 0.0) - first[w]) for w in first) > 1e-3
