"""CPU oracle for the Talon hot path -- TEST INFRASTRUCTURE, not a product path.

A plain, slow, fp64 NumPy statement of what the paper's method computes, written from the
paper and used only by the tests, by ``__graft_entry__.smoke()`` and by the benchmark's
CPU-baseline leg.  It shares no code with the CUDA path and imports nothing from it.

What follows which passage:

* ``expand_layer`` / ``expand``  -- Algorithm 2 (adaptive tree construction), with the
  candidate pool and path probability of Eq. 3, the confidence gate of Eq. 4, the budget
  truncation stated after Eq. 4, and the Top-K root initialisation of Eq. 5.  Path scores
  are Eq. 2's products, kept as log-probabilities (a monotone re-expression: products
  become sums and ``p >= mu*m`` becomes ``log p >= log mu + log m``).
* ``finalize``                   -- positions and the ancestor ("tree attention") mask of
  Fig. 2(b) / Appendix B: a node sees itself and its root-to-leaf predecessors.
* ``tree_attention``             -- Appendix B: every tree token attends to the whole
  prefix and to its predecessors on its own path, softmax(QK^T/sqrt(d))V written out.
* ``target_argmax`` / ``accept`` -- Appendix B steps (1)-(2) at temperature 0: the longest
  root-to-leaf prefix whose tokens equal the target's greedy choices, plus the target's
  token at the point of divergence.
* ``accept_stochastic``          -- Appendix B steps (1)-(3) under sampling (the paper's
  temperature-1 setting): the target's posterior at each visited node, the children of
  that node tried one after the other as proposals, and on rejection of all of them a
  correction token drawn from what is left of the posterior.  The appendix names the three
  steps and the property they must have (the emitted tokens are distributed exactly as the
  target model's) and leaves the procedure to the tree-verification literature it cites; the
  procedure written here is the recursive rejection scheme of that literature for proposals
  that are fixed rather than sampled, and the property is what pins it.
* ``commit`` / ``draft_efficiency`` / ``speedup`` -- the bookkeeping either side of one
  draft-and-verify step in the generation loop of Section 5.3: the accepted tokens' keys and
  values join the prefix cache, the correction token becomes the next root, and the counts
  N_p (verification passes), N_q (draft passes) and L (tokens produced) feed the draft
  efficiency delta = N_q / N_p, the mean accepted tokens tau = L / N_p and the speed-up
  R = tau / (1 + c delta) of Section 5.3 and its derivation in the appendix.

* ``expand_static`` / ``prune_static`` -- Algorithm 1 (the static tree the paper compares with): at
  every depth 0..D each parent proposes its Top-K tokens, the K x K pool is cut to the K best path
  probabilities, which join the tree and become the next parents; at the end the tree is pruned to
  the N best path probabilities.
Readings taken where the paper is silent (all listed in the design notes): the budget N
counts the root; ``max_depth`` is an extra stop; a per-parent candidate cap ``cand_topk``
(== vocabulary size gives the paper's full pool); ties go to the lower parent index, then
the lower token id; nodes are stored layer by layer, each layer sorted by (parent, token).

Parity pins live in ``tests/test_oracle_*.py``: brute-force enumeration in probability
space, a hand-worked example, closed forms, structural invariants, causal attention.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Callable, List, Optional, Sequence

import numpy as np


class NonFiniteLogits(ValueError):
    """A logit row holds NaN or +inf, or nothing but -inf (its softmax is undefined)."""


@dataclass
class Params:
    budget: int                 # N: maximum number of tree nodes, root included
    root_topk: int              # K: width of the Top-K initialisation (Eq. 5)
    cand_topk: int              # per-parent candidate cap k; >= vocabulary size = Eq. 3's full pool
    mu: float = 0.03            # gate threshold of Eq. 4
    max_depth: int = 1 << 30    # extra stop: no node deeper than this
    init_layers: int = 1        # how many leading layers use Top-K instead of the gate


@dataclass
class Tree:
    budget: int
    max_depth: int
    n_nodes: int = 1
    layers_run: int = 0
    token: np.ndarray = None
    parent: np.ndarray = None
    depth: np.ndarray = None
    score: np.ndarray = None            # log of Eq. 2's path probability
    mask: np.ndarray = None             # [N, W] uint64, bit j of row i: node i sees node j
    layer_off: List[int] = field(default_factory=list)

    @property
    def frontier(self) -> range:
        d = self.layers_run
        return range(self.layer_off[d], self.layer_off[d + 1])


def new_tree(root_token: int, budget: int, max_depth: int) -> Tree:
    """Algorithm 2, initialisation: T = {x_t}, P_0 = {x_t}, p(x_t) = 1."""
    n = budget
    w = (n + 63) // 64
    t = Tree(budget=budget, max_depth=max_depth)
    t.token = np.full(n, -1, np.int32)
    t.parent = np.full(n, -1, np.int32)
    t.depth = np.full(n, -1, np.int32)
    t.score = np.full(n, -np.inf, np.float64)
    t.mask = np.zeros((n, w), np.uint64)
    t.token[0] = root_token
    t.depth[0] = 0
    t.score[0] = 0.0
    t.mask[0, 0] = np.uint64(1)
    t.layer_off = [0, 1]
    return t


def log_softmax_norm(z32: np.ndarray) -> float:
    """log sum_w exp(z_w) of one fp32 logit row, in fp64 (the softmax normaliser)."""
    z = np.asarray(z32, dtype=np.float64)
    if np.isnan(z).any() or np.isposinf(z).any():
        raise NonFiniteLogits("NaN or +inf logit")
    m = float(z.max())
    if m == -np.inf:
        raise NonFiniteLogits("row is all -inf")
    return m + math.log(float(np.exp(z - m).sum()))


def row_topk(z32: np.ndarray, k: int) -> np.ndarray:
    """Token ids of the k largest logits of a row, larger first, equal logits by lower id."""
    z = np.asarray(z32, dtype=np.float64)
    order = np.argsort(-z, kind="stable")
    return order[: min(k, z.shape[0])].astype(np.int64)


def is_active(tree: Tree) -> bool:
    """Loop condition of Algorithm 2 (|T| < N) plus the depth stop and a non-empty frontier."""
    return (tree.n_nodes < tree.budget and tree.layers_run < tree.max_depth
            and len(tree.frontier) > 0)


def layer_pool(tree: Tree, rows: Sequence[np.ndarray], p: Params):
    """Candidate pool S_d of Eq. 3 for the current frontier: (log p(u), parent v, token w)."""
    pool = []
    for v, z32 in zip(tree.frontier, rows):
        lse = log_softmax_norm(z32)
        for w in row_topk(z32, p.cand_topk):
            logp = float(np.float64(z32[w])) - lse          # log P_Md(w | x_<=v)
            if logp == -np.inf:
                continue                                     # p(u) = 0 is never a candidate
            pool.append((float(tree.score[v]) + logp, int(v), int(w)))   # p(u) = p(v) * P(w|v)
    return pool


def select_layer(pool, d: int, remaining: int, p: Params):
    """Hybrid expansion of Algorithm 2 on a pool: Top-K at the root, the gate below it,
    then the budget check.  Returns the selected (score, parent, token) triples."""
    by_rank = sorted(pool, key=lambda u: (-u[0], u[1], u[2]))
    if d < p.init_layers:
        chosen = by_rank[: p.root_topk]                      # Eq. 5
    else:
        if not by_rank:
            return []
        m_d = by_rank[0][0]                                  # anchor confidence (log)
        thr = math.log(p.mu) + m_d
        chosen = [u for u in by_rank if u[0] >= thr]         # Eq. 4, inclusive
    if len(chosen) > remaining:                              # budget check
        chosen = chosen[:remaining]
    return chosen


def expand_layer(tree: Tree, rows: Sequence[np.ndarray], p: Params) -> int:
    """One pass of Algorithm 2's while-body.  ``rows[j]`` is the fp32 draft-logit row of the
    j-th frontier node (ascending node index).  Returns the number of nodes appended."""
    if not is_active(tree):
        return 0
    d = tree.layers_run
    assert len(rows) == len(tree.frontier)
    pool = layer_pool(tree, rows, p)
    chosen = select_layer(pool, d, tree.budget - tree.n_nodes, p)
    chosen.sort(key=lambda u: (u[1], u[2]))                  # storage order inside the layer
    for s, v, w in chosen:
        i = tree.n_nodes
        tree.token[i] = w
        tree.parent[i] = v
        tree.depth[i] = tree.depth[v] + 1
        tree.score[i] = s
        tree.mask[i] = tree.mask[v]
        tree.mask[i, i // 64] |= np.uint64(1) << np.uint64(i % 64)
        tree.n_nodes += 1
    tree.layer_off.append(tree.n_nodes)
    tree.layers_run += 1
    return len(chosen)


def path_tokens(tree: Tree, node: int) -> List[int]:
    out = []
    while node >= 0:
        out.append(int(tree.token[node]))
        node = int(tree.parent[node])
    return out[::-1]


def expand(root_token: int, logits_fn: Callable[[List[int]], np.ndarray], p: Params) -> Tree:
    """Algorithm 2 in full.  ``logits_fn(path)`` returns the draft row of the node whose
    root-to-node token path is ``path`` (stands in for the draft model forward)."""
    tree = new_tree(root_token, p.budget, p.max_depth)
    while is_active(tree):
        rows = [logits_fn(path_tokens(tree, v)) for v in tree.frontier]
        expand_layer(tree, rows, p)
    return tree


def expand_static(root_token: int, logits_fn: Callable[[List[int]], np.ndarray], width: int, depth: int) -> Tree:
    """Algorithm 1 up to its pruning step: for d = 0..depth every parent v of the layer proposes
    C_v = Top-K of its next-token distribution with p(u) = p(v) * P(u | v); the pool S_d of all
    proposals is cut to its K best by p(u); those join the tree and are the parents of the next
    layer.  The tree holds 1 + K * (depth + 1) nodes (fewer if a vocabulary is smaller than K).
    Ties and storage order as everywhere in this file."""
    cap = 1 + width * (depth + 1)
    tree = new_tree(root_token, cap, depth + 1)
    parents = [0]
    for d in range(depth + 1):
        pool = []
        for v in parents:
            z32 = logits_fn(path_tokens(tree, v))
            lse = log_softmax_norm(z32)
            for w in row_topk(z32, width):                                  # C_v
                logp = float(np.float64(z32[w])) - lse
                if logp > -np.inf:
                    pool.append((float(tree.score[v]) + logp, int(v), int(w)))   # p(u) = p(v) P(u | v)
        nxt = sorted(pool, key=lambda u: (-u[0], u[1], u[2]))[:width]      # Top-K of S_d by p(u)
        nxt.sort(key=lambda u: (u[1], u[2]))
        parents = []
        for s, v, w in nxt:
            i = tree.n_nodes
            tree.token[i], tree.parent[i], tree.depth[i], tree.score[i] = w, v, tree.depth[v] + 1, s
            tree.mask[i] = tree.mask[v]
            tree.mask[i, i // 64] |= np.uint64(1) << np.uint64(i % 64)
            tree.n_nodes += 1
            parents.append(i)
        tree.layer_off.append(tree.n_nodes)
        tree.layers_run += 1
    return tree


def prune_static(tree: Tree, keep: int) -> Tree:
    """Algorithm 1's last step: T <- Top-N(T by p(u)).  Equal scores go to the lower node index, so
    a kept node's parent (whose probability is at least as large and whose index is lower) is
    kept too.  The survivors keep their relative order; parents and mask bits are renumbered."""
    n = tree.n_nodes
    order = sorted(range(n), key=lambda i: (-float(tree.score[i]), i))[:keep]
    kept = sorted(order)
    new_of = {old: new for new, old in enumerate(kept)}
    out = new_tree(int(tree.token[0]), tree.budget, tree.max_depth)
    out.n_nodes = len(kept)
    for new, old in enumerate(kept):
        out.token[new], out.depth[new], out.score[new] = tree.token[old], tree.depth[old], tree.score[old]
        out.parent[new] = -1 if tree.parent[old] < 0 else new_of[int(tree.parent[old])]
        out.mask[new] = 0
        for j in range(n):
            if (int(tree.mask[old, j // 64]) >> (j % 64)) & 1:
                out.mask[new, new_of[j] // 64] |= np.uint64(1) << np.uint64(new_of[j] % 64)
    out.layers_run = tree.layers_run
    out.layer_off = [sum(1 for i in kept if tree.depth[i] < d) for d in range(tree.layers_run + 2)]
    return out


def dense_mask(tree: Tree) -> np.ndarray:
    """[N, N] bool view of the bit mask."""
    n = tree.budget
    out = np.zeros((n, n), bool)
    for i in range(n):
        for j in range(n):
            out[i, j] = bool((int(tree.mask[i, j // 64]) >> (j % 64)) & 1)
    return out


def finalize(tree: Tree, prefix_len: int) -> dict:
    """Arrays handed to the target model: positions (prefix length + depth), parent links,
    depths, the ancestor mask; unused slots hold sentinels and see only themselves."""
    n, cap = tree.n_nodes, tree.budget
    token = tree.token.copy()
    parent = tree.parent.copy()
    depth = tree.depth.copy()
    score = tree.score.copy()
    mask = tree.mask.copy()
    position = np.full(cap, -1, np.int32)
    position[:n] = prefix_len + depth[:n]
    for i in range(n, cap):
        token[i] = parent[i] = depth[i] = -1
        score[i] = -np.inf
        mask[i] = 0
        mask[i, i // 64] = np.uint64(1) << np.uint64(i % 64)
    layer_off = list(tree.layer_off) + [n] * (tree.max_depth + 2 - len(tree.layer_off))
    return dict(n_nodes=n, token=token, parent=parent, depth=depth, position=position,
                score=score, mask=mask, layer_off=np.asarray(layer_off, np.int32),
                layers_run=tree.layers_run)


def tree_attention(q, k_prefix, v_prefix, k_tree, v_tree, tree: Tree, sm_scale: float) -> np.ndarray:
    """Tree attention of Appendix B for one sequence, direct softmax in fp64.

    q [N, Hq, Dh]; k_prefix/v_prefix [L, Hkv, Dh]; k_tree/v_tree [N, Hkv, Dh] -- values
    already rounded to bf16.  Query head h uses kv head h // (Hq/Hkv).  Node i sees every
    prefix key and the tree keys j whose mask bit (i, j) is set.  Rows of unused node
    slots are zero.  Returns [N, Hq, Dh] fp64.
    """
    q = np.asarray(q, np.float64)
    cap, hq, dh = q.shape
    hkv = k_tree.shape[1]
    g = hq // hkv
    n = tree.n_nodes
    L = k_prefix.shape[0]
    vis = np.concatenate([np.ones((n, L), bool), dense_mask(tree)[:n, :n]], axis=1)
    out = np.zeros((cap, hq, dh), np.float64)
    for h in range(hq):
        kv = h // g
        K = np.concatenate([np.asarray(k_prefix[:, kv], np.float64), np.asarray(k_tree[:n, kv], np.float64)])
        V = np.concatenate([np.asarray(v_prefix[:, kv], np.float64), np.asarray(v_tree[:n, kv], np.float64)])
        S = (q[:n, h] @ K.T) * sm_scale
        S = np.where(vis, S, -np.inf)
        P = np.exp(S - S.max(axis=1, keepdims=True))
        P /= P.sum(axis=1, keepdims=True)
        out[:n, h] = P @ V
    return out


def target_argmax(target_logits: np.ndarray, n_nodes: int) -> np.ndarray:
    """Greedy target token after each tree node (lowest id among equal maxima); -1 for unused slots."""
    y = np.asarray(target_logits)
    if np.isnan(y[:n_nodes]).any():
        raise NonFiniteLogits("NaN target logit")
    t = np.full(y.shape[0], -1, np.int32)
    t[:n_nodes] = np.argmax(y[:n_nodes], axis=1)
    return t


def accept(tree: Tree, t: np.ndarray):
    """Greedy acceptance: walk down from the root while some child carries the target's
    token.  Returns (accept_len, accepted node indices incl. root, bonus token)."""
    cur = 0
    path = [0]
    while True:
        nxt = -1
        for c in range(tree.n_nodes):
            if tree.parent[c] == cur and tree.token[c] == t[cur]:
                nxt = c
                break
        if nxt < 0:
            break
        path.append(nxt)
        cur = nxt
    return len(path) - 1, path, int(t[cur])


def children_of(tree: Tree, node: int) -> List[int]:
    """Children of ``node`` in storage order (ascending token id within a parent)."""
    return [c for c in range(tree.n_nodes) if tree.parent[c] == node]


def target_posterior(z32: np.ndarray, temperature: float = 1.0) -> np.ndarray:
    """Appendix B step (1): softmax(z / T) of one target-logit row, in fp64."""
    z = np.asarray(z32, dtype=np.float64) / float(temperature)
    if np.isnan(z).any() or np.isposinf(z).any() or not np.isfinite(z.max()):
        raise NonFiniteLogits("target row has no softmax")
    e = np.exp(z - z.max())
    return e / e.sum()


def accept_stochastic(tree: Tree, target_logits: np.ndarray, u_accept: np.ndarray, u_sample: float,
                      temperature: float = 1.0):
    """Sampling verification (Appendix B steps 1-3).

    At the current node (the root first) let p be the target's posterior there.  Its children
    are proposals that were fixed by the draft tree, not drawn, so each is a proposal
    distribution with all its mass on one token: child c with token w is accepted with
    probability p(w) / (mass still unclaimed), decided by the uniform ``u_accept[c]``; a rejected
    child's token is struck from p.  The first accepted child becomes the current node.  When
    every child of the current node is rejected (or it has none), the correction token is drawn
    from what is left of p by inverse CDF in token order with ``u_sample``.  Returns
    (accept_len, accepted node indices incl. root, correction token).

    The uniforms lie in [0, 1) and come from the caller: node c consumes ``u_accept[c]`` at most
    once (it has one parent), the sequence consumes ``u_sample`` once.
    """
    cur = 0
    path = [0]
    while True:
        p = target_posterior(target_logits[cur], temperature)
        mass = 1.0
        nxt = -1
        for c in children_of(tree, cur):
            w = int(tree.token[c])
            if float(u_accept[c]) * mass < p[w]:
                nxt = c
                break
            mass -= p[w]
            p[w] = 0.0
        if nxt < 0:
            break
        path.append(nxt)
        cur = nxt
    cdf = np.cumsum(p)
    total = cdf[-1]
    tok = int(np.searchsorted(cdf, float(u_sample) * total, side="right"))
    last = int(np.nonzero(p > 0.0)[0][-1])           # rounding at u -> 1 must not leave the support
    tok = min(tok, last)
    return len(path) - 1, path, tok


def commit(tree: Tree, accept_len: int, path: Sequence[int], next_tok: int, k_tree: np.ndarray, v_tree: np.ndarray,
           k_prefix: np.ndarray, v_prefix: np.ndarray):
    """What one finished step leaves for the next one (generation loop of Section 5.3).

    The tokens on the accepted path, root first, are now part of the sequence: their key and
    value rows (``k_tree[node]``, ``[Hkv, Dh]`` each) are appended to the prefix cache in path
    order.  The next step starts from ``next_tok``.  Returns (k_prefix', v_prefix', next root,
    counts) with counts = (verification passes, draft passes, tokens produced) of this step:
    one target pass, one draft pass per expanded layer (Algorithm 2's loop body), and the
    accepted tokens plus the correction token."""
    nodes = [int(x) for x in path[: accept_len + 1]]
    assert nodes[0] == 0 and len(nodes) == accept_len + 1
    k_new = np.concatenate([k_prefix, k_tree[nodes]], axis=0)
    v_new = np.concatenate([v_prefix, v_tree[nodes]], axis=0)
    return k_new, v_new, int(next_tok), (1, int(tree.layers_run), accept_len + 1)


def draft_efficiency(n_q: int, n_p: int) -> float:
    """delta = N_q / N_p: draft passes invested per verification pass (Section 5.3)."""
    return n_q / n_p


def mean_accepted_tokens(length: int, n_p: int) -> float:
    """tau = L / N_p: tokens produced per verification pass (Section 5.3)."""
    return length / n_p


def speedup(tau: float, delta: float, c: float) -> float:
    """R = tau / (1 + c delta), c the draft pass's cost relative to the target pass (Section 5.3)."""
    return tau / (1.0 + c * delta)
