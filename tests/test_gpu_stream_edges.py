"""Adversarial logit rows for the streaming expansion kernel, at vocabularies that span many tiles
per warp: rows whose elements all tie, rows sorted either way, plateaus of equal maxima, steps.
They drive the paths that ordinary rows rarely reach (a candidate buffer that overflows inside a
tile, cut-backs, a CTA pool that cannot hold every survivor, a row merge with more keys at the
bound than its fast path holds), with a row cut into one chunk and into many.  Every node has the
same row, so scores tie across parents as well and the tie rule decides the whole tree."""
import numpy as np
import pytest
import torch

from oracle import talon_oracle as O
from tests import parity_util as PU

pytestmark = pytest.mark.gpu

V = 50_001                      # not a multiple of 4: the last tile is ragged


def _row(kind: str) -> np.ndarray:
    i = np.arange(V, dtype=np.float64)
    if kind == "all_equal":
        z = np.zeros(V)
    elif kind == "ascending":
        z = i * 1e-3
    elif kind == "descending":
        z = -i * 1e-3
    elif kind == "plateau":      # 700 equal maxima scattered over the row, the rest lower
        z = -1.0 - (i % 97) * 1e-2
        z[(np.arange(700) * 71) % V] = 3.0
    elif kind == "steps":        # long runs of equal values, the best run last
        z = np.floor(i / 6000.0)
    elif kind == "two_values":   # half the row ties for the maximum
        z = (i % 2).astype(np.float64)
    else:
        raise ValueError(kind)
    return z.astype(np.float32)


# (batch, K): few rows per layer (a row is cut into chunks of its own), 320 rows per layer (every CTA
# takes an equal share of the line of rows and crosses row boundaries), frontiers wider than eight
# rows (rows are merged wherever their last chunk finishes)
SHAPES = [(2, 8), (40, 8), (3, 12)]


@pytest.mark.parametrize("max_split", [1, 15])
@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("kind", ["all_equal", "ascending", "descending", "plateau", "steps", "two_values"])
def test_adversarial_rows(kind, shape, max_split, monkeypatch):
    from paper_2601_07353_b200 import talon
    monkeypatch.setenv("TALON_EXPAND_MAX_SPLIT", str(max_split))      # read when the context is made
    B, K = shape
    N, D = 3 * K, 6
    t = talon.Talon(batch_max=B, vocab=V, budget=N, root_topk=K, cand_topk=K, max_depth=D, n_q_heads=4, n_kv_heads=2,
                    mu=0.03)
    tree = t.alloc_tree(B)
    row = _row(kind)
    logits = torch.from_numpy(row).cuda().expand(B, N, V).contiguous()
    # rows must be 16-byte aligned: pad the stride to a multiple of 4 with NaN, which must never be read as data
    stride = (V + 3) // 4 * 4
    padded = torch.full((B, N, stride), float("nan"), device="cuda")
    padded[:, :, :V] = logits
    root = torch.zeros(B, dtype=torch.int32, device="cuda")
    plen = torch.zeros(B, dtype=torch.int32, device="cuda")
    t.reset(tree, root, plen)
    for _ in range(D):
        t.expand_layer(tree, padded[:, :, :V])
    t.build_tree(tree)
    torch.cuda.synchronize()
    assert t.poll_status() == talon.OK
    # Every candidate of a layer has the same score in exact arithmetic.  When all rows are cut the
    # same way their fp32 partial sums agree bit for bit and the tie rule (lower parent first) is
    # visible in the result; when the CTAs take equal shares of the whole line, rows are cut at
    # different offsets, their normalisers differ in the last bits and which of the tied parents
    # wins is a choice inside the 1e-5 tie tolerance: the oracle then follows the GPU's choice.
    params = O.Params(N, K, K, 0.03, D)
    rows_differ_in_cut = B * K > 222
    for b in range(B):
        n = int(tree.n_nodes[b])
        tok, par = tree.token[b].cpu().numpy(), tree.parent[b].cpu().numpy()
        ref, tolerated = PU.follow_tree(None, params, 0, lambda path: row, tok, par, n, tree.layer_off[b].cpu().numpy(),
                                        f"{kind} seq {b}")
        if not rows_differ_in_cut:
            assert tolerated == 0, kind
        assert (tok[:n] == np.asarray(ref.token[:n])).all() and (par[:n] == np.asarray(ref.parent[:n])).all(), kind
        assert (tree.depth[b, :n].cpu().numpy() == np.asarray(ref.depth[:n])).all(), kind
        assert np.abs(tree.score[b, :n].cpu().numpy() - np.asarray(ref.score[:n])).max() <= 2e-5, kind
    t.close()
