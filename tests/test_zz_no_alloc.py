"""The allocation-free argmax entry point against the ordinary verification call and the oracle.

Some callers of this library may not allocate device memory at the point where they verify a
draft tree: they live inside a fixed memory pool, or in a stretch of a serving loop where a
cudaMalloc (which synchronises the device and can fail under memory pressure) is ruled out.
``talon_target_argmax_noalloc`` serves them with a scratch array that is part of the library
image.  These tests call it through the C ABI twice in a row, because the array keeps the previous
call's contents, and compare both results with the target tokens that ``talon_accept`` reports and
with the oracle's argmax.  The comparison is exact: these are token ids."""
import numpy as np
import pytest
import torch

from oracle import talon_oracle as O
from paper_2601_07353_b200 import synth

pytestmark = pytest.mark.gpu


def test_noalloc_argmax_matches_accept_twice_in_a_row():
    from paper_2601_07353_b200 import talon, workload
    cfg = synth.CONFIGS["tiny"].scaled(vocab=40000, batch=3, prefix_min=16, prefix_max=48)
    t = workload.make_talon(cfg)
    wl = workload.build_workload(cfg, t, seed=99)
    wl.target[1, 0, 123] = 50.0                    # two equal maxima: the lower id wins
    wl.target[1, 0, 30123] = 50.0
    workload.run_step(t, wl)
    assert t.poll_status() == talon.OK
    want = wl.target_tok.clone()                   # from talon_accept; -1 in unused node slots
    n_nodes = wl.tree.n_nodes.cpu().tolist()
    rows = wl.target.view(-1, cfg.vocab)
    for call in range(2):
        got = torch.full((rows.shape[0],), -7, dtype=torch.int32, device=rows.device)
        talon.target_argmax_noalloc(rows, got)
        torch.cuda.synchronize()
        got = got.view(cfg.batch, cfg.budget)
        for b in range(cfg.batch):
            n = n_nodes[b]
            assert torch.equal(got[b, :n], want[b, :n]), f"call {call}, sequence {b}"
            oracle_tok = O.target_argmax(wl.target[b].cpu().numpy(), n)
            assert (got[b, :n].cpu().numpy() == oracle_tok[:n]).all(), f"call {call}, sequence {b} vs the oracle"
        assert got[1, 0].item() == 123
        # a different input on the second call: stale keys of the first call must not leak
        if call == 0:
            rows = rows.clone()
            rows[:, :] -= 1000.0                  # every key of this call is smaller than the first call's
            rows[:, 7] = -900.0
            shifted = torch.empty(rows.shape[0], dtype=torch.int32, device=rows.device)
            talon.target_argmax_noalloc(rows, shifted)
            torch.cuda.synchronize()
            assert (shifted == 7).all()
            rows = wl.target.view(-1, cfg.vocab)
    t.close()


@pytest.mark.parametrize("n_rows", [6, 2000])      # few rows: a row is cut into chunks; many rows: one chunk per row
def test_noalloc_argmax_nan_and_minus_inf_rows(n_rows):
    """A NaN never competes, wherever it sits; a row of NaN only gives -1; a row of -inf only gives
    token 0.  Rows without NaN must equal the oracle's argmax."""
    from paper_2601_07353_b200 import talon
    V = 5000
    g = torch.Generator(device="cuda").manual_seed(5)
    x = torch.randn(n_rows, V, device="cuda", generator=g)
    nan, ninf = float("nan"), float("-inf")
    x[0, :] = nan                                   # nothing but NaN
    x[1, 0] = nan                                   # NaN at index 0, a finite maximum elsewhere
    x[2, 5] = nan                                   # NaN at index 5
    x[3, :] = ninf                                  # -inf only
    x[4, :] = ninf; x[4, 0] = nan; x[4, 4097] = nan  # -inf and NaN only: the lowest non-NaN index
    x[5, 1234] = 9.0; x[5, 4321] = 9.0              # equal maxima, NaN in between
    x[5, 3000] = nan
    h = x.cpu().numpy()
    want = np.full(n_rows, -1, np.int32)
    for i in range(n_rows):
        ok = ~np.isnan(h[i])
        if not ok.any():
            continue
        if ok.all():
            want[i] = O.target_argmax(h[i:i + 1], 1)[0]
        else:                                       # the stated rule: the oracle's argmax over what is not NaN
            idx = np.nonzero(ok)[0]
            want[i] = idx[O.target_argmax(h[i:i + 1, idx], 1)[0]]
    assert want[0] == -1 and want[3] == 0 and want[4] == 1 and want[5] == 1234
    for call in range(2):
        got = torch.full((n_rows,), -7, dtype=torch.int32, device="cuda")
        talon.target_argmax_noalloc(x, got)
        torch.cuda.synchronize()
        assert (got.cpu().numpy() == want).all(), f"call {call}"


def test_noalloc_rejects_sizes_beyond_its_scratch():
    from paper_2601_07353_b200 import talon
    x = torch.zeros(4, 64, device="cuda")
    out = torch.zeros(4, dtype=torch.int32, device="cuda")
    big = x.expand(4, 64)          # only the row count matters for the check
    with pytest.raises(talon.TalonError) as e:
        talon._check(talon._lib.talon_target_argmax_noalloc(talon._ptr(big), 64, 64, talon.NOALLOC_MAX_ROWS + 1,
                                                            talon._ptr(out), None), "noalloc")
    assert e.value.code == talon.ERR_CAPACITY
