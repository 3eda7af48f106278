"""The allocation-free argmax entry point against the ordinary verification call.

Some callers of this library may not allocate device memory at the point where they verify a
draft tree: they live inside a fixed memory pool, or in a stretch of a serving loop where a
cudaMalloc (which synchronises the device and can fail under memory pressure) is ruled out.
``talon_target_argmax_noalloc`` serves them with a scratch array that is part of the library
image.  This test calls it through the C ABI twice in a row, because the array keeps the previous
call's contents, and compares both results with the target tokens that ``talon_accept`` reports.
The comparison is exact: these are token ids."""
import pytest
import torch

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


def test_noalloc_rejects_sizes_beyond_its_scratch():
    from paper_2601_07353_b200 import talon
    x = torch.zeros(4, 64, device="cuda")
    out = torch.zeros(4, dtype=torch.int32, device="cuda")
    big = x.expand(4, 64)          # only the row count matters for the check
    with pytest.raises(talon.TalonError) as e:
        talon._check(talon._lib.talon_target_argmax_noalloc(talon._ptr(big), 64, 64, talon.NOALLOC_MAX_ROWS + 1,
                                                            talon._ptr(out), None), "noalloc")
    assert e.value.code == talon.ERR_CAPACITY
