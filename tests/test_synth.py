"""The seeded input generator: deterministic, backend-independent, and shaped as documented."""
import numpy as np
import torch

from paper_2601_07353_b200 import synth


def test_gaussian_is_bit_identical_between_numpy_and_torch():
    key = synth.row_key(5, synth.STREAM_DRAFT, 3, synth.fold_path([1, 2, 3]))
    a = synth.gaussian(key, 5000)
    b = synth.gaussian(key, 5000, device="cpu").numpy()
    assert a.dtype == np.float32 and (a.view(np.int32) == b.view(np.int32)).all()
    c = synth.gaussian(key, 100, start=400)
    assert (c == a[400:500]).all()


def test_gaussian_moments():
    g = synth.gaussian(12345, 400000).astype(np.float64)
    assert abs(g.mean()) < 0.01 and abs(g.var() - 1.0) < 0.01
    assert 4.0 < g.max() < 6.0 and (np.abs(g) > 3).mean() < 0.004


def test_bf16_rounding_matches_torch():
    x = synth.gaussian(99, 20000)
    want = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert (synth.round_to_bf16(x) == want).all()
    assert (synth.round_to_bf16(torch.from_numpy(x)).numpy() == want).all()


def test_rows_depend_on_seed_sequence_and_path_only():
    cfg = synth.CONFIGS["tiny"].scaled(vocab=1000)
    a = synth.draft_logits_row(cfg, 1, 0, [5, 6])
    assert (a == synth.draft_logits_row(cfg, 1, 0, [5, 6])).all()
    for other in (synth.draft_logits_row(cfg, 2, 0, [5, 6]), synth.draft_logits_row(cfg, 1, 1, [5, 6]),
                  synth.draft_logits_row(cfg, 1, 0, [6, 5])):
        assert (a != other).mean() > 0.9
    t = synth.draft_logits_row(cfg, 1, 0, [5, 6], device="cpu").numpy()
    assert (t.view(np.int32) == a.view(np.int32)).all()
    y = synth.target_logits_row(cfg, 1, 0, [5, 6])
    yt = synth.target_logits_row(cfg, 1, 0, [5, 6], device="cpu").numpy()
    assert (y.view(np.int32) == yt.view(np.int32)).all()


def test_spike_mix_and_prefix_lengths():
    cfg = synth.CONFIGS["llama8b"]
    hs = [synth.spike_height(cfg, 1, 0, synth.fold_path([i])) for i in range(4000)]
    assert abs(np.mean(np.array(hs) == 8.0) - 0.5) < 0.04
    cfgb = synth.CONFIGS["llama8b_batched"]
    ls = [synth.prefix_len(cfgb, 1, b) for b in range(500)]
    assert min(ls) >= 1024 and max(ls) <= 4096 and max(ls) - min(ls) > 2500
    lo = np.mean([synth.spike_height(cfgb, 1, 0, synth.fold_path([i])) == 8.0 for i in range(2000)])
    hi = np.mean([synth.spike_height(cfgb, 1, 15, synth.fold_path([i])) == 8.0 for i in range(2000)])
    assert lo < 0.1 and hi > 0.9
    ex = [synth.spike_height(synth.CONFIGS["longctx"], 1, 0, synth.fold_path([i])) for i in range(4000)]
    assert abs(np.mean(ex) - 4.0) < 0.3


def test_zipf_row_is_a_permuted_power_law():
    z = synth.zipf_logits_row(1000, 1.35, 1, 0).astype(np.float64)
    want = -1.35 * np.log(np.arange(1, 1001))
    assert np.allclose(np.sort(z)[::-1], want, atol=1e-5)
