"""The algorithmic-work model that the benchmark's roofline figures use (host logic only)."""
from paper_2601_07353_b200 import roofline, synth


def test_expanded_rows_counts_frontiers_that_still_have_budget():
    # budget 7: layers of 1, 2, 2, 2 nodes -> frontiers of layers 0..2 are expanded (1 + 2 + 2 rows)
    assert roofline.expanded_rows([0, 1, 3, 5, 7, 7, 7], 7, 6) == 5
    # depth stop: only the layers that were enqueued count
    assert roofline.expanded_rows([0, 1, 3, 5, 7, 7, 7], 7, 2) == 3
    # a tree that stays below its budget expands its last frontier too, then meets an empty layer
    assert roofline.expanded_rows([0, 1, 2, 3, 3, 3], 10, 5) == 3


def test_bytes_match_the_stated_per_unit_figures():
    cfg = synth.CONFIGS["llama8b"]
    assert roofline.expand_bytes(3, cfg.vocab) == 3 * 4 * cfg.vocab
    assert roofline.argmax_bytes(60, cfg.vocab) == 60 * 4 * cfg.vocab
    b = roofline.attention_bytes(2048, 60, 32, 8, 128, 60)
    assert b == 2 * 2 * 128 * 8 * (2048 + 60) + 2 * 2 * 60 * 32 * 128 + 8 * 1 * 60
    f = roofline.attention_flops(2048, 60, 32, 128)
    assert f == 4 * 128 * 32 * 60 * 2108
    # arithmetic intensity is g * N flop per KV byte up to the Q/O and mask terms
    assert abs(f / (2 * 2 * 128 * 8 * 2108) - 4 * 60) < 1e-9


def test_peaks_fall_back_when_the_file_is_missing(tmp_path):
    p = roofline.load_peaks(str(tmp_path))
    assert p["source"] == "fallback" and p["hbm_gbs"] == roofline.FALLBACK_HBM_GBS
    (tmp_path / "MEASURED_PEAKS.json").write_text('{"hbm_gbs": 6000.0, "bf16_tflops": 1500.0}')
    p = roofline.load_peaks(str(tmp_path))
    assert p["source"] == "measured" and p["hbm_gbs"] == 6000.0 and p["bf16_tflops_sustained"] == 1500.0


def test_traffic_ratio_is_void_once_the_kernel_source_changed(tmp_path):
    import json
    (tmp_path / "profiles").mkdir()
    (tmp_path / "csrc").mkdir()
    (tmp_path / "csrc" / "k.cu").write_text("__global__ void k() {}\n")
    rec = {"expand_rows": {"sources": ["csrc/k.cu"], "sha256": roofline.source_hash(str(tmp_path), ["csrc/k.cu"]),
                           "dram_bytes_per_algorithmic_byte": {"llama8b": 1.05}}}
    (tmp_path / "profiles" / "traffic_capture.json").write_text(json.dumps(rec))
    assert roofline.captured_traffic_ratio(str(tmp_path), "expand_rows", "llama8b") == 1.05
    assert roofline.captured_traffic_ratio(str(tmp_path), "expand_rows", "longctx") is None      # no capture on that workload
    assert roofline.captured_traffic_ratio(str(tmp_path), "no_such_kernel", "llama8b") is None
    with open(tmp_path / "csrc" / "k.cu", "a") as f:
        f.write("// changed\n")
    assert roofline.captured_traffic_ratio(str(tmp_path), "expand_rows", "llama8b") is None


def test_the_committed_traffic_record_names_existing_sources():
    import json, os
    root = os.path.dirname(os.path.dirname(os.path.abspath(roofline.__file__)))
    rec = json.load(open(os.path.join(root, "profiles", "traffic_capture.json")))
    for kernel, r in rec.items():
        assert len(r["sha256"]) == 64 and all(os.path.exists(os.path.join(root, s)) for s in r["sources"]), kernel
