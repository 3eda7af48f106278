"""Algorithmic work of each kernel of the path, for roofline accounting.

"Algorithmic" means what the method itself has to move or compute, whatever the kernels do:
one read of each expanded logit row, one read of each target-logit row, one read of the
prefix and tree K/V per kv head plus Q in and O out.  Scratch traffic (split-KV partials,
per-chunk top-k lists) is deliberately not counted, so it shows up as lost bandwidth.
"""
from __future__ import annotations

import hashlib
import json
import os
from typing import Dict, Sequence

FALLBACK_HBM_GBS = 6650.0          # earlier copy measurement on the same kind of GPU
FALLBACK_BF16_TFLOPS = 1590.0


def load_peaks(root: str) -> Dict[str, object]:
    """Measured copy bandwidth and bf16 matmul rate of this machine's GPUs, else the fallback."""
    path = os.path.join(root, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            j = json.load(f)
        return dict(hbm_gbs=float(j["hbm_gbs"]), bf16_tflops=float(j["bf16_tflops"]),
                    bf16_tflops_sustained=float(j.get("bf16_tflops_sustained", j["bf16_tflops"])),
                    source="measured")
    except (OSError, KeyError, ValueError):
        return dict(hbm_gbs=FALLBACK_HBM_GBS, bf16_tflops=FALLBACK_BF16_TFLOPS,
                    bf16_tflops_sustained=FALLBACK_BF16_TFLOPS, source="fallback")


def expanded_rows(layer_off: Sequence[int], budget: int, layers_enqueued: int) -> int:
    """Logit rows one sequence reads in a step: the frontier of every layer that starts with
    budget left (a full tree or an empty frontier reads nothing)."""
    rows = 0
    for d in range(layers_enqueued):
        lo, hi = int(layer_off[d]), int(layer_off[d + 1])     # nodes of depth d; hi = |T| before the layer
        if hi <= lo or hi >= budget:
            break
        rows += hi - lo
    return rows


def expand_bytes(rows: int, vocab: int) -> int:
    return 4 * vocab * rows


def argmax_bytes(n_nodes: int, vocab: int) -> int:
    return 4 * vocab * n_nodes


def attention_bytes(prefix_len: int, n_nodes: int, n_q_heads: int, n_kv_heads: int, head_dim: int,
                    budget: int) -> int:
    words = (budget + 63) // 64
    kv = 2 * 2 * head_dim * n_kv_heads * (prefix_len + n_nodes)
    qo = 2 * 2 * n_nodes * n_q_heads * head_dim
    return kv + qo + 8 * words * n_nodes


def attention_flops(prefix_len: int, n_nodes: int, n_q_heads: int, head_dim: int) -> int:
    return 4 * head_dim * n_q_heads * n_nodes * (prefix_len + n_nodes)


def source_hash(root: str, sources: Sequence[str]) -> str:
    h = hashlib.sha256()
    for rel in sources:
        with open(os.path.join(root, rel), "rb") as src:
            h.update(src.read())
    return h.hexdigest()


def captured_traffic_ratio(root: str, kernel: str, workload: str):
    """DRAM bytes per algorithmic byte of ``kernel`` on ``workload`` from its last ncu capture, or None.

    ``profiles/traffic_capture.json`` under ``root`` records, per kernel, the ratios measured under
    ncu (one per workload) together with a hash of the kernel's source files at that time; a kernel
    whose source changed since then has no valid counters, so None is returned and the benchmark
    reports ``traffic`` as null."""
    try:
        with open(os.path.join(root, "profiles", "traffic_capture.json")) as f:
            rec = json.load(f)[kernel]
        if source_hash(root, rec["sources"]) != rec["sha256"]:
            return None
        return float(rec["dram_bytes_per_algorithmic_byte"][workload])
    except (OSError, KeyError, ValueError, TypeError):
        return None
