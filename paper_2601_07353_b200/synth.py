"""Seeded synthetic inputs for the Talon hot path (draft logits, target logits, Q/K/V).

This module is the only code shared by the CPU oracle's tests and the CUDA path's
tests/benchmark.  It holds none of the method's arithmetic: it only turns
(seed, sequence id, parent-token path) into input tensors.  Everything is built from
64-bit integer hashing plus one int->float conversion and a power-of-two scale, so the
same function gives bit-identical arrays with NumPy on the host and with torch on a GPU.

Array arguments/returns are NumPy arrays unless a torch ``device`` is given, in which
case the same integer recipe runs through torch ops on that device.

Workload shapes follow the paper's setting (vocabularies of 32K/128K/152K, node budget
60, width K <= 10; Section 6 "setup" and the tree-construction micro-benchmark in the
appendix) and five benchmark configurations.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace
from typing import Optional, Sequence

import numpy as np

_M64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15
_C1 = 0xBF58476D1CE4E5B9
_C2 = 0x94D049BB133111EB
_ODD_A = 0xD6E8FEB86659FD93
_ODD_B = 0xA0761D6478BD642F

# stream ids: which tensor a hash feeds
STREAM_ROOT = 1
STREAM_DRAFT = 2
STREAM_TARGET = 3
STREAM_SPIKE = 4
STREAM_Q = 5
STREAM_K = 6
STREAM_V = 7
STREAM_KT = 8
STREAM_VT = 9
STREAM_PREFIX = 10
STREAM_ZIPF = 11
STREAM_UACCEPT = 12
STREAM_USAMPLE = 13

DEFAULT_SEED = 20260107


def _s64(c: int) -> int:
    """Two's-complement view of a 64-bit pattern as a signed Python int."""
    c &= _M64
    return c - (1 << 64) if c >= (1 << 63) else c


def mix64(x: int) -> int:
    """64-bit finaliser (splitmix64-style xor-shift-multiply) on a Python int."""
    x &= _M64
    x ^= x >> 30
    x = (x * _C1) & _M64
    x ^= x >> 27
    x = (x * _C2) & _M64
    x ^= x >> 31
    return x


def _lsr(x, s: int):
    """Logical shift right of int64 arrays (NumPy or torch)."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix64_arr(x):
    """``mix64`` on int64 arrays with wrap-around multiplication (NumPy or torch)."""
    x = x ^ _lsr(x, 30)
    x = x * _s64(_C1)
    x = x ^ _lsr(x, 27)
    x = x * _s64(_C2)
    x = x ^ _lsr(x, 31)
    return x


def fold_path(tokens: Sequence[int]) -> int:
    """Hash of the root-to-node token path (root token first)."""
    ph = 0x243F6A8885A308D3
    for t in tokens:
        ph = mix64((ph * _GOLDEN + int(t) + 1) & _M64)
    return ph


def row_key(seed: int, stream: int, seq_id: int, path_hash: int = 0) -> int:
    a = mix64((seed * _GOLDEN + stream) & _M64)
    b = mix64((seq_id * _ODD_A + path_hash) & _M64)
    return mix64(a ^ ((b * _ODD_B) & _M64))


def uniform01(key: int) -> float:
    """One uniform in (0,1) with 53 bits, from a key (host scalar)."""
    return ((mix64(key) >> 11) + 0.5) * (1.0 / (1 << 53))


def verify_uniforms(seed: int, seq_id: int, n: int, draw: int = 0):
    """The uniforms a sampling verification of one sequence consumes: one per tree node (NumPy
    fp64 array of length ``n``) and one for the correction token, all in (0, 1) with 53 bits.
    ``draw`` numbers independent repetitions."""
    ku = row_key(seed, STREAM_UACCEPT, seq_id, draw)
    u = np.array([uniform01((ku + i * _ODD_A) & _M64) for i in range(n)], dtype=np.float64)
    return u, uniform01(row_key(seed, STREAM_USAMPLE, seq_id, draw))


def _arange64(n: int, device=None, start: int = 0):
    if device is None:
        return np.arange(start, start + n, dtype=np.int64)
    import torch
    return torch.arange(start, start + n, dtype=torch.int64, device=device)


def gaussian(key: int, n: int, device=None, start: int = 0):
    """``n`` approximately N(0,1) fp32 values (elements start..start+n-1 of stream ``key``).

    Irwin-Hall: the sum of twelve 16-bit uniforms taken from three 64-bit hashes,
    centred and scaled by 2^-16.  Integer-only up to the final exact conversion, so the
    NumPy and torch results are bit-identical.  Range is +-6.
    """
    idx = _arange64(n, device, start)
    with np.errstate(over="ignore"):
        acc = None
        for j in range(3):
            h = _mix64_arr(idx * _s64(_GOLDEN) + _s64((key + j * _ODD_A) & _M64))
            part = (h & 0xFFFF) + (_lsr(h, 16) & 0xFFFF) + (_lsr(h, 32) & 0xFFFF) + _lsr(h, 48)
            acc = part if acc is None else acc + part
        acc = acc - 6 * 65535
    if device is None:
        return acc.astype(np.float32) * np.float32(1.0 / 65536.0)
    import torch
    return acc.to(torch.float32) * (1.0 / 65536.0)


def round_to_bf16(x):
    """Round fp32 values to the nearest bf16 (ties to even), returned as fp32.

    Bit arithmetic only, so NumPy and torch agree and the later fp32->bf16 cast is exact.
    """
    if isinstance(x, np.ndarray):
        bits = x.view(np.int32)
        with np.errstate(over="ignore"):
            r = (bits + 0x7FFF + ((bits >> 16) & 1)) & np.int32(-65536)
        return r.view(np.float32)
    import torch
    bits = x.view(torch.int32)
    r = (bits + 0x7FFF + ((bits >> 16) & 1)) & (-65536)
    return r.view(torch.float32)


# --------------------------------------------------------------------------------------
# Workload configurations
# --------------------------------------------------------------------------------------
@dataclass(frozen=True)
class TalonConfig:
    name: str
    batch: int
    vocab: int
    budget: int          # N, root included
    max_depth: int
    topk: int            # K: root top-k and per-parent candidate cap
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    prefix_min: int
    prefix_max: int      # inclusive; == prefix_min for a fixed prefix
    temp: float          # noise scale T of the logit generator
    spike: str           # how the per-row spike height h is drawn
    mu: float = 0.03     # the paper's default threshold

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    def scaled(self, **kw) -> "TalonConfig":
        return replace(self, **kw)


CONFIGS = {
    "tiny": TalonConfig("tiny", 1, 32000, 16, 8, 4, 32, 8, 128, 512, 512, 0.5, "uniform3"),
    "llama8b": TalonConfig("llama8b", 1, 128256, 60, 12, 8, 32, 8, 128, 2048, 2048, 0.5, "half8"),
    "llama8b_batched": TalonConfig("llama8b_batched", 16, 128256, 60, 12, 8, 32, 8, 128, 1024, 4096, 0.5, "perseq"),
    "qwen32b": TalonConfig("qwen32b", 8, 151936, 60, 16, 10, 64, 8, 128, 8192, 8192, 0.7, "p30"),
    "longctx": TalonConfig("longctx", 32, 128256, 128, 24, 8, 32, 8, 128, 32768, 32768, 0.5, "exp4"),
}
CONFIG_ORDER = ["tiny", "llama8b", "llama8b_batched", "qwen32b", "longctx"]


def spike_height(cfg: TalonConfig, seed: int, seq_id: int, path_hash: int) -> float:
    """Per-row spike height h (host scalar) according to the configuration's mix."""
    u = uniform01(row_key(seed, STREAM_SPIKE, seq_id, path_hash))
    if cfg.spike == "uniform3":
        return (8.0, 2.0, 0.0)[min(2, int(u * 3.0))]
    if cfg.spike in ("half8", "p30", "perseq"):
        if cfg.spike == "half8":
            p8 = 0.5
        elif cfg.spike == "p30":
            p8 = 0.3
        else:
            p8 = (seq_id % cfg.batch + 0.5) / cfg.batch
        if u < p8:
            return 8.0
        return 2.0 if u < p8 + 0.5 * (1.0 - p8) else 0.0
    if cfg.spike == "exp4":
        return float(np.float32(-4.0 * math.log(u)))
    if cfg.spike == "all8":
        return 8.0
    if cfg.spike == "none":
        return 0.0
    raise ValueError(cfg.spike)


def root_token(cfg: TalonConfig, seed: int, seq_id: int) -> int:
    return mix64(row_key(seed, STREAM_ROOT, seq_id)) % cfg.vocab


def prefix_len(cfg: TalonConfig, seed: int, seq_id: int) -> int:
    span = cfg.prefix_max - cfg.prefix_min + 1
    return cfg.prefix_min + (mix64(row_key(seed, STREAM_PREFIX, seq_id)) % span)


def _add_at(z, tok: int, h: float):
    if isinstance(z, np.ndarray):
        z[tok] = np.float32(z[tok] + np.float32(h))
    else:
        z[tok] = z[tok] + h
    return z


def draft_logits_row(cfg: TalonConfig, seed: int, seq_id: int, path: Sequence[int], device=None):
    """fp32 draft logits of the node reached by ``path`` (root token first): T*g + h*[w == spike]."""
    ph = fold_path(path)
    key = row_key(seed, STREAM_DRAFT, seq_id, ph)
    g = gaussian(key, cfg.vocab, device)
    if device is None:
        z = g * np.float32(cfg.temp)
    else:
        z = g * float(np.float32(cfg.temp))
    h = spike_height(cfg, seed, seq_id, ph)
    if h != 0.0:
        z = _add_at(z, mix64(key ^ _ODD_B) % cfg.vocab, h)
    return z


def target_logits_row(cfg: TalonConfig, seed: int, seq_id: int, path: Sequence[int], device=None):
    """fp32 target logits after the node at ``path``: the draft row plus half-scale fresh noise."""
    z = draft_logits_row(cfg, seed, seq_id, path, device)
    ph = fold_path(path)
    g2 = gaussian(row_key(seed, STREAM_TARGET, seq_id, ph), cfg.vocab, device)
    if device is None:
        return z + g2 * np.float32(0.5)
    return z + g2 * 0.5


def zipf_logits_row(vocab: int, alpha: float, seed: int, row_id: int, device=None):
    """Zipfian row of the paper's tree-construction micro-benchmark: P(r) ~ r^-alpha.

    The logit of the token holding rank r is -alpha*ln(r).  Ranks are spread over the token
    ids by a hashed permutation: an affine map with an odd multiplier modulo the next
    power of two, cycle-walked until the image falls inside the vocabulary.  (The log is
    taken by the host or device math library, so generate a row once and hand the same
    array to every consumer.)
    """
    key = row_key(seed, STREAM_ZIPF, row_id)
    nbits = max(1, (vocab - 1).bit_length())
    size = 1 << nbits
    a = (mix64(key) | 1) & (size - 1)
    c = mix64(key ^ _ODD_A) & (size - 1)
    w = _arange64(vocab, device)
    # cycle-walk the affine map on [0, size) until the image falls in [0, vocab)
    r = (w * a + c) & (size - 1)
    for _ in range(64):
        bad = r >= vocab
        if not bool(bad.any()):
            break
        r2 = (r * a + c) & (size - 1)
        if device is None:
            r = np.where(bad, r2, r)
        else:
            import torch
            r = torch.where(bad, r2, r)
    if device is None:
        return (-alpha * np.log((r + 1).astype(np.float64))).astype(np.float32)
    import torch
    return (-alpha * torch.log((r + 1).to(torch.float64))).to(torch.float32)


def qkv_block(seed: int, stream: int, seq_id: int, n_elems: int, device=None, start: int = 0):
    """``n_elems`` N(0,1) values rounded to bf16 (returned as fp32) for one tensor of one sequence."""
    return round_to_bf16(gaussian(row_key(seed, stream, seq_id), n_elems, device, start))
