"""Thin ctypes binding over ``libtalon.so`` (the C ABI declared in ``include/talon.h``).

Only argument marshalling happens here: torch supplies device memory and streams, every step
of the path runs in the library's CUDA kernels.  There is no CPU fallback: if the library has
not been built (``python -m paper_2601_07353_b200.build``) importing this module raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional

import torch

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libtalon.so")
if not os.path.exists(_LIB_PATH):
    raise ImportError(
        f"{_LIB_PATH} is missing: build the CUDA library first with "
        "`python -m paper_2601_07353_b200.build` (needs nvcc); there is no CPU fallback")
_lib = C.CDLL(_LIB_PATH)

OK, ERR_INVALID_ARG, ERR_CAPACITY, ERR_CUDA, ERR_TIMEOUT, ERR_NONFINITE, ERR_UNSUPPORTED = range(7)
ROWS_BY_NODE, ROWS_PACKED = 0, 1


class TalonParams(C.Structure):
    _fields_ = [("batch_max", C.c_int32), ("vocab", C.c_int32), ("budget", C.c_int32),
                ("root_topk", C.c_int32), ("cand_topk", C.c_int32), ("max_depth", C.c_int32),
                ("init_layers", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("mu", C.c_double)]


class TalonTreeStruct(C.Structure):
    _fields_ = [("n_nodes", C.c_void_p), ("token", C.c_void_p), ("parent", C.c_void_p),
                ("depth", C.c_void_p), ("position", C.c_void_p), ("layer_off", C.c_void_p),
                ("score", C.c_void_p), ("mask", C.c_void_p)]


_vp, _i32, _i64, _f32 = C.c_void_p, C.c_int32, C.c_int64, C.c_float
_TP = C.POINTER(TalonTreeStruct)
_lib.talon_create.argtypes = [C.POINTER(_vp), C.POINTER(TalonParams), C.c_int]
_lib.talon_destroy.argtypes = [_vp]
_lib.talon_reset.argtypes = [_vp, _TP, _vp, _vp, _i32, _vp]
_lib.talon_expand_layer.argtypes = [_vp, _TP, _vp, _i64, _i32, _i32, _vp]
_lib.talon_layers_run.argtypes = [_vp]
_lib.talon_build_tree.argtypes = [_vp, _TP, _vp, _vp]
_lib.talon_prune_tree.argtypes = [_vp, _TP, _i32, _vp]
_lib.talon_tree_attention_paged.argtypes = [_vp, _TP, _vp, _vp, _vp, _vp, _vp, _vp, _i32, _i64, _i64, _i64, _i32, _f32, _vp, _vp]
_lib.talon_commit_paged.argtypes = [_vp, _TP] + [_vp] * 8 + [_i32, _vp, _i64, _i64, _i64, _vp, _vp, _vp, _vp]
_lib.talon_loop.argtypes = ([_vp, _TP, _i32, _i32, _vp, _vp, _vp, _i64, _i64, _i32, _vp, _i64, _vp, _vp, _vp, _vp, _i64, _vp, _vp,
                            _i64, _i64, _i64, _i32, _f32, _vp, _vp, _i64, _i64, _vp, _vp, _vp, _vp, _i64, _vp, _vp])
_lib.talon_loop_metrics.argtypes = [_vp, _i32, C.c_double, C.POINTER(C.c_double), C.POINTER(C.c_double), C.POINTER(C.c_double)]
_lib.talon_tree_attention.argtypes = [_vp, _TP, _vp, _vp, _vp, _vp, _vp, _vp, _i64, _i64, _i64, _i32, _f32, _vp, _vp]
_lib.talon_accept.argtypes = [_vp, _TP, _vp, _i64, _vp, _vp, _vp, _vp, _vp]
_lib.talon_close_and_accept.argtypes = [_vp, _TP, _vp, _i64, _vp, _vp, _vp, _vp, _vp]
_lib.talon_accept_sample.argtypes = [_vp, _TP, _vp, _i64, C.c_double, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.talon_commit.argtypes = [_vp, _TP] + [_vp] * 9 + [_i64, _i64, _i64, _vp, _vp, _vp, _vp]
_lib.talon_poll_status.argtypes = [_vp, _vp]
_lib.talon_step_host.argtypes = [_vp, _i32] + [_vp] * 9 + [_f32] + [_vp] * 10
_lib.talon_step.argtypes = ([_vp, _TP, _i32, _vp, _vp, _vp, _i64, _i32] + [_vp] * 6 + [_i64, _i64, _i64, _i32, _f32, _vp,
                            _vp, _i64] + [_vp] * 5)
_lib.talon_timing_enable.argtypes = [_vp, _i32, C.c_uint32]
_lib.talon_timing_pause.argtypes = [_vp, _i32]
_lib.talon_timing_read.argtypes = [_vp, _vp, C.POINTER(C.c_double), C.POINTER(C.c_int64)]
_lib.talon_kernel_name.argtypes = [_i32]
_lib.talon_kernel_name.restype = C.c_char_p
_lib.talon_target_argmax_noalloc.argtypes = [_vp, _i64, _i32, _i32, _vp, _vp]
_lib.talon_launch_count.argtypes = [_vp]
_lib.talon_launch_count.restype = C.c_int64
_lib.talon_status_string.argtypes = [C.c_int]
_lib.talon_status_string.restype = C.c_char_p
for _n in ("talon_create", "talon_destroy", "talon_reset", "talon_expand_layer", "talon_layers_run",
           "talon_build_tree", "talon_tree_attention", "talon_accept", "talon_poll_status", "talon_step_host",
           "talon_step", "talon_timing_enable", "talon_timing_read", "talon_timing_pause",
           "talon_target_argmax_noalloc", "talon_accept_sample", "talon_commit", "talon_prune_tree",
           "talon_tree_attention_paged", "talon_commit_paged", "talon_loop", "talon_loop_metrics",
           "talon_close_and_accept"):
    getattr(_lib, _n).restype = C.c_int

EXPORTED = ["talon_create", "talon_destroy", "talon_reset", "talon_expand_layer", "talon_layers_run",
            "talon_build_tree", "talon_tree_attention", "talon_accept", "talon_poll_status",
            "talon_step_host", "talon_step", "talon_timing_enable", "talon_timing_read", "talon_timing_pause",
            "talon_kernel_name",
            "talon_launch_count", "talon_status_string", "talon_target_argmax_noalloc", "talon_accept_sample",
            "talon_commit", "talon_prune_tree", "talon_tree_attention_paged", "talon_commit_paged", "talon_loop",
            "talon_loop_metrics", "talon_close_and_accept"]
PAGE_TOKENS = 128
NOALLOC_MAX_ROWS = 8192
N_KERNELS = 11
KERNEL_NAMES = [_lib.talon_kernel_name(i).decode() for i in range(N_KERNELS)]


class TalonError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {_lib.talon_status_string(code).decode()} ({code})")


def _check(code: int, where: str):
    if code != OK:
        raise TalonError(code, where)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(device) -> C.c_void_p:
    return C.c_void_p(torch.cuda.current_stream(device).cuda_stream)


def loop_metrics(counters: torch.Tensor, cost_ratio: float) -> dict:
    """``talon_loop_metrics``: Section 5.3's delta, tau and speed-up from the counters ``talon_commit``
    keeps ([B, 3] int64).  The arithmetic is the library's; this only copies the counters to the host."""
    host = counters.detach().to("cpu", torch.int64).contiguous()
    d, t, r = C.c_double(), C.c_double(), C.c_double()
    _check(_lib.talon_loop_metrics(C.c_void_p(host.data_ptr()), host.shape[0], float(cost_ratio), C.byref(d), C.byref(t),
                                   C.byref(r)), "talon_loop_metrics")
    n_p, n_q, length = (int(x) for x in host.sum(dim=0).tolist())
    return {"n_p": n_p, "n_q": n_q, "tokens": length, "delta": d.value, "tau": t.value, "speedup": r.value}


def target_argmax_noalloc(target_logits: torch.Tensor, target_tok: torch.Tensor) -> None:
    """``talon_target_argmax_noalloc``: greedy target token of every row of ``target_logits``
    ([rows, V] fp32 on the current CUDA device) into ``target_tok`` ([rows] int32), with no context
    and no allocation in the library: for callers that are not allowed to call cudaMalloc.  At most
    ``NOALLOC_MAX_ROWS`` rows; the library's single scratch array is shared by all calls, so calls
    must not overlap on the GPU."""
    rows = target_logits.numel() // target_logits.shape[-1]
    _check(_lib.talon_target_argmax_noalloc(_ptr(target_logits), target_logits.stride(-2), target_logits.shape[-1],
                                            rows, _ptr(target_tok), _stream(target_logits.device)),
           "talon_target_argmax_noalloc")


@dataclass
class Tree:
    """Caller-owned device arrays of the draft tree (``talon_tree`` in the header)."""
    n_nodes: torch.Tensor
    token: torch.Tensor
    parent: torch.Tensor
    depth: torch.Tensor
    position: torch.Tensor
    layer_off: torch.Tensor
    score: torch.Tensor
    mask: torch.Tensor

    def struct(self) -> TalonTreeStruct:
        return TalonTreeStruct(*(t.data_ptr() for t in (self.n_nodes, self.token, self.parent, self.depth,
                                                          self.position, self.layer_off, self.score, self.mask)))


class Talon:
    """One library context (``talon_ctx``) on one CUDA device; methods mirror the C calls."""

    def __init__(self, *, batch_max, vocab, budget, root_topk, cand_topk, max_depth, n_q_heads, n_kv_heads,
                 head_dim=128, mu=0.03, init_layers=1, device=0):
        if not torch.cuda.is_available():
            raise RuntimeError("talon needs a CUDA device; there is no CPU path")
        self.device = torch.device("cuda", device)
        self.params = TalonParams(batch_max, vocab, budget, root_topk, cand_topk, max_depth, init_layers,
                                  n_q_heads, n_kv_heads, head_dim, mu)
        self._ctx = C.c_void_p()
        _check(_lib.talon_create(C.byref(self._ctx), C.byref(self.params), device), "talon_create")
        self.N, self.V, self.W = budget, vocab, (budget + 63) // 64

    def close(self):
        if self._ctx:
            _lib.talon_destroy(self._ctx)
            self._ctx = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def alloc_tree(self, B: int) -> Tree:
        d, N = self.device, self.N
        i32 = dict(dtype=torch.int32, device=d)
        return Tree(torch.zeros(B, **i32), torch.zeros(B, N, **i32), torch.zeros(B, N, **i32),
                    torch.zeros(B, N, **i32), torch.zeros(B, N, **i32),
                    torch.zeros(B, self.params.max_depth + 2, **i32),
                    torch.zeros(B, N, dtype=torch.float64, device=d),
                    torch.zeros(B, N, self.W, dtype=torch.int64, device=d))

    def reset(self, tree: Tree, root_tok: torch.Tensor, prefix_len: torch.Tensor):
        B = root_tok.shape[0]
        ts = tree.struct()
        _check(_lib.talon_reset(self._ctx, C.byref(ts), _ptr(root_tok), _ptr(prefix_len), B,
                                _stream(self.device)), "talon_reset")

    def expand_layer(self, tree: Tree, logits: torch.Tensor, rows_per_seq: Optional[int] = None,
                     layout: int = ROWS_BY_NODE, row_stride: Optional[int] = None):
        ts = tree.struct()
        if row_stride is None:
            row_stride = logits.stride(-2)
        if rows_per_seq is None:
            rows_per_seq = logits.shape[-2]
        _check(_lib.talon_expand_layer(self._ctx, C.byref(ts), _ptr(logits), row_stride, rows_per_seq, layout,
                                       _stream(self.device)), "talon_expand_layer")

    def layers_run(self) -> int:
        return _lib.talon_layers_run(self._ctx)

    def build_tree(self, tree: Tree, dense_mask: Optional[torch.Tensor] = None):
        ts = tree.struct()
        _check(_lib.talon_build_tree(self._ctx, C.byref(ts), _ptr(dense_mask), _stream(self.device)),
               "talon_build_tree")

    def prune_tree(self, tree: Tree, keep: int):
        """``talon_prune_tree``: the final Top-N step of the static construction (Algorithm 1)."""
        ts = tree.struct()
        _check(_lib.talon_prune_tree(self._ctx, C.byref(ts), int(keep), _stream(self.device)), "talon_prune_tree")

    def tree_attention(self, tree: Tree, q, k_prefix, v_prefix, k_tree, v_tree, kv_start, kv_tokens, kv_stride_t,
                       kv_stride_h, max_prefix_len, sm_scale, out):
        ts = tree.struct()
        _check(_lib.talon_tree_attention(self._ctx, C.byref(ts), _ptr(q), _ptr(k_prefix), _ptr(v_prefix),
                                         _ptr(k_tree), _ptr(v_tree), _ptr(kv_start), kv_tokens, kv_stride_t, kv_stride_h,
                                         max_prefix_len, sm_scale, _ptr(out), _stream(self.device)),
               "talon_tree_attention")

    def accept(self, tree: Tree, target_logits, accept_len, accept_nodes, bonus_tok, target_tok=None,
               row_stride: Optional[int] = None):
        ts = tree.struct()
        if row_stride is None:
            row_stride = target_logits.stride(-2)
        _check(_lib.talon_accept(self._ctx, C.byref(ts), _ptr(target_logits), row_stride, _ptr(target_tok),
                                 _ptr(accept_len), _ptr(accept_nodes), _ptr(bonus_tok), _stream(self.device)),
               "talon_accept")

    def close_and_accept(self, tree: Tree, target_logits, accept_len, accept_nodes, bonus_tok, target_tok=None,
                         row_stride: Optional[int] = None):
        ts = tree.struct()
        if row_stride is None:
            row_stride = target_logits.stride(-2)
        _check(_lib.talon_close_and_accept(self._ctx, C.byref(ts), _ptr(target_logits), row_stride, _ptr(target_tok),
                                           _ptr(accept_len), _ptr(accept_nodes), _ptr(bonus_tok), _stream(self.device)),
               "talon_close_and_accept")

    def accept_sample(self, tree: Tree, target_logits, temperature: float, u_accept, u_sample, accept_len,
                      accept_nodes, out_tok, row_stride: Optional[int] = None):
        ts = tree.struct()
        if row_stride is None:
            row_stride = target_logits.stride(-2)
        assert u_accept.dtype == torch.float64 and u_sample.dtype == torch.float64
        _check(_lib.talon_accept_sample(self._ctx, C.byref(ts), _ptr(target_logits), row_stride, float(temperature),
                                        _ptr(u_accept), _ptr(u_sample), _ptr(accept_len), _ptr(accept_nodes),
                                        _ptr(out_tok), _stream(self.device)), "talon_accept_sample")

    def commit(self, tree: Tree, accept_len, accept_nodes, next_tok, k_tree, v_tree, k_prefix, v_prefix, kv_start,
               kv_limit, kv_tokens, kv_stride_t, kv_stride_h, prefix_len, root_tok, counters=None):
        ts = tree.struct()
        _check(_lib.talon_commit(self._ctx, C.byref(ts), _ptr(accept_len), _ptr(accept_nodes), _ptr(next_tok),
                                 _ptr(k_tree), _ptr(v_tree), _ptr(k_prefix), _ptr(v_prefix), _ptr(kv_start),
                                 _ptr(kv_limit), kv_tokens, kv_stride_t, kv_stride_h, _ptr(prefix_len), _ptr(root_tok),
                                 _ptr(counters), _stream(self.device)), "talon_commit")

    def tree_attention_paged(self, tree: Tree, q, k_pages, v_pages, k_tree, v_tree, block_table, n_pages, kv_stride_t,
                             kv_stride_h, max_prefix_len, sm_scale, out):
        ts = tree.struct()
        _check(_lib.talon_tree_attention_paged(self._ctx, C.byref(ts), _ptr(q), _ptr(k_pages), _ptr(v_pages), _ptr(k_tree),
                                               _ptr(v_tree), _ptr(block_table), block_table.stride(0), n_pages, kv_stride_t,
                                               kv_stride_h, max_prefix_len, sm_scale, _ptr(out), _stream(self.device)),
               "talon_tree_attention_paged")

    def commit_paged(self, tree: Tree, accept_len, accept_nodes, next_tok, k_tree, v_tree, k_pages, v_pages, block_table,
                     n_blocks, n_pages, kv_stride_t, kv_stride_h, prefix_len, root_tok, counters=None):
        ts = tree.struct()
        _check(_lib.talon_commit_paged(self._ctx, C.byref(ts), _ptr(accept_len), _ptr(accept_nodes), _ptr(next_tok),
                                       _ptr(k_tree), _ptr(v_tree), _ptr(k_pages), _ptr(v_pages), _ptr(block_table),
                                       block_table.stride(0), _ptr(n_blocks), n_pages, kv_stride_t, kv_stride_h,
                                       _ptr(prefix_len), _ptr(root_tok), _ptr(counters), _stream(self.device)),
               "talon_commit_paged")

    def loop(self, tree: Tree, n_steps, root_tok, prefix_len, draft, n_layers, q, k_prefix, v_prefix, k_tree, v_tree,
             kv_start, kv_limit, kv_tokens, kv_stride_t, kv_stride_h, max_prefix_len, sm_scale, out, target, target_tok,
             accept_len, accept_nodes, bonus_tok, counters, keep_results: bool = True):
        """``talon_loop``: ``n_steps`` draft-and-verify steps with the commit between them.  ``draft`` and
        ``target`` are [S, B, N, V]; ``q``, ``k_tree``, ``v_tree`` [S, B, N, H, Dh]; with ``keep_results`` the
        result arrays are [S, B(, D_max + 1)], else the last step's."""
        ts = tree.struct()
        B = root_tok.shape[0]
        _check(_lib.talon_loop(self._ctx, C.byref(ts), B, n_steps, _ptr(root_tok), _ptr(prefix_len), _ptr(draft),
                               draft.stride(-2), draft.stride(0), n_layers, _ptr(q), q.stride(0), _ptr(k_prefix),
                               _ptr(v_prefix), _ptr(k_tree), _ptr(v_tree), k_tree.stride(0), _ptr(kv_start), _ptr(kv_limit),
                               kv_tokens, kv_stride_t, kv_stride_h, max_prefix_len, sm_scale, _ptr(out), _ptr(target),
                               target.stride(-2), target.stride(0), _ptr(target_tok), _ptr(accept_len), _ptr(accept_nodes),
                               _ptr(bonus_tok), B if keep_results else 0, _ptr(counters), _stream(self.device)),
               "talon_loop")

    def poll_status(self) -> int:
        return _lib.talon_poll_status(self._ctx, _stream(self.device))

    def launch_count(self) -> int:
        return _lib.talon_launch_count(self._ctx)

    def step(self, tree: Tree, root_tok, prefix_len, draft_logits, n_layers, q, k_prefix, v_prefix, k_tree, v_tree,
             kv_start, kv_tokens, kv_stride_t, kv_stride_h, max_prefix_len, sm_scale, out, target_logits, target_tok,
             accept_len, accept_nodes, bonus_tok):
        """``talon_step``: the whole draft-and-verify step on device-resident inputs, one library call."""
        ts = tree.struct()
        _check(_lib.talon_step(self._ctx, C.byref(ts), root_tok.shape[0], _ptr(root_tok), _ptr(prefix_len),
                               _ptr(draft_logits), draft_logits.stride(-2), n_layers, _ptr(q), _ptr(k_prefix),
                               _ptr(v_prefix), _ptr(k_tree), _ptr(v_tree), _ptr(kv_start), kv_tokens, kv_stride_t,
                               kv_stride_h, max_prefix_len, sm_scale, _ptr(out), _ptr(target_logits), target_logits.stride(-2),
                               _ptr(target_tok), _ptr(accept_len), _ptr(accept_nodes), _ptr(bonus_tok),
                               _stream(self.device)), "talon_step")

    def timing_enable(self, max_launches: int, kernels=None):
        """Bracket launches with CUDA events; ``kernels`` = names to time (None: all); 0 switches off."""
        mask = 0
        for k in kernels or ():
            mask |= 1 << KERNEL_NAMES.index(k)
        _check(_lib.talon_timing_enable(self._ctx, max_launches, mask), "talon_timing_enable")

    def timing_pause(self, paused: bool):
        _check(_lib.talon_timing_pause(self._ctx, 1 if paused else 0), "talon_timing_pause")

    def timing_read(self):
        """Returns {kernel name: (summed ms, launches)} since the last read (synchronises the stream)."""
        ms = (C.c_double * N_KERNELS)()
        n = (C.c_int64 * N_KERNELS)()
        _check(_lib.talon_timing_read(self._ctx, _stream(self.device), ms, n), "talon_timing_read")
        return {KERNEL_NAMES[i]: (ms[i], n[i]) for i in range(N_KERNELS)}

    def step_host(self, root_tok, prefix_len, draft_logits, target_logits, q, k_prefix, v_prefix, k_tree, v_tree,
                  sm_scale, out_attn, n_nodes, token, parent, depth, position, accept_len, accept_nodes,
                  bonus_tok) -> int:
        """All arguments are HOST tensors (pinned for asynchronous copies).  Returns the status."""
        B = root_tok.shape[0]
        return _lib.talon_step_host(self._ctx, B, _ptr(root_tok), _ptr(prefix_len), _ptr(draft_logits),
                                    _ptr(target_logits), _ptr(q), _ptr(k_prefix), _ptr(v_prefix), _ptr(k_tree),
                                    _ptr(v_tree), sm_scale, _ptr(out_attn), _ptr(n_nodes), _ptr(token),
                                    _ptr(parent), _ptr(depth), _ptr(position), _ptr(accept_len),
                                    _ptr(accept_nodes), _ptr(bonus_tok), _stream(self.device))
