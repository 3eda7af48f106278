"""Device-resident synthetic workloads for the tests and the benchmark.

``build_workload`` plays the role of the two model forwards that are out of scope: it fills a
per-node cache of draft-logit rows while the library grows the tree (each row depends on the
node's root-to-node token path, so the tree has to exist before its rows do), then the target
logits of every node and random bf16 Q/K/V.  It calls the library only through the binding and
holds none of the method's arithmetic.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional, Sequence

import numpy as np
import torch

from . import synth
from .talon import Talon, Tree, ROWS_BY_NODE


@dataclass
class Workload:
    cfg: synth.TalonConfig
    seed: int
    seq_ids: List[int]
    root_tok: torch.Tensor        # [B] i32
    prefix_len: torch.Tensor      # [B] i32
    kv_start: torch.Tensor        # [B] i64 (token offsets into the ragged prefix KV)
    max_prefix_len: int
    draft: torch.Tensor           # [B, N, V] fp32, row i = draft logits of node i (BY_NODE)
    target: torch.Tensor          # [B, N, V] fp32
    q: torch.Tensor               # [B, N, Hq, Dh] bf16
    k_prefix: torch.Tensor        # [sum L_b, Hkv, Dh] bf16
    v_prefix: torch.Tensor
    k_tree: torch.Tensor          # [B, N, Hkv, Dh] bf16
    v_tree: torch.Tensor
    tree: Tree
    out: torch.Tensor             # [B, N, Hq, Dh] bf16
    accept_len: torch.Tensor
    accept_nodes: torch.Tensor
    bonus_tok: torch.Tensor
    target_tok: torch.Tensor
    layers_run: int = 0

    @property
    def B(self) -> int:
        return len(self.seq_ids)


def make_talon(cfg: synth.TalonConfig, batch_max: Optional[int] = None, cand_topk: Optional[int] = None,
               device: int = 0, init_layers: int = 1) -> Talon:
    return Talon(batch_max=batch_max or cfg.batch, vocab=cfg.vocab, budget=cfg.budget, root_topk=cfg.topk,
                 cand_topk=cfg.topk if cand_topk is None else cand_topk, max_depth=cfg.max_depth,
                 n_q_heads=cfg.n_q_heads, n_kv_heads=cfg.n_kv_heads, head_dim=cfg.head_dim, mu=cfg.mu,
                 init_layers=init_layers, device=device)


def node_paths(token: np.ndarray, parent: np.ndarray, n: int) -> List[List[int]]:
    paths: List[List[int]] = []
    for i in range(n):
        paths.append([int(token[i])] if parent[i] < 0 else paths[int(parent[i])] + [int(token[i])])
    return paths


def _bf16(x32: torch.Tensor) -> torch.Tensor:
    return x32.to(torch.bfloat16)


def logit_rows(B: int, N: int, V: int, row_pad: int, dev) -> torch.Tensor:
    """[B, N, V] fp32 rows that start 16 bytes aligned: the row stride is V rounded up to a multiple
    of four elements plus ``row_pad``; what lies between the rows holds NaN, which no kernel may use."""
    assert row_pad % 4 == 0
    stride = (V + 3) // 4 * 4 + row_pad
    if stride == V:
        return torch.zeros(B, N, V, dtype=torch.float32, device=dev)
    buf = torch.full((B, N, stride), float("nan"), dtype=torch.float32, device=dev)
    rows = buf[:, :, :V]
    rows.zero_()
    return rows


def build_workload(cfg: synth.TalonConfig, talon: Talon, seed: int = synth.DEFAULT_SEED,
                   seq_ids: Optional[Sequence[int]] = None, with_verify: bool = True, row_pad: int = 0,
                   prefix_lens: Optional[Sequence[int]] = None, host_inputs: bool = False,
                   root_tokens: Optional[Sequence[int]] = None) -> Workload:
    """``row_pad`` widens the logit rows' stride (NaN padding); ``prefix_lens`` overrides the hashed
    prefix lengths of the sequences (the generated K/V of a sequence are cut to that length);
    ``root_tokens`` overrides the hashed root tokens (a later step of a generation loop starts from
    the previous step's correction token);
    ``host_inputs`` generates every input with NumPy on the host and uploads it (bit-identical to
    the device generator), so that the only kernels the GPU runs are the library's."""
    dev = talon.device
    gen_dev = None if host_inputs else dev
    up = (lambda x: torch.from_numpy(np.ascontiguousarray(x))) if host_inputs else (lambda x: x)
    seq_ids = list(range(cfg.batch)) if seq_ids is None else list(seq_ids)
    B, N, V = len(seq_ids), cfg.budget, cfg.vocab
    i32 = dict(dtype=torch.int32, device=dev)
    roots = [synth.root_token(cfg, seed, s) for s in seq_ids] if root_tokens is None else [int(x) for x in root_tokens]
    assert len(roots) == B
    root = torch.tensor(roots, **i32)
    plens = [synth.prefix_len(cfg, seed, s) for s in seq_ids] if prefix_lens is None else [int(x) for x in prefix_lens]
    assert len(plens) == B
    prefix_len = torch.tensor(plens, **i32)
    starts = np.concatenate([[0], np.cumsum(plens)[:-1]]).astype(np.int64)
    kv_start = torch.tensor(starts, dtype=torch.int64, device=dev)
    draft = logit_rows(B, N, V, row_pad, dev)
    tree = talon.alloc_tree(B)

    talon.reset(tree, root, prefix_len)
    done_rows = [0] * B                # nodes whose draft row is already in the cache
    layers = 0
    for d in range(cfg.max_depth):
        n_nodes = tree.n_nodes.cpu().numpy()
        token = tree.token.cpu().numpy()
        parent = tree.parent.cpu().numpy()
        lo = tree.layer_off.cpu().numpy()
        any_active = False
        for bi, s in enumerate(seq_ids):
            n = int(n_nodes[bi])
            if n >= N or lo[bi, d + 1] <= lo[bi, d]:
                continue
            any_active = True
            paths = node_paths(token[bi], parent[bi], n)
            for i in range(max(done_rows[bi], int(lo[bi, d])), int(lo[bi, d + 1])):
                draft[bi, i] = up(synth.draft_logits_row(cfg, seed, s, paths[i], device=gen_dev))
            done_rows[bi] = int(lo[bi, d + 1])
        if not any_active:
            break
        talon.expand_layer(tree, draft)
        layers += 1
    talon.build_tree(tree)

    Hq, Hkv, Dh = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    bf = dict(dtype=torch.bfloat16, device=dev)
    total = int(sum(plens))
    wl = Workload(cfg, seed, seq_ids, root, prefix_len, kv_start, max(plens), draft,
                  target=logit_rows(B, N, V, row_pad, dev) if with_verify else torch.zeros(1, 1, 4, dtype=torch.float32, device=dev),
                  q=torch.zeros(B, N, Hq, Dh, **bf), k_prefix=torch.zeros(max(total, 1), Hkv, Dh, **bf),
                  v_prefix=torch.zeros(max(total, 1), Hkv, Dh, **bf), k_tree=torch.zeros(B, N, Hkv, Dh, **bf),
                  v_tree=torch.zeros(B, N, Hkv, Dh, **bf), tree=tree, out=torch.zeros(B, N, Hq, Dh, **bf),
                  accept_len=torch.zeros(B, **i32), accept_nodes=torch.zeros(B, cfg.max_depth + 1, **i32),
                  bonus_tok=torch.zeros(B, **i32), target_tok=torch.zeros(B, N, **i32), layers_run=layers)
    if not with_verify:
        return wl

    n_nodes = tree.n_nodes.cpu().numpy()
    token = tree.token.cpu().numpy()
    parent = tree.parent.cpu().numpy()
    for bi, s in enumerate(seq_ids):
        n = int(n_nodes[bi])
        paths = node_paths(token[bi], parent[bi], n)
        for i in range(n):
            wl.target[bi, i] = up(synth.target_logits_row(cfg, seed, s, paths[i], device=gen_dev))
        wl.q[bi] = _bf16(up(synth.qkv_block(seed, synth.STREAM_Q, s, N * Hq * Dh, gen_dev))).view(N, Hq, Dh)
        wl.k_tree[bi] = _bf16(up(synth.qkv_block(seed, synth.STREAM_KT, s, N * Hkv * Dh, gen_dev))).view(N, Hkv, Dh)
        wl.v_tree[bi] = _bf16(up(synth.qkv_block(seed, synth.STREAM_VT, s, N * Hkv * Dh, gen_dev))).view(N, Hkv, Dh)
        L = plens[bi]
        if L:
            a = int(starts[bi])
            step = 4096                       # tokens per generation chunk (bounds temporaries)
            for t0 in range(0, L, step):
                t1 = min(L, t0 + step)
                cnt, off = (t1 - t0) * Hkv * Dh, t0 * Hkv * Dh
                wl.k_prefix[a + t0:a + t1] = _bf16(up(synth.qkv_block(seed, synth.STREAM_K, s, cnt, gen_dev, off))).view(-1, Hkv, Dh)
                wl.v_prefix[a + t0:a + t1] = _bf16(up(synth.qkv_block(seed, synth.STREAM_V, s, cnt, gen_dev, off))).view(-1, Hkv, Dh)
    return wl


def run_step(talon: Talon, wl: Workload, sm_scale: Optional[float] = None, expand_layers: Optional[int] = None):
    """One whole draft-and-verify step on device-resident inputs (what the benchmark times)."""
    cfg = wl.cfg
    if sm_scale is None:
        sm_scale = 1.0 / float(np.sqrt(cfg.head_dim))
    talon.reset(wl.tree, wl.root_tok, wl.prefix_len)
    for _ in range(cfg.max_depth if expand_layers is None else expand_layers):
        talon.expand_layer(wl.tree, wl.draft)
    talon.build_tree(wl.tree)
    talon.tree_attention(wl.tree, wl.q, wl.k_prefix, wl.v_prefix, wl.k_tree, wl.v_tree, wl.kv_start,
                         wl.k_prefix.shape[0], cfg.n_kv_heads * cfg.head_dim, cfg.head_dim, wl.max_prefix_len, sm_scale, wl.out)
    talon.accept(wl.tree, wl.target, wl.accept_len, wl.accept_nodes, wl.bonus_tok, wl.target_tok)


def run_step_fused(talon: Talon, wl: Workload, sm_scale: Optional[float] = None, n_layers: Optional[int] = None):
    """The same step through the single ``talon_step`` call."""
    cfg = wl.cfg
    if sm_scale is None:
        sm_scale = 1.0 / float(np.sqrt(cfg.head_dim))
    talon.step(wl.tree, wl.root_tok, wl.prefix_len, wl.draft, cfg.max_depth if n_layers is None else n_layers,
               wl.q, wl.k_prefix, wl.v_prefix, wl.k_tree, wl.v_tree, wl.kv_start, wl.k_prefix.shape[0],
               cfg.n_kv_heads * cfg.head_dim,
               cfg.head_dim, wl.max_prefix_len, sm_scale, wl.out, wl.target, wl.target_tok, wl.accept_len,
               wl.accept_nodes, wl.bonus_tok)
