"""talon_commit on the GPU against the oracle's bookkeeping (Section 5.3's generation loop):
cache rows bit for bit, prefix lengths, next roots, counters; the committed cache then serves a
second step's tree attention; a block without room is refused."""
import math

import numpy as np
import pytest
import torch

from oracle import talon_oracle as O
from paper_2601_07353_b200 import synth
from tests import parity_util as PU

pytestmark = pytest.mark.gpu
SEED = synth.DEFAULT_SEED


def _setup(cfg, seqs, room):
    """A verified step plus a prefix cache with `room[b]` free tokens behind each sequence's prefix."""
    from paper_2601_07353_b200 import talon, workload
    t = workload.make_talon(cfg, batch_max=len(seqs))
    wl = workload.build_workload(cfg, t, SEED, seqs)
    workload.run_step(t, wl)
    assert t.poll_status() == talon.OK
    dev = wl.q.device
    plens = wl.prefix_len.cpu().numpy()
    old = wl.kv_start.cpu().numpy()
    blocks = [int(plens[b]) + room[b] for b in range(wl.B)]
    starts = np.concatenate([[0], np.cumsum(blocks)[:-1]]).astype(np.int64)
    limits = starts + np.asarray(blocks, np.int64)
    total = int(limits[-1]) + 3                      # a little slack behind the last block
    Hkv, Dh = cfg.n_kv_heads, cfg.head_dim
    kc = torch.full((total, Hkv, Dh), 7.0, dtype=torch.bfloat16, device=dev)
    vc = torch.full((total, Hkv, Dh), -7.0, dtype=torch.bfloat16, device=dev)
    for b in range(wl.B):
        L = int(plens[b])
        kc[starts[b]:starts[b] + L] = wl.k_prefix[old[b]:old[b] + L]
        vc[starts[b]:starts[b] + L] = wl.v_prefix[old[b]:old[b] + L]
    i64 = lambda x: torch.tensor(x, dtype=torch.int64, device=dev)
    return talon, t, wl, kc, vc, i64(starts), i64(limits), total, plens


def bits(x):
    return x.view(torch.int16).cpu().numpy()


def test_commit_matches_the_oracle_and_feeds_the_next_step():
    cfg = synth.CONFIGS["tiny"].scaled(batch=4, prefix_min=40, prefix_max=300)
    seqs = [0, 1, 2, 3]
    talon, t, wl, kc, vc, starts, limits, total, plens = _setup(cfg, seqs, [cfg.max_depth + 1] * 4)
    dev = wl.q.device
    B, N, Hkv, Dh = wl.B, cfg.budget, cfg.n_kv_heads, cfg.head_dim
    k_before, v_before = kc.clone(), vc.clone()
    plen = wl.prefix_len.clone()
    root = torch.zeros(B, dtype=torch.int32, device=dev)
    counters = torch.tensor([[5, 6, 7]] * B, dtype=torch.int64, device=dev)
    t.commit(wl.tree, wl.accept_len, wl.accept_nodes, wl.bonus_tok, wl.k_tree, wl.v_tree, kc, vc, starts, limits,
             total, Hkv * Dh, Dh, plen, root, counters)
    assert t.poll_status() == talon.OK
    p = PU.oracle_params(cfg)
    st = starts.cpu().numpy()
    touched = np.zeros(total, bool)
    for b, s in enumerate(seqs):
        tree = O.expand(synth.root_token(cfg, SEED, s), lambda path: synth.draft_logits_row(cfg, SEED, s, path), p)
        alen = int(wl.accept_len[b])
        path = wl.accept_nodes[b].cpu().numpy()
        L = int(plens[b])
        f = lambda x: x.to(torch.float32).cpu().numpy()
        k2, v2, nxt, cnt = O.commit(tree, alen, path, int(wl.bonus_tok[b]), f(wl.k_tree[b]), f(wl.v_tree[b]),
                                    f(k_before[st[b]:st[b] + L]), f(v_before[st[b]:st[b] + L]))
        n2 = L + alen + 1
        assert int(plen[b]) == n2 and int(root[b]) == nxt
        assert counters[b].cpu().tolist() == [5 + cnt[0], 6 + cnt[1], 7 + cnt[2]]
        assert (f(kc[st[b]:st[b] + n2]) == k2).all() and (f(vc[st[b]:st[b] + n2]) == v2).all()
        touched[st[b] + L: st[b] + n2] = True
    # nothing outside the appended rows changed, bit for bit
    keep = torch.from_numpy(~touched).to(dev)
    assert np.array_equal(bits(kc[keep]), bits(k_before[keep])) and np.array_equal(bits(vc[keep]), bits(v_before[keep]))

    # the next step's root attends to the longer prefix: root-only tree over the committed cache
    tree2 = t.alloc_tree(B)
    t.reset(tree2, root, plen)
    t.build_tree(tree2)
    out = torch.zeros_like(wl.out)
    scale = 1.0 / math.sqrt(Dh)
    t.tree_attention(tree2, wl.q, kc, vc, wl.k_tree, wl.v_tree, starts, total, Hkv * Dh, Dh, int(plen.max()), scale, out)
    assert t.poll_status() == talon.OK
    for b in range(B):
        g = PU.tree_to_host(tree2, b)
        assert g["n_nodes"] == 1 and g["position"][0] == int(plen[b])
        ot = PU.oracle_tree_from_arrays(g, N, cfg.max_depth)
        f = lambda x: x.to(torch.float32).cpu().numpy()
        n2 = int(plen[b])
        want = O.tree_attention(f(wl.q[b]), f(kc[st[b]:st[b] + n2]), f(vc[st[b]:st[b] + n2]), f(wl.k_tree[b]),
                                f(wl.v_tree[b]), ot, scale)
        err = np.abs(out[b, :1].to(torch.float64).cpu().numpy() - want[:1])
        assert err.max() <= 1e-2 and err.mean() <= 1e-3
    t.close()


def test_commit_refuses_a_block_without_room():
    cfg = synth.CONFIGS["tiny"].scaled(batch=3, prefix_min=20, prefix_max=60)
    talon, t, wl, kc, vc, starts, limits, total, plens = _setup(cfg, [0, 1, 2], [cfg.max_depth + 1, 0, cfg.max_depth + 1])
    dev = wl.q.device
    B, Hkv, Dh = wl.B, cfg.n_kv_heads, cfg.head_dim
    k_before = kc.clone()
    plen = wl.prefix_len.clone()
    root = torch.full((B,), -5, dtype=torch.int32, device=dev)
    t.commit(wl.tree, wl.accept_len, wl.accept_nodes, wl.bonus_tok, wl.k_tree, wl.v_tree, kc, vc, starts, limits,
             total, Hkv * Dh, Dh, plen, root, None)
    assert t.poll_status() == talon.ERR_CAPACITY
    st, lim = starts.cpu().numpy(), limits.cpu().numpy()
    assert int(plen[1]) == int(plens[1]) and int(root[1]) == -5            # untouched
    assert np.array_equal(bits(kc[st[1]:lim[1]]), bits(k_before[st[1]:lim[1]]))
    for b in (0, 2):
        assert int(plen[b]) == int(plens[b]) + int(wl.accept_len[b]) + 1 and int(root[b]) == int(wl.bonus_tok[b])
    t.close()


def test_commit_after_sampling_verification_on_a_full_size_tree():
    cfg = synth.CONFIGS["llama8b"]
    talon, t, wl, kc, vc, starts, limits, total, plens = _setup(cfg, [0], [cfg.max_depth + 1])
    dev = wl.q.device
    N, Hkv, Dh = cfg.budget, cfg.n_kv_heads, cfg.head_dim
    u, us = synth.verify_uniforms(SEED, 0, N, 1)
    tok = torch.zeros(1, dtype=torch.int32, device=dev)
    t.accept_sample(wl.tree, wl.target, 0.2, torch.from_numpy(u[None]).to(dev),
                    torch.tensor([us], dtype=torch.float64, device=dev), wl.accept_len, wl.accept_nodes, tok)
    plen = wl.prefix_len.clone()
    root = torch.zeros(1, dtype=torch.int32, device=dev)
    counters = torch.zeros(1, 3, dtype=torch.int64, device=dev)
    t.commit(wl.tree, wl.accept_len, wl.accept_nodes, tok, wl.k_tree, wl.v_tree, kc, vc, starts, limits, total,
             Hkv * Dh, Dh, plen, root, counters)
    assert t.poll_status() == talon.OK
    alen, L = int(wl.accept_len[0]), int(plens[0])
    path = wl.accept_nodes[0].cpu().numpy()
    for j in range(alen + 1):
        assert np.array_equal(bits(kc[L + j]), bits(wl.k_tree[0, int(path[j])]))
        assert np.array_equal(bits(vc[L + j]), bits(wl.v_tree[0, int(path[j])]))
    assert int(plen[0]) == L + alen + 1 and int(root[0]) == int(tok[0])
    g = PU.tree_to_host(wl.tree, 0)
    assert counters[0].cpu().tolist() == [1, int(g["depth"][: g["n_nodes"]].max()), alen + 1]
    t.close()
