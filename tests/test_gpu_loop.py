"""The steps either side of one draft-and-verify step (Section 5.3's generation loop) on the GPU:
a paged prefix cache for the tree attention and the commit, and several steps with the commit
between them in one call, against the oracle run step by step."""
import math

import numpy as np
import pytest
import torch

from oracle import talon_oracle as O
from paper_2601_07353_b200 import synth
from tests import parity_util as PU

pytestmark = pytest.mark.gpu
SEED = 1357
ATT_MAX_ABS, ATT_MEAN_ABS = 1e-2, 1e-3
PAGE = 128


def _mods():
    from paper_2601_07353_b200 import talon, workload
    return talon, workload


def bits(x):
    return x.contiguous().view(torch.int16).cpu().numpy()


def test_paged_cache_attention_and_commit():
    talon, workload = _mods()
    cfg = synth.CONFIGS["tiny"].scaled(batch=3, prefix_min=0, prefix_max=400)
    t = workload.make_talon(cfg)
    plens = [130, 0, 300]
    wl = workload.build_workload(cfg, t, SEED, prefix_lens=plens)
    workload.run_step(t, wl)                                     # contiguous cache: the reference output
    assert t.poll_status() == talon.OK
    dev = wl.q.device
    B, N, Hkv, Dh = wl.B, cfg.budget, cfg.n_kv_heads, cfg.head_dim
    # ---- scatter every sequence's prefix over pages of a shuffled pool ----
    need = [(L + cfg.max_depth + 1 + PAGE - 1) // PAGE for L in plens]     # room for the commit
    n_pages = sum(need) + 3
    order = np.random.default_rng(3).permutation(n_pages)
    table = np.full((B, max(need) + 1), -1, np.int32)
    nxt = 0
    for b in range(B):
        for j in range(need[b]):
            table[b, j] = order[nxt]; nxt += 1
    kpg = torch.full((n_pages * PAGE, Hkv, Dh), 3.0, dtype=torch.bfloat16, device=dev)
    vpg = torch.full((n_pages * PAGE, Hkv, Dh), -3.0, dtype=torch.bfloat16, device=dev)
    starts = wl.kv_start.cpu().numpy()
    for b in range(B):
        for tk in range(plens[b]):
            dst = int(table[b, tk // PAGE]) * PAGE + tk % PAGE
            kpg[dst] = wl.k_prefix[int(starts[b]) + tk]
            vpg[dst] = wl.v_prefix[int(starts[b]) + tk]
    bt = torch.tensor(np.maximum(table, 0), dtype=torch.int32, device=dev)
    nb = torch.tensor(need, dtype=torch.int32, device=dev)
    out = torch.zeros_like(wl.out)
    t.tree_attention_paged(wl.tree, wl.q, kpg, vpg, wl.k_tree, wl.v_tree, bt, n_pages, Hkv * Dh, Dh, max(plens),
                           1.0 / math.sqrt(Dh), out)
    assert t.poll_status() == talon.OK
    assert (bits(out) == bits(wl.out)).all()                     # the same tiles in the same order: the same bits
    f32 = lambda x: x.to(torch.float32).cpu().numpy()
    for b in range(B):
        g = PU.tree_to_host(wl.tree, b)
        tr = PU.oracle_tree_from_arrays(g, N, cfg.max_depth)
        a, L = int(starts[b]), plens[b]
        want = O.tree_attention(f32(wl.q[b]), f32(wl.k_prefix[a:a + L]), f32(wl.v_prefix[a:a + L]), f32(wl.k_tree[b]),
                                f32(wl.v_tree[b]), tr, 1.0 / math.sqrt(Dh))
        err = np.abs(out[b].to(torch.float64).cpu().numpy() - want)
        assert err.max() <= ATT_MAX_ABS and err.mean() <= ATT_MEAN_ABS
    # ---- commit through the page table against the oracle's commit on the gathered cache ----
    plen = wl.prefix_len.clone()
    root = torch.zeros(B, dtype=torch.int32, device=dev)
    counters = torch.zeros(B, 3, dtype=torch.int64, device=dev)
    t.commit_paged(wl.tree, wl.accept_len, wl.accept_nodes, wl.bonus_tok, wl.k_tree, wl.v_tree, kpg, vpg, bt, nb, n_pages,
                   Hkv * Dh, Dh, plen, root, counters)
    assert t.poll_status() == talon.OK
    for b in range(B):
        g = PU.tree_to_host(wl.tree, b)
        tr = PU.oracle_tree_from_arrays(g, N, cfg.max_depth)
        alen = int(wl.accept_len[b]); path = wl.accept_nodes[b].cpu().numpy()
        a, L = int(starts[b]), plens[b]
        k_new, v_new, nroot, _ = O.commit(tr, alen, path, int(wl.bonus_tok[b]), bits(wl.k_tree[b]), bits(wl.v_tree[b]),
                                          bits(wl.k_prefix[a:a + L]), bits(wl.v_prefix[a:a + L]))
        assert int(plen[b]) == L + alen + 1 and int(root[b]) == nroot
        idx = [int(table[b, tk // PAGE]) * PAGE + tk % PAGE for tk in range(L + alen + 1)]
        assert (bits(kpg[idx]) == k_new).all() and (bits(vpg[idx]) == v_new).all()
    # a sequence without room is refused
    nb_small = torch.tensor([(L + PAGE - 1) // PAGE for L in plens], dtype=torch.int32, device=dev)
    plen2 = torch.tensor([PAGE * int(x) for x in nb_small.cpu()], dtype=torch.int32, device=dev)    # pages exactly full
    t.commit_paged(wl.tree, wl.accept_len, wl.accept_nodes, wl.bonus_tok, wl.k_tree, wl.v_tree, kpg, vpg, bt, nb_small,
                   n_pages, Hkv * Dh, Dh, plen2, root, None)
    assert t.poll_status() == talon.ERR_CAPACITY
    t.close()


def test_multi_step_loop_in_one_call_matches_the_oracle_step_by_step():
    talon, workload = _mods()
    cfg = synth.CONFIGS["tiny"].scaled(batch=2, prefix_min=60, prefix_max=200, vocab=8000)
    S, seqs = 3, [4, 9]
    t = workload.make_talon(cfg)
    dev = t.device
    B, N, V, D, Hq, Hkv, Dh = 2, cfg.budget, cfg.vocab, cfg.max_depth, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    scale = 1.0 / math.sqrt(Dh)
    room = S * (D + 1)
    # ---- build the steps one after the other with plain calls: step s + 1 starts from step s's result ----
    lens = [synth.prefix_len(cfg, SEED, s) for s in seqs]
    roots = [synth.root_token(cfg, SEED, s) for s in seqs]
    blocks = [L + room for L in lens]
    starts = np.concatenate([[0], np.cumsum(blocks)[:-1]]).astype(np.int64)
    limits = starts + np.asarray(blocks, np.int64)
    total = int(limits[-1])
    i64 = lambda x: torch.tensor(np.asarray(x), dtype=torch.int64, device=dev)
    kv_start, kv_limit = i64(starts), i64(limits)
    kc = torch.zeros(total, Hkv, Dh, dtype=torch.bfloat16, device=dev)
    vc = torch.zeros(total, Hkv, Dh, dtype=torch.bfloat16, device=dev)
    plen = torch.tensor(lens, dtype=torch.int32, device=dev)
    root = torch.tensor(roots, dtype=torch.int32, device=dev)
    counters = torch.zeros(B, 3, dtype=torch.int64, device=dev)
    steps, ref_results = [], []
    k_host = [None] * B; v_host = [None] * B
    for s in range(S):
        cur_lens, cur_roots = plen.cpu().tolist(), root.cpu().tolist()
        wl = workload.build_workload(cfg, t, SEED + s, seqs, prefix_lens=cur_lens, root_tokens=cur_roots)
        if s == 0:
            ws = wl.kv_start.cpu().numpy()
            for b in range(B):
                kc[starts[b]:starts[b] + lens[b]] = wl.k_prefix[int(ws[b]):int(ws[b]) + lens[b]]
                vc[starts[b]:starts[b] + lens[b]] = wl.v_prefix[int(ws[b]):int(ws[b]) + lens[b]]
                k_host[b] = bits(kc[starts[b]:starts[b] + lens[b]]); v_host[b] = bits(vc[starts[b]:starts[b] + lens[b]])
            k0, v0 = kc.clone(), vc.clone()
        t.reset(wl.tree, root, plen)
        for _ in range(D):
            t.expand_layer(wl.tree, wl.draft)
        t.build_tree(wl.tree)
        t.tree_attention(wl.tree, wl.q, kc, vc, wl.k_tree, wl.v_tree, kv_start, total, Hkv * Dh, Dh, max(cur_lens), scale, wl.out)
        t.accept(wl.tree, wl.target, wl.accept_len, wl.accept_nodes, wl.bonus_tok, wl.target_tok)
        # ---- the oracle's step on the same inputs ----
        p = PU.oracle_params(cfg)
        for b, sq in enumerate(seqs):
            fn = lambda path: synth.draft_logits_row(cfg, SEED + s, sq, path)
            tr = O.expand(cur_roots[b], fn, p)
            g = PU.tree_to_host(wl.tree, b)
            assert g["n_nodes"] == tr.n_nodes and (g["token"][:tr.n_nodes] == tr.token[:tr.n_nodes]).all()
            tt = O.target_argmax(wl.target[b].cpu().numpy(), tr.n_nodes)
            alen, path, bonus = O.accept(tr, tt)
            assert int(wl.accept_len[b]) == alen and int(wl.bonus_tok[b]) == bonus
            k_host[b], v_host[b], nroot, cnt = O.commit(tr, alen, path, bonus, bits(wl.k_tree[b]), bits(wl.v_tree[b]),
                                                        k_host[b], v_host[b])
        ref_results.append((wl.accept_len.clone(), wl.accept_nodes.clone(), wl.bonus_tok.clone(), wl.out.clone()))
        t.commit(wl.tree, wl.accept_len, wl.accept_nodes, wl.bonus_tok, wl.k_tree, wl.v_tree, kc, vc, kv_start, kv_limit,
                 total, Hkv * Dh, Dh, plen, root, counters)
        assert t.poll_status() == talon.OK
        steps.append(wl)
    for b in range(B):                                           # the cache the plain calls left is the oracle's
        L = int(plen[b])
        assert L == len(k_host[b])
        assert (bits(kc[starts[b]:starts[b] + L]) == k_host[b]).all() and (bits(vc[starts[b]:starts[b] + L]) == v_host[b]).all()
    ref_state = (plen.clone(), root.clone(), counters.clone(), kc.clone(), vc.clone())

    # ---- the same loop as ONE call, captured in one CUDA graph and replayed ----
    draft = torch.stack([w.draft for w in steps]); target = torch.stack([w.target for w in steps])
    q = torch.stack([w.q for w in steps]); kt = torch.stack([w.k_tree for w in steps]); vt = torch.stack([w.v_tree for w in steps])
    tree = t.alloc_tree(B)
    out = torch.zeros(B, N, Hq, Dh, dtype=torch.bfloat16, device=dev)
    al = torch.zeros(S, B, dtype=torch.int32, device=dev); an = torch.zeros(S, B, D + 1, dtype=torch.int32, device=dev)
    bo = torch.zeros(S, B, dtype=torch.int32, device=dev); tt = torch.zeros(B, N, dtype=torch.int32, device=dev)
    plen2 = torch.zeros(B, dtype=torch.int32, device=dev); root2 = torch.zeros(B, dtype=torch.int32, device=dev)
    cnt2 = torch.zeros(B, 3, dtype=torch.int64, device=dev)
    kc2, vc2 = k0.clone(), v0.clone()
    max_len = max(lens) + room

    def fresh():
        plen2.copy_(torch.tensor(lens, dtype=torch.int32)); root2.copy_(torch.tensor(roots, dtype=torch.int32))
        cnt2.zero_(); kc2.copy_(k0); vc2.copy_(v0)

    call = lambda: t.loop(tree, S, root2, plen2, draft, D, q, kc2, vc2, kt, vt, kv_start, kv_limit, total, Hkv * Dh, Dh,
                          max_len, scale, out, target, tt, al, an, bo, cnt2)
    side = torch.cuda.Stream()
    fresh()
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        call()                                                  # plain launches first
        side.synchronize()
        launches = t.launch_count()
        g = torch.cuda.CUDAGraph()
        fresh()
        side.synchronize()
        with torch.cuda.graph(g, stream=side):
            call()
        per_loop = t.launch_count() - launches
        for rep in range(2):                                    # replay twice from the same start
            fresh()
            side.synchronize()
            g.replay()
            side.synchronize()
            assert t.poll_status() == talon.OK
            assert torch.equal(plen2, ref_state[0]) and torch.equal(root2, ref_state[1]) and torch.equal(cnt2, ref_state[2])
            assert (bits(kc2) == bits(ref_state[3])).all() and (bits(vc2) == bits(ref_state[4])).all()
            for s in range(S):
                assert torch.equal(al[s], ref_results[s][0]) and torch.equal(bo[s], ref_results[s][2])
                assert torch.equal(an[s], ref_results[s][1])
            assert (bits(out) == bits(ref_results[-1][3])).all()
    # per step at least: reset, D layers, attention, arg-max (its last CTA walks and closes the tree), 2 for the commit
    assert per_loop >= S * (D + 5)
    # Section 5.3's figures from the counters, against the oracle's formulas
    m = talon.loop_metrics(cnt2, 0.1)
    n_p, n_q, length = (int(x) for x in cnt2.sum(dim=0).tolist())
    assert n_p == S * B
    assert abs(m["delta"] - O.draft_efficiency(n_q, n_p)) < 1e-12
    assert abs(m["tau"] - O.mean_accepted_tokens(length, n_p)) < 1e-12
    assert abs(m["speedup"] - O.speedup(m["tau"], m["delta"], 0.1)) < 1e-12
    t.close()
