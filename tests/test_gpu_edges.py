"""GPU edge cases through the C ABI: degenerate inputs, error reporting, layouts, the host-buffer step."""
import math

import numpy as np
import pytest
import torch

from oracle import talon_oracle as O
from paper_2601_07353_b200 import synth
from tests import parity_util as PU

pytestmark = pytest.mark.gpu
SEED = 77


def _mods():
    from paper_2601_07353_b200 import talon, workload
    return talon, workload


def _simple_ctx(V=512, N=16, K=4, k=4, D=8, B=2, Hq=4, Hkv=2, mu=0.03):
    talon, _ = _mods()
    return talon.Talon(batch_max=B, vocab=V, budget=N, root_topk=K, cand_topk=k, max_depth=D, n_q_heads=Hq,
                       n_kv_heads=Hkv, mu=mu)


def _expand_all(t, tree, logits, root, plen, layers):
    t.reset(tree, root, plen)
    for _ in range(layers):
        t.expand_layer(tree, logits)
    t.build_tree(tree)
    torch.cuda.synchronize()


def test_all_equal_logits_follow_the_tie_break_rule():
    talon, _ = _mods()
    V, N, K = 64, 14, 3
    t = _simple_ctx(V=V, N=N, K=K, k=K, B=1)
    tree = t.alloc_tree(1)
    logits = torch.zeros(1, N, V, device="cuda")
    _expand_all(t, tree, logits, torch.zeros(1, dtype=torch.int32, device="cuda"),
                torch.zeros(1, dtype=torch.int32, device="cuda"), 8)
    ref = O.expand(0, lambda path: np.zeros(V, np.float32), O.Params(N, K, K, 0.03, 8))
    assert tree.n_nodes.item() == N
    assert (tree.token[0].cpu().numpy() == ref.token).all() and (tree.parent[0].cpu().numpy() == ref.parent).all()
    t.close()


def test_minus_inf_logits_are_legal_and_never_selected():
    talon, _ = _mods()
    V, N = 200, 10
    t = _simple_ctx(V=V, N=N, B=1)
    tree = t.alloc_tree(1)
    logits = torch.full((1, N, V), float("-inf"), device="cuda")
    logits[:, :, 7] = 1.0
    logits[:, :, 100] = 0.5
    _expand_all(t, tree, logits, torch.zeros(1, dtype=torch.int32, device="cuda"),
                torch.zeros(1, dtype=torch.int32, device="cuda"), 8)
    assert t.poll_status() == talon.OK
    ref = O.expand(0, lambda path: logits[0, 0].cpu().numpy(), O.Params(N, 4, 4, 0.03, 8))
    n = tree.n_nodes.item()
    assert n == ref.n_nodes
    assert (tree.token[0].cpu().numpy()[:n] == ref.token[:n]).all()
    assert set(tree.token[0].cpu().numpy()[1:n]) <= {7, 100}
    t.close()


@pytest.mark.parametrize("bad", [float("nan"), float("inf"), "all_minus_inf"])
def test_nonfinite_rows_set_the_status_word_and_stop_the_sequence(bad):
    talon, _ = _mods()
    V, N = 300, 12
    t = _simple_ctx(V=V, N=N, B=2)
    tree = t.alloc_tree(2)
    g = torch.Generator(device="cuda").manual_seed(1)
    logits = torch.randn(2, N, V, device="cuda", generator=g)
    if bad == "all_minus_inf":
        logits[1, 0, :] = float("-inf")
    else:
        logits[1, 0, 17] = bad
    _expand_all(t, tree, logits, torch.zeros(2, dtype=torch.int32, device="cuda"),
                torch.zeros(2, dtype=torch.int32, device="cuda"), 8)
    assert t.poll_status() == talon.ERR_NONFINITE
    assert tree.n_nodes[1].item() == 1 and tree.n_nodes[0].item() == N      # the clean sequence is unaffected
    # reset clears the word
    t.reset(tree, torch.zeros(2, dtype=torch.int32, device="cuda"), torch.zeros(2, dtype=torch.int32, device="cuda"))
    assert t.poll_status() == talon.OK
    t.close()


def test_host_side_validation():
    talon, _ = _mods()
    with pytest.raises(talon.TalonError):
        talon.Talon(batch_max=1, vocab=100, budget=300, root_topk=4, cand_topk=4, max_depth=4, n_q_heads=4, n_kv_heads=2)
    with pytest.raises(talon.TalonError) as e:
        talon.Talon(batch_max=1, vocab=100, budget=8, root_topk=4, cand_topk=4, max_depth=4, n_q_heads=4, n_kv_heads=2,
                    head_dim=64)
    assert e.value.code == talon.ERR_UNSUPPORTED
    t = _simple_ctx(V=512, B=2)
    tree = t.alloc_tree(2)
    z = torch.zeros(2, 16, 512, device="cuda")
    with pytest.raises(talon.TalonError):          # expand before reset
        t.expand_layer(tree, z)
    root = torch.zeros(3, dtype=torch.int32, device="cuda")
    with pytest.raises(talon.TalonError) as e:     # batch larger than batch_max
        t.reset(tree, root, root)
    assert e.value.code == talon.ERR_CAPACITY
    t.reset(tree, root[:2], root[:2])
    with pytest.raises(talon.TalonError):          # misaligned rows
        t.expand_layer(tree, z.view(-1)[1:1 + 2 * 15 * 512].view(2, 15, 512), rows_per_seq=16)
    with pytest.raises(talon.TalonError):          # stride not a multiple of 4
        t.expand_layer(tree, z, row_stride=513)
    t.close()


def test_packed_layout_equals_by_node_layout():
    talon, workload = _mods()
    cfg = synth.CONFIGS["tiny"].scaled(vocab=2048, batch=3, budget=24)
    t = workload.make_talon(cfg)
    wl = workload.build_workload(cfg, t, SEED, with_verify=False)
    ref = PU.tree_to_host(wl.tree, 1)
    lo_all = wl.tree.layer_off.cpu().numpy()
    tree2 = t.alloc_tree(3)
    t.reset(tree2, wl.root_tok, wl.prefix_len)
    cap = cfg.budget
    for d in range(wl.layers_run):
        packed = torch.zeros(3, cap, cfg.vocab, device="cuda")
        for b in range(3):
            lo, hi = int(lo_all[b, d]), int(lo_all[b, d + 1])
            packed[b, : hi - lo] = wl.draft[b, lo:hi]
        t.expand_layer(tree2, packed, rows_per_seq=cap, layout=talon.ROWS_PACKED)
    t.build_tree(tree2)
    got = PU.tree_to_host(tree2, 1)
    for k in ("token", "parent", "depth", "position", "mask", "layer_off"):
        assert (got[k] == ref[k]).all()
    t.close()


def test_dense_mask_output():
    talon, workload = _mods()
    cfg = synth.CONFIGS["longctx"].scaled(vocab=1024, batch=2, prefix_min=3, prefix_max=9)
    t = workload.make_talon(cfg)
    wl = workload.build_workload(cfg, t, SEED, with_verify=False)
    dense = torch.zeros(2, cfg.budget, cfg.budget, dtype=torch.uint8, device="cuda")
    t.build_tree(wl.tree, dense)
    for b in range(2):
        g = PU.tree_to_host(wl.tree, b)
        want = O.dense_mask(PU.oracle_tree_from_arrays(g, cfg.budget, cfg.max_depth))
        n = g["n_nodes"]
        got = dense[b].cpu().numpy().astype(bool)
        assert (got[:n, :n] == want[:n, :n]).all()
        for i in range(n, cfg.budget):
            assert got[i].sum() == 1 and got[i, i]
    t.close()


def test_chain_tree_attention_is_causal_attention():
    """A chain-shaped tree must reduce to causal attention (Appendix B), checked against torch SDPA on CPU."""
    talon, workload = _mods()
    cfg = synth.CONFIGS["llama8b"].scaled(vocab=1024, spike="all8", mu=1.0, topk=1, budget=20, max_depth=30,
                                          prefix_min=77, prefix_max=77)
    t = workload.make_talon(cfg)
    wl = workload.build_workload(cfg, t, SEED)
    workload.run_step(t, wl)
    torch.cuda.synchronize()
    n, L, Hq, g = cfg.budget, 77, cfg.n_q_heads, cfg.group
    assert wl.tree.parent[0].cpu().tolist() == [-1] + list(range(n - 1))
    K = torch.cat([wl.k_prefix[:L], wl.k_tree[0]]).double().cpu().permute(1, 0, 2).repeat_interleave(g, 0)
    V = torch.cat([wl.v_prefix[:L], wl.v_tree[0]]).double().cpu().permute(1, 0, 2).repeat_interleave(g, 0)
    Q = torch.zeros(Hq, L + n, cfg.head_dim, dtype=torch.float64)
    Q[:, L:] = wl.q[0].double().cpu().permute(1, 0, 2)
    ref = torch.nn.functional.scaled_dot_product_attention(Q, K, V, is_causal=True)[:, L:].permute(1, 0, 2)
    err = (wl.out[0].double().cpu() - ref).abs()
    assert err.max() <= 1e-2 and err.mean() <= 1e-3
    t.close()


def test_host_buffer_step_matches_device_calls():
    talon, workload = _mods()
    cfg = synth.CONFIGS["tiny"].scaled(vocab=4096, batch=3, prefix_min=40, prefix_max=200)
    t = workload.make_talon(cfg)
    wl = workload.build_workload(cfg, t, SEED)
    workload.run_step(t, wl)
    torch.cuda.synchronize()
    B, N, D = 3, cfg.budget, cfg.max_depth
    pin = lambda x: x.cpu().pin_memory()
    hi32 = lambda *s: torch.zeros(*s, dtype=torch.int32).pin_memory()
    out = torch.zeros(B, N, cfg.n_q_heads, cfg.head_dim, dtype=torch.bfloat16).pin_memory()
    n_nodes, token, parent, depth, position = hi32(B), hi32(B, N), hi32(B, N), hi32(B, N), hi32(B, N)
    alen, anodes, bonus = hi32(B), hi32(B, D + 1), hi32(B)
    for _ in range(2):
        st = t.step_host(pin(wl.root_tok), pin(wl.prefix_len), pin(wl.draft), pin(wl.target), pin(wl.q),
                         pin(wl.k_prefix), pin(wl.v_prefix), pin(wl.k_tree), pin(wl.v_tree),
                         1.0 / math.sqrt(cfg.head_dim), out, n_nodes, token, parent, depth, position, alen, anodes, bonus)
        assert st == talon.OK
        assert torch.equal(n_nodes, wl.tree.n_nodes.cpu()) and torch.equal(token, wl.tree.token.cpu())
        assert torch.equal(parent, wl.tree.parent.cpu()) and torch.equal(position, wl.tree.position.cpu())
        assert torch.equal(out, wl.out.cpu())
        assert torch.equal(alen, wl.accept_len.cpu()) and torch.equal(anodes, wl.accept_nodes.cpu())
        assert torch.equal(bonus, wl.bonus_tok.cpu())
    t.close()


def test_target_argmax_ties_and_nan():
    talon, workload = _mods()
    cfg = synth.CONFIGS["tiny"].scaled(vocab=40000, batch=2, prefix_min=8, prefix_max=8)
    t = workload.make_talon(cfg)
    wl = workload.build_workload(cfg, t, SEED)
    wl.target[0, 0, :] = 0.0                       # all equal: lowest id wins
    wl.target[0, 1, :] = float("-inf")
    wl.target[0, 1, 39999] = -3.0
    wl.target[1, 0, 123] = 50.0
    wl.target[1, 0, 30123] = 50.0
    workload.run_step(t, wl)
    assert t.poll_status() == talon.OK
    tt = wl.target_tok.cpu().numpy()
    assert tt[0, 0] == 0 and tt[0, 1] == 39999 and tt[1, 0] == 123
    wl.target[1, 1, 5] = float("nan")
    workload.run_step(t, wl)
    assert t.poll_status() == talon.ERR_NONFINITE
    t.close()
