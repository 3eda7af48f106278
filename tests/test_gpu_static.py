"""GPU parity of the static tree construction (Algorithm 1) built from the same kernels: the depth
loop is the expansion call with Top-K at every layer, the last step is ``talon_prune_tree``."""
import numpy as np
import pytest
import torch

from oracle import talon_oracle as O
from paper_2601_07353_b200 import synth
from tests import parity_util as PU

pytestmark = pytest.mark.gpu
SEED = 20260107


def _static(cfg, K, D, keep, seqs):
    from paper_2601_07353_b200 import talon, workload
    cap = 1 + K * (D + 1)
    scfg = cfg.scaled(budget=cap, topk=K, max_depth=D + 1, batch=len(seqs))
    t = workload.make_talon(scfg, init_layers=D + 1)
    wl = workload.build_workload(scfg, t, SEED, seqs, with_verify=False)     # runs the D + 1 Top-K layers
    assert t.poll_status() == talon.OK
    before = [PU.tree_to_host(wl.tree, bi) for bi in range(len(seqs))]
    t.prune_tree(wl.tree, keep)
    t.build_tree(wl.tree)
    torch.cuda.synchronize()
    for bi, s in enumerate(seqs):
        fn = lambda path: synth.draft_logits_row(scfg, SEED, s, path)
        ref = O.expand_static(synth.root_token(scfg, SEED, s), fn, K, D)
        g0 = before[bi]
        n0 = ref.n_nodes
        assert g0["n_nodes"] == n0 == cap
        assert (g0["token"][:n0] == ref.token[:n0]).all() and (g0["parent"][:n0] == ref.parent[:n0]).all()
        assert np.abs(g0["score"][:n0] - ref.score[:n0]).max() <= 2e-5
        # Scores differ from the fp64 oracle in the last digits, so prune the oracle's tree with the
        # GPU's scores: the pruning rule itself must then agree bit for bit.
        ref.score[:n0] = g0["score"][:n0]
        pr = O.prune_static(ref, keep)
        fin = O.finalize(pr, synth.prefix_len(scfg, SEED, s))
        g = PU.tree_to_host(wl.tree, bi)
        n = pr.n_nodes
        assert g["n_nodes"] == n == min(keep, cap)
        for name in ("token", "parent", "depth", "position"):
            assert (g[name] == fin[name]).all(), f"{name} after pruning, sequence {s}"
        assert (g["mask"] == fin["mask"]).all()
        assert (g["layer_off"][: len(pr.layer_off)] == np.asarray(pr.layer_off)).all()
        assert (g["score"][:n] == fin["score"][:n]).all()
        # and with the oracle's own scores the same nodes survive unless two scores are within 1e-5
        own = O.prune_static(O.expand_static(synth.root_token(scfg, SEED, s), fn, K, D), keep)
        if not (own.token[:n] == g["token"][:n]).all():
            sc = np.sort(g0["score"][:n0])[::-1]
            assert abs(sc[keep - 1] - sc[keep]) < 1e-5, "pruning differs beyond the tie tolerance"
    t.close()


def test_static_tree_tiny():
    _static(synth.CONFIGS["tiny"], K=4, D=3, keep=12, seqs=[0, 1, 2, 3])


def test_static_tree_llama_shape_k10_d7_n60():
    _static(synth.CONFIGS["llama8b"], K=10, D=7, keep=60, seqs=[0, 1])


def test_static_tree_keep_larger_than_tree_changes_nothing():
    _static(synth.CONFIGS["tiny"], K=3, D=2, keep=64, seqs=[5])
