"""The C-ABI library loads and exports every function that include/talon.h declares (no GPU needed)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "talon.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(talon_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2601_07353_b200 import build
    path = build.build()
    lib = ctypes.CDLL(path)
    names = declared_functions()
    assert {"talon_expand_layer", "talon_build_tree", "talon_tree_attention", "talon_accept"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in talon.h but not exported"


def test_status_strings_and_host_side_argument_checks():
    from paper_2601_07353_b200 import build
    lib = ctypes.CDLL(build.build())
    lib.talon_status_string.restype = ctypes.c_char_p
    assert lib.talon_status_string(0) == b"ok"
    assert len({lib.talon_status_string(i) for i in range(7)}) == 7
    # null arguments are rejected before any CUDA call
    assert lib.talon_create(None, None, 0) == 1
    assert lib.talon_destroy(None) == 0
    assert lib.talon_reset(None, None, None, None, 1, None) == 1
    assert lib.talon_expand_layer(None, None, None, ctypes.c_int64(0), 0, 0, None) == 1
    assert lib.talon_build_tree(None, None, None, None) == 1
    assert lib.talon_poll_status(None, None) == 1
    # the later additions reject a missing context the same way
    i64 = ctypes.c_int64
    assert lib.talon_accept(None, None, None, i64(0), None, None, None, None, None) == 1
    assert lib.talon_close_and_accept(None, None, None, i64(0), None, None, None, None, None) == 1
    assert lib.talon_prune_tree(None, None, 1, None) == 1
    assert lib.talon_loop_metrics(None, 1, ctypes.c_double(0.05), None, None, None) == 1
    # delta, tau and R of Eq. 6-7 are host arithmetic behind the C ABI: 3 verification passes, 12 draft
    # passes, 9 tokens give delta 4, tau 3 and R = 3 / (1 + 0.1 * 4)
    cnt = (i64 * 6)(1, 5, 2, 2, 7, 7)
    d, tau, r = ctypes.c_double(), ctypes.c_double(), ctypes.c_double()
    assert lib.talon_loop_metrics(cnt, 2, ctypes.c_double(0.1), ctypes.byref(d), ctypes.byref(tau), ctypes.byref(r)) == 0
    assert d.value == 4.0 and tau.value == 3.0 and abs(r.value - 3.0 / 1.4) < 1e-15


def test_binding_names_match_header():
    src = open(os.path.join(ROOT, "paper_2601_07353_b200", "talon.py")).read()
    for n in declared_functions():
        assert n in src, f"binding does not mention {n}"


def test_the_product_has_no_cpu_route():
    """The package never imports the oracle, and without a CUDA device a context cannot be made."""
    import glob
    import pytest
    import torch
    for path in glob.glob(os.path.join(ROOT, "paper_2601_07353_b200", "*.py")):
        src = open(path).read()
        assert "oracle" not in src or "talon_oracle" not in src, f"{path} mentions the oracle module"
        assert not re.search(r"^\s*(from|import)\s+oracle\b", src, flags=re.M), f"{path} imports the oracle"
    for path in glob.glob(os.path.join(ROOT, "oracle", "*.py")):
        src = open(path).read()
        assert not re.search(r"^\s*(from|import)\s+paper_2601_07353_b200\b", src, flags=re.M), f"{path} imports the package"
    if not torch.cuda.is_available():
        from paper_2601_07353_b200 import talon
        with pytest.raises(RuntimeError):
            talon.Talon(batch_max=1, vocab=100, budget=8, root_topk=4, cand_topk=4, max_depth=4, n_q_heads=4, n_kv_heads=2)
