"""The C-ABI library builds, loads without a GPU and exports every symbol include/hsd.h declares."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "hsd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(hsd_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2510_19705_b200 import build
    path = build.build()
    lib = ctypes.CDLL(path)
    names = _declared_symbols()
    assert "hsd_verify_level" in names and "hsd_strerror" in names
    for n in names:
        assert hasattr(lib, n), n


def test_strerror_and_argument_validation_need_no_gpu():
    from paper_2510_19705_b200 import binding
    lib = binding.library()
    assert lib.hsd_strerror(0) == b"ok"
    assert lib.hsd_strerror(-2) == b"workspace too small"
    # null pointers / bad sizes are rejected before any CUDA call
    assert lib.hsd_draft_sample(None, 1, 1, 8, 0, 0, 0, None, None) == -1
    assert lib.hsd_verify_level(0, None, None, None, 1, 1, 8, 0, 0, 0, None, 0, None, None, None) == -1
    assert lib.hsd_verify_workspace_bytes(0, 3) == 0
    assert lib.hsd_verify_workspace_bytes(4, 3) == 256 + 4 * 7 * 16      # counters (one per sequence, padded) + row statistics


def test_context_setters_reject_a_null_context_without_a_gpu():
    from paper_2510_19705_b200 import binding
    lib = binding.library()
    binding._declare_engine(lib)
    alphas = (ctypes.c_double * 2)(0.5, 0.5)
    assert lib.hsd_set_iid_acceptance(None, alphas) == -1
    assert lib.hsd_set_exit_heads(None, None, None) == -1
    assert lib.hsd_set_trace(None, None, 0) == -1
