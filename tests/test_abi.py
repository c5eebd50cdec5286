"""The C-ABI library loads and exports every symbol the header declares (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib_path():
    from paper_2609_34420_b200 import build
    return build.build()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "gt_attn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gt_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_four_entry_points():
    syms = declared_symbols()
    for name in ("gt_spd_build", "gt_biased_attn_fwd", "gt_biased_attn_bwd", "gt_biased_attn_fwd_chunked"):
        assert name in syms


def test_library_exports_every_declared_symbol(lib_path):
    L = ctypes.CDLL(lib_path)
    missing = [s for s in declared_symbols() if not hasattr(L, s)]
    assert not missing, missing


def test_binding_lists_the_same_symbols(lib_path):
    from paper_2609_34420_b200 import binding
    assert sorted(binding.EXPORTS) == declared_symbols()


def test_status_strings_and_host_side_validation(lib_path):
    from paper_2609_34420_b200 import binding
    L = binding.lib()
    assert L.gt_status_string(0) == b"GT_OK" and L.gt_status_string(5) == b"GT_ERR_DEVICE_TIMEOUT"
    bad = binding._GtBatch(0, 1, None, 0)
    assert L.gt_spd_build_workspace(ctypes.byref(bad), 0, 4) == 0
    # argument errors are returned before any CUDA call is made
    assert L.gt_spd_build(None, None, 0, ctypes.byref(bad), 4, None, None, None, 0, None) == 1
