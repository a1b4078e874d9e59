"""CPU-side checks of the C-ABI library: it loads, exports every declared symbol, and its host-only
entry points and argument validation behave as the header says (no kernel is launched here)."""

import ctypes
import os
import re

import pytest

import paper_2607_21271_b200 as eq
from paper_2607_21271_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "eqlinear.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(eqlinear_\w+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = eq.load_library()
    names = declared_symbols()
    assert len(names) >= 15
    for name in names:
        assert hasattr(lib, name), f"{name} is declared in eqlinear.h but not exported"
    assert set(names) == set(binding.EXPORTED_SYMBOLS)


def test_binding_has_the_same_names():
    for name in binding.EXPORTED_SYMBOLS:
        if name == "eqlinear_status_string":
            assert callable(binding.status_string)
        else:
            assert callable(getattr(eq.binding, name)), name


def test_mac_counts_match_the_paper():
    # Theorem 1: 6/16 of the dense N*D*C at T = 4; Table 1 at c = 64: 1024 tokens, D = C = 256.
    spectral, dense = eq.eqlinear_count_macs(4, 64, 64, 1024)
    assert dense == 1024 * 256 * 256
    assert spectral * 16 == dense * 6
    assert abs(2 * dense / 1e9 - 0.134) < 1e-3            # Table 1: 0.134 GFLOPs for the dense layer
    # exact count for even T: (2T - 2) N Ci Co; never more than the paper's bound 4NDC/T^2 (T/2+1)
    for T in (2, 4, 6, 8, 12, 16, 32):
        s, d = eq.eqlinear_count_macs(T, 3, 5, 7)
        assert s == (2 * T - 2) * 7 * 3 * 5
        assert d == 7 * (3 * T) * (5 * T)
        assert s <= 4 * d // (T * T) * (T // 2 + 1)
    s, _ = eq.eqlinear_count_macs(5, 2, 2, 1)
    assert s == (2 * 5 - 1) * 4


def test_status_strings():
    for code in range(0, 8):
        assert len(eq.status_string(code)) > 0
    assert "unknown" in eq.status_string(99)


def test_workspace_bytes_validation():
    assert eq.eqlinear_workspace_bytes(8, 96, 384, eq.EQL_FP16) >= 2 * 8 * 96 * 384 * 4
    for bad_T in (9, 11, 24, 64):
        with pytest.raises(eq.EqlError) as e:
            eq.eqlinear_workspace_bytes(bad_T, 8, 8, eq.EQL_FP32)
        assert e.value.status == binding.EQL_ERR_UNSUPPORTED
    for T in (1, 3, 5, 6, 7, 12):                          # odd and other non-power-of-two orders are planned for
        assert eq.eqlinear_workspace_bytes(T, 8, 8, eq.EQL_FP32) >= 2 * T * 64 * 4
    with pytest.raises(eq.EqlError) as e:
        eq.eqlinear_workspace_bytes(4, 0, 8, eq.EQL_FP32)
    assert e.value.status == binding.EQL_ERR_INVALID_ARG
    with pytest.raises(eq.EqlError) as e:                  # 3 channels * 2 * 2 bytes = 12-byte rows
        eq.eqlinear_workspace_bytes(2, 3, 4, eq.EQL_FP16)
    assert e.value.status == binding.EQL_ERR_ALIGNMENT
    with pytest.raises(eq.EqlError) as e:
        eq.eqlinear_workspace_bytes(4, 8, 8, 7)
    assert e.value.status == binding.EQL_ERR_INVALID_ARG


def test_workspace_bytes_with_flags():
    """The dihedral flag doubles the tuple length (2T elements per channel) and has its own list of group orders."""
    D = binding.EQL_FLAG_DIHEDRAL
    plain = eq.eqlinear_workspace_bytes_flags(5, 8, 8, eq.EQL_FP32, 0)
    assert plain == eq.eqlinear_workspace_bytes(5, 8, 8, eq.EQL_FP32)
    dih = eq.eqlinear_workspace_bytes_flags(5, 8, 8, eq.EQL_FP32, D)
    assert dih >= 2 * 10 * 64 * 4 and dih > plain
    for bad_T in (1, 7, 12, 16):
        with pytest.raises(eq.EqlError) as e:
            eq.eqlinear_workspace_bytes_flags(bad_T, 8, 8, eq.EQL_FP32, D)
        assert e.value.status == binding.EQL_ERR_UNSUPPORTED
    with pytest.raises(eq.EqlError) as e:                  # D_3 in half precision: 3 channels * 6 * 2 bytes = 36-byte rows
        eq.eqlinear_workspace_bytes_flags(3, 3, 4, eq.EQL_FP16, D)
    assert e.value.status == binding.EQL_ERR_ALIGNMENT
    assert eq.eqlinear_workspace_bytes(8, 96, 384, eq.EQL_BF16) == eq.eqlinear_workspace_bytes(8, 96, 384, eq.EQL_FP16)


def test_plan_argument_errors_are_caught_before_any_cuda_call():
    lib = eq.load_library()
    h = ctypes.c_void_p(1234)
    # NULL weight
    assert lib.eqlinear_plan(ctypes.byref(h), 4, 8, 8, 0, None, None, 256, 1 << 20, 0, None) == binding.EQL_ERR_INVALID_ARG
    assert h.value is None
    # unsupported group order
    assert lib.eqlinear_plan(ctypes.byref(h), 9, 8, 8, 0, 256, None, 256, 1 << 20, 0, None) == binding.EQL_ERR_UNSUPPORTED
    # misaligned weight / workspace
    assert lib.eqlinear_plan(ctypes.byref(h), 4, 8, 8, 0, 260, None, 256, 1 << 20, 0, None) == binding.EQL_ERR_ALIGNMENT
    assert lib.eqlinear_plan(ctypes.byref(h), 4, 8, 8, 0, 256, None, 272, 1 << 20, 0, None) == binding.EQL_ERR_ALIGNMENT
    # short workspace
    assert lib.eqlinear_plan(ctypes.byref(h), 4, 8, 8, 0, 256, None, 256, 16, 0, None) == binding.EQL_ERR_WORKSPACE
    # unknown flag
    assert lib.eqlinear_plan(ctypes.byref(h), 4, 8, 8, 0, 256, None, 256, 1 << 20, 1 << 9, None) == binding.EQL_ERR_INVALID_ARG
    # NULL plan handles
    assert lib.eqlinear_fwd(None, 256, 512, 1, None) == binding.EQL_ERR_INVALID_ARG
    assert lib.eqlinear_bwd_data(None, 256, 512, 1, None) == binding.EQL_ERR_INVALID_ARG
    assert lib.eqlinear_bwd_weight(None, 256, 512, 768, None, 1, 1024, 0, None) == binding.EQL_ERR_INVALID_ARG
    assert lib.eqlinear_plan_destroy(None) == binding.EQL_OK


def test_missing_library_fails_loudly(tmp_path):
    with pytest.raises(FileNotFoundError):
        eq.load_library(str(tmp_path / "libeqlinear.so"))
