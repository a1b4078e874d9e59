"""Thin ctypes binding of libeqlinear's C ABI (include/eqlinear.h): argument marshalling only.

Every step of the path runs inside the library's CUDA kernels.  PyTorch is used by callers for
device memory and streams; this module only needs `.data_ptr()`-style integers and never falls
back to another implementation: if the shared library is missing, loading fails loudly.
"""

from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, byref, c_char_p, c_int, c_int32, c_int64, c_size_t, c_uint, c_uint32, c_void_p

_PKG_DIR = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG_DIR, "libeqlinear.so")

EQL_OK = 0
EQL_ERR_INVALID_ARG = 1
EQL_ERR_UNSUPPORTED = 2
EQL_ERR_ALIGNMENT = 3
EQL_ERR_WORKSPACE = 4
EQL_ERR_ARCH = 5
EQL_ERR_CUDA = 6
EQL_ERR_DEVICE_TIMEOUT = 7

EQL_FP32 = 0
EQL_FP16 = 1
EQL_BF16 = 2

EQL_FLAG_CORRELATION = 1
EQL_FLAG_FORCE_SIMT = 2
EQL_FLAG_FORCE_STREAMING = 4
EQL_FLAG_CTA_PAIR = 8
EQL_FLAG_NO_CTA_PAIR = 16
EQL_FLAG_GELU = 32
EQL_FLAG_DIHEDRAL = 64

EQL_STATIC_SCRATCH_BYTES = 32 << 20

# Every symbol include/eqlinear.h declares.
EXPORTED_SYMBOLS = (
    "eqlinear_status_string", "eqlinear_count_macs", "eqlinear_workspace_bytes", "eqlinear_plan",
    "eqlinear_plan_set_weight", "eqlinear_plan_info", "eqlinear_plan_device_status", "eqlinear_plan_destroy",
    "eqlinear_fwd", "eqlinear_bwd_data", "eqlinear_bwd_weight_scratch_bytes", "eqlinear_bwd_weight",
    "eqlinear_fwd_host", "eqlinear_bwd_data_host", "eqlinear_bwd_weight_host", "eqlinear_step_host", "eqlinear_bwd_weight_static",
    "eqlinear_spectrum_bytes", "eqlinear_fwd_save_spectrum", "eqlinear_bwd_weight_from_spectrum",
    "eqlinear_plan_clear_device_status", "eqlinear_plan_selftest_expired_wait", "eqlinear_plan_launch_counts",
    "eqlinear_workspace_bytes_flags",
)


class EqlInfo(ctypes.Structure):
    _fields_ = [
        ("T", c_int32), ("C_in", c_int32), ("C_out", c_int32), ("dtype", c_int32),
        ("flags", c_uint32),
        ("fwd_kernel", c_int32), ("bwd_data_kernel", c_int32), ("bwd_weight_kernel", c_int32),
        ("macs_per_token", c_int64), ("dense_macs_per_token", c_int64),
        ("bytes_per_token_fwd", c_int64), ("bytes_per_token_bwd_data", c_int64),
        ("bytes_per_token_bwd_weight", c_int64),
        ("workspace_bytes", c_size_t),
    ]


class EqlError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


_lib = None


def load_library(path: str | None = None) -> ctypes.CDLL:
    """Load libeqlinear.so (built by paper_2607_21271_b200.build). No fallback exists."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or os.environ.get("EQLINEAR_LIB") or LIB_PATH     # EQLINEAR_LIB: explicit path to another build
    if not os.path.exists(p):
        raise FileNotFoundError(
            f"{p} not found: build it with `python -m paper_2607_21271_b200.build` "
            "(there is no CPU or PyTorch fallback for this library)")
    lib = ctypes.CDLL(p)
    V, I, I64, SZ = c_void_p, c_int, c_int64, c_size_t
    lib.eqlinear_status_string.restype = c_char_p
    lib.eqlinear_status_string.argtypes = [I]
    sigs = {
        "eqlinear_count_macs": [I, I, I, I64, POINTER(I64), POINTER(I64)],
        "eqlinear_workspace_bytes": [I, I, I, I, POINTER(SZ)],
        "eqlinear_workspace_bytes_flags": [I, I, I, I, c_uint, POINTER(SZ)],
        "eqlinear_plan": [POINTER(V), I, I, I, I, V, V, V, SZ, c_uint, V],
        "eqlinear_plan_set_weight": [V, V, V, V],
        "eqlinear_plan_info": [V, POINTER(EqlInfo)],
        "eqlinear_plan_launch_counts": [V, I64, POINTER(c_int32)],
        "eqlinear_plan_device_status": [V, V],
        "eqlinear_plan_clear_device_status": [V, V],
        "eqlinear_plan_selftest_expired_wait": [V, V],
        "eqlinear_plan_destroy": [V],
        "eqlinear_fwd": [V, V, V, I64, V],
        "eqlinear_bwd_data": [V, V, V, I64, V],
        "eqlinear_bwd_weight_scratch_bytes": [V, I64, POINTER(SZ)],
        "eqlinear_bwd_weight": [V, V, V, V, V, I64, V, SZ, V],
        "eqlinear_fwd_host": [V, V, V, I64, V, V, V],
        "eqlinear_bwd_data_host": [V, V, V, I64, V, V, V],
        "eqlinear_bwd_weight_host": [V, V, V, V, V, I64, V, V, V, V, V, SZ, V],
        "eqlinear_bwd_weight_static": [V, V, V, V, V, I64, V],
        "eqlinear_step_host": [V, V, V, V, V, V, V, I64, V, V, V, V, V, V, V, SZ, V],
        "eqlinear_spectrum_bytes": [V, I64, POINTER(SZ)],
        "eqlinear_fwd_save_spectrum": [V, V, V, I64, V, SZ, V],
        "eqlinear_bwd_weight_from_spectrum": [V, V, SZ, V, V, V, I64, V, SZ, V],
    }
    for name, argtypes in sigs.items():
        fn = getattr(lib, name)
        fn.restype = I
        fn.argtypes = argtypes
    if path is None:
        _lib = lib
    return lib


def _check(status: int, where: str) -> None:
    if status != EQL_OK:
        raise EqlError(status, where)


def _ptr(t) -> int | None:
    """Address of a tensor-like (torch tensor / numpy array), a raw int, or None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if hasattr(t, "data_ptr"):
        return t.data_ptr()
    if hasattr(t, "ctypes"):
        return t.ctypes.data
    raise TypeError(f"cannot take the address of {type(t)}")


def status_string(status: int) -> str:
    return load_library().eqlinear_status_string(status).decode()


def eqlinear_count_macs(T: int, C_in: int, C_out: int, N: int) -> tuple[int, int]:
    s, d = c_int64(0), c_int64(0)
    _check(load_library().eqlinear_count_macs(T, C_in, C_out, N, byref(s), byref(d)), "eqlinear_count_macs")
    return s.value, d.value


def eqlinear_workspace_bytes(T: int, C_in: int, C_out: int, dtype: int) -> int:
    out = c_size_t(0)
    _check(load_library().eqlinear_workspace_bytes(T, C_in, C_out, dtype, byref(out)), "eqlinear_workspace_bytes")
    return out.value


def eqlinear_workspace_bytes_flags(T: int, C_in: int, C_out: int, dtype: int, flags: int) -> int:
    out = c_size_t(0)
    _check(load_library().eqlinear_workspace_bytes_flags(T, C_in, C_out, dtype, flags, byref(out)), "eqlinear_workspace_bytes_flags")
    return out.value


def eqlinear_plan(T, C_in, C_out, dtype, w, bias, workspace, workspace_bytes, flags=0, stream=0) -> int:
    """Returns the opaque plan handle (an integer address)."""
    h = c_void_p(None)
    _check(load_library().eqlinear_plan(byref(h), T, C_in, C_out, dtype, _ptr(w), _ptr(bias), _ptr(workspace),
                                        workspace_bytes, flags, stream or None), "eqlinear_plan")
    return h.value


def eqlinear_plan_set_weight(plan, w, bias, stream=0) -> None:
    _check(load_library().eqlinear_plan_set_weight(plan, _ptr(w), _ptr(bias), stream or None), "eqlinear_plan_set_weight")


def eqlinear_plan_info(plan) -> EqlInfo:
    info = EqlInfo()
    _check(load_library().eqlinear_plan_info(plan, byref(info)), "eqlinear_plan_info")
    return info


def eqlinear_plan_launch_counts(plan, N) -> dict:
    """Kernel launches one call of each entry point makes for N tokens with this plan."""
    c = (c_int32 * 4)()
    _check(load_library().eqlinear_plan_launch_counts(plan, N, c), "eqlinear_plan_launch_counts")
    return {"fwd": c[0], "bwd_data": c[1], "bwd_weight": c[2], "fwd_save_spectrum_extra": c[3]}


def eqlinear_plan_device_status(plan, stream=0) -> int:
    return load_library().eqlinear_plan_device_status(plan, stream or None)


def eqlinear_plan_clear_device_status(plan, stream=0) -> None:
    _check(load_library().eqlinear_plan_clear_device_status(plan, stream or None), "eqlinear_plan_clear_device_status")


def eqlinear_plan_selftest_expired_wait(plan, stream=0) -> None:
    _check(load_library().eqlinear_plan_selftest_expired_wait(plan, stream or None), "eqlinear_plan_selftest_expired_wait")


def eqlinear_plan_destroy(plan) -> None:
    _check(load_library().eqlinear_plan_destroy(plan), "eqlinear_plan_destroy")


def eqlinear_fwd(plan, x, y, N, stream=0) -> None:
    _check(load_library().eqlinear_fwd(plan, _ptr(x), _ptr(y), N, stream or None), "eqlinear_fwd")


def eqlinear_bwd_data(plan, dy, dx, N, stream=0) -> None:
    _check(load_library().eqlinear_bwd_data(plan, _ptr(dy), _ptr(dx), N, stream or None), "eqlinear_bwd_data")


def eqlinear_bwd_weight_scratch_bytes(plan, N) -> int:
    out = c_size_t(0)
    _check(load_library().eqlinear_bwd_weight_scratch_bytes(plan, N, byref(out)), "eqlinear_bwd_weight_scratch_bytes")
    return out.value


def eqlinear_bwd_weight(plan, x, dy, dw, db, N, scratch, scratch_bytes, stream=0) -> None:
    _check(load_library().eqlinear_bwd_weight(plan, _ptr(x), _ptr(dy), _ptr(dw), _ptr(db), N, _ptr(scratch),
                                              scratch_bytes, stream or None), "eqlinear_bwd_weight")


def eqlinear_fwd_host(plan, x_host, y_host, N, x_staging, y_staging, stream=0) -> None:
    _check(load_library().eqlinear_fwd_host(plan, _ptr(x_host), _ptr(y_host), N, _ptr(x_staging), _ptr(y_staging),
                                            stream or None), "eqlinear_fwd_host")


def eqlinear_bwd_data_host(plan, dy_host, dx_host, N, dy_staging, dx_staging, stream=0) -> None:
    _check(load_library().eqlinear_bwd_data_host(plan, _ptr(dy_host), _ptr(dx_host), N, _ptr(dy_staging),
                                                 _ptr(dx_staging), stream or None), "eqlinear_bwd_data_host")


def eqlinear_bwd_weight_host(plan, x_host, dy_host, dw_host, db_host, N, x_staging, dy_staging, dw_staging,
                             db_staging, scratch, scratch_bytes, stream=0) -> None:
    _check(load_library().eqlinear_bwd_weight_host(plan, _ptr(x_host), _ptr(dy_host), _ptr(dw_host), _ptr(db_host), N,
                                                   _ptr(x_staging), _ptr(dy_staging), _ptr(dw_staging),
                                                   _ptr(db_staging), _ptr(scratch), scratch_bytes, stream or None),
           "eqlinear_bwd_weight_host")


def eqlinear_step_host(plan, x_host, dy_host, y_host, dx_host, dw_host, db_host, N, x_staging, dy_staging, y_staging,
                       dx_staging, dw_staging, db_staging, scratch, scratch_bytes, stream=0) -> None:
    _check(load_library().eqlinear_step_host(plan, _ptr(x_host), _ptr(dy_host), _ptr(y_host), _ptr(dx_host),
                                             _ptr(dw_host), _ptr(db_host), N, _ptr(x_staging), _ptr(dy_staging),
                                             _ptr(y_staging), _ptr(dx_staging), _ptr(dw_staging), _ptr(db_staging),
                                             _ptr(scratch), scratch_bytes, stream or None), "eqlinear_step_host")


def eqlinear_spectrum_bytes(plan, N) -> int:
    out = c_size_t(0)
    _check(load_library().eqlinear_spectrum_bytes(plan, N, byref(out)), "eqlinear_spectrum_bytes")
    return out.value


def eqlinear_fwd_save_spectrum(plan, x, y, N, spectrum, spectrum_bytes, stream=0) -> None:
    """eqlinear_fwd that also saves the fp16 spectrum of x for eqlinear_bwd_weight_from_spectrum."""
    _check(load_library().eqlinear_fwd_save_spectrum(plan, _ptr(x), _ptr(y), N, _ptr(spectrum), spectrum_bytes,
                                                     stream or None), "eqlinear_fwd_save_spectrum")


def eqlinear_bwd_weight_from_spectrum(plan, spectrum, spectrum_bytes, dy, dw, db, N, scratch, scratch_bytes, stream=0) -> None:
    _check(load_library().eqlinear_bwd_weight_from_spectrum(plan, _ptr(spectrum), spectrum_bytes, _ptr(dy), _ptr(dw),
                                                            _ptr(db), N, _ptr(scratch), scratch_bytes, stream or None),
           "eqlinear_bwd_weight_from_spectrum")


def eqlinear_bwd_weight_static(plan, x, dy, dw, db, N, stream=0) -> None:
    """eqlinear_bwd_weight for callers that cannot allocate device scratch: the library's built-in
    32 MiB device array is used instead (shared by all calls; do not overlap two of them)."""
    _check(load_library().eqlinear_bwd_weight_static(plan, _ptr(x), _ptr(dy), _ptr(dw), _ptr(db), N, stream or None),
           "eqlinear_bwd_weight_static")
