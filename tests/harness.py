"""Shared helpers for the GPU parity tests: run the C-ABI library on a workload and compare with the oracle."""

from __future__ import annotations

import numpy as np
import torch

import paper_2607_21271_b200 as eq
from oracle import eqlinear_oracle as orc

# max|err| / max|ref|.  FP32 and FP16: the stated parity bars.  BF16 (not among the stated configurations): derived from
# the arithmetic -- the scheme is the FP16 one (spectra of activations and weight rounded once, float accumulation, one
# rounding of the output) with unit roundoff u = 2^-9 instead of 2^-11; the FP16 path measures 0.8-1.3 u_half against
# its bar of 6 u_half, the BF16 bar is the same 6 u = 1.2e-2.
TOL = {"fp32": 1e-5, "fp16": 3e-3, "bf16": 6 * 2.0 ** -9}
CANARY = 64                                  # guard elements after every output buffer


def torch_dtype(dtype: str):
    return {"fp32": torch.float32, "fp16": torch.float16, "bf16": torch.bfloat16}[dtype]


def eql_dtype(dtype: str) -> int:
    return {"fp32": eq.EQL_FP32, "fp16": eq.EQL_FP16, "bf16": eq.EQL_BF16}[dtype]


def to_device(a: np.ndarray, dtype: str, dev):
    """Host array of a workload -> device tensor of the plan's dtype (bf16 inputs are float32 arrays holding
    bfloat16-representable values: the narrowing is exact)."""
    return torch.from_numpy(np.ascontiguousarray(a)).to(dev).to(torch_dtype(dtype))


def to_host(t) -> np.ndarray:
    return (t.float() if t.dtype == torch.bfloat16 else t).cpu().numpy()


def rel_max_err(got: np.ndarray, ref: np.ndarray) -> float:
    scale = float(np.abs(ref).max())
    err = float(np.abs(got.astype(np.float64) - ref).max())
    return err / scale if scale > 0 else err


class GpuLayer:
    """One plan plus its buffers, all through the C ABI."""

    def __init__(self, T, Ci, Co, dtype, w, bias, flags=0, device="cuda:0"):
        self.T, self.Ci, self.Co, self.dtype = T, Ci, Co, dtype
        self.L = 2 * T if flags & eq.EQL_FLAG_DIHEDRAL else T        # elements per group tuple
        self.dev = torch.device(device)
        self.td = torch_dtype(dtype)
        self.w = to_device(w, dtype, self.dev)
        self.bias = None if bias is None else to_device(bias, dtype, self.dev)
        self.ws_bytes = eq.eqlinear_workspace_bytes_flags(T, Ci, Co, eql_dtype(dtype), flags & eq.EQL_FLAG_DIHEDRAL)
        self.ws = torch.empty(self.ws_bytes + 256, dtype=torch.uint8, device=self.dev)
        assert self.ws.data_ptr() % 256 == 0
        self.stream = torch.cuda.current_stream(self.dev).cuda_stream
        self.plan = eq.eqlinear_plan(T, Ci, Co, eql_dtype(dtype), self.w, self.bias, self.ws, self.ws_bytes,
                                     flags, self.stream)

    def raw_status(self) -> int:
        """The plan's device status word (0 = ok, else the code of the wait that gave up)."""
        torch.cuda.synchronize(self.dev)
        return int(self.ws[:4].view(torch.int32).item())

    def close(self):
        if self.plan:
            torch.cuda.synchronize(self.dev)
            eq.eqlinear_plan_destroy(self.plan)
            self.plan = None

    def _out(self, rows, cols, dtype=None):
        """Output buffer with a canary tail; returns (flat buffer, view)."""
        dtype = dtype or self.td
        n = rows * cols
        buf = torch.full((n + CANARY,), -77.0, dtype=dtype, device=self.dev)
        return buf, buf[:n].view(rows, cols) if rows > 0 else buf[:0].view(0, cols)

    @staticmethod
    def _canary_ok(buf, n):
        return bool((buf[n:] == -77.0).all().item())

    def fwd(self, x_np):
        N = x_np.shape[0]
        x = to_device(x_np, self.dtype, self.dev)
        buf, y = self._out(N, self.Co * self.L)
        eq.eqlinear_fwd(self.plan, x if N else None, buf if N else None, N, self.stream)
        torch.cuda.synchronize(self.dev)
        assert self._canary_ok(buf, N * self.Co * self.L), "fwd wrote past its output"
        return to_host(y)

    def bwd_data(self, dy_np):
        N = dy_np.shape[0]
        dy = to_device(dy_np, self.dtype, self.dev)
        buf, dx = self._out(N, self.Ci * self.L)
        eq.eqlinear_bwd_data(self.plan, dy if N else None, buf if N else None, N, self.stream)
        torch.cuda.synchronize(self.dev)
        assert self._canary_ok(buf, N * self.Ci * self.L), "bwd_data wrote past its output"
        return to_host(dx)

    def bwd_weight(self, x_np, dy_np, want_db=True):
        N = x_np.shape[0]
        x = to_device(x_np, self.dtype, self.dev)
        dy = to_device(dy_np, self.dtype, self.dev)
        nw = self.Co * self.Ci * self.L
        wbuf, _ = self._out(1, nw, torch.float32)
        bbuf, _ = self._out(1, self.Co, torch.float32)
        sb = eq.eqlinear_bwd_weight_scratch_bytes(self.plan, N)
        scratch = torch.empty(sb + 256, dtype=torch.uint8, device=self.dev)
        eq.eqlinear_bwd_weight(self.plan, x if N else None, dy if N else None, wbuf, bbuf if want_db else None, N,
                               scratch, sb, self.stream)
        torch.cuda.synchronize(self.dev)
        assert self._canary_ok(wbuf, nw), "bwd_weight wrote past dw"
        assert self._canary_ok(bbuf, self.Co), "bwd_weight wrote past db"
        dw = wbuf[:nw].view(self.Co, self.Ci, self.L).cpu().numpy()
        db = bbuf[:self.Co].cpu().numpy() if want_db else None
        return dw, db


def check_workload(wl, passes=None, flags=0, data=None):
    """Runs the named passes on the GPU and returns {tensor: max|err|/max|ref|} against the oracle."""
    data = data or eq.workloads.generate(wl)
    passes = passes or wl.passes
    corr = bool(flags & eq.EQL_FLAG_CORRELATION)
    layer = GpuLayer(wl.T, wl.Ci, wl.Co, wl.dtype, data["w"], data["bias"], flags)
    errs = {}
    try:
        if "fwd" in passes:
            y = layer.fwd(data["x"])
            errs["y"] = rel_max_err(y, orc.fwd(data["x"], data["w"], data["bias"], corr))
        if "bwd_data" in passes:
            dx = layer.bwd_data(data["dy"])
            errs["dx"] = rel_max_err(dx, orc.bwd_data(data["dy"], data["w"], corr))
        if "bwd_weight" in passes:
            dw, db = layer.bwd_weight(data["x"], data["dy"])
            rdw, rdb = orc.bwd_weight(data["x"], data["dy"], wl.T, corr)
            errs["dw"] = rel_max_err(dw, rdw)
            errs["db"] = rel_max_err(db, rdb)
        assert eq.eqlinear_plan_device_status(layer.plan, layer.stream) == eq.binding.EQL_OK
    finally:
        layer.close()
    return errs
