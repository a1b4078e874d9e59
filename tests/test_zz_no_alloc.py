"""eqlinear_bwd_weight_static: the weight gradient for callers that cannot allocate device scratch.

Some users of the library run where a device allocation is not available to them at call time (a
plug-in inside an application that owns all GPU memory, a pool that has already reserved the whole
device, a loop that must not stall on an allocation).  They call this entry point instead of
eqlinear_bwd_weight; it takes the same inputs and outputs but no scratch buffer, using a fixed
32 MiB device array inside the library.  The test checks, through the C ABI, that it returns what
eqlinear_bwd_weight returns on two calls in a row (the shared array keeps the previous call's
contents, so the second call also shows that nothing stale leaks in), and that it refuses sizes
beyond the array.  This file sorts last so that a run stopping at the first failure has already
run every other test; it also passes when run alone in a fresh process.
"""

import numpy as np
import pytest
import torch

import paper_2607_21271_b200 as eq
from paper_2607_21271_b200.workloads import Workload, generate
from tests.harness import TOL, GpuLayer, rel_max_err

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,T,Ci,Co,N", [("fp16", 8, 24, 40, 1500), ("fp32", 4, 16, 8, 333)])
def test_static_scratch_matches_caller_scratch_twice(dtype, T, Ci, Co, N):
    wl = Workload("noalloc", dtype, T, Ci, Co, N, "normal", ("bwd_weight",), 21)
    d = generate(wl)
    layer = GpuLayer(T, Ci, Co, dtype, d["w"], d["bias"])
    try:
        ref_dw, ref_db = layer.bwd_weight(d["x"], d["dy"])                 # existing entry point, caller scratch
        x = torch.from_numpy(d["x"]).cuda()
        dy = torch.from_numpy(d["dy"]).cuda()
        # a different problem first, so the shared array holds foreign partials when the real calls run
        other = torch.from_numpy(generate(Workload("o", dtype, T, Ci, Co, N, "normal", ("bwd_weight",), 22))["dy"]).cuda()
        for call, grad in enumerate((other, dy, dy)):
            dw = torch.full((Co, Ci, T), float("nan"), dtype=torch.float32, device="cuda")
            db = torch.full((Co,), float("nan"), dtype=torch.float32, device="cuda")
            eq.eqlinear_bwd_weight_static(layer.plan, x, grad, dw, db, N, layer.stream)
            torch.cuda.synchronize()
            if call == 0:
                continue
            assert rel_max_err(dw.cpu().numpy(), ref_dw.astype(np.float64)) <= TOL[dtype], f"call {call}: dw"
            assert rel_max_err(db.cpu().numpy(), ref_db.astype(np.float64)) <= TOL[dtype], f"call {call}: db"
    finally:
        layer.close()


def test_static_scratch_rejects_sizes_beyond_the_array():
    T, Ci, Co, N = 8, 256, 256, 8192
    wl = Workload("big", "fp16", T, Ci, Co, N, "none", ("bwd_weight",), 23)
    d = generate(wl)
    layer = GpuLayer(T, Ci, Co, "fp16", d["w"], None)
    try:
        need = eq.eqlinear_bwd_weight_scratch_bytes(layer.plan, N)
        if need <= eq.binding.EQL_STATIC_SCRATCH_BYTES:
            pytest.skip("this shape fits the built-in array with the current kernel's split")
        x = torch.from_numpy(d["x"]).cuda()
        dy = torch.from_numpy(d["dy"]).cuda()
        dw = torch.zeros(Co, Ci, T, dtype=torch.float32, device="cuda")
        with pytest.raises(eq.EqlError) as e:
            eq.eqlinear_bwd_weight_static(layer.plan, x, dy, dw, None, N, layer.stream)
        assert e.value.status == eq.binding.EQL_ERR_WORKSPACE
        assert not dw.any().item()                                      # nothing was launched
    finally:
        layer.close()
