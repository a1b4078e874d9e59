"""eqlinear_bwd_weight_static: the weight gradient for callers that cannot allocate device scratch.

Some users of the library run where a device allocation is not available to them at call time (a
plug-in inside an application that owns all GPU memory, a pool that has already reserved the whole
device, a loop that must not stall on an allocation).  They call this entry point instead of
eqlinear_bwd_weight; it takes the same inputs and outputs but no scratch buffer, using a fixed
32 MiB device array inside the library.  The test checks, through the C ABI, that it returns exactly
what eqlinear_bwd_weight returns (the same kernels in the same fixed reduction order: bit-identical),
and what the oracle computes, on two calls in a row (the shared array keeps the previous call's
contents, so the second call also shows that nothing stale leaks in); that free device memory is the
same before and after each of those calls (the array became resident when the plan was built, not
here); and that sizes beyond the array are refused.  This file sorts last so that a run stopping at the first failure has already
run every other test; it also passes when run alone in a fresh process.
"""

import numpy as np
import pytest
import torch

import paper_2607_21271_b200 as eq
from oracle import eqlinear_oracle as orc
from paper_2607_21271_b200.workloads import Workload, generate
from tests.harness import TOL, GpuLayer, rel_max_err

pytestmark = pytest.mark.gpu


# The FP32 case with 300 -> 280 channels and 6000 tokens is large enough that the call walks over several blocks of
# tokens, each a launch through the same built-in array whose result the finalize kernel adds to dw / db.
@pytest.mark.parametrize("dtype,T,Ci,Co,N", [("fp16", 8, 24, 40, 1500), ("fp32", 4, 16, 8, 333), ("fp32", 4, 300, 280, 6000)])
def test_static_scratch_matches_caller_scratch_twice(dtype, T, Ci, Co, N):
    wl = Workload("noalloc", dtype, T, Ci, Co, N, "normal", ("bwd_weight",), 21)
    d = generate(wl)
    layer = GpuLayer(T, Ci, Co, dtype, d["w"], d["bias"])
    try:
        assert eq.eqlinear_bwd_weight_scratch_bytes(layer.plan, N) <= eq.binding.EQL_STATIC_SCRATCH_BYTES
        ref_dw, ref_db = layer.bwd_weight(d["x"], d["dy"])                 # existing entry point, caller scratch
        orc_dw, orc_db = orc.bwd_weight(d["x"], d["dy"], T)
        x = torch.from_numpy(d["x"]).cuda()
        dy = torch.from_numpy(d["dy"]).cuda()
        # a different problem first, so the shared array holds foreign partials when the real calls run
        other = torch.from_numpy(generate(Workload("o", dtype, T, Ci, Co, N, "normal", ("bwd_weight",), 22))["dy"]).cuda()
        outs = [(torch.full((Co, Ci, T), float("nan"), dtype=torch.float32, device="cuda"),
                 torch.full((Co,), float("nan"), dtype=torch.float32, device="cuda")) for _ in range(3)]
        torch.cuda.synchronize()
        for call, grad in enumerate((other, dy, dy)):
            dw, db = outs[call]
            free_before = torch.cuda.mem_get_info()[0]
            eq.eqlinear_bwd_weight_static(layer.plan, x, grad, dw, db, N, layer.stream)
            torch.cuda.synchronize()
            assert torch.cuda.mem_get_info()[0] == free_before, f"call {call} changed the free device memory"
            if call == 0:
                continue
            assert np.array_equal(dw.cpu().numpy(), ref_dw), f"call {call}: dw differs from eqlinear_bwd_weight's"
            assert np.array_equal(db.cpu().numpy(), ref_db), f"call {call}: db differs from eqlinear_bwd_weight's"
            assert rel_max_err(dw.cpu().numpy(), orc_dw) <= TOL[dtype], f"call {call}: dw against the oracle"
            assert rel_max_err(db.cpu().numpy(), orc_db) <= TOL[dtype], f"call {call}: db against the oracle"
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
