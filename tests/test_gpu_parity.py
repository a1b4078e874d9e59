"""GPU parity: the CUDA library (through its C ABI) against the float64 oracle, element by element.

Bars (max|gpu - ref| / max|ref| over the whole tensor): 1e-5 for FP32, 3e-3 for FP16 I/O with
float accumulation.
"""

import numpy as np
import pytest
import torch

import paper_2607_21271_b200 as eq
from oracle import eqlinear_oracle as orc
from paper_2607_21271_b200.workloads import BLOCK_SHAPES, CONFIGS, OPERATOR_SHAPES, Workload, generate, sample_rows
from tests.harness import TOL, GpuLayer, check_workload, rel_max_err

pytestmark = pytest.mark.gpu


# ------------------------------------------------------------------ the five configurations, full size
@pytest.mark.parametrize("name", list(CONFIGS))
def test_config_matches_oracle(name):
    wl = CONFIGS[name]
    errs = check_workload(wl)
    print(name, {k: f"{v:.2e}" for k, v in errs.items()})
    assert set(errs) >= {"y"}
    for k, v in errs.items():
        assert v <= TOL[wl.dtype], f"{name}: {k} error {v:.3e} above {TOL[wl.dtype]:.0e}"


@pytest.mark.parametrize("name", list(BLOCK_SHAPES))
def test_transformer_block_layers_match_oracle(name):
    """The fused q/k/v projection (one layer, 96 -> 3 x 96 channels: x is transformed once for the three blocks) and fc2
    (384 -> 96) of the EQ-ViT-B block, full size, every output against the oracle."""
    wl = BLOCK_SHAPES[name]
    for k, v in check_workload(wl).items():
        assert v <= TOL[wl.dtype], f"{name}: {k} error {v:.3e}"


def _gelu(a):
    from scipy.special import erf
    return 0.5 * a * (1.0 + erf(a / np.sqrt(2.0)))


@pytest.mark.parametrize("dtype,T,Ci,Co,N,flags,kernel", [
    ("fp16", 8, 96, 384, 1500, 0, 2),                                        # resident-activation kernel (fc1 -> GELU)
    ("fp16", 8, 96, 384, 1500, eq.EQL_FLAG_FORCE_STREAMING, 1),              # streaming kernel
    ("fp16", 4, 64, 200, 777, eq.EQL_FLAG_FORCE_STREAMING | eq.EQL_FLAG_CTA_PAIR, 3),   # its CTA-pair form
    ("fp16", 16, 17, 33, 333, 0, 1),
    ("fp32", 8, 48, 48, 1000, 0, 1),                                         # 3xTF32
    ("fp16", 2, 40, 300, 333, 0, 1),                                        # T = 2 on the streaming kernel
    ("fp32", 5, 8, 24, 333, 0, 0), ("fp16", 2, 8, 16, 333, eq.EQL_FLAG_FORCE_SIMT, 0),   # CUDA-core kernels
])
def test_fused_gelu_epilogue(dtype, T, Ci, Co, N, flags, kernel):
    """EQL_FLAG_GELU: the forward pass returns GELU(layer(x)), applied in FP32 before the one rounding of the output;
    the gradients of a plan built with the flag remain those of the linear layer."""
    wl = Workload("gelu", dtype, T, Ci, Co, N, "normal", ("fwd", "bwd_data"), 33)
    d = generate(wl)
    layer = GpuLayer(T, Ci, Co, dtype, d["w"], d["bias"], flags | eq.EQL_FLAG_GELU)
    try:
        assert eq.eqlinear_plan_info(layer.plan).fwd_kernel == kernel
        y = layer.fwd(d["x"])
        dx = layer.bwd_data(d["dy"])
        assert layer.raw_status() == 0
    finally:
        layer.close()
    assert rel_max_err(y, _gelu(orc.fwd(d["x"], d["w"], d["bias"]))) <= TOL[dtype]
    assert rel_max_err(dx, orc.bwd_data(d["dy"], d["w"])) <= TOL[dtype]


# ------------------------------------------------------------------ bfloat16 I/O
@pytest.mark.parametrize("T,Ci,Co,N,flags,kernels", [
    (8, 96, 384, 1500, 0, (2, 2, 1)),                                         # resident activations / ring mode / tcgen05 dW
    (4, 24, 96, 1111, 0, (2, 1, 1)),
    (8, 96, 384, 1000, eq.EQL_FLAG_FORCE_STREAMING, (1, 1, 1)),               # streaming kernel
    (4, 100, 130, 515, eq.EQL_FLAG_FORCE_STREAMING | eq.EQL_FLAG_CTA_PAIR, (3, 3, 1)),   # CTA pairs
    (16, 17, 33, 333, 0, (1, 1, 1)), (32, 32, 32, 500, 0, (1, 1, 1)),
    (2, 8, 16, 333, 0, (1, 1, 0)), (2, 72, 264, 1000, 0, (1, 1, 0)),          # T = 2: streaming kernel, CUDA-core weight gradient
    (5, 8, 24, 333, 0, (0, 0, 0)),                                            # CUDA-core kernels
])
def test_bf16_matches_oracle(T, Ci, Co, N, flags, kernels):
    """EQL_BF16: bfloat16 inputs and outputs, float accumulation -- every pass of every kernel family against the oracle
    fed the same bfloat16-representable values.  The bar is derived in tests/harness.py (6 unit roundoffs, as for FP16)."""
    wl = Workload("bf16", "bf16", T, Ci, Co, N, "normal", ("fwd", "bwd_data", "bwd_weight"), 35)
    d = generate(wl)
    layer = GpuLayer(T, Ci, Co, "bf16", d["w"], d["bias"], flags)
    try:
        info = eq.eqlinear_plan_info(layer.plan)
        assert (info.fwd_kernel, info.bwd_data_kernel, info.bwd_weight_kernel) == kernels
        saved = {}
        if info.bwd_weight_kernel == 1:                                       # training with a saved spectrum, in bfloat16
            x = torch.from_numpy(d["x"]).cuda().to(torch.bfloat16)
            dy = torch.from_numpy(d["dy"]).cuda().to(torch.bfloat16)
            sb = eq.eqlinear_spectrum_bytes(layer.plan, N)
            spec = torch.full((sb + 64,), 0x7F, dtype=torch.uint8, device="cuda")
            y = torch.empty(N, Co * T, dtype=torch.bfloat16, device="cuda")
            eq.eqlinear_fwd_save_spectrum(layer.plan, x, y, N, spec, sb, layer.stream)
            scb = eq.eqlinear_bwd_weight_scratch_bytes(layer.plan, N)
            sc = torch.empty(scb, dtype=torch.uint8, device="cuda")
            dw = torch.full((Co, Ci, T), float("nan"), dtype=torch.float32, device="cuda")
            db = torch.full((Co,), float("nan"), dtype=torch.float32, device="cuda")
            eq.eqlinear_bwd_weight_from_spectrum(layer.plan, spec, sb, dy, dw, db, N, sc, scb, layer.stream)
            assert layer.raw_status() == 0
            assert bool((spec[sb:] == 0x7F).all().item())
            rdw, rdb = orc.bwd_weight(d["x"], d["dy"], T)
            saved = {"y_saved": rel_max_err(y.float().cpu().numpy(), orc.fwd(d["x"], d["w"], d["bias"])),
                     "dw_saved": rel_max_err(dw.cpu().numpy(), rdw), "db_saved": rel_max_err(db.cpu().numpy(), rdb)}
        else:
            with pytest.raises(eq.EqlError) as e:                             # no saved-spectrum path behind CUDA-core kernels
                eq.eqlinear_spectrum_bytes(layer.plan, N)
            assert e.value.status == eq.binding.EQL_ERR_UNSUPPORTED
    finally:
        layer.close()
    errs = {**check_workload(wl, flags=flags, data=d), **saved}
    print({k: f"{v:.2e}" for k, v in errs.items()})
    for k, v in errs.items():
        assert v <= TOL["bf16"], f"T={T} Ci={Ci} Co={Co} N={N} flags={flags}: {k} error {v:.3e}"


def test_bf16_full_size_headline_shape_with_gelu():
    """The headline layer's shape in bfloat16 at full size, forward with the fused GELU, data and weight gradients."""
    wl = Workload("bf16_fc1", "bf16", 8, 96, 384, 128 * 197, "normal", ("fwd", "bwd_data", "bwd_weight"), 36)
    d = generate(wl)
    errs = check_workload(wl, passes=("bwd_data", "bwd_weight"), data=d)
    layer = GpuLayer(wl.T, wl.Ci, wl.Co, "bf16", d["w"], d["bias"], eq.EQL_FLAG_GELU)
    try:
        errs["gelu(y)"] = rel_max_err(layer.fwd(d["x"]), _gelu(orc.fwd(d["x"], d["w"], d["bias"])))
        assert layer.raw_status() == 0
    finally:
        layer.close()
    print({k: f"{v:.2e}" for k, v in errs.items()})
    for k, v in errs.items():
        assert v <= TOL["bf16"], f"{k} error {v:.3e}"


def test_fused_gelu_is_refused_where_the_forward_sum_is_split():
    """FP32 plans on the tensor cores with more than 256 input channels add segments of the reduction in global memory:
    no place to apply an activation to the finished sum."""
    wl = Workload("gelu", "fp32", 4, 300, 16, 64, "normal", ("fwd",), 34)
    d = generate(wl)
    with pytest.raises(eq.EqlError) as e:
        GpuLayer(wl.T, wl.Ci, wl.Co, "fp32", d["w"], d["bias"], eq.EQL_FLAG_GELU)
    assert e.value.status == eq.binding.EQL_ERR_UNSUPPORTED


def test_repeated_full_size_runs_are_identical():
    """Races in the multi-stage pipelines show up as rare corrupted rows: at the headline size (eight work
    units per SM) every pass must return bit-identical results on every repetition, and match the oracle."""
    wl = CONFIGS["vit_b_fc1_fp16"]
    d = generate(wl)
    layer = GpuLayer(wl.T, wl.Ci, wl.Co, wl.dtype, d["w"], d["bias"])
    try:
        y0, dx0 = layer.fwd(d["x"]), layer.bwd_data(d["dy"])
        dw0, db0 = layer.bwd_weight(d["x"], d["dy"])
        assert rel_max_err(y0, orc.fwd(d["x"], d["w"], d["bias"])) <= TOL["fp16"]
        assert rel_max_err(dx0, orc.bwd_data(d["dy"], d["w"])) <= TOL["fp16"]
        for _ in range(6):
            assert np.array_equal(layer.fwd(d["x"]), y0)
            assert np.array_equal(layer.bwd_data(d["dy"]), dx0)
            dw, db = layer.bwd_weight(d["x"], d["dy"])
            assert np.array_equal(dw, dw0) and np.array_equal(db, db0)
    finally:
        layer.close()


# ------------------------------------------------------------------ ragged token counts, several tiles
@pytest.mark.parametrize("dtype", ["fp32", "fp16"])
@pytest.mark.parametrize("N", [1, 2, 127, 128, 129, 197, 1000])
def test_ragged_token_counts(dtype, N):
    wl = Workload(f"ragged{N}", dtype, 8, 24, 40, N, "normal", ("fwd", "bwd_data", "bwd_weight"), 11)
    for k, v in check_workload(wl).items():
        assert v <= TOL[dtype], f"N={N} {dtype}: {k} error {v:.3e}"


@pytest.mark.parametrize("dtype", ["fp32", "fp16"])
@pytest.mark.parametrize("T,Ci,Co", [(2, 8, 16), (4, 64, 64), (4, 6, 10), (8, 96, 384), (8, 384, 96),
                                       (16, 17, 33), (32, 32, 32), (32, 5, 3), (2, 136, 520),
                                       # Algorithm 1 for other cyclic groups: odd and non-power-of-two orders, and the trivial group
                                       (1, 16, 8), (3, 8, 16), (5, 8, 24), (6, 12, 20), (7, 8, 8), (12, 10, 6)])
def test_shapes(dtype, T, Ci, Co):
    wl = Workload("shape", dtype, T, Ci, Co, 333, "normal", ("fwd", "bwd_data", "bwd_weight"), 12)
    for k, v in check_workload(wl).items():
        assert v <= TOL[dtype], f"T={T} Ci={Ci} Co={Co} {dtype}: {k} error {v:.3e}"


@pytest.mark.parametrize("T,Ci,Co,N", [(8, 162, 254, 9473), (8, 297, 219, 4099), (4, 300, 280, 6000), (8, 380, 40, 2049),
                                         (4, 512, 520, 1500), (4, 1040, 72, 700)])
def test_fp32_long_reductions_stay_inside_the_bar(T, Ci, Co, N):
    """FP32 plans on the tensor cores: the accumulator adds with truncation, so the error grows with the number of
    accumulation steps.  Layers with many channel tiles leave few CTAs per tile, i.e. long token ranges per
    accumulator (weight gradient), and wide layers have long channel reductions (forward, data gradient: run as
    segments of at most 256 channels whose results are added in global memory); both must stay inside the FP32 bar
    (these shapes measured 1.8e-5 ... 3.8e-5 on dw before the token range was bounded)."""
    wl = Workload("fp32long", "fp32", T, Ci, Co, N, "none", ("fwd", "bwd_data", "bwd_weight"), 31)
    for k, v in check_workload(wl).items():
        assert v <= 0.6 * TOL["fp32"], f"T={T} Ci={Ci} Co={Co} N={N}: {k} error {v:.3e}"


# ------------------------------------------------------------------ the paper's operator-benchmark shapes (Tables 1-2)
@pytest.mark.parametrize("name", ["op_c16_fp16", "op_c64_fp16", "op_c256_fp16", "op_c512_fp16", "op_c1024_fp16", "op_c2048_fp16",
                                  "op_c16_fp32", "op_c64_fp32", "op_c256_fp32", "op_c512_fp32"])
def test_operator_benchmark_shapes_on_sampled_outputs(name):
    """32 x 1024 tokens, T = 4, c channels per group element on both sides: the GPU runs the full size; the oracle
    computes a sample of it one piece at a time - sampled token rows x sampled output channels of y (the dense weight
    of those channels only), sampled rows x sampled input channels of dx, and dw for sampled channel pairs over ALL
    tokens (dw[o, i, :] depends only on channel i of x and channel o of dy)."""
    wl = OPERATOR_SHAPES[name]
    d = generate(wl)
    T, c, N = wl.T, wl.Ci, wl.N
    rows = sample_rows(N, 96, seed=1)
    g = np.random.Generator(np.random.PCG64(77))
    ch = np.unique(np.concatenate([[0, c - 1], g.choice(c, size=min(c, 10) - 2, replace=False)]))
    cols = (ch[:, None] * T + np.arange(T)[None, :]).reshape(-1)
    layer = GpuLayer(T, c, c, wl.dtype, d["w"], d["bias"])
    try:
        y = layer.fwd(d["x"])
        dx = layer.bwd_data(d["dy"])
        dw, db = layer.bwd_weight(d["x"], d["dy"])
        assert layer.raw_status() == 0
    finally:
        layer.close()
    tol = TOL[wl.dtype]
    ry = orc.fwd(d["x"][rows], d["w"][ch], d["bias"][ch])                    # [rows, sampled output channels x T]
    assert rel_max_err(y[rows][:, cols], ry) <= tol
    rdx = orc.bwd_data(d["dy"][rows], d["w"][:, ch])                         # [rows, sampled input channels x T]
    assert rel_max_err(dx[rows][:, cols], rdx) <= tol
    rdw, rdb = orc.bwd_weight(d["x"][:, cols], d["dy"][:, cols], T)          # [sampled o, sampled i, T], all tokens
    assert rel_max_err(dw[np.ix_(ch, ch)], rdw) <= tol
    assert rel_max_err(db[ch], rdb) <= tol


# ------------------------------------------------------------------ the two tensor-core kernels of fwd / bwd_data
@pytest.mark.parametrize("T,Ci,Co,N,ids", [(8, 96, 384, 1000, (2, 2)), (8, 24, 200, 777, (2, 1)), (8, 10, 64, 130, (2, 1)),
                                             (8, 16, 520, 6500, (2, 1)), (8, 64, 64, 900, (2, 2)), (4, 24, 96, 1111, (2, 1)),
                                             (4, 100, 130, 515, (2, 2)), (4, 8, 300, 20000, (2, 1)),
                                             (8, 384, 96, 12000, (2, 2)), (4, 320, 100, 600, (2, 2)), (8, 200, 100, 3333, (2, 1))])
def test_resident_and_streaming_kernels_agree_with_oracle(T, Ci, Co, N, ids):
    """Layers with few input channels run the kernel that keeps a token tile's spectrum in shared memory (id 2), and so
    do layers with at most 128 output channels (one channel tile: the spectrum then streams through a ring of three
    chunk buffers, e.g. 384 -> 96 channels); EQL_FLAG_FORCE_STREAMING selects the streaming kernel (id 1) for the same
    plan shape, and EQL_FLAG_CTA_PAIR on top of it the streaming kernel's CTA-pair form (id 3: two CTAs, one
    tcgen05.mma.cta_group::2 over both).  All must meet the bar, on channel counts that are not multiples of the
    128-channel / 16-channel tiles, ragged token counts, odd numbers of token tiles (a pair's second CTA then has no
    rows), and token counts large enough that a CTA's range of work starts and ends in the middle of a token tile and
    covers several units.  The pair form computes the same products in the same order as the single-CTA form: its
    results must be bit-identical to it."""
    wl = Workload("res", "fp16", T, Ci, Co, N, "normal", ("fwd", "bwd_data"), 21)
    data = eq.workloads.generate(wl)
    outs = {}
    for flags, want in ((0, ids), (eq.EQL_FLAG_FORCE_STREAMING, (1, 1)),   # (narrow layers: no pair form by default)
                        (eq.EQL_FLAG_FORCE_STREAMING | eq.EQL_FLAG_CTA_PAIR, (3, 3))):
        layer = GpuLayer(T, Ci, Co, "fp16", data["w"], data["bias"], flags)
        try:
            info = eq.eqlinear_plan_info(layer.plan)
            assert (info.fwd_kernel, info.bwd_data_kernel) == want
            outs[flags] = (layer.fwd(data["x"]), layer.bwd_data(data["dy"]))
            assert layer.raw_status() == 0
        finally:
            layer.close()
        for k, v in check_workload(wl, flags=flags, data=data).items():
            assert v <= TOL["fp16"], f"T={T} Ci={Ci} Co={Co} N={N} flags={flags}: {k} error {v:.3e}"
    single, pair = outs[eq.EQL_FLAG_FORCE_STREAMING], outs[eq.EQL_FLAG_FORCE_STREAMING | eq.EQL_FLAG_CTA_PAIR]
    assert np.array_equal(single[0], pair[0]) and np.array_equal(single[1], pair[1])


def test_cta_pair_form_at_full_size_is_repeatable():
    """A wide layer at full size (32 x 1024 tokens, 512 -> 512 channels, T = 4): the plan takes the CTA-pair form by
    itself (id 3).  Sampled outputs against the oracle, bit-identical results on every repetition (a race between the two
    CTAs of a pair would show up as rare corrupted rows), and bit-identical to the single-CTA form
    (EQL_FLAG_NO_CTA_PAIR, id 1)."""
    wl = OPERATOR_SHAPES["op_c512_fp16"]
    d = generate(wl)
    rows = sample_rows(wl.N, 64, seed=5)
    layer = GpuLayer(wl.T, wl.Ci, wl.Co, "fp16", d["w"], d["bias"])
    try:
        info = eq.eqlinear_plan_info(layer.plan)
        assert (info.fwd_kernel, info.bwd_data_kernel) == (3, 3)
        y0, dx0 = layer.fwd(d["x"]), layer.bwd_data(d["dy"])
        assert rel_max_err(y0[rows], orc.fwd(d["x"][rows], d["w"], d["bias"])) <= TOL["fp16"]
        assert rel_max_err(dx0[rows], orc.bwd_data(d["dy"][rows], d["w"])) <= TOL["fp16"]
        for _ in range(4):
            assert np.array_equal(layer.fwd(d["x"]), y0)
            assert np.array_equal(layer.bwd_data(d["dy"]), dx0)
        assert layer.raw_status() == 0
    finally:
        layer.close()
    layer = GpuLayer(wl.T, wl.Ci, wl.Co, "fp16", d["w"], d["bias"], eq.EQL_FLAG_NO_CTA_PAIR)
    try:
        info = eq.eqlinear_plan_info(layer.plan)
        assert (info.fwd_kernel, info.bwd_data_kernel) == (1, 1)
        assert np.array_equal(layer.fwd(d["x"]), y0) and np.array_equal(layer.bwd_data(d["dy"]), dx0)
    finally:
        layer.close()


# ------------------------------------------------------------------ training with a saved spectrum
@pytest.mark.parametrize("T,Ci,Co,N", [(8, 96, 384, 1000), (8, 96, 384, 12000), (8, 10, 24, 77), (4, 24, 96, 1111),
                                         (4, 256, 256, 700), (8, 384, 96, 640), (16, 17, 33, 333), (32, 32, 32, 500)])
def test_saved_spectrum_path_matches_oracle(T, Ci, Co, N):
    """eqlinear_fwd_save_spectrum + eqlinear_bwd_weight_from_spectrum: the forward result and the weight gradient
    computed from the saved spectrum of x meet the same bars as the plain calls.  The shapes cover the forward kernel
    that writes the spectrum itself (resident and ring mode), the pre-pass fallback behind the streaming kernel,
    token counts that are not multiples of the 16-token chunk, and channel counts that are not multiples of a tile."""
    wl = Workload("spec", "fp16", T, Ci, Co, N, "normal", ("fwd", "bwd_weight"), 23)
    d = generate(wl)
    layer = GpuLayer(T, Ci, Co, "fp16", d["w"], d["bias"])
    try:
        x = torch.from_numpy(d["x"]).cuda()
        dy = torch.from_numpy(d["dy"]).cuda()
        sb = eq.eqlinear_spectrum_bytes(layer.plan, N)
        spec = torch.full((sb + 64,), 0x7F, dtype=torch.uint8, device="cuda")       # NaN pattern: nothing stale may be read
        y = torch.empty(N, Co * T, dtype=torch.float16, device="cuda")
        eq.eqlinear_fwd_save_spectrum(layer.plan, x, y, N, spec, sb, layer.stream)
        scb = eq.eqlinear_bwd_weight_scratch_bytes(layer.plan, N)
        sc = torch.empty(scb, dtype=torch.uint8, device="cuda")
        outs = []
        for _ in range(2):                                                          # twice: bit-identical results
            dw = torch.full((Co, Ci, T), float("nan"), dtype=torch.float32, device="cuda")
            db = torch.full((Co,), float("nan"), dtype=torch.float32, device="cuda")
            eq.eqlinear_bwd_weight_from_spectrum(layer.plan, spec, sb, dy, dw, db, N, sc, scb, layer.stream)
            torch.cuda.synchronize()
            outs.append((dw.cpu().numpy(), db.cpu().numpy()))
        assert layer.raw_status() == 0
        assert bool((spec[sb:] == 0x7F).all().item()), "the spectrum write went past its buffer"
        assert rel_max_err(y.cpu().numpy(), orc.fwd(d["x"], d["w"], d["bias"])) <= TOL["fp16"]
        rdw, rdb = orc.bwd_weight(d["x"], d["dy"], T)
        assert rel_max_err(outs[0][0], rdw) <= TOL["fp16"]
        assert rel_max_err(outs[0][1], rdb) <= TOL["fp16"]
        assert np.array_equal(outs[0][0], outs[1][0]) and np.array_equal(outs[0][1], outs[1][1])
    finally:
        layer.close()


def test_benchmarked_step_sequence_at_full_size():
    """The call sequence bench.py times on the headline workload, at its full size (N = 25 216): eqlinear_fwd_save_spectrum,
    eqlinear_bwd_data, eqlinear_bwd_weight_from_spectrum, every output against the oracle."""
    wl = CONFIGS["vit_b_fc1_fp16"]
    d = generate(wl)
    T, Ci, Co, N = wl.T, wl.Ci, wl.Co, wl.N
    layer = GpuLayer(T, Ci, Co, "fp16", d["w"], d["bias"])
    try:
        info = eq.eqlinear_plan_info(layer.plan)
        assert (info.fwd_kernel, info.bwd_data_kernel, info.bwd_weight_kernel) == (2, 2, 1)
        x, dy = torch.from_numpy(d["x"]).cuda(), torch.from_numpy(d["dy"]).cuda()
        sb = eq.eqlinear_spectrum_bytes(layer.plan, N)
        spec = torch.full((sb + 64,), 0x7F, dtype=torch.uint8, device="cuda")
        y = torch.empty(N, Co * T, dtype=torch.float16, device="cuda")
        dx = torch.empty(N, Ci * T, dtype=torch.float16, device="cuda")
        dw = torch.full((Co, Ci, T), float("nan"), dtype=torch.float32, device="cuda")
        db = torch.full((Co,), float("nan"), dtype=torch.float32, device="cuda")
        scb = eq.eqlinear_bwd_weight_scratch_bytes(layer.plan, N)
        sc = torch.empty(scb, dtype=torch.uint8, device="cuda")
        eq.eqlinear_fwd_save_spectrum(layer.plan, x, y, N, spec, sb, layer.stream)
        eq.eqlinear_bwd_data(layer.plan, dy, dx, N, layer.stream)
        eq.eqlinear_bwd_weight_from_spectrum(layer.plan, spec, sb, dy, dw, db, N, sc, scb, layer.stream)
        assert layer.raw_status() == 0
        assert bool((spec[sb:] == 0x7F).all().item())
        rdw, rdb = orc.bwd_weight(d["x"], d["dy"], T)
        errs = {"y": rel_max_err(y.cpu().numpy(), orc.fwd(d["x"], d["w"], d["bias"])),
                "dx": rel_max_err(dx.cpu().numpy(), orc.bwd_data(d["dy"], d["w"])),
                "dw": rel_max_err(dw.cpu().numpy(), rdw), "db": rel_max_err(db.cpu().numpy(), rdb)}
        print({k: f"{v:.2e}" for k, v in errs.items()})
        for k, v in errs.items():
            assert v <= TOL["fp16"], f"{k} error {v:.3e}"
    finally:
        layer.close()


def test_saved_spectrum_argument_errors():
    d = generate(Workload("spec", "fp32", 8, 16, 16, 64, "normal", ("fwd",), 24))
    layer = GpuLayer(8, 16, 16, "fp32", d["w"], d["bias"])
    try:
        with pytest.raises(eq.EqlError) as e:                                        # FP32 plans have no such path
            eq.eqlinear_spectrum_bytes(layer.plan, 64)
        assert e.value.status == eq.binding.EQL_ERR_UNSUPPORTED
    finally:
        layer.close()
    d = generate(Workload("spec", "fp16", 8, 16, 16, 64, "normal", ("fwd",), 24))
    layer = GpuLayer(8, 16, 16, "fp16", d["w"], d["bias"])
    try:
        x = torch.from_numpy(d["x"]).cuda()
        y = torch.empty(64, 128, dtype=torch.float16, device="cuda")
        sb = eq.eqlinear_spectrum_bytes(layer.plan, 64)
        spec = torch.empty(sb, dtype=torch.uint8, device="cuda")
        with pytest.raises(eq.EqlError) as e:                                        # buffer too small
            eq.eqlinear_fwd_save_spectrum(layer.plan, x, y, 64, spec, sb - 1, layer.stream)
        assert e.value.status == eq.binding.EQL_ERR_WORKSPACE
        eq.eqlinear_fwd_save_spectrum(layer.plan, x, y, 0, None, 0, layer.stream)   # N = 0: no-op
        dw = torch.full((16, 16, 8), 1.0, dtype=torch.float32, device="cuda")
        eq.eqlinear_bwd_weight_from_spectrum(layer.plan, None, 0, None, dw, None, 0, None, 0, layer.stream)
        torch.cuda.synchronize()
        assert float(dw.abs().max().item()) == 0.0                                   # N = 0: gradients are zero
    finally:
        layer.close()


@pytest.mark.parametrize("dtype", ["fp32", "fp16"])
def test_paper_parity_shape(dtype):
    """The shape of the paper's numerical-equivalence table (Table 4): (B, N, c, T) = (32, 1024, 64, 4)."""
    wl = Workload("table4", dtype, 4, 64, 64, 32 * 1024, "normal", ("fwd", "bwd_data", "bwd_weight"), 13)
    for k, v in check_workload(wl).items():
        assert v <= TOL[dtype], f"{k} error {v:.3e}"


@pytest.mark.parametrize("dtype", ["fp32", "fp16"])
@pytest.mark.parametrize("T", [8, 5, 6])
def test_correlation_flag_and_no_bias(dtype, T):
    wl = Workload("corr", dtype, T, 16, 24, 300, "none", ("fwd", "bwd_data", "bwd_weight"), 14)
    for k, v in check_workload(wl, flags=eq.EQL_FLAG_CORRELATION).items():
        assert v <= TOL[dtype], f"{k} error {v:.3e}"


# ------------------------------------------------------------------ plan life cycle
def test_empty_batch_and_repeated_calls_and_set_weight():
    wl = Workload("life", "fp32", 4, 8, 12, 200, "normal", ("fwd",), 15)
    d = generate(wl)
    layer = GpuLayer(wl.T, wl.Ci, wl.Co, wl.dtype, d["w"], d["bias"])
    try:
        # N = 0 is a no-op / zero gradients
        assert layer.fwd(d["x"][:0]).shape == (0, wl.Co * wl.T)
        dw0, db0 = layer.bwd_weight(d["x"][:0], d["dy"][:0])
        assert not dw0.any() and not db0.any()
        ref = orc.fwd(d["x"], d["w"], d["bias"])
        y1, y2 = layer.fwd(d["x"]), layer.fwd(d["x"])
        assert np.array_equal(y1, y2)
        assert rel_max_err(y1, ref) <= TOL["fp32"]
        # new parameter values through set_weight
        w2 = (d["w"] * 0.5 + 0.25).astype(np.float32)
        b2 = (d["bias"] - 1.0).astype(np.float32)
        w2_t, b2_t = torch.from_numpy(w2).cuda(), torch.from_numpy(b2).cuda()
        eq.eqlinear_plan_set_weight(layer.plan, w2_t, b2_t, layer.stream)
        assert rel_max_err(layer.fwd(d["x"]), orc.fwd(d["x"], w2, b2)) <= TOL["fp32"]
        assert rel_max_err(layer.bwd_data(d["dy"]), orc.bwd_data(d["dy"], w2)) <= TOL["fp32"]
        # weight gradient is bit-reproducible (fixed reduction order)
        a, _ = layer.bwd_weight(d["x"], d["dy"])
        b, _ = layer.bwd_weight(d["x"], d["dy"])
        assert np.array_equal(a, b)
        # db may be omitted
        dw, db = layer.bwd_weight(d["x"], d["dy"], want_db=False)
        assert db is None and np.array_equal(dw, a)
    finally:
        layer.close()


def test_two_plans_interleaved_on_one_stream():
    wa = Workload("a", "fp16", 4, 24, 96, 500, "normal", ("fwd",), 16)
    wb = Workload("b", "fp32", 8, 48, 48, 300, "normal", ("fwd",), 17)
    da, db_ = generate(wa), generate(wb)
    la = GpuLayer(wa.T, wa.Ci, wa.Co, wa.dtype, da["w"], da["bias"])
    lb = GpuLayer(wb.T, wb.Ci, wb.Co, wb.dtype, db_["w"], db_["bias"])
    try:
        ya1 = la.fwd(da["x"]); yb1 = lb.fwd(db_["x"]); ya2 = la.fwd(da["x"])
        assert np.array_equal(ya1, ya2)
        assert rel_max_err(ya1, orc.fwd(da["x"], da["w"], da["bias"])) <= TOL["fp16"]
        assert rel_max_err(yb1, orc.fwd(db_["x"], db_["w"], db_["bias"])) <= TOL["fp32"]
    finally:
        la.close(); lb.close()


def test_runtime_argument_errors():
    wl = Workload("err", "fp32", 4, 8, 8, 16, "none", ("fwd",), 18)
    d = generate(wl)
    layer = GpuLayer(wl.T, wl.Ci, wl.Co, wl.dtype, d["w"], None)
    lib = eq.load_library()
    B = eq.binding
    try:
        x = torch.zeros(16 * 32 + 4, dtype=torch.float32, device="cuda")
        y = torch.zeros(16 * 32 + 4, dtype=torch.float32, device="cuda")
        p = layer.plan
        assert lib.eqlinear_fwd(p, x.data_ptr(), y.data_ptr(), -1, None) == B.EQL_ERR_INVALID_ARG
        assert lib.eqlinear_fwd(p, None, y.data_ptr(), 4, None) == B.EQL_ERR_INVALID_ARG
        assert lib.eqlinear_fwd(p, x.data_ptr(), x.data_ptr(), 4, None) == B.EQL_ERR_INVALID_ARG
        assert lib.eqlinear_fwd(p, x.data_ptr() + 4, y.data_ptr(), 4, None) == B.EQL_ERR_ALIGNMENT
        assert lib.eqlinear_bwd_data(p, x.data_ptr(), y.data_ptr() + 8, 4, None) == B.EQL_ERR_ALIGNMENT
        dw = torch.zeros(8 * 8 * 4, dtype=torch.float32, device="cuda")
        sc = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
        assert lib.eqlinear_bwd_weight(p, x.data_ptr(), y.data_ptr(), dw.data_ptr(), None, 16, sc.data_ptr(), 8,
                                       None) == B.EQL_ERR_WORKSPACE
        assert lib.eqlinear_plan_set_weight(p, layer.w.data_ptr(), layer.w.data_ptr(), None) == B.EQL_ERR_INVALID_ARG
        info = eq.eqlinear_plan_info(p)
        assert (info.T, info.C_in, info.C_out) == (4, 8, 8)
        assert info.macs_per_token == 6 * 8 * 8 and info.dense_macs_per_token == 32 * 32
        assert info.bytes_per_token_fwd == (8 + 8) * 4 * 4
    finally:
        layer.close()


def test_plan_on_a_second_stream():
    """A plan is not tied to the stream it was built on: built on one stream (the build is ordered before later use by a
    stream synchronisation here), then used from another non-default stream, with results equal bit for bit to those on
    the first."""
    wl = Workload("stream", "fp16", 8, 96, 200, 3000, "normal", ("fwd", "bwd_data", "bwd_weight"), 29)
    d = generate(wl)
    layer = GpuLayer(wl.T, wl.Ci, wl.Co, wl.dtype, d["w"], d["bias"])
    try:
        y0, dx0 = layer.fwd(d["x"]), layer.bwd_data(d["dy"])
        dw0, db0 = layer.bwd_weight(d["x"], d["dy"])
        torch.cuda.synchronize()
        side = torch.cuda.Stream()
        x, dy = torch.from_numpy(d["x"]).cuda(), torch.from_numpy(d["dy"]).cuda()
        y = torch.empty(wl.N, wl.Dout, dtype=torch.float16, device="cuda")
        dx = torch.empty(wl.N, wl.Din, dtype=torch.float16, device="cuda")
        dw = torch.empty(wl.Co, wl.Ci, wl.T, dtype=torch.float32, device="cuda")
        db = torch.empty(wl.Co, dtype=torch.float32, device="cuda")
        sb = eq.eqlinear_bwd_weight_scratch_bytes(layer.plan, wl.N)
        sc = torch.empty(sb, dtype=torch.uint8, device="cuda")
        torch.cuda.synchronize()
        with torch.cuda.stream(side):
            s = side.cuda_stream
            eq.eqlinear_fwd(layer.plan, x, y, wl.N, s)
            eq.eqlinear_bwd_data(layer.plan, dy, dx, wl.N, s)
            eq.eqlinear_bwd_weight(layer.plan, x, dy, dw, db, wl.N, sc, sb, s)
            assert eq.eqlinear_plan_device_status(layer.plan, s) == eq.binding.EQL_OK
        side.synchronize()
        assert np.array_equal(y.cpu().numpy(), y0) and np.array_equal(dx.cpu().numpy(), dx0)
        assert np.array_equal(dw.cpu().numpy(), dw0) and np.array_equal(db.cpu().numpy(), db0)
        assert rel_max_err(y0, orc.fwd(d["x"], d["w"], d["bias"])) <= TOL["fp16"]
    finally:
        layer.close()


def test_plan_is_refused_on_another_device():
    """A plan's workspace and tensor maps belong to the GPU it was built on: with another device current every entry
    point that takes the plan must return EQL_ERR_INVALID_ARG before launching anything (needs two GPUs)."""
    if torch.cuda.device_count() < 2:
        pytest.skip("needs a second GPU to make another device current")
    wl = Workload("dev", "fp16", 8, 24, 40, 64, "normal", ("fwd",), 28)
    d = generate(wl)
    layer = GpuLayer(wl.T, wl.Ci, wl.Co, wl.dtype, d["w"], d["bias"])
    lib, B = eq.load_library(), eq.binding
    try:
        x = torch.zeros(64, wl.Din, dtype=torch.float16, device="cuda:0")
        y = torch.full((64, wl.Dout), -5.0, dtype=torch.float16, device="cuda:0")
        dw = torch.zeros(wl.Co * wl.Ci * wl.T, dtype=torch.float32, device="cuda:0")
        sc = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda:0")
        p = layer.plan
        with torch.cuda.device(1):
            assert lib.eqlinear_fwd(p, x.data_ptr(), y.data_ptr(), 64, None) == B.EQL_ERR_INVALID_ARG
            assert lib.eqlinear_bwd_data(p, y.data_ptr(), x.data_ptr(), 64, None) == B.EQL_ERR_INVALID_ARG
            assert lib.eqlinear_bwd_weight(p, x.data_ptr(), y.data_ptr(), dw.data_ptr(), None, 64, sc.data_ptr(), 1 << 20,
                                           None) == B.EQL_ERR_INVALID_ARG
            assert lib.eqlinear_bwd_weight_static(p, x.data_ptr(), y.data_ptr(), dw.data_ptr(), None, 64, None) == B.EQL_ERR_INVALID_ARG
            assert lib.eqlinear_plan_set_weight(p, layer.w.data_ptr(), layer.bias.data_ptr(), None) == B.EQL_ERR_INVALID_ARG
            assert lib.eqlinear_plan_device_status(p, None) == B.EQL_ERR_INVALID_ARG
        torch.cuda.synchronize()
        assert bool((y == -5.0).all().item())                                          # nothing ran
    finally:
        layer.close()


# ------------------------------------------------------------------ invariants on the GPU output alone
@pytest.mark.parametrize("dtype,T", [("fp32", 4), ("fp32", 8), ("fp16", 16), ("fp32", 5), ("fp32", 12)])
def test_gpu_equivariance_and_adjoint(dtype, T):
    wl = Workload("inv", dtype, T, 16, 24, 512, "normal", ("fwd", "bwd_data", "bwd_weight"), 19)
    d = generate(wl)
    layer = GpuLayer(wl.T, wl.Ci, wl.Co, wl.dtype, d["w"], d["bias"])
    try:
        y = layer.fwd(d["x"]).astype(np.float64).reshape(wl.N, wl.Co, T)
        for r in (1, T - 1):
            xr = np.roll(d["x"].reshape(wl.N, wl.Ci, T), r, axis=-1).reshape(wl.N, wl.Ci * T)
            yr = layer.fwd(np.ascontiguousarray(xr)).astype(np.float64).reshape(wl.N, wl.Co, T)
            nmse = ((yr - np.roll(y, r, axis=-1)) ** 2).sum() / (y ** 2).sum()
            assert nmse <= (1e-12 if dtype == "fp32" else 1e-5), nmse   # paper's Table 5: 4e-8 in FP32
    finally:
        layer.close()
    # adjoint identity <dy, fwd0(x)> = <dx, x> = <dw, w> with the bias-free layer
    layer = GpuLayer(wl.T, wl.Ci, wl.Co, wl.dtype, d["w"], None)
    try:
        f64 = lambda a: a.astype(np.float64)
        lhs = np.vdot(f64(d["dy"]), f64(layer.fwd(d["x"])))
        dx = layer.bwd_data(d["dy"])
        dw, _ = layer.bwd_weight(d["x"], d["dy"])
        tol = 1e-5 if dtype == "fp32" else 3e-3
        assert abs(lhs - np.vdot(f64(dx), f64(d["x"]))) <= tol * abs(lhs)
        assert abs(lhs - np.vdot(f64(dw), f64(d["w"]))) <= tol * abs(lhs)
    finally:
        layer.close()


# ------------------------------------------------------------------ the error path of the bounded waits
def test_expired_wait_is_reported_and_the_plan_stays_usable():
    """Every wait inside the tensor-core kernels is bounded; when one runs out the kernel ends by itself and leaves a code
    in the plan's status word.  The self-test kernel waits (with the same helper) on a barrier nothing arrives on: the
    host must read EQL_ERR_DEVICE_TIMEOUT, nothing may fault, and after clearing the status the plan computes as before."""
    wl = Workload("err", "fp16", 8, 24, 40, 300, "normal", ("fwd",), 27)
    d = generate(wl)
    layer = GpuLayer(wl.T, wl.Ci, wl.Co, wl.dtype, d["w"], d["bias"])
    try:
        ref = orc.fwd(d["x"], d["w"], d["bias"])
        assert rel_max_err(layer.fwd(d["x"]), ref) <= TOL["fp16"]
        assert eq.eqlinear_plan_device_status(layer.plan, layer.stream) == eq.binding.EQL_OK
        eq.eqlinear_plan_selftest_expired_wait(layer.plan, layer.stream)
        assert eq.eqlinear_plan_device_status(layer.plan, layer.stream) == eq.binding.EQL_ERR_DEVICE_TIMEOUT
        assert layer.raw_status() == 901                                             # the code of the wait that gave up
        torch.cuda.synchronize()                                                     # no sticky CUDA error
        eq.eqlinear_plan_clear_device_status(layer.plan, layer.stream)
        assert eq.eqlinear_plan_device_status(layer.plan, layer.stream) == eq.binding.EQL_OK
        assert rel_max_err(layer.fwd(d["x"]), ref) <= TOL["fp16"]
        assert eq.eqlinear_plan_device_status(layer.plan, layer.stream) == eq.binding.EQL_OK
    finally:
        layer.close()


# ------------------------------------------------------------------ host-buffer variants
@pytest.mark.parametrize("N", [700, 9001])
def test_host_buffer_variants(N):
    """N = 9001 goes through the chunked three-stream copy pipeline (15 chunks of 640 tokens and a ragged last one)."""
    wl = Workload("host", "fp16", 8, 24, 40, N, "normal", ("fwd", "bwd_data", "bwd_weight"), 20)
    d = generate(wl)
    layer = GpuLayer(wl.T, wl.Ci, wl.Co, wl.dtype, d["w"], d["bias"])
    try:
        N = wl.N
        xh = torch.from_numpy(d["x"]).pin_memory(); dyh = torch.from_numpy(d["dy"]).pin_memory()
        yh = torch.empty(N, wl.Dout, dtype=torch.float16).pin_memory()
        dxh = torch.empty(N, wl.Din, dtype=torch.float16).pin_memory()
        dwh = torch.empty(wl.Co, wl.Ci, wl.T, dtype=torch.float32).pin_memory()
        dbh = torch.empty(wl.Co, dtype=torch.float32).pin_memory()
        xs = torch.empty(N, wl.Din, dtype=torch.float16, device="cuda"); dys = torch.empty(N, wl.Dout, dtype=torch.float16, device="cuda")
        ys = torch.empty_like(dys); dxs = torch.empty_like(xs)
        dws = torch.empty(wl.Co, wl.Ci, wl.T, dtype=torch.float32, device="cuda"); dbs = torch.empty(wl.Co, dtype=torch.float32, device="cuda")
        sb = eq.eqlinear_bwd_weight_scratch_bytes(layer.plan, N)
        sc = torch.empty(sb, dtype=torch.uint8, device="cuda")
        eq.eqlinear_fwd_host(layer.plan, xh, yh, N, xs, ys, layer.stream)
        eq.eqlinear_bwd_data_host(layer.plan, dyh, dxh, N, dys, dxs, layer.stream)
        eq.eqlinear_bwd_weight_host(layer.plan, xh, dyh, dwh, dbh, N, xs, dys, dws, dbs, sc, sb, layer.stream)
        torch.cuda.synchronize()
        ry, rdx = orc.fwd(d["x"], d["w"], d["bias"]), orc.bwd_data(d["dy"], d["w"])
        rdw, rdb = orc.bwd_weight(d["x"], d["dy"], wl.T)
        assert rel_max_err(yh.numpy(), ry) <= TOL["fp16"]
        assert rel_max_err(dxh.numpy(), rdx) <= TOL["fp16"]
        assert rel_max_err(dwh.numpy(), rdw) <= TOL["fp16"]
        assert rel_max_err(dbh.numpy(), rdb) <= TOL["fp16"]
        # the whole step in one call, twice in a row on the same buffers
        for _ in range(2):
            for t in (yh, dxh, dwh, dbh):
                t.zero_()
            eq.eqlinear_step_host(layer.plan, xh, dyh, yh, dxh, dwh, dbh, N, xs, dys, ys, dxs, dws, dbs, sc, sb, layer.stream)
            torch.cuda.synchronize()
            assert rel_max_err(yh.numpy(), ry) <= TOL["fp16"]
            assert rel_max_err(dxh.numpy(), rdx) <= TOL["fp16"]
            assert rel_max_err(dwh.numpy(), rdw) <= TOL["fp16"]
            assert rel_max_err(dbh.numpy(), rdb) <= TOL["fp16"]
    finally:
        layer.close()
