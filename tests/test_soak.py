"""Opt-in long checks of the CUDA path (`python -m pytest tests/test_soak.py -m soak -s`; they are deselected by
`-m gpu` and skipped everywhere else): a random-shape parity fuzz over every kernel family, tensors beyond 4 GB (the
64-bit offset paths), and a soak of repeated full steps whose results must stay bit-identical.  Too long for the
regular suite; the output of their last run is kept in tests/soak_last_run.txt.

EQL_SOAK_SHAPES (default 300) random shapes, EQL_SOAK_STEPS (default 300) repeated steps per layer."""

import os
import random

import numpy as np
import pytest
import torch

import paper_2607_21271_b200 as eq
from oracle import eqlinear_oracle as orc
from paper_2607_21271_b200.workloads import CONFIGS, Workload, generate
from tests.harness import TOL, GpuLayer, rel_max_err

pytestmark = pytest.mark.soak


def test_random_shapes_match_the_oracle():
    """Every pass of every kernel family on random shapes: both dtypes, every supported group order, ragged token counts,
    all bias kinds, the correlation flag, the streaming / CTA-pair / CUDA-core kernels forced at random, and for FP16 the
    saved-spectrum path; bfloat16 plans and the fused GELU epilogue at random.  Stops at the first device time-out."""
    count = int(os.environ.get("EQL_SOAK_SHAPES", "300"))
    rng = random.Random(int(os.environ.get("EQL_SOAK_SEED", "0")))
    bad, kinds = [], {}
    for it in range(count):
        dtype = rng.choice(["fp16", "fp16", "fp32", "fp32", "bf16"])
        T = rng.choice([4, 4, 8, 8, 8, 8, 16, 16, 32, 32, 2, 3, 5, 6, 7, 12, 1])
        e = 4 if dtype == "fp32" else 2
        step = next(s for s in range(1, 17) if (s * T * e) % 16 == 0)      # row bytes C*T*e must be a multiple of 16
        cmax = 600 if T <= 8 else 96 if T <= 16 else 48
        if not (T in (4, 8, 16, 32)):
            cmax = min(cmax, 64)                                            # CUDA-core kernels: keep the oracle pass short
        Ci = step * rng.randint(1, max(1, cmax // step)); Co = step * rng.randint(1, max(1, cmax // step))
        if rng.random() < 0.3:
            Ci = max(step, (c := rng.choice([8, 16, 24, 48, 96, 128, 256, 384])) - c % step)
        if rng.random() < 0.3:
            Co = max(step, (c := rng.choice([8, 16, 24, 48, 96, 128, 256, 384])) - c % step)
        if T > 8 or T not in (4, 8, 16, 32):
            Ci, Co = min(Ci, cmax), min(Co, cmax)
        N = rng.choice([1, 7, 15, 16, 17, 31, 33, 63, 64, 65, 100, 127, 129, 255, 300, 511, 640, 1000, 2049, 4099, 9473, 20011])
        if Ci * Co * T * T * N > 6e10:
            N = 300
        flags = eq.EQL_FLAG_CORRELATION if rng.random() < 0.15 else 0
        r = rng.random()
        if r < 0.15:
            flags |= eq.EQL_FLAG_FORCE_STREAMING
        elif r < 0.30:
            flags |= eq.EQL_FLAG_FORCE_STREAMING | eq.EQL_FLAG_CTA_PAIR
        elif r < 0.35:
            flags |= eq.EQL_FLAG_FORCE_SIMT
        corr = bool(flags & eq.EQL_FLAG_CORRELATION)
        gelu = rng.random() < 0.2 and not (dtype == "fp32" and T in (4, 8) and Ci > 256 and not flags & eq.EQL_FLAG_FORCE_SIMT)
        if gelu:
            flags |= eq.EQL_FLAG_GELU
        wl = Workload("fz", dtype, T, Ci, Co, N, rng.choice(["normal", "zero", "none"]), ("fwd", "bwd_data", "bwd_weight"), 1000 + it)
        d = generate(wl)
        layer = GpuLayer(T, Ci, Co, dtype, d["w"], d["bias"], flags)
        info = eq.eqlinear_plan_info(layer.plan)
        key = (dtype, info.fwd_kernel, info.bwd_data_kernel, info.bwd_weight_kernel)
        kinds[key] = kinds.get(key, 0) + 1
        errs = {}
        try:
            ref_y = orc.fwd(d["x"], d["w"], d["bias"], corr)
            if gelu:
                from scipy.special import erf
                ref_y = 0.5 * ref_y * (1.0 + erf(ref_y / np.sqrt(2.0)))
            errs["y"] = rel_max_err(layer.fwd(d["x"]), ref_y)
            errs["dx"] = rel_max_err(layer.bwd_data(d["dy"]), orc.bwd_data(d["dy"], d["w"], corr))
            dw, db = layer.bwd_weight(d["x"], d["dy"])
            rdw, rdb = orc.bwd_weight(d["x"], d["dy"], T, corr)
            errs["dw"], errs["db"] = rel_max_err(dw, rdw), rel_max_err(db, rdb)
            if dtype == "fp16" and info.bwd_weight_kernel == 1:
                x_t, dy_t = torch.from_numpy(d["x"]).cuda(), torch.from_numpy(d["dy"]).cuda()
                sb = eq.eqlinear_spectrum_bytes(layer.plan, N)
                spec = torch.full((sb + 64,), 0x7F, dtype=torch.uint8, device="cuda")
                y2 = torch.empty(N, Co * T, dtype=torch.float16, device="cuda")
                eq.eqlinear_fwd_save_spectrum(layer.plan, x_t, y2, N, spec, sb, layer.stream)
                scb = eq.eqlinear_bwd_weight_scratch_bytes(layer.plan, N)
                sc = torch.empty(scb + 16, dtype=torch.uint8, device="cuda")
                dw2 = torch.full((Co, Ci, T), float("nan"), dtype=torch.float32, device="cuda")
                db2 = torch.full((Co,), float("nan"), dtype=torch.float32, device="cuda")
                eq.eqlinear_bwd_weight_from_spectrum(layer.plan, spec, sb, dy_t, dw2, db2, N, sc, scb, layer.stream)
                torch.cuda.synchronize()
                errs["y_s"] = rel_max_err(y2.cpu().numpy(), ref_y)
                errs["dw_s"], errs["db_s"] = rel_max_err(dw2.cpu().numpy(), rdw), rel_max_err(db2.cpu().numpy(), rdb)
                if not bool((spec[sb:] == 0x7F).all().item()):
                    errs["spectrum_overrun"] = 1.0
            st = layer.raw_status()
        finally:
            layer.close()
        ok = all(v <= TOL[dtype] for v in errs.values()) and st == 0
        print(f"{'ok ' if ok else 'BAD'} #{it} {dtype} T={T} Ci={Ci} Co={Co} N={N} flags={flags} bias={wl.bias} kernels={key[1:]} "
              f"status={st} " + " ".join(f"{k}={v:.2e}" for k, v in errs.items()), flush=True)
        if not ok:
            bad.append((it, dtype, T, Ci, Co, N, flags))
            if st != 0:
                break
    print("plans per (dtype, fwd, bwd_data, bwd_weight kernel):", kinds)
    assert not bad, bad


def test_tensors_beyond_4_gb():
    """800 003 tokens of the headline layer: y is 4.9 GB, so byte offsets pass 2^31 and 2^32.  Sampled rows (both ends,
    random ones, and rows around those two offsets) of the forward result of both tensor-core kernels and of the data
    gradient, and sampled channel pairs of the weight gradient over all tokens, against the oracle."""
    T, Ci, Co, N = 8, 96, 384, 800_003
    d = generate(Workload("s", "fp16", T, Ci, Co, 16, "normal", ("fwd",), 5))
    g = torch.Generator(device="cuda").manual_seed(1)
    x = torch.randn(N, Ci * T, device="cuda", dtype=torch.float16, generator=g)
    rows = np.unique(np.concatenate([np.arange(0, 40), np.arange(N - 70, N), np.random.default_rng(0).integers(0, N, 300),
                                     np.arange(699_040, 699_100), np.arange(349_500, 349_560)]))
    ri = torch.from_numpy(rows).cuda()
    xr = x[ri].cpu().numpy()
    ref = orc.fwd(xr, d["w"], d["bias"])
    y = None
    for flags in (0, eq.EQL_FLAG_FORCE_STREAMING):
        layer = GpuLayer(T, Ci, Co, "fp16", d["w"], d["bias"], flags)
        try:
            yk = torch.full((N, Co * T), float("nan"), device="cuda", dtype=torch.float16)
            eq.eqlinear_fwd(layer.plan, x, yk, N, layer.stream)
            assert layer.raw_status() == 0
            err = rel_max_err(yk[ri].cpu().numpy(), ref)
            nan_rows = int(torch.isnan(yk).any(dim=1).sum().item())
            print(f"fwd flags={flags}: y is {yk.numel() * 2 / 1e9:.2f} GB, sampled error {err:.2e}, rows with NaN {nan_rows}", flush=True)
            assert err <= TOL["fp16"] and nan_rows == 0
            if y is None:
                y = yk
                dx = torch.full((N, Ci * T), float("nan"), device="cuda", dtype=torch.float16)
                eq.eqlinear_bwd_data(layer.plan, y, dx, N, layer.stream)            # y as the incoming gradient
                assert layer.raw_status() == 0
                e2 = rel_max_err(dx[ri].cpu().numpy(), orc.bwd_data(y[ri].cpu().numpy(), d["w"]))
                print(f"bwd_data: sampled error {e2:.2e}, rows with NaN {int(torch.isnan(dx).any(dim=1).sum().item())}", flush=True)
                assert e2 <= TOL["fp16"] and not bool(torch.isnan(dx).any().item())
                del dx
                dw = torch.empty(Co, Ci, T, device="cuda", dtype=torch.float32)
                db = torch.empty(Co, device="cuda", dtype=torch.float32)
                sb = eq.eqlinear_bwd_weight_scratch_bytes(layer.plan, N)
                sc = torch.empty(sb, dtype=torch.uint8, device="cuda")
                eq.eqlinear_bwd_weight(layer.plan, x, y, dw, db, N, sc, sb, layer.stream)
                assert layer.raw_status() == 0
                ch_o, ch_i = np.array([0, 100, 383]), np.array([0, 50, 95])
                co = (ch_o[:, None] * T + np.arange(T)).reshape(-1)
                ci = (ch_i[:, None] * T + np.arange(T)).reshape(-1)
                rdw, rdb = orc.bwd_weight(x[:, torch.from_numpy(ci).cuda()].cpu().numpy(),
                                          y[:, torch.from_numpy(co).cuda()].cpu().numpy(), T)
                e3 = rel_max_err(dw.cpu().numpy()[np.ix_(ch_o, ch_i)], rdw)
                e4 = rel_max_err(db.cpu().numpy()[ch_o], rdb)
                print(f"bwd_weight: sampled errors dw {e3:.2e} db {e4:.2e}", flush=True)
                assert e3 <= TOL["fp16"] and e4 <= TOL["fp16"]
            else:
                assert float((yk[ri].float() - y[ri].float()).abs().max()) <= 2e-2 * float(y[ri].float().abs().max())
            del yk
        finally:
            layer.close()


@pytest.mark.parametrize("name,tokens", [("vit_b_fc1_fp16", None), ("sweep_T8_fp16", 20000), ("swin_t_s1_fp16", 60000),
                                         ("vit_s_fp32", None), ("sweep_T4_fp16", 20000), ("op_c512_pair", None)])
def test_repeated_steps_stay_bit_identical(name, tokens):
    """A race in one of the shared-memory pipelines shows up as a rare corrupted row: hundreds of repeated full steps of
    each kernel family (the CTA-pair form included) must produce identical bits."""
    steps = int(os.environ.get("EQL_SOAK_STEPS", "300"))
    wl = Workload("op_c512_pair", "fp16", 4, 512, 512, 8192, "normal", ("fwd", "bwd_data", "bwd_weight"), 9) if name == "op_c512_pair" \
        else CONFIGS[name]
    if tokens:
        wl = wl.with_tokens(tokens)
    d = generate(wl)
    td = torch.float16 if wl.dtype == "fp16" else torch.float32
    it = torch.int16 if wl.dtype == "fp16" else torch.int32
    layer = GpuLayer(wl.T, wl.Ci, wl.Co, wl.dtype, d["w"], d["bias"])
    try:
        plan, stream = layer.plan, layer.stream
        has_bwd = "bwd_weight" in wl.passes
        x = torch.from_numpy(d["x"]).cuda(); dy = torch.from_numpy(d["dy"]).cuda()
        y = torch.empty(wl.N, wl.Dout, dtype=td, device="cuda"); dx = torch.empty(wl.N, wl.Din, dtype=td, device="cuda")
        dw = torch.empty(wl.Co, wl.Ci, wl.T, dtype=torch.float32, device="cuda"); db = torch.empty(wl.Co, dtype=torch.float32, device="cuda")
        sb = eq.eqlinear_bwd_weight_scratch_bytes(plan, wl.N); sc = torch.empty(max(sb, 256), dtype=torch.uint8, device="cuda")
        saved = wl.dtype == "fp16" and eq.eqlinear_plan_info(plan).bwd_weight_kernel == 1
        if saved:
            spb = eq.eqlinear_spectrum_bytes(plan, wl.N); spec = torch.empty(spb, dtype=torch.uint8, device="cuda")
        ref, mismatches = None, 0
        for _ in range(steps):
            y.fill_(float("nan")); dx.fill_(float("nan")); dw.fill_(float("nan"))
            if saved:
                eq.eqlinear_fwd_save_spectrum(plan, x, y, wl.N, spec, spb, stream)
            else:
                eq.eqlinear_fwd(plan, x, y, wl.N, stream)
            if has_bwd:
                eq.eqlinear_bwd_data(plan, dy, dx, wl.N, stream)
                if saved:
                    eq.eqlinear_bwd_weight_from_spectrum(plan, spec, spb, dy, dw, db, wl.N, sc, sb, stream)
                else:
                    eq.eqlinear_bwd_weight(plan, x, dy, dw, db, wl.N, sc, sb, stream)
            sig = (y.view(it).long().sum().item(), dx.view(it).long().sum().item() if has_bwd else 0,
                   dw.view(torch.int32).long().sum().item() if has_bwd else 0)
            if ref is None:
                ref = sig
            elif sig != ref:
                mismatches += 1
        status = layer.raw_status()
        print(f"{wl.name}: {steps} steps, {mismatches} mismatches, device status {status}", flush=True)
        assert mismatches == 0 and status == 0
    finally:
        layer.close()
