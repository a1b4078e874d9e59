#!/usr/bin/env python
"""Benchmark of the Flash EQ-Linear hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME|all] [--impl ours|reference]

One "step" is one pass of the whole hot path -- eqlinear_fwd, eqlinear_bwd_data and
eqlinear_bwd_weight -- over one batch of the workload (default: the EQ-ViT-B fc1-shaped FP16
layer, T=8, 96 -> 384 channels per group element, 128 x 197 tokens).  Forward-only workloads
(Swin stage 1, the tiny FP32 case) time eqlinear_fwd alone.  Rank 0 prints ONE JSON line per
workload; `--workload all` runs the five configurations (eight workloads: the sweep has four
points) one after the other, one line each.

Each line carries, besides the contract's keys:
  roofline      the slowest of the step's calls against its floor (algorithmic bytes at the measured
                copy bandwidth, or spectral flops at the measured tensor throughput), per-call figures,
                and the DRAM traffic of a committed ncu capture where one exists (profiles/dram_traffic.md)
  sustained     the same step run back to back for --sustain-seconds (default 3 s) with the SM clock
                sampled, so that the number under a long load stands beside the short run's
  cpu_baseline  the float64 oracle timed on the host cores on a bounded sample, and `check`: sampled
                outputs of the LAST TIMED STEP (the exact call sequence that was timed) against the oracle
  dense_context torch.nn.functional.linear on the unrolled dense weight on the same GPU, forward and
                backward (fp16; fp32 with TF32 off and on) -- context, not part of the path
  e2e           the same metric through the host-buffer C-ABI call, copies inside the timed region

With N > 1 ranks every rank runs the same per-rank batch (weak scaling); the only exchange step of the
data-parallel path is the sum of dw / db over ranks (NCCL all-reduce), inside the timed step.  Without
torchrun, `--gpus N` (N > 1) starts the N ranks itself.

`--impl reference` times the float64 CPU oracle on the host cores, on a bounded sample of the same
workload, and prints the same line with "impl": "reference".
`--render-table FILE` prints a Markdown table of the JSON lines in FILE (formatting only).
"""

from __future__ import annotations

import argparse
import json
import math
import os
import socket
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# Used only when MEASURED_PEAKS.json is absent (the line then says "of fallback").
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0
L2_BYTES = 126e6


def torch_dtype_of(wl):
    import torch
    return {"fp32": torch.float32, "fp16": torch.float16, "bf16": torch.bfloat16}[wl.dtype]


def host_np(t):
    """Device tensor -> numpy (bfloat16 widened to float32 first: numpy has no bfloat16)."""
    import torch
    return (t.float() if t.dtype == torch.bfloat16 else t).cpu().numpy()


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": FALLBACK_HBM_GBS, "bf16_tflops": FALLBACK_BF16_TFLOPS,
            "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def load_committed_traffic():
    """DRAM bytes per launch from the committed ncu captures: rows of profiles/dram_traffic.md,
    | workload | call | dram read MB | dram write MB | summary file |.  Missing rows mean "not captured"."""
    table = {}
    path = os.path.join(ROOT, "profiles", "dram_traffic.md")
    if not os.path.exists(path):
        return table
    for line in open(path):
        cells = [c.strip() for c in line.strip().strip("|").split("|")]
        if len(cells) < 5:
            continue
        try:
            rd, wr = float(cells[2]), float(cells[3])
        except ValueError:
            continue
        table[(cells[0], cells[1])] = {"bytes": (rd + wr) * 1e6, "profile": cells[4]}
    return table


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons for one GPU while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int, tag: str = ""):
        self.index, self.proc, self.path = index, None, f"/tmp/eql_clocks_{os.getpid()}{tag}.csv"

    def start(self):
        try:
            self.fh = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=self.fh, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.fh.close()
        sm, mx, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in open(self.path):
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1])); power.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        try:
            os.remove(self.path)
        except OSError:
            pass
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm), "power_w_max": max(power)}


def workload_config(wl, n_gpus, extra=None):
    cfg = {"workload": wl.name, "T": wl.T, "C_in": wl.Ci, "C_out": wl.Co, "tokens_per_gpu": wl.N,
           "global_tokens": wl.N * n_gpus, "passes": list(wl.passes), "io_dtype": wl.dtype,
           "accumulate": "fp32", "parallelism": f"dp{n_gpus}" if n_gpus > 1 else "single"}
    if extra:
        cfg.update(extra)
    return cfg


def metric_name(wl):
    kind = "fwd+bwd" if "bwd_weight" in wl.passes else "fwd"
    return f"EQ-Linear tokens/s {kind} ({wl.dtype.upper()} I/O, FP32 accumulate)"


# ------------------------------------------------------------------------------------------------ oracle legs
def oracle_step(orc, wl, d, rows):
    """One pass of the workload's passes through the oracle on `rows` tokens."""
    x, dy = d["x"][:rows], d["dy"][:rows]
    out = None
    if "fwd" in wl.passes:
        out = orc.fwd(x, d["w"], d["bias"])
    if "bwd_data" in wl.passes:
        out = orc.bwd_data(dy, d["w"])
    if "bwd_weight" in wl.passes:
        out = orc.bwd_weight(x, dy, wl.T)
    return out


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 1) for i in threadpool_info() if i.get("user_api") == "blas"]
        return max(n) if n else (os.cpu_count() or 1)
    except Exception:
        return os.cpu_count() or 1


def pick_sample_rows(orc, wl, d, target_seconds):
    """Choose how many tokens of the batch the oracle can process in about `target_seconds`."""
    probe = min(wl.N, 512)
    t0 = time.perf_counter()
    oracle_step(orc, wl, d, probe)
    dt = max(time.perf_counter() - t0, 1e-4)
    rows = int(min(wl.N, max(probe, probe * target_seconds / dt)))
    return rows


def run_reference(args, wl):
    """The oracle, as it stands, timed on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from oracle import eqlinear_oracle as orc
    from paper_2607_21271_b200.workloads import generate

    d = generate(wl)
    total_budget = 150.0                                   # seconds for warm-up + timed steps
    per_step = max(0.1, min(15.0, total_budget / max(1, args.steps + args.warmup)))   # 1000 steps still end in ~3 min
    rows = pick_sample_rows(orc, wl, d, per_step)
    for _ in range(args.warmup):
        oracle_step(orc, wl, d, rows)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(orc, wl, d, rows)
    dt = time.perf_counter() - t0
    value = rows * args.steps / dt
    cores = blas_threads()
    sample = f"first {rows} of {wl.N} tokens per step, float64 dense unroll, passes {'+'.join(wl.passes)}"
    line = {"impl": "reference", "metric": metric_name(wl), "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(wl, 1),
            "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def check_against_oracle(orc, wl, d, outs):
    """Sampled outputs of the step that was timed against the oracle: sampled token rows x sampled channels of y and
    dx, and dw for sampled channel pairs over ALL tokens (dw[o, i, :] depends only on channel i of x and channel o of
    dy).  Returns max|gpu - ref| / max|ref| per tensor."""
    import numpy as np

    from paper_2607_21271_b200.workloads import sample_rows

    T = wl.T
    rows = sample_rows(wl.N, 64, seed=3)
    g = np.random.Generator(np.random.PCG64(99))

    def pick(c):
        k = min(c, 8)
        return np.unique(np.concatenate([[0, c - 1], g.choice(c, size=max(k - 2, 0), replace=False)])) if c > 1 else np.arange(1)

    ch_i, ch_o = pick(wl.Ci), pick(wl.Co)
    cols_i = (ch_i[:, None] * T + np.arange(T)[None, :]).reshape(-1)
    cols_o = (ch_o[:, None] * T + np.arange(T)[None, :]).reshape(-1)

    def rel(got, ref):
        scale = float(np.abs(ref).max())
        err = float(np.abs(got.astype(np.float64) - ref).max())
        return err / scale if scale > 0 else err

    res = {"rows": int(len(rows)), "channels": [int(len(ch_i)), int(len(ch_o))]}
    bias = None if d["bias"] is None else d["bias"][ch_o]
    if "y" in outs:
        res["y"] = rel(host_np(outs["y"][rows][:, cols_o]), orc.fwd(d["x"][rows], d["w"][ch_o], bias))
    if "dx" in outs:
        res["dx"] = rel(host_np(outs["dx"][rows][:, cols_i]), orc.bwd_data(d["dy"][rows], d["w"][:, ch_i]))
    if "dw" in outs:
        rdw, rdb = orc.bwd_weight(d["x"][:, cols_i], d["dy"][:, cols_o], T)
        res["dw"] = rel(outs["dw"].cpu().numpy()[np.ix_(ch_o, ch_i)], rdw)
        res["db"] = rel(outs["db"].cpu().numpy()[ch_o], rdb)
    tol = {"fp32": 1e-5, "fp16": 3e-3, "bf16": 6 * 2.0 ** -9}[wl.dtype]      # bf16: six unit roundoffs, as the FP16 bar
    res["tolerance"] = tol
    res["ok"] = all(res[k] <= tol for k in ("y", "dx", "dw", "db") if k in res)
    return res


# ------------------------------------------------------------------------------------------------ context legs
_FP32_PEAKS = None


def measure_fp32_peaks(dev):
    """Dense fp32 matmul throughput of this GPU, measured here: with TF32 tensor cores allowed (the class of peak an
    FP32 plan's kind::tf32 contractions run against) and with TF32 off (FFMA pipe).  cuBLAS, context only."""
    global _FP32_PEAKS
    if _FP32_PEAKS is not None:
        return _FP32_PEAKS
    import torch

    out = {}
    old = torch.backends.cuda.matmul.allow_tf32
    try:
        for name, allow, n in (("tf32_tflops", True, 8192), ("ffma_tflops", False, 4096)):
            torch.backends.cuda.matmul.allow_tf32 = allow
            a = torch.randn(n, n, device=dev)
            b = torch.randn(n, n, device=dev)
            best = float("inf")
            for i in range(6):
                s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                s.record()
                torch.matmul(a, b)
                e.record()
                torch.cuda.synchronize(dev)
                if i > 0:
                    best = min(best, s.elapsed_time(e))
            out[name] = 2 * n ** 3 / (best * 1e-3) / 1e12
            del a, b
    finally:
        torch.backends.cuda.matmul.allow_tf32 = old
    out["how"] = "torch.matmul fp32, 8192^3 with TF32 allowed / 4096^3 with TF32 off, best of 5, CUDA events"
    _FP32_PEAKS = out
    return out


def dense_context(wl, d, dev, iters=8):
    """torch.nn.functional.linear on the UNROLLED dense weight (Eq. 1: the layer the paper calls Naive EQ-Linear /
    Standard Linear of the same width), forward and backward, on the same GPU.  Context only: cuBLAS through PyTorch."""
    import torch
    import torch.nn.functional as F

    T, Ci, Co = wl.T, wl.Ci, wl.Co
    td = torch_dtype_of(wl)
    w = torch.from_numpy(d["w"]).to(dev).to(td)
    t_idx = torch.arange(T, device=dev)
    r = (t_idx[:, None] - t_idx[None, :]) % T                       # [t, s] -> group offset (t - s) mod T
    W = w[:, :, r].permute(0, 2, 1, 3).reshape(Co * T, Ci * T).contiguous()   # W[(o,t),(i,s)] = w[o,i,(t-s) mod T]
    b = None if d["bias"] is None else torch.from_numpy(d["bias"]).to(dev).to(td).repeat_interleave(T)
    x = torch.from_numpy(d["x"]).to(dev).to(td).requires_grad_(True)
    dy = torch.from_numpy(d["dy"]).to(dev).to(td) if "bwd_weight" in wl.passes else None
    W.requires_grad_(True)
    if b is not None:
        b.requires_grad_(True)
    modes = [(wl.dtype, None)] if td != torch.float32 else [("fp32_tf32_off", False), ("fp32_tf32_on", True)]
    res = {}
    old = torch.backends.cuda.matmul.allow_tf32
    try:
        for name, allow in modes:
            if allow is not None:
                torch.backends.cuda.matmul.allow_tf32 = allow
            fw, bw = [], []
            for i in range(iters + 2):
                x.grad = W.grad = None
                if b is not None:
                    b.grad = None
                e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
                e[0].record()
                y = F.linear(x, W, b)
                e[1].record()
                if dy is not None:
                    y.backward(dy)
                e[2].record()
                torch.cuda.synchronize(dev)
                if i >= 2:
                    fw.append(e[0].elapsed_time(e[1]))
                    bw.append(e[1].elapsed_time(e[2]))
                del y
            res[name] = {"fwd_ms": statistics.mean(fw), "bwd_ms": statistics.mean(bw) if dy is not None else None}
    finally:
        torch.backends.cuda.matmul.allow_tf32 = old
    res["what"] = (f"F.linear on the dense [{Co * T} x {Ci * T}] unrolled weight, {wl.N} tokens, warm inputs, "
                   f"mean of {iters}; backward = autograd (dx, dW, db)")
    return res


# ------------------------------------------------------------------------------------------------ our arm
def run_workload(args, wl, rt):
    """Times one workload on this rank's GPU; returns the JSON line (rank 0) or None."""
    import numpy as np
    import torch
    import torch.distributed as dist

    import paper_2607_21271_b200 as eq
    from paper_2607_21271_b200 import parallel
    from paper_2607_21271_b200.workloads import generate

    dev, world, rank, local_rank, use_dist = rt["dev"], rt["world"], rt["rank"], rt["local_rank"], rt["use_dist"]
    n_gpus = world
    peaks = load_peaks()
    td = torch_dtype_of(wl)
    code = {"fp32": eq.EQL_FP32, "fp16": eq.EQL_FP16, "bf16": eq.EQL_BF16}[wl.dtype]
    esz = 4 if wl.dtype == "fp32" else 2
    has_bwd = "bwd_weight" in wl.passes
    d = generate(wl)
    stream = torch.cuda.current_stream(dev).cuda_stream

    w = torch.from_numpy(d["w"]).to(dev).to(td)
    b = None if d["bias"] is None else torch.from_numpy(d["bias"]).to(dev).to(td)
    ws_bytes = eq.eqlinear_workspace_bytes(wl.T, wl.Ci, wl.Co, code)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    flags = eq.EQL_FLAG_FORCE_SIMT if args.force_simt else 0
    plan = eq.eqlinear_plan(wl.T, wl.Ci, wl.Co, code, w, b, ws, ws_bytes, flags, stream)
    info = eq.eqlinear_plan_info(plan)

    # Rotating buffer sets: more bytes than the 126 MB L2 between two uses of the same buffer.
    bytes_per_set = wl.N * (wl.Din + wl.Dout) * esz * (2 if has_bwd else 1)
    n_sets = max(2, int(np.ceil(3 * L2_BYTES / bytes_per_set)) + 1)
    n_sets = min(n_sets, 16)
    # Workloads too small for that (the tiny and small configurations) get an explicit L2 flush before every step instead:
    # a 256 MB buffer is overwritten, and the step time is the sum of the per-call event times (the flush excluded).
    flush_l2 = n_sets * bytes_per_set < 2.5 * L2_BYTES
    flush_buf = torch.empty(int(2 * L2_BYTES + 4e6), dtype=torch.uint8, device=dev) if flush_l2 else None
    x0 = torch.from_numpy(d["x"]).to(dev).to(td)
    dy0 = torch.from_numpy(d["dy"]).to(dev).to(td) if has_bwd else None
    sets = []
    for i in range(n_sets):
        s = {"x": x0 if i == 0 else x0.clone(), "y": torch.empty(wl.N, wl.Dout, dtype=td, device=dev)}
        if has_bwd:
            s["dy"] = dy0 if i == 0 else dy0.clone()
            s["dx"] = torch.empty(wl.N, wl.Din, dtype=td, device=dev)
        sets.append(s)
    grads, dw, db = parallel.grad_buffers(wl.Co, wl.Ci, wl.T, dev)      # one buffer: one all-reduce at N > 1
    sb = eq.eqlinear_bwd_weight_scratch_bytes(plan, wl.N) if has_bwd else 0
    scratch = torch.empty(max(sb, 256), dtype=torch.uint8, device=dev)
    # Training with a saved spectrum: the forward kernel that transforms x once per token tile also writes x^ for
    # the weight gradient (same step, same results within the same bars).  Used where that forward kernel runs and
    # x is the small tensor of the layer (else writing x^ costs more than repeating the transform).
    # Also on very wide layers, where the weight gradient repeats the transform of x once per output-channel tile
    # (16 times at 2048 channels) and the pre-pass that writes x^ is cheap next to the GEMMs.
    use_saved = (has_bwd and not args.no_saved_spectrum and wl.dtype != "fp32" and info.bwd_weight_kernel == 1
                 and ((info.fwd_kernel == 2 and wl.Co >= 2 * wl.Ci) or wl.Co >= 1024))
    spec_bytes = eq.eqlinear_spectrum_bytes(plan, wl.N) if use_saved else 0
    if use_saved:
        for s in sets:
            s["spec"] = torch.empty(spec_bytes, dtype=torch.uint8, device=dev)
    launches = eq.eqlinear_plan_launch_counts(plan, wl.N)
    launches_per_step = launches["fwd"] + (launches["fwd_save_spectrum_extra"] if use_saved else 0)
    if has_bwd:
        launches_per_step += launches["bwd_data"] + launches["bwd_weight"]

    comm_stream = torch.cuda.Stream(device=dev) if use_dist else None

    def step(s, events=None):
        mark = (lambda i: events[i].record()) if events is not None else None
        if flush_buf is not None:
            flush_buf.zero_()

        def fwd():
            if use_saved:
                eq.eqlinear_fwd_save_spectrum(plan, s["x"], s["y"], wl.N, s["spec"], spec_bytes, stream)
            else:
                eq.eqlinear_fwd(plan, s["x"], s["y"], wl.N, stream)

        def weight_grad():
            if use_saved:
                eq.eqlinear_bwd_weight_from_spectrum(plan, s["spec"], spec_bytes, s["dy"], dw, db, wl.N, scratch, sb, stream)
            else:
                eq.eqlinear_bwd_weight(plan, s["x"], s["dy"], dw, db, wl.N, scratch, sb, stream)

        def data_grad():
            eq.eqlinear_bwd_data(plan, s["dy"], s["dx"], wl.N, stream)

        if not has_bwd:
            if mark:
                mark(0)
            fwd()
            if mark:
                mark(1)
        elif use_dist:
            # N > 1: weight gradient first, its all-reduce on a side stream beside the data gradient (parallel.py)
            parallel.dp_training_step(fwd, weight_grad, data_grad, grads, side_stream=comm_stream, mark=mark)
        else:
            if mark:
                mark(0)
            fwd()
            if mark:
                mark(1)
            data_grad()
            if mark:
                mark(2)
            weight_grad()
            if mark:
                mark(3)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    for i in range(args.warmup):
        step(sets[i % n_sets])
    barrier()

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t_begin.record()
    for i in range(args.steps):
        step(sets[(args.warmup + i) % n_sets], ev[i])
    t_end.record()
    barrier()
    total_ms = t_begin.elapsed_time(t_end)
    last_set = sets[(args.warmup + args.steps - 1) % n_sets]
    clocks = None
    if rank == 0:
        time.sleep(0.1)
        clocks = sampler.stop()
    if world > 1:
        t = torch.tensor([total_ms], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t.item())
    status = eq.eqlinear_plan_device_status(plan, stream)
    if status != 0:
        raise RuntimeError(f"device status {status}: {eq.status_string(status)}")

    ms_per_step = total_ms / args.steps
    if flush_l2:                                               # the flush sits between the steps: count the calls only
        last = 3 if has_bwd else 1
        per = torch.tensor([statistics.mean(ev[i][0].elapsed_time(ev[i][last]) for i in range(args.steps))],
                           dtype=torch.float64, device=dev)
        if world > 1:
            dist.all_reduce(per, op=dist.ReduceOp.MAX)
        ms_per_step = float(per.item())
    value = wl.N * n_gpus / (ms_per_step * 1e-3)

    # the outputs the last timed step left behind, for the check against the oracle below
    outs = {"y": last_set["y"].clone()}
    if has_bwd:
        outs.update(dx=last_set["dx"].clone(), dw=dw.clone(), db=db.clone())

    # per-call times (mean over the timed steps), from the events recorded inside the timed region
    names = (["fwd", "bwd_weight", "bwd_data"] if use_dist else ["fwd", "bwd_data", "bwd_weight"]) if has_bwd else ["fwd"]
    kern_ms = {name: statistics.mean(ev[i][k].elapsed_time(ev[i][k + 1]) for i in range(args.steps))
               for k, name in enumerate(names)}
    alg_bytes = {"fwd": wl.N * info.bytes_per_token_fwd, "bwd_data": wl.N * info.bytes_per_token_bwd_data,
                 "bwd_weight": wl.N * info.bytes_per_token_bwd_weight + 4 * wl.T * wl.Ci * wl.Co}
    flops = 2 * info.macs_per_token * wl.N
    dom = max(names, key=lambda n: kern_ms[n])
    dom_s = kern_ms[dom] * 1e-3
    hbm_time = alg_bytes[dom] / (peaks["hbm_gbs"] * 1e9)
    kernel_kind = {"fwd": info.fwd_kernel, "bwd_data": info.bwd_data_kernel, "bwd_weight": info.bwd_weight_kernel}
    # The slowest call is bound by whichever of its two floors is higher: algorithmic bytes at the measured copy
    # bandwidth, or spectral flops at the tensor throughput of its dtype.  fp16 runs at the measured bf16 rate.  FP32
    # plans compute in TF32 with the 3xTF32 split (three tensor-core products per spectral product), against the fp32
    # matmul throughput with TF32 allowed measured in this run; their CUDA-core kernels against the FFMA figure.
    fp32_peaks = measure_fp32_peaks(dev) if wl.dtype == "fp32" else None
    if wl.dtype in ("fp16", "bf16"):
        tc_peak, tc_flops, tc_note = peaks["bf16_tflops"], flops, f"bf16 dense matmul, of {peaks['source']}"
    elif kernel_kind[dom]:
        tc_peak, tc_flops, tc_note = fp32_peaks["tf32_tflops"], 3 * flops, "fp32 matmul with TF32 allowed, measured in this run; 3xTF32 = 3 products per spectral product"
    else:
        tc_peak, tc_flops, tc_note = fp32_peaks["ffma_tflops"], flops, "fp32 matmul with TF32 off (FFMA), measured in this run"
    tc_time = tc_flops / (tc_peak * 1e12)
    traffic = load_committed_traffic()
    if tc_time > hbm_time:
        head = {"bound": "tensor" if (wl.dtype != "fp32" or kernel_kind[dom]) else "alu", "kernel": f"eqlinear_{dom}",
                "achieved": tc_flops / dom_s / 1e12, "peak": tc_peak, "unit": "TFLOP/s", "frac": tc_flops / dom_s / 1e12 / tc_peak}
    else:
        head = {"bound": "hbm", "kernel": f"eqlinear_{dom}", "achieved": alg_bytes[dom] / dom_s / 1e9,
                "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": alg_bytes[dom] / dom_s / 1e9 / peaks["hbm_gbs"]}
    tr = traffic.get((wl.name, dom))
    roofline = {**head,
                "traffic": tr["bytes"] if tr else None, "traffic_source": tr["profile"] if tr else None,
                "peak_source": f"of {peaks['source']}" if head["bound"] == "hbm" else tc_note,
                "algorithmic_bytes": alg_bytes[dom], "ms": kern_ms[dom],
                "tensor_tflops": flops / dom_s / 1e12, "tensor_frac_of_burst_peak": flops / dom_s / 1e12 / peaks["bf16_tflops"],
                "hbm_bound_us": hbm_time * 1e6, "tensor_bound_us": tc_time * 1e6,
                "fp32_peaks": fp32_peaks,
                "per_kernel": {n: {"ms": kern_ms[n], "GBps": alg_bytes[n] / (kern_ms[n] * 1e-3) / 1e9,
                                   "hbm_frac": alg_bytes[n] / (kern_ms[n] * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                   "tflops": flops / (kern_ms[n] * 1e-3) / 1e12,
                                   "tcgen05": bool(kernel_kind[n]), "kernel_id": kernel_kind[n],
                                   "traffic": traffic[(wl.name, n)]["bytes"] if (wl.name, n) in traffic else None}
                               for n in names}}

    # the same step back to back for a few seconds: what it costs once the clocks have settled under load
    sustained = None
    if world == 1 and args.sustain_seconds > 0:
        n_sus = int(min(200000, max(args.steps, math.ceil(args.sustain_seconds * 1e3 / ms_per_step))))
        sus = ClockSampler(local_rank, "s")
        a, z = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        sus.start()
        time.sleep(0.1)
        torch.cuda.synchronize(dev)
        wall0 = time.perf_counter()
        a.record()
        for i in range(n_sus):
            step(sets[i % n_sets])
        z.record()
        torch.cuda.synchronize(dev)
        wall = time.perf_counter() - wall0
        sc = sus.stop()
        sus_ms = a.elapsed_time(z) / n_sus
        sustained = {"steps": n_sus, "seconds": wall, "ms_per_step": sus_ms, "value": wl.N / (sus_ms * 1e-3),
                     "sm_mhz": sc.get("sm_mhz"), "power_w_max": sc.get("power_w_max"), "reasons": sc.get("reasons"),
                     "ms_x_mhz": sus_ms * sc["sm_mhz"] if sc.get("sm_mhz") else None,
                     "short_run_ms_x_mhz": ms_per_step * clocks["sm_mhz"] if clocks and clocks.get("sm_mhz") else None}

    # end to end through the host-buffer C-ABI call: pinned host buffers, copies inside the timed region
    e2e = None
    if not args.no_e2e:
        xh = torch.from_numpy(d["x"]).to(td).pin_memory()
        yh = torch.empty(wl.N, wl.Dout, dtype=td).pin_memory()
        s0 = sets[0]
        if has_bwd:
            dyh = torch.from_numpy(d["dy"]).to(td).pin_memory()
            dxh = torch.empty(wl.N, wl.Din, dtype=td).pin_memory()
            dwh = torch.empty(wl.Co, wl.Ci, wl.T, dtype=torch.float32).pin_memory()
            dbh = torch.empty(wl.Co, dtype=torch.float32).pin_memory()
            h2d = xh.numel() * esz + dyh.numel() * esz
            d2h = yh.numel() * esz + dxh.numel() * esz + dwh.numel() * 4 + dbh.numel() * 4

            def e2e_step():
                eq.eqlinear_step_host(plan, xh, dyh, yh, dxh, dwh, dbh, wl.N, s0["x"], s0["dy"], s0["y"], s0["dx"],
                                      dw, db, scratch, sb, stream)
        else:
            h2d, d2h = xh.numel() * esz, yh.numel() * esz

            def e2e_step():
                eq.eqlinear_fwd_host(plan, xh, yh, wl.N, s0["x"], s0["y"], stream)
        e_steps = max(3, min(args.steps, 10))
        for _ in range(2):
            e2e_step()
        barrier()
        a, z = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(e_steps):
            e2e_step()
        z.record()
        barrier()
        e_ms = a.elapsed_time(z) / e_steps
        if world > 1:
            t = torch.tensor([e_ms], dtype=torch.float64, device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            e_ms = float(t.item())
        e2e = {"value": wl.N * n_gpus / (e_ms * 1e-3), "unit": "tokens/s", "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": e_ms, "steps": e_steps,
               "api": "eqlinear_step_host" if has_bwd else "eqlinear_fwd_host"}

    eq.eqlinear_plan_destroy(plan)
    del sets, scratch, ws

    context = None
    if rank == 0 and n_gpus == 1 and not args.no_context:
        torch.cuda.empty_cache()
        context = dense_context(wl, d, dev)

    cpu_baseline = None
    if rank == 0 and n_gpus == 1 and not args.no_cpu_baseline:
        from oracle import eqlinear_oracle as orc
        rows = pick_sample_rows(orc, wl, d, args.cpu_seconds)
        t0 = time.perf_counter()
        oracle_step(orc, wl, d, rows)
        dt = time.perf_counter() - t0
        cpu_baseline = {"value": rows / dt, "unit": "tokens/s", "cores": blas_threads(), "kind": "oracle",
                        "sample": f"first {rows} of {wl.N} tokens, one pass of {'+'.join(wl.passes)}, float64 dense unroll",
                        "seconds": dt,
                        "check": check_against_oracle(orc, wl, d, outs)}

    if rank != 0:
        return None
    return {"metric": metric_name(wl), "value": value, "unit": "tokens/s", "n_gpus": n_gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": {"fp16": "f16", "bf16": "bf16", "fp32": "f32"}[wl.dtype],
            "data": "synthetic",
            "config": workload_config(wl, n_gpus, {"l2": ("flushed before every step (256 MB overwrite), step time = sum of the calls' event times"
                                                          if flush_l2 else f"rotating {n_sets} buffer sets "
                                                          f"({n_sets * bytes_per_set / 1e6:.0f} MB > 126 MB L2)"),
                                                    "saved_spectrum": bool(use_saved)}),
            "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step * args.steps,
            "roofline": roofline, "sustained": sustained, "cpu_baseline": cpu_baseline, "dense_context": context}


# ------------------------------------------------------------------------------------------------ formatting
def render_table(path):
    """Markdown table of the JSON lines in `path` (one row per call of each workload)."""
    rows = []
    for line in open(path):
        line = line.strip()
        if not line.startswith("{"):
            continue
        j = json.loads(line)
        if j.get("impl") == "reference":
            continue
        cfg, rf = j["config"], j["roofline"]
        ctx, cpu, sus = j.get("dense_context") or {}, j.get("cpu_baseline") or {}, j.get("sustained") or {}
        chk = cpu.get("check") or {}
        err_of = {"fwd": "y", "bwd_data": "dx", "bwd_weight": "dw"}
        for name, k in rf["per_kernel"].items():
            dense = []
            for mode, v in ctx.items():
                if isinstance(v, dict):
                    t = v["fwd_ms"] if name == "fwd" else v["bwd_ms"]
                    if t is not None:
                        dense.append(f"{mode} {'fwd' if name == 'fwd' else 'bwd (dx+dW+db)'} {t * 1e3:.0f} us")
            err = chk.get(err_of[name])
            rows.append(f"| {cfg['workload']} | {name} | {k['ms'] * 1e3:.1f} us | {cfg['tokens_per_gpu'] / (k['ms'] * 1e-3):.3g} | "
                        f"{k['GBps']:.0f} ({k['hbm_frac']:.2f}) | {k['tflops']:.0f} | "
                        f"{'tcgen05' if k['tcgen05'] else 'FFMA'} #{k['kernel_id']} | "
                        f"{'' if err is None else f'{err:.1e}'} | {'; '.join(dense) if name != 'bwd_data' else ''} |")
        rows.append(f"| {cfg['workload']} | **step** | {j['ms_per_step'] * 1e3:.1f} us @ {j['clocks']['sm_mhz']:.0f} MHz; "
                    f"sustained {sus.get('ms_per_step', float('nan')) * 1e3:.1f} us @ {sus.get('sm_mhz') or float('nan'):.0f} MHz | "
                    f"{j['value']:.3g} | | | | check ok: {chk.get('ok')} | oracle CPU {cpu.get('value', float('nan')):.3g} tokens/s "
                    f"({cpu.get('cores')} cores); e2e {j['e2e']['value'] if j.get('e2e') else float('nan'):.3g} tokens/s |")
    print("| workload | call | GPU time | tokens/s | algorithmic GB/s (of 6456) | spectral TFLOP/s | kernel | max err / max ref (sampled, oracle) | context |")
    print("|---|---|---|---|---|---|---|---|---|")
    print("\n".join(rows))


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default=None, help="a workload name, or 'all' for the five configurations")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--sustain-seconds", type=float, default=3.0, help="length of the back-to-back run (0: skip)")
    ap.add_argument("--cpu-seconds", type=float, default=15.0, help="target length of the oracle's timed sample")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-context", action="store_true", help="skip the F.linear-on-the-dense-weight context leg")
    ap.add_argument("--force-simt", action="store_true", help="use the CUDA-core kernels (context numbers)")
    ap.add_argument("--no-saved-spectrum", action="store_true",
                    help="weight gradient from x (eqlinear_bwd_weight) instead of from the spectrum saved by the forward pass")
    ap.add_argument("--render-table", default=None, metavar="FILE")
    args = ap.parse_args()
    if args.render_table:
        render_table(args.render_table)
        return
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    from paper_2607_21271_b200.workloads import ALL_WORKLOADS, CONFIGS, HEADLINE
    names = list(CONFIGS) if args.workload == "all" else [args.workload or HEADLINE]

    if args.impl == "reference":
        for name in names:
            run_reference(args, ALL_WORKLOADS[name])
        return

    # --gpus N without torchrun: start the N ranks here (one process per GPU, NCCL over NVLink for the exchange step)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__), *sys.argv[1:]]
        sys.exit(subprocess.call(cmd))

    import torch
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the library has no CPU fallback")
    dev = torch.device(f"cuda:{local_rank}")
    torch.cuda.set_device(dev)
    # EQL_BENCH_FORCE_DIST: run the N > 1 form of the step in a one-rank group (to exercise it on one GPU)
    use_dist = world > 1 or bool(os.environ.get("EQL_BENCH_FORCE_DIST"))
    if use_dist:
        dist.init_process_group("nccl", device_id=dev)
    rt = {"dev": dev, "world": world, "rank": rank, "local_rank": local_rank, "use_dist": use_dist}
    for name in names:
        line = run_workload(args, ALL_WORKLOADS[name], rt)
        if line is not None:
            print(json.dumps(line), flush=True)
        torch.cuda.empty_cache()
    if use_dist:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
