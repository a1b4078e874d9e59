#!/usr/bin/env python
"""Benchmark of the Flash EQ-Linear hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

One "step" is one pass of the whole hot path -- eqlinear_fwd, eqlinear_bwd_data and
eqlinear_bwd_weight -- over one batch of the workload (default: the EQ-ViT-B fc1-shaped FP16
layer, T=8, 96 -> 384 channels per group element, 128 x 197 tokens).  Forward-only workloads
(Swin stage 1) time eqlinear_fwd alone.  Prints ONE JSON line on rank 0.

With N > 1 ranks (torchrun) every rank runs the same per-rank batch (weak scaling); the only
exchange step of the data-parallel path is the sum of dw / db over ranks (NCCL all-reduce),
which is inside the timed step.

`--impl reference` times the float64 CPU oracle on the host cores, on a bounded sample of the
same workload, and prints the same line with "impl": "reference".
"""

from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

FALLBACK_HBM_GBS = 6650.0        # earlier measurement on this machine, used only without MEASURED_PEAKS.json
FALLBACK_BF16_TFLOPS = 1590.0

# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per launch from the committed ncu capture
# profiles/umma_kernels_fp16_vit_b_fc1.md (None = not captured for that workload / kernel).
NCU_TRAFFIC_BYTES = {
    ("vit_b_fc1_fp16", "fwd"): 48.6e6 + 145.4e6,          # includes the 38.7 MB spectrum of x saved for the weight gradient
    ("vit_b_fc1_fp16", "bwd_data"): 156.1e6 + 17.3e6,
    ("vit_b_fc1_fp16", "bwd_weight"): 193.7e6 + 3.7e6,
}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": FALLBACK_HBM_GBS, "bf16_tflops": FALLBACK_BF16_TFLOPS,
            "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons for one GPU while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.path = index, None, f"/tmp/eql_clocks_{os.getpid()}.csv"

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
    import numpy as np  # noqa: F401

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
    print(json.dumps(line))


def metric_name(wl):
    kind = "fwd+bwd" if "bwd_weight" in wl.passes else "fwd"
    return f"EQ-Linear tokens/s {kind} ({wl.dtype.upper()} I/O, FP32 accumulate)"


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--force-simt", action="store_true", help="use the CUDA-core kernels (context numbers)")
    ap.add_argument("--no-saved-spectrum", action="store_true",
                    help="weight gradient from x (eqlinear_bwd_weight) instead of from the spectrum saved by the forward pass")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    from paper_2607_21271_b200.workloads import ALL_WORKLOADS, HEADLINE, generate
    wl = ALL_WORKLOADS[args.workload or HEADLINE]

    if args.impl == "reference":
        run_reference(args, wl)
        return

    import numpy as np
    import torch
    import torch.distributed as dist

    import paper_2607_21271_b200 as eq
    from paper_2607_21271_b200 import parallel

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
    n_gpus = world

    peaks = load_peaks()
    td = torch.float32 if wl.dtype == "fp32" else torch.float16
    code = eq.EQL_FP32 if wl.dtype == "fp32" else eq.EQL_FP16
    esz = 4 if wl.dtype == "fp32" else 2
    has_bwd = "bwd_weight" in wl.passes
    d = generate(wl)
    stream = torch.cuda.current_stream(dev).cuda_stream

    w = torch.from_numpy(d["w"]).to(dev)
    b = None if d["bias"] is None else torch.from_numpy(d["bias"]).to(dev)
    ws_bytes = eq.eqlinear_workspace_bytes(wl.T, wl.Ci, wl.Co, code)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    flags = eq.EQL_FLAG_FORCE_SIMT if args.force_simt else 0
    plan = eq.eqlinear_plan(wl.T, wl.Ci, wl.Co, code, w, b, ws, ws_bytes, flags, stream)
    info = eq.eqlinear_plan_info(plan)

    # Rotating buffer sets: more bytes than the 126 MB L2 between two uses of the same buffer.
    bytes_per_set = wl.N * (wl.Din + wl.Dout) * esz * (2 if has_bwd else 1)
    n_sets = max(2, int(np.ceil(3 * 126e6 / bytes_per_set)) + 1)
    n_sets = min(n_sets, 16)
    x0 = torch.from_numpy(d["x"]).to(dev)
    dy0 = torch.from_numpy(d["dy"]).to(dev) if has_bwd else None
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
    use_saved = (has_bwd and not args.no_saved_spectrum and wl.dtype == "fp16" and info.bwd_weight_kernel == 1
                 and ((info.fwd_kernel == 2 and wl.Co >= 2 * wl.Ci) or wl.Co >= 1024))
    spec_bytes = eq.eqlinear_spectrum_bytes(plan, wl.N) if use_saved else 0
    if use_saved:
        for s in sets:
            s["spec"] = torch.empty(spec_bytes, dtype=torch.uint8, device=dev)

    # N > 1: the weight gradient goes first, and its all-reduce is issued from a side stream that waits only for it, so
    # that the exchange overlaps the data gradient of the same step (the step still ends with the summed dw / db:
    # the compute stream waits for the collective before the step is over).
    comm_stream = torch.cuda.Stream(device=dev) if use_dist else None
    dw_ready = torch.cuda.Event() if use_dist else None

    def step(s, events=None):
        if events is not None:
            events[0].record()
        if use_saved:
            eq.eqlinear_fwd_save_spectrum(plan, s["x"], s["y"], wl.N, s["spec"], spec_bytes, stream)
        else:
            eq.eqlinear_fwd(plan, s["x"], s["y"], wl.N, stream)
        if events is not None:
            events[1].record()
        if has_bwd:
            def weight_grad():
                if use_saved:
                    eq.eqlinear_bwd_weight_from_spectrum(plan, s["spec"], spec_bytes, s["dy"], dw, db, wl.N, scratch, sb, stream)
                else:
                    eq.eqlinear_bwd_weight(plan, s["x"], s["dy"], dw, db, wl.N, scratch, sb, stream)

            work = None
            if use_dist:
                weight_grad()
                dw_ready.record()
                with torch.cuda.stream(comm_stream):
                    comm_stream.wait_event(dw_ready)
                    work = parallel.allreduce_weight_grads(dw, db, flat=grads, async_op=True)
                if events is not None:
                    events[2].record()
                eq.eqlinear_bwd_data(plan, s["dy"], s["dx"], wl.N, stream)
                if events is not None:
                    events[3].record()
                if work is not None:
                    work.wait()                                # the compute stream waits for the collective
            else:
                eq.eqlinear_bwd_data(plan, s["dy"], s["dx"], wl.N, stream)
                if events is not None:
                    events[2].record()
                weight_grad()
                if events is not None:
                    events[3].record()

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
    value = wl.N * n_gpus / (ms_per_step * 1e-3)

    # per-kernel times (mean over the timed steps), from the events recorded inside the timed region
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
    # The dominant kernel is bound by whichever of its two floors is higher: algorithmic bytes at the measured copy
    # bandwidth, or spectral flops at the measured dense tensor throughput (fp16 runs at the bf16 rate; FP32 plans
    # compute in TF32, nominally 1.1 / 2.25 of it).
    tc_peak = peaks["bf16_tflops"] * (1.0 if wl.dtype == "fp16" else 1.1 / 2.25)
    tc_time = flops / (tc_peak * 1e12)
    if tc_time > hbm_time:
        head = {"bound": "tensor", "kernel": f"eqlinear_{dom}", "achieved": flops / dom_s / 1e12, "peak": tc_peak,
                "unit": "TFLOP/s", "frac": flops / dom_s / 1e12 / tc_peak}
    else:
        head = {"bound": "hbm", "kernel": f"eqlinear_{dom}", "achieved": alg_bytes[dom] / dom_s / 1e9,
                "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": alg_bytes[dom] / dom_s / 1e9 / peaks["hbm_gbs"]}
    roofline = {**head,
                "traffic": NCU_TRAFFIC_BYTES.get((wl.name, dom)), "peak_source": f"of {peaks['source']}",
                "algorithmic_bytes": alg_bytes[dom], "ms": kern_ms[dom],
                "tensor_tflops": flops / dom_s / 1e12, "tensor_frac_of_burst_peak": flops / dom_s / 1e12 / peaks["bf16_tflops"],
                "hbm_bound_us": hbm_time * 1e6, "tensor_bound_us": tc_time * 1e6,
                "per_kernel": {n: {"ms": kern_ms[n], "GBps": alg_bytes[n] / (kern_ms[n] * 1e-3) / 1e9,
                                   "hbm_frac": alg_bytes[n] / (kern_ms[n] * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                   "tcgen05": bool(kernel_kind[n]),
                                   "traffic": NCU_TRAFFIC_BYTES.get((wl.name, n))} for n in names}}

    # end to end through the host-buffer C-ABI call: pinned host buffers, copies inside the timed region
    e2e = None
    if not args.no_e2e:
        xh = torch.from_numpy(d["x"]).pin_memory()
        yh = torch.empty(wl.N, wl.Dout, dtype=td).pin_memory()
        s0 = sets[0]
        if has_bwd:
            dyh = torch.from_numpy(d["dy"]).pin_memory()
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
               "d2h_bytes_per_step": d2h, "ms_per_step": e_ms, "steps": e_steps}

    cpu_baseline = None
    if rank == 0 and n_gpus == 1 and not args.no_cpu_baseline:
        from oracle import eqlinear_oracle as orc
        rows = pick_sample_rows(orc, wl, d, 15.0)
        t0 = time.perf_counter()
        oracle_step(orc, wl, d, rows)
        dt = time.perf_counter() - t0
        cpu_baseline = {"value": rows / dt, "unit": "tokens/s", "cores": blas_threads(), "kind": "oracle",
                        "sample": f"first {rows} of {wl.N} tokens, one pass of {'+'.join(wl.passes)}, float64 dense unroll",
                        "seconds": dt}

    eq.eqlinear_plan_destroy(plan)
    if rank == 0:
        launches_per_step = 1 + (3 if has_bwd else 0)      # fwd, bwd_data, bwd_weight (2 kernels)
        line = {"metric": metric_name(wl), "value": value, "unit": "tokens/s", "n_gpus": n_gpus,
                "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f16" if wl.dtype == "fp16" else "f32",
                "data": "synthetic",
                "config": workload_config(wl, n_gpus, {"l2": f"rotating {n_sets} buffer sets "
                                                              f"({n_sets * bytes_per_set / 1e6:.0f} MB > 126 MB L2)",
                                                        "saved_spectrum": bool(use_saved)}),
                "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step * args.steps,
                "roofline": roofline, "cpu_baseline": cpu_baseline}
        print(json.dumps(line))
    if use_dist:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
