#!/usr/bin/env python
"""Benchmark of the IDKM hot path on B200: weight-iterations/sec and fraction of the roofline.

One *step* is one pass of the whole hot path over one synthetic layer batch: the soft k-means loop
(forward steps), the final pass (Wq), the implicit backward (codebook gradient, adjoint loop, dL/dW
pass) and the Jacobian-free backward (codebook gradient + dL/dW pass).  The metric counts the loop
iterations: value = m * (forward iterations + adjoint iterations) / time of the step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg4] [--impl ours|reference]

Under torchrun every rank runs its own replica of the workload (the path has no exchange step);
the time is the maximum over ranks and the value the sum over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2312_07759_b200 import workloads as WL  # noqa: E402

SM_COUNT = 148
SM_MAX_MHZ = 1965.0
FP32_LANES_PER_SM = 128     # fp32 add/mul/fma results per clock per SM (compute capability 10.0)
SFU_LANES_PER_SM = 16       # ex2 / rsqrt / rcp / sqrt results per clock per SM


def make_workload(name: str):
    if name == "cfg1":
        return WL.config1()
    if name == "cfg2":
        wl = WL.config2()
        wl.tol, wl.adj_tol = 0.0, 0.0       # fixed 100 + 100 iterations so that the count is known
        return wl
    if name == "cfg3":
        return WL.config3()
    if name == "cfg4":
        return WL.config4()
    if name.startswith("cfg5:"):             # cfg5:m,d,b,tau,iters
        m, d, b, tau, it = name[5:].split(",")
        wl = WL.config5_point(int(m), int(d), int(b), float(tau), max_iter=int(it))
        wl.tol, wl.adj_tol = 0.0, 0.0
        return wl
    raise SystemExit(f"unknown workload {name}")


def pair_ops(d: int):
    """Algorithmic work of one fused forward step per (weight-vector, centroid) pair:
    (fp32-pipe instruction lanes, special-function lanes)."""
    if d == 1:
        return 6, 1          # sub|abs, min, fma(scale), add(sum), fma(S), fma(N)  + ex2
    return 3 * d + 5, 2      # d sub, d fma (square), mul(D), min, fma, add, fma(S), d fma(N)  + rsqrt, ex2


def adjoint_pair_ops(d: int):
    """Algorithmic work of one fused adjoint step per pair (Eq. 14's vector-Jacobian product): the softmax of the
    forward step without its S / N sums, then p_ij (d fma), its attention-weighted mean (fma), e_ij(p) / (tau D_ij)
    (sub, 3 mul; 2 mul and a sign for d = 1) and the d sums of e_ij n_ij."""
    if d == 1:
        return 11, 1         # sub|abs, min, fma, add, fma(p), fma(mean), sub, mul, mul, sign, fma  + ex2
    return 4 * d + 9, 2      # d sub, d fma, mul(D), min, fma, add, d fma(p), fma(mean), sub, 3 mul, d fma  + rsqrt, ex2


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.index, self.samples, self.reasons, self.max_mhz = index, [], set(), None
        self._halt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self._halt.is_set():
            try:
                self.samples.append(float(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                try:
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, nm in names.items():
                    if r & bit:
                        self.reasons.add(nm)
            except Exception:
                pass
            time.sleep(0.05)

    def stop(self):
        self._halt.set()
        if self.is_alive():
            self.join(timeout=2)
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def max_over_ranks(x: float, device=None) -> float:
    """Maximum of a per-rank number over the process group (the rank's own value without one)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_value(rows_per_rank: int, iterations: int, world: int, ms_per_step: float) -> float:
    """Whole-job weight-iterations/sec: every rank runs its own replica (no exchange step on the path), the step
    time is the slowest rank's."""
    return world * rows_per_rank * iterations / (ms_per_step * 1e-3)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}, "fallback"


def stored_traffic(workload_name):
    """DRAM bytes per launch of the loop kernels from the stored ncu capture (profiles/traffic_cfg4.json): a map
    "<pass>:<centroids per lane>x<lanes per weight>" -> bytes, empty when the file is for another workload or was
    written for another version of the kernel source."""
    import hashlib
    path = os.path.join(ROOT, "profiles", "traffic_cfg4.json")
    src = os.path.join(ROOT, "paper_2312_07759_b200", "csrc", "idkm_kernels.cuh")
    if workload_name is None or not os.path.exists(path) or not os.path.exists(src):
        return {}
    with open(path) as f:
        t = json.load(f)
    with open(src, "rb") as f:
        sha = hashlib.sha256(f.read()).hexdigest()
    if t.get("workload") != workload_name or t.get("kernel_source_sha256") != sha:
        return {}
    return {key: v["dram_bytes_read"] + v["dram_bytes_write"] for key, v in t.get("kernels", {}).items()}


def store_traffic(workload_name, entries, source):
    """Writes profiles/traffic_cfg4.json from figures read off an ncu capture: entries maps
    "<pass>:<centroids per lane>x<lanes per weight>" to (dram__bytes_read.sum, dram__bytes_write.sum) of one launch.  The
    sha256 of the kernel source goes with them, so that a later change of the kernels voids the figures."""
    import hashlib
    src = os.path.join(ROOT, "paper_2312_07759_b200", "csrc", "idkm_kernels.cuh")
    with open(src, "rb") as f:
        sha = hashlib.sha256(f.read()).hexdigest()
    out = {"workload": workload_name, "kernel_source_sha256": sha, "source": source,
           "kernels": {key: {"dram_bytes_read": float(r), "dram_bytes_write": float(w)} for key, (r, w) in entries.items()}}
    with open(os.path.join(ROOT, "profiles", "traffic_cfg4.json"), "w") as f:
        json.dump(out, f, indent=1)
        f.write("\n")


def time_oracle_sample(wl, rows: int, it_f: int, it_a: int):
    """Times the float64 oracle on the first `rows` rows of the workload: it_f forward iterations and it_a
    adjoint iterations (plus the final pass and the codebook gradient they need).  Returns
    (weight-iterations/sec, seconds, threads)."""
    from oracle import idkm_ref as R
    rows = min(rows, wl.m if wl.n_layers == 1 else int(wl.layer_offsets[1]))
    W = wl.W[:rows].astype(np.float64)
    G = wl.G[:rows].astype(np.float64)
    C0 = wl.C0[:wl.k].astype(np.float64)
    t0 = time.perf_counter()
    Ct, _, _, _ = R.forward(W, C0, wl.tau, 0.0, it_f)
    t_f = time.perf_counter() - t0
    _, _, S, F = R.final(W, Ct, wl.tau, want_Wq=False)
    g = R.codebook_grad(W, G, Ct, wl.tau)
    t0 = time.perf_counter()
    R.adjoint_solve(W, Ct, wl.tau, S, F, g, 1.0, 0.0, it_a)
    t_a = time.perf_counter() - t0
    sec = t_f + t_a
    return rows * (it_f + it_a) / sec, sec, R.threads(), rows * it_f / t_f, rows * it_a / t_a


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = make_workload(args.workload)
    rows, it_f, it_a = args.cpu_rows, 2, 2
    vals = []
    for s in range(args.warmup + args.steps):
        v, sec, thr, _, _ = time_oracle_sample(wl, rows, it_f, it_a)
        if s >= args.warmup:
            vals.append((v, sec))
    v = float(np.mean([x[0] for x in vals]))
    ms = float(np.mean([x[1] for x in vals]) * 1e3)
    sample = f"first {min(rows, wl.m)} rows of {wl.name}, {it_f} forward + {it_a} adjoint iterations per step"
    line = {
        "impl": "reference", "metric": "weight-iterations/sec", "value": v, "unit": "weight-iterations/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "m": wl.m, "d": wl.d, "k": wl.k, "tau": wl.tau},
        "cpu_baseline": {"value": v, "unit": "weight-iterations/s", "cores": thr, "kind": "oracle", "sample": sample},
        "e2e": {"value": v, "unit": "weight-iterations/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg4")
    ap.add_argument("--cpu-rows", type=int, default=1 << 19, help="rows of the workload the oracle is timed on")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--collapse-step", type=int, default=0, choices=[0, 1],
                    help="step of collapsing layers: 0 fp32 increment form (default), 1 fp64")
    ap.add_argument("--iters", type=int, default=0, help="override the forward and adjoint iteration counts "
                    "(short runs for profiler captures; the reported value is then not the configured workload's)")
    ap.add_argument("--store-traffic", nargs="+", metavar="KEY=READ,WRITE", default=None,
                    help="record dram bytes per launch read off an ncu capture of this workload's loop kernels, e.g. "
                    "'idkm_pass<ADJ>:16x16=100764160,3399680' (no GPU work is done)")
    args = ap.parse_args()
    if args.store_traffic:
        entries = {}
        for item in args.store_traffic:
            key, val = item.split("=")
            r, w = val.split(",")
            entries[key] = (float(r), float(w))
        store_traffic(make_workload(args.workload).name, entries,
                      "ncu --set full captures summarised in profiles/adjoint_kernel_cfg4.txt and profiles/step_kernel_cfg4.txt")
        return
    if args.warmup < 3:
        args.warmup = 3 if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import torch.distributed as dist
    from paper_2312_07759_b200 import binding as B      # raises if the CUDA library is missing

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    wl = make_workload(args.workload)
    if args.iters > 0:
        wl.max_iter = wl.adj_max_iter = args.iters
    m, d, k, L = wl.m, wl.d, wl.k, wl.n_layers
    offs = [int(x) for x in wl.layer_offsets]
    T_f, T_a = wl.max_iter, wl.adj_max_iter
    W = torch.from_numpy(wl.W).to(dev)
    C0 = torch.from_numpy(wl.C0).to(dev)
    G = torch.from_numpy(wl.G).to(dev)
    ctx = B.Context()
    ctx.set_collapse_step(args.collapse_step)
    ctx.set_timing(True)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)     # > 126 MB L2

    launches_before = [0]

    def step():
        fr = ctx.forward(W, C0, wl.tau, 0.0, T_f, layer_offsets=offs, want_Wq=True)
        dWj, dCj = ctx.backward(G, B.JFB, 0.0, 0, 1.0)
        dW, dC = ctx.backward(G, B.IMPLICIT, 0.0, T_a, 1.0)
        return fr, dW, dC, dWj

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    # The clock sampler starts before the last warm-up step: the first NVML queries of a process are slow and were
    # seen to delay kernel launches of the step they coincided with (one timed step 20-70 ms longer than the others).
    sampler = ClockSampler(local)
    for w in range(args.warmup):
        if w == args.warmup - 1:
            sampler.start()
        out = step()                        # kept, as in the timed loop, so that torch's allocator reaches its steady state
        flush.fill_(1)
    barrier()
    launches_before[0] = ctx.launches
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    phases = []
    for s in range(args.steps):
        flush.fill_(s)                      # L2 flush between timed steps (outside the timed events)
        ev[s][0].record()
        out = step()
        ev[s][1].record()
        ev[s][1].synchronize()
        phases.append(ctx.phase_ms())       # forward and implicit-backward phases of this step
    barrier()
    clocks = sampler.stop()
    n_launch = ctx.launches - launches_before[0]
    step_ms = [a.elapsed_time(b) for a, b in ev]
    total_ms = float(sum(step_ms))
    total_ms = max_over_ranks(total_ms, dev)
    ms_per_step = total_ms / args.steps
    value = job_value(m, T_f + T_a, world, ms_per_step)

    info = ctx.info()
    ph = {key: float(np.mean([p[key] for p in phases])) for key in phases[0]}
    step_kernel_ms = ph["steps"] / max(T_f, 1)
    adj_kernel_ms = ph["adjoint"] / max(T_a, 1)

    # ---- rooflines of the two loop kernels; `roofline` is the one with the larger share of the step -----------------
    pairs = float(m) * k
    peaks, which = measured_peaks()
    fp32_rate, sfu_rate = B.measure_pipe_rates()      # register-only micro-benchmarks of the two pipes, measured now
    path = B.describe_path(d, k, T_a, 0)
    traffic_table = stored_traffic(wl.name if args.iters == 0 else None)

    def kernel_roofline(label, layout, kernel_ms, ops, share, bytes_per_row):
        fp32_ops, sfu_ops = ops
        t_hbm = (bytes_per_row * m) / (peaks["hbm_gbs"] * 1e9)
        fp32_peak = SM_COUNT * FP32_LANES_PER_SM * SM_MAX_MHZ * 1e6
        sfu_peak = SM_COUNT * SFU_LANES_PER_SM * SM_MAX_MHZ * 1e6
        t_fp32, t_sfu = pairs * fp32_ops / fp32_peak, pairs * sfu_ops / sfu_peak
        sec = kernel_ms * 1e-3
        if t_hbm >= max(t_fp32, t_sfu):
            r = {"bound": "hbm", "achieved": bytes_per_row * m / sec / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                 "peak_source": f"MEASURED_PEAKS.json hbm_gbs ({which})"}
        elif t_fp32 >= t_sfu:
            r = {"bound": "alu", "achieved": pairs * fp32_ops / sec / 1e12, "peak": fp32_peak / 1e12,
                 "unit": "Tinst-lanes/s (fp32 pipe)", "peak_source": "148 SMs x 128 fp32 lanes/clk x 1965 MHz"}
        else:
            r = {"bound": "alu", "achieved": pairs * sfu_ops / sec / 1e12, "peak": sfu_peak / 1e12,
                 "unit": "Tinst-lanes/s (sfu pipe)", "peak_source": "148 SMs x 16 sfu lanes/clk x 1965 MHz"}
        r["frac"] = r["achieved"] / r["peak"]
        r["kernel"] = f"{label}, layout {layout[0]} centroids/lane x {layout[1]} lanes/weight"
        r["kernel_ms"] = kernel_ms
        r["share_of_step"] = share
        r["roofline_ms"] = max(t_hbm, t_fp32, t_sfu) * 1e3
        r["fp32_ops_per_pair"], r["sfu_ops_per_pair"] = fp32_ops, sfu_ops
        r["algorithmic_bytes_per_launch"] = bytes_per_row * m
        # dram__bytes_read.sum + dram__bytes_write.sum of one launch from the stored ncu capture of this kernel (ncu
        # flushes the caches before the launch, so this is the cold-L2 figure); null when none is stored for this
        # workload and layout, or when the kernel source has changed since the capture
        r["traffic"] = traffic_table.get(f"{label.split(' ')[0]}:{layout[0]}x{layout[1]}")
        r["frac_of_measured_pipes"] = max(t_hbm, pairs * fp32_ops / fp32_rate, pairs * sfu_ops / sfu_rate) / sec
        return r

    step_total = float(np.mean(step_ms))
    roof_step = kernel_roofline("idkm_pass<STEP> (fused forward step)", path["step_layout"], step_kernel_ms, pair_ops(d),
                                ph["steps"] / step_total, 4.0 * d) if T_f > 0 and step_kernel_ms > 0 else None
    roof_adj = None
    if T_a > 0 and adj_kernel_ms > 0 and path["adjoint_route"] == "fused passes":
        # the group-per-weight adjoint layouts also read each row's cached softmax reference and normaliser (8 bytes)
        roof_adj = kernel_roofline("idkm_pass<ADJ> (fused adjoint step)", path["adjoint_layout"], adj_kernel_ms,
                                   adjoint_pair_ops(d), ph["adjoint"] / step_total,
                                   4.0 * d + (8.0 if path["adjoint_layout"][1] > 1 else 0.0))
    ranked = sorted([r for r in (roof_step, roof_adj) if r is not None], key=lambda r: -r["share_of_step"])
    roof = ranked[0] if ranked else None
    roof_second = ranked[1] if len(ranked) > 1 else None
    if roof is not None:
        roof["pipes_measured"] = {"fp32_lane_ops_per_s": fp32_rate, "sfu_lane_ops_per_s": sfu_rate,
                                  "fp32_lanes_per_clk_per_sm_at_max_clock": fp32_rate / (SM_COUNT * SM_MAX_MHZ * 1e6),
                                  "sfu_lanes_per_clk_per_sm_at_max_clock": sfu_rate / (SM_COUNT * SM_MAX_MHZ * 1e6)}
        roof["adjoint_route"] = path["adjoint_route"]

    # ---- end to end through the host-buffer entry point: the same work as the timed step ----------------------------
    e2e = None
    if not args.no_e2e:
        hW = torch.from_numpy(wl.W).pin_memory()
        hG = torch.from_numpy(wl.G).pin_memory()
        hC0 = torch.from_numpy(wl.C0).pin_memory()
        outs = {"C": torch.empty_like(hC0).pin_memory().numpy(), "Wq": torch.empty_like(hW).pin_memory().numpy(),
                "dW": torch.empty_like(hW).pin_memory().numpy(), "dC": torch.empty_like(hC0).pin_memory().numpy(),
                "dW_jfb": torch.empty_like(hW).pin_memory().numpy(), "dC_jfb": torch.empty_like(hC0).pin_memory().numpy()}
        hctx = B.Context()
        n_e2e = max(2, min(args.steps, 3))

        def host_step():
            # forward + Jacobian-free backward + implicit backward from one forward, as in step() above
            return hctx.quantize_host(hW.numpy(), hC0.numpy(), hG.numpy(), wl.tau, 0.0, T_f, B.IMPLICIT, 0.0, T_a, 1.0,
                                      layer_offsets=offs, out=outs, also_jfb=True)

        host_step()
        barrier()
        e2e_ms = []
        for _ in range(n_e2e):
            flush.fill_(3)
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            host_step()                      # returns after the last copy has landed
            e2e_ms.append((time.perf_counter() - t0) * 1e3)
        e2e_s = max_over_ranks(float(np.mean(e2e_ms)) * 1e-3, dev)
        e2e = {"value": job_value(m, T_f + T_a, world, e2e_s * 1e3), "unit": "weight-iterations/s",
               "h2d_bytes_per_step": int(hW.numel() * 4 + hG.numel() * 4 + hC0.numel() * 4),
               "d2h_bytes_per_step": int(3 * hW.numel() * 4 + 3 * hC0.numel() * 4), "ms_per_step": e2e_s * 1e3,
               "api": "idkm_quantize_host_ex (forward + Jacobian-free backward + implicit backward, pinned host "
                      "buffers; the upload of dL/dWq overlaps the forward loop, the downloads of Wq and the "
                      "Jacobian-free dL/dW overlap the backward)"}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, sec, thr, vf, va = time_oracle_sample(wl, 2 * args.cpu_rows, 10, 10)     # about 10-20 s of CPU work
        cpu = {"value": v, "unit": "weight-iterations/s", "cores": thr, "kind": "oracle",
               "sample": f"first {min(2 * args.cpu_rows, m)} rows of {wl.name}, 10 forward + 10 adjoint iterations, {sec:.1f} s",
               "forward_value": vf, "adjoint_value": va}

    if rank == 0:
        line = {
            "metric": "weight-iterations/sec", "value": value, "unit": "weight-iterations/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": wl.name, "m": m, "d": d, "k": k, "n_layers": L, "tau": wl.tau,
                       "forward_iters": T_f, "adjoint_iters": T_a, "parallelism": f"replicas x{world}",
                       "l2": "256 MB buffer written between timed steps; W (%.0f MB) stays L2-resident across the "
                             "iterations inside a step" % (m * d * 4 / 1e6)},
            "forward_wit_per_s": world * m * T_f / (ph["steps"] * 1e-3) if T_f else None,
            "adjoint_wit_per_s": world * m * T_a / (ph["adjoint"] * 1e-3) if T_a else None,
            "step_ms": [round(x, 3) for x in step_ms],
            "step_phase_sum_ms": [round(sum(p.values()), 3) for p in phases], "phase_ms": ph, "step_kernel_ms": step_kernel_ms, "adjoint_kernel_ms": adj_kernel_ms,
            "roofline": roof, "roofline_second": roof_second, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": int(n_launch), "clocks": clocks,
            "info": {"status": [i.status for i in info][:4], "fwd_residual": info[0].fwd_residual,
                     "adj_residual": info[0].adj_residual},
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
