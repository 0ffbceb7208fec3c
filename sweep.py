#!/usr/bin/env python
"""Scaling sweep of the IDKM hot path on one B200 (the fifth benchmark configuration).

For every point of m x d x b x tau (weights N(0, 0.02^2)): forward to a relative centroid change of 1e-6
(capped), then the implicit backward (adjoint solve to 1e-6, capped) against the Jacobian-free backward, on
time and on gradient error measured against a 200-iteration adjoint reference computed by the library itself
(as the configuration specifies).  Prints one JSON line per point and, with --markdown, a table.

    python sweep.py [--m 1048576 4194304] [--d 1 2 4] [--b 1 2 4 8] [--tau 0.1 0.01 0.001] [--cap 500]

Every step of the path runs in the CUDA library; this script only times calls and subtracts tensors.
"""
from __future__ import annotations

import argparse
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2312_07759_b200 import workloads as WL  # noqa: E402
from bench import SM_COUNT, SM_MAX_MHZ, FP32_LANES_PER_SM, SFU_LANES_PER_SM, measured_peaks, pair_ops  # noqa: E402


def step_roofline_ms(m, d, k, hbm_gbs):
    f, s = pair_ops(d)
    pairs = float(m) * k
    return 1e3 * max(4.0 * d * m / (hbm_gbs * 1e9), pairs * f / (SM_COUNT * FP32_LANES_PER_SM * SM_MAX_MHZ * 1e6),
                     pairs * s / (SM_COUNT * SFU_LANES_PER_SM * SM_MAX_MHZ * 1e6))


def rel(x, ref):
    return float((x - ref).abs().max() / ref.abs().max().clamp_min(1e-30))


def run_point(ctx, B, torch, m, d, b, tau, cap):
    wl = WL.config5_point(m, d, b, tau, max_iter=cap)
    dev = torch.device("cuda", 0)
    W, C0, G = (torch.from_numpy(x).to(dev) for x in (wl.W, wl.C0, wl.G))
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(6)]
    # warm-up: every kernel the timed calls use is launched once before (the first launch of a kernel loads it, which
    # takes up to a millisecond and would otherwise land in the first point of each (d, k))
    ctx.forward(W, C0, wl.tau, wl.tol, 3)
    ctx.forward(W, C0, wl.tau, 0.0, 3)
    ctx.backward(G, B.JFB, 0.0, 0, 1.0)
    ctx.backward(G, B.IMPLICIT, wl.adj_tol, 3, 1.0)
    ctx.backward(G, B.IMPLICIT, 0.0, 20, 1.0)
    torch.cuda.synchronize()
    ev[0].record()
    ctx.forward(W, C0, wl.tau, wl.tol, cap)
    ev[1].record()
    dWj, dCj = ctx.backward(G, B.JFB, 0.0, 0, 1.0)
    ev[2].record()
    dWi, dCi = ctx.backward(G, B.IMPLICIT, wl.adj_tol, cap, 1.0)
    ev[3].record()
    torch.cuda.synchronize()
    info = ctx.info()[0]
    # the same number of iterations at a fixed count: the time of the executed iterations alone (launches queued
    # after convergence return at once but still cost a few microseconds each)
    # (timed by the library's own events around the loop, second of two calls: an event pair around the call would
    # also count the host's allocation of the call's outputs, which stalls the stream when a new size appears)
    ctx.set_timing(True)
    for _ in range(2):
        ctx.forward(W, C0, wl.tau, 0.0, max(info.fwd_iters, 1))
        torch.cuda.synchronize()
    fixed_ms = ctx.phase_ms()["steps"]
    ctx.set_timing(False)
    ctx.forward(W, C0, wl.tau, wl.tol, cap)                    # restore the tolerance-mode state for the reference
    dWr, dCr = ctx.backward(G, B.IMPLICIT, 0.0, 200, 1.0)     # the 200-iteration reference
    torch.cuda.synchronize()
    ref_info = ctx.info()[0]
    k = 1 << b
    peaks, _ = measured_peaks()
    fwd_ms = ev[0].elapsed_time(ev[1])
    it = max(info.fwd_iters, 1)
    out = {
        "m": m, "d": d, "k": k, "tau": tau, "fwd_iters": info.fwd_iters, "fwd_residual": info.fwd_residual,
        "fwd_status": info.status, "fwd_ms": fixed_ms, "fwd_wit_per_s": m * it / (fixed_ms * 1e-3),
        "fwd_ms_per_iter": fixed_ms / it, "fwd_ms_tol_mode": fwd_ms, "step_roofline_ms": step_roofline_ms(m, d, k, peaks["hbm_gbs"]),
        "jfb_ms": ev[1].elapsed_time(ev[2]), "implicit_ms": ev[2].elapsed_time(ev[3]),
        "adj_iters": info.adj_iters, "adj_residual": info.adj_residual,
        "ref_adj_residual": ref_info.adj_residual, "ref_status": ref_info.status,
        "dW_err_implicit": rel(dWi, dWr), "dW_err_jfb": rel(dWj, dWr),
        "dC_err_implicit": rel(dCi, dCr), "dC_err_jfb": rel(dCj, dCr),
    }
    out["frac_of_roofline"] = out["step_roofline_ms"] / out["fwd_ms_per_iter"]
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--m", type=int, nargs="+", default=list(WL.SWEEP_M))
    ap.add_argument("--d", type=int, nargs="+", default=list(WL.SWEEP_D))
    ap.add_argument("--b", type=int, nargs="+", default=list(WL.SWEEP_B))
    ap.add_argument("--tau", type=float, nargs="+", default=list(WL.SWEEP_TAU))
    ap.add_argument("--cap", type=int, default=500)
    ap.add_argument("--markdown", action="store_true")
    args = ap.parse_args()

    import torch
    from paper_2312_07759_b200 import binding as B
    if not torch.cuda.is_available():
        raise SystemExit("sweep.py needs a CUDA device")
    torch.cuda.set_device(0)
    ctx = B.Context()
    rows = []
    for m in args.m:
        for d in args.d:
            for b in args.b:
                for tau in args.tau:
                    r = run_point(ctx, B, torch, m, d, b, tau, args.cap)
                    rows.append(r)
                    print(json.dumps(r), flush=True)
    if args.markdown:
        print("\n| m | d | k | tau | fwd iters | residual | ms/iter | roofline ms | frac | JFB ms | implicit ms (iters) | "
              "dW err implicit | dW err JFB |")
        print("|---|---|---|---|---|---|---|---|---|---|---|---|---|")
        for r in rows:
            print(f"| {r['m']} | {r['d']} | {r['k']} | {r['tau']} | {r['fwd_iters']} | {r['fwd_residual']:.1e} | "
                  f"{r['fwd_ms_per_iter']:.4f} | {r['step_roofline_ms']:.4f} | {r['frac_of_roofline']:.2f} | "
                  f"{r['jfb_ms']:.3f} | {r['implicit_ms']:.3f} ({r['adj_iters']}) | {r['dW_err_implicit']:.1e} | "
                  f"{r['dW_err_jfb']:.1e} |")


if __name__ == "__main__":
    main()
