"""Writes tests/golden/cfg4_full.json: the float64 oracle's small outputs for the full-size vector-quantisation
workload (m = 2^22, d = 4, k = 256, 50 forward + 50 adjoint iterations).

Calls only the oracle and the seeded input generator; takes about ten minutes on 8 cores.  The GPU tests compare
the library's centroids and adjoint with these values and recompute per-row outputs (Wq, dL/dW) of sampled rows
from them with the oracle's per-row functions.

    python tests/golden/make_cfg4_golden.py
"""
import json
import os
import sys
import time

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(os.path.dirname(HERE))
sys.path.insert(0, ROOT)

from oracle import idkm_ref as R  # noqa: E402
from paper_2312_07759_b200 import workloads as WL  # noqa: E402


def state_at(W, G, C, tau, T_adj):
    _, _, S, F = R.final(W, C, tau, want_Wq=False)
    g = R.codebook_grad(W, G, C, tau)
    u, it, res = R.adjoint_solve(W, C, tau, S, F, g, 1.0, 0.0, T_adj)
    return {"C": C.tolist(), "S": S.tolist(), "F": F.tolist(), "g": g.tolist(), "u": u.tolist(),
            "adj_iters": it, "adj_residual": res}


def main():
    wl = WL.config4()
    W, C0, G = wl.W.astype(np.float64), wl.C0.astype(np.float64), wl.G.astype(np.float64)
    t0 = time.time()
    Ct, it, res, dead = R.forward(W, C0, wl.tau, 0.0, wl.max_iter)
    print(f"forward {it} iterations, residual {res:.3e}, {time.time() - t0:.0f} s", flush=True)
    out = {"workload": wl.name, "m": wl.m, "d": wl.d, "k": wl.k, "tau": wl.tau, "seed": wl.seed,
           "fwd_iters": it, "fwd_residual": res, "dead": dead}
    out["at_C_T"] = state_at(W, G, Ct, wl.tau, wl.adj_max_iter)
    print(f"backward at C_T done, {time.time() - t0:.0f} s", flush=True)
    Cr = Ct.astype(np.float32).astype(np.float64)
    out["at_fp32_C_T"] = state_at(W, G, Cr, wl.tau, wl.adj_max_iter)
    print(f"backward at fp32(C_T) done, {time.time() - t0:.0f} s", flush=True)
    with open(os.path.join(HERE, "cfg4_full.json"), "w") as f:
        json.dump(out, f)
    print("written")


if __name__ == "__main__":
    main()
