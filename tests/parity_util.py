"""Shared helpers of the GPU parity tests: run the CUDA path and the float64 oracle on the same
seeded fp32 inputs and compare element by element."""
import os

import numpy as np

# Stated tolerances of the fp32 CUDA path against the float64 oracle at a fixed iteration count
TOL_C = 1e-5      # centroids and Wq, relative
TOL_GRAD = 1e-4   # dL/dW and dL/dC, relative

# Achieved errors of the checks that carry a `record` tag, in the order they ran.  When the environment variable
# IDKM_PARITY_TABLE names a file, the session writes them there as a markdown table (tests/conftest.py).
RECORDS = []


def rel_err(x, ref):
    """(max-norm error / max|ref|, l2 error / ||ref||_2)."""
    x = np.asarray(x, np.float64)
    ref = np.asarray(ref, np.float64)
    e = np.abs(x - ref)
    mx = np.abs(ref).max()
    l2 = np.linalg.norm(ref)
    return float(e.max() / max(mx, 1e-300)), float(np.linalg.norm(e) / max(l2, 1e-300))


ELEM_FLOOR = 5.0   # in units of rms(ref)


def elem_err(x, ref):
    """Element-wise relative error with a floor: max_i |x_i - ref_i| / (|ref_i| + ELEM_FLOOR rms(ref)).  Unlike the
    two norms above it does not let the few largest entries hide an error in the many small ones (most rows of
    dL/dW are far below the largest).  The floor is there because an entry is a sum of k terms of either sign: its
    rounding error scales with the terms, whose size the typical entry shows, not with the entry itself."""
    x = np.asarray(x, np.float64)
    ref = np.asarray(ref, np.float64)
    floor = max(ELEM_FLOOR * float(np.sqrt(np.mean(ref * ref))), 1e-300)
    return float((np.abs(x - ref) / (np.abs(ref) + floor)).max())


def assert_close(x, ref, tol, what, l2_only=False, record=None):
    """max-norm, l2 and element-wise (see elem_err) relative errors all within `tol`; `l2_only` keeps the l2 bound
    alone (chained d = 1 runs with kink crossings, where single rows legitimately differ by O(1))."""
    rm, r2 = rel_err(x, ref)
    el = elem_err(x, ref)
    if record is not None:
        RECORDS.append((record, what, rm, r2, el, tol, "l2 only" if l2_only else ""))
    ok = r2 <= tol and (l2_only or (rm <= tol and el <= tol))
    assert ok, f"{what}: rel max {rm:.3e}, rel l2 {r2:.3e}, element-wise {el:.3e} > {tol:.1e}"
    return rm, r2


def write_records(path):
    """The recorded errors as a markdown table."""
    lines = ["| test | quantity | max-norm / max abs ref | l2 / l2 ref | element-wise, floor 5 rms(ref) | bound | note |",
             "|---|---|---|---|---|---|---|"]
    # per-layer rows of a batched configuration collapse to the worst layer per quantity
    import re
    merged, order = {}, []
    for tag, what, rm, r2, el, tol, note in RECORDS:
        mt = re.match(r"^(\S+) layer \d+ \(m = \d+\)$", tag)
        if mt:
            tag = f"{mt.group(1)}, worst of the layers"
            what = re.sub(r"^layer \d+ ", "", re.sub(r" \(\d+ kink crossings\)", " (kink crossings)", what))
        key = (tag, what, tol, note)
        if key not in merged:
            merged[key] = [rm, r2, el]
            order.append(key)
        else:
            merged[key] = [max(a, b) for a, b in zip(merged[key], (rm, r2, el))]
    for (tag, what, tol, note) in order:
        rm, r2, el = merged[(tag, what, tol, note)]
        lines.append(f"| {tag} | {what} | {rm:.2e} | {r2:.2e} | {el:.2e} | {tol:.0e} | {note} |")
    os.makedirs(os.path.dirname(os.path.abspath(path)), exist_ok=True)
    with open(path, "w") as f:
        f.write("\n".join(lines) + "\n")


def assert_grad_close(x, ref, what, crossings, tol, tol_kink, record=None):
    """Gradient check of a chained run.  With no kink crossing: max-norm and l2 at `tol`.  With crossings the
    rows of the crossed weights legitimately differ by O(1), so only the l2 error is bounded, by `tol_kink`."""
    if crossings == 0:
        return assert_close(x, ref, tol, what, record=record)
    return assert_close(x, ref, tol_kink, what + f" ({crossings} kink crossings)", l2_only=True, record=record)


def oracle_run(wl, mode="implicit", alpha=1.0, fixed=True, want_A=False, want_dW=True, squared=False):
    """Oracle forward + final + backward of a single-layer workload (fixed iteration counts when
    ``fixed``: tolerances disabled).  ``squared``: the squared-distance variant."""
    from oracle import idkm_ref as R
    tol = 0.0 if fixed else wl.tol
    adj_tol = 0.0 if fixed else wl.adj_tol
    W, C0, G = wl.W.astype(np.float64), wl.C0.astype(np.float64), wl.G.astype(np.float64)
    with R.squared_distance(squared):
        Ct, it, res, dead = R.forward(W, C0, wl.tau, tol, wl.max_iter)
        Wq, A, S, F = R.final(W, Ct, wl.tau, want_A=want_A)
        dW, dC, ait, ares = R.backward(W, G, Ct, wl.tau, S, F, mode=mode, alpha=alpha, adj_tol=adj_tol,
                                       adj_max_iter=wl.adj_max_iter, want_dW=want_dW)
    return dict(C=Ct, Wq=Wq, A=A, S=S, F=F, dW=dW, dC=dC, iters=it, res=res, adj_iters=ait, adj_res=ares, dead=dead)


def gpu_run(wl, mode="implicit", alpha=1.0, fixed=True, want_A=False, ctx=None, want_dW=True, squared=False):
    """The same through the C-ABI library on cuda:0."""
    import torch
    from paper_2312_07759_b200 import binding as B
    dev = torch.device("cuda:0")
    ctx = ctx or B.Context()
    ctx.set_distance(squared)
    W = torch.from_numpy(wl.W).to(dev)
    C0 = torch.from_numpy(wl.C0).to(dev)
    G = torch.from_numpy(wl.G).to(dev)
    tol = 0.0 if fixed else wl.tol
    adj_tol = 0.0 if fixed else wl.adj_tol
    offs = [int(x) for x in wl.layer_offsets]
    fr = ctx.forward(W, C0, wl.tau, tol, wl.max_iter, layer_offsets=offs, want_A=want_A)
    dW, dC = ctx.backward(G, B.IMPLICIT if mode == "implicit" else B.JFB, adj_tol, wl.adj_max_iter, alpha,
                          want_dW=want_dW)
    info = ctx.info()
    torch.cuda.synchronize()
    return dict(C=fr.C.cpu().numpy(), Wq=fr.Wq.cpu().numpy(), A=None if fr.A is None else fr.A.cpu().numpy(),
                dW=None if dW is None else dW.cpu().numpy(), dC=dC.cpu().numpy(), info=info, ctx=ctx)


def oracle_backward_at(wl, C, mode="implicit", alpha=1.0, want_dW=True, squared=False):
    """Oracle final pass + backward evaluated at the given centroids (fixed adjoint count)."""
    from oracle import idkm_ref as R
    W, G, C = wl.W.astype(np.float64), wl.G.astype(np.float64), np.asarray(C, np.float64)
    with R.squared_distance(squared):
        Wq, _, S, F = R.final(W, C, wl.tau)
        dW, dC, ait, ares = R.backward(W, G, C, wl.tau, S, F, mode=mode, alpha=alpha, adj_tol=0.0,
                                       adj_max_iter=wl.adj_max_iter, want_dW=want_dW)
    return dict(C=C, Wq=Wq, dW=dW, dC=dC)


def at_centroids(wl, C):
    """The same workload with the clustering loop switched off and C as the starting (= returned) centroids."""
    import copy
    w2 = copy.copy(wl)
    w2.C0 = np.ascontiguousarray(np.asarray(C, np.float32))
    w2.max_iter = 0
    return w2


def kink_crossings(W, C_a, C_b):
    """For d = 1 the Jacobians of the map jump when a centroid crosses a weight (n_ij = sign(w_i - c_j)).
    Number of (weight, centroid) pairs whose sign differs between two centroid sets; 0 for d > 1."""
    if W.shape[1] != 1:
        return 0
    w = W[:, 0].astype(np.float64)
    n = 0
    for ca, cb in zip(np.asarray(C_a, np.float64)[:, 0], np.asarray(C_b, np.float64)[:, 0]):
        lo, hi = min(ca, cb), max(ca, cb)
        n += int(((w >= lo) & (w <= hi)).sum()) if lo != hi else 0
    return n
