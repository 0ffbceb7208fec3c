"""Gradient of the TRUNCATED clustering loop by reverse-mode differentiation through every stored iteration -- what
DKM does (Section 3.4: backpropagation through all t iterations, memory O(t m 2^b)) and what IDKM replaces by the
implicit gradient (Section 4.2) or its Jacobian-free shortcut (Section 4.3).

TEST INFRASTRUCTURE ONLY, like the rest of ``oracle/``: it quantifies how the implicit gradient, which treats the
returned centroids as an exact fixed point, differs from the true derivative of the T-step program when the loop has
not converged.  float64; composed from the oracle's own per-pass routines (``idkm_ref``), in the plain order of the
chain rule, with nothing fused.

The program differentiated, with C_0 held constant:

    C_{t+1} = F(C_t, W)  for t = 0 .. T-1,      Wq = A(W, C_T) C_T,      L = <G, Wq>.

Reverse sweep:  v_T = (dWq/dC)^T G at C_T;  for t = T-1 .. 0:  dW += (dF/dW)^T v_{t+1} at C_t  and
v_t = (dF/dC)^T v_{t+1} at C_t;  finally dW += (dWq/dW)^T G at C_T.  The T centroid sets are stored; the attention
matrices (the O(t m 2^b) term of DKM) are recomputed instead, which changes memory, not the result.
"""
from __future__ import annotations

import numpy as np

from . import idkm_ref as R


def forward_iterates(W, C0, tau: float, T: int):
    """[C_0, C_1, ..., C_T] of Algorithm 1 with a fixed count."""
    Cs = [np.asarray(C0, np.float64).copy()]
    for _ in range(T):
        Cs.append(R.step(W, Cs[-1], tau)[0])
    return Cs


def gradients(W, G, C0, tau: float, T: int):
    """(dL/dW [m, d], dL/dC_0 [k, d], C_T) of L = <G, Wq(W, C_T(W))> for the T-step loop started at the constant C_0."""
    W = np.asarray(W, np.float64)
    G = np.asarray(G, np.float64)
    Cs = forward_iterates(W, C0, tau, T)
    CT = Cs[-1]
    zeros_G = np.zeros_like(G)
    _, _, S_T, F_T = R.final(W, CT, tau, want_Wq=False)
    v = R.codebook_grad(W, G, CT, tau)                                   # (dWq/dC)^T G
    # (dWq/dW)^T G: the scatter pass with a zero adjoint keeps only its direct term
    dW = R.scatter(W, G, CT, tau, S_T, F_T, np.zeros_like(CT))
    for t in range(T - 1, -1, -1):
        Ct = Cs[t]
        _, _, S, F = R.final(W, Ct, tau, want_Wq=False)                  # S, F(C_t, W) = C_{t+1} of this application
        dW += R.scatter(W, zeros_G, Ct, tau, S, F, v)                    # (dF/dW)^T v   (zero upstream: no direct term)
        v = R.adjoint_apply(W, Ct, tau, S, F, v)                         # (dF/dC)^T v
    return dW, v, CT
