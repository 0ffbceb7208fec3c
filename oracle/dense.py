"""Dense (explicit-Jacobian) route to the IDKM gradients, for tiny problems only.

TEST INFRASTRUCTURE ONLY.  Second, independent route inside the oracle: it materialises the
attention matrix, writes the four Jacobians of one application of the map as full matrices
and solves the linear system of the implicit-gradient equation
``dC*/dW = (I - dF/dC)^-1 dF/dW`` (Section 4.2) by LU, where ``idkm_ref.c`` iterates vector
products.  float64 numpy; O(m k^2 d^2) memory, so m and k must be small.

Index convention: a centroid coordinate (j, a) is flattened to j*d + a, a weight coordinate
(i, b) to i*d + b.
"""
from __future__ import annotations

import numpy as np


def attention(W: np.ndarray, C: np.ndarray, tau: float, squared: bool = False):
    """A = rowsoftmax_tau(-D), D_ij = ||w_i - c_j|| (squared: ||w_i - c_j||^2, the variant in which the objectives
    of Sections 3.1 / 3.2 are written); also returns D and n_ij = dD_ij/dw_i (unit vectors; squared: 2 (w_i - c_j))."""
    diff = W[:, None, :] - C[None, :, :]                  # [m, k, d]
    D2 = (diff ** 2).sum(-1)                              # [m, k]
    D = D2 if squared else np.sqrt(D2)
    X = -(D - D.min(axis=1, keepdims=True)) / tau
    E = np.exp(X)
    A = E / E.sum(axis=1, keepdims=True)
    if squared:
        n = 2.0 * diff
    else:
        with np.errstate(invalid="ignore", divide="ignore"):
            n = np.where(D[..., None] > 0, diff / D[..., None], 0.0)
    return A, D, n


def fixed_point_map(W, C, tau, squared: bool = False):
    """F(C, W)_j = sum_i A_ij w_i / sum_i A_ij."""
    A, _, _ = attention(W, C, tau, squared)
    S = A.sum(0)
    return (A.T @ W) / S[:, None], S, A


def soft_quantise(W, C, tau, squared: bool = False):
    """Wq = A C."""
    A, _, _ = attention(W, C, tau, squared)
    return A @ C


def jacobians(W: np.ndarray, C: np.ndarray, tau: float, squared: bool = False):
    """Explicit J_C = dF/dC [kd, kd], dF/dW [kd, md], dWq/dC [md, kd], dWq/dW [md, md] at (C, W)."""
    m, d = W.shape
    k = C.shape[0]
    A, D, n = attention(W, C, tau, squared)
    S = A.sum(0)
    F = (A.T @ W) / S[:, None]
    eye_k = np.eye(k)
    eye_d = np.eye(d)
    # dA_ij/dc_l = (1/tau) A_ij (delta_jl - A_il) n_il          -> [m, k(j), k(l), d]
    dA_dC = (A[:, :, None] * (eye_k[None] - A[:, None, :]))[..., None] * n[:, None, :, :] / tau
    # dA_ij/dw_i = -(1/tau) A_ij (n_ij - sum_l A_il n_il)        -> [m, k(j), d]
    nbar = (A[..., None] * n).sum(1)                             # [m, d]
    dA_dW = -(A[..., None] * (n - nbar[:, None, :])) / tau
    dev = (W[:, None, :] - F[None, :, :]) / S[None, :, None]    # (w_i - F_j)/S_j  [m, k, d]
    # J_C[(j,a),(l,b)] = sum_i dev_ija dA_ij/dc_lb
    J_C = np.einsum("ija,ijlb->jalb", dev, dA_dC).reshape(k * d, k * d)
    # dF/dW[(j,a),(i,b)] = A_ij/S_j delta_ab + dev_ija dA_ij/dw_ib
    dF_dW = (np.einsum("ij,ab->jaib", A / S[None, :], eye_d)
             + np.einsum("ija,ijb->jaib", dev, dA_dW)).reshape(k * d, m * d)
    # dWq/dC[(i,a),(l,b)] = A_il delta_ab + sum_j c_ja dA_ij/dc_lb
    dWq_dC = (np.einsum("il,ab->ialb", A, eye_d)
              + np.einsum("ja,ijlb->ialb", C, dA_dC)).reshape(m * d, k * d)
    # dWq/dW is block diagonal: [(i,a),(i,b)] = sum_j c_ja dA_ij/dw_ib
    blocks = np.einsum("ja,ijb->iab", C, dA_dW)
    dWq_dW = np.zeros((m, d, m, d))
    for i in range(m):
        dWq_dW[i, :, i, :] = blocks[i]
    return J_C, dF_dW, dWq_dC, dWq_dW.reshape(m * d, m * d), S, F


def gradients(W, G, C, tau, mode="implicit", squared: bool = False):
    """(dL/dW [m, d], u [k, d]) of L = <G, Wq(W, C*(W))> with the linear system solved exactly.

    implicit: u = (I - J_C^T)^-1 g;  jfb: u = g  (zeroth Neumann term, Section 4.3)."""
    m, d = W.shape
    k = C.shape[0]
    J_C, dF_dW, dWq_dC, dWq_dW, _, _ = jacobians(W, C, tau, squared)
    gflat = G.reshape(-1)
    g = dWq_dC.T @ gflat
    if mode == "implicit":
        u = np.linalg.solve(np.eye(k * d) - J_C.T, g)
    elif mode == "jfb":
        u = g
    else:
        raise ValueError(mode)
    dW = dWq_dW.T @ gflat + dF_dW.T @ u
    return dW.reshape(m, d), u.reshape(k, d), g.reshape(k, d)
