"""Seeded synthetic layers shaped like the paper's workloads.

This module only draws random numbers and arranges them; it holds none of the
clustering arithmetic.  Both the CUDA path's callers and the CPU oracle's tests
take their inputs from here, so the two sides always see identical fp32 bits.

The paper clusters the conv / fc weight tensors of a small MNIST CNN and of a
ResNet-18 (Section 5); neither the data nor trained weights are available, so
weight tensors are drawn from the distributions those layers are initialised
with (Kaiming-normal by fan-in), or from the stated stand-in distributions.

Every recipe: ``numpy.random.default_rng(seed)``, float64 draws, one cast to
float32.  ``W`` is row-major ``[m, d]``, ``C0`` row-major ``[k, d]``, ``G`` (the
upstream gradient dL/dWq) has the shape of ``W``.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np

# (out_channels, in_channels, kh, kw) of the 20 conv tensors of a ResNet-18,
# then the 1000x512 classifier (Section 5.2 clusters such a network).
RESNET18_SHAPES = (
    [(64, 3, 7, 7)]
    + [(64, 64, 3, 3)] * 4
    + [(128, 64, 3, 3)] + [(128, 128, 3, 3)] * 3 + [(128, 64, 1, 1)]
    + [(256, 128, 3, 3)] + [(256, 256, 3, 3)] * 3 + [(256, 128, 1, 1)]
    + [(512, 256, 3, 3)] + [(512, 512, 3, 3)] * 3 + [(512, 256, 1, 1)]
    + [(1000, 512, 1, 1)]
)


@dataclass
class Workload:
    """One clustering problem (or a batch of per-layer problems sharing d, k, tau)."""
    name: str
    W: np.ndarray                 # float32 [m_total, d]
    C0: np.ndarray                # float32 [n_layers * k, d]
    G: np.ndarray                 # float32 [m_total, d]
    d: int
    k: int
    tau: float
    tol: float
    max_iter: int
    adj_tol: float
    adj_max_iter: int
    layer_offsets: np.ndarray = field(default_factory=lambda: np.zeros(0, np.int64))  # int64 [L+1], rows
    seed: int = 0

    @property
    def m(self) -> int:
        return int(self.W.shape[0])

    @property
    def n_layers(self) -> int:
        return int(len(self.layer_offsets) - 1)


def quantile_centroids(w: np.ndarray, k: int) -> np.ndarray:
    """k evenly spaced order statistics of a scalar weight set: sorted[floor((j+1/2) m / k)]."""
    flat = np.sort(np.asarray(w, dtype=np.float32).reshape(-1))
    m = flat.shape[0]
    idx = np.minimum(((np.arange(k) + 0.5) * m / k).astype(np.int64), m - 1)
    return flat[idx].reshape(k, 1).astype(np.float32)


def sampled_row_centroids(W: np.ndarray, k: int, rng: np.random.Generator) -> np.ndarray:
    """k distinct rows of W, kept in drawn order."""
    idx = rng.choice(W.shape[0], size=k, replace=False)
    return np.ascontiguousarray(W[idx]).astype(np.float32)


def _normal(rng, n, d, std):
    return (rng.standard_normal((n, d)) * std).astype(np.float32)


def single_layer(m: int, d: int, k: int, tau: float, *, std: float = 0.02, dist: str = "normal",
                 init: str = "auto", g_std: float = 1e-2, seed: int = 0, tol: float = 0.0,
                 max_iter: int = 30, adj_tol: float = 0.0, adj_max_iter: int = 30,
                 name: Optional[str] = None) -> Workload:
    """A single [m, d] layer.  ``dist``: "normal" (std) or "laplace" (scale = std)."""
    rng = np.random.default_rng(seed)
    if dist == "normal":
        W = _normal(rng, m, d, std)
    elif dist == "laplace":
        W = rng.laplace(0.0, std, size=(m, d)).astype(np.float32)
    else:
        raise ValueError(dist)
    if init == "auto":
        init = "quantile" if d == 1 else "rows"
    if init == "quantile":
        C0 = quantile_centroids(W, k)
    elif init == "rows":
        C0 = sampled_row_centroids(W, k, rng)
    else:
        raise ValueError(init)
    G = _normal(np.random.default_rng(seed + 1000), m, d, g_std)
    return Workload(name or f"layer_m{m}_d{d}_k{k}", W, C0, G, d, k, float(np.float32(tau)), tol, max_iter,
                    adj_tol, adj_max_iter, np.array([0, m], np.int64), seed)


def config1() -> Workload:
    """4096 scalar weights N(0, 0.05^2), k=4, quantile init, tau=0.05, 30+30 fixed iterations, seed 0."""
    return single_layer(4096, 1, 4, 0.05, std=0.05, g_std=1.0, seed=0, tol=0.0, max_iter=30,
                        adj_tol=0.0, adj_max_iter=30, name="cfg1_single_layer")


def config2() -> Workload:
    """64x64x3x3 conv layer, Kaiming-normal std=sqrt(2/576), k=8, tau=0.01, tol 1e-6 / 100 iterations."""
    return single_layer(64 * 64 * 9, 1, 8, 0.01, std=float(np.sqrt(2.0 / 576.0)), g_std=1e-2, seed=2,
                        tol=1e-6, max_iter=100, adj_tol=1e-6, adj_max_iter=100, name="cfg2_conv64")


def config3(shapes=RESNET18_SHAPES, k: int = 4, tau: float = 0.02, iters: int = 50, seed: int = 3) -> Workload:
    """All 21 ResNet-18-shaped tensors, each Kaiming-normal by its own fan-in, clustered per layer."""
    rng = np.random.default_rng(seed)
    grng = np.random.default_rng(seed + 1000)
    Ws, Cs, Gs, offs = [], [], [], [0]
    for (o, i, kh, kw) in shapes:
        n = o * i * kh * kw
        std = float(np.sqrt(2.0 / (i * kh * kw)))
        w = _normal(rng, n, 1, std)
        Ws.append(w)
        Cs.append(quantile_centroids(w, k))
        Gs.append(_normal(grng, n, 1, 1e-2))
        offs.append(offs[-1] + n)
    return Workload("cfg3_resnet18_batched", np.concatenate(Ws), np.concatenate(Cs), np.concatenate(Gs),
                    1, k, float(np.float32(tau)), 0.0, iters, 0.0, iters, np.array(offs, np.int64), seed)


def config4(m: int = 1 << 22, k: int = 256, iters: int = 50, seed: int = 4) -> Workload:
    """Vector quantisation: m rows of d=4 drawn Laplace(0, 0.02), k=256 sampled rows, tau=0.005."""
    return single_layer(m, 4, k, 0.005, std=0.02, dist="laplace", init="rows", g_std=1e-2, seed=seed,
                        tol=0.0, max_iter=iters, adj_tol=0.0, adj_max_iter=iters,
                        name=f"cfg4_vq_m{m}_d4_k{k}")


SWEEP_M = (1 << 20, 1 << 22, 1 << 24, 1 << 26)
SWEEP_D = (1, 2, 4)
SWEEP_B = (1, 2, 4, 8)
SWEEP_TAU = (0.1, 0.01, 0.001)


def config5_point(m: int, d: int, b: int, tau: float, *, max_iter: int = 500, seed: int = 5) -> Workload:
    """One point of the scaling sweep: N(0, 0.02^2) weights, forward to tol 1e-6 (capped)."""
    return single_layer(m, d, 1 << b, tau, std=0.02, g_std=1e-2, seed=seed, tol=1e-6, max_iter=max_iter,
                        adj_tol=1e-6, adj_max_iter=max_iter, name=f"cfg5_m{m}_d{d}_b{b}_tau{tau}")


def split_layers(wl: Workload) -> List[Workload]:
    """The per-layer problems of a batched workload, as independent single-layer workloads."""
    out = []
    for l in range(wl.n_layers):
        a, b = int(wl.layer_offsets[l]), int(wl.layer_offsets[l + 1])
        out.append(Workload(f"{wl.name}[{l}]", wl.W[a:b], wl.C0[l * wl.k:(l + 1) * wl.k], wl.G[a:b], wl.d, wl.k,
                            wl.tau, wl.tol, wl.max_iter, wl.adj_tol, wl.adj_max_iter,
                            np.array([0, b - a], np.int64), wl.seed))
    return out
