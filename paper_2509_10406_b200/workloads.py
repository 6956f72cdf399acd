"""Seeded synthetic inputs for the MuSe attention layer.

This module serves both the CUDA path's tests/benchmarks and the CPU oracle's
tests.  It contains input generation only (Gaussian mixtures, rotary position
encoding, k-means++ seeding indices) and none of the method's arithmetic; it
imports neither the CUDA binding nor the oracle.

The paper evaluates on Q/K/V activations of trained language models
(Section "Experiments", Appendix "96M Model Microbenchmarks"), which are not
available; Gaussian-mixture tensors of the same shapes stand in for them.

All arrays are produced with numpy's PCG64 generator in float32 and, where a
workload is bf16, rounded to bf16 (round-to-nearest-even) *before* either side
sees them, so the GPU and the oracle consume identical bits.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Optional

import numpy as np

__all__ = [
    "Workload", "WORKLOADS", "make_head_inputs", "make_inputs", "round_bf16",
    "kmeanspp_indices", "random_init_indices", "rope",
]


@dataclasses.dataclass(frozen=True)
class Workload:
    """One synthetic workload.  Field names follow the paper's notation:
    N tokens, D head dim, Cq/Ck query/key clusters, m = k_1 retrieved clusters,
    S spatial blocks, T Lloyd iterations."""
    name: str
    B: int
    Hq: int
    Hkv: int
    N: int
    D: int
    Cq: int
    Ck: int
    m: int
    S: int = 8
    T: int = 3
    dtype: str = "bf16"            # "bf16" | "f32"
    components: int = 32           # mixture components per head
    anisotropic: bool = True
    rope_theta: Optional[float] = None
    student_t_nu: Optional[float] = None
    outlier_frac: float = 0.0
    outlier_scale: float = 5.0
    init: str = "random"           # "kmeans++" | "random"
    seed: int = 20250910

    def with_(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


WORKLOADS = {
    "tiny": Workload("tiny", 1, 1, 1, 1024, 64, 8, 16, 4, T=5, dtype="f32", components=32,
                     anisotropic=False, init="kmeans++", seed=20250910),
    "small": Workload("small", 2, 8, 8, 8192, 64, 64, 128, 8, components=256,
                      rope_theta=1.0e4, seed=20250911),
    "gqa1b": Workload("gqa1b", 1, 32, 8, 16384, 64, 128, 256, 16, components=512,
                      rope_theta=5.0e5, student_t_nu=4.0, seed=20250912),
    "headline": Workload("headline", 1, 16, 16, 65536, 128, 256, 1024, 32, components=1024,
                         rope_theta=5.0e5, seed=20250913),
    # the configuration of the paper's runtime comparison (Section "Experiments", Table 1): 64 heads of
    # dimension 64, two sequences of 64k tokens, 128 query and 128 key clusters, 8 retrieved clusters, 8k blocks
    "paper1b": Workload("paper1b", 2, 64, 64, 65536, 64, 128, 128, 8, components=128,
                        rope_theta=5.0e5, seed=20250915),
    "gqa8b": Workload("gqa8b", 1, 32, 8, 131072, 128, 512, 2048, 32, components=2048,
                      rope_theta=5.0e5, student_t_nu=4.0, outlier_frac=0.01, seed=20250914),
}


def round_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 (ties to even); result stays float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    u = (u + 0x7FFF + lsb) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(x.shape)


def rope(x: np.ndarray, theta: float) -> np.ndarray:
    """Rotary position encoding, rotate-half convention, positions 0..N-1.  x: [N, D] float32."""
    N, D = x.shape
    half = D // 2
    inv = theta ** (-np.arange(half, dtype=np.float64) / half)
    ang = np.arange(N, dtype=np.float64)[:, None] * inv[None, :]
    c, s = np.cos(ang), np.sin(ang)
    x1, x2 = x[:, :half].astype(np.float64), x[:, half:].astype(np.float64)
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=1).astype(np.float32)


def _mixture(rng: np.random.Generator, w: Workload) -> np.ndarray:
    """One head's [N, D] draw from the workload's Gaussian mixture."""
    N, D, M = w.N, w.D, w.components
    centres = rng.standard_normal((M, D)) / math.sqrt(D)
    z = rng.integers(0, M, size=N)
    xi = rng.standard_normal((N, D))
    if w.student_t_nu:
        chi2 = rng.chisquare(w.student_t_nu, size=N)
        xi = xi * np.sqrt(w.student_t_nu / chi2)[:, None]
    if w.anisotropic:
        lam = np.exp(rng.uniform(math.log(0.1), math.log(1.0), size=(M, D)))
        rot, _ = np.linalg.qr(rng.standard_normal((D, D)))
        eps = (xi * np.sqrt(lam[z] / D)) @ rot.T
    else:
        eps = xi * (0.3 / math.sqrt(D))
    return (centres[z] + eps).astype(np.float32)


def make_head_inputs(w: Workload, b: int, h: int, *, gain: float = 1.0):
    """Q (query head h), K, V (the kv head that h maps to), dO for one (batch, head).

    Returns float32 arrays [N, D] whose values are exactly representable in the
    workload's dtype.  `gain` multiplies Q (a power of two keeps bf16 exactness);
    gain > 1 makes attention sharp, as in trained models, so that selection and
    retrieval matter."""
    g = h * w.Hkv // w.Hq
    def stream(kind: int, head: int) -> np.random.Generator:
        return np.random.default_rng([w.seed, kind, b, head])
    Q = _mixture(stream(0, h), w)
    K = _mixture(stream(1, g), w)
    if w.rope_theta:
        Q = rope(Q, w.rope_theta)
        K = rope(K, w.rope_theta)
    if w.outlier_frac > 0:
        r = stream(4, g)
        idx = r.choice(w.N, size=max(1, int(round(w.outlier_frac * w.N))), replace=False)
        K[idx] *= w.outlier_scale
    V = stream(2, g).standard_normal((w.N, w.D)).astype(np.float32)
    dO = stream(3, h).standard_normal((w.N, w.D)).astype(np.float32)
    Q = Q * np.float32(gain)
    if w.dtype == "bf16":
        Q, K, V, dO = (round_bf16(a) for a in (Q, K, V, dO))
    return Q, K, V, dO


def make_inputs(w: Workload, *, gain: float = 1.0):
    """Whole-workload tensors: Q, dO [B,Hq,N,D]; K, V [B,Hkv,N,D] (float32 values)."""
    Q = np.empty((w.B, w.Hq, w.N, w.D), np.float32)
    dO = np.empty_like(Q)
    K = np.empty((w.B, w.Hkv, w.N, w.D), np.float32)
    V = np.empty_like(K)
    per = w.Hq // w.Hkv
    for b in range(w.B):
        for h in range(w.Hq):
            q, k, v, do = make_head_inputs(w, b, h, gain=gain)
            Q[b, h], dO[b, h] = q, do
            if h % per == 0:
                K[b, h // per], V[b, h // per] = k, v
    return Q, K, V, dO


def random_init_indices(N: int, C: int, seed: int, stream: int) -> np.ndarray:
    """C distinct seeded start indices (int32) for Lloyd's algorithm."""
    rng = np.random.default_rng([seed, 7, stream])
    return np.sort(rng.choice(N, size=C, replace=False)).astype(np.int32)


def kmeanspp_indices(X: np.ndarray, C: int, seed: int, stream: int) -> np.ndarray:
    """Plain (non-greedy) k-means++ seeding in float64; returns C start indices.

    This is harness-side input preparation: the indices are handed to both the
    oracle and the CUDA path, so its random draws never enter their comparison."""
    X = np.asarray(X, np.float64)
    N = X.shape[0]
    rng = np.random.default_rng([seed, 11, stream])
    idx = [int(rng.integers(0, N))]
    d2 = ((X - X[idx[0]]) ** 2).sum(1)
    for _ in range(1, C):
        tot = d2.sum()
        if tot <= 0:
            cand = np.setdiff1d(np.arange(N), np.array(idx))
            nxt = int(cand[0])
        else:
            cdf = np.cumsum(d2)
            nxt = int(min(np.searchsorted(cdf, rng.random() * tot, side="right"), N - 1))
        idx.append(nxt)
        d2 = np.minimum(d2, ((X - X[nxt]) ** 2).sum(1))
    return np.asarray(idx, np.int32)
