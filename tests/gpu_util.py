"""Helpers for the GPU parity tests: build a synthetic case, run the oracle on it (numpy fp64,
per head) and hand identical bits to the CUDA library."""
from __future__ import annotations

import numpy as np
import torch

from oracle import muse_oracle as orc
from paper_2509_10406_b200 import workloads as wl


def tol(dtype: str) -> float:
    """max-abs error relative to the oracle tensor's max-abs: 1e-4 (fp32 mode), 2e-2 (bf16 mode)."""
    return 1e-4 if dtype == "f32" else 2e-2


def rel_err(x: np.ndarray, ref: np.ndarray) -> float:
    return float(np.abs(x - ref).max() / max(np.abs(ref).max(), 1e-30))


def to_dev(x: np.ndarray, dtype: str) -> torch.Tensor:
    """dtype "bf16" converts float32 values (already bf16-exact) to bfloat16; anything else keeps the array type."""
    t = torch.from_numpy(np.ascontiguousarray(x))
    if t.dtype == torch.float32 and dtype == "bf16":
        t = t.to(torch.bfloat16)
    return t.cuda()


def to_np(t: torch.Tensor) -> np.ndarray:
    t = t.detach().cpu()
    if t.dtype == torch.bfloat16:
        t = t.float()
    return t.numpy()


class Case:
    """Inputs of one workload plus oracle clustering (per head), ready for teacher forcing."""

    def __init__(self, w: wl.Workload, gain: float = 1.0, cluster: bool = True):
        self.w = w
        self.Q, self.K, self.V, self.dO = wl.make_inputs(w, gain=gain)
        self.sigma = 1.0 / np.sqrt(w.D)
        self.hm = [h * w.Hkv // w.Hq for h in range(w.Hq)]
        B, Hq, Hkv = w.B, w.Hq, w.Hkv
        self.init_q = np.zeros((B, Hq, w.Cq), np.int32); self.init_k = np.zeros((B, Hkv, w.Ck), np.int32)
        for b in range(B):
            for h in range(Hq):
                self.init_q[b, h] = self._init(self.Q[b, h], w.Cq, (b * Hq + h) * 2)
            for g in range(Hkv):
                self.init_k[b, g] = self._init(self.K[b, g], w.Ck, (b * Hkv + g) * 2 + 1)
        if cluster:
            self.a_q = np.zeros((B, Hq, w.N), np.int32); self.a_k = np.zeros((B, Hkv, w.N), np.int32)
            self.qbar = np.zeros((B, Hq, w.Cq, w.D)); self.kcent = np.zeros((B, Hkv, w.Ck, w.D))
            for b in range(B):
                for h in range(Hq):
                    self.a_q[b, h], self.qbar[b, h] = orc.lloyd(self.Q[b, h], w.T, init_idx=self.init_q[b, h])
                for g in range(Hkv):
                    self.a_k[b, g], self.kcent[b, g] = orc.lloyd(self.K[b, g], w.T, init_idx=self.init_k[b, g])

    def _init(self, X, C, stream):
        if self.w.init == "kmeans++":
            return wl.kmeanspp_indices(X, C, self.w.seed, stream)
        return wl.random_init_indices(X.shape[0], C, self.w.seed, stream)

    def params(self, **kw):
        from paper_2509_10406_b200 import binding as mb
        w = self.w
        args = dict(B=w.B, Hq=w.Hq, Hkv=w.Hkv, N=w.N, D=w.D, Cq=w.Cq, Ck=w.Ck, m=w.m, n_blocks=w.S,
                    dtype=w.dtype, kmeans_iters=w.T)
        args.update(kw)
        return mb.make_params(**args)

    def dev(self):
        d = self.w.dtype
        return to_dev(self.Q, d), to_dev(self.K, d), to_dev(self.V, d), to_dev(self.dO, d)


class kernels_launched:
    """Context manager: records the library's kernel names launched inside the block (through the
    library's own per-kernel timing hook), so that a test can assert which path ran."""

    def __enter__(self):
        from paper_2509_10406_b200 import binding as mb
        self.mb = mb
        mb.muse_profile(True)
        self.names = set()
        return self

    def __exit__(self, *exc):
        torch.cuda.synchronize()
        self.names = set(self.mb.muse_profile_report())
        self.mb.muse_profile(False)
        return False
