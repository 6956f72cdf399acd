"""Thin ctypes binding of libmuse.so: argument marshalling only.

Function names and argument order mirror include/muse.h.  Tensors are torch CUDA tensors
(torch is used for device memory and streams only); every step of the computation runs in
the library's CUDA kernels.  There is no CPU fallback: a missing library raises.
"""
from __future__ import annotations

import ctypes
import math
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# MUSE_LIBRARY names another build of the same sources beside this file (the bounds-checked libmuse_debug.so)
LIB_PATH = os.path.join(_HERE, os.path.basename(os.environ.get("MUSE_LIBRARY", "libmuse.so")))

MUSE_BF16, MUSE_F32 = 0, 1
MUSE_SEL_PER_QUERY, MUSE_SEL_PER_QCLUSTER = 0, 1
MUSE_INIT_INDICES, MUSE_INIT_STRIDED, MUSE_INIT_CENTRES, MUSE_INIT_KMEANSPP = 0, 1, 2, 3

EXPORTS = ("muse_workspace_bytes", "muse_summaries_layout", "muse_cluster", "muse_summarize",
           "muse_attn_fwd", "muse_attn_bwd", "muse_stream_workspace_bytes", "muse_stream_kmeans", "muse_balanced_assign",
           "muse_kmeanspp_init", "muse_dipole_layout", "muse_dipole_tilt_point",
           "muse_cluster_streaming", "muse_cluster_noalloc", "muse_cluster_noalloc_max_bytes",
           "muse_cluster_noalloc_status_copy", "muse_status_copy", "muse_test_force_paths",
           "muse_test_wait_timeout", "muse_debug_report", "muse_profile", "muse_profile_report", "muse_strerror")

# bits of muse_test_force_paths
FORCE_SUMM_FWD_SIMT, FORCE_FAR_SIMT, FORCE_SUMM_BWD_SIMT, FORCE_RET_FWD_STREAM = 1, 2, 4, 8
FORCE_RET_BWD_SPLIT, FORCE_DIPOLE_SIMT, FORCE_BLOCK_SELECT_WARP = 16, 32, 64


class MuseParams(ctypes.Structure):
    """Mirror of muse_params_t."""
    _fields_ = [
        ("B", ctypes.c_int32), ("Hq", ctypes.c_int32), ("Hkv", ctypes.c_int32), ("N", ctypes.c_int32),
        ("D", ctypes.c_int32), ("Cq", ctypes.c_int32), ("Ck", ctypes.c_int32), ("m", ctypes.c_int32),
        ("causal", ctypes.c_int32), ("n_blocks", ctypes.c_int32), ("k2", ctypes.c_int32),
        ("dtype", ctypes.c_int32), ("softmax_scale", ctypes.c_float), ("kmeans_iters", ctypes.c_int32),
        ("init_mode", ctypes.c_int32), ("seed", ctypes.c_uint64), ("sel_mode", ctypes.c_int32),
        ("dipole", ctypes.c_int32), ("agg_grad", ctypes.c_int32), ("head_map", ctypes.POINTER(ctypes.c_int32)),
    ]

    @property
    def S(self) -> int:
        return (self.n_blocks or 8) if self.causal else 1

    @property
    def SB(self) -> int:
        return self.S - 1 if self.causal else 1

    @property
    def sigma(self) -> float:
        return self.softmax_scale if self.softmax_scale > 0 else 1.0 / math.sqrt(self.D)


def make_params(*, B, Hq, Hkv, N, D, Cq, Ck, m, causal=True, n_blocks=8, dtype="bf16", softmax_scale=0.0,
                kmeans_iters=3, init_mode=MUSE_INIT_INDICES, seed=0, sel_mode=MUSE_SEL_PER_QUERY,
                agg_grad=True, head_map=None, k2=0, dipole=0) -> MuseParams:
    p = MuseParams(B=B, Hq=Hq, Hkv=Hkv, N=N, D=D, Cq=Cq, Ck=Ck, m=m, causal=int(causal), n_blocks=n_blocks,
                   k2=k2, dtype=MUSE_F32 if dtype in ("f32", torch.float32) else MUSE_BF16,
                   softmax_scale=softmax_scale, kmeans_iters=kmeans_iters, init_mode=init_mode, seed=seed,
                   sel_mode=sel_mode, dipole=dipole, agg_grad=int(agg_grad))
    if head_map is not None:
        arr = (ctypes.c_int32 * Hq)(*[int(x) for x in head_map])
        p._head_map_keepalive = arr
        p.head_map = ctypes.cast(arr, ctypes.POINTER(ctypes.c_int32))
    return p


_lib = None


def lib() -> ctypes.CDLL:
    """Loads libmuse.so (once).  Raises if it has not been built: there is no fallback."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2509_10406_b200.build`")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32p, f32p, sz = ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t
        pp = ctypes.POINTER(MuseParams)
        L.muse_strerror.restype = ctypes.c_char_p
        L.muse_strerror.argtypes = [ctypes.c_int]
        L.muse_workspace_bytes.argtypes = [pp, ctypes.POINTER(sz)]
        L.muse_summaries_layout.argtypes = [pp, ctypes.POINTER(sz)]
        L.muse_cluster.argtypes = [pp, vp, vp, i32p, i32p, i32p, i32p, f32p, f32p, vp, sz, vp]
        L.muse_summarize.argtypes = [pp, vp, vp, i32p, f32p, i32p, i32p, i32p, f32p, f32p, vp, vp, sz, vp]
        L.muse_attn_fwd.argtypes = [pp, vp, vp, vp, i32p, f32p, i32p, i32p, vp, i32p, i32p, vp, f32p, i32p, i32p, vp, sz, vp]
        L.muse_attn_bwd.argtypes = [pp, vp, vp, vp, vp, f32p, vp, i32p, f32p, i32p, i32p, vp, i32p, i32p, vp, vp, vp,
                                    vp, sz, vp]
        fl, ci = ctypes.c_float, ctypes.c_int
        L.muse_stream_workspace_bytes.argtypes = [pp, ctypes.POINTER(sz)]
        L.muse_stream_kmeans.argtypes = [pp, vp, ci, fl, ci, ci, f32p, f32p, f32p, i32p, vp, sz, vp]
        L.muse_balanced_assign.argtypes = [pp, vp, ci, f32p, fl, i32p, vp, sz, vp]
        L.muse_cluster_streaming.argtypes = [pp, vp, vp, fl, fl, i32p, i32p, f32p, f32p, vp, sz, vp]
        L.muse_cluster_noalloc.argtypes = [pp, vp, vp, i32p, i32p, i32p, i32p, f32p, f32p, vp]
        L.muse_cluster_noalloc_max_bytes.argtypes = []
        L.muse_cluster_noalloc_status_copy.argtypes = [vp, vp]
        L.muse_status_copy.argtypes = [vp, vp, vp]
        L.muse_test_force_paths.argtypes = [ctypes.c_uint]
        L.muse_test_wait_timeout.argtypes = [vp, ctypes.c_uint, vp]
        L.muse_debug_report.argtypes = [ctypes.c_char_p, sz, ctypes.c_int]
        L.muse_profile.argtypes = [ctypes.c_int]
        L.muse_profile_report.argtypes = [ctypes.c_char_p, sz]
        for name in EXPORTS[:-1]:
            getattr(L, name).restype = ctypes.c_int
        L.muse_profile_report.restype = ctypes.c_long
        L.muse_cluster_noalloc_max_bytes.restype = ctypes.c_size_t
        _lib = L
    return _lib


class MuseError(RuntimeError):
    pass


def _check(rc: int, what: str) -> None:
    if rc != 0:
        raise MuseError(f"{what}: {lib().muse_strerror(rc).decode()} ({rc})")


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "tensors must be contiguous CUDA tensors"
    return ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def muse_workspace_bytes(p: MuseParams):
    """(cluster, summarize, attn_fwd, attn_bwd, summaries, attn_bwd without stored summaries) sizes in bytes."""
    out = (ctypes.c_size_t * 6)()
    _check(lib().muse_workspace_bytes(ctypes.byref(p), out), "muse_workspace_bytes")
    return tuple(int(x) for x in out)


def muse_profile(enable: bool) -> None:
    _check(lib().muse_profile(int(enable)), "muse_profile")


def muse_profile_report() -> dict:
    """{kernel name: (launches, total ms)} since muse_profile(True)."""
    buf = ctypes.create_string_buffer(1 << 16)
    n = lib().muse_profile_report(buf, len(buf))
    if n < 0:
        _check(int(n), "muse_profile_report")
    out = {}
    for line in buf.value.decode().splitlines():
        name, launches, ms = line.split()
        out[name] = (int(launches), float(ms))
    return out


def muse_summaries_layout(p: MuseParams):
    """Byte offsets (mu, beta, kappa, kappa_lo, nu, K bucketed, V bucketed, dipole matrices, per-block set)."""
    out = (ctypes.c_size_t * 9)()
    _check(lib().muse_summaries_layout(ctypes.byref(p), out), "muse_summaries_layout")
    return tuple(int(x) for x in out)


def muse_cluster(p, Q, K, init_q, init_k, assign_q, assign_k, qbar, kcent, ws):
    _check(lib().muse_cluster(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(init_q), _ptr(init_k), _ptr(assign_q),
                              _ptr(assign_k), _ptr(qbar), _ptr(kcent), _ptr(ws), ws.numel() * ws.element_size(),
                              _stream()), "muse_cluster")


def muse_cluster_noalloc(p, Q, K, init_q, init_k, assign_q, assign_k, qbar, kcent):
    """muse_cluster on the library's built-in 32 MiB scratch: no workspace argument, no device
    allocation.  For callers that may not allocate (see include/muse.h); raises MuseError with
    'workspace too small' when the problem needs more scratch than the built-in array holds.
    Calls that overlap on the GPU share the array and must be serialised by the caller."""
    _check(lib().muse_cluster_noalloc(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(init_q), _ptr(init_k), _ptr(assign_q),
                                      _ptr(assign_k), _ptr(qbar), _ptr(kcent), _stream()), "muse_cluster_noalloc")


def muse_cluster_noalloc_max_bytes() -> int:
    return int(lib().muse_cluster_noalloc_max_bytes())


def muse_summarize(p, K, V, assign_k, qbar, off_k, perm_k, summaries, ws, counts=None, ksum=None, vsum=None):
    _check(lib().muse_summarize(ctypes.byref(p), _ptr(K), _ptr(V), _ptr(assign_k), _ptr(qbar), _ptr(off_k),
                                _ptr(perm_k), _ptr(counts), _ptr(ksum), _ptr(vsum), _ptr(summaries), _ptr(ws),
                                ws.numel() * ws.element_size(), _stream()), "muse_summarize")


def muse_status(ws) -> int:
    """Status word 0 of a workspace after the stream has drained (0 = every kernel of the last call
    that used `ws` ran to completion; otherwise a MUSE_STATUS_* code)."""
    out = torch.zeros(1, dtype=torch.int32, device=ws.device)
    _check(lib().muse_status_copy(_ptr(ws), _ptr(out), _stream()), "muse_status_copy")
    return int(out.item())


def muse_stream_workspace_bytes(p) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().muse_stream_workspace_bytes(ctypes.byref(p), ctypes.byref(out)), "muse_stream_workspace_bytes")
    return int(out.value)


def muse_stream_kmeans(p, X, side, totals, counts, centres, ws, beta=0.9, first_batch=0, n_batches=-1, assign_stream=None):
    _check(lib().muse_stream_kmeans(ctypes.byref(p), _ptr(X), int(side), float(beta), int(first_batch), int(n_batches),
                                    _ptr(totals), _ptr(counts), _ptr(centres), _ptr(assign_stream), _ptr(ws),
                                    ws.numel() * ws.element_size(), _stream()), "muse_stream_kmeans")


def muse_dipole_layout(p):
    """Byte offsets (cbar, cov, pw, zall, qstar) of the dipole arrays inside the summaries buffer."""
    off = (ctypes.c_size_t * 5)()
    _check(lib().muse_dipole_layout(ctypes.byref(p), off), "muse_dipole_layout")
    return [int(x) for x in off]


def muse_dipole_tilt_point(p, assign_q, qbar, summaries):
    _check(lib().muse_dipole_tilt_point(ctypes.byref(p), _ptr(assign_q), _ptr(qbar), _ptr(summaries), _stream()),
           "muse_dipole_tilt_point")


def muse_kmeanspp_init(p, X, side, idx_out, ws):
    _check(lib().muse_kmeanspp_init(ctypes.byref(p), _ptr(X), int(side), _ptr(idx_out), _ptr(ws),
                                    ws.numel() * ws.element_size(), _stream()), "muse_kmeanspp_init")


def muse_balanced_assign(p, X, side, centres, assign, ws, cap_factor=4.0):
    _check(lib().muse_balanced_assign(ctypes.byref(p), _ptr(X), int(side), _ptr(centres), float(cap_factor), _ptr(assign),
                                      _ptr(ws), ws.numel() * ws.element_size(), _stream()), "muse_balanced_assign")


def muse_cluster_streaming(p, Q, K, assign_q, assign_k, qbar, kcent, ws, beta=0.9, cap_factor=4.0):
    _check(lib().muse_cluster_streaming(ctypes.byref(p), _ptr(Q), _ptr(K), float(beta), float(cap_factor), _ptr(assign_q),
                                        _ptr(assign_k), _ptr(qbar), _ptr(kcent), _ptr(ws), ws.numel() * ws.element_size(),
                                        _stream()), "muse_cluster_streaming")


def muse_cluster_noalloc_status() -> int:
    out = torch.zeros(1, dtype=torch.int32, device="cuda")
    _check(lib().muse_cluster_noalloc_status_copy(_ptr(out), _stream()), "muse_cluster_noalloc_status_copy")
    return int(out.item())


def muse_debug_report(reset: bool = True):
    """(files with an out-of-range index, text) of a bounds-checked build; (MUSE_ERR_UNSUPPORTED, "") for the product build."""
    buf = ctypes.create_string_buffer(4096)
    n = lib().muse_debug_report(buf, 4096, int(reset))
    return n, buf.value.decode()


def muse_test_force_paths(mask: int) -> None:
    _check(lib().muse_test_force_paths(int(mask)), "muse_test_force_paths")


def muse_test_wait_timeout(ws, limit_clocks: int) -> None:
    _check(lib().muse_test_wait_timeout(_ptr(ws), int(limit_clocks), _stream()), "muse_test_wait_timeout")


def muse_attn_fwd(p, Q, K, V, assign_q, qbar, off_k, perm_k, summaries, sel_in, O, LSE, sel_out, ws, bsel_in=None,
                  bsel_out=None):
    _check(lib().muse_attn_fwd(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(assign_q), _ptr(qbar), _ptr(off_k),
                               _ptr(perm_k), _ptr(summaries), _ptr(sel_in), _ptr(bsel_in), _ptr(O), _ptr(LSE), _ptr(sel_out),
                               _ptr(bsel_out), _ptr(ws), ws.numel() * ws.element_size(), _stream()), "muse_attn_fwd")


def muse_attn_bwd(p, Q, K, V, O, LSE, dO, assign_q, qbar, off_k, perm_k, summaries, sel, dQ, dK, dV, ws, bsel=None):
    _check(lib().muse_attn_bwd(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(LSE), _ptr(dO),
                               _ptr(assign_q), _ptr(qbar), _ptr(off_k), _ptr(perm_k), _ptr(summaries), _ptr(sel), _ptr(bsel),
                               _ptr(dQ), _ptr(dK), _ptr(dV), _ptr(ws), ws.numel() * ws.element_size(), _stream()),
           "muse_attn_bwd")


# ---------------------------------------------------------------------------------------------
# Buffer plumbing (allocation only)
# ---------------------------------------------------------------------------------------------

class MuseBuffers:
    """Owns the device buffers one layer call needs (outputs, intermediates, workspaces)."""

    def __init__(self, p: MuseParams, device="cuda", backward=True):
        self.p = p
        dt = torch.float32 if p.dtype == MUSE_F32 else torch.bfloat16
        i32, f32 = torch.int32, torch.float32
        B, Hq, Hkv, N, D, m = p.B, p.Hq, p.Hkv, p.N, p.D, p.m
        sizes = muse_workspace_bytes(p)
        e = lambda *s, dtype: torch.empty(*s, dtype=dtype, device=device)
        self.assign_q = e(B, Hq, N, dtype=i32); self.assign_k = e(B, Hkv, N, dtype=i32)
        self.qbar = e(B, Hq, p.Cq, D, dtype=f32); self.kcent = e(B, Hkv, p.Ck, D, dtype=f32)
        self.off_k = e(B, Hkv, p.Ck * p.S + 1, dtype=i32); self.perm_k = e(B, Hkv, N, dtype=i32)
        self.summaries = e(sizes[4], dtype=torch.uint8)
        self.O = e(B, Hq, N, D, dtype=dt); self.LSE = e(B, Hq, N, dtype=f32)
        self.sel = e(B, Hq, N, max(m, 1), dtype=i32)
        self.bsel = e(B, Hq, N, max(m, 1), max(p.k2, 1), dtype=i32) if p.k2 > 0 else None
        need = max(sizes[:3] + ((sizes[3],) if backward else ()))
        self.sizes = sizes
        self.ws = e(need, dtype=torch.uint8)
        if backward:
            self.dQ = e(B, Hq, N, D, dtype=dt); self.dK = e(B, Hkv, N, D, dtype=dt); self.dV = e(B, Hkv, N, D, dtype=dt)

    def summary_planes(self):
        """(mu, beta, kappa, nu) of the accumulated summaries as fp32 tensors
        [B,Hq,SB,Cq,Ck(,D)]; in bf16 mode kappa is rebuilt as hi + lo."""
        p = self.p
        off = muse_summaries_layout(p)
        ent = p.B * p.Hq * p.SB * p.Cq * p.Ck
        shp = (p.B, p.Hq, p.SB, p.Cq, p.Ck)
        f32 = lambda o, n: self.summaries[o:o + 4 * n].view(torch.float32)
        b16 = lambda o, n: self.summaries[o:o + 2 * n].view(torch.bfloat16).float()
        mu, beta = f32(off[0], ent).view(shp), f32(off[1], ent).view(shp)
        if p.dtype == MUSE_F32:
            ka, nu = f32(off[2], ent * p.D), f32(off[4], ent * p.D)
        else:
            ka, nu = b16(off[2], ent * p.D) + b16(off[3], ent * p.D), b16(off[4], ent * p.D)
        return mu, beta, ka.view(*shp, p.D), nu.view(*shp, p.D)


def muse_layer_forward(p, buf: MuseBuffers, Q, K, V, init_q=None, init_k=None, sel_in=None):
    """cluster -> summarize -> attention forward on the current stream."""
    muse_cluster(p, Q, K, init_q, init_k, buf.assign_q, buf.assign_k, buf.qbar, buf.kcent, buf.ws)
    if p.dipole == 2:
        muse_dipole_tilt_point(p, buf.assign_q, buf.qbar, buf.summaries)
    muse_summarize(p, K, V, buf.assign_k, buf.qbar, buf.off_k, buf.perm_k, buf.summaries, buf.ws)
    muse_attn_fwd(p, Q, K, V, buf.assign_q, buf.qbar, buf.off_k, buf.perm_k, buf.summaries, sel_in, buf.O, buf.LSE,
                  buf.sel, buf.ws, bsel_out=buf.bsel)
    return buf.O


def muse_layer_backward(p, buf: MuseBuffers, Q, K, V, dO, sel=None):
    muse_attn_bwd(p, Q, K, V, buf.O, buf.LSE, dO, buf.assign_q, buf.qbar, buf.off_k, buf.perm_k, buf.summaries,
                  buf.sel if sel is None else sel, buf.dQ, buf.dK, buf.dV, buf.ws, bsel=buf.bsel)
    return buf.dQ, buf.dK, buf.dV
