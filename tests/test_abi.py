"""The C-ABI library builds, loads and exports every symbol include/muse.h declares; host-side
argument checking works without a GPU (no compute is launched here)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def mb():
    from paper_2509_10406_b200 import build, binding
    build.build()
    binding.lib()
    return binding


def test_header_symbols_are_exported(mb):
    hdr = open(os.path.join(ROOT, "include", "muse.h")).read()
    declared = set(re.findall(r"MUSE_API\s+[\w\s\*]+?\b(muse_\w+)\s*\(", hdr))
    assert declared == set(mb.EXPORTS)
    lib = ctypes.CDLL(mb.LIB_PATH)
    for name in declared:
        assert getattr(lib, name) is not None


def test_params_struct_layout(mb):
    assert ctypes.sizeof(mb.MuseParams) == 96
    assert mb.MuseParams.seed.offset == 64 and mb.MuseParams.head_map.offset == 88


def test_workspace_sizes_and_layout(mb):
    p = mb.make_params(B=1, Hq=16, Hkv=16, N=65536, D=128, Cq=256, Ck=1024, m=32)
    sizes = mb.muse_workspace_bytes(p)
    ent = 16 * 7 * 256 * 1024
    assert sizes[4] >= ent * (3 * 128 * 2 + 8) + 2 * 16 * 65536 * 128 * 2
    off = mb.muse_summaries_layout(p)
    assert off[0] == 0 and off[1] >= ent * 4 and off[3] - off[2] >= ent * 128 * 2 and all(o % 256 == 0 for o in off)
    assert len(off) == 9 and list(off) == sorted(off) and off[8] == sizes[4]        # no per-block set without k2
    p2 = mb.make_params(B=1, Hq=16, Hkv=16, N=65536, D=128, Cq=256, Ck=1024, m=32, k2=1)
    off2 = mb.muse_summaries_layout(p2)
    assert mb.muse_workspace_bytes(p2)[4] - off2[8] >= ent * (3 * 128 * 2 + 8)      # the per-block set has the same size
    assert all(s % 256 == 0 for s in sizes)


@pytest.mark.parametrize("kw,code", [
    (dict(D=96), -2), (dict(m=2000), -1), (dict(N=1001), -1), (dict(Cq=0), -1), (dict(k2=9), -2), (dict(k2=1, dtype="f32"), -2),
    (dict(dipole=1, k2=1), -2), (dict(dipole=3), -1), (dict(Hq=3, Hkv=2), -1), (dict(m=65, Ck=128), -2), (dict(Ck=8192, N=16384), -2),
])
def test_invalid_parameters_are_rejected_on_the_host(mb, kw, code):
    args = dict(B=1, Hq=2, Hkv=2, N=1024, D=64, Cq=8, Ck=16, m=4)
    args.update(kw)
    p = mb.make_params(**args)
    out = (ctypes.c_size_t * 6)()
    assert mb.lib().muse_workspace_bytes(ctypes.byref(p), out) == code
    assert mb.lib().muse_strerror(code)


def test_null_and_small_workspace_are_rejected(mb):
    p = mb.make_params(B=1, Hq=1, Hkv=1, N=1024, D=64, Cq=8, Ck=16, m=4)
    L = mb.lib()
    z = ctypes.c_void_p(0)
    assert L.muse_cluster(ctypes.byref(p), z, z, z, z, z, z, z, z, z, 0, z) == -1
    fake = ctypes.c_void_p(4096)      # aligned, never dereferenced: the size check comes first
    assert L.muse_summarize(ctypes.byref(p), fake, fake, fake, fake, fake, fake, z, z, z, fake, fake, 16, z) == -3
    # the three untilted outputs come together
    assert L.muse_summarize(ctypes.byref(p), fake, fake, fake, fake, fake, fake, fake, z, z, fake, fake, 1 << 30, z) == -1
    assert L.muse_attn_fwd(ctypes.byref(p), fake, fake, fake, fake, fake, fake, fake, fake, z, z, fake, fake, z, z, fake, 16, z) == -3
    odd = ctypes.c_void_p(4100)
    assert L.muse_summarize(ctypes.byref(p), odd, fake, fake, fake, fake, fake, z, z, z, fake, fake, 1 << 30, z) == -1
    # backward without summaries needs the larger scratch
    need = mb.muse_workspace_bytes(p)
    assert need[5] == need[3] + need[4] + need[1]
    a16 = [fake] * 9
    assert L.muse_attn_bwd(ctypes.byref(p), fake, fake, fake, fake, fake, fake, fake, fake, fake, fake, z, fake, z,
                           fake, fake, fake, fake, need[3], z) == -3
    # two-level retrieval: the backward pass needs the forward's chosen blocks
    p2 = mb.make_params(B=1, Hq=1, Hkv=1, N=1024, D=64, Cq=8, Ck=16, m=4, k2=1)
    assert L.muse_attn_bwd(ctypes.byref(p2), fake, fake, fake, fake, fake, fake, fake, fake, fake, fake, fake, fake, z,
                           fake, fake, fake, fake, 1 << 40, z) == -1


def test_head_map(mb):
    p = mb.make_params(B=1, Hq=3, Hkv=2, N=1024, D=64, Cq=8, Ck=16, m=4, head_map=[0, 1, 1])
    assert len(mb.muse_workspace_bytes(p)) == 6
    p = mb.make_params(B=1, Hq=3, Hkv=2, N=1024, D=64, Cq=8, Ck=16, m=4, head_map=[0, 1, 2])
    out = (ctypes.c_size_t * 6)()
    assert mb.lib().muse_workspace_bytes(ctypes.byref(p), out) == -1


def test_streaming_clustering_entry_points_check_their_arguments(mb):
    p = mb.make_params(B=1, Hq=2, Hkv=1, N=1024, D=64, Cq=8, Ck=16, m=4)
    L = mb.lib()
    z, fake, odd = ctypes.c_void_p(0), ctypes.c_void_p(4096), ctypes.c_void_p(4100)
    need = mb.muse_stream_workspace_bytes(p)
    assert need % 256 == 0 and need > mb.muse_workspace_bytes(p)[0]          # the balanced step adds its sort and rank arrays
    assert L.muse_stream_workspace_bytes(ctypes.byref(p), None) == -1
    # muse_stream_kmeans: side in {0, 1}, beta in (0, 1], pointers present and aligned
    args = lambda **kw: [kw.get("X", fake), kw.get("side", 0), ctypes.c_float(kw.get("beta", 0.9)), kw.get("first", 0), kw.get("nb", -1),
                         kw.get("tot", fake), fake, fake, z, kw.get("ws", fake), kw.get("wsb", 1 << 20), z]
    assert L.muse_stream_kmeans(ctypes.byref(p), *args(side=2)) == -1
    assert L.muse_stream_kmeans(ctypes.byref(p), *args(beta=0.0)) == -1
    assert L.muse_stream_kmeans(ctypes.byref(p), *args(beta=1.5)) == -1
    assert L.muse_stream_kmeans(ctypes.byref(p), *args(X=z)) == -1
    assert L.muse_stream_kmeans(ctypes.byref(p), *args(tot=odd)) == -1
    assert L.muse_stream_kmeans(ctypes.byref(p), *args(wsb=16)) == -3
    # muse_balanced_assign and muse_cluster_streaming: workspace from muse_stream_workspace_bytes
    assert L.muse_balanced_assign(ctypes.byref(p), fake, 1, fake, ctypes.c_float(4.0), fake, fake, 1024, z) == -3
    assert L.muse_balanced_assign(ctypes.byref(p), fake, 3, fake, ctypes.c_float(4.0), fake, fake, need, z) == -1
    assert L.muse_cluster_streaming(ctypes.byref(p), fake, fake, ctypes.c_float(0.9), ctypes.c_float(4.0), fake, fake, fake, fake,
                                    fake, need - 256, z) == -3
    assert L.muse_cluster_streaming(ctypes.byref(p), z, z, ctypes.c_float(0.9), ctypes.c_float(4.0), z, z, z, z, fake, need, z) == -1
