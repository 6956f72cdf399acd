"""GPU parity: clustering stage (muse_cluster) and bucketing, against the fp64 oracle.

Gate (per step, teacher-forced): assignments given centres are bit-exact except near-ties
(relative gap of the two smallest true squared distances below 1e-4), which are counted;
centres given assignments agree to 1e-6 relative."""
import numpy as np
import pytest
import torch

from oracle import muse_oracle as orc
from paper_2509_10406_b200 import workloads as wl
from tests.gpu_util import Case, to_dev, to_np

pytestmark = pytest.mark.gpu

CASES = {
    "tiny": wl.WORKLOADS["tiny"],
    "gqa_bf16": wl.WORKLOADS["small"].with_(B=2, Hq=4, Hkv=2, N=2000, Cq=16, Ck=40, m=6, components=64),
    "d128": wl.WORKLOADS["headline"].with_(Hq=2, Hkv=1, N=3072, Cq=24, Ck=128, m=8, components=96),
    "d128_wide": wl.WORKLOADS["headline"].with_(name="headline_wide", Hq=1, Hkv=1, N=2048, Cq=4, Ck=256, m=16, components=64),
    # D = 64 with C_k a multiple of 128: the shapes at which the D = 64 instances of the tensor-core far-field kernels run
    "d64": wl.WORKLOADS["small"].with_(name="small_d64", B=1, Hq=2, Hkv=1, N=3072, Cq=24, Ck=128, m=8, components=96),
}


def _mb():
    from paper_2509_10406_b200 import binding as mb
    return mb


@pytest.mark.parametrize("name", list(CASES))
@pytest.mark.parametrize("gain", [1.0, 128.0])
def test_assign_and_update_teacher_forced(name, gain):
    mb = _mb()
    c = Case(CASES[name], gain=gain)
    w = c.w
    Q, K, V, _ = c.dev()
    # start centres: fp32 values shared by both sides
    cq0 = np.stack([[c.Q[b, h][c.init_q[b, h]] for h in range(w.Hq)] for b in range(w.B)]).astype(np.float32)
    ck0 = np.stack([[c.K[b, g][c.init_k[b, g]] for g in range(w.Hkv)] for b in range(w.B)]).astype(np.float32)
    outs = {}
    for T in (0, 1):
        p = c.params(kmeans_iters=T, init_mode=mb.MUSE_INIT_CENTRES)
        buf = mb.MuseBuffers(p, backward=False)
        buf.qbar.copy_(torch.from_numpy(cq0)); buf.kcent.copy_(torch.from_numpy(ck0))
        mb.muse_cluster(p, Q, K, None, None, buf.assign_q, buf.assign_k, buf.qbar, buf.kcent, buf.ws)
        torch.cuda.synchronize()
        outs[T] = (to_np(buf.assign_q), to_np(buf.assign_k), to_np(buf.qbar), to_np(buf.kcent))
    near = total = 0
    for X, c0, a0, c1, a1 in ((c.Q, cq0, outs[0][0], outs[1][2], outs[1][0]), (c.K, ck0, outs[0][1], outs[1][3], outs[1][1])):
        for b in range(X.shape[0]):
            for h in range(X.shape[1]):
                # assign | centres
                exp = orc.assign_nearest(X[b, h], c0[b, h])
                gaps = orc.assignment_gaps(X[b, h], c0[b, h])
                bad = np.nonzero(exp != a0[b, h])[0]
                assert np.all(gaps[bad] < 1e-4), (name, "assignment differs away from a near-tie", gaps[bad].max())
                near += bad.size; total += exp.size
                # update | assignment (the GPU's own a0, so both sides average the same members)
                c1_exp = orc.update_centres(X[b, h], a0[b, h], c0[b, h])
                assert np.abs(c1[b, h] - c1_exp).max() <= 1e-6 * np.abs(c1_exp).max()
                # final assign | updated centres
                exp1 = orc.assign_nearest(X[b, h], c1[b, h])
                gaps1 = orc.assignment_gaps(X[b, h], c1[b, h])
                bad1 = np.nonzero(exp1 != a1[b, h])[0]
                assert np.all(gaps1[bad1] < 1e-4)
                near += bad1.size; total += exp1.size
    print(f"[{name} gain={gain}] near-tie assignment differences: {near} of {total}")
    assert near <= max(2, 2e-3 * total)


def test_lloyd_free_running_tiny():
    mb = _mb()
    c = Case(CASES["tiny"])
    w = c.w
    Q, K, V, _ = c.dev()
    p = c.params()
    buf = mb.MuseBuffers(p, backward=False)
    mb.muse_cluster(p, Q, K, to_dev(c.init_q, "i"), to_dev(c.init_k, "i"), buf.assign_q, buf.assign_k, buf.qbar,
                    buf.kcent, buf.ws)
    torch.cuda.synchronize()
    assert mb.muse_status(buf.ws) == 0
    aq, ak = to_np(buf.assign_q), to_np(buf.assign_k)
    ndiff = int((aq != c.a_q).sum() + (ak != c.a_k).sum())
    print("free-running Lloyd: differing assignments", ndiff, "of", aq.size + ak.size)
    assert ndiff < 0.01 * (aq.size + ak.size)
    if ndiff == 0:
        # same trajectory on both sides: the centres are the same member means
        assert np.abs(to_np(buf.qbar) - c.qbar).max() <= 1e-5 * np.abs(c.qbar).max()
        assert np.abs(to_np(buf.kcent) - c.kcent).max() <= 1e-5 * np.abs(c.kcent).max()
    # whatever the trajectory, the result is a fixed point of its own last step: every point sits in the
    # cluster nearest to the returned centres (near-ties excepted) ...
    for X, a, cen in ((c.Q[0, 0], aq[0, 0], to_np(buf.qbar)[0, 0]), (c.K[0, 0], ak[0, 0], to_np(buf.kcent)[0, 0])):
        exp = orc.assign_nearest(X, cen.astype(np.float64))
        bad = np.nonzero(exp != a)[0]
        assert np.all(orc.assignment_gaps(X, cen.astype(np.float64))[bad] < 1e-4)
    # ... and its k-means objective is within a hair of the oracle trajectory's
    inertia = lambda X, a, cen: float(((X - cen[a]) ** 2).sum())
    for X, a, cen, a0, cen0 in ((c.Q[0, 0], aq[0, 0], to_np(buf.qbar)[0, 0], c.a_q[0, 0], c.qbar[0, 0]),
                                (c.K[0, 0], ak[0, 0], to_np(buf.kcent)[0, 0], c.a_k[0, 0], c.kcent[0, 0])):
        assert abs(inertia(X, a, cen) - inertia(X, a0, cen0)) <= 1e-2 * inertia(X, a0, cen0)


def test_nan_and_infinite_rows_get_a_valid_cluster():
    """A row of NaN or infinities (a diverged training step) compares below no running minimum: the
    assignment kernels must still write an index inside [0, C), and the later stages must run without a
    CUDA error on such an assignment."""
    mb = _mb()
    for name in ("tiny", "d128"):
        c = Case(CASES[name], cluster=False)
        w = c.w
        c.Q[0, 0, 5] = np.nan; c.K[0, 0, 7] = np.inf; c.K[0, 0, 9] = np.nan
        Q, K, V, _ = c.dev()
        p = c.params()
        buf = mb.MuseBuffers(p, backward=False)
        mb.muse_cluster(p, Q, K, to_dev(c.init_q, "i"), to_dev(c.init_k, "i"), buf.assign_q, buf.assign_k, buf.qbar,
                        buf.kcent, buf.ws)
        torch.cuda.synchronize()
        aq, ak = to_np(buf.assign_q), to_np(buf.assign_k)
        assert aq.min() >= 0 and aq.max() < w.Cq and ak.min() >= 0 and ak.max() < w.Ck
        mb.muse_summarize(p, K, V, buf.assign_k, buf.qbar, buf.off_k, buf.perm_k, buf.summaries, buf.ws)
        torch.cuda.synchronize()
        perm = to_np(buf.perm_k)
        assert all(np.array_equal(np.sort(perm[b, g]), np.arange(w.N)) for b in range(w.B) for g in range(w.Hkv))


def test_out_of_range_assignments_from_the_caller_are_pinned():
    mb = _mb()
    c = Case(CASES["gqa_bf16"])
    w = c.w
    Q, K, V, _ = c.dev()
    a_k = c.a_k.copy()
    a_k[0, 0, 3] = 0x7fffffff; a_k[0, 0, 4] = -5; a_k[1, 1, 11] = w.Ck
    p = c.params()
    buf = mb.MuseBuffers(p, backward=False)
    mb.muse_summarize(p, K, V, to_dev(a_k, "i"), to_dev(c.qbar.astype(np.float32), "f32"), buf.off_k, buf.perm_k,
                      buf.summaries, buf.ws)
    torch.cuda.synchronize()
    pinned = np.clip(a_k.astype(np.int64), 0, w.Ck - 1)
    Bs = w.N // w.S
    for b in range(w.B):
        for g in range(w.Hkv):
            key = pinned[b, g] * w.S + np.arange(w.N) // Bs
            assert np.array_equal(to_np(buf.perm_k)[b, g], np.argsort(key, kind="stable"))


def test_bounded_wait_reports_through_the_status_word():
    """A wait that can never be satisfied (nothing arrives at its barrier) runs out after the given number
    of clocks; the kernel then returns, word 0 of the workspace carries the code, and the context is usable."""
    mb = _mb()
    ws = torch.empty(4096, dtype=torch.uint8, device="cuda")
    mb.muse_test_wait_timeout(ws, 200000)
    torch.cuda.synchronize()
    assert mb.muse_status(ws) == 9
    assert float(torch.ones(8, device="cuda").sum().item()) == 8.0


def test_strided_init_matches_integer_spec():
    mb = _mb()
    c = Case(CASES["gqa_bf16"], cluster=False)
    w = c.w
    Q, K, V, _ = c.dev()
    p = c.params(kmeans_iters=0, init_mode=mb.MUSE_INIT_STRIDED, seed=991)
    buf = mb.MuseBuffers(p, backward=False)
    mb.muse_cluster(p, Q, K, None, None, buf.assign_q, buf.assign_k, buf.qbar, buf.kcent, buf.ws)
    torch.cuda.synchronize()
    qb, kc = to_np(buf.qbar), to_np(buf.kcent)
    for b in range(w.B):
        for h in range(w.Hq):
            idx = orc.strided_init(w.N, w.Cq, 991, (b * w.Hq + h) * 2)
            assert np.array_equal(qb[b, h], c.Q[b, h][idx])
        for g in range(w.Hkv):
            idx = orc.strided_init(w.N, w.Ck, 991, (b * w.Hkv + g) * 2 + 1)
            assert np.array_equal(kc[b, g], c.K[b, g][idx])


@pytest.mark.parametrize("name", ["tiny", "gqa_bf16"])
def test_bucketing_is_stable_counting_sort(name):
    mb = _mb()
    c = Case(CASES[name])
    w = c.w
    Q, K, V, _ = c.dev()
    p = c.params()
    buf = mb.MuseBuffers(p, backward=False)
    mb.muse_summarize(p, K, V, to_dev(c.a_k, "i"), to_dev(c.qbar.astype(np.float32), "f32"), buf.off_k, buf.perm_k,
                      buf.summaries, buf.ws)
    torch.cuda.synchronize()
    off, perm = to_np(buf.off_k), to_np(buf.perm_k)
    Bs = w.N // w.S
    for b in range(w.B):
        for g in range(w.Hkv):
            key = c.a_k[b, g].astype(np.int64) * w.S + np.arange(w.N) // Bs
            assert np.array_equal(perm[b, g], np.argsort(key, kind="stable"))
            cnt = np.bincount(key, minlength=w.Ck * w.S)
            assert np.array_equal(off[b, g], np.concatenate([[0], np.cumsum(cnt)]))
