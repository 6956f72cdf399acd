"""GPU parity of the paper's own clustering (Appendix "Clustering Details") against the fp64 oracle.

Streaming mini-batch k-means is a chain of dependent minibatches, so the gate is teacher-forced per step, like the
Lloyd gate: from the ORACLE's state (t, c) before a sampled minibatch the GPU runs that one minibatch; its 64
assignments are bit-exact except near-ties (relative gap of the two smallest squared distances below 1e-4), and
when they all agree the updated state agrees to 1e-5 relative.  A free-running pass is compared on separated blobs,
where no assignment is ambiguous.  The balanced assignment is compared vector by vector on inputs where the cap
binds and no vector is a near-tie."""
import numpy as np
import pytest
import torch

from oracle import muse_oracle as orc
from paper_2509_10406_b200 import workloads as wl
from tests.gpu_util import Case, to_dev, to_np, tol, rel_err, kernels_launched
from tests.test_gpu_cluster import CASES

pytestmark = pytest.mark.gpu


def _mb():
    from paper_2509_10406_b200 import binding as mb
    return mb


def _ws(mb, p):
    return torch.zeros(mb.muse_stream_workspace_bytes(p), dtype=torch.uint8, device="cuda")


# shapes that exercise the tensor-core kernel's splits: (centroids per CTA, tiles per CTA) = (128, 1) over 4 CTAs, (256, 2) over
# 2 CTAs, and ragged slices of 100 centroids over 2 CTAs
STREAM_CASES = dict(CASES)
STREAM_CASES.update({
    "tc_split4": wl.WORKLOADS["headline"].with_(name="s4", B=1, Hq=1, Hkv=1, N=1024, Cq=512, Ck=512, m=4, components=64),
    "tc_two_tiles": wl.WORKLOADS["small"].with_(name="s2", B=5, Hq=8, Hkv=8, N=1024, Cq=512, Ck=512, m=4, components=64),
    "tc_ragged": wl.WORKLOADS["headline"].with_(name="sr", B=1, Hq=2, Hkv=2, N=1000, Cq=200, Ck=200, m=4, S=4, components=64),
})


@pytest.mark.parametrize("name", ["tiny", "gqa_bf16", "d128", "tc_split4", "tc_two_tiles", "tc_ragged"])
def test_streaming_minibatch_teacher_forced(name):
    mb = _mb()
    c = Case(STREAM_CASES[name], gain=1.0, cluster=False)
    w = c.w
    p = c.params(seed=w.seed)
    ws = _ws(mb, p)
    Q, K, _, _ = c.dev()
    nb_all = (w.N + 63) // 64
    near = total = 0
    for side, X, Xd, H, C in ((0, c.Q, Q, w.Hq, w.Cq), (1, c.K, K, w.Hkv, w.Ck)):
        P = w.B * H
        orders = [orc.stream_order(w.N, w.seed, pr * 2 + side) for pr in range(P)]
        inits = [orc.strided_init(w.N, C, w.seed, pr * 2 + side) for pr in range(P)]
        Xf = X.reshape(P, w.N, w.D)
        for s in sorted({0, 1, 7 % nb_all, nb_all - 1}):
            t0 = np.zeros((P, C, w.D)); c0 = np.zeros((P, C)); exp = []
            for pr in range(P):
                _, t0[pr], c0[pr], _ = orc.streaming_kmeans(Xf[pr], C, orders[pr], inits[pr], n_batches=s)
                exp.append(orc.streaming_kmeans(Xf[pr], C, orders[pr], inits[pr], first_batch=s, n_batches=1, totals=t0[pr], counts=c0[pr]))
            tot = to_dev(t0.astype(np.float32), "f32"); cnt = to_dev(c0.astype(np.float32), "f32")
            cen = torch.zeros(P, C, w.D, device="cuda"); a_s = torch.full((P, w.N), -7, dtype=torch.int32, device="cuda")
            with kernels_launched() as rec:
                mb.muse_stream_kmeans(p, Xd, side, tot, cnt, cen, ws, beta=0.9, first_batch=s, n_batches=1, assign_stream=a_s)
            assert rec.names == ({"k_stream_kmeans"} if w.dtype == "f32" else {"k_stream_kmeans_tc"}), rec.names
            torch.cuda.synchronize()
            assert mb.muse_status(ws) == 0
            a_gpu, t_gpu, c_gpu, cen_gpu = to_np(a_s), to_np(tot), to_np(cnt), to_np(cen)
            for pr in range(P):
                lo, hi = s * 64, min(w.N, (s + 1) * 64)
                idx = orders[pr][lo:hi]
                gaps = orc.assignment_gaps(Xf[pr][idx], t0[pr] / c0[pr][:, None])
                bad = np.nonzero(a_gpu[pr, lo:hi] != exp[pr][3])[0]
                assert np.all(gaps[bad] < 1e-4), (name, side, s, "assignment differs away from a near-tie")
                assert np.all(a_gpu[pr, :lo] == -7) and np.all(a_gpu[pr, hi:] == -7)      # nothing outside the minibatch is written
                near += bad.size; total += hi - lo
                if bad.size == 0:
                    assert np.abs(t_gpu[pr] - exp[pr][1]).max() <= 1e-5 * np.abs(exp[pr][1]).max(), (name, side, s)
                    assert np.abs(c_gpu[pr] - exp[pr][2]).max() <= 1e-5 * np.abs(exp[pr][2]).max()
                    assert np.abs(cen_gpu[pr] - exp[pr][0]).max() <= 1e-5 * np.abs(exp[pr][0]).max()
    print(f"[{name}] near-tie differences {near} of {total}")
    assert near <= max(2, 5e-3 * total)


@pytest.mark.parametrize("dtype,D", [("f32", 64), ("bf16", 128)])
def test_streaming_full_pass_on_separated_blobs(dtype, D):
    mb = _mb()
    N, C, seed = 2000, 8, 11                                        # N is not a multiple of 64: the last minibatch is short
    rng = np.random.default_rng(0)
    order = orc.stream_order(N, seed, 0)
    init = orc.strided_init(N, C, seed, 0)
    label = rng.integers(0, C, size=N); label[init] = np.arange(C)
    X = (8.0 * np.eye(C, D)[label] + 0.05 * rng.normal(size=(N, D))).astype(np.float32)
    if dtype == "bf16":
        X = torch.from_numpy(X).to(torch.bfloat16).float().numpy()
    p = mb.make_params(B=1, Hq=1, Hkv=1, N=N, D=D, Cq=C, Ck=C, m=2, n_blocks=4, dtype=dtype, seed=seed)
    ws = _ws(mb, p)
    Xd = to_dev(X.reshape(1, 1, N, D), dtype)
    tot = torch.zeros(1, C, D, device="cuda"); cnt = torch.zeros(1, C, device="cuda"); cen = torch.zeros(1, C, D, device="cuda")
    a_s = torch.zeros(1, N, dtype=torch.int32, device="cuda")
    mb.muse_stream_kmeans(p, Xd, 0, tot, cnt, cen, ws, assign_stream=a_s)
    torch.cuda.synchronize()
    assert mb.muse_status(ws) == 0
    cen_o, t_o, c_o, a_o = orc.streaming_kmeans(X, C, order, init)
    assert np.array_equal(to_np(a_s)[0], a_o) and np.array_equal(a_o, label[order])
    assert rel_err(to_np(cen)[0], cen_o) <= 1e-5 and rel_err(to_np(cnt)[0], c_o) <= 1e-5 and rel_err(to_np(tot)[0], t_o) <= 1e-5
    # two calls that split the pass give the same state as one
    tot2 = torch.zeros_like(tot); cnt2 = torch.zeros_like(cnt); cen2 = torch.zeros_like(cen)
    mb.muse_stream_kmeans(p, Xd, 0, tot2, cnt2, cen2, ws, first_batch=0, n_batches=9)
    mb.muse_stream_kmeans(p, Xd, 0, tot2, cnt2, cen2, ws, first_batch=9, n_batches=-1)
    torch.cuda.synchronize()
    assert torch.equal(tot2, tot) and torch.equal(cnt2, cnt) and torch.equal(cen2, cen)


def _lattice(N, C, D, seed):
    """Integer-valued vectors and centroids, elongated along the first axis so that a few centroids attract most
    vectors.  Every |c|^2 - 2 x.c is a small integer, exact in fp32 (and in the bf16 hi/lo operands of the tensor-core
    assignment), so both sides see the same distances, exact ties included."""
    rng = np.random.default_rng(seed)
    X = rng.integers(-3, 4, size=(N, D)).astype(np.float32)
    X[:, 0] = rng.integers(-30, 31, size=N)
    cen = rng.integers(-2, 3, size=(C, D)).astype(np.float32)
    cen[:, 0] = rng.integers(-15, 16, size=C)
    return X, cen


@pytest.mark.parametrize("dtype,D,C", [("f32", 64, 16), ("bf16", 128, 128), ("bf16", 64, 40)])
def test_balanced_assignment_matches_oracle(dtype, D, C):
    mb = _mb()
    N, S = 4096, 4
    X, cen = _lattice(N, C, D, 3)
    p = mb.make_params(B=1, Hq=1, Hkv=1, N=N, D=D, Cq=C, Ck=C, m=2, n_blocks=S, dtype=dtype)
    ws = _ws(mb, p)
    Xd = to_dev(X.reshape(1, 1, N, D), dtype); cd = to_dev(cen.reshape(1, C, D), "f32")
    near = orc.assign_nearest(X, cen)
    Bs = N // S
    for factor in (1.0, 1.5, 4.0, 0.0):
        a = torch.full((1, N), -1, dtype=torch.int32, device="cuda")
        mb.muse_balanced_assign(p, Xd, 1, cd, a, ws, cap_factor=factor)
        torch.cuda.synchronize()
        assert mb.muse_status(ws) == 0
        a_gpu = to_np(a)[0]
        exp = orc.balanced_assign(X, cen, S, factor) if factor > 0 else near
        print(f"[{dtype} D={D} C={C} factor={factor}] the cap displaces {(exp != near).sum()} of {N} vectors")
        assert np.array_equal(a_gpu, exp), np.nonzero(a_gpu != exp)[0][:10]
        if factor == 1.0:
            assert (exp != near).sum() > N // 8                       # the cap binds hard in this case
            cap = orc.balanced_cap(Bs, C, factor)
            assert max(np.bincount(a_gpu[b * Bs:(b + 1) * Bs], minlength=C).max() for b in range(S)) == cap


def test_streaming_clustering_feeds_the_rest_of_the_path():
    """muse_cluster_streaming in place of muse_cluster: the forward pass with its assignments and centroids agrees with
    the oracle's forward evaluated on the same assignments and centroids."""
    mb = _mb()
    c = Case(CASES["d128"], gain=128.0, cluster=False)
    w = c.w
    p = c.params(seed=w.seed)
    buf = mb.MuseBuffers(p, backward=False)
    ws = _ws(mb, p)
    Q, K, V, _ = c.dev()
    mb.muse_cluster_streaming(p, Q, K, buf.assign_q, buf.assign_k, buf.qbar, buf.kcent, ws)
    torch.cuda.synchronize()
    assert mb.muse_status(ws) == 0
    a_q, a_k, qbar = to_np(buf.assign_q), to_np(buf.assign_k), to_np(buf.qbar)
    Bs, capq, capk = w.N // w.S, orc.balanced_cap(w.N // w.S, w.Cq, 4.0), orc.balanced_cap(w.N // w.S, w.Ck, 4.0)
    for a, C, cap in ((a_q, w.Cq, capq), (a_k, w.Ck, capk)):
        assert a.min() >= 0 and a.max() < C
        for pr in range(a.shape[0] * a.shape[1]):
            for b in range(w.S):
                assert np.bincount(a.reshape(-1, w.N)[pr, b * Bs:(b + 1) * Bs], minlength=C).max() <= cap
    mb.muse_summarize(p, K, V, buf.assign_k, buf.qbar, buf.off_k, buf.perm_k, buf.summaries, buf.ws)
    mb.muse_attn_fwd(p, Q, K, V, buf.assign_q, buf.qbar, buf.off_k, buf.perm_k, buf.summaries, None, buf.O, buf.LSE, buf.sel, buf.ws)
    torch.cuda.synchronize()
    assert mb.muse_status(buf.ws) == 0
    O, sel = to_np(buf.O), to_np(buf.sel)[..., :w.m]
    for b in range(w.B):
        for h in range(w.Hq):
            g = c.hm[h]
            f = orc.forward(c.Q[b, h], c.K[b, g], c.V[b, g], a_q[b, h], a_k[b, g], qbar[b, h].astype(np.float64),
                            sigma=c.sigma, S=w.S, Ck=w.Ck, m=w.m, sel=sel[b, h])
            assert rel_err(O[b, h], f["O"]) <= tol(w.dtype)
