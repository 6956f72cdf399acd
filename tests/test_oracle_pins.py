"""Pins for the fp64 oracle: every function is checked against something other than itself —
a library routine, a closed form, an invariant the paper states, brute force on tiny inputs,
or central finite differences."""
import itertools

import numpy as np
import pytest

from oracle import muse_oracle as orc
from tests.helpers import toy_problem, dense_causal_attention, dense_causal_grads


# ------------------------------------------------------------------ clustering

def _blobs(seed, N=600, D=5, C=6):
    rng = np.random.default_rng(seed)
    c = 3.0 * rng.standard_normal((C, D))
    X = c[rng.integers(0, C, N)] + 0.5 * rng.standard_normal((N, D))
    return X


def test_assign_is_bruteforce_nearest():
    rng = np.random.default_rng(0)
    X = rng.standard_normal((50, 3)); C = rng.standard_normal((7, 3))
    a = orc.assign_nearest(X, C)
    for t in range(50):
        d = [sum((X[t, k] - C[c, k]) ** 2 for k in range(3)) for c in range(7)]
        assert a[t] == int(np.argmin(d))


def test_assign_ties_go_to_lowest_index():
    X = np.array([[0.0, 0.0]])
    C = np.array([[1.0, 0.0], [-1.0, 0.0], [0.0, 1.0]])
    assert orc.assign_nearest(X, C)[0] == 0


@pytest.mark.parametrize("T", [1, 3, 5])
def test_lloyd_matches_sklearn(T):
    from sklearn.cluster import KMeans
    X = _blobs(1)
    init = np.arange(0, 600, 100)
    a, c = orc.lloyd(X, T, init_idx=init)
    km = KMeans(n_clusters=6, init=X[init].copy(), n_init=1, max_iter=T, tol=0.0, algorithm="lloyd").fit(X)
    assert np.array_equal(np.bincount(a, minlength=6) > 0, np.ones(6, bool))  # no empties here
    np.testing.assert_allclose(c, km.cluster_centers_, rtol=0, atol=1e-12)
    assert np.array_equal(a, km.labels_)


def test_lloyd_centres_match_scipy():
    from scipy.cluster.vq import kmeans2
    X = _blobs(2)
    init = np.arange(0, 600, 100)
    _, c = orc.lloyd(X, 4, init_idx=init)
    c2, _ = kmeans2(X, X[init].copy(), iter=4, minit="matrix")
    np.testing.assert_allclose(c, c2, rtol=0, atol=1e-12)


def test_lloyd_inertia_monotone_and_fixed_point():
    X = _blobs(3)
    init = np.arange(0, 600, 100)
    prev = np.inf
    for T in range(0, 8):
        a, c = orc.lloyd(X, T, init_idx=init)
        inertia = ((X - c[a]) ** 2).sum()
        assert inertia <= prev + 1e-9
        prev = inertia
    a, c = orc.lloyd(X, 60, init_idx=init)
    for k in range(6):
        np.testing.assert_allclose(c[k], X[a == k].mean(0), atol=1e-12)


def test_empty_cluster_keeps_centre():
    X = np.array([[0.0], [0.1], [0.2]])
    start = np.array([[0.1], [100.0]])
    a, c = orc.lloyd(X, 2, init_centres=start)
    assert np.all(a == 0) and c[1, 0] == 100.0 and abs(c[0, 0] - 0.1) < 1e-15


def test_assignment_gaps():
    X = np.array([[0.0, 0.0], [0.9, 0.0]])
    C = np.array([[1.0, 0.0], [-1.0, 0.0]])
    g = orc.assignment_gaps(X, C)
    assert g[0] == 0.0
    assert abs(g[1] - (1.9 ** 2 - 0.1 ** 2) / 1.9 ** 2) < 1e-12


@pytest.mark.parametrize("N", [2, 7, 64, 1000, 1024, 4097])
def test_feistel_is_bijection(N):
    img = sorted(orc.feistel_permute(x, N, 1234, 5) for x in range(N))
    assert img == list(range(N))


def test_strided_init_distinct_and_seeded():
    a = orc.strided_init(1000, 37, 42, 0)
    assert len(set(a.tolist())) == 37 and a.min() >= 0 and a.max() < 1000
    assert not np.array_equal(a, orc.strided_init(1000, 37, 43, 0))
    assert not np.array_equal(a, orc.strided_init(1000, 37, 42, 1))
    assert np.array_equal(a, orc.strided_init(1000, 37, 42, 0))


# ------------------------------------------------------------------ summaries

def test_recurrence_equals_direct_definition():
    p = toy_problem(4)
    mu, ka, nu = orc.block_summaries(p["K"], p["V"], p["a_k"], p["qbar"], p["sigma"], p["S"], p["Ck"])
    r = orc.accumulate(mu, ka, nu)
    d = orc.accumulated_summaries(p["K"], p["V"], p["a_k"], p["qbar"], p["sigma"], p["S"], p["Ck"])
    for x, y in zip(r, d):
        assert np.array_equal(np.isfinite(x), np.isfinite(y))
        np.testing.assert_allclose(np.where(np.isfinite(x), x, 0), np.where(np.isfinite(y), y, 0), atol=1e-12)
    assert np.all(np.isneginf(d[0][0]))  # exclusive: block 0 sees nothing


def test_zero_centroid_gives_plain_means_and_log_counts():
    p = toy_problem(5)
    qbar0 = np.zeros_like(p["qbar"])
    muh, kah, nuh = orc.accumulated_summaries(p["K"], p["V"], p["a_k"], qbar0, p["sigma"], p["S"], p["Ck"])
    Bs = p["N"] // p["S"]
    for b in range(1, p["S"]):
        for j in range(p["Ck"]):
            mem = np.nonzero((np.arange(p["N"]) // Bs < b) & (p["a_k"] == j))[0]
            if mem.size:
                np.testing.assert_allclose(muh[b, :, j], np.log(mem.size), atol=1e-13)
                np.testing.assert_allclose(kah[b, 0, j], p["K"][mem].mean(0), atol=1e-13)
                np.testing.assert_allclose(nuh[b, 1, j], p["V"][mem].mean(0), atol=1e-13)


def test_summary_is_attention_from_centroid_and_jensen():
    p = toy_problem(6)
    muh, kah, nuh = orc.accumulated_summaries(p["K"], p["V"], p["a_k"], p["qbar"], p["sigma"], p["S"], p["Ck"])
    Bs = p["N"] // p["S"]
    b, i, j = 3, 1, 2
    mem = np.nonzero((np.arange(p["N"]) // Bs < b) & (p["a_k"] == j))[0]
    w = np.array([np.exp(p["sigma"] * p["qbar"][i] @ p["K"][u]) for u in mem])
    assert abs(muh[b, i, j] - np.log(w.sum())) < 1e-12
    np.testing.assert_allclose(kah[b, i, j], (w[:, None] * p["K"][mem]).sum(0) / w.sum(), atol=1e-12)
    np.testing.assert_allclose(nuh[b, i, j], (w[:, None] * p["V"][mem]).sum(0) / w.sum(), atol=1e-12)
    # Jensen: log-mean-exp >= mean of the logits
    assert muh[b, i, j] >= np.log(mem.size) + p["sigma"] * p["qbar"][i] @ p["K"][mem].mean(0) - 1e-12


# ------------------------------------------------------------------ forward

def _bruteforce_forward(p, m, sel_mode=0):
    """The whole layer, query by query and key by key, as one softmax over exact keys and
    far-cluster virtual keys (no shared code with the oracle)."""
    N, S, Ck, sg = p["N"], p["S"], p["Ck"], p["sigma"]
    Bs = N // S
    O = np.zeros_like(p["V"]); L = np.zeros(N); SEL = []
    for t in range(N):
        b = t // Bs; i = p["a_q"][t]
        qb = p["qbar"][i]; q = p["Q"][t]
        cl = {}
        for j in range(Ck):
            mem = [u for u in range(b * Bs) if p["a_k"][u] == j]
            if not mem:
                continue
            w = np.array([np.exp(sg * qb @ p["K"][u]) for u in mem])
            mass = w.sum()
            kap = sum(w[x] * p["K"][u] for x, u in enumerate(mem)) / mass
            nu = sum(w[x] * p["V"][u] for x, u in enumerate(mem)) / mass
            cl[j] = (np.log(mass), sg * (q - qb) @ kap + np.log(mass), nu, mem)
        ranked = sorted(cl, key=lambda j: (-(cl[j][1] if sel_mode == 0 else cl[j][0]), j))[:m]
        SEL.append(sorted(ranked))
        logits, vals = [], []
        for j, (_, sc, nu, mem) in cl.items():
            if j in ranked:
                for u in mem:
                    logits.append(sg * q @ p["K"][u]); vals.append(p["V"][u])
            else:
                logits.append(sc); vals.append(nu)
        for u in range(b * Bs, t + 1):
            logits.append(sg * q @ p["K"][u]); vals.append(p["V"][u])
        logits = np.array(logits); vals = np.array(vals)
        mx = logits.max(); w = np.exp(logits - mx)
        L[t] = mx + np.log(w.sum()); O[t] = (w / w.sum()) @ vals
    return O, L, SEL


@pytest.mark.parametrize("m,sel_mode", [(0, 0), (2, 0), (3, 1), (6, 0)])
def test_forward_equals_bruteforce_union_softmax(m, sel_mode):
    p = toy_problem(7, N=64, D=4, Cq=3, Ck=6, S=4)
    f = orc.forward(p["Q"], p["K"], p["V"], p["a_q"], p["a_k"], p["qbar"], sigma=p["sigma"], S=p["S"],
                    Ck=p["Ck"], m=m, sel_mode=sel_mode)
    O, L, SEL = _bruteforce_forward(p, m, sel_mode)
    np.testing.assert_allclose(f["O"], O, atol=1e-12)
    np.testing.assert_allclose(f["LSE"], L, atol=1e-12)
    for t in range(p["N"]):
        assert sorted(x for x in f["sel"][t] if x >= 0) == SEL[t]


def test_select_clusters_bruteforce_and_ties():
    rng = np.random.default_rng(8)
    sc = np.round(rng.standard_normal((20, 9)), 1)          # rounding creates ties
    sc[rng.random((20, 9)) < 0.3] = -np.inf
    sel = orc.select_clusters(sc, sc, 4)
    for r in range(20):
        cand = [j for j in range(9) if np.isfinite(sc[r, j])]
        exp = sorted(cand, key=lambda j: (-sc[r, j], j))[:4]
        assert [x for x in sel[r] if x >= 0] == exp
        assert list(sel[r][len(exp):]) == [-1] * (4 - len(exp))


def test_all_clusters_retrieved_is_dense_attention():
    p = toy_problem(9)
    f = orc.forward(p["Q"], p["K"], p["V"], p["a_q"], p["a_k"], p["qbar"], sigma=p["sigma"], S=p["S"],
                    Ck=p["Ck"], m=p["Ck"])
    O, L = dense_causal_attention(p["Q"], p["K"], p["V"], p["sigma"])
    np.testing.assert_allclose(f["O"], O, atol=1e-13)
    np.testing.assert_allclose(f["LSE"], L, atol=1e-12)


@pytest.mark.parametrize("m", [0, 3])
def test_singleton_key_clusters_are_exact(m):
    p = toy_problem(10, N=48, S=4)
    a_k = np.arange(48, dtype=np.int32)
    f = orc.forward(p["Q"], p["K"], p["V"], p["a_q"], a_k, p["qbar"], sigma=p["sigma"], S=4, Ck=48, m=m)
    O, _ = dense_causal_attention(p["Q"], p["K"], p["V"], p["sigma"])
    np.testing.assert_allclose(f["O"], O, atol=1e-12)


def test_singleton_query_clusters_are_exact():
    p = toy_problem(11, N=48, S=4)
    a_q = np.arange(48, dtype=np.int32)
    f = orc.forward(p["Q"], p["K"], p["V"], a_q, p["a_k"], p["Q"].copy(), sigma=p["sigma"], S=4,
                    Ck=p["Ck"], m=1)
    O, _ = dense_causal_attention(p["Q"], p["K"], p["V"], p["sigma"])
    np.testing.assert_allclose(f["O"], O, atol=1e-12)


def test_key_translation_invariance():
    p = toy_problem(12)
    kw = dict(sigma=p["sigma"], S=p["S"], Ck=p["Ck"], m=2)
    f0 = orc.forward(p["Q"], p["K"], p["V"], p["a_q"], p["a_k"], p["qbar"], **kw)
    shift = np.random.default_rng(0).standard_normal(p["D"])
    f1 = orc.forward(p["Q"], p["K"] + shift, p["V"], p["a_q"], p["a_k"], p["qbar"], **kw)
    np.testing.assert_allclose(f0["O"], f1["O"], atol=1e-12)
    assert np.array_equal(f0["sel"], f1["sel"])


def test_weights_sum_to_one_and_are_causal():
    p = toy_problem(13, N=64)
    N = 64
    kw = dict(sigma=p["sigma"], S=p["S"], Ck=p["Ck"], m=2)
    ones = orc.forward(p["Q"], p["K"], np.ones((N, 3)), p["a_q"], p["a_k"], p["qbar"], **kw)
    np.testing.assert_allclose(ones["O"], 1.0, atol=1e-13)
    W = orc.forward(p["Q"], p["K"], np.eye(N), p["a_q"], p["a_k"], p["qbar"], **kw)["O"]
    assert W.min() >= 0 and np.abs(np.triu(W, 1)).max() == 0
    np.testing.assert_allclose(W.sum(1), 1.0, atol=1e-13)


def test_monopole_error_is_bilinear_in_residuals():
    rng = np.random.default_rng(14)
    N, D, Cq, Ck, S = 96, 6, 3, 5, 4
    a_q = rng.integers(0, Cq, N).astype(np.int32); a_k = rng.integers(0, Ck, N).astype(np.int32)
    qc, kc = rng.standard_normal((Cq, D)), rng.standard_normal((Ck, D))
    rq, rk = rng.standard_normal((N, D)), rng.standard_normal((N, D))
    V = rng.standard_normal((N, D))

    def err(eq, ek):
        Q, K = qc[a_q] + eq * rq, kc[a_k] + ek * rk
        f = orc.forward(Q, K, V, a_q, a_k, qc, sigma=1.0, S=S, Ck=Ck, m=0)
        O, _ = dense_causal_attention(Q, K, V, 1.0)
        return np.abs(f["O"] - O).max()
    e = err(0.02, 0.02)
    assert 1.8 < e / err(0.01, 0.02) < 2.2
    assert 1.8 < e / err(0.02, 0.01) < 2.2
    assert err(0.0, 0.5) < 1e-13 and err(0.5, 0.0) < 1e-13


def test_component_merge_matches_components():
    p = toy_problem(15)
    f = orc.forward(p["Q"], p["K"], p["V"], p["a_q"], p["a_k"], p["qbar"], sigma=p["sigma"], S=p["S"],
                    Ck=p["Ck"], m=2)
    lses = np.stack([f["lse_far"], f["lse_ret"], f["lse_loc"]], 1)
    mx = lses.max(1, keepdims=True)
    L = (mx + np.log(np.exp(lses - mx).sum(1, keepdims=True)))[:, 0]
    np.testing.assert_allclose(L, f["LSE"], atol=1e-13)
    assert np.all(np.isneginf(f["lse_far"][: p["N"] // p["S"]]))   # block 0 is local-only


def test_rows_subset_matches_full():
    p = toy_problem(16)
    kw = dict(sigma=p["sigma"], S=p["S"], Ck=p["Ck"], m=2)
    full = orc.forward(p["Q"], p["K"], p["V"], p["a_q"], p["a_k"], p["qbar"], **kw)
    rows = np.array([3, 40, 41, 95])
    part = orc.forward(p["Q"], p["K"], p["V"], p["a_q"], p["a_k"], p["qbar"], rows=rows, **kw)
    np.testing.assert_allclose(part["O"][rows], full["O"][rows], atol=1e-14)


def test_noncausal_all_clusters_is_dense_noncausal():
    p = toy_problem(17)
    f = orc.forward(p["Q"], p["K"], p["V"], p["a_q"], p["a_k"], p["qbar"], sigma=p["sigma"], S=1,
                    Ck=p["Ck"], m=p["Ck"], causal=False)
    O, _ = dense_causal_attention(p["Q"], p["K"], p["V"], p["sigma"], causal=False)
    np.testing.assert_allclose(f["O"], O, atol=1e-13)


# ------------------------------------------------------------------ backward

def _fd(fun, X, h=1e-5):
    g = np.zeros_like(X)
    for idx in itertools.product(*map(range, X.shape)):
        old = X[idx]
        X[idx] = old + h; fp = fun()
        X[idx] = old - h; fm = fun()
        X[idx] = old
        g[idx] = (fp - fm) / (2 * h)
    return g


@pytest.mark.parametrize("m,sel_mode", [(0, 0), (2, 0), (2, 1)])
def test_backward_matches_finite_differences(m, sel_mode):
    p = toy_problem(18, N=32, D=4, Dv=3, Cq=3, Ck=4, S=4, gain=2.0)
    kw = dict(sigma=p["sigma"], S=p["S"], Ck=p["Ck"], m=m, sel_mode=sel_mode)
    sel = orc.forward(p["Q"], p["K"], p["V"], p["a_q"], p["a_k"], p["qbar"], **kw)["sel"]
    Q, K, V = p["Q"].copy(), p["K"].copy(), p["V"].copy()

    def loss():
        return (orc.forward(Q, K, V, p["a_q"], p["a_k"], p["qbar"], sel=sel, **kw)["O"] * p["dO"]).sum()
    dQ, dK, dV, _ = orc.backward(Q, K, V, p["dO"], p["a_q"], p["a_k"], p["qbar"], sel=sel, **kw)
    for g, X in ((dQ, Q), (dK, K), (dV, V)):
        fd = _fd(loss, X)
        assert np.abs(g - fd).max() <= 1e-6 * np.abs(fd).max()


def test_backward_without_aggregation_gradient():
    """agg_grad=False: the tilted aggregation weights are constants.  Reference: finite
    differences of a forward whose summaries are rebuilt with the weights frozen."""
    p = toy_problem(19, N=32, D=4, Dv=3, Cq=3, Ck=4, S=4, gain=2.0)
    N, S, Ck, sg = p["N"], p["S"], p["Ck"], p["sigma"]
    kw = dict(sigma=sg, S=S, Ck=Ck, m=1)
    f0 = orc.forward(p["Q"], p["K"], p["V"], p["a_q"], p["a_k"], p["qbar"], **kw)
    sel, (muh, _, _) = f0["sel"], f0["summ"]
    Bs = N // S
    K0 = p["K"].copy()
    Q, K, V = p["Q"].copy(), p["K"].copy(), p["V"].copy()

    def frozen_summaries():
        kah = np.zeros((S, p["Cq"], Ck, p["D"])); nuh = np.zeros((S, p["Cq"], Ck, V.shape[1]))
        for b in range(S):
            for j in range(Ck):
                mem = np.nonzero((np.arange(N) // Bs < b) & (p["a_k"] == j))[0]
                if mem.size:
                    w = np.exp(sg * p["qbar"] @ K0[mem].T - muh[b, :, j][:, None])   # frozen
                    kah[b, :, j] = w @ K[mem]; nuh[b, :, j] = w @ V[mem]
        return muh, kah, nuh

    def loss():
        return (orc.forward(Q, K, V, p["a_q"], p["a_k"], p["qbar"], sel=sel, summ=frozen_summaries(),
                            **kw)["O"] * p["dO"]).sum()
    dQ, dK, dV, _ = orc.backward(Q, K, V, p["dO"], p["a_q"], p["a_k"], p["qbar"], sel=sel,
                                 agg_grad=False, **kw)
    for g, X in ((dQ, Q), (dK, K), (dV, V)):
        fd = _fd(loss, X)
        assert np.abs(g - fd).max() <= 1e-6 * np.abs(fd).max()
    dK_full = orc.backward(Q, K, V, p["dO"], p["a_q"], p["a_k"], p["qbar"], sel=sel, **kw)[1]
    assert np.abs(dK_full - dK).max() > 1e-6     # the dropped term is not zero


def test_backward_all_retrieved_equals_dense_gradient():
    p = toy_problem(20)
    dQ, dK, dV, _ = orc.backward(p["Q"], p["K"], p["V"], p["dO"], p["a_q"], p["a_k"], p["qbar"],
                                 sigma=p["sigma"], S=p["S"], Ck=p["Ck"], m=p["Ck"])
    eQ, eK, eV = dense_causal_grads(p["Q"], p["K"], p["V"], p["dO"], p["sigma"])
    np.testing.assert_allclose(dQ, eQ, atol=1e-12)
    np.testing.assert_allclose(dK, eK, atol=1e-12)
    np.testing.assert_allclose(dV, eV, atol=1e-12)


def test_backward_rows_are_additive():
    p = toy_problem(21)
    kw = dict(sigma=p["sigma"], S=p["S"], Ck=p["Ck"], m=2)
    sel = orc.forward(p["Q"], p["K"], p["V"], p["a_q"], p["a_k"], p["qbar"], **kw)["sel"]
    full = orc.backward(p["Q"], p["K"], p["V"], p["dO"], p["a_q"], p["a_k"], p["qbar"], sel=sel, **kw)
    lo = orc.backward(p["Q"], p["K"], p["V"], p["dO"], p["a_q"], p["a_k"], p["qbar"], sel=sel,
                      rows=np.arange(0, 50), **kw)
    hi = orc.backward(p["Q"], p["K"], p["V"], p["dO"], p["a_q"], p["a_k"], p["qbar"], sel=sel,
                      rows=np.arange(50, 96), **kw)
    for k in range(3):
        np.testing.assert_allclose(lo[k] + hi[k], full[k], atol=1e-12)


def test_gqa_layer_sums_key_gradients_over_group():
    rng = np.random.default_rng(22)
    B, Hq, Hkv, N, D, Cq, Ck, S = 1, 4, 2, 32, 4, 2, 3, 4
    Q = rng.standard_normal((B, Hq, N, D)); K = rng.standard_normal((B, Hkv, N, D))
    V = rng.standard_normal((B, Hkv, N, D)); dO = rng.standard_normal((B, Hq, N, D))
    a_q = rng.integers(0, Cq, (B, Hq, N)).astype(np.int32)
    a_k = rng.integers(0, Ck, (B, Hkv, N)).astype(np.int32)
    qbar = rng.standard_normal((B, Hq, Cq, D))
    kw = dict(sigma=0.5, S=S, Ck=Ck, m=1)
    O, LSE, sel = orc.layer_forward(Q, K, V, a_q, a_k, qbar, **kw)
    dQ, dK, dV = orc.layer_backward(Q, K, V, dO, a_q, a_k, qbar, sel=sel, **kw)
    acc = np.zeros((N, D))
    for h in (2, 3):
        acc += orc.backward(Q[0, h], K[0, 1], V[0, 1], dO[0, h], a_q[0, h], a_k[0, 1], qbar[0, h],
                            sel=sel[0, h], **kw)[1]
    np.testing.assert_allclose(dK[0, 1], acc, atol=1e-13)
    f = orc.forward(Q[0, 3], K[0, 1], V[0, 1], a_q[0, 3], a_k[0, 1], qbar[0, 3], **kw)
    np.testing.assert_allclose(O[0, 3], f["O"], atol=0)
