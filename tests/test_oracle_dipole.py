"""Pins for the oracle's dipole correction (Appendix "Error Analysis": "Dipole Correction",
"Untilted (Partially Specialized) Covariances"): library covariance, library softmax, the
dense-attention Jacobian in closed form, the order of the error, invariances."""
import itertools

import numpy as np
import pytest
import scipy.special

from oracle import muse_oracle as orc
from tests.helpers import toy_problem, dense_causal_attention


def test_untilted_covariance_is_numpy_cov_over_visible_members():
    p = toy_problem(31, N=128, D=5, Dv=3, Ck=4, S=4)
    cov = orc.untilted_covariances(p["K"], p["V"], p["a_k"], p["S"], p["Ck"])
    Bs = p["N"] // p["S"]
    assert np.abs(cov[0]).max() == 0                       # nothing is visible before block 0
    for b in range(1, p["S"]):
        for j in range(p["Ck"]):
            mem = [u for u in range(b * Bs) if p["a_k"][u] == j]
            full = np.cov(np.hstack([p["V"][mem], p["K"][mem]]).T, bias=True)
            np.testing.assert_allclose(cov[b, j], full[:3, 3:], atol=1e-13)


def test_untilted_covariance_ignores_current_and_later_blocks():
    p = toy_problem(32, N=128, S=4)
    c0 = orc.untilted_covariances(p["K"], p["V"], p["a_k"], p["S"], p["Ck"])
    K2, V2 = p["K"].copy(), p["V"].copy()
    K2[64:] += 3.0; V2[64:] -= 2.0                          # blocks 2 and 3
    c1 = orc.untilted_covariances(K2, V2, p["a_k"], p["S"], p["Ck"])
    np.testing.assert_array_equal(c0[:3], c1[:3])
    assert np.abs(c0[3] - c1[3]).max() > 1e-3


def test_merge_weights_are_softmax_of_log_masses():
    rng = np.random.default_rng(33)
    S, Cq, Ck, D = 3, 4, 6, 2
    muh = rng.standard_normal((S, Cq, Ck)) * 3
    muh[0] = -np.inf; muh[1, :, 2] = -np.inf
    # covariance j = indicator matrix scaled by (j+1): the merge then spells out its weights
    cov = np.zeros((S, Ck, D, D))
    for j in range(Ck):
        cov[:, j, 0, 0] = 1.0; cov[:, j, 1, 1] = j + 1.0
    cbar = orc.merged_dipole(muh, cov)
    assert np.abs(cbar[0]).max() == 0
    for b in (1, 2):
        pw = scipy.special.softmax(muh[b], axis=1)          # exp(-inf) = 0 handles empty clusters
        np.testing.assert_allclose(cbar[b, :, 0, 0], pw.sum(1), atol=1e-14)
        np.testing.assert_allclose(cbar[b, :, 1, 1], pw @ (np.arange(Ck) + 1.0), atol=1e-13)
        assert np.abs(cbar[b, :, 0, 1]).max() == 0


def _zero_tilt_problem(seed, N=96, D=5, Ck=5, S=4):
    rng = np.random.default_rng(seed)
    a_k = rng.integers(0, Ck, N).astype(np.int32)
    kc = rng.standard_normal((Ck, D))
    K = kc[a_k] + 0.5 * rng.standard_normal((N, D))
    V = rng.standard_normal((N, 4))
    rq = rng.standard_normal((N, D))
    return dict(N=N, D=D, Ck=Ck, S=S, a_k=a_k, K=K, V=V, rq=rq, a_q=np.zeros(N, np.int32), qbar=np.zeros((1, D)))


@pytest.mark.parametrize("causal", [True, False])
def test_jacobian_at_zero_residual_is_the_dense_attention_jacobian(causal):
    """One query cluster with centroid 0: tilted = untilted, so monopole (between clusters) +
    merged dipole (within clusters) must reproduce d/dq softmax-attention at q = 0, which is
    sigma * Cov(v, k) under uniform weights over the visible keys (total covariance)."""
    z = _zero_tilt_problem(34)
    sigma, eps, t = 0.7, 1e-5, 77                            # a query in block 3
    kw = dict(sigma=sigma, S=z["S"], Ck=z["Ck"], m=0, causal=causal, rows=[t], dipole=1)
    J = np.zeros((4, z["D"]))
    for d in range(z["D"]):
        Qp = np.zeros((z["N"], z["D"])); Qm = Qp.copy()
        Qp[t, d], Qm[t, d] = eps, -eps
        op = orc.forward(Qp, z["K"], z["V"], z["a_q"], z["a_k"], z["qbar"], **kw)["O"][t]
        om = orc.forward(Qm, z["K"], z["V"], z["a_q"], z["a_k"], z["qbar"], **kw)["O"][t]
        J[:, d] = (op - om) / (2 * eps)
    n = t + 1 if causal else z["N"]
    total = np.cov(np.hstack([z["V"][:n], z["K"][:n]]).T, bias=True)[:4, 4:]
    np.testing.assert_allclose(J, sigma * total, atol=1e-8)
    # without the dipole the within-cluster part is missing
    kw["dipole"] = 0
    Qp = np.zeros((z["N"], z["D"])); Qp[t, 0] = eps
    o1 = orc.forward(Qp, z["K"], z["V"], z["a_q"], z["a_k"], z["qbar"], **kw)["O"][t]
    o0 = orc.forward(0 * Qp, z["K"], z["V"], z["a_q"], z["a_k"], z["qbar"], **kw)["O"][t]
    assert np.abs((o1 - o0) / eps - sigma * total[:, 0]).max() > 1e-3


def test_dipole_error_is_second_order_in_the_query_residual():
    z = _zero_tilt_problem(35)

    def err(eq, dipole):
        Q = eq * z["rq"]
        f = orc.forward(Q, z["K"], z["V"], z["a_q"], z["a_k"], z["qbar"], sigma=1.0, S=z["S"], Ck=z["Ck"],
                        m=0, dipole=dipole)
        O, _ = dense_causal_attention(Q, z["K"], z["V"], 1.0)
        return np.abs(f["O"] - O).max()
    assert 3.6 < err(0.02, 1) / err(0.01, 1) < 4.4          # O(residual^2) with the dipole
    assert 1.8 < err(0.02, 0) / err(0.01, 0) < 2.2          # O(residual) without
    assert err(0.02, 1) < 0.1 * err(0.02, 0)


def test_dipole_leaves_mass_unchanged_and_keeps_invariances():
    p = toy_problem(36)
    kw = dict(sigma=p["sigma"], S=p["S"], Ck=p["Ck"], m=0)
    f0 = orc.forward(p["Q"], p["K"], p["V"], p["a_q"], p["a_k"], p["qbar"], **kw)
    f1 = orc.forward(p["Q"], p["K"], p["V"], p["a_q"], p["a_k"], p["qbar"], dipole=1, **kw)
    np.testing.assert_array_equal(f0["LSE"], f1["LSE"])
    np.testing.assert_array_equal(f0["lse_far"], f1["lse_far"])
    np.testing.assert_array_equal(f0["o_loc"], f1["o_loc"])
    assert np.abs(f0["O"] - f1["O"]).max() > 1e-3
    Bs = p["N"] // p["S"]
    np.testing.assert_array_equal(f0["O"][:Bs], f1["O"][:Bs])   # block 0 has no far field
    # key translation: covariances and masses are translation invariant
    shift = np.random.default_rng(1).standard_normal(p["D"])
    f2 = orc.forward(p["Q"], p["K"] + shift, p["V"], p["a_q"], p["a_k"], p["qbar"], dipole=1, **kw)
    np.testing.assert_allclose(f1["O"], f2["O"], atol=1e-12)
    # constant values have zero covariance with the keys: output stays 1
    ones = orc.forward(p["Q"], p["K"], np.ones((p["N"], 2)), p["a_q"], p["a_k"], p["qbar"], dipole=1, **kw)
    np.testing.assert_allclose(ones["O"], 1.0, atol=1e-13)
    # the correction is the merged matrix applied to the residual, weighted by the far share
    t = p["N"] - 1
    i, b = p["a_q"][t], p["S"] - 1
    qres = p["sigma"] * (p["Q"][t] - p["qbar"][i])
    w_far = np.exp(f1["lse_far"][t] - f1["LSE"][t])
    np.testing.assert_allclose(f1["O"][t] - f0["O"][t], w_far * (f1["cbar"][b, i] @ qres), atol=1e-13)


# ------------------------------------------------------------------ shared covariance with one tilt point

def test_tilted_covariance_is_the_derivative_of_the_tilted_value_mean():
    """d/d(tilt) of the tilted value mean of a key set is sigma times its tilted cross-covariance
    (a cumulant identity); the value mean comes from the summaries, which have their own pins."""
    p = toy_problem(41, N=96, D=4, Dv=3, Ck=3, S=4)
    rng = np.random.default_rng(41)
    tilt, sigma, h = rng.standard_normal(4), 0.6, 1e-6
    cov = orc.tilted_covariances(p["K"], p["V"], p["a_k"], p["S"], p["Ck"], tilt, sigma)
    for d in range(4):
        e = np.zeros(4); e[d] = h
        nu_p = orc.accumulated_summaries(p["K"], p["V"], p["a_k"], (tilt + e)[None], sigma, p["S"], p["Ck"])[2]
        nu_m = orc.accumulated_summaries(p["K"], p["V"], p["a_k"], (tilt - e)[None], sigma, p["S"], p["Ck"])[2]
        np.testing.assert_allclose((nu_p - nu_m)[:, 0] / (2 * h), sigma * cov[..., d], atol=1e-8)
    assert np.abs(cov[1:]).max() > 1e-2


def test_zero_tilt_is_the_untilted_covariance_and_tilt_is_key_translation_invariant():
    p = toy_problem(42, N=96, D=4, Dv=3, Ck=3, S=4)
    c0 = orc.untilted_covariances(p["K"], p["V"], p["a_k"], p["S"], p["Ck"])
    np.testing.assert_allclose(orc.tilted_covariances(p["K"], p["V"], p["a_k"], p["S"], p["Ck"], np.zeros(4), 1.0), c0,
                               atol=1e-14)
    t = np.array([0.3, -1.0, 0.5, 0.2])
    c1 = orc.tilted_covariances(p["K"], p["V"], p["a_k"], p["S"], p["Ck"], t, 0.8)
    c2 = orc.tilted_covariances(p["K"] + 2.5, p["V"], p["a_k"], p["S"], p["Ck"], t, 0.8)
    np.testing.assert_allclose(c1, c2, atol=1e-12)
    assert np.abs(c1 - c0).max() > 1e-3
    nc = orc.tilted_covariances(p["K"], p["V"], p["a_k"], p["S"], p["Ck"], t, 0.8, causal=False)
    assert nc.shape[0] == 1


def test_mean_query_centroid_is_the_mean_query_when_centroids_are_cluster_means():
    p = toy_problem(43)                                     # toy qbar = per-cluster means of Q
    np.testing.assert_allclose(orc.mean_query_centroid(p["qbar"], p["a_q"]), p["Q"].mean(0), atol=1e-13)
    # weights are the cluster sizes, not uniform
    a = np.array([0, 0, 0, 1], np.int32)
    np.testing.assert_allclose(orc.mean_query_centroid(np.array([[4.0], [8.0]]), a), [5.0])


def test_tilt_at_the_only_centroid_restores_second_order_error():
    """One query cluster with a non-zero centroid: the untilted covariance is off by the third
    cumulant times the centroid, so its error stays first order in the residual; tilting the shared
    covariance at the mean centroid (here: the centroid itself) is the fully tilted dipole."""
    z = _zero_tilt_problem(44)
    qb = 0.8 * np.random.default_rng(44).standard_normal((1, z["D"]))

    def err(eq, dipole):
        Q = qb + eq * z["rq"]
        f = orc.forward(Q, z["K"], z["V"], z["a_q"], z["a_k"], qb, sigma=1.0, S=z["S"], Ck=z["Ck"], m=0,
                        dipole=dipole)
        O, _ = dense_causal_attention(Q, z["K"], z["V"], 1.0)
        return np.abs(f["O"] - O).max()
    assert 3.6 < err(0.02, 2) / err(0.01, 2) < 4.4
    assert 1.8 < err(0.02, 1) / err(0.01, 1) < 2.3
    assert err(0.01, 2) < 0.2 * err(0.01, 1) < 0.2 * err(0.01, 0)


# ------------------------------------------------------------------ dipole next to retrieval

@pytest.mark.parametrize("m", [1, 2])
def test_jacobian_with_retrieval_is_still_the_dense_jacobian(m):
    """Retrieved clusters are exact, the others carry monopole + their share of the dipole: at zero
    residual (zero centroid) the whole output must again have the dense-attention Jacobian.  Leaving
    the retrieved clusters inside the merged matrix, or not renormalising, breaks it."""
    z = _zero_tilt_problem(45)
    sigma, eps, t = 0.7, 1e-5, 80
    base = dict(sigma=sigma, S=z["S"], Ck=z["Ck"], m=m, rows=[t])
    sel = orc.forward(np.zeros((z["N"], z["D"])), z["K"], z["V"], z["a_q"], z["a_k"], z["qbar"], **base)["sel"]

    def jac(dipole):
        J = np.zeros((4, z["D"]))
        for d in range(z["D"]):
            Qp = np.zeros((z["N"], z["D"])); Qm = Qp.copy()
            Qp[t, d], Qm[t, d] = eps, -eps
            op = orc.forward(Qp, z["K"], z["V"], z["a_q"], z["a_k"], z["qbar"], sel=sel, dipole=dipole, **base)["O"][t]
            om = orc.forward(Qm, z["K"], z["V"], z["a_q"], z["a_k"], z["qbar"], sel=sel, dipole=dipole, **base)["O"][t]
            J[:, d] = (op - om) / (2 * eps)
        return J
    n = t + 1
    total = np.cov(np.hstack([z["V"][:n], z["K"][:n]]).T, bias=True)[:4, 4:]
    np.testing.assert_allclose(jac(1), sigma * total, atol=1e-8)
    assert np.abs(jac(0) - sigma * total).max() > 1e-3
    # the naive composition (whole merged matrix next to retrieval) is not first-order exact
    f = orc.forward(np.zeros((z["N"], z["D"])), z["K"], z["V"], z["a_q"], z["a_k"], z["qbar"], dipole=1, **base)
    w_far = np.exp(f["lse_far"][t] - f["LSE"][t])
    naive = jac(0) + sigma * w_far * f["cbar"][3, 0]
    assert np.abs(naive - sigma * total).max() > 1e-4


def test_correction_with_retrieval_is_the_merged_matrix_minus_the_retrieved_share():
    p = toy_problem(46)
    kw = dict(sigma=p["sigma"], S=p["S"], Ck=p["Ck"], m=2)
    f0 = orc.forward(p["Q"], p["K"], p["V"], p["a_q"], p["a_k"], p["qbar"], **kw)
    f1 = orc.forward(p["Q"], p["K"], p["V"], p["a_q"], p["a_k"], p["qbar"], dipole=1, **kw)
    np.testing.assert_array_equal(f0["LSE"], f1["LSE"])
    np.testing.assert_array_equal(f0["sel"], f1["sel"])
    pw = orc.dipole_weights(f1["summ"][0])
    np.testing.assert_allclose(pw[1:].sum(2), 1.0, atol=1e-13)
    assert np.abs(pw[0]).max() == 0
    Bs = p["N"] // p["S"]
    checked = 0
    for t in range(Bs, p["N"]):
        i, b = p["a_q"][t], t // Bs
        if not np.isfinite(f1["lse_far"][t]):
            continue
        s = f1["sel"][t][f1["sel"][t] >= 0]
        M = f1["cbar"][b, i] - np.tensordot(pw[b, i][s], f1["cov"][b][s], axes=(0, 0))
        qres = p["sigma"] * (p["Q"][t] - p["qbar"][i])
        w_far = np.exp(f1["lse_far"][t] - f1["LSE"][t])
        np.testing.assert_allclose(f1["O"][t] - f0["O"][t], w_far * (M @ qres) / (1.0 - pw[b, i][s].sum()), atol=1e-11)
        checked += 1
    assert checked > p["N"] // 2


def test_m0_correction_is_the_same_on_both_routes():
    """backward() always takes the per-query route; at m = 0 it must reproduce the pre-merged one."""
    p = toy_problem(47)
    kw = dict(sigma=p["sigma"], S=p["S"], Ck=p["Ck"], m=0)
    for dip in (1, 2):
        f = orc.forward(p["Q"], p["K"], p["V"], p["a_q"], p["a_k"], p["qbar"], dipole=dip, **kw)
        fb = orc.backward(p["Q"], p["K"], p["V"], p["dO"], p["a_q"], p["a_k"], p["qbar"], dipole=dip, **kw)[3]
        np.testing.assert_allclose(fb["O"], f["O"], atol=1e-13)
    with pytest.raises(ValueError):
        orc.forward(p["Q"], p["K"], p["V"], p["a_q"], p["a_k"], p["qbar"], dipole=1, k2=1, **kw)
    with pytest.raises(ValueError):
        orc.forward(p["Q"], p["K"], p["V"], p["a_q"], p["a_k"], p["qbar"], dipole=3, **kw)


# ------------------------------------------------------------------ backward through the dipole

def _fd(fun, X, h=1e-5):
    g = np.zeros_like(X)
    for idx in itertools.product(*map(range, X.shape)):
        old = X[idx]
        X[idx] = old + h; fp = fun()
        X[idx] = old - h; fm = fun()
        X[idx] = old
        g[idx] = (fp - fm) / (2 * h)
    return g


@pytest.mark.parametrize("m,dipole,causal", [(0, 1, True), (2, 1, True), (0, 2, True), (2, 2, True), (1, 1, False)])
def test_dipole_backward_matches_finite_differences(m, dipole, causal):
    p = toy_problem(48, N=32, D=4, Dv=3, Cq=3, Ck=4, S=4, gain=2.0)
    kw = dict(sigma=p["sigma"], S=p["S"], Ck=p["Ck"], m=m, causal=causal)
    sel = orc.forward(p["Q"], p["K"], p["V"], p["a_q"], p["a_k"], p["qbar"], **kw)["sel"]
    Q, K, V = p["Q"].copy(), p["K"].copy(), p["V"].copy()

    def loss():
        return (orc.forward(Q, K, V, p["a_q"], p["a_k"], p["qbar"], sel=sel, dipole=dipole, **kw)["O"] * p["dO"]).sum()
    dQ, dK, dV, _ = orc.backward(Q, K, V, p["dO"], p["a_q"], p["a_k"], p["qbar"], sel=sel, dipole=dipole, **kw)
    for g, X in ((dQ, Q), (dK, K), (dV, V)):
        fd = _fd(loss, X)
        assert np.abs(g - fd).max() <= 1e-6 * np.abs(fd).max()
    plain = orc.backward(Q, K, V, p["dO"], p["a_q"], p["a_k"], p["qbar"], sel=sel, **kw)
    assert np.abs(plain[1] - dK).max() > 1e-4 and np.abs(plain[0] - dQ).max() > 1e-4


def test_dipole_backward_with_frozen_weights():
    """agg_grad=False: neither the tilted summary weights, nor the centroid weights p_ib(j) (functions
    of the log-masses), nor the tilt weights of the shared covariance depend on the keys."""
    p = toy_problem(49, N=32, D=4, Dv=3, Cq=3, Ck=4, S=4, gain=2.0)
    N, S, Ck, sg = p["N"], p["S"], p["Ck"], p["sigma"]
    kw = dict(sigma=sg, S=S, Ck=Ck, m=0)
    Bs = N // S
    K0 = p["K"].copy()
    Q, K, V = p["Q"].copy(), p["K"].copy(), p["V"].copy()
    muh = orc.accumulated_summaries(K0, V, p["a_k"], p["qbar"], sg, S, Ck)[0]
    pw = orc.dipole_weights(muh)
    qstar = orc.mean_query_centroid(p["qbar"], p["a_q"])

    def loss():
        # forward written out with every weight taken at K0 (m = 0: far field + dipole + local block)
        tot = 0.0
        for t in range(N):
            i, b = p["a_q"][t], t // Bs
            qp = sg * Q[t]; qres = qp - sg * p["qbar"][i]
            logits, values = [], []
            cbar = np.zeros((V.shape[1], p["D"]))
            for j in range(Ck):
                mem = np.nonzero((np.arange(N) // Bs < b) & (p["a_k"] == j))[0]
                if mem.size == 0:
                    continue
                w = np.exp(sg * K0[mem] @ p["qbar"][i] - muh[b, i, j])
                logits.append(muh[b, i, j] + qres @ (w @ K[mem])); values.append(w @ V[mem])
                ws = np.exp(sg * K0[mem] @ qstar); ws /= ws.sum()
                cbar += pw[b, i, j] * ((ws[:, None] * V[mem]).T @ K[mem] - np.outer(ws @ V[mem], ws @ K[mem]))
            nfar = len(logits)
            corr = cbar @ qres
            for u in range(b * Bs, t + 1):
                logits.append(qp @ K[u]); values.append(V[u])
            lg = np.array(logits); w = np.exp(lg - lg.max()); w /= w.sum()
            vals = np.array(values); vals[:nfar] += corr
            tot += (w @ vals) @ p["dO"][t]
        return tot
    f = orc.forward(Q, K, V, p["a_q"], p["a_k"], p["qbar"], dipole=2, **kw)
    np.testing.assert_allclose(loss(), (f["O"] * p["dO"]).sum(), rtol=1e-12)
    dQ, dK, dV, _ = orc.backward(Q, K, V, p["dO"], p["a_q"], p["a_k"], p["qbar"], dipole=2, agg_grad=False, **kw)
    for g, X in ((dQ, Q), (dK, K), (dV, V)):
        fd = _fd(loss, X)
        assert np.abs(g - fd).max() <= 1e-6 * np.abs(fd).max()
