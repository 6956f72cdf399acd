"""Pins for the oracle's dipole correction (Appendix "Error Analysis": "Dipole Correction",
"Untilted (Partially Specialized) Covariances"): library covariance, library softmax, the
dense-attention Jacobian in closed form, the order of the error, invariances."""
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


def test_dipole_with_retrieval_is_rejected():
    p = toy_problem(37)
    with pytest.raises(ValueError):
        orc.forward(p["Q"], p["K"], p["V"], p["a_q"], p["a_k"], p["qbar"], sigma=1.0, S=p["S"], Ck=p["Ck"], m=2, dipole=1)
