"""Pins for the oracle's two-level retrieval (Section "Two-Level Retrieval": cluster selection, then
spatial block selection inside the selected clusters with the pre-accumulation per-block summaries;
Section "Output merging": four components).  The brute force below shares no code with the oracle."""
import numpy as np
import pytest

from oracle import muse_oracle as orc
from tests.helpers import toy_problem, dense_causal_attention


def _bruteforce_two_level(p, m, k2):
    """Query by query: one softmax over
       exact keys of the k2 best earlier blocks of each of the m best clusters,
       one stand-in key per other earlier block of those clusters (per-block tilted summary),
       one stand-in key per remaining cluster (summary of all its earlier keys),
       the causal keys of the query's own block."""
    N, S, Ck, sg = p["N"], p["S"], p["Ck"], p["sigma"]
    Bs = N // S
    O = np.zeros_like(p["V"]); L = np.zeros(N); CH = []

    def tilted(qb, mem):
        w = np.array([np.exp(sg * qb @ p["K"][u]) for u in mem])
        mass = w.sum()
        return (np.log(mass), sum(w[x] * p["K"][u] for x, u in enumerate(mem)) / mass,
                sum(w[x] * p["V"][u] for x, u in enumerate(mem)) / mass)

    for t in range(N):
        b = t // Bs; i = p["a_q"][t]
        qb = p["qbar"][i]; q = p["Q"][t]; res = sg * (q - qb)
        cl = {}
        for j in range(Ck):
            mem = [u for u in range(b * Bs) if p["a_k"][u] == j]
            if mem:
                mu, kap, nu = tilted(qb, mem)
                cl[j] = (res @ kap + mu, nu)
        ranked = sorted(cl, key=lambda j: (-cl[j][0], j))[:m]
        logits, vals, chosen_all = [], [], {}
        for j, (sc, nu) in cl.items():
            if j not in ranked:
                logits.append(sc); vals.append(nu)
                continue
            blocks = {}
            for bp in range(b):
                mem = [u for u in range(bp * Bs, (bp + 1) * Bs) if p["a_k"][u] == j]
                if mem:
                    mu, kap, nu_b = tilted(qb, mem)
                    blocks[bp] = (res @ kap + mu, nu_b, mem)
            chosen = sorted(blocks, key=lambda bp: (-blocks[bp][0], bp))[:k2]
            chosen_all[j] = sorted(chosen)
            for bp, (sc_b, nu_b, mem) in blocks.items():
                if bp in chosen:
                    for u in mem:
                        logits.append(sg * q @ p["K"][u]); vals.append(p["V"][u])
                else:
                    logits.append(sc_b); vals.append(nu_b)
        for u in range(b * Bs, t + 1):
            logits.append(sg * q @ p["K"][u]); vals.append(p["V"][u])
        logits = np.array(logits); vals = np.array(vals)
        mx = logits.max(); w = np.exp(logits - mx)
        L[t] = mx + np.log(w.sum()); O[t] = (w / w.sum()) @ vals
        CH.append(chosen_all)
    return O, L, CH


@pytest.mark.parametrize("m,k2", [(2, 1), (3, 2), (6, 1), (1, 3)])
def test_two_level_equals_bruteforce_union_softmax(m, k2):
    p = toy_problem(21, N=64, D=4, Cq=3, Ck=6, S=4)
    f = orc.forward(p["Q"], p["K"], p["V"], p["a_q"], p["a_k"], p["qbar"], sigma=p["sigma"], S=p["S"],
                    Ck=p["Ck"], m=m, k2=k2)
    O, L, CH = _bruteforce_two_level(p, m, k2)
    np.testing.assert_allclose(f["O"], O, atol=1e-12)
    np.testing.assert_allclose(f["LSE"], L, atol=1e-12)
    for t in range(p["N"]):
        for k, j in enumerate(f["sel"][t]):
            if j >= 0:
                assert sorted(x for x in f["bsel"][t, k] if x >= 0) == CH[t][int(j)]


def test_all_blocks_selected_is_single_level():
    p = toy_problem(22)
    kw = dict(sigma=p["sigma"], S=p["S"], Ck=p["Ck"], m=2)
    f0 = orc.forward(p["Q"], p["K"], p["V"], p["a_q"], p["a_k"], p["qbar"], **kw)
    for k2 in (p["S"] - 1, p["S"] + 3):
        f = orc.forward(p["Q"], p["K"], p["V"], p["a_q"], p["a_k"], p["qbar"], k2=k2, **kw)
        np.testing.assert_array_equal(f["O"], f0["O"])
        np.testing.assert_array_equal(f["LSE"], f0["LSE"])
        assert np.all(~np.isfinite(f["lse_near"]))


def test_select_blocks_order_ties_and_padding():
    bl = np.array([0.5, -np.inf, 0.5, 2.0, -np.inf])
    assert orc.select_blocks(bl, 1).tolist() == [3]
    assert orc.select_blocks(bl, 2).tolist() == [3, 0]             # tie between blocks 0 and 2 -> lower index
    assert orc.select_blocks(bl, 4).tolist() == [3, 0, 2, -1]      # only three blocks hold keys


@pytest.mark.parametrize("k2", [1, 2])
def test_two_level_singleton_key_clusters_are_exact(k2):
    # a block summary of a single key is that key: every stand-in is exact
    p = toy_problem(23, N=48, S=4)
    a_k = np.arange(48, dtype=np.int32)
    f = orc.forward(p["Q"], p["K"], p["V"], p["a_q"], a_k, p["qbar"], sigma=p["sigma"], S=4, Ck=48, m=5, k2=k2)
    O, L = dense_causal_attention(p["Q"], p["K"], p["V"], p["sigma"])
    np.testing.assert_allclose(f["O"], O, atol=1e-12)
    np.testing.assert_allclose(f["LSE"], L, atol=1e-12)


def test_two_level_singleton_query_clusters_are_exact():
    # zero residual: every summary carries the exact mass and value mean of its keys
    p = toy_problem(24, N=48, S=4)
    a_q = np.arange(48, dtype=np.int32)
    f = orc.forward(p["Q"], p["K"], p["V"], a_q, p["a_k"], p["Q"].copy(), sigma=p["sigma"], S=4,
                    Ck=p["Ck"], m=2, k2=1)
    O, _ = dense_causal_attention(p["Q"], p["K"], p["V"], p["sigma"])
    np.testing.assert_allclose(f["O"], O, atol=1e-12)


def test_two_level_weights_sum_to_one_and_are_causal():
    p = toy_problem(25, N=64)
    N = 64
    kw = dict(sigma=p["sigma"], S=p["S"], Ck=p["Ck"], m=3, k2=1)
    ones = orc.forward(p["Q"], p["K"], np.ones((N, 3)), p["a_q"], p["a_k"], p["qbar"], **kw)
    np.testing.assert_allclose(ones["O"], 1.0, atol=1e-13)
    W = orc.forward(p["Q"], p["K"], np.eye(N), p["a_q"], p["a_k"], p["qbar"], **kw)["O"]
    assert W.min() >= 0 and np.abs(np.triu(W, 1)).max() == 0
    np.testing.assert_allclose(W.sum(1), 1.0, atol=1e-13)


def test_two_level_merge_matches_components_and_forced_blocks():
    p = toy_problem(26)
    kw = dict(sigma=p["sigma"], S=p["S"], Ck=p["Ck"], m=2, k2=1)
    f = orc.forward(p["Q"], p["K"], p["V"], p["a_q"], p["a_k"], p["qbar"], **kw)
    lses = np.stack([f["lse_far"], f["lse_near"], f["lse_ret"], f["lse_loc"]], 1)
    mx = lses.max(1, keepdims=True)
    L = (mx + np.log(np.exp(lses - mx).sum(1, keepdims=True)))[:, 0]
    np.testing.assert_allclose(f["LSE"], L, atol=1e-12)
    O = sum(np.exp(f["lse_" + c] - L)[:, None] * f["o_" + c] for c in ("far", "near", "ret", "loc"))
    np.testing.assert_allclose(f["O"], O, atol=1e-12)
    # forcing the clusters and blocks it chose reproduces the result; forcing others changes it
    g = orc.forward(p["Q"], p["K"], p["V"], p["a_q"], p["a_k"], p["qbar"], sel=f["sel"], bsel=f["bsel"], **kw)
    np.testing.assert_array_equal(g["O"], f["O"])
    other = np.where(f["bsel"] >= 0, 0, -1).astype(np.int32)
    h = orc.forward(p["Q"], p["K"], p["V"], p["a_q"], p["a_k"], p["qbar"], sel=f["sel"], bsel=other, **kw)
    assert np.abs(h["O"] - f["O"]).max() > 1e-6


def test_two_level_argument_rules():
    p = toy_problem(27)
    with pytest.raises(ValueError):
        orc.forward(p["Q"], p["K"], p["V"], p["a_q"], p["a_k"], p["qbar"], sigma=p["sigma"], S=p["S"], Ck=p["Ck"], m=2, k2=-1)
    with pytest.raises(ValueError):
        orc.forward(p["Q"], p["K"], p["V"], p["a_q"], p["a_k"], p["qbar"], sigma=p["sigma"], S=p["S"], Ck=p["Ck"], m=0, k2=1, dipole=1)


# ------------------------------------------------------------------ backward with two-level retrieval

def _fd(fun, X, h=1e-5):
    import itertools
    g = np.zeros_like(X)
    for idx in itertools.product(*map(range, X.shape)):
        old = X[idx]
        X[idx] = old + h; fp = fun()
        X[idx] = old - h; fm = fun()
        X[idx] = old
        g[idx] = (fp - fm) / (2 * h)
    return g


@pytest.mark.parametrize("m,k2,agg", [(2, 1, True), (3, 2, True), (2, 1, False)])
def test_two_level_backward_matches_finite_differences(m, k2, agg):
    """Central differences of sum(O * dO) with the chosen clusters and blocks held fixed.  With agg = False the
    reference forward rebuilds both kinds of summaries with the tilt weights frozen at their initial values."""
    p = toy_problem(23, N=40, D=4, Dv=3, Cq=3, Ck=4, S=5, gain=2.0)
    N, S, Ck, sg = p["N"], p["S"], p["Ck"], p["sigma"]
    kw = dict(sigma=sg, S=S, Ck=Ck, m=m, k2=k2)
    f0 = orc.forward(p["Q"], p["K"], p["V"], p["a_q"], p["a_k"], p["qbar"], **kw)
    sel, bsel = f0["sel"], f0["bsel"]
    assert (bsel >= 0).any() and np.isfinite(f0["lse_near"]).any()          # both kinds of key occur
    Q, K, V = p["Q"].copy(), p["K"].copy(), p["V"].copy()
    K0 = p["K"].copy()
    Bs = N // S
    blk = np.arange(N) // Bs

    def frozen(kind):
        """accumulated ('acc') or per-block ('blk') summaries with weights from K0 and the original log-masses"""
        mu0 = f0["summ"][0] if kind == "acc" else orc.block_summaries(K0, p["V"], p["a_k"], p["qbar"], sg, S, Ck)[0]
        ka = np.zeros((S, p["Cq"], Ck, p["D"])); nu = np.zeros((S, p["Cq"], Ck, V.shape[1]))
        for b in range(S):
            for j in range(Ck):
                mem = np.nonzero(((blk < b) if kind == "acc" else (blk == b)) & (p["a_k"] == j))[0]
                if mem.size:
                    w = np.exp(sg * p["qbar"] @ K0[mem].T - mu0[b, :, j][:, None])
                    ka[b, :, j] = w @ K[mem]; nu[b, :, j] = w @ V[mem]
        return mu0, ka, nu

    def loss():
        extra = {} if agg else dict(summ=frozen("acc"), blocks=frozen("blk"))
        return (orc.forward(Q, K, V, p["a_q"], p["a_k"], p["qbar"], sel=sel, bsel=bsel, **extra, **kw)["O"] * p["dO"]).sum()
    dQ, dK, dV, fwd = orc.backward(Q, K, V, p["dO"], p["a_q"], p["a_k"], p["qbar"], sel=sel, bsel=bsel, agg_grad=agg, **kw)
    np.testing.assert_allclose(fwd["O"], f0["O"], atol=1e-13)
    for g, X in ((dQ, Q), (dK, K), (dV, V)):
        fd = _fd(loss, X)
        assert np.abs(g - fd).max() <= 1e-6 * np.abs(fd).max()


def test_two_level_backward_with_every_block_chosen_is_the_single_level_backward():
    p = toy_problem(24, N=32, D=4, Dv=3, Cq=3, Ck=4, S=4, gain=2.0)
    kw = dict(sigma=p["sigma"], S=p["S"], Ck=p["Ck"], m=2)
    a = orc.backward(p["Q"], p["K"], p["V"], p["dO"], p["a_q"], p["a_k"], p["qbar"], **kw)
    b = orc.backward(p["Q"], p["K"], p["V"], p["dO"], p["a_q"], p["a_k"], p["qbar"], k2=p["S"] - 1, **kw)
    for x, y in zip(a[:3], b[:3]):
        np.testing.assert_allclose(x, y, atol=1e-12)
