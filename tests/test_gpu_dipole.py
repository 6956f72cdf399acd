"""GPU parity for the dipole correction of the far field (untilted, pre-merged; alone with m = 0 and next to
retrieval with m > 0, where the retrieved clusters leave the merged matrix): merged matrices and forward outputs
against the fp64 oracle, teacher-forced clustering (and, with m > 0, the GPU's own selection handed to the oracle).
Tolerance: max-abs error relative to the oracle tensor's max-abs <= 1e-4 (fp32 mode), 2e-2 (bf16 mode)."""
import numpy as np
import pytest
import torch

from oracle import muse_oracle as orc
from tests.gpu_util import Case, to_dev, to_np, tol, rel_err, kernels_launched
from tests.test_gpu_cluster import CASES

pytestmark = pytest.mark.gpu

DIPOLE_CASES = {
    "tiny_f32": (CASES["tiny"].with_(m=0), True),
    "tiny_f32_noncausal": (CASES["tiny"].with_(m=0), False),
    "gqa_bf16_d64": (CASES["gqa_bf16"].with_(B=1, Hq=2, Hkv=1, m=0), True),            # tensor merge, D = 64, Cq < 128
    "d128_bf16": (CASES["d128"].with_(m=0), True),                                      # tensor merge, ragged Cq = 24
    "d128_bf16_two_halves": (CASES["d128"].with_(m=0, Hq=1, Hkv=1, N=2048, Cq=160, Ck=64), True),
    "d128_f32_odd_ck": (CASES["d128"].with_(dtype="f32", m=0, Hq=1, Hkv=1, N=1000, Cq=8, Ck=24, S=4), True),
    # next to retrieval
    "tiny_f32_m2": (CASES["tiny"].with_(m=2), True),
    "tiny_f32_m2_noncausal": (CASES["tiny"].with_(m=2), False),
    "gqa_bf16_d64_m6": (CASES["gqa_bf16"].with_(B=1, Hq=4, Hkv=2, m=6), True),
    "d128_bf16_m8": (CASES["d128"].with_(m=8), True),
    "d128_f32_odd_ck_m5": (CASES["d128"].with_(dtype="f32", m=5, Hq=1, Hkv=1, N=1000, Cq=8, Ck=24, S=4), True),
}


def _cbar(mb, p, buf):
    off = mb.muse_summaries_layout(p)
    n = p.B * p.Hq * p.SB * p.Cq * p.D * p.D
    if p.dtype == mb.MUSE_F32 or p.m > 0:
        t = buf.summaries[off[7]:off[7] + 4 * n].view(torch.float32)
    else:
        t = buf.summaries[off[7]:off[7] + 2 * n].view(torch.bfloat16).float()
    return to_np(t).reshape(p.B, p.Hq, p.SB, p.Cq, p.D, p.D)


@pytest.mark.parametrize("name", list(DIPOLE_CASES))
@pytest.mark.parametrize("gain", [1.0, 128.0])
def test_dipole_forward_matches_oracle(name, gain):
    from paper_2509_10406_b200 import binding as mb
    w, causal = DIPOLE_CASES[name]
    c = Case(w, gain=gain)
    qbar32 = c.qbar.astype(np.float32)
    p = c.params(dipole=1, causal=causal)
    buf = mb.MuseBuffers(p, backward=False)
    Q, K, V, _ = c.dev()
    a_q, a_k, qb = to_dev(c.a_q, "i"), to_dev(c.a_k, "i"), to_dev(qbar32, "f32")
    mb.muse_summarize(p, K, V, a_k, qb, buf.off_k, buf.perm_k, buf.summaries, buf.ws)
    mb.muse_attn_fwd(p, Q, K, V, a_q, qb, buf.off_k, buf.perm_k, buf.summaries, None, buf.O, buf.LSE, buf.sel, buf.ws)
    torch.cuda.synchronize()
    assert int(buf.ws[:4].view(torch.int32)[0]) == 0
    O, L, cb, sel = to_np(buf.O), to_np(buf.LSE), _cbar(mb, p, buf), to_np(buf.sel)
    t = tol(w.dtype)
    S = w.S if causal else 1
    moved = 0.0
    for b in range(w.B):
        for h in range(w.Hq):
            g = c.hm[h]
            kw = dict(sigma=c.sigma, S=w.S, Ck=w.Ck, m=w.m, causal=causal, sel=sel[b, h] if w.m > 0 else None)
            f1 = orc.forward(c.Q[b, h], c.K[b, g], c.V[b, g], c.a_q[b, h], c.a_k[b, g], qbar32[b, h].astype(np.float64), dipole=1, **kw)
            f0 = orc.forward(c.Q[b, h], c.K[b, g], c.V[b, g], c.a_q[b, h], c.a_k[b, g], qbar32[b, h].astype(np.float64),
                             summ=f1["summ"], **kw)
            ref = f1["cbar"][1:] if causal else f1["cbar"]
            assert ref.shape == cb[b, h].shape and len(ref) == (S - 1 if causal else 1)
            # the matrices only matter for query clusters that own queries in the plane's block
            assert rel_err(cb[b, h], ref) <= t
            assert rel_err(O[b, h], f1["O"]) <= t
            assert np.abs(L[b, h] - f1["LSE"]).max() <= 1e-3 * max(1.0, np.abs(f1["LSE"]).max())
            moved = max(moved, rel_err(f0["O"], f1["O"]))
            # the GPU result must be closer to the oracle with the correction than to the one without,
            # wherever the correction is larger than the tolerance
            if rel_err(f0["O"], f1["O"]) > 4 * t:
                assert rel_err(O[b, h], f1["O"]) < rel_err(O[b, h], f0["O"])
    assert moved > 0.0


def test_dipole_argument_rules():
    from paper_2509_10406_b200 import binding as mb
    w = CASES["tiny"]
    with pytest.raises(mb.MuseError):
        mb.muse_workspace_bytes(mb.make_params(B=1, Hq=1, Hkv=1, N=w.N, D=w.D, Cq=w.Cq, Ck=w.Ck, m=2, dipole=1, k2=1))
    with pytest.raises(mb.MuseError):
        mb.muse_workspace_bytes(mb.make_params(B=1, Hq=1, Hkv=1, N=w.N, D=w.D, Cq=w.Cq, Ck=w.Ck, m=2, dipole=3))
    p0 = mb.make_params(B=1, Hq=1, Hkv=1, N=w.N, D=w.D, Cq=w.Cq, Ck=w.Ck, m=0, dtype="f32")
    p1 = mb.make_params(B=1, Hq=1, Hkv=1, N=w.N, D=w.D, Cq=w.Cq, Ck=w.Ck, m=0, dtype="f32", dipole=1)
    s0, s1 = mb.muse_workspace_bytes(p0), mb.muse_workspace_bytes(p1)
    assert s1[4] >= s0[4] + 7 * (w.Cq + w.Ck) * w.D * w.D * 4
    assert mb.muse_summaries_layout(p0)[7] == s0[4]


# ------------------------------------------------------------------ backward through the dipole correction

BWD_CASES = {
    "tiny_f32": (CASES["tiny"].with_(m=0), True, True),
    "tiny_f32_m2": (CASES["tiny"].with_(m=2), True, True),
    "tiny_f32_m2_noncausal": (CASES["tiny"].with_(m=2), False, True),
    "tiny_f32_m2_frozen": (CASES["tiny"].with_(m=2), True, False),
    "gqa_bf16_d64": (CASES["gqa_bf16"].with_(B=1, Hq=4, Hkv=2, m=0), True, True),
    "gqa_bf16_d64_m6": (CASES["gqa_bf16"].with_(B=1, Hq=4, Hkv=2, m=6), True, True),
    "d128_bf16_m8": (CASES["d128"].with_(m=8), True, True),                             # tensor-core far field and key-side pass
    "d128_f32_odd_ck_m5": (CASES["d128"].with_(dtype="f32", m=5, Hq=1, Hkv=1, N=1000, Cq=8, Ck=24, S=4), True, True),
    # C_q a multiple of 64: the two dense contractions of the backward run on the tensor cores
    "d128_bf16_tc_m4": (CASES["d128"].with_(Hq=1, Hkv=1, N=1024, Cq=64, Ck=128, m=4, S=4), True, True),
    "d64_bf16_tc_ragged_ck": (CASES["gqa_bf16"].with_(B=1, Hq=2, Hkv=1, N=1024, Cq=128, Ck=72, m=3, S=4), True, True),
    "d64_bf16_tc_m0": (CASES["gqa_bf16"].with_(B=1, Hq=2, Hkv=2, N=1024, Cq=64, Ck=200, m=0, S=4), True, True),
    # odd sizes everywhere, three query heads per kv head, two batches
    "odd_f32_gqa3": (CASES["tiny"].with_(name="odd3", B=2, Hq=3, Hkv=1, N=720, S=3, Cq=5, Ck=13, m=3, components=16), True, True),
    "odd_f32_d128_noncausal": (CASES["d128"].with_(name="odd128", dtype="f32", Hq=2, Hkv=2, N=516, S=2, Cq=3, Ck=7, m=2, components=8), False, True),
}
TC_DIPOLE_BWD = {"k_dipole_dcov_tc", "k_dipole_dpw_tc"}


@pytest.mark.parametrize("name", list(BWD_CASES))
def test_dipole_backward_matches_oracle(name):
    from paper_2509_10406_b200 import binding as mb
    w, causal, agg = BWD_CASES[name]
    with kernels_launched() as rec:
        _dipole_backward_case(mb, name, w, causal, agg)
    assert ("_tc_" in name) == TC_DIPOLE_BWD.issubset(rec.names), sorted(rec.names)


def test_dipole_backward_contractions_on_the_plain_kernels_at_a_tensor_shape():
    from paper_2509_10406_b200 import binding as mb
    w, causal, agg = BWD_CASES["d64_bf16_tc_ragged_ck"]
    mb.muse_test_force_paths(mb.FORCE_DIPOLE_SIMT)
    try:
        with kernels_launched() as rec:
            _dipole_backward_case(mb, "forced", w, causal, agg)
    finally:
        mb.muse_test_force_paths(0)
    assert {"k_dipole_dcov", "k_dipole_dpw"}.issubset(rec.names) and not (TC_DIPOLE_BWD & rec.names)


def _dipole_backward_case(mb, name, w, causal, agg):
    gain = 128.0
    c = Case(w, gain=gain)
    qbar32 = c.qbar.astype(np.float32)
    p = c.params(dipole=1, causal=causal, agg_grad=agg)
    buf = mb.MuseBuffers(p, backward=True)
    Q, K, V, dO = c.dev()
    aq, qb = to_dev(c.a_q, "i"), to_dev(qbar32, "f32")
    mb.muse_summarize(p, K, V, to_dev(c.a_k, "i"), qb, buf.off_k, buf.perm_k, buf.summaries, buf.ws)
    mb.muse_attn_fwd(p, Q, K, V, aq, qb, buf.off_k, buf.perm_k, buf.summaries, None, buf.O, buf.LSE, buf.sel, buf.ws)
    assert mb.muse_status(buf.ws) == 0
    mb.muse_attn_bwd(p, Q, K, V, buf.O, buf.LSE, dO, aq, qb, buf.off_k, buf.perm_k, buf.summaries, buf.sel, buf.dQ, buf.dK, buf.dV, buf.ws)
    torch.cuda.synchronize()
    assert mb.muse_status(buf.ws) == 0
    sel = to_np(buf.sel)[..., :w.m]
    dQ, dK, dV = to_np(buf.dQ), to_np(buf.dK), to_np(buf.dV)
    kw = dict(sigma=c.sigma, S=w.S, Ck=w.Ck, m=w.m, causal=causal, sel=sel, agg_grad=agg)
    args = (c.Q.astype(np.float64), c.K.astype(np.float64), c.V.astype(np.float64), c.dO.astype(np.float64), c.a_q, c.a_k,
            qbar32.astype(np.float64))
    eQ, eK, eV = orc.layer_backward(*args, dipole=1, **kw)
    pQ, pK, pV = orc.layer_backward(*args, **kw)                 # without the correction
    errs = dict(dQ=rel_err(dQ, eQ), dK=rel_err(dK, eK), dV=rel_err(dV, eV))
    moved = dict(dQ=rel_err(pQ, eQ), dK=rel_err(pK, eK), dV=rel_err(pV, eV))
    print(name, errs, "correction moves the gradients by", moved)
    t = tol(w.dtype)
    assert all(v <= t for v in errs.values()), errs
    # the comparison must be able to see the dipole terms: where they exceed the tolerance, the GPU is on the right side
    for key, got, e, plain in (("dQ", dQ, eQ, pQ), ("dK", dK, eK, pK), ("dV", dV, eV, pV)):
        if moved[key] > 4 * t:
            assert rel_err(got, e) < rel_err(got, plain), key
    assert max(moved.values()) > 4 * t or w.dtype != "f32"


# ------------------------------------------------------------------ shared covariance tilted at the mean query centroid

TILT_CASES = {
    "tiny_f32": (CASES["tiny"].with_(m=0), True, True),
    "tiny_f32_m2": (CASES["tiny"].with_(m=2), True, True),
    "tiny_f32_m2_frozen": (CASES["tiny"].with_(m=2), True, False),
    "tiny_f32_m2_noncausal": (CASES["tiny"].with_(m=2), False, True),
    "gqa_bf16_d64_m6": (CASES["gqa_bf16"].with_(B=1, Hq=4, Hkv=2, m=6), True, True),     # covariances per query head
    "d128_bf16_m8": (CASES["d128"].with_(m=8), True, True),
    "odd_f32_gqa3": (CASES["tiny"].with_(name="odd3", B=2, Hq=3, Hkv=1, N=720, S=3, Cq=5, Ck=13, m=3, components=16), True, True),
    "odd_bf16_d128_m0": (CASES["d128"].with_(name="odd128", Hq=2, Hkv=2, N=516, S=2, Cq=3, Ck=7, m=0, components=8), True, False),
}


@pytest.mark.parametrize("name", list(TILT_CASES))
def test_tilted_dipole_forward_and_backward_match_oracle(name):
    from paper_2509_10406_b200 import binding as mb
    w, causal, agg = TILT_CASES[name]
    c = Case(w, gain=128.0)
    qbar32 = c.qbar.astype(np.float32)
    p = c.params(dipole=2, causal=causal, agg_grad=agg)
    buf = mb.MuseBuffers(p, backward=True)
    Q, K, V, dO = c.dev()
    aq, qb = to_dev(c.a_q, "i"), to_dev(qbar32, "f32")
    mb.muse_dipole_tilt_point(p, aq, qb, buf.summaries)
    mb.muse_summarize(p, K, V, to_dev(c.a_k, "i"), qb, buf.off_k, buf.perm_k, buf.summaries, buf.ws)
    mb.muse_attn_fwd(p, Q, K, V, aq, qb, buf.off_k, buf.perm_k, buf.summaries, None, buf.O, buf.LSE, buf.sel, buf.ws)
    assert mb.muse_status(buf.ws) == 0
    mb.muse_attn_bwd(p, Q, K, V, buf.O, buf.LSE, dO, aq, qb, buf.off_k, buf.perm_k, buf.summaries, buf.sel, buf.dQ, buf.dK, buf.dV, buf.ws)
    torch.cuda.synchronize()
    assert mb.muse_status(buf.ws) == 0
    off = mb.muse_dipole_layout(p)
    qstar = to_np(buf.summaries[off[4]:off[4] + 4 * w.B * w.Hq * w.D].view(torch.float32)).reshape(w.B, w.Hq, w.D)
    sel = to_np(buf.sel)[..., :w.m]
    O, dQ, dK, dV = to_np(buf.O), to_np(buf.dQ), to_np(buf.dK), to_np(buf.dV)
    t = tol(w.dtype)
    kw = dict(sigma=c.sigma, S=w.S, Ck=w.Ck, m=w.m, causal=causal)
    far_apart = 0.0
    for b in range(w.B):
        for h in range(w.Hq):
            g = c.hm[h]
            q64 = qbar32[b, h].astype(np.float64)
            np.testing.assert_allclose(qstar[b, h], orc.mean_query_centroid(q64, c.a_q[b, h]), rtol=1e-5, atol=1e-6)
            f2 = orc.forward(c.Q[b, h], c.K[b, g], c.V[b, g], c.a_q[b, h], c.a_k[b, g], q64, dipole=2, sel=sel[b, h] if w.m else None, **kw)
            f1 = orc.forward(c.Q[b, h], c.K[b, g], c.V[b, g], c.a_q[b, h], c.a_k[b, g], q64, dipole=1, sel=sel[b, h] if w.m else None,
                             summ=f2["summ"], **kw)
            assert rel_err(O[b, h], f2["O"]) <= t
            far_apart = max(far_apart, rel_err(f1["O"], f2["O"]))
            if rel_err(f1["O"], f2["O"]) > 4 * t:
                assert rel_err(O[b, h], f2["O"]) < rel_err(O[b, h], f1["O"])
    args = (c.Q.astype(np.float64), c.K.astype(np.float64), c.V.astype(np.float64), c.dO.astype(np.float64), c.a_q, c.a_k,
            qbar32.astype(np.float64))
    eQ, eK, eV = orc.layer_backward(*args, dipole=2, sel=sel, agg_grad=agg, **kw)
    uQ, uK, uV = orc.layer_backward(*args, dipole=1, sel=sel, agg_grad=agg, **kw)
    errs = dict(dQ=rel_err(dQ, eQ), dK=rel_err(dK, eK), dV=rel_err(dV, eV))
    moved = dict(dQ=rel_err(uQ, eQ), dK=rel_err(uK, eK), dV=rel_err(uV, eV))
    print(name, errs, "tilt moves the output by", far_apart, "and the gradients by", moved)
    assert all(v <= t for v in errs.values()), errs
    for key, got, e, plain in (("dQ", dQ, eQ, uQ), ("dK", dK, eK, uK), ("dV", dV, eV, uV)):
        if moved[key] > 4 * t:
            assert rel_err(got, e) < rel_err(got, plain), key
    if w.dtype == "f32":
        assert far_apart > 4 * t and max(moved.values()) > 4 * t


@pytest.mark.parametrize("dipole", [1, 2])
def test_dipole_backward_rebuilds_summaries_when_not_given(dipole):
    """muse_attn_bwd with summaries == NULL rebuilds them (with the dipole's arrays and, for dipole == 2, the tilt point)
    in the tail of its scratch: same gradients as with the forward's buffer."""
    from paper_2509_10406_b200 import binding as mb
    w = CASES["tiny"].with_(m=2)
    c = Case(w, gain=128.0)
    qbar32 = c.qbar.astype(np.float32)
    p = c.params(dipole=dipole)
    buf = mb.MuseBuffers(p, backward=True)
    Q, K, V, dO = c.dev()
    aq, qb = to_dev(c.a_q, "i"), to_dev(qbar32, "f32")
    if dipole == 2:
        mb.muse_dipole_tilt_point(p, aq, qb, buf.summaries)
    mb.muse_summarize(p, K, V, to_dev(c.a_k, "i"), qb, buf.off_k, buf.perm_k, buf.summaries, buf.ws)
    mb.muse_attn_fwd(p, Q, K, V, aq, qb, buf.off_k, buf.perm_k, buf.summaries, None, buf.O, buf.LSE, buf.sel, buf.ws)
    res = []
    for summ, ws in ((buf.summaries, buf.ws), (None, torch.empty(buf.sizes[5], dtype=torch.uint8, device="cuda"))):
        mb.muse_attn_bwd(p, Q, K, V, buf.O, buf.LSE, dO, aq, qb, buf.off_k, buf.perm_k, summ, buf.sel, buf.dQ, buf.dK, buf.dV, ws)
        torch.cuda.synchronize()
        assert mb.muse_status(ws) == 0
        res.append((to_np(buf.dQ).copy(), to_np(buf.dK).copy(), to_np(buf.dV).copy()))
    for a, b in zip(*res):
        assert rel_err(b, a) <= 1e-5


def test_dipole_with_selection_per_query_cluster_and_with_a_single_block():
    """Selection per query cluster (every query of a segment retrieves the same clusters) next to the dipole, forward and
    backward; and one causal block (no far field at all): the dipole then changes nothing and nothing faults."""
    from paper_2509_10406_b200 import binding as mb
    w = CASES["tiny"].with_(m=2)
    c = Case(w, gain=128.0)
    qbar32 = c.qbar.astype(np.float32)
    Q, K, V, dO = c.dev()
    aq, qb = to_dev(c.a_q, "i"), to_dev(qbar32, "f32")
    args = (c.Q.astype(np.float64), c.K.astype(np.float64), c.V.astype(np.float64), c.dO.astype(np.float64), c.a_q, c.a_k,
            qbar32.astype(np.float64))

    def run(p):
        buf = mb.MuseBuffers(p, backward=True)
        if p.dipole == 2:
            mb.muse_dipole_tilt_point(p, aq, qb, buf.summaries)
        mb.muse_summarize(p, K, V, to_dev(c.a_k, "i"), qb, buf.off_k, buf.perm_k, buf.summaries, buf.ws)
        mb.muse_attn_fwd(p, Q, K, V, aq, qb, buf.off_k, buf.perm_k, buf.summaries, None, buf.O, buf.LSE, buf.sel, buf.ws)
        mb.muse_attn_bwd(p, Q, K, V, buf.O, buf.LSE, dO, aq, qb, buf.off_k, buf.perm_k, buf.summaries, buf.sel, buf.dQ, buf.dK, buf.dV, buf.ws)
        torch.cuda.synchronize()
        assert mb.muse_status(buf.ws) == 0
        return to_np(buf.O), to_np(buf.dQ), to_np(buf.dK), to_np(buf.dV), to_np(buf.sel)[..., :w.m]

    O, dQ, dK, dV, sel = run(c.params(dipole=2, sel_mode=1))
    kw = dict(sigma=c.sigma, S=w.S, Ck=w.Ck, m=w.m, sel=sel, sel_mode=1, dipole=2)
    eO, _, _ = orc.layer_forward(*args[:3], *args[4:], **kw)
    eQ, eK, eV = orc.layer_backward(*args, **kw)
    for got, ref in ((O, eO), (dQ, eQ), (dK, eK), (dV, eV)):
        assert rel_err(got, ref) <= 1e-4
    # every query of a segment carries its cluster's selection
    Bs = w.N // w.S
    for t in range(Bs, w.N, 37):
        same = (c.a_q[0, 0] == c.a_q[0, 0, t]) & (np.arange(w.N) // Bs == t // Bs)
        assert (sel[0, 0][same] == sel[0, 0, t]).all()
    one = run(c.params(dipole=1, n_blocks=1))
    ref = run(c.params(dipole=0, n_blocks=1))
    for a, b in zip(one[:4], ref[:4]):
        np.testing.assert_array_equal(a, b)
