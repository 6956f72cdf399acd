"""GPU parity at the benchmark's full size and launch configuration (headline workload,
all 16 heads in one call).  The oracle cannot run the whole problem, so it is evaluated on
sampled points / queries of one head with the GPU's assignments, centroids and selections
forced on it, and properties that hold at any size cover the rest:
  * assignments of sampled points vs brute-force nearest centre (near-ties excepted),
  * O, LSE and dQ of sampled queries vs the oracle (bf16-mode tolerance 2e-2),
  * sum_u dV_u = sum_t dO_t   (attention weights, exact and far-field, sum to one),
  * sum_u dK_u = 0            (softmax is invariant to a translation of all keys)."""
import numpy as np
import pytest
import torch

from oracle import muse_oracle as orc
from paper_2509_10406_b200 import workloads as wl
from tests.gpu_util import Case, to_dev, to_np, rel_err, kernels_launched

pytestmark = pytest.mark.gpu


def test_headline_full_size_sampled_parity():
    import bench
    from paper_2509_10406_b200 import binding as mb
    w = wl.WORKLOADS["headline"]
    gain = 128.0                                     # sharp attention, so that selection and retrieval matter
    Qh, Kh, Vh, dOh, iq, ik = bench.gen_inputs(w, gain)
    dev = lambda a: torch.from_numpy(a).to(torch.bfloat16).cuda()
    Q, K, V, dO = dev(Qh), dev(Kh), dev(Vh), dev(dOh)
    p = mb.make_params(B=w.B, Hq=w.Hq, Hkv=w.Hkv, N=w.N, D=w.D, Cq=w.Cq, Ck=w.Ck, m=w.m, n_blocks=w.S, dtype=w.dtype,
                       kmeans_iters=w.T)
    buf = mb.MuseBuffers(p, backward=True)
    mb.muse_layer_forward(p, buf, Q, K, V, torch.from_numpy(iq).cuda(), torch.from_numpy(ik).cuda())
    mb.muse_layer_backward(p, buf, Q, K, V, dO)
    torch.cuda.synchronize()
    assert mb.muse_status(buf.ws) == 0                            # no bounded wait gave up (backward call)
    h = 5
    a_q, a_k = to_np(buf.assign_q[0, h]), to_np(buf.assign_k[0, h])
    qbar, kcent = to_np(buf.qbar[0, h]).astype(np.float64), to_np(buf.kcent[0, h]).astype(np.float64)
    rng = np.random.default_rng(0)
    # --- assignments of sampled points against the final centres
    pts = rng.choice(w.N, 4096, replace=False)
    for X, a, c in ((Qh[0, h], a_q, qbar), (Kh[0, h], a_k, kcent)):
        exp = orc.assign_nearest(X[pts], c)
        gaps = orc.assignment_gaps(X[pts], c)
        bad = np.nonzero(exp != a[pts])[0]
        assert np.all(gaps[bad] < 1e-4) and bad.size <= 8, (bad.size, gaps[bad])
    assert np.bincount(a_k, minlength=w.Ck).min() >= 0 and a_k.max() < w.Ck
    # --- sampled queries: O, LSE, dQ with the GPU's selections forced on the oracle
    rows = np.sort(np.concatenate([rng.choice(np.arange(b * 8192, (b + 1) * 8192), 3, replace=False) for b in range(8)]))
    sel = to_np(buf.sel[0, h])
    Q64, K64, V64, dO64 = (x[0, h].astype(np.float64) for x in (Qh, Kh, Vh, dOh))
    kw = dict(sigma=1.0 / np.sqrt(w.D), S=w.S, Ck=w.Ck, m=w.m, sel=sel, rows=rows)
    dQ, _, _, f = orc.backward(Q64, K64, V64, dO64, a_q, a_k, qbar, **kw)
    O, LSE, gQ = to_np(buf.O[0, h]), to_np(buf.LSE[0, h]), to_np(buf.dQ[0, h])
    errs = dict(O=rel_err(O[rows], f["O"][rows]), LSE=float(np.abs(LSE[rows] - f["LSE"][rows]).max() / np.abs(f["LSE"][rows]).max()),
                dQ=rel_err(gQ[rows], dQ[rows]))
    print("full-size sampled parity (head %d, %d queries):" % (h, rows.size), errs)
    assert all(v <= 2e-2 for v in errs.values()), errs
    # --- selections are valid: distinct, non-empty clusters with visible keys, none for block 0
    blk = rows // (w.N // w.S)
    for t, b in zip(rows, blk):
        s = sel[t][sel[t] >= 0]
        assert len(set(s.tolist())) == s.size and (b > 0 or s.size == 0)
        vis = np.bincount(a_k[: b * (w.N // w.S)], minlength=w.Ck) > 0
        assert np.all(vis[s])
    # --- identities that hold at any size (all heads)
    dV, dK = buf.dV.float(), buf.dK.float()
    sum_dO = dO.float().sum(2)
    assert float((dV.sum(2) - sum_dO).abs().max() / sum_dO.abs().max()) <= 2e-2
    assert float(dK.sum(2).abs().max() / dK.abs().sum(2).max()) <= 2e-2


def test_headline_shaped_head_elementwise_gradients():
    """One head with the headline workload's proportions (D = 128, 64 keys per key cluster, 32 retrieved
    clusters, 8 blocks, 32 queries per (cluster, block) segment) at a length the oracle can afford in full:
    O, LSE, dQ and — element by element — dK and dV against the oracle, so that a key-side term landing on
    the wrong key cannot hide behind a sum."""
    from paper_2509_10406_b200 import binding as mb
    w = wl.WORKLOADS["headline"].with_(name="headline_16k", Hq=1, Hkv=1, N=16384, Cq=64, Ck=256, m=32, components=256)
    c = Case(w, gain=128.0)
    qbar32 = c.qbar.astype(np.float32)
    p = c.params()
    buf = mb.MuseBuffers(p, backward=True)
    Q, K, V, dO = c.dev()
    aq, qb = to_dev(c.a_q, "i"), to_dev(qbar32, "f32")
    with kernels_launched() as rec:
        mb.muse_summarize(p, K, V, to_dev(c.a_k, "i"), qb, buf.off_k, buf.perm_k, buf.summaries, buf.ws)
        mb.muse_attn_fwd(p, Q, K, V, aq, qb, buf.off_k, buf.perm_k, buf.summaries, None, buf.O, buf.LSE, buf.sel, buf.ws)
        mb.muse_attn_bwd(p, Q, K, V, buf.O, buf.LSE, dO, aq, qb, buf.off_k, buf.perm_k, buf.summaries, buf.sel,
                         buf.dQ, buf.dK, buf.dV, buf.ws)
    assert mb.muse_status(buf.ws) == 0
    assert {"k_summarize_tc", "k_far_fwd_tc", "k_far_bwd_tc", "k_summ_bwd_tc", "k_local_fwd_tc"} <= rec.names, sorted(rec.names)
    sel = to_np(buf.sel)[..., :w.m]
    kw = dict(sigma=c.sigma, S=w.S, Ck=w.Ck, m=w.m)
    f = orc.forward(c.Q[0, 0], c.K[0, 0], c.V[0, 0], c.a_q[0, 0], c.a_k[0, 0], qbar32[0, 0].astype(np.float64), sel=sel[0, 0], **kw)
    eQ, eK, eV = orc.layer_backward(c.Q.astype(np.float64), c.K.astype(np.float64), c.V.astype(np.float64),
                                    c.dO.astype(np.float64), c.a_q, c.a_k, qbar32.astype(np.float64), causal=True, sel=sel,
                                    sel_mode=0, agg_grad=True, **kw)
    errs = dict(O=rel_err(to_np(buf.O)[0, 0], f["O"]), dQ=rel_err(to_np(buf.dQ), eQ), dK=rel_err(to_np(buf.dK), eK),
                dV=rel_err(to_np(buf.dV), eV))
    print("headline-shaped head, N = 16384:", errs)
    assert all(v <= 2e-2 for v in errs.values()), errs


def test_headline_full_size_tilted_dipole_next_to_retrieval_sampled_parity():
    """The dipole options at the benchmark's full size and launch configuration (`bench.py --dipole 2
    --dipole-with-retrieval`): shared covariance tilted at the mean query centroid, correction restricted to the clusters a
    query did not retrieve, forward and backward.  O, LSE and dQ of sampled queries of one head against the oracle with the
    GPU's assignments, centroids and selections; the sum identities on all heads (the correction has zero total weight:
    it moves values, not mass)."""
    import bench
    from paper_2509_10406_b200 import binding as mb
    w = wl.WORKLOADS["headline"]
    Qh, Kh, Vh, dOh, iq, ik = bench.gen_inputs(w, 128.0)
    dev = lambda a: torch.from_numpy(a).to(torch.bfloat16).cuda()
    Q, K, V, dO = dev(Qh), dev(Kh), dev(Vh), dev(dOh)
    p = mb.make_params(B=w.B, Hq=w.Hq, Hkv=w.Hkv, N=w.N, D=w.D, Cq=w.Cq, Ck=w.Ck, m=w.m, n_blocks=w.S, dtype=w.dtype,
                       kmeans_iters=w.T, dipole=2)
    buf = mb.MuseBuffers(p, backward=True)
    mb.muse_layer_forward(p, buf, Q, K, V, torch.from_numpy(iq).cuda(), torch.from_numpy(ik).cuda())
    mb.muse_layer_backward(p, buf, Q, K, V, dO)
    torch.cuda.synchronize()
    assert mb.muse_status(buf.ws) == 0
    h = 3
    a_q, a_k = to_np(buf.assign_q[0, h]), to_np(buf.assign_k[0, h])
    qbar = to_np(buf.qbar[0, h]).astype(np.float64)
    rng = np.random.default_rng(1)
    rows = np.sort(np.concatenate([rng.choice(np.arange(b * 8192, (b + 1) * 8192), 2, replace=False) for b in range(8)]))
    sel = to_np(buf.sel[0, h])
    Q64, K64, V64, dO64 = (x[0, h].astype(np.float64) for x in (Qh, Kh, Vh, dOh))
    kw = dict(sigma=1.0 / np.sqrt(w.D), S=w.S, Ck=w.Ck, m=w.m, sel=sel, rows=rows)
    dQ, _, _, f = orc.backward(Q64, K64, V64, dO64, a_q, a_k, qbar, dipole=2, **kw)
    plain = orc.forward(Q64, K64, V64, a_q, a_k, qbar, **kw)
    O, LSE, gQ = to_np(buf.O[0, h]), to_np(buf.LSE[0, h]), to_np(buf.dQ[0, h])
    errs = dict(O=rel_err(O[rows], f["O"][rows]), LSE=float(np.abs(LSE[rows] - f["LSE"][rows]).max() / np.abs(f["LSE"][rows]).max()),
                dQ=rel_err(gQ[rows], dQ[rows]))
    moved = rel_err(plain["O"][rows], f["O"][rows])
    print("full-size tilted dipole next to retrieval (head %d, %d queries):" % (h, rows.size), errs, "correction moves O by", moved)
    assert all(v <= 2e-2 for v in errs.values()), errs
    dV, dK = buf.dV.float(), buf.dK.float()
    sum_dO = dO.float().sum(2)
    assert float((dV.sum(2) - sum_dO).abs().max() / sum_dO.abs().max()) <= 2e-2
    assert float(dK.sum(2).abs().max() / dK.abs().sum(2).max()) <= 2e-2
