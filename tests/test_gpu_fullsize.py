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
from tests.gpu_util import to_np, rel_err

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
    assert int(buf.ws[:4].view(torch.int32).item()) == 0          # no bounded wait gave up
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
