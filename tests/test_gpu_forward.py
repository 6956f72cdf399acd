"""GPU parity: summaries and forward attention against the fp64 oracle, teacher-forced
(identical assignments and query centroids on both sides).  Tolerance: max-abs error
relative to the oracle tensor's max-abs <= 1e-4 in fp32 mode, 2e-2 in bf16 mode."""
import numpy as np
import pytest
import torch

from oracle import muse_oracle as orc
from paper_2509_10406_b200 import workloads as wl
from tests.gpu_util import Case, to_dev, to_np, tol, rel_err, kernels_launched
from tests.test_gpu_cluster import CASES

pytestmark = pytest.mark.gpu

EDGE = {
    "m0": CASES["gqa_bf16"].with_(B=1, Hq=2, Hkv=1, m=0),
    "one_block": CASES["tiny"].with_(S=1),
    # one causal block in bf16: the block-diagonal tensor-core kernels alone, over the whole sequence
    "one_block_bf16": CASES["d128"].with_(Hq=1, Hkv=1, N=2048, S=1, Cq=1, Ck=1, m=0),
    "one_qcluster": CASES["tiny"].with_(Cq=1, N=512),
    "tiny_blocks": CASES["tiny"].with_(N=64, Cq=2, Ck=8, m=8, components=4),
    "ragged_f32_d128": CASES["d128"].with_(dtype="f32", N=1000, Hq=1, Cq=8, Ck=24, m=3),
    # segments of ~128 queries (several 64-query sweeps per segment in the tensor far-field kernels) and key
    # clusters of ~128 keys (several key sweeps in the retrieval kernels)
    "long_segments": CASES["d128"].with_(Hq=1, Hkv=1, N=4096, S=4, Cq=8, Ck=128, m=4),
    "long_clusters": CASES["d128"].with_(Hq=1, Hkv=1, N=4096, S=4, Cq=16, Ck=16, m=4),
    # four key clusters that every query retrieves: ~48 tiles of 128 pairs per cluster, so that each cluster's
    # tiles are dealt to several CTAs of the retrieval kernels, and ~2000 keys per cluster (many key sweeps)
    "shared_clusters": CASES["d128"].with_(Hq=1, Hkv=1, N=8192, S=4, Cq=16, Ck=4, m=4),
    # 2048 key clusters: sixteen cluster tiles per segment in the tensor far-field backward (the forward far
    # field takes its other path above 1024 clusters)
    "many_key_clusters": CASES["d128"].with_(Hq=1, Hkv=1, N=4096, S=4, Cq=8, Ck=2048, m=4),
}


def _mb():
    from paper_2509_10406_b200 import binding as mb
    return mb


def _run_summaries(mb, c, p, buf, K, V):
    mb.muse_summarize(p, K, V, to_dev(c.a_k, "i"), to_dev(c.qbar32, "f32"), buf.off_k, buf.perm_k, buf.summaries, buf.ws)


def _prep(w, gain, **pk):
    mb = _mb()
    c = Case(w, gain=gain)
    c.qbar32 = c.qbar.astype(np.float32)
    p = c.params(**pk)
    buf = mb.MuseBuffers(p, backward=True)
    return mb, c, p, buf


@pytest.mark.parametrize("name", list(CASES))
@pytest.mark.parametrize("gain", [1.0, 128.0])
def test_summaries_match_oracle(name, gain):
    mb, c, p, buf = _prep(CASES[name], gain)
    w = c.w
    Q, K, V, _ = c.dev()
    _run_summaries(mb, c, p, buf, K, V)
    torch.cuda.synchronize()
    mu, beta, ka, nu = (to_np(x) for x in buf.summary_planes())
    t_nu = 1e-4 if w.dtype == "f32" else tol(w.dtype)     # nu is stored in bf16 in bf16 mode
    for b in range(w.B):
        for h in range(w.Hq):
            g = c.hm[h]
            muh, kah, nuh = orc.accumulated_summaries(c.K[b, g], c.V[b, g], c.a_k[b, g], c.qbar32[b, h].astype(np.float64),
                                                      c.sigma, w.S, w.Ck)
            e_mu, g_mu = muh[1:], mu[b, h]
            assert np.array_equal(np.isfinite(e_mu), np.isfinite(g_mu))
            fin = np.isfinite(e_mu)
            assert np.abs(e_mu[fin] - g_mu[fin]).max() <= 1e-4 * max(1.0, np.abs(e_mu[fin]).max())
            assert rel_err(ka[b, h], kah[1:]) <= 1e-4
            assert rel_err(nu[b, h], nuh[1:]) <= t_nu
            e_beta = e_mu - c.sigma * np.einsum("id,bijd->bij", c.qbar32[b, h].astype(np.float64), kah[1:])
            assert np.abs(e_beta[fin] - beta[b, h][fin]).max() <= 1e-4 * max(1.0, np.abs(e_beta[fin]).max())


# bf16, D = 128, C_k a multiple of 128, C_q a multiple of 8: shapes at which every far-field, summary and
# retrieval step runs its tcgen05 kernel; "tc_gqa4" has four query heads per kv head (the key-side group sum)
TC = {
    "tc": CASES["d128"].with_(name="tc", Hq=2, Hkv=1, N=4096, S=4, Cq=16, Ck=256, m=4),
    "tc_gqa4": CASES["d128"].with_(name="tc_gqa4", Hq=4, Hkv=1, N=2048, S=4, Cq=8, Ck=128, m=4),
    "tc_d64": CASES["d64"].with_(name="tc_d64", Hq=2, Hkv=1, N=4096, S=4, Cq=16, Ck=256, m=4),
    "tc_d64_gqa4": CASES["d64"].with_(name="tc_d64_gqa4", Hq=4, Hkv=1, N=2048, S=4, Cq=8, Ck=128, m=4),
}
TC_FWD_KERNELS = {"k_summarize_tc", "k_far_fwd_tc", "k_local_fwd_tc"}
TC_BWD_KERNELS = {"k_far_bwd_tc", "k_summ_bwd_tc"}


def _forward_parity(w, gain, sel_mode=0, causal=True, expect_kernels=()):
    with kernels_launched() as rec:
        _forward_parity_run(w, gain, sel_mode, causal)
    missing = set(expect_kernels) - rec.names
    assert not missing, ("expected kernels did not run", missing, sorted(rec.names))


def _forward_parity_run(w, gain, sel_mode=0, causal=True):
    mb, c, p, buf = _prep(w, gain, sel_mode=sel_mode, causal=causal)
    Q, K, V, _ = c.dev()
    _run_summaries(mb, c, p, buf, K, V)
    kw = dict(sigma=c.sigma, S=w.S, Ck=w.Ck, m=w.m, sel_mode=sel_mode, causal=causal)
    t = tol(w.dtype)
    # free selection on the GPU
    mb.muse_attn_fwd(p, Q, K, V, to_dev(c.a_q, "i"), to_dev(c.qbar32, "f32"), buf.off_k, buf.perm_k, buf.summaries,
                     None, buf.O, buf.LSE, buf.sel, buf.ws)
    torch.cuda.synchronize()
    assert mb.muse_status(buf.ws) == 0
    O_free, L_free, sel_gpu = to_np(buf.O), to_np(buf.LSE), to_np(buf.sel)[..., :w.m]
    stats = dict(sel_rows_differ=0, rows=0, err_forced_gpu_sel=0.0, err_forced_orc_sel=0.0)
    sel_orc = np.full((w.B, w.Hq, w.N, max(w.m, 1)), -1, np.int32)
    for b in range(w.B):
        for h in range(w.Hq):
            g = c.hm[h]
            args = (c.Q[b, h], c.K[b, g], c.V[b, g], c.a_q[b, h], c.a_k[b, g], c.qbar32[b, h].astype(np.float64))
            f = orc.forward(*args, **kw)
            sel_orc[b, h, :, :w.m] = f["sel"]
            # selections: equal as sets except where the oracle's margin is below tolerance
            same = np.array([set(x) == set(y) for x, y in zip(f["sel"].tolist(), sel_gpu[b, h].tolist())])
            assert np.all(f["sel_gap"][~same] < t), ("selection differs away from a near-tie", f["sel_gap"][~same].max())
            stats["sel_rows_differ"] += int((~same).sum()); stats["rows"] += w.N
            # outputs: oracle forced to the GPU's selections
            ff = orc.forward(*args, sel=sel_gpu[b, h], summ=f["summ"], **kw)
            e = max(rel_err(O_free[b, h], ff["O"]), float(np.abs(L_free[b, h] - ff["LSE"]).max() / max(1.0, np.abs(ff["LSE"]).max())))
            stats["err_forced_gpu_sel"] = max(stats["err_forced_gpu_sel"], e)
    assert stats["err_forced_gpu_sel"] <= t, stats
    # GPU forced to the oracle's selections
    mb.muse_attn_fwd(p, Q, K, V, to_dev(c.a_q, "i"), to_dev(c.qbar32, "f32"), buf.off_k, buf.perm_k, buf.summaries,
                     to_dev(sel_orc, "i"), buf.O, buf.LSE, buf.sel, buf.ws)
    torch.cuda.synchronize()
    O_f = to_np(buf.O)
    for b in range(w.B):
        for h in range(w.Hq):
            g = c.hm[h]
            f = orc.forward(c.Q[b, h], c.K[b, g], c.V[b, g], c.a_q[b, h], c.a_k[b, g], c.qbar32[b, h].astype(np.float64),
                            sel=sel_orc[b, h, :, :w.m], **kw)
            stats["err_forced_orc_sel"] = max(stats["err_forced_orc_sel"], rel_err(O_f[b, h], f["O"]))
    print(w.name, gain, stats)
    assert stats["err_forced_orc_sel"] <= t, stats
    assert stats["sel_rows_differ"] <= 0.02 * stats["rows"] + 2


@pytest.mark.parametrize("name", list(CASES))
@pytest.mark.parametrize("gain", [1.0, 128.0])
def test_forward_matches_oracle(name, gain):
    _forward_parity(CASES[name], gain)


@pytest.mark.parametrize("name", list(EDGE))
def test_forward_edge_cases(name):
    _forward_parity(EDGE[name], 128.0)


def test_forward_per_query_cluster_selection():
    _forward_parity(CASES["gqa_bf16"], 128.0, sel_mode=1)


def test_forward_noncausal():
    _forward_parity(CASES["tiny"], 128.0, causal=False)


@pytest.mark.parametrize("name", list(TC))
@pytest.mark.parametrize("opt", ["default", "per_qcluster", "noncausal"])
def test_forward_options_on_the_tensor_core_path(name, opt):
    """Selection per query cluster and the non-causal (single block) mode on the shapes where the
    tcgen05 kernels run, checked against the oracle like the default options."""
    kern = TC_FWD_KERNELS - ({"k_local_fwd_tc"} if opt == "noncausal" else set())
    _forward_parity(TC[name], 128.0, sel_mode=1 if opt == "per_qcluster" else 0, causal=opt != "noncausal",
                    expect_kernels=kern)


def test_untilted_bucket_statistics():
    """counts, key sums and value sums per (cluster, block) bucket against their definition."""
    for name in ("tiny", "gqa_bf16", "d128"):
        mb, c, p, buf = _prep(CASES[name], 1.0)
        w = c.w
        Q, K, V, _ = c.dev()
        dev = dict(device="cuda")
        counts = torch.empty(w.B, w.Hkv, w.Ck, w.S, dtype=torch.int32, **dev)
        ksum = torch.empty(w.B, w.Hkv, w.Ck, w.S, w.D, dtype=torch.float32, **dev)
        vsum = torch.empty_like(ksum)
        mb.muse_summarize(p, K, V, to_dev(c.a_k, "i"), to_dev(c.qbar32, "f32"), buf.off_k, buf.perm_k, buf.summaries, buf.ws,
                          counts=counts, ksum=ksum, vsum=vsum)
        torch.cuda.synchronize()
        Bs = w.N // w.S
        for b in range(w.B):
            for g in range(w.Hkv):
                key = c.a_k[b, g].astype(np.int64) * w.S + np.arange(w.N) // Bs
                ec = np.bincount(key, minlength=w.Ck * w.S).reshape(w.Ck, w.S)
                ek = np.zeros((w.Ck * w.S, w.D)); ev = np.zeros((w.Ck * w.S, w.D))
                np.add.at(ek, key, c.K[b, g].astype(np.float64)); np.add.at(ev, key, c.V[b, g].astype(np.float64))
                assert np.array_equal(to_np(counts)[b, g], ec)
                assert rel_err(to_np(ksum)[b, g].reshape(-1, w.D), ek) <= 1e-5
                assert rel_err(to_np(vsum)[b, g].reshape(-1, w.D), ev) <= 1e-5


def test_out_of_range_selection_entries_count_as_none():
    """sel_in entries outside [0, Ck) are treated as -1: same output as with -1 in their place, no CUDA error."""
    mb, c, p, buf = _prep(TC["tc"], 128.0)
    w = c.w
    Q, K, V, _ = c.dev()
    _run_summaries(mb, c, p, buf, K, V)
    rng = np.random.default_rng(5)
    sel = rng.integers(0, w.Ck, (w.B, w.Hq, w.N, w.m)).astype(np.int32)
    sel[..., 1:] = -1                                  # one cluster per query, so that entries stay distinct
    bad = sel.copy(); good = sel.copy()
    rows = rng.choice(w.N, 64, replace=False)
    bad[0, 0, rows, 1] = 0x7fffffff; bad[0, 1, rows, 2] = w.Ck; bad[0, 1, rows, 3] = -9
    outs = []
    for s_ in (good, bad):
        mb.muse_attn_fwd(p, Q, K, V, to_dev(c.a_q, "i"), to_dev(c.qbar32, "f32"), buf.off_k, buf.perm_k, buf.summaries,
                         to_dev(s_, "i"), buf.O, buf.LSE, buf.sel, buf.ws)
        torch.cuda.synchronize()
        assert mb.muse_status(buf.ws) == 0
        outs.append((to_np(buf.O).copy(), to_np(buf.sel).copy()))
    assert np.array_equal(outs[0][0], outs[1][0])
    assert outs[1][1].max() < w.Ck and outs[1][1].min() >= -1


@pytest.mark.parametrize("groups", [8, 2])
def test_selection_with_exact_ties_takes_the_lowest_cluster_indices(groups):
    """Key clusters with identical contents have bit-identical summaries and scores, on both sides.  512
    clusters in `groups` classes: the threshold of the top 32 falls inside a class of 64 (compacted selection,
    more ties than places) or 256 (too many candidates to compact: the general path).  Both sides break ties
    towards the lowest cluster index, so the selected sets must be equal for every query."""
    w = CASES["d128"].with_(Hq=1, Hkv=1, N=8192, S=4, Cq=8, Ck=512, m=32)
    mb, c, p, buf = _prep(w, 128.0)
    rng = np.random.default_rng(1234 + groups)
    t = np.arange(w.N)
    bf = lambda x: to_np(torch.from_numpy(x.astype(np.float32)).to(torch.bfloat16)).astype(np.float32)
    proto_k = bf(rng.standard_normal((w.N // w.Ck, groups, w.D)) * 2.0)       # [round][class][D]
    proto_v = bf(rng.standard_normal((w.N // w.Ck, groups, w.D)))
    c.K[0, 0] = proto_k[t // w.Ck, (t % w.Ck) % groups]
    c.V[0, 0] = proto_v[t // w.Ck, (t % w.Ck) % groups]
    c.a_k[0, 0] = (t % w.Ck).astype(np.int32)
    Q, K, V, _ = c.dev()
    _run_summaries(mb, c, p, buf, K, V)
    mb.muse_attn_fwd(p, Q, K, V, to_dev(c.a_q, "i"), to_dev(c.qbar32, "f32"), buf.off_k, buf.perm_k, buf.summaries,
                     None, buf.O, buf.LSE, buf.sel, buf.ws)
    torch.cuda.synchronize()
    sel_gpu = to_np(buf.sel)[0, 0, :, :w.m]
    f = orc.forward(c.Q[0, 0], c.K[0, 0], c.V[0, 0], c.a_q[0, 0], c.a_k[0, 0], c.qbar32[0, 0].astype(np.float64),
                    sigma=c.sigma, S=w.S, Ck=w.Ck, m=w.m)
    rows = np.arange(w.N // w.S, w.N)                    # the first block has no far field
    differ = [r for r in rows if set(sel_gpu[r].tolist()) != set(f["sel"][r].tolist())]
    assert not differ, (len(differ), differ[:5], sorted(sel_gpu[differ[0]].tolist()), sorted(f["sel"][differ[0]].tolist()))
    assert rel_err(to_np(buf.O)[0, 0], f["O"]) <= tol(w.dtype)
