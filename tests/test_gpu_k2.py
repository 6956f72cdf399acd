"""GPU parity of the two-level retrieval (Section "Two-Level Retrieval": inside every selected cluster only the
k2 best-scoring earlier blocks are retrieved exactly, the others enter through their per-block summaries; Section
"Output merging": the four-way merge) against the fp64 oracle, forward pass, bf16 mode (2e-2 relative max-abs),
with cluster and block selections forced both ways."""
import numpy as np
import pytest
import torch

from oracle import muse_oracle as orc
from tests.gpu_util import Case, to_dev, to_np, tol, rel_err, kernels_launched
from tests.test_gpu_cluster import CASES
from tests.test_gpu_forward import TC

pytestmark = pytest.mark.gpu

K2_CASES = {"d128": CASES["d128"], "tc": TC["tc"], "tc_d64": TC["tc_d64"]}


def _run(mb, c, p, buf, Q, K, V, qbar32, sel_in=None, bsel_in=None):
    mb.muse_attn_fwd(p, Q, K, V, to_dev(c.a_q, "i"), to_dev(qbar32, "f32"), buf.off_k, buf.perm_k, buf.summaries,
                     None if sel_in is None else to_dev(sel_in, "i"), buf.O, buf.LSE, buf.sel, buf.ws,
                     bsel_in=None if bsel_in is None else to_dev(bsel_in, "i"), bsel_out=buf.bsel)
    torch.cuda.synchronize()
    assert mb.muse_status(buf.ws) == 0
    return to_np(buf.O), to_np(buf.LSE), to_np(buf.sel)[..., :c.w.m], to_np(buf.bsel)


@pytest.mark.parametrize("name,force", [(n, 0) for n in K2_CASES] + [("tc", 64)])
@pytest.mark.parametrize("k2", [1, 2])
def test_two_level_forward_matches_oracle(name, k2, force):
    """force = 64: the block selection kernel with a warp per query (the one for more than 8 earlier blocks) at a shape where
    the lane-per-query kernel is the default."""
    from paper_2509_10406_b200 import binding as mb
    mb.muse_test_force_paths(force)
    try:
        _two_level_forward(mb, name, k2, force)
    finally:
        mb.muse_test_force_paths(0)


def _two_level_forward(mb, name, k2, force):
    w = K2_CASES[name]
    c = Case(w, gain=128.0)
    qbar32 = c.qbar.astype(np.float32)
    p = c.params(k2=k2)
    buf = mb.MuseBuffers(p, backward=False)
    Q, K, V, _ = c.dev()
    with kernels_launched() as rec:
        mb.muse_summarize(p, K, V, to_dev(c.a_k, "i"), to_dev(qbar32, "f32"), buf.off_k, buf.perm_k, buf.summaries, buf.ws)
        O_free, L_free, sel_gpu, bsel_gpu = _run(mb, c, p, buf, Q, K, V, qbar32)
    assert {"k_block_select" if force == 64 else "k_block_select_q", "k_ret_fwd_pairs_tc"} <= rec.names, sorted(rec.names)
    t = tol(w.dtype)
    kw = dict(sigma=c.sigma, S=w.S, Ck=w.Ck, m=w.m, k2=k2)
    sel_orc = np.full((w.B, w.Hq, w.N, w.m), -1, np.int32)
    bsel_orc = np.full((w.B, w.Hq, w.N, w.m, k2), -1, np.int32)
    worst = dict(forced_gpu=0.0, forced_orc=0.0, block_rows_differ=0, pairs=0)
    for b in range(w.B):
        for h in range(w.Hq):
            g = c.hm[h]
            args = (c.Q[b, h], c.K[b, g], c.V[b, g], c.a_q[b, h], c.a_k[b, g], qbar32[b, h].astype(np.float64))
            f = orc.forward(*args, **kw)
            sel_orc[b, h], bsel_orc[b, h] = f["sel"], f["bsel"]
            # the oracle forced to the GPU's cluster AND block selections
            ff = orc.forward(*args, sel=sel_gpu[b, h], bsel=bsel_gpu[b, h], summ=f["summ"], **kw)
            e = max(rel_err(O_free[b, h], ff["O"]), float(np.abs(L_free[b, h] - ff["LSE"]).max() / max(1.0, np.abs(ff["LSE"]).max())))
            worst["forced_gpu"] = max(worst["forced_gpu"], e)
            # the GPU's blocks are valid: earlier than the query's block, distinct, inside non-empty buckets of the cluster
            Bs = w.N // w.S
            cnt = np.zeros((w.Ck, w.S), np.int64)
            np.add.at(cnt, (c.a_k[b, g], np.arange(w.N) // Bs), 1)
            for tq in range(0, w.N, 37):
                for k in range(w.m):
                    j = sel_gpu[b, h, tq, k]
                    bl = bsel_gpu[b, h, tq, k]; bl = bl[bl >= 0]
                    assert j >= 0 or bl.size == 0
                    assert len(set(bl.tolist())) == bl.size and np.all(bl < tq // Bs)
                    if j >= 0:
                        assert np.all(cnt[j, bl] > 0)
                        assert bl.size == min(k2, int((cnt[j, :tq // Bs] > 0).sum()))
            # free selections compared where the cluster selections agree slot for slot after sorting by cluster
            for tq in range(0, w.N, 11):
                so, sg = f["sel"][tq], sel_gpu[b, h, tq]
                if set(so.tolist()) != set(sg.tolist()):
                    continue
                for k in range(w.m):
                    if so[k] < 0:
                        continue
                    kg = int(np.nonzero(sg == so[k])[0][0])
                    worst["pairs"] += 1
                    worst["block_rows_differ"] += int(set(f["bsel"][tq, k].tolist()) != set(bsel_gpu[b, h, tq, kg].tolist()))
    assert worst["forced_gpu"] <= t, worst
    # the GPU forced to the oracle's cluster and block selections
    O_f, _, _, _ = _run(mb, c, p, buf, Q, K, V, qbar32, sel_in=sel_orc, bsel_in=bsel_orc)
    for b in range(w.B):
        for h in range(w.Hq):
            g = c.hm[h]
            f = orc.forward(c.Q[b, h], c.K[b, g], c.V[b, g], c.a_q[b, h], c.a_k[b, g], qbar32[b, h].astype(np.float64),
                            sel=sel_orc[b, h], bsel=bsel_orc[b, h], **kw)
            worst["forced_orc"] = max(worst["forced_orc"], rel_err(O_f[b, h], f["O"]))
    print(name, k2, worst)
    assert worst["forced_orc"] <= t, worst
    # block choices may differ from the oracle's only at near-ties of the block logits: a small fraction
    assert worst["block_rows_differ"] <= 0.02 * worst["pairs"] + 2, worst


def test_retrieving_every_block_equals_single_level():
    """k2 >= S - 1 retrieves every earlier block of the selected clusters: the near field is empty and the result is
    that of k2 = 0 (up to the order of the floating-point sums)."""
    from paper_2509_10406_b200 import binding as mb
    w = TC["tc"]
    c = Case(w, gain=128.0)
    qbar32 = c.qbar.astype(np.float32)
    Q, K, V, _ = c.dev()
    outs = []
    for k2 in (0, w.S - 1):
        p = c.params(k2=k2)
        buf = mb.MuseBuffers(p, backward=False)
        mb.muse_summarize(p, K, V, to_dev(c.a_k, "i"), to_dev(qbar32, "f32"), buf.off_k, buf.perm_k, buf.summaries, buf.ws)
        mb.muse_attn_fwd(p, Q, K, V, to_dev(c.a_q, "i"), to_dev(qbar32, "f32"), buf.off_k, buf.perm_k, buf.summaries, None,
                         buf.O, buf.LSE, buf.sel, buf.ws, bsel_out=buf.bsel)
        torch.cuda.synchronize()
        assert mb.muse_status(buf.ws) == 0
        outs.append((to_np(buf.O), to_np(buf.LSE)))
    assert rel_err(outs[1][0], outs[0][0]) <= 1e-2
    assert np.abs(outs[1][1] - outs[0][1]).max() <= 1e-3 * max(1.0, np.abs(outs[0][1]).max())


@pytest.mark.parametrize("name,k2,agg,force", [("d128", 1, True, 0), ("d128", 2, True, 0), ("tc_d64", 1, True, 0), ("tc", 1, False, 0),
                                               ("tc_gqa4", 2, True, 0), ("tc", 1, True, 4), ("tc_d64", 2, False, 4)])
def test_two_level_backward_matches_oracle(name, k2, agg, force):
    """Backward with k2 > 0: the chosen clusters and blocks of the forward pass are constants; dQ, dK, dV against the oracle's
    backward evaluated on the same selections (bf16 mode, 2e-2 relative max-abs)."""
    from paper_2509_10406_b200 import binding as mb
    w = TC[name] if name in TC else K2_CASES[name]
    c = Case(w, gain=128.0)
    qbar32 = c.qbar.astype(np.float32)
    p = c.params(k2=k2, agg_grad=agg)
    buf = mb.MuseBuffers(p, backward=True)
    Q, K, V, dO = c.dev()
    aq, qb = to_dev(c.a_q, "i"), to_dev(qbar32, "f32")
    mb.muse_test_force_paths(force)        # 4: the key-side passes (accumulated and per-block) on the FFMA kernel
    try:
        with kernels_launched() as rec:
            mb.muse_summarize(p, K, V, to_dev(c.a_k, "i"), qb, buf.off_k, buf.perm_k, buf.summaries, buf.ws)
            mb.muse_attn_fwd(p, Q, K, V, aq, qb, buf.off_k, buf.perm_k, buf.summaries, None, buf.O, buf.LSE, buf.sel, buf.ws, bsel_out=buf.bsel)
            torch.cuda.synchronize()
            assert mb.muse_status(buf.ws) == 0
            mb.muse_attn_bwd(p, Q, K, V, buf.O, buf.LSE, dO, aq, qb, buf.off_k, buf.perm_k, buf.summaries, buf.sel, buf.dQ, buf.dK, buf.dV,
                             buf.ws, bsel=buf.bsel)
            torch.cuda.synchronize()
    finally:
        mb.muse_test_force_paths(0)
    assert mb.muse_status(buf.ws) == 0
    assert {"k_near_bwd", "k_ret_bwd_pairs_tc"} <= rec.names, sorted(rec.names)
    assert ("k_summ_bwd" in rec.names) == (force == 4) and ("k_grad_to_bf16" in rec.names) == (force == 0), sorted(rec.names)
    sel, bsel = to_np(buf.sel)[..., :w.m], to_np(buf.bsel)
    assert (bsel >= 0).any()
    ref = orc.layer_backward(c.Q.astype(np.float64), c.K.astype(np.float64), c.V.astype(np.float64), c.dO.astype(np.float64),
                             c.a_q, c.a_k, qbar32.astype(np.float64), sigma=c.sigma, S=w.S, Ck=w.Ck, m=w.m, causal=True,
                             sel=sel, sel_mode=0, agg_grad=agg, k2=k2, bsel=bsel)
    errs = dict(dQ=rel_err(to_np(buf.dQ), ref[0]), dK=rel_err(to_np(buf.dK), ref[1]), dV=rel_err(to_np(buf.dV), ref[2]))
    print(f"[{name} k2={k2} agg={agg} force={force}] backward errors {errs}")
    assert all(v <= tol(w.dtype) for v in errs.values()), errs
    # the near-field term is not negligible in this case: dropping it (the single-level formulas on the same selections)
    # would not pass
    ref0 = orc.layer_backward(c.Q.astype(np.float64), c.K.astype(np.float64), c.V.astype(np.float64), c.dO.astype(np.float64),
                              c.a_q, c.a_k, qbar32.astype(np.float64), sigma=c.sigma, S=w.S, Ck=w.Ck, m=w.m, causal=True,
                              sel=sel, sel_mode=0, agg_grad=agg)
    print("   distance of the single-level gradients:", {k: rel_err(ref0[i], ref[i]) for i, k in enumerate(("dQ", "dK", "dV"))})


def test_two_level_backward_rebuilds_both_summary_sets_when_not_given():
    """summaries = NULL with k2 > 0: the backward pass rebuilds the accumulated AND the per-block summaries in its scratch
    and returns the same gradients as with the caller's copy (dQ bit for bit; dK, dV end in float atomics)."""
    from paper_2509_10406_b200 import binding as mb
    w = TC["tc"]
    c = Case(w, gain=128.0)
    qbar32 = c.qbar.astype(np.float32)
    p = c.params(k2=1)
    buf = mb.MuseBuffers(p, backward=True)
    Q, K, V, dO = c.dev()
    aq, qb = to_dev(c.a_q, "i"), to_dev(qbar32, "f32")
    mb.muse_summarize(p, K, V, to_dev(c.a_k, "i"), qb, buf.off_k, buf.perm_k, buf.summaries, buf.ws)
    mb.muse_attn_fwd(p, Q, K, V, aq, qb, buf.off_k, buf.perm_k, buf.summaries, None, buf.O, buf.LSE, buf.sel, buf.ws, bsel_out=buf.bsel)
    outs = []
    for summ, ws in ((buf.summaries, buf.ws), (None, torch.empty(buf.sizes[5], dtype=torch.uint8, device="cuda"))):
        mb.muse_attn_bwd(p, Q, K, V, buf.O, buf.LSE, dO, aq, qb, buf.off_k, buf.perm_k, summ, buf.sel, buf.dQ, buf.dK, buf.dV, ws, bsel=buf.bsel)
        torch.cuda.synchronize()
        assert mb.muse_status(ws) == 0
        outs.append((to_np(buf.dQ), to_np(buf.dK), to_np(buf.dV)))
    assert np.array_equal(outs[0][0], outs[1][0])
    assert rel_err(outs[1][1], outs[0][1]) <= 1e-2 and rel_err(outs[1][2], outs[0][2]) <= 1e-2
