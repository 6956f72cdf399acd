#!/usr/bin/env python
"""Benchmark of the MuSe attention layer (cluster + summarize + forward + backward) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload headline] [--impl muse|reference]

One "step" is one pass of the whole hot path over one batch of seeded synthetic input.
Prints ONE JSON line (rank 0).  With --gpus N > 1 (under torchrun) every rank runs an
independent replica of the workload on its own GPU (the layer has no inter-GPU exchange);
the value is the units all ranks processed divided by the slowest rank's time.
"""
from __future__ import annotations

import argparse
import concurrent.futures
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2509_10406_b200 import workloads as wl  # noqa: E402

METRIC = "muse_attn_fwd_bwd_tokens_per_s"
UNIT = "tokens/s"


# ------------------------------------------------------------------------------------------
# work models: algorithmic FLOPs / bytes per step for each kernel
# ------------------------------------------------------------------------------------------
def work_model(w: wl.Workload):
    B, Hq, Hkv, N, D, Cq, Ck, m, S, T = w.B, w.Hq, w.Hkv, w.N, w.D, w.Cq, w.Ck, w.m, w.S, w.T
    e = 4 if w.dtype == "f32" else 2
    Bs, SB = N // S, S - 1
    heads, kvh = B * Hq, B * Hkv
    nd = N * D
    ret_keys = m * (N / Ck) * (S - 1) / (2 * S)             # nominal retrieved keys per query
    local = 2 * D * N * Bs                                  # 2 matmuls over the causal half
    # Accumulated summaries as the method defines them: (mu, kappa[D], nu[D]) per (head, plane, i, j) in the
    # storage type e' (bf16 / fp32); their gradients have the same shape.  What the kernels move on top of
    # that (a second kappa plane, beta) is implementation traffic: see impl_bytes().
    summ = heads * SB * Cq * Ck * (2 * D + 1) * e
    grads = heads * SB * Cq * Ck * (2 * D + 1) * e
    part = heads * N * m * D * (2 if w.dtype == "bf16" else 4)                       # retrieval partials (o or dq)
    M = {
        # clustering
        "k_assign": ("tensor", 2.0 * N * D * (T + 1) * (Cq * heads + Ck * kvh)),
        "k_assign_tc": ("tensor", 2.0 * N * D * (T + 1) * (Cq * heads + Ck * kvh)),
        "k_update": ("hbm", T * (heads + kvh) * nd * e),
        "k_gather_rows": ("hbm", 2 * kvh * nd * e * 2),
        # summaries: bound by the write of the summaries
        "k_summarize": ("hbm", summ + 2 * kvh * nd * e),
        "k_summarize_tc": ("hbm", summ + 2 * kvh * nd * e),
        # far field: bound by the read of the summaries
        "k_far_fwd": ("hbm", summ + heads * nd * (e + 4)),
        "k_far_fwd_tc": ("hbm", summ + heads * nd * (e + 4)),
        "k_far_bwd": ("hbm", summ + grads + heads * nd * (2 * e + 8)),
        "k_far_bwd_tc": ("hbm", summ + grads + heads * nd * (2 * e + 8)),
        "k_summ_bwd": ("hbm", grads + 2 * kvh * nd * e + 4 * heads * nd * 4),
        "k_summ_bwd_tc": ("hbm", grads + 2 * kvh * nd * e + 4 * heads * nd * 4),
        # exact attention: tensor bound
        "k_local_fwd": ("tensor", heads * float(local)),
        "k_local_fwd_tc": ("tensor", heads * float(local)),
        "k_local_bwd_dkdv": ("tensor", heads * 2.0 * local),      # S, dP, dV, dK
        "k_local_bwd_dkdv_tc": ("tensor", heads * 2.0 * local),
        "k_local_bwd_dq": ("tensor", heads * 1.5 * local),        # S, dP, dQ
        "k_local_bwd_dq_tc": ("tensor", heads * 1.5 * local),
        "k_ret_fwd": ("tensor", heads * 4.0 * D * N * ret_keys),
        "k_ret_fwd_tc": ("tensor", heads * 4.0 * D * N * ret_keys),
        "k_ret_bwd": ("tensor", heads * 10.0 * D * N * ret_keys),
        "k_ret_bwd_dkdv_tc": ("tensor", heads * 8.0 * D * N * ret_keys),
        "k_ret_bwd_dq_tc": ("tensor", heads * 6.0 * D * N * ret_keys),
        "k_ret_fwd_pairs_tc": ("tensor", heads * 4.0 * D * N * ret_keys),
        "k_ret_bwd_pairs_tc": ("tensor", heads * 10.0 * D * N * ret_keys),    # S, dP, dQ, dK, dV from one gather
        # merges and assembly
        "k_merge": ("hbm", heads * nd * (8 + e) + part + heads * N * m * 4),
        "k_final_dq": ("hbm", heads * nd * (4 + e) + part),
        "k_final_dkv": ("hbm", heads * 4 * nd * 4 + kvh * 2 * nd * e),
        # dipole correction (only with --dipole): covariances written once, merged by one GEMM per
        # (head, plane), consumed once per query
        "k_dipole_cov": ("hbm", kvh * SB * Ck * D * D * e + 2 * kvh * nd * e),
        "k_dipole_merge_tc": ("tensor", 2.0 * heads * SB * Cq * Ck * D * D),
        "k_dipole_merge": ("tensor", 2.0 * heads * SB * Cq * Ck * D * D),
        "k_dipole_apply": ("hbm", heads * SB * Cq * D * D * e + heads * nd * (e + 8)),
        # ... next to retrieval, and its backward: matrix-vector products per (query, slot) pair and per query,
        # the two dense contractions over the query and key clusters (all FFMA, counted against the tensor peak
        # of the same contraction), and the covariance backward to the keys
        "k_dipole_sub": ("tensor", 2.0 * heads * N * m * (S - 1) / S * D * D),
        "k_dipole_bwd_pairs": ("tensor", 6.0 * heads * N * m * (S - 1) / S * D * D),
        "k_dipole_sub_tc": ("tensor", 2.0 * heads * N * m * (S - 1) / S * D * D),
        "k_dipole_bwd_pairs_tc": ("tensor", 4.0 * heads * N * m * (S - 1) / S * D * D),
        "k_dipole_bwd_seg": ("tensor", 4.0 * heads * N * (S - 1) / S * D * D),
        "k_dipole_dcov": ("tensor", 2.0 * heads * SB * Cq * Ck * D * D),
        "k_dipole_dpw": ("tensor", 2.0 * heads * SB * Cq * Ck * D * D),
        "k_dipole_dcov_tc": ("tensor", 2.0 * heads * SB * Cq * Ck * D * D),
        "k_dipole_dpw_tc": ("tensor", 2.0 * heads * SB * Cq * Ck * D * D),
        "k_dipole_cov_bwd": ("hbm", heads * SB * Ck * D * D * 4 + 2 * heads * nd * (e + 8)),
        # seeded k-means++ start: every draw reads every vector once
        "k_kmeanspp": ("hbm", float(nd) * e * (heads * (Cq - 1) + kvh * (Ck - 1))),
    }
    return M


def impl_bytes(w: wl.Workload):
    """Bytes the summary-streaming kernels actually move per step in this implementation (stored layout),
    for comparison with the algorithmic bytes of work_model: the difference is overhead, not work."""
    B, Hq, Hkv, N, D, Cq, Ck, S = w.B, w.Hq, w.Hkv, w.N, w.D, w.Cq, w.Ck, w.S
    e = 4 if w.dtype == "f32" else 2
    heads, kvh, nd, ent = B * Hq, B * Hkv, N * D, B * Hq * (S - 1) * Cq * Ck
    st = stored_summary_bytes_per_entry(w)
    gr = (2 * D * 2 + 4) if w.dtype == "bf16" else (2 * D + 1) * 4
    return {"k_summarize_tc": ent * st + 2 * kvh * nd * e, "k_summarize": ent * st + 2 * kvh * nd * e,
            "k_far_fwd_tc": ent * st + heads * nd * (e + 4), "k_far_fwd": ent * st + heads * nd * (e + 4),
            "k_far_bwd_tc": ent * (st + gr) + heads * nd * (2 * e + 8), "k_far_bwd": ent * (st + gr) + heads * nd * (2 * e + 8),
            "k_summ_bwd_tc": ent * gr + 2 * kvh * nd * e + 4 * heads * nd * 4, "k_summ_bwd": ent * gr + 2 * kvh * nd * e + 4 * heads * nd * 4}


def stored_summary_bytes_per_entry(w: wl.Workload) -> int:
    if w.dtype == "f32":
        return (2 * w.D + 2) * 4
    return SUMMARY_KAPPA_PLANES * w.D * 2 + w.D * 2 + 8       # kappa plane(s) + nu, bf16; mu and beta fp32


SUMMARY_KAPPA_PLANES = 2      # bf16 mode stores kappa as a hi + lo pair


NOMINAL = dict(hbm=8000.0, tensor=2250.0)     # "roughly 8 TB/s" and the dense bf16 peak, for context


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm=p["hbm_gbs"], tensor_burst=p["bf16_tflops"], tensor_sustained=p["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm=6650.0, tensor_burst=1590.0, tensor_sustained=1400.0, source="fallback")


# ------------------------------------------------------------------------------------------
class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass
        sm = [float(r[0]) for r in self.rows if r and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) > 1 and r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for k, n in enumerate(names) if any(len(r) > 3 + k and r[3 + k] == "Active" for r in self.rows)]
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm)}


# ------------------------------------------------------------------------------------------
def gen_inputs(w: wl.Workload, gain: float):
    Q = np.empty((w.B, w.Hq, w.N, w.D), np.float32); dO = np.empty_like(Q)
    K = np.empty((w.B, w.Hkv, w.N, w.D), np.float32); V = np.empty_like(K)
    per = w.Hq // w.Hkv

    def one(bh):
        b, h = bh
        q, k, v, do = wl.make_head_inputs(w, b, h, gain=gain)
        Q[b, h], dO[b, h] = q, do
        if h % per == 0:
            K[b, h // per], V[b, h // per] = k, v
    with concurrent.futures.ThreadPoolExecutor(max_workers=min(16, os.cpu_count() or 4)) as ex:
        list(ex.map(one, [(b, h) for b in range(w.B) for h in range(w.Hq)]))
    iq = np.stack([[wl.random_init_indices(w.N, w.Cq, w.seed, (b * w.Hq + h) * 2) for h in range(w.Hq)] for b in range(w.B)])
    ik = np.stack([[wl.random_init_indices(w.N, w.Ck, w.seed, (b * w.Hkv + g) * 2 + 1) for g in range(w.Hkv)] for b in range(w.B)])
    return Q, K, V, dO, iq, ik


def oracle_sample_seconds(w: wl.Workload, gain: float, rows_n: int, gpu=None):
    """Times the fp64 oracle, as it stands, on one (batch 0, head 0) problem: full clustering and
    summaries, forward+backward for `rows_n` sampled queries; scales the per-query part to N
    queries and everything to all heads.  Returns (estimated seconds per step, description, stats).
    `gpu` (optional): the CUDA path's results for that head (assign_q, assign_k, qbar, kcent, sel, O, dQ as
    numpy arrays).  The oracle's per-query part then runs on the GPU's clustering, so that its selections
    and outputs for the sampled queries can be compared with the GPU's (reported statistics, not a gate)."""
    from oracle import muse_oracle as orc
    Q, K, V, dO = (x.astype(np.float64) for x in wl.make_head_inputs(w, 0, 0, gain=gain))
    iq = wl.random_init_indices(w.N, w.Cq, w.seed, 0); ik = wl.random_init_indices(w.N, w.Ck, w.seed, 1)
    sigma = 1.0 / np.sqrt(w.D)
    t0 = time.perf_counter()
    a_q, qbar = orc.lloyd(Q, w.T, init_idx=iq)
    a_k, kcent = orc.lloyd(K, w.T, init_idx=ik)
    t1 = time.perf_counter()
    rows = np.sort(np.random.default_rng(0).choice(w.N, size=min(rows_n, w.N), replace=False))
    stats = None
    if gpu is not None:
        stats = {"free_running_lloyd_assignments_differing": int((gpu["assign_q"] != a_q).sum() + (gpu["assign_k"] != a_k).sum()),
                 "of": int(a_q.size + a_k.size)}
        pts = np.sort(np.random.default_rng(1).choice(w.N, size=min(4096, w.N), replace=False))
        near = bad = 0
        for X, a, c in ((Q, gpu["assign_q"], gpu["qbar"]), (K, gpu["assign_k"], gpu["kcent"])):
            gaps = orc.assignment_gaps(X[pts], c.astype(np.float64))
            near += int((gaps < 1e-4).sum())
            bad += int((orc.assign_nearest(X[pts], c.astype(np.float64)) != a[pts]).sum())
        stats.update(sampled_points=int(2 * pts.size), near_tie_assignments=near, assignments_differing_from_fp64_argmin=bad)
        a_q, a_k, qbar = gpu["assign_q"], gpu["assign_k"], gpu["qbar"].astype(np.float64)
    dQ, dK, dV, f = orc.backward(Q, K, V, dO, a_q, a_k, qbar, sigma=sigma, S=w.S, Ck=w.Ck, m=w.m, rows=rows)
    t2 = time.perf_counter()
    if gpu is not None and w.m > 0:
        same = np.array([set(f["sel"][t].tolist()) == set(gpu["sel"][t].tolist()) for t in rows])
        gap = f["sel_gap"][rows][~same]
        stats.update(sampled_queries=int(rows.size), selection_rows_differing=int((~same).sum()),
                     largest_oracle_margin_where_differing=float(gap.max()) if gap.size else 0.0)
        ok_rows = rows[same]
        if ok_rows.size:
            rel = lambda x, r: float(np.abs(x - r).max() / max(np.abs(r).max(), 1e-30))
            stats.update(O_err_rows_with_equal_selection=rel(gpu["O"][ok_rows], f["O"][ok_rows]),
                         dQ_err_rows_with_equal_selection=rel(gpu["dQ"][ok_rows], dQ[ok_rows]) if gpu.get("dQ") is not None else None)
    # backward() = summaries + per-query forward/backward of the sampled rows + key-side pass;
    # time the row-independent part separately to scale only the per-query part
    t3 = time.perf_counter()
    orc.backward(Q, K, V, dO, a_q, a_k, qbar, sigma=sigma, S=w.S, Ck=w.Ck, m=w.m, rows=rows[:0])
    t4 = time.perf_counter()
    fixed = t4 - t3
    per_row = max(t2 - t1 - fixed, 0.0) / max(len(rows), 1)
    est = ((t1 - t0) * (w.Hq + w.Hkv) / 2.0 + (fixed + per_row * w.N) * w.Hq) * w.B
    desc = (f"batch 0 / head 0 of '{w.name}': Lloyd T={w.T} on Q and K ({t1 - t0:.1f}s), summaries + key-side "
            f"backward ({fixed:.1f}s), forward+backward of {len(rows)} sampled queries ({per_row * 1e3:.1f} ms/query); "
            f"per-query part scaled to N={w.N}, all scaled to {w.B * w.Hq} heads")
    return est, desc, stats


def run_reference(args, w, gain):
    """--impl reference: the oracle on the host cores, a bounded sample per step."""
    import torch
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cores = torch.get_num_threads()
    times = []
    for k in range(args.warmup + args.steps):
        est, desc, _ = oracle_sample_seconds(w, gain, args.ref_rows)
        if k >= args.warmup:
            times.append(est)
    t = statistics.mean(times)
    val = w.B * w.N / t
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(w, gain),
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def workload_config(w, gain):
    return {"workload": f"{w.name}: B={w.B} Hq={w.Hq} Hkv={w.Hkv} N={w.N} D={w.D} {w.dtype} causal S={w.S} "
                        f"Cq={w.Cq} Ck={w.Ck} m={w.m} T={w.T}",
            "inputs": f"{w.components}-component Gaussian mixture per head, RoPE theta={w.rope_theta}, Q gain {gain}",
            "l2": "inputs and intermediates (>1 GB per step) exceed the 126 MB L2; no explicit flush",
            "parallelism": "replicas"}


# DRAM bytes per (batch, head) problem from an ncu capture (--set full) of the headline workload cut
# to one head: dram__bytes_read.sum + dram__bytes_write.sum per launch.  Traffic grows in proportion
# to the problem count.
NCU_TRAFFIC_PER_HEAD = {"k_summarize_tc": 1.430e9, "k_local_fwd_tc": 0.055e9, "k_far_fwd_tc": 1.630e9,
                        "k_ret_bwd_pairs_tc": 1.235e9, "k_ret_fwd_pairs_tc": 0.498e9, "k_far_bwd_tc": 2.415e9,
                        "k_summ_bwd_tc": 1.100e9, "k_local_bwd_dkdv_tc": 0.087e9, "k_local_bwd_dq_tc": 0.074e9,
                        "k_merge": 0.566e9, "k_final_dq": 0.528e9}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="headline", choices=list(wl.WORKLOADS))
    ap.add_argument("--impl", default="muse", choices=["muse", "reference"])
    ap.add_argument("--gain", type=float, default=1.0, help="multiplier on Q (1 = literal workload)")
    ap.add_argument("--m", type=int, default=None, help="override retrieved clusters per query")
    ap.add_argument("--kmeans-iters", type=int, default=None, help="override the number of Lloyd iterations T")
    ap.add_argument("--heads", type=int, default=None, help="override head count (smaller captures)")
    ap.add_argument("--head-groups", type=int, default=0,
                    help="run the KV-head groups in this many sequential stages over one set of buffers "
                         "(0 = as few as keep the summaries under 64 GB)")
    ap.add_argument("--forward-only", action="store_true", help="time cluster + summarize + forward only")
    ap.add_argument("--k2", type=int, default=0,
                    help="spatial blocks retrieved inside each selected cluster (0 = all visible blocks)")
    ap.add_argument("--clustering", default="lloyd", choices=["lloyd", "streaming"],
                    help="lloyd = muse_cluster (the measured path); streaming = the paper's one-pass mini-batch k-means "
                         "with the balanced per-block assignment (muse_cluster_streaming; device-timed line only)")
    ap.add_argument("--dipole", type=int, nargs="?", const=1, default=0, choices=[0, 1, 2],
                    help="far field with the dipole correction: 1 untilted, 2 tilted at the mean query centroid; replaces "
                         "retrieval (m = 0) unless --dipole-with-retrieval is given (device-timed line only)")
    ap.add_argument("--dipole-with-retrieval", action="store_true", help="keep m > 0 next to the dipole correction")
    ap.add_argument("--init", default="indices", choices=["indices", "kmeans++"],
                    help="start points of Lloyd: indices handed in by the harness (the measured path), or the seeded "
                         "k-means++ draws on the GPU (MUSE_INIT_KMEANSPP)")
    ap.add_argument("--ref-rows", type=int, default=128, help="sampled queries for the oracle timing")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-dense", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-sharp", action="store_true", help="skip the extra timing on the sharp variant of the inputs")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "muse" else args.warmup

    w = wl.WORKLOADS[args.workload]
    if args.m is not None:
        w = w.with_(m=args.m)
    if args.dipole:
        if not args.dipole_with_retrieval:
            w = w.with_(m=0)
        args.no_e2e = True
        args.no_cpu_baseline = True
    if args.clustering == "streaming":                    # a device-timed comparison line: no staged run, no oracle sample
        args.no_e2e = True
        args.no_cpu_baseline = True
    if args.kmeans_iters is not None:
        w = w.with_(T=args.kmeans_iters)
    if args.heads is not None:
        w = w.with_(Hq=args.heads, Hkv=max(1, args.heads * w.Hkv // w.Hq))
    if args.impl == "reference":
        return run_reference(args, w, args.gain)

    import torch
    import torch.distributed as dist
    from paper_2509_10406_b200 import binding as mb

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the MuSe path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    mb.lib()   # fail loudly if the CUDA library is missing

    dt = torch.float32 if w.dtype == "f32" else torch.bfloat16
    Qh, Kh, Vh, dOh, iq, ik = gen_inputs(w, args.gain)
    pin = lambda a: torch.from_numpy(a).to(dt).pin_memory()
    hQ, hK, hV, hdO = pin(Qh), pin(Kh), pin(Vh), pin(dOh)
    Q, K, V, dO = (x.cuda(non_blocking=True) for x in (hQ, hK, hV, hdO))
    init_q, init_k = torch.from_numpy(iq).cuda(), torch.from_numpy(ik).cuda()
    # Head staging: every KV-head group is an independent problem, so a layer whose summaries do
    # not fit the device at once runs its groups one after another over one set of buffers.
    groups = args.head_groups
    if groups <= 0:
        full = mb.make_params(B=w.B, Hq=w.Hq, Hkv=w.Hkv, N=w.N, D=w.D, Cq=w.Cq, Ck=w.Ck, m=w.m, n_blocks=w.S,
                              dtype=w.dtype, kmeans_iters=w.T)
        need = mb.muse_workspace_bytes(full)[4]
        groups = 1
        while need / groups > 64e9 and groups < w.Hkv:
            groups *= 2
    if groups > 1 and (w.B != 1 or w.Hkv % groups):
        raise SystemExit("head staging needs B == 1 and a group count that divides the KV heads")
    hq, hkv = w.Hq // groups, w.Hkv // groups
    p = mb.make_params(B=w.B, Hq=hq, Hkv=hkv, N=w.N, D=w.D, Cq=w.Cq, Ck=w.Ck, m=w.m, n_blocks=w.S,
                       dtype=w.dtype, kmeans_iters=w.T, dipole=int(args.dipole), k2=args.k2,
                       init_mode=mb.MUSE_INIT_KMEANSPP if args.init == "kmeans++" else mb.MUSE_INIT_INDICES, seed=w.seed)
    buf = mb.MuseBuffers(p, backward=not args.forward_only)
    stream_ws = (torch.zeros(mb.muse_stream_workspace_bytes(p), dtype=torch.uint8, device="cuda")
                 if args.clustering == "streaming" else None)
    O_all = torch.empty_like(Q)
    dQ_all, dK_all, dV_all = (None, None, None) if args.forward_only else (torch.empty_like(Q), torch.empty_like(K), torch.empty_like(V))

    marks = []                                            # (stage, event) pairs of the timed steps, when asked for

    def step(mark=False):
        def m_(name):
            if mark:
                e = torch.cuda.Event(enable_timing=True); e.record(); marks.append((name, e))
        m_("start")
        for g in range(groups):
            qs, ks = slice(g * hq, (g + 1) * hq), slice(g * hkv, (g + 1) * hkv)
            Qg, Kg, Vg = Q[:, qs], K[:, ks], V[:, ks]
            if args.clustering == "streaming":
                mb.muse_cluster_streaming(p, Qg, Kg, buf.assign_q, buf.assign_k, buf.qbar, buf.kcent, stream_ws, beta=0.9, cap_factor=4.0)
            else:
                kpp = args.init == "kmeans++"
                mb.muse_cluster(p, Qg, Kg, None if kpp else init_q[:, qs], None if kpp else init_k[:, ks], buf.assign_q, buf.assign_k,
                                buf.qbar, buf.kcent, buf.ws)
            m_("cluster")
            if args.dipole == 2:
                mb.muse_dipole_tilt_point(p, buf.assign_q, buf.qbar, buf.summaries)
            mb.muse_summarize(p, Kg, Vg, buf.assign_k, buf.qbar, buf.off_k, buf.perm_k, buf.summaries, buf.ws)
            m_("summarize")
            mb.muse_attn_fwd(p, Qg, Kg, Vg, buf.assign_q, buf.qbar, buf.off_k, buf.perm_k, buf.summaries, None,
                             O_all[:, qs], buf.LSE, buf.sel, buf.ws, bsel_out=buf.bsel)
            m_("forward")
            if not args.forward_only:
                mb.muse_attn_bwd(p, Qg, Kg, Vg, O_all[:, qs], buf.LSE, dO[:, qs], buf.assign_q, buf.qbar, buf.off_k,
                                 buf.perm_k, buf.summaries, buf.sel, dQ_all[:, qs], dK_all[:, ks], dV_all[:, ks], buf.ws, bsel=buf.bsel)
                m_("backward")

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    mb.muse_profile(True)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record()
    for _ in range(args.steps):
        step(mark=True)
    ev1.record()
    barrier()
    ms = ev0.elapsed_time(ev1) / args.steps
    # per public call and per step, from events recorded between the calls of the timed steps
    stages, per_step, t_step = {}, [], 0.0
    for (n0, e0), (n1, e1) in zip(marks, marks[1:]):
        if n1 == "start":
            per_step.append(t_step); t_step = 0.0
            continue
        dt = e0.elapsed_time(e1)
        stages[n1] = stages.get(n1, 0.0) + dt / args.steps
        t_step += dt
    per_step.append(t_step)
    prof = mb.muse_profile_report()
    mb.muse_profile(False)
    clocks = sampler.stop() if rank == 0 else None
    if world > 1:
        t = torch.tensor([ms], device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    tokens = w.B * w.N
    value = world * tokens / (ms * 1e-3)
    O_first = O_all.clone() if (groups == 1 and not args.no_dense) else None
    dev_status = mb.muse_status(buf.ws)           # 0 = no kernel of the last call reported a wait that ran out
    # the CUDA path's results for (batch 0, head 0), for the reported parity statistics
    gpu_head0 = None
    if rank == 0 and groups == 1 and not args.no_cpu_baseline:
        npy = lambda t: t.detach().float().cpu().numpy() if t.dtype in (torch.bfloat16, torch.float32) else t.cpu().numpy()
        gpu_head0 = dict(assign_q=npy(buf.assign_q[0, 0]), assign_k=npy(buf.assign_k[0, 0]), qbar=npy(buf.qbar[0, 0]),
                         kcent=npy(buf.kcent[0, 0]), sel=npy(buf.sel[0, 0])[:, :max(w.m, 0)], O=npy(O_all[0, 0]),
                         dQ=None if args.forward_only else npy(dQ_all[0, 0]))

    # end to end: host buffers in, host buffers out, through the same public calls
    e2e = None
    if not args.no_e2e:
        pinned_like = lambda x: torch.empty(x.shape, dtype=x.dtype, pin_memory=True)
        O_dev = O_all.clone()                         # the device-timed run's output, to check the staged run against
        hO = pinned_like(hQ)
        outs = [(hO, O_all)]
        if not args.forward_only:
            hdQ, hdK, hdV = pinned_like(hQ), pinned_like(hK), pinned_like(hK)
            outs += [(hdQ, dQ_all), (hdK, dK_all), (hdV, dV_all)]

        # The heads are processed in stages through the same public calls, so that the copies of the next stage's
        # inputs and of the previous stage's results overlap the kernels of the current one (two copy streams;
        # PCIe is full duplex).  Every byte still crosses the bus inside the timed region, every step.
        eg = groups
        if w.B == 1:
            while eg < 4 and w.Hkv % (2 * eg) == 0 and w.Hq % (2 * eg) == 0:
                eg *= 2
        ehq, ehkv = w.Hq // eg, w.Hkv // eg
        if eg == groups:
            ep, ebuf = p, buf
        else:
            ep = mb.make_params(B=w.B, Hq=ehq, Hkv=ehkv, N=w.N, D=w.D, Cq=w.Cq, Ck=w.Ck, m=w.m, n_blocks=w.S,
                                dtype=w.dtype, kmeans_iters=w.T, dipole=int(args.dipole), k2=args.k2)
            ebuf = mb.MuseBuffers(ep, backward=not args.forward_only)
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()

        def e2e_step():
            cur = torch.cuda.current_stream()
            s_in.wait_stream(cur)                     # the previous step's kernels have read their inputs
            s_out.wait_stream(cur)
            ev = []
            with torch.cuda.stream(s_in):
                for g in range(eg):
                    qs, ks = slice(g * ehq, (g + 1) * ehq), slice(g * ehkv, (g + 1) * ehkv)
                    Q[:, qs].copy_(hQ[:, qs], non_blocking=True); K[:, ks].copy_(hK[:, ks], non_blocking=True)
                    e_qk = torch.cuda.Event(); e_qk.record(s_in)
                    V[:, ks].copy_(hV[:, ks], non_blocking=True)
                    e_v = torch.cuda.Event(); e_v.record(s_in)
                    dO[:, qs].copy_(hdO[:, qs], non_blocking=True)
                    e_do = torch.cuda.Event(); e_do.record(s_in)
                    ev.append((e_qk, e_v, e_do))
            for g in range(eg):
                qs, ks = slice(g * ehq, (g + 1) * ehq), slice(g * ehkv, (g + 1) * ehkv)
                Qg, Kg, Vg = Q[:, qs], K[:, ks], V[:, ks]
                e_qk, e_v, e_do = ev[g]
                cur.wait_event(e_qk)
                mb.muse_cluster(ep, Qg, Kg, init_q[:, qs], init_k[:, ks], ebuf.assign_q, ebuf.assign_k, ebuf.qbar, ebuf.kcent, ebuf.ws)
                cur.wait_event(e_v)
                mb.muse_summarize(ep, Kg, Vg, ebuf.assign_k, ebuf.qbar, ebuf.off_k, ebuf.perm_k, ebuf.summaries, ebuf.ws)
                mb.muse_attn_fwd(ep, Qg, Kg, Vg, ebuf.assign_q, ebuf.qbar, ebuf.off_k, ebuf.perm_k, ebuf.summaries, None,
                                 O_all[:, qs], ebuf.LSE, ebuf.sel, ebuf.ws, bsel_out=ebuf.bsel)
                e_o = torch.cuda.Event(); e_o.record(cur)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(e_o)
                    hO[:, qs].copy_(O_all[:, qs], non_blocking=True)
                if not args.forward_only:
                    cur.wait_event(e_do)
                    mb.muse_attn_bwd(ep, Qg, Kg, Vg, O_all[:, qs], ebuf.LSE, dO[:, qs], ebuf.assign_q, ebuf.qbar, ebuf.off_k,
                                     ebuf.perm_k, ebuf.summaries, ebuf.sel, dQ_all[:, qs], dK_all[:, ks], dV_all[:, ks], ebuf.ws, bsel=ebuf.bsel)
                    e_g = torch.cuda.Event(); e_g.record(cur)
                    with torch.cuda.stream(s_out):
                        s_out.wait_event(e_g)
                        hdQ[:, qs].copy_(dQ_all[:, qs], non_blocking=True)
                        hdK[:, ks].copy_(dK_all[:, ks], non_blocking=True)
                        hdV[:, ks].copy_(dV_all[:, ks], non_blocking=True)
            cur.wait_stream(s_out)                    # the step ends when its results are in host memory
            cur.wait_stream(s_in)
        e2e_step()
        barrier()
        ev0.record()
        for _ in range(args.steps):
            e2e_step()
        ev1.record()
        barrier()
        ems = ev0.elapsed_time(ev1) / args.steps
        if world > 1:
            t = torch.tensor([ems], device="cuda")
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ems = float(t.item())
        nb = lambda *ts: int(sum(x.numel() * x.element_size() for x in ts))
        e2e = {"value": world * tokens / (ems * 1e-3), "unit": UNIT, "ms_per_step": ems,
               "h2d_bytes_per_step": nb(hQ, hK, hV, hdO), "d2h_bytes_per_step": nb(*[h for h, _ in outs]),
               "head_stages": eg, "copy_streams": 2,
               # (the two runs pass different numbers of heads per call)
               "output_max_abs_diff_vs_device_run_rel": float(((hO.cuda().float() - O_dev.float()).abs().max()
                                                                / O_dev.float().abs().max()).item())}
        del O_dev

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # per-kernel table and the roofline of the dominant kernel
    pk = peaks()
    model = work_model(w)
    total_ms = sum(v[1] for v in prof.values())
    launches = sum(v[0] for v in prof.values() if True)
    kernels = {k: {"launches": v[0] // args.steps, "ms_per_step": v[1] / args.steps, "share": v[1] / total_ms}
               for k, v in sorted(prof.items(), key=lambda kv: -kv[1][1])}
    top = next(iter(kernels))
    roof = {"kernel": top, "bound": None, "achieved": None, "peak": None, "unit": None, "frac": None, "traffic": None}
    if top in model:
        bound, work = model[top]
        sec = kernels[top]["ms_per_step"] * 1e-3
        if bound == "tensor":
            ach, peak, unit = work / sec / 1e12, pk["tensor_sustained"], "TFLOP/s"
        else:
            ach, peak, unit = work / sec / 1e9, pk["hbm"], "GB/s"
        traffic = None
        if w.name == "headline" and w.m == 32 and top in NCU_TRAFFIC_PER_HEAD:
            traffic = NCU_TRAFFIC_PER_HEAD[top] * w.B * w.Hq    # one launch per step covers all heads
        roof.update(bound=bound, achieved=ach, peak=peak, unit=unit, frac=ach / peak, traffic=traffic,
                    peak_source=pk["source"] + (" (sustained bf16)" if bound == "tensor" else " (copy)"),
                    frac_of_nominal=ach / NOMINAL[bound], nominal_peak=NOMINAL[bound],
                    algorithmic_work_per_step=work, kernel_ms_per_step=kernels[top]["ms_per_step"])
    impl = impl_bytes(w)
    for k, v in kernels.items():
        if k in model:
            bound, work = model[k]
            sec = max(v["ms_per_step"], 1e-9) * 1e-3
            v["bound"] = bound
            v["achieved"] = work / sec / (1e12 if bound == "tensor" else 1e9)
            v["frac"] = v["achieved"] / (pk["tensor_sustained"] if bound == "tensor" else pk["hbm"])
            v["frac_of_nominal"] = v["achieved"] / NOMINAL[bound]
            if k in impl:                        # bytes the stored layout makes the kernel move, beside the algorithmic ones
                v["implementation_gbs"] = impl[k] / sec / 1e9
                v["implementation_over_algorithmic_bytes"] = impl[k] / work

    context = {}
    if not args.no_dense:
        try:
            import torch.nn.functional as F
            q = Q.clone().requires_grad_(True)
            k = K.repeat_interleave(w.Hq // w.Hkv, dim=1).clone().requires_grad_(True)
            v = V.repeat_interleave(w.Hq // w.Hkv, dim=1).clone().requires_grad_(True)

            def dense():
                o = F.scaled_dot_product_attention(q, k, v, is_causal=True)
                if not args.forward_only:
                    o.backward(dO)
                    q.grad = k.grad = v.grad = None
                return o
            dense(); torch.cuda.synchronize()
            ev0.record()
            for _ in range(3):
                o_dense = dense()
            ev1.record(); torch.cuda.synchronize()
            dms = ev0.elapsed_time(ev1) / 3
            context["dense_sdpa_forward_only_ms" if args.forward_only else "dense_sdpa_fwd_bwd_ms"] = dms
            context["speedup_vs_dense_sdpa"] = dms / ms
            if groups == 1 and O_first is not None:
                # relative squared error of the approximation against exact attention, averaged over queries
                # (Appendix "Hyperparameters", "Evaluation metrics"); context only: synthetic mixtures have none of
                # the structure of trained-model attention
                od = o_dense.detach().float()
                num = (O_first.float() - od).pow(2).sum(-1); den = od.pow(2).sum(-1).clamp_min(1e-30)
                context["rse_vs_dense_mean_over_queries"] = float((num / den).mean().item())
            del q, k, v, o_dense
        except Exception as ex:  # bench-only comparator; never fatal
            context["dense_sdpa_error"] = repr(ex)[:200]
        try:
            # exact causal attention through this library's own kernels: one spatial block, nothing retrieved,
            # no far field (the block-diagonal kernels then cover the whole sequence)
            pd = mb.make_params(B=w.B, Hq=w.Hq, Hkv=w.Hkv, N=w.N, D=w.D, Cq=1, Ck=1, m=0, n_blocks=1, dtype=w.dtype,
                                kmeans_iters=0, init_mode=mb.MUSE_INIT_STRIDED)
            bd = mb.MuseBuffers(pd, backward=True)
            mb.muse_cluster(pd, Q, K, None, None, bd.assign_q, bd.assign_k, bd.qbar, bd.kcent, bd.ws)
            mb.muse_summarize(pd, K, V, bd.assign_k, bd.qbar, bd.off_k, bd.perm_k, bd.summaries, bd.ws)

            def own():
                mb.muse_attn_fwd(pd, Q, K, V, bd.assign_q, bd.qbar, bd.off_k, bd.perm_k, bd.summaries, None, bd.O, bd.LSE, bd.sel, bd.ws)
                mb.muse_attn_bwd(pd, Q, K, V, bd.O, bd.LSE, dO, bd.assign_q, bd.qbar, bd.off_k, bd.perm_k, bd.summaries, bd.sel,
                                 bd.dQ, bd.dK, bd.dV, bd.ws)
            own(); torch.cuda.synchronize()
            ev0.record()
            for _ in range(3):
                own()
            ev1.record(); torch.cuda.synchronize()
            context["dense_own_kernels_fwd_bwd_ms"] = ev0.elapsed_time(ev1) / 3
            del bd
        except Exception as ex:
            context["dense_own_kernels_error"] = repr(ex)[:200]
    if args.clustering == "streaming":
        # quality beside the time: the k-means objective (mean squared distance to the assigned centroid, head 0 of the
        # last head group) under the streaming pass + balanced assignment and under Lloyd, and how many vectors the cap
        # moved away from their nearest centroid.  Bench-only arithmetic (torch), outside every timed region.
        def objective(X, a, c):
            return float(((X.float() - c[a.long()]) ** 2).sum(-1).mean().item())
        g0 = groups - 1
        Qg, Kg = Q[:, g0 * hq:(g0 + 1) * hq], K[:, g0 * hkv:(g0 + 1) * hkv]
        qual = {"streaming_objective_q": objective(Qg[0, 0], buf.assign_q[0, 0], buf.qbar[0, 0]),
                "streaming_objective_k": objective(Kg[0, 0], buf.assign_k[0, 0], buf.kcent[0, 0])}
        near = torch.empty_like(buf.assign_k)
        mb.muse_balanced_assign(p, Kg, 1, buf.kcent, near, stream_ws, cap_factor=0.0)
        qual["keys_moved_by_the_cap_fraction"] = float((near != buf.assign_k).float().mean().item())
        nearq = torch.empty_like(buf.assign_q)
        mb.muse_balanced_assign(p, Qg, 0, buf.qbar, nearq, stream_ws, cap_factor=0.0)
        qual["queries_moved_by_the_cap_fraction"] = float((nearq != buf.assign_q).float().mean().item())
        mb.muse_cluster(p, Qg, Kg, init_q[:, g0 * hq:(g0 + 1) * hq], init_k[:, g0 * hkv:(g0 + 1) * hkv], buf.assign_q, buf.assign_k,
                        buf.qbar, buf.kcent, buf.ws)
        qual["lloyd_objective_q"] = objective(Qg[0, 0], buf.assign_q[0, 0], buf.qbar[0, 0])
        qual["lloyd_objective_k"] = objective(Kg[0, 0], buf.assign_k[0, 0], buf.kcent[0, 0])
        context["clustering_quality_head0"] = qual
    if not args.no_sharp and args.gain == 1.0:
        # the same step on the sharp variant of the inputs (Q x 128, exact in bf16): attention is then peaked,
        # so selection and retrieval matter; k-means and the tile schedule are scale-free
        Q.mul_(128.0)
        for _ in range(2):
            step()
        torch.cuda.synchronize()
        ev0.record()
        for _ in range(3):
            step()
        ev1.record(); torch.cuda.synchronize()
        context["sharp_inputs_ms_per_step"] = ev0.elapsed_time(ev1) / 3
        context["sharp_inputs_device_status"] = mb.muse_status(buf.ws)
        Q.mul_(1.0 / 128.0)
    if not args.no_sharp and args.clustering == "lloyd" and args.k2 == 0 and not args.dipole and w.dtype == "bf16" and groups == 1:
        # the path's options on the same inputs, device-timed, as context beside the headline numbers: the paper's own
        # clustering in place of Lloyd and Lloyd from the k-means++ start drawn on the GPU (cluster stage only), the two-level
        # retrieval with k2 = 1 and the dipole correction with m = 0 (summarize + forward)
        try:
            sws = torch.zeros(mb.muse_stream_workspace_bytes(p), dtype=torch.uint8, device="cuda")
            for it in range(3):
                if it == 1:
                    ev0.record()
                mb.muse_cluster_streaming(p, Q, K, buf.assign_q, buf.assign_k, buf.qbar, buf.kcent, sws, beta=0.9, cap_factor=4.0)
            ev1.record(); torch.cuda.synchronize()
            context["streaming_clustering_stage_ms"] = ev0.elapsed_time(ev1) / 2
            context["streaming_clustering_device_status"] = mb.muse_status(sws)
            del sws
            pk = mb.make_params(B=w.B, Hq=hq, Hkv=hkv, N=w.N, D=w.D, Cq=w.Cq, Ck=w.Ck, m=w.m, n_blocks=w.S, dtype=w.dtype,
                                kmeans_iters=w.T, init_mode=mb.MUSE_INIT_KMEANSPP, seed=w.seed)
            for it in range(3):
                if it == 1:
                    ev0.record()
                mb.muse_cluster(pk, Q, K, None, None, buf.assign_q, buf.assign_k, buf.qbar, buf.kcent, buf.ws)
            ev1.record(); torch.cuda.synchronize()
            context["kmeanspp_start_clustering_stage_ms"] = ev0.elapsed_time(ev1) / 2
            context["kmeanspp_start_device_status"] = mb.muse_status(buf.ws)
            mb.muse_cluster(p, Q, K, init_q, init_k, buf.assign_q, buf.assign_k, buf.qbar, buf.kcent, buf.ws)
            p2 = mb.make_params(B=w.B, Hq=hq, Hkv=hkv, N=w.N, D=w.D, Cq=w.Cq, Ck=w.Ck, m=w.m, n_blocks=w.S, dtype=w.dtype,
                                kmeans_iters=w.T, k2=1)
            need2 = mb.muse_workspace_bytes(p2)
            if need2[4] < 60e9:
                aq, ak, qb = buf.assign_q.clone(), buf.assign_k.clone(), buf.qbar.clone()
                del buf
                torch.cuda.empty_cache()
                b2 = mb.MuseBuffers(p2, backward=False)
                for it in range(3):
                    if it == 1:
                        ev0.record()
                    mb.muse_summarize(p2, K, V, ak, qb, b2.off_k, b2.perm_k, b2.summaries, b2.ws)
                    mb.muse_attn_fwd(p2, Q, K, V, aq, qb, b2.off_k, b2.perm_k, b2.summaries, None, O_all, b2.LSE, b2.sel, b2.ws,
                                     bsel_out=b2.bsel)
                ev1.record(); torch.cuda.synchronize()
                context["two_level_k2_1_summarize_plus_forward_ms"] = ev0.elapsed_time(ev1) / 2
                context["k2_all_summarize_plus_forward_ms"] = stages.get("summarize", 0.0) + stages.get("forward", 0.0)
                context["two_level_device_status"] = mb.muse_status(b2.ws)
                del b2
                torch.cuda.empty_cache()
                # the dipole correction as the paper defines it (no retrieval): summarize + forward
                p3 = mb.make_params(B=w.B, Hq=hq, Hkv=hkv, N=w.N, D=w.D, Cq=w.Cq, Ck=w.Ck, m=0, n_blocks=w.S, dtype=w.dtype,
                                    kmeans_iters=w.T, dipole=1)
                b3 = mb.MuseBuffers(p3, backward=False)
                for it in range(3):
                    if it == 1:
                        ev0.record()
                    mb.muse_summarize(p3, K, V, ak, qb, b3.off_k, b3.perm_k, b3.summaries, b3.ws)
                    mb.muse_attn_fwd(p3, Q, K, V, aq, qb, b3.off_k, b3.perm_k, b3.summaries, None, O_all, b3.LSE, b3.sel, b3.ws)
                ev1.record(); torch.cuda.synchronize()
                context["dipole_m0_summarize_plus_forward_ms"] = ev0.elapsed_time(ev1) / 2
                context["dipole_device_status"] = mb.muse_status(b3.ws)
                del b3
        except Exception as ex:
            context["options_error"] = repr(ex)[:200]
    context["paper"] = ("2x over cuDNN flash attention at 64k and +36% pretraining throughput, 8xA100, "
                        "D=64, QK128R8SP1B8k (other hardware and configuration: context only)")

    cpu = None
    parity_stats = None
    if not args.no_cpu_baseline:
        est, desc, parity_stats = oracle_sample_seconds(w, args.gain, args.ref_rows, gpu=gpu_head0)
        cpu = {"value": tokens / est, "unit": UNIT, "cores": torch.get_num_threads(), "kind": "oracle",
               "sample": desc, "est_seconds_per_step": est}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": w.dtype,
            "data": "synthetic",
            "config": dict(workload_config(w, args.gain), head_stages=groups,
                           dipole=int(args.dipole), k2=args.k2,
                           clustering="lloyd" if args.clustering == "lloyd" else "streaming mini-batch k-means (batch 64, beta 0.9) + balanced assignment (cap 4 B/K)",
                           passes="cluster+summarize+forward" if args.forward_only else "cluster+summarize+forward+backward"),
            "ms_per_step_median": statistics.median(per_step), "ms_per_step_best": min(per_step), "stages_ms": stages,
            "clocks": clocks, "e2e": e2e,
            "gpu_launches": launches, "roofline": roof, "cpu_baseline": cpu, "kernels": kernels, "context": context,
            "device_status": dev_status, "parity_stats_head0": parity_stats}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
