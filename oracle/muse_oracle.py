"""fp64 CPU oracle for the MuSe (Multipole Semantic Attention) layer.

TEST INFRASTRUCTURE ONLY.  This file is the independent, slow, plain statement
of what the layer computes, written from the paper.  Only the tests, the smoke
check and the benchmark's CPU-baseline leg may import it; the CUDA product path
never does, and the two share no code.  Everything is numpy float64; a library
matmul / argsort is used as a step, nothing is blocked, fused or reordered.

One (batch, query head) at a time.  Notation follows the paper: queries q,
keys k, values v, query centroids qbar_i, key clusters j, spatial blocks b of
size B_s = N / S, per-block summaries (mu, kappa, nu)_{ijb} = (log mass,
tilted key centroid, tilted value centroid), accumulated (exclusive over
blocks) summaries (muh, kah, nuh)_{ijb}, k_1 = m retrieved clusters.

Readings taken where the paper is silent (listed again in the design notes):
 * the softmax scale sigma multiplies every logit: exp(sigma q.k); the paper
   writes exp(q.k).  qbar is in the units of q, so tilt logits are
   sigma qbar_i . k and the residual is qres = sigma (q - qbar_i).
 * clustering: T Lloyd iterations (assign, update) from given start points,
   then a final assignment against the last centres; qbar := those centres.
   Empty clusters keep their centre; ties go to the lowest index.
 * spatial selection k_2 = all causally visible blocks on the hot path, so the merge has three
   non-empty components (far approximation, retrieved exact, local exact).  forward(k2 > 0)
   also states the two-level retrieval (block selection with per-block summaries and the
   fourth, near-field component); block ties go to the lower block index.  backward(k2 > 0)
   holds the chosen blocks constant like the chosen clusters.
 * top-m: among clusters with at least one visible key, largest score first,
   ties to the lower cluster index; fewer than m candidates -> take them all.

Pins (tests/test_oracle_*.py): Lloyd vs scikit-learn / scipy on the same start
centres; the Algorithm-1 recurrence vs the direct definition of accumulated
summaries; m = C_k, singleton key clusters or singleton query clusters give
dense causal softmax attention (textbook formula written separately in the
test); key-translation invariance; weights sum to one and are causal;
error bilinear in the residuals; backward vs central finite differences and,
for m = C_k, vs the closed-form dense-attention gradient.  Two-level retrieval: k2 >= S - 1
reproduces k2 = all; a separately written single softmax over exact and stand-in keys on tiny
inputs; singleton key or query clusters stay exact for every k2; weights causal, sum to one; its
backward vs central finite differences with clusters and blocks held fixed, and k2 >= S - 1 vs the
single-level backward.  Dipole: the Jacobian
of the far field at zero residual equals the dense-attention Jacobian (a
cross-covariance written separately in the test), the error falls from first
to second order in the residual, causality and key-translation invariance; a covariance tilted at a
point is the derivative of the tilted value mean at that point (central differences); with retrieval
(m > 0) the Jacobian at zero residual is still the dense one and the correction is the merge over the
clusters that were not retrieved; its backward vs central finite differences.  k-means++ seeding: draw
frequencies against D^2 / sum D^2, distinct indices, one start per separated blob.  Streaming k-means: closed-form
exponentially weighted means for one cluster and for separated blobs, a hand-computed case that tells
minibatch assignment from immediate updates, continuation from a saved state; balanced assignment: equals
the nearest centroid when the cap does not bind, hand-computed overflow cases, size and placement invariants.
"""
from __future__ import annotations

import numpy as np

__all__ = [
    "lloyd", "assign_nearest", "assignment_gaps", "strided_init", "feistel_permute",
    "block_summaries", "accumulate", "accumulated_summaries",
    "select_clusters", "forward", "backward", "layer_forward", "layer_backward",
    "untilted_covariances", "tilted_covariances", "mean_query_centroid", "merged_dipole", "dipole_weights",
    "kmeanspp_init", "kmeanspp_step",
    "stream_order", "streaming_kmeans", "balanced_cap", "balanced_assign",
]

_M64 = (1 << 64) - 1


# --------------------------------------------------------------------------------------------
# Clustering (Section "Clustering"; Appendix "Clustering Details")
# --------------------------------------------------------------------------------------------

def assign_nearest(X, centres):
    """argmin_c (|c|^2 - 2 x.c): the |x|^2 term cancels between centres
    (Appendix "Balanced Assignment", distance identity).  Ties -> lowest c."""
    X = np.asarray(X, np.float64)
    centres = np.asarray(centres, np.float64)
    d = (centres * centres).sum(1)[None, :] - 2.0 * (X @ centres.T)
    return np.argmin(d, axis=1).astype(np.int32)


def assignment_gaps(X, centres):
    """Relative gap (d2 - d1) / max(d2, 1e-30) between the two smallest true squared
    distances of every point; a point whose gap is below 1e-4 is a near-tie."""
    X = np.asarray(X, np.float64)
    centres = np.asarray(centres, np.float64)
    d = ((X * X).sum(1)[:, None] + (centres * centres).sum(1)[None, :] - 2.0 * (X @ centres.T))
    d = np.maximum(d, 0.0)
    if d.shape[1] == 1:
        return np.ones(d.shape[0])
    part = np.partition(d, 1, axis=1)
    d1, d2 = part[:, 0], part[:, 1]
    return (d2 - d1) / np.maximum(d2, 1e-30)


def update_centres(X, a, centres):
    """Mean of the members of each cluster; an empty cluster keeps its centre."""
    X = np.asarray(X, np.float64)
    new = np.array(centres, np.float64, copy=True)
    for c in range(new.shape[0]):
        mem = np.nonzero(a == c)[0]
        if mem.size:
            new[c] = X[mem].sum(0) / mem.size
    return new


def lloyd(X, T, init_idx=None, init_centres=None):
    """T x (assign, update) then a final assignment.  Returns (assign, centres)."""
    X = np.asarray(X, np.float64)
    centres = (np.array(init_centres, np.float64, copy=True) if init_centres is not None
               else X[np.asarray(init_idx, np.int64)].copy())
    for _ in range(T):
        a = assign_nearest(X, centres)
        centres = update_centres(X, a, centres)
    return assign_nearest(X, centres), centres


def _splitmix64(x: int) -> int:
    z = (x + 0x9E3779B97F4A7C15) & _M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
    return z ^ (z >> 31)


def feistel_permute(x: int, N: int, seed: int, stream: int) -> int:
    """A seeded bijection of [0, N): 4-round balanced Feistel network over the smallest
    even-width power of two >= N, cycle-walked back into range.  Integer-only, so two
    independent implementations agree bit for bit."""
    bits = max(2, (N - 1).bit_length())
    bits += bits & 1
    half = bits // 2
    mask = (1 << half) - 1
    while True:
        L, R = x >> half, x & mask
        for r in range(4):
            f = _splitmix64((seed ^ (stream << 32) ^ (r << 56) ^ R) & _M64) & mask
            L, R = R, L ^ f
        x = (L << half) | R
        if x < N:
            return x


def strided_init(N: int, C: int, seed: int, stream: int) -> np.ndarray:
    """Start indices by the paper's rule (Appendix "Centroid Computation", step 1): shuffle
    with a fixed seed, then take every floor(N/C)-th vector.  The shuffle is the seeded
    bijection above: index r -> position pi(r * floor(N/C))."""
    stride = N // C
    return np.array([feistel_permute(r * stride, N, seed, stream) for r in range(C)], np.int32)


def _kpp_uniforms(N: int, c: int, seed: int, stream: int) -> np.ndarray:
    """The N uniforms in (0, 1) of draw number c: integer hash of (seed, stream, c, t) -> 23 bits,
    centred in their cell, so that every value is exact in single and double precision alike."""
    key = _splitmix64((seed ^ (stream << 32) ^ (0xA5 << 56) ^ c) & _M64)
    return np.array([((_splitmix64(key ^ t) >> 41) + 0.5) / 8388608.0 for t in range(N)])


def kmeanspp_step(d2, c: int, seed: int, stream: int):
    """Draw number c (c >= 1) of k-means++ seeding: one index with probability proportional to d2
    (squared distance to the nearest start point chosen so far).  The draw is an exponential race:
    every point gets e_t = -log(u_t) from its own uniform and the largest d2_t / e_t wins (lowest
    index on exact ties), which selects t with probability d2_t / sum(d2) and needs no prefix sum.
    If every distance is zero the lowest index wins.  Returns (index, race keys)."""
    d2 = np.asarray(d2, np.float64)
    e = -np.log(_kpp_uniforms(d2.shape[0], c, seed, stream))
    keys = d2 / e
    return int(np.argmax(keys)), keys


def kmeanspp_init(X, C: int, seed: int, stream: int) -> np.ndarray:
    """Seeded k-means++ start indices (plain, one candidate per draw): the first is position 0 of the
    seeded shuffle, each further one is drawn by kmeanspp_step from the squared distances to the
    nearest start point so far."""
    X = np.asarray(X, np.float64)
    N = X.shape[0]
    idx = [feistel_permute(0, N, seed, stream)]
    d2 = ((X - X[idx[0]]) ** 2).sum(1)
    for c in range(1, C):
        nxt, _ = kmeanspp_step(d2, c, seed, stream)
        idx.append(nxt)
        d2 = np.minimum(d2, ((X - X[nxt]) ** 2).sum(1))
    return np.asarray(idx, np.int32)


# --------------------------------------------------------------------------------------------
# The paper's own clustering (Appendix "Clustering Details": "Centroid Computation",
# "Balanced Assignment"): one pass of streaming mini-batch k-means, then a per-block assignment
# under a size cap.  Readings where the appendix is silent: the stream visits the vectors in the
# order of the seeded shuffle (position s of the stream is vector pi(s)); centroid r starts as
# the r-th strided sample with total t = x and count c = 1; a minibatch is assigned against the
# centroids as they stand when it starts, then its updates are applied one vector after the
# other; the cap is ceil(factor * B / K) per (block, cluster); a vector that loses its nearest
# centroid to the cap is placed by the two-step rule stated at balanced_assign.  Arithmetic in
# fp64 here (the paper runs it in half precision for speed; nothing in the method depends on that).
# --------------------------------------------------------------------------------------------

def stream_order(N: int, seed: int, stream: int) -> np.ndarray:
    """The shuffled visiting order of the single pass: position s -> vector pi(s)."""
    return np.array([feistel_permute(s, N, seed, stream) for s in range(N)], np.int64)


def streaming_kmeans(X, C, order, init_idx, batch=64, beta=0.9, first_batch=0, n_batches=None,
                     totals=None, counts=None):
    """Appendix "Centroid Computation", step 2.  For each minibatch of `batch` vectors of the
    stream: assign every vector to its nearest current centroid t_j / c_j, then for each vector x
    in stream order t_j <- beta t_j + x, c_j <- beta c_j + 1 for its centroid j.  Runs minibatches
    [first_batch, first_batch + n_batches) from the given state (first_batch = 0: the start state
    t = X[init_idx], c = 1).  Returns (centres, totals, counts, assignments of the streamed vectors)."""
    X = np.asarray(X, np.float64)
    N = X.shape[0]
    nb_all = (N + batch - 1) // batch
    if n_batches is None:
        n_batches = nb_all - first_batch
    if totals is None:
        totals = X[np.asarray(init_idx, np.int64)].copy()
        counts = np.ones(C)
    else:
        totals, counts = np.array(totals, np.float64, copy=True), np.array(counts, np.float64, copy=True)
    seen = []
    for s in range(first_batch, first_batch + n_batches):
        idx = np.asarray(order[s * batch:min(N, (s + 1) * batch)], np.int64)
        a = assign_nearest(X[idx], totals / counts[:, None])
        for u, j in zip(idx, a):
            totals[j] = beta * totals[j] + X[u]
            counts[j] = beta * counts[j] + 1.0
        seen.append(a)
    return totals / counts[:, None], totals, counts, (np.concatenate(seen) if seen else np.zeros(0, np.int32))


def balanced_cap(Bs: int, C: int, factor: float) -> int:
    """Largest allowed size of a (block, cluster) bucket: factor x the average B / K, rounded up."""
    return int(np.ceil(factor * Bs / C))


def balanced_assign(X, centres, S, factor=4.0):
    """Appendix "Balanced Assignment": independently in each spatial block, every vector goes to its
    nearest centroid subject to a maximum bucket size.  Step 1: every vector names its nearest
    centroid; of the vectors of a block that name centroid j, the first cap in position order keep it.
    Step 2: the others, in position order, take the nearest centroid whose bucket still has room
    (counting the step-1 members and the step-2 vectors placed before).  Ties -> lowest centroid."""
    X = np.asarray(X, np.float64)
    centres = np.asarray(centres, np.float64)
    N, C = X.shape[0], centres.shape[0]
    Bs = N // S
    cap = balanced_cap(Bs, C, factor)
    d = (centres * centres).sum(1)[None, :] - 2.0 * (X @ centres.T)
    out = np.full(N, -1, np.int32)
    for b in range(S):
        size = np.zeros(C, np.int64)
        late = []
        for t in range(b * Bs, (b + 1) * Bs):
            j = int(np.argmin(d[t]))
            if size[j] < cap:
                out[t] = j
                size[j] += 1
            else:
                late.append(t)
        for t in late:
            dd = np.where(size < cap, d[t], np.inf)
            j = int(np.argmin(dd))
            out[t] = j
            size[j] += 1
    return out


# --------------------------------------------------------------------------------------------
# Summaries (Section "Summary Computation and Causal Accumulation", Eq. 3-5; Algorithm 1)
# --------------------------------------------------------------------------------------------

def _tilted(qbar, Kmem, Vmem, sigma):
    """Exact attention from every query centroid to a set of keys: (log mass, key mean, value mean)."""
    Cq = qbar.shape[0]
    if Kmem.shape[0] == 0:
        return (np.full(Cq, -np.inf), np.zeros((Cq, Kmem.shape[1])), np.zeros((Cq, Vmem.shape[1])))
    l = sigma * (qbar @ Kmem.T)                          # [Cq, n]
    mx = l.max(1, keepdims=True)
    w = np.exp(l - mx)
    s = w.sum(1, keepdims=True)
    mu = (mx + np.log(s))[:, 0]
    w = w / s
    return mu, w @ Kmem, w @ Vmem


def block_summaries(K, V, a_k, qbar, sigma, S, Ck):
    """Per-block summaries of Eq. 3-5: for block b, query cluster i, key cluster j,
    S_ijb = sum_{k in (b,j)} exp(sigma qbar_i.k); mu = log S; kappa, nu = weighted means.
    Shapes [S,Cq,Ck], [S,Cq,Ck,D], [S,Cq,Ck,Dv]."""
    K = np.asarray(K, np.float64); V = np.asarray(V, np.float64); qbar = np.asarray(qbar, np.float64)
    N, D = K.shape; Dv = V.shape[1]; Cq = qbar.shape[0]; Bs = N // S
    blk = np.arange(N) // Bs
    mu = np.full((S, Cq, Ck), -np.inf)
    kappa = np.zeros((S, Cq, Ck, D)); nu = np.zeros((S, Cq, Ck, Dv))
    for b in range(S):
        for j in range(Ck):
            mem = np.nonzero((blk == b) & (a_k == j))[0]
            mu[b, :, j], kappa[b, :, j], nu[b, :, j] = _tilted(qbar, K[mem], V[mem], sigma)
    return mu, kappa, nu


def accumulate(mu, kappa, nu):
    """Exclusive causal accumulation by the recurrence of Algorithm 1:
    accum_b = accum_{b-1} (+) summary_{b-1}, where (+) adds masses (log-sum-exp of mu)
    and averages kappa, nu with the masses as weights.  accum_0 is empty."""
    S = mu.shape[0]
    muh = np.full_like(mu, -np.inf); kah = np.zeros_like(kappa); nuh = np.zeros_like(nu)
    for b in range(1, S):
        a, c = muh[b - 1], mu[b - 1]
        mx = np.maximum(a, c)
        safe = np.where(np.isfinite(mx), mx, 0.0)
        wa, wc = np.exp(a - safe), np.exp(c - safe)      # exp(-inf) = 0 for empty parts
        tot = wa + wc
        with np.errstate(divide="ignore", invalid="ignore"):
            muh[b] = np.where(tot > 0, safe + np.log(tot), -np.inf)
            fa = np.where(tot > 0, wa / tot, 0.0)[..., None]
            fc = np.where(tot > 0, wc / tot, 0.0)[..., None]
        kah[b] = fa * kah[b - 1] + fc * kappa[b - 1]
        nuh[b] = fa * nuh[b - 1] + fc * nu[b - 1]
    return muh, kah, nuh


def accumulated_summaries(K, V, a_k, qbar, sigma, S, Ck, causal=True):
    """Accumulated summaries by their direct definition ("accumulated_ijb summarizes all
    keys/values in blocks 0..b-1 belonging to key cluster j, specialised for query cluster
    i"): the tilted statistics over M_jb = {u : a_k[u] = j, block(u) < b}.
    Non-causal: one block whose summary covers every key of the cluster."""
    K = np.asarray(K, np.float64); V = np.asarray(V, np.float64); qbar = np.asarray(qbar, np.float64)
    N, D = K.shape; Dv = V.shape[1]; Cq = qbar.shape[0]
    if not causal:
        S = 1
    Bs = N // S
    blk = np.arange(N) // Bs
    muh = np.full((S, Cq, Ck), -np.inf)
    kah = np.zeros((S, Cq, Ck, D)); nuh = np.zeros((S, Cq, Ck, Dv))
    for b in range(S):
        for j in range(Ck):
            vis = (blk < b) if causal else np.ones(N, bool)
            mem = np.nonzero(vis & (a_k == j))[0]
            muh[b, :, j], kah[b, :, j], nuh[b, :, j] = _tilted(qbar, K[mem], V[mem], sigma)
    return muh, kah, nuh


# --------------------------------------------------------------------------------------------
# Dipole correction (Appendix "Error Analysis", paragraphs "Dipole Correction" and "Untilted
# (Partially Specialized) Covariances")
# --------------------------------------------------------------------------------------------

def untilted_covariances(K, V, a_k, S, Ck, causal=True):
    """Shared, untilted within-cluster cross-covariance of values and keys, one per key cluster
    and spatial block: over M_jb = {u : a_k[u] = j, block(u) < b} with uniform weights,
    Cov_0jb(v,k) = mean(v k^T) - mean(v) mean(k)^T  (rows = value dims, columns = key dims).
    Empty sets give zero.  Shape [S, Ck, Dv, D]."""
    K = np.asarray(K, np.float64); V = np.asarray(V, np.float64)
    N, D = K.shape; Dv = V.shape[1]
    if not causal:
        S = 1
    Bs = N // S
    blk = np.arange(N) // Bs
    cov = np.zeros((S, Ck, Dv, D))
    for b in range(S):
        vis = (blk < b) if causal else np.ones(N, bool)
        for j in range(Ck):
            mem = np.nonzero(vis & (a_k == j))[0]
            if mem.size == 0:
                continue
            k, v = K[mem], V[mem]
            cov[b, j] = v.T @ k / mem.size - np.outer(v.mean(0), k.mean(0))
    return cov


def mean_query_centroid(qbar, a_q):
    """qbar_star: the mean of the query centroids weighted by the number of queries each holds
    (the single shared tilt point of "Untilted (Partially Specialized) Covariances")."""
    qbar = np.asarray(qbar, np.float64)
    n = np.bincount(np.asarray(a_q, np.int64), minlength=qbar.shape[0]).astype(np.float64)
    return (n[:, None] * qbar).sum(0) / n.sum()


def tilted_covariances(K, V, a_k, S, Ck, tilt, sigma, causal=True):
    """Shared covariance with one tilt point: as untilted_covariances, but the members of M_jb carry
    the weights w_u proportional to exp(sigma tilt . k_u), normalised inside the set:
    Cov_jb = sum_u w_u v_u k_u^T - (sum_u w_u v_u)(sum_u w_u k_u)^T.  tilt = 0 is the untilted case."""
    K = np.asarray(K, np.float64); V = np.asarray(V, np.float64); tilt = np.asarray(tilt, np.float64)
    N, D = K.shape; Dv = V.shape[1]
    if not causal:
        S = 1
    Bs = N // S
    blk = np.arange(N) // Bs
    cov = np.zeros((S, Ck, Dv, D))
    for b in range(S):
        vis = (blk < b) if causal else np.ones(N, bool)
        for j in range(Ck):
            mem = np.nonzero(vis & (a_k == j))[0]
            if mem.size == 0:
                continue
            k, v = K[mem], V[mem]
            l = sigma * (k @ tilt)
            w = np.exp(l - l.max()); w /= w.sum()
            cov[b, j] = (w[:, None] * v).T @ k - np.outer(w @ v, w @ k)
    return cov


def dipole_weights(muh):
    """Centroid attention weights p_ib(j) = softmax_j muh_ijb over the non-empty key clusters
    (zero elsewhere, and all zero where nothing is visible).  muh [S,Cq,Ck] -> [S,Cq,Ck]."""
    p = np.zeros_like(muh)
    S, Cq, _ = muh.shape
    for b in range(S):
        for i in range(Cq):
            fin = np.isfinite(muh[b, i])
            if fin.any():
                e = np.where(fin, np.exp(np.where(fin, muh[b, i], 0.0) - muh[b, i][fin].max()), 0.0)
                p[b, i] = e / e.sum()
    return p


def merged_dipole(muh, cov):
    """Pre-merged dipole matrix per query cluster and block: Cbar_ib = sum_j p_ib(j) Cov_0jb
    with the centroid attention weights p_ib(j) = softmax_j muh_ijb over the non-empty key
    clusters.  muh [S,Cq,Ck], cov [S,Ck,Dv,D] -> [S,Cq,Dv,D]; zero where no cluster is visible."""
    S, Cq, Ck = muh.shape
    cbar = np.zeros((S, Cq) + cov.shape[2:])
    for b in range(S):
        for i in range(Cq):
            fin = np.isfinite(muh[b, i])
            if not fin.any():
                continue
            mx = muh[b, i][fin].max()
            p = np.where(fin, np.exp(np.where(fin, muh[b, i], mx) - mx), 0.0)
            p /= p.sum()
            cbar[b, i] = np.tensordot(p, cov[b], axes=(0, 0))
    return cbar


# --------------------------------------------------------------------------------------------
# Per-query attention (Section "Two-Level Retrieval", Eq. 6; "Exact Retrieval and Local
# Attention"; "Output merging")
# --------------------------------------------------------------------------------------------

def select_clusters(score, rank_key, m):
    """Top-m key clusters per row.  `rank_key` [n, Ck] is what is ranked (the Eq. 6 score, or
    mu alone for per-query-cluster selection); -inf marks clusters with no visible key.
    Returns int32 [n, m], padded with -1."""
    n, Ck = rank_key.shape
    sel = np.full((n, m), -1, np.int32)
    if m == 0:
        return sel
    order = np.argsort(-rank_key, axis=1, kind="stable")      # ties -> lower index
    for r in range(n):
        cand = order[r][np.isfinite(rank_key[r, order[r]])][:m]
        sel[r, :cand.size] = cand
    return sel


def _lse(x, axis):
    mx = np.max(x, axis=axis, keepdims=True)
    safe = np.where(np.isfinite(mx), mx, 0.0)
    with np.errstate(divide="ignore"):
        out = safe + np.log(np.sum(np.exp(x - safe), axis=axis, keepdims=True))
    return np.squeeze(out, axis=axis)


def _softmax_part(logits, values):
    """(o, lse) of one component: softmax over the finite logits of each row; rows with no
    finite logit give lse = -inf and o = 0."""
    lse = _lse(logits, 1)
    safe = np.where(np.isfinite(lse), lse, 0.0)
    p = np.exp(logits - safe[:, None])
    p[~np.isfinite(lse)] = 0.0
    return p @ values, lse


def select_blocks(bl, k2):
    """Top-k2 spatial blocks of one (query, selected cluster) pair.  `bl` [nb] are the logits of
    the per-block summaries (-inf: no visible key of the cluster in that block).  Largest first,
    ties to the lower block index, fewer than k2 candidates -> all of them.  int32 [k2], -1 padded."""
    out = np.full(k2, -1, np.int32)
    order = np.argsort(-bl, kind="stable")
    cand = order[np.isfinite(bl[order])][:k2]
    out[:cand.size] = cand
    return out


def _segment(Q, K, V, a_k, qbar_i, muh_ib, kah_ib, nuh_ib, rows, b, *, sigma, Bs, m, causal,
             sel_rows, sel_mode, cbar_ib=None, k2=0, blk_i=None, bsel_rows=None, dip=None):
    """All quantities of Algorithm 1's per-query loop for the queries `rows`, which share the
    query cluster (centroid qbar_i) and the spatial block b.
    k2 > 0 (Section "Two-Level Retrieval", spatial block selection): inside every selected cluster
    only the k2 best-scoring earlier blocks are retrieved exactly; its other earlier blocks enter
    through their PER-BLOCK summaries `blk_i` = (mu, kappa, nu)[b', j] of this query cluster.
    `dip` = (p_ib [Ck], cov_b [Ck,Dv,D]): dipole correction next to retrieval (Appendix "Compatibility
    with Retrieval"): the retrieved clusters are attended exactly, so their share leaves the merged
    matrix -- the correction of a query is the merge over the clusters it did NOT retrieve, with the
    centroid weights renormalised over those: (sum_{j far} p(j) Cov_jb) qres / sum_{j far} p(j)."""
    N = K.shape[0]
    Ck = muh_ib.shape[0]
    qp = sigma * Q[rows]                                   # full (scaled) query
    qres = qp - sigma * qbar_i[None, :]                    # residual
    score = qres @ kah_ib.T + muh_ib[None, :]              # Eq. 6
    nonempty = np.isfinite(muh_ib)
    score = np.where(nonempty[None, :], score, -np.inf)
    rank = score if sel_mode == 0 else np.broadcast_to(np.where(nonempty, muh_ib, -np.inf), score.shape)
    if sel_rows is None:
        sel_rows = select_clusters(score, rank, m)
    # diagnostic only: margin between the m-th and (m+1)-th ranked cluster (inf if no choice)
    srt = -np.sort(-rank, axis=1)
    if 0 < m < Ck:
        with np.errstate(invalid="ignore"):
            gap = np.where(np.isfinite(srt[:, m]), srt[:, m - 1] - srt[:, m], np.inf)
    else:
        gap = np.full(len(rows), np.inf)
    selmask = np.zeros((len(rows), Ck), bool)
    for r in range(len(rows)):
        s = sel_rows[r][sel_rows[r] >= 0]
        selmask[r, s] = True
    # 1. far field: approximate attention over the clusters that were not retrieved
    far_logit = np.where(nonempty[None, :] & ~selmask, score, -np.inf)
    o_far, lse_far = _softmax_part(far_logit, nuh_ib)
    if cbar_ib is not None:
        # dipole: the linear value term, merged over clusters; the mass (lse_far) is unchanged
        o_far = o_far + np.where(np.isfinite(lse_far)[:, None], qres @ cbar_ib.T, 0.0)
    dip_c = np.zeros((len(rows), V.shape[1])); dip_Z = np.zeros(len(rows))
    if dip is not None:
        p_ib, cov_b = dip
        for r in range(len(rows)):
            far = nonempty & ~selmask[r]
            dip_Z[r] = p_ib[far].sum()
            if np.isfinite(lse_far[r]) and dip_Z[r] > 0:
                dip_c[r] = np.tensordot(p_ib[far], cov_b[far], axes=(0, 0)) @ qres[r] / dip_Z[r]
        o_far = o_far + dip_c
    # 3. exact attention over the retrieved clusters' visible keys (full query)
    u = np.arange(N)
    vis = (u // Bs < b) if causal else np.ones(N, bool)
    ret_mask = vis[None, :] & selmask[:, a_k]
    o_near = np.zeros((len(rows), V.shape[1])); lse_near = np.full(len(rows), -np.inf)
    bsel = None
    near_logit = None
    if k2 > 0 and causal:
        # 2. block selection inside the selected clusters, with the pre-accumulation summaries
        mu_b, ka_b, nu_b = blk_i                           # [S, Ck], [S, Ck, D], [S, Ck, Dv]
        bsel = np.full((len(rows), max(m, 1), k2), -1, np.int32)
        blk_of = u // Bs
        ret_mask = np.zeros((len(rows), N), bool)
        near_logit = np.full((len(rows), max(b, 1), Ck), -np.inf)   # logit of the stand-in key (b', j) for each query
        for r in range(len(rows)):
            near_logits, near_values = [], []
            for k, j in enumerate(sel_rows[r]):
                if j < 0:
                    continue
                bl = np.full(b, -np.inf)
                for bp in range(b):                        # block-index causal mask: b' < b
                    if np.isfinite(mu_b[bp, j]):
                        bl[bp] = qres[r] @ ka_b[bp, j] + mu_b[bp, j]
                chosen = select_blocks(bl, k2) if bsel_rows is None else np.asarray(bsel_rows[r][k], np.int32)
                bsel[r, k] = chosen
                for bp in range(b):
                    if not np.isfinite(bl[bp]):
                        continue
                    if bp in chosen[chosen >= 0]:
                        ret_mask[r] |= (a_k == j) & (blk_of == bp)
                    else:                                  # not retrieved: its per-block summary stands in
                        near_logits.append(bl[bp]); near_values.append(nu_b[bp, j])
                        near_logit[r, bp, j] = bl[bp]
            if near_logits:
                o1, l1 = _softmax_part(np.asarray(near_logits)[None, :], np.asarray(near_values))
                o_near[r], lse_near[r] = o1[0], l1[0]
    logit = qp @ K.T
    ret_logit = np.where(ret_mask, logit, -np.inf)
    o_ret, lse_ret = _softmax_part(ret_logit, V)
    # 4. exact causal attention inside the query's own block
    if causal:
        loc_mask = (u[None, :] // Bs == b) & (u[None, :] <= np.asarray(rows)[:, None])
    else:
        loc_mask = np.zeros((len(rows), N), bool)
    loc_logit = np.where(loc_mask, logit, -np.inf)
    o_loc, lse_loc = _softmax_part(loc_logit, V)
    # merge by log-sum-exp weights (component 2, the near field, is empty when k_2 = all)
    lses = np.stack([lse_far, lse_ret, lse_loc, lse_near], 1)
    L = _lse(lses, 1)
    wts = np.exp(lses - L[:, None])
    O = wts[:, 0:1] * o_far + wts[:, 1:2] * o_ret + wts[:, 2:3] * o_loc + wts[:, 3:4] * o_near
    return dict(O=O, L=L, sel=sel_rows, bsel=bsel, dip_c=dip_c, dip_Z=dip_Z, nonempty=nonempty, near_logit=near_logit, o_near=o_near, lse_near=lse_near, sel_gap=gap, selmask=selmask, score=score, qp=qp, qres=qres,
                far_logit=far_logit, exact_logit=np.where(ret_mask | loc_mask, logit, -np.inf),
                o_far=o_far, lse_far=lse_far, o_ret=o_ret, lse_ret=lse_ret,
                o_loc=o_loc, lse_loc=lse_loc)


def _segments(a_q, N, S, causal, rows):
    Bs = N // S
    blk = np.arange(N) // Bs if causal else np.zeros(N, np.int64)
    keep = np.zeros(N, bool)
    keep[np.arange(N) if rows is None else np.asarray(rows)] = True
    for b in range(S if causal else 1):
        for i in np.unique(a_q[(blk == b) & keep]):
            yield b, int(i), np.nonzero((blk == b) & (a_q == i) & keep)[0]


def forward(Q, K, V, a_q, a_k, qbar, *, sigma, S, Ck, m, causal=True, sel=None, sel_mode=0,
            summ=None, rows=None, dipole=0, k2=0, bsel=None, blocks=None):
    """MuSe attention for one head.  Returns a dict with O [N,Dv], LSE [N], sel [N,m] and the
    three component (o, lse) pairs.  `sel` forces the retrieved clusters (teacher forcing);
    `rows` restricts the computation to some queries (others are left zero / -inf / -1).
    `dipole=1` adds the untilted dipole correction to the far field, `dipole=2` the one whose shared
    covariance is tilted at the mass-weighted mean query centroid (`a_q` gives the masses).  The paper
    defines the pre-merged correction without retrieval (m = 0); with m > 0 each query's correction is
    the merge over the clusters it did not retrieve (see _segment).
    `k2` > 0: two-level retrieval; per (query, selected cluster) only the k2 best earlier blocks
    are retrieved exactly (returned as bsel [N, m, k2], -1 padded; `bsel` forces them), the other
    earlier blocks of the selected clusters are approximated by their per-block summaries
    (`blocks` = block_summaries(...) may be passed in).  k2 = 0 retrieves every visible block."""
    if dipole not in (0, 1, 2):
        raise ValueError("dipole is 0 (off), 1 (untilted) or 2 (tilted at the mean query centroid)")
    if k2 < 0 or (k2 > 0 and dipole):
        raise ValueError("k2 must be >= 0 and is not combined with the dipole correction")
    Q = np.asarray(Q, np.float64); K = np.asarray(K, np.float64); V = np.asarray(V, np.float64)
    qbar = np.asarray(qbar, np.float64)
    N, D = Q.shape; Dv = V.shape[1]
    if not causal:
        S = 1
    Bs = N // S
    if summ is None:
        summ = accumulated_summaries(K, V, a_k, qbar, sigma, S, Ck, causal)
    muh, kah, nuh = summ
    if k2 > 0 and causal and blocks is None:
        blocks = block_summaries(K, V, a_k, qbar, sigma, S, Ck)
    cbar = cov = pw = None
    if dipole:
        cov = (untilted_covariances(K, V, a_k, S, Ck, causal) if dipole == 1 else
               tilted_covariances(K, V, a_k, S, Ck, mean_query_centroid(qbar, a_q), sigma, causal))
        cbar = merged_dipole(muh, cov)
        pw = dipole_weights(muh)
    out = dict(O=np.zeros((N, Dv)), LSE=np.full(N, -np.inf), sel=np.full((N, m), -1, np.int32),
               sel_gap=np.full(N, np.inf))
    for name in ("o_far", "o_ret", "o_loc", "o_near"):
        out[name] = np.zeros((N, Dv))
    for name in ("lse_far", "lse_ret", "lse_loc", "lse_near"):
        out[name] = np.full(N, -np.inf)
    if k2 > 0:
        out["bsel"] = np.full((N, max(m, 1), k2), -1, np.int32)
    for b, i, r in _segments(a_q, N, S, causal, rows):
        seg = _segment(Q, K, V, a_k, qbar[i], muh[b, i], kah[b, i], nuh[b, i], r, b,
                       sigma=sigma, Bs=Bs, m=m, causal=causal,
                       sel_rows=None if sel is None else sel[r], sel_mode=sel_mode,
                       cbar_ib=cbar[b, i] if (dipole and m == 0) else None, k2=k2,
                       blk_i=None if blocks is None else (blocks[0][:, i], blocks[1][:, i], blocks[2][:, i]),
                       bsel_rows=None if bsel is None else bsel[r],
                       dip=(pw[b, i], cov[b]) if (dipole and m > 0) else None)
        out["O"][r], out["LSE"][r], out["sel"][r] = seg["O"], seg["L"], seg["sel"]
        out["sel_gap"][r] = seg["sel_gap"]
        for name in ("o_far", "lse_far", "o_ret", "lse_ret", "o_loc", "lse_loc", "o_near", "lse_near"):
            out[name][r] = seg[name]
        if k2 > 0 and seg["bsel"] is not None:
            out["bsel"][r] = seg["bsel"]
    out["summ"] = summ
    out["cbar"] = cbar
    out["cov"] = cov
    return out


def backward(Q, K, V, dO, a_q, a_k, qbar, *, sigma, S, Ck, m, causal=True, sel=None, sel_mode=0,
             agg_grad=True, rows=None, k2=0, bsel=None, dipole=0):
    """Gradients of sum(O * dO) w.r.t. Q, K, V with the assignments, the selections and the
    query centroids held constant (Appendix "Centroid Gradient Flow"; assignments and
    selections are discrete).  agg_grad=False also treats the tilted aggregation weights as
    constants (Appendix "Aggregation Weight Gradient Flow").  k2 > 0: two-level retrieval; the
    chosen blocks (`bsel`) are constants like the clusters, and the stand-in keys of the other
    blocks pass their gradient on through the per-block summaries.  `dipole` as in forward(): the
    correction is differentiated through the residual, the shared covariances (to keys and values) and
    the centroid weights p_ib(j) (to the log-masses, hence dropped with agg_grad=False, as is the
    dependence of the dipole=2 tilt weights on the keys); the tilt point is a constant like qbar.
    Returns (dQ, dK, dV, fwd)."""
    if dipole not in (0, 1, 2) or (dipole and k2 > 0):
        raise ValueError("dipole is 0, 1 or 2 and is not combined with k2 > 0")
    Q = np.asarray(Q, np.float64); K = np.asarray(K, np.float64); V = np.asarray(V, np.float64)
    dO = np.asarray(dO, np.float64); qbar = np.asarray(qbar, np.float64)
    N, D = Q.shape; Dv = V.shape[1]; Cq = qbar.shape[0]
    if not causal:
        S = 1
    Bs = N // S
    muh, kah, nuh = accumulated_summaries(K, V, a_k, qbar, sigma, S, Ck, causal)
    two_level = k2 > 0 and causal
    if two_level:
        mu_b, ka_b, nu_b = block_summaries(K, V, a_k, qbar, sigma, S, Ck)
        dmu_b = np.zeros_like(mu_b); dka_b = np.zeros_like(ka_b); dnu_b = np.zeros_like(nu_b)
    dQ = np.zeros((N, D)); dK = np.zeros((N, D)); dV = np.zeros((N, Dv))
    dmu = np.zeros_like(muh); dka = np.zeros_like(kah); dnu = np.zeros_like(nuh)
    if dipole:
        qstar = np.zeros(D) if dipole == 1 else mean_query_centroid(qbar, a_q)
        cov = tilted_covariances(K, V, a_k, S, Ck, qstar, sigma, causal)
        pw = dipole_weights(muh)
        dcov = np.zeros_like(cov); dpw = np.zeros_like(pw)
    fwd = dict(O=np.zeros((N, Dv)), LSE=np.full(N, -np.inf), sel=np.full((N, m), -1, np.int32),
               sel_gap=np.full(N, np.inf))
    for b, i, r in _segments(a_q, N, S, causal, rows):
        seg = _segment(Q, K, V, a_k, qbar[i], muh[b, i], kah[b, i], nuh[b, i], r, b,
                       sigma=sigma, Bs=Bs, m=m, causal=causal,
                       sel_rows=None if sel is None else sel[r], sel_mode=sel_mode, k2=k2 if two_level else 0,
                       blk_i=(mu_b[:, i], ka_b[:, i], nu_b[:, i]) if two_level else None,
                       bsel_rows=None if bsel is None else bsel[r],
                       dip=(pw[b, i], cov[b]) if dipole else None)
        fwd["O"][r], fwd["LSE"][r], fwd["sel"][r] = seg["O"], seg["L"], seg["sel"]
        fwd["sel_gap"][r] = seg["sel_gap"]
        L = seg["L"][:, None]
        g_out = dO[r]
        delta = (g_out * seg["O"]).sum(1, keepdims=True)
        # the merged output is one softmax over {exact keys} U {far clusters}
        P = np.exp(seg["exact_logit"] - L)                 # [n, N], zero where masked
        dV += P.T @ g_out
        G = P * (g_out @ V.T - delta)
        dqp = G @ K
        dK += G.T @ seg["qp"]
        Pf = np.exp(seg["far_logit"] - L)                  # [n, Ck]
        dnu[b, i] += Pf.T @ g_out
        # with the dipole every far cluster's value is nuh_j + c_t (c_t = the query's correction)
        Gf = Pf * (g_out @ nuh[b, i].T + (g_out * seg["dip_c"]).sum(1, keepdims=True) - delta)
        dqp += Gf @ kah[b, i]                              # d score / d q = kah (qbar constant)
        dka[b, i] += Gf.T @ seg["qres"]
        dmu[b, i] += Gf.sum(0)
        if two_level and seg["near_logit"] is not None:
            # the stand-in keys (b', j) of the non-retrieved blocks of the selected clusters: logit
            # qres . kappa_b'j + mu_b'j, value nu_b'j (per-block summaries of this query cluster)
            for bp in range(b):
                Pn = np.exp(seg["near_logit"][:, bp, :] - L)       # [n, Ck], zero where there is no stand-in key
                dnu_b[bp, i] += Pn.T @ g_out
                Gn = Pn * (g_out @ nu_b[bp, i].T - delta)
                dqp += Gn @ ka_b[bp, i]
                dka_b[bp, i] += Gn.T @ seg["qres"]
                dmu_b[bp, i] += Gn.sum(0)
        if dipole:
            # c_t = M_t qres_t / Z_t,  M_t = sum_{j far} p(j) Cov_jb,  Z_t = sum_{j far} p(j)
            w_far = np.exp(seg["lse_far"] - seg["L"])
            for x in range(len(r)):
                Z = seg["dip_Z"][x]
                if not (np.isfinite(seg["lse_far"][x]) and Z > 0):
                    continue
                far = seg["nonempty"] & ~seg["selmask"][x]
                dc = w_far[x] * g_out[x]
                M = np.tensordot(pw[b, i][far], cov[b][far], axes=(0, 0))
                dqp[x] += M.T @ dc / Z
                dM = np.outer(dc, seg["qres"][x]) / Z
                dcov[b][far] += pw[b, i][far][:, None, None] * dM
                dpw[b, i][far] += (cov[b][far] * dM).sum((1, 2)) - (dc @ seg["dip_c"][x]) / Z
        dQ[r] = sigma * dqp
    if dipole:
        # softmax backward of the centroid weights into the accumulated log-masses
        dmu += pw * (dpw - (pw * dpw).sum(2, keepdims=True))
    # through the accumulated summaries to the keys and values they were built from
    blk = np.arange(N) // Bs
    for b in range(S):
        for j in range(Ck):
            vis = (blk < b) if causal else np.ones(N, bool)
            mem = np.nonzero(vis & (a_k == j))[0]
            if mem.size == 0:
                continue
            l = sigma * (qbar @ K[mem].T)                  # [Cq, n]
            w = np.exp(l - muh[b, :, j][:, None])          # normalised tilt weights
            dK[mem] += w.T @ dka[b, :, j]
            dV[mem] += w.T @ dnu[b, :, j]
            if agg_grad:
                dl = w * (dmu[b, :, j][:, None]
                          + dka[b, :, j] @ K[mem].T - (dka[b, :, j] * kah[b, :, j]).sum(1)[:, None]
                          + dnu[b, :, j] @ V[mem].T - (dnu[b, :, j] * nuh[b, :, j]).sum(1)[:, None])
                dK[mem] += sigma * (dl.T @ qbar)
    if dipole:
        # through the shared covariances: Cov = sum_u w_u (v_u - vm)(k_u - km)^T over the visible members
        for b in range(S):
            for j in range(Ck):
                vis = (blk < b) if causal else np.ones(N, bool)
                mem = np.nonzero(vis & (a_k == j))[0]
                if mem.size == 0:
                    continue
                l = sigma * (K[mem] @ qstar)
                w = np.exp(l - l.max()); w /= w.sum()
                kc = K[mem] - w @ K[mem]; vc = V[mem] - w @ V[mem]
                G = dcov[b, j]
                dV[mem] += w[:, None] * (kc @ G.T)
                dK[mem] += w[:, None] * (vc @ G)
                if agg_grad and dipole == 2:
                    dl = w * (((vc @ G) * kc).sum(1) - (G * cov[b, j]).sum())
                    dK[mem] += sigma * dl[:, None] * qstar[None, :]
    if two_level:
        # ... and through the per-block summaries to the keys and values of their own bucket
        for bp in range(S):
            for j in range(Ck):
                mem = np.nonzero((blk == bp) & (a_k == j))[0]
                if mem.size == 0:
                    continue
                l = sigma * (qbar @ K[mem].T)
                w = np.exp(l - mu_b[bp, :, j][:, None])
                dK[mem] += w.T @ dka_b[bp, :, j]
                dV[mem] += w.T @ dnu_b[bp, :, j]
                if agg_grad:
                    dl = w * (dmu_b[bp, :, j][:, None]
                              + dka_b[bp, :, j] @ K[mem].T - (dka_b[bp, :, j] * ka_b[bp, :, j]).sum(1)[:, None]
                              + dnu_b[bp, :, j] @ V[mem].T - (dnu_b[bp, :, j] * nu_b[bp, :, j]).sum(1)[:, None])
                    dK[mem] += sigma * (dl.T @ qbar)
    return dQ, dK, dV, fwd


# --------------------------------------------------------------------------------------------
# Whole layer with grouped-query heads: [B,Hq,N,D] queries over [B,Hkv,N,D] keys/values
# --------------------------------------------------------------------------------------------

def _head_map(Hq, Hkv, head_map):
    return [h * Hkv // Hq for h in range(Hq)] if head_map is None else list(head_map)


def layer_forward(Q, K, V, a_q, a_k, qbar, *, sigma, S, Ck, m, causal=True, sel=None, sel_mode=0,
                  head_map=None, dipole=0):
    B, Hq, N, D = Q.shape
    Hkv = K.shape[1]
    hm = _head_map(Hq, Hkv, head_map)
    O = np.zeros((B, Hq, N, V.shape[-1])); LSE = np.zeros((B, Hq, N))
    SEL = np.full((B, Hq, N, m), -1, np.int32)
    for b in range(B):
        for h in range(Hq):
            g = hm[h]
            f = forward(Q[b, h], K[b, g], V[b, g], a_q[b, h], a_k[b, g], qbar[b, h], sigma=sigma,
                        S=S, Ck=Ck, m=m, causal=causal, sel=None if sel is None else sel[b, h],
                        sel_mode=sel_mode, dipole=dipole)
            O[b, h], LSE[b, h], SEL[b, h] = f["O"], f["LSE"], f["sel"]
    return O, LSE, SEL


def layer_backward(Q, K, V, dO, a_q, a_k, qbar, *, sigma, S, Ck, m, causal=True, sel=None,
                   sel_mode=0, agg_grad=True, head_map=None, k2=0, bsel=None, dipole=0):
    """dK, dV of a kv head are the sums over the query heads that share it."""
    B, Hq, N, D = Q.shape
    Hkv = K.shape[1]
    hm = _head_map(Hq, Hkv, head_map)
    dQ = np.zeros(Q.shape); dK = np.zeros(K.shape); dV = np.zeros(V.shape)
    for b in range(B):
        for h in range(Hq):
            g = hm[h]
            q, k, v, _ = backward(Q[b, h], K[b, g], V[b, g], dO[b, h], a_q[b, h], a_k[b, g],
                                  qbar[b, h], sigma=sigma, S=S, Ck=Ck, m=m, causal=causal,
                                  sel=None if sel is None else sel[b, h], sel_mode=sel_mode,
                                  agg_grad=agg_grad, k2=k2, bsel=None if bsel is None else bsel[b, h],
                                  dipole=dipole)
            dQ[b, h] = q
            dK[b, g] += k
            dV[b, g] += v
    return dQ, dK, dV
