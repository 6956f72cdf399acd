"""Pins of the oracle's statement of the paper's own clustering (Appendix "Clustering Details": "Centroid
Computation" = one pass of streaming mini-batch k-means; "Balanced Assignment" = per-block nearest centroid under
a size cap).  Each pin is something other than the oracle's own formula: closed forms, hand-computed cases,
invariants, brute force written separately."""
import numpy as np
import pytest

from oracle import muse_oracle as orc


def test_stream_order_is_a_permutation_and_starts_are_strided_samples():
    N, C = 1000, 8
    order = orc.stream_order(N, 5, 3)
    assert sorted(order.tolist()) == list(range(N))
    init = orc.strided_init(N, C, 5, 3)
    assert np.array_equal(init, order[np.arange(C) * (N // C)])        # every floor(N/C)-th vector of the shuffled sequence


def test_one_cluster_is_an_exponentially_weighted_mean_of_the_stream():
    """C = 1: every vector updates the single centroid, so t = beta^N x0 + sum_s beta^(N-1-s) x_pi(s), c likewise."""
    rng = np.random.default_rng(0)
    N, D, beta = 300, 5, 0.9
    X = rng.normal(size=(N, D))
    order = orc.stream_order(N, 1, 0)
    init = orc.strided_init(N, 1, 1, 0)
    cen, t, c, a = orc.streaming_kmeans(X, 1, order, init, batch=64, beta=beta)
    w = beta ** (N - 1 - np.arange(N))
    t_ref = beta ** N * X[init[0]] + (w[:, None] * X[order]).sum(0)
    c_ref = beta ** N + w.sum()
    assert np.allclose(t[0], t_ref, rtol=1e-12, atol=1e-12) and np.isclose(c[0], c_ref, rtol=1e-12)
    assert np.allclose(cen[0], t_ref / c_ref) and np.all(a == 0)


def test_beta_one_gives_plain_running_means():
    """beta = 1 and separated blobs whose starts sit in distinct blobs: centroid j = (start + sum of blob j) / (1 + n_j)."""
    rng = np.random.default_rng(1)
    N, C, D = 512, 4, 3
    order = orc.stream_order(N, 9, 2)
    init = orc.strided_init(N, C, 9, 2)
    label = rng.integers(0, C, size=N)
    label[init] = np.arange(C)
    means = 100.0 * np.eye(C, D)
    X = means[label] + 0.01 * rng.normal(size=(N, D))
    cen, t, c, a = orc.streaming_kmeans(X, C, order, init, batch=64, beta=1.0)
    assert np.array_equal(a, label[order])
    for j in range(C):
        mem = X[label == j]
        assert np.allclose(cen[j], (X[init[j]] + mem.sum(0)) / (1 + len(mem)), rtol=1e-12)
        assert np.isclose(c[j], 1 + len(mem))


def test_separated_blobs_give_per_cluster_weighted_means_in_stream_order():
    rng = np.random.default_rng(2)
    N, C, D, beta = 640, 5, 4, 0.9
    order = orc.stream_order(N, 4, 1)
    init = orc.strided_init(N, C, 4, 1)
    label = rng.integers(0, C, size=N)
    label[init] = np.arange(C)
    X = 50.0 * np.eye(C, D)[label] + 0.01 * rng.normal(size=(N, D))
    cen, t, c, _ = orc.streaming_kmeans(X, C, order, init, batch=64, beta=beta)
    for j in range(C):
        mem = [u for u in order if label[u] == j]                    # the cluster's vectors as the stream meets them
        n = len(mem)
        w = beta ** (n - 1 - np.arange(n))
        assert np.allclose(t[j], beta ** n * X[init[j]] + (w[:, None] * X[mem]).sum(0), rtol=1e-11)
        assert np.isclose(c[j], beta ** n + w.sum(), rtol=1e-12)


def test_a_minibatch_is_assigned_before_any_of_its_updates():
    """Hand-computed, 1-D, two centroids at 0 and 10 (vectors 0 and 1), one minibatch holding 4.9 then 5.5.
    Assigned against the centroids at the start: 4.9 -> 0, 5.5 -> 10.  (Had the first update been applied at once,
    centroid 0 would sit at 4.9 / 1.9 = 2.58 and take 5.5 as well.)  All four vectors stream, in two minibatches of 2:
    minibatch 1 = the two start vectors themselves (0 -> centroid 0, 10 -> centroid 1):
      t0 = 0.9*0 + 0 = 0, c0 = 1.9;  t1 = 0.9*10 + 10 = 19, c1 = 1.9  -> centroids 0 and 10
    minibatch 2: t0 = 0.9*0 + 4.9 = 4.9, c0 = 0.9*1.9 + 1 = 2.71;  t1 = 0.9*19 + 5.5 = 22.6, c1 = 2.71."""
    X = np.array([[0.0], [10.0], [4.9], [5.5]])
    cen, t, c, a = orc.streaming_kmeans(X, 2, order=np.arange(4), init_idx=[0, 1], batch=2, beta=0.9)
    assert a.tolist() == [0, 1, 0, 1]
    assert np.allclose(t[:, 0], [4.9, 22.6]) and np.allclose(c, [2.71, 2.71])
    assert np.allclose(cen[:, 0], [4.9 / 2.71, 22.6 / 2.71])
    # the same stream with minibatches of one vector updates at once, and 5.5 then falls to centroid 0
    _, _, _, a1 = orc.streaming_kmeans(X, 2, order=np.arange(4), init_idx=[0, 1], batch=1, beta=0.9)
    assert a1.tolist() == [0, 1, 0, 0]


def test_updates_inside_a_minibatch_are_sequential():
    """Two vectors of one minibatch on the same centroid: t <- beta (beta t + x1) + x2, not beta t + x1 + x2."""
    X = np.array([[1.0], [2.0], [3.0]])
    _, t, c, _ = orc.streaming_kmeans(X, 1, order=[1, 2], init_idx=[0], batch=2, beta=0.5, n_batches=1)
    assert np.isclose(t[0, 0], 0.5 * (0.5 * 1.0 + 2.0) + 3.0) and np.isclose(c[0], 0.5 * (0.5 * 1.0 + 1.0) + 1.0)


def test_continuing_from_a_saved_state_equals_one_pass():
    rng = np.random.default_rng(3)
    N, C = 500, 6
    X = rng.normal(size=(N, 4))
    order, init = orc.stream_order(N, 2, 0), orc.strided_init(N, C, 2, 0)
    full = orc.streaming_kmeans(X, C, order, init)
    _, t, c, a0 = orc.streaming_kmeans(X, C, order, init, n_batches=3)
    part = orc.streaming_kmeans(X, C, order, init, first_batch=3, totals=t, counts=c)
    assert np.array_equal(full[1], part[1]) and np.array_equal(full[2], part[2])
    assert np.array_equal(full[3], np.concatenate([a0, part[3]]))


def test_streaming_step_matches_scalar_brute_force():
    """The same recurrence written out with scalar loops (no shared helper): nearest by true squared distance."""
    rng = np.random.default_rng(4)
    N, C, D, beta, batch = 40, 3, 2, 0.9, 8
    X = rng.normal(size=(N, D))
    order = orc.stream_order(N, 7, 0)
    init = orc.strided_init(N, C, 7, 0)
    t = [[float(X[i][d]) for d in range(D)] for i in init]
    c = [1.0] * C
    for s in range(0, N, batch):
        chunk = [int(u) for u in order[s:s + batch]]
        cents = [[t[j][d] / c[j] for d in range(D)] for j in range(C)]
        picks = []
        for u in chunk:
            best, bj = None, -1
            for j in range(C):
                dist = sum((X[u][d] - cents[j][d]) ** 2 for d in range(D))
                if best is None or dist < best:
                    best, bj = dist, j
            picks.append(bj)
        for u, j in zip(chunk, picks):
            t[j] = [beta * t[j][d] + X[u][d] for d in range(D)]
            c[j] = beta * c[j] + 1.0
    cen, tt, cc, _ = orc.streaming_kmeans(X, C, order, init, batch=batch, beta=beta)
    assert np.allclose(tt, np.array(t), rtol=1e-12) and np.allclose(cc, c, rtol=1e-12)


# ---------------------------------------------------------------------------------------------
# Balanced assignment
# ---------------------------------------------------------------------------------------------

def test_cap_is_factor_times_average_rounded_up():
    assert orc.balanced_cap(8192, 128, 4) == 256 and orc.balanced_cap(10, 3, 1) == 4 and orc.balanced_cap(8, 2, 1) == 4


def test_unbinding_cap_is_the_nearest_centroid_per_block():
    rng = np.random.default_rng(5)
    X, cen = rng.normal(size=(256, 3)), rng.normal(size=(8, 3))
    a = orc.balanced_assign(X, cen, S=4, factor=64.0)                # cap = 512 > block size
    d = ((X[:, None, :] - cen[None]) ** 2).sum(-1)
    assert np.array_equal(a, d.argmin(1))


def test_hand_computed_overflow():
    """One block of 8 vectors on a line, centroids at 0 and 10, factor 1 -> cap 4.  All are nearer 0; the first four
    in position order keep it, the other four go to the only centroid with room."""
    X = np.array([[0.1], [0.2], [0.3], [0.4], [0.5], [0.6], [0.7], [0.8]])
    a = orc.balanced_assign(X, np.array([[0.0], [10.0]]), S=1, factor=1.0)
    assert a.tolist() == [0, 0, 0, 0, 1, 1, 1, 1]


def test_step_one_members_are_seated_before_any_displaced_vector():
    """Centroids at 0, 10, 20; cap = ceil(1 * 6 / 3) = 2; vectors (position order): 0.1, 0.2, 0.3 (all nearest 0),
    then 9.0, 9.5, 10.5 (all nearest 10).  Step 1 seats 0.1, 0.2 at 0 and 9.0, 9.5 at 10.  Step 2: 0.3 (nearest
    with room: 20, since 0 and 10 are full) and 10.5 -> 20.  A single greedy pass in position order would instead
    send 0.3 to centroid 10 and push 9.5 out of it."""
    X = np.array([[0.1], [0.2], [0.3], [9.0], [9.5], [10.5]])
    a = orc.balanced_assign(X, np.array([[0.0], [10.0], [20.0]]), S=1, factor=1.0)
    assert a.tolist() == [0, 0, 2, 1, 1, 2]


def test_blocks_are_independent_and_sizes_respect_the_cap():
    rng = np.random.default_rng(6)
    N, C, S = 512, 8, 4
    X = rng.normal(size=(N, 2)) * np.array([3.0, 0.2])               # elongated: a few centroids attract most vectors
    cen = rng.normal(size=(C, 2))
    a = orc.balanced_assign(X, cen, S=S, factor=1.0)
    Bs, cap = N // S, orc.balanced_cap(N // S, C, 1.0)
    d = ((X[:, None, :] - cen[None]) ** 2).sum(-1)
    near = d.argmin(1)
    for b in range(S):
        blk = slice(b * Bs, (b + 1) * Bs)
        sizes = np.bincount(a[blk], minlength=C)
        assert sizes.max() <= cap and sizes.sum() == Bs
        # a vector that does not sit at its nearest centroid found that bucket full of earlier-or-nearest claimants
        for t in range(b * Bs, (b + 1) * Bs):
            if a[t] != near[t]:
                assert sizes[near[t]] == cap
        # a block on its own gives the same answer
        assert np.array_equal(a[blk], orc.balanced_assign(X[blk], cen, S=1, factor=1.0))
    assert (a != near).any()                                         # the cap does bind in this case
