"""The seeded input generators: determinism, dtype exactness, shapes."""
import numpy as np
import torch

from paper_2509_10406_b200 import workloads as wl


def test_round_bf16_matches_torch():
    x = np.random.default_rng(0).standard_normal(4096).astype(np.float32) * 37.0
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(wl.round_bf16(x), ref)


def test_head_inputs_are_seeded_and_bf16_exact():
    w = wl.WORKLOADS["small"].with_(N=512, components=16)
    a = wl.make_head_inputs(w, 1, 3)
    b = wl.make_head_inputs(w, 1, 3)
    for x, y in zip(a, b):
        assert np.array_equal(x, y) and x.shape == (512, 64) and x.dtype == np.float32
        assert np.array_equal(wl.round_bf16(x), x)
    c = wl.make_head_inputs(w, 1, 4)
    assert not np.array_equal(a[0], c[0])


def test_gqa_heads_share_keys():
    w = wl.WORKLOADS["gqa1b"].with_(N=256, components=8)
    _, k0, v0, _ = wl.make_head_inputs(w, 0, 4)
    _, k1, v1, _ = wl.make_head_inputs(w, 0, 7)
    _, k2, _, _ = wl.make_head_inputs(w, 0, 8)
    assert np.array_equal(k0, k1) and np.array_equal(v0, v1) and not np.array_equal(k0, k2)
    Q, K, V, dO = wl.make_inputs(w.with_(Hq=8, Hkv=2))
    assert Q.shape == (1, 8, 256, 64) and K.shape == (1, 2, 256, 64)


def test_rope_preserves_norms_and_position_zero():
    x = np.random.default_rng(1).standard_normal((32, 16)).astype(np.float32)
    y = wl.rope(x, 1e4)
    np.testing.assert_allclose(np.linalg.norm(y, axis=1), np.linalg.norm(x, axis=1), rtol=1e-5)
    np.testing.assert_allclose(y[0], x[0], atol=1e-7)


def test_init_indices_distinct():
    X = np.random.default_rng(2).standard_normal((300, 4))
    i1 = wl.kmeanspp_indices(X, 10, 5, 0)
    assert len(set(i1.tolist())) == 10
    i2 = wl.random_init_indices(300, 10, 5, 0)
    assert len(set(i2.tolist())) == 10 and np.array_equal(i2, wl.random_init_indices(300, 10, 5, 0))
