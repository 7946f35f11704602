"""Checks of the seeded workload generators (no attention arithmetic involved)."""
import numpy as np
import torch

from paper_2603_04127_b200 import inputs


def test_bf16_rounding_matches_torch():
    rng = np.random.default_rng(0)
    x = (rng.standard_normal(5000) * 10 ** rng.uniform(-6, 6, 5000)).astype(np.float32)
    want = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    got = inputs.round_to_bf16(x)
    assert np.array_equal(got, want)
    bits = inputs.bf16_bits(got)
    back = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(back, want)


def test_spectrum_and_orthogonal_factor():
    lam = inputs.covariance_spectrum(64, 0.9)
    assert np.isclose(lam.sum(), 64) and np.isclose(lam[1] / lam[0], 0.9)
    lam4 = inputs.covariance_spectrum(64, 0.9, 4.0)
    assert np.isclose(lam4[0], 4 * lam[0]) and np.allclose(lam4[1:], lam[1:])
    U = inputs.random_orthogonal(16, np.random.default_rng(1))
    np.testing.assert_allclose(U @ U.T, np.eye(16), atol=1e-12)


def test_subset_of_pairs_reproduces_full_tensor():
    wl = inputs.small(B=2, H=3, N=8, d=4, m=8, dtype="bf16", causal=True)
    full = inputs.generate(wl)
    sub = inputs.generate(wl, pairs=[(1, 2), (0, 1)])
    assert np.array_equal(sub.Q[0, 0], full.Q[1, 2]) and np.array_equal(sub.K[0, 1], full.K[0, 1])
    assert np.array_equal(sub.V[0, 0], full.V[1, 2]) and np.array_equal(sub.dO[0, 1], full.dO[0, 1])
    assert np.array_equal(sub.M, full.M[[2, 1]]) and np.array_equal(sub.W, full.W)
    bat = inputs.generate(wl, pairs=[(0, 1), (1, 1)], as_batch=True)
    assert bat.Q.shape == (2, 1, 8, 4) and np.array_equal(bat.Q[1, 0], full.Q[1, 1])
    assert np.array_equal(bat.M, full.M[1:2])
    # bf16 workloads hold bf16-representable values
    assert np.array_equal(inputs.round_to_bf16(full.Q).astype(np.float64), full.Q)


def test_workload_statistics():
    wl = inputs.WORKLOADS["c1"]
    t = inputs.generate(wl)
    B, H, N, d, r, m, dv = wl.dims()
    assert t.Q.shape == (B, H, N, d) and t.M.shape == (H, r, d) and t.W.shape == (m, r)
    # trace of the query covariance is d, so the mean squared row norm is close to d
    assert abs((t.Q ** 2).sum(-1).mean() / d - 1.0) < 0.25
    np.testing.assert_allclose(t.M[0], np.eye(d), atol=0.1)
