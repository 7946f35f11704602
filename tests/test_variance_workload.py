"""The second synthetic workload (orthogonal projection rows, variance-optimal sampling geometry) and the
Monte-Carlo variance harness of Section 3, on the CPU."""
import numpy as np
import pytest

from oracle import ref, variance
from paper_2603_04127_b200 import inputs


def test_orthogonal_rows_are_orthogonal_within_a_block_and_gaussian_in_norm():
    rng = np.random.default_rng(3)
    W = inputs.orthogonal_projection_rows(40, 16, rng)
    assert W.shape == (40, 16)
    for b in range(2):
        G = W[16 * b:16 * (b + 1)] @ W[16 * b:16 * (b + 1)].T
        assert np.abs(G - np.diag(np.diag(G))).max() < 1e-12
    # squared row norms are chi-square with 16 degrees of freedom: mean 16, variance 32
    n2 = np.concatenate([np.sum(inputs.orthogonal_projection_rows(64, 16, rng) ** 2, axis=1) for _ in range(200)])
    assert abs(n2.mean() - 16.0) < 0.2 and abs(n2.var() - 32.0) < 2.0


def test_optimal_proposal_is_isotropic_exactly_when_the_inputs_are():
    """Theorem 3.2, item 1, and the formula's domain."""
    assert np.allclose(inputs.optimal_proposal_spectrum(np.full(5, 0.1)), 1.2 / 0.8)
    s = inputs.optimal_proposal_spectrum(np.array([0.4, 0.1, 0.0]))
    assert np.allclose(s, [9.0, 1.5, 1.0]) and len(set(np.round(s, 12))) == 3
    with pytest.raises(ValueError):
        inputs.optimal_proposal_spectrum(np.array([0.5, 0.1]))
    rng = np.random.default_rng(5)
    U = inputs.random_orthogonal(4, rng)
    lam = np.array([0.3, 0.2, 0.1, 0.05])
    M = inputs.aligned_M(U, lam)
    Lambda = U @ np.diag(lam) @ U.T
    want = (np.eye(4) + 2 * Lambda) @ np.linalg.inv(np.eye(4) - 2 * Lambda)
    assert np.allclose(M.T @ M, want)


def test_importance_sampled_estimator_is_unbiased_and_matches_its_closed_form_variance():
    """Lemma 3.1's estimator with a Gaussian proposal: mean exp(q.k), per-term second moment as derived."""
    rng = np.random.default_rng(7)
    d = 3
    q, k = 0.5 * rng.standard_normal(d), 0.5 * rng.standard_normal(d)
    for Sigma in (np.eye(d), np.diag([1.6, 1.2, 1.0])):
        omega = rng.standard_normal((400000, d)) @ np.linalg.cholesky(Sigma).T
        lw = variance.log_importance_factor(omega, Sigma)
        terms = np.exp(lw + omega @ (q + k) - 0.5 * q @ q - 0.5 * k @ k)
        assert abs(terms.mean() - np.exp(q @ k)) < 5 * terms.std() / np.sqrt(len(terms))
        m2 = variance.term_second_moment(q, k, Sigma)
        assert abs((terms ** 2).mean() - m2) < 0.03 * m2
        assert abs(variance.prf_estimate(q, k, omega, Sigma) - terms.mean()) < 1e-12
    # Sigma = I: the textbook second moment of positive random features
    assert np.isclose(variance.term_second_moment(q, k, np.eye(d)), np.exp(2 * (q + k) @ (q + k) - q @ q - k @ k))


def test_data_aligned_proposal_has_the_smaller_expected_variance():
    """Theorem 3.2, item 2, numerically: for anisotropic Gaussian inputs the proposal N(0, Sigma*) beats N(0, I)."""
    rng = np.random.default_rng(11)
    d = 4
    U = inputs.random_orthogonal(d, rng)
    lam = np.array([0.30, 0.15, 0.05, 0.02])
    Lambda = U @ np.diag(lam) @ U.T
    Sigma_star = U @ np.diag(inputs.optimal_proposal_spectrum(lam)) @ U.T
    v_iso = variance.expected_term_variance(Lambda, np.eye(d), 4000, np.random.default_rng(12))
    v_opt = variance.expected_term_variance(Lambda, Sigma_star, 4000, np.random.default_rng(12))
    assert v_opt < v_iso
    # and a proposal stretched the wrong way is worse than the isotropic one
    Sigma_bad = U @ np.diag(inputs.optimal_proposal_spectrum(lam[::-1].copy())) @ U.T
    v_bad = variance.expected_term_variance(Lambda, Sigma_bad, 4000, np.random.default_rng(12))
    assert v_bad > v_opt


def test_hot_path_estimates_the_aligned_kernel_on_the_variance_workload():
    """The hot path on this workload (scale 1, M aligned, orthogonal W) is the random-feature attention of the
    kernel exp(q^T Sigma* k): its output approaches the exact kernel attention as the number of features grows."""
    err = {}
    for m in (1024, 16384):
        t = inputs.variance_workload(wid=21, B=1, H=1, N=24, d=4, m=m, lam_max=0.05, aligned=True, dtype="f32", backward=False)
        got = ref.forward(t.Q, t.K, t.V, t.M, t.W, causal=False, scale=1.0)[0, 0]
        q, k, v, M = t.Q[0, 0], t.K[0, 0], t.V[0, 0], t.M[0]
        A = np.exp(q @ (M.T @ M) @ k.T)
        want = (A / A.sum(axis=1, keepdims=True)) @ v
        err[m] = np.abs(got - want).max() / np.abs(want).max()
    assert err[1024] < 0.1 and err[16384] < 0.02 and err[16384] < err[1024] / 3
