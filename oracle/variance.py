"""Monte-Carlo variance of the importance-sampled positive-random-feature estimator (Section 3).

TEST INFRASTRUCTURE ONLY, like the rest of this package. Plain numpy, float64.

Section 3 studies the estimator of the softmax kernel exp(q.k) that draws its projections omega_j from a
proposal psi instead of N(0, I) and corrects each term by p_I(omega_j) / psi(omega_j) (Lemma 3.1), and shows
that for Gaussian inputs of covariance Lambda the expected variance is smallest for psi = N(0, Sigma*),
Sigma* = (I + 2 Lambda)(I - 2 Lambda)^-1 (Theorem 3.2). The functions below evaluate that estimator, its
per-term second moment in closed form for a Gaussian proposal, and the expectation of the variance over q, k.
"""
from __future__ import annotations

import numpy as np


def log_importance_factor(omega: np.ndarray, Sigma: np.ndarray) -> np.ndarray:
    """log( p_I(omega) / psi(omega) ) for psi = N(0, Sigma); omega [m, d]."""
    _, logdet = np.linalg.slogdet(Sigma)
    quad_i = np.einsum("md,md->m", omega, omega)
    quad_s = np.einsum("md,md->m", omega @ np.linalg.inv(Sigma), omega)
    return -0.5 * quad_i + 0.5 * quad_s + 0.5 * logdet


def prf_estimate(q: np.ndarray, k: np.ndarray, omega: np.ndarray, Sigma: np.ndarray) -> float:
    """The estimator of Lemma 3.1 with omega_j ~ N(0, Sigma): mean over j of
    (p_I / psi)(omega_j) exp(omega_j.q - |q|^2/2) exp(omega_j.k - |k|^2/2)."""
    lw = log_importance_factor(omega, Sigma)
    terms = np.exp(lw + omega @ (q + k) - 0.5 * (q @ q) - 0.5 * (k @ k))
    return float(terms.mean())


def term_second_moment(q: np.ndarray, k: np.ndarray, Sigma: np.ndarray) -> float:
    """E_psi of the squared single term of the estimator, in closed form for psi = N(0, Sigma):
    with s = q + k and A = 2 I - Sigma^-1 (which must be positive definite),
    sqrt(det Sigma / det A) exp(2 s^T A^-1 s - |q|^2 - |k|^2). For Sigma = I this is the textbook
    exp(2 |q + k|^2 - |q|^2 - |k|^2)."""
    d = q.shape[0]
    A = 2.0 * np.eye(d) - np.linalg.inv(Sigma)
    if np.linalg.eigvalsh(A).min() <= 0.0:
        return float("inf")
    s = q + k
    _, ld_s = np.linalg.slogdet(Sigma)
    _, ld_a = np.linalg.slogdet(A)
    return float(np.exp(0.5 * (ld_s - ld_a) + 2.0 * s @ np.linalg.solve(A, s) - q @ q - k @ k))


def term_variance(q: np.ndarray, k: np.ndarray, Sigma: np.ndarray) -> float:
    """Variance of one term; the estimator with m independent projections has this divided by m."""
    return term_second_moment(q, k, Sigma) - float(np.exp(2.0 * (q @ k)))


def expected_term_variance(Lambda: np.ndarray, Sigma: np.ndarray, pairs: int, rng: np.random.Generator) -> float:
    """Average of term_variance over `pairs` draws q, k ~ N(0, Lambda) (the quantity Theorem 3.2 compares)."""
    L = np.linalg.cholesky(Lambda)
    d = Lambda.shape[0]
    total = 0.0
    for _ in range(pairs):
        q, k = L @ rng.standard_normal(d), L @ rng.standard_normal(d)
        total += term_variance(q, k, Sigma)
    return total / pairs
