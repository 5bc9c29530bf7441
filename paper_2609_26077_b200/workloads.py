"""Seeded synthetic operand generators (numpy only; none of the method's arithmetic).

The same host arrays feed the CUDA library and the CPU oracle in the tests.  Shapes,
value distributions and seeds follow the benchmark configurations: iid Gaussian and
signed-uniform operands (the families the paper's emulated sweep and covariance
diagnostic use), an activation-times-weight shaped pair with per-channel outliers,
and a wide-dynamic-range / heavy-tailed family that stresses the per-block scales.
"""
from __future__ import annotations

import numpy as np


def _rng(seed, stream):
    return np.random.default_rng([int(seed), int(stream)])


def gaussian(M, K, N, seed, sigma_a=1.0, sigma_b=1.0):
    """A, B iid N(0, sigma^2), fp32."""
    A = _rng(seed, 0).standard_normal((M, K), dtype=np.float32) * np.float32(sigma_a)
    B = _rng(seed, 1).standard_normal((K, N), dtype=np.float32) * np.float32(sigma_b)
    return A, B


def uniform(M, K, N, seed):
    """A, B iid U(-1, 1), fp32 (signed-uniform family)."""
    A = (_rng(seed, 0).random((M, K), dtype=np.float32) * np.float32(2) - np.float32(1))
    B = (_rng(seed, 1).random((K, N), dtype=np.float32) * np.float32(2) - np.float32(1))
    return A.astype(np.float32), B.astype(np.float32)


def llm_shaped(M, K, N, seed, outlier_sigma=1.5, weight_sigma=0.02):
    """Activation x weight: A[i,k] = z_ik * f_k with lognormal per-channel factors
    f_k = exp(outlier_sigma * g_k); B iid N(0, weight_sigma^2)."""
    z = _rng(seed, 0).standard_normal((M, K), dtype=np.float32)
    g = _rng(seed, 2).standard_normal(K).astype(np.float32)
    f = np.exp(np.float32(outlier_sigma) * g).astype(np.float32)
    A = (z * f[None, :]).astype(np.float32)
    B = _rng(seed, 1).standard_normal((K, N), dtype=np.float32) * np.float32(weight_sigma)
    return A, B


def llm_hetero_weights(M, K, N, seed, outlier_sigma=1.5, weight_sigma=0.02, col_sigma=1.0, row_sigma=0.5):
    """As llm_shaped, with a weight matrix whose output channels (columns) and input channels (rows) carry
    lognormal magnitude factors: the block-to-block heterogeneity that makes the weight-scale granularity
    (one scale per column block vs per 128 x 128 tile, App. E.5) matter.  Stand-in for stored checkpoint
    tiles, which are not available here."""
    A, B = llm_shaped(M, K, N, seed, outlier_sigma, weight_sigma)
    c = np.exp(np.float32(col_sigma) * _rng(seed, 3).standard_normal(N).astype(np.float32))
    r = np.exp(np.float32(row_sigma) * _rng(seed, 4).standard_normal(K).astype(np.float32))
    return A, (B * r[:, None] * c[None, :]).astype(np.float32)


def log_uniform_sigma(seed, stream, lo=-3.0, hi=3.0):
    return float(10.0 ** _rng(seed, stream).uniform(lo, hi))


def scaled_gaussian(M, K, N, seed):
    """N(0, sigma^2) with sigma = 10^u, u ~ U[-3, 3] drawn per trial, independently for A and B."""
    sa, sb = log_uniform_sigma(seed, 10), log_uniform_sigma(seed, 11)
    return gaussian(M, K, N, seed, sa, sb)


def student_t3(M, K, N, seed):
    """Mixed-sign heavy-tailed Student-t(nu=3) entries scaled by the log-uniform sigma law."""
    sa, sb = log_uniform_sigma(seed, 10), log_uniform_sigma(seed, 11)
    A = (_rng(seed, 0).standard_t(3.0, (M, K)) * sa).astype(np.float32)
    B = (_rng(seed, 1).standard_t(3.0, (K, N)) * sb).astype(np.float32)
    return A, B


def rademacher(M, K, N, seed, scale=1.0):
    """Entries +-scale with equal probability."""
    A = (_rng(seed, 0).integers(0, 2, (M, K)) * 2 - 1).astype(np.float32) * np.float32(scale)
    B = (_rng(seed, 1).integers(0, 2, (K, N)) * 2 - 1).astype(np.float32) * np.float32(scale)
    return A, B


def small_integers(M, K, N, seed, amp=8):
    """Integer-valued entries in [-amp, amp]: every fp32 +-1 combination is exact."""
    A = _rng(seed, 0).integers(-amp, amp + 1, (M, K)).astype(np.float32)
    B = _rng(seed, 1).integers(-amp, amp + 1, (K, N)).astype(np.float32)
    return A, B


def unit_uniform(M, K, N, seed):
    """iid U(-sqrt 3, sqrt 3): unit variance."""
    A, B = uniform(M, K, N, seed)
    r3 = np.float32(np.sqrt(3.0))
    return A * r3, B * r3


def unit_laplace(M, K, N, seed):
    """iid Laplace with unit variance (scale 1/sqrt 2)."""
    A = _rng(seed, 0).laplace(0.0, 1.0 / np.sqrt(2.0), (M, K)).astype(np.float32)
    B = _rng(seed, 1).laplace(0.0, 1.0 / np.sqrt(2.0), (K, N)).astype(np.float32)
    return A, B


def unit_t5(M, K, N, seed):
    """iid Student-t(nu = 5) scaled to unit variance (variance of t5 is 5/3)."""
    c = np.sqrt(3.0 / 5.0)
    A = (_rng(seed, 0).standard_t(5.0, (M, K)) * c).astype(np.float32)
    B = (_rng(seed, 1).standard_t(5.0, (K, N)) * c).astype(np.float32)
    return A, B


def rademacher10(M, K, N, seed):
    return rademacher(M, K, N, seed, scale=10.0)


FAMILIES = {
    "gaussian": gaussian,
    "uniform": uniform,
    "llm": llm_shaped,
    "llm_hetero": llm_hetero_weights,
    "scaled_gaussian": scaled_gaussian,
    "student_t3": student_t3,
    "rademacher": rademacher,
    "small_integers": small_integers,
    "unit_uniform": unit_uniform,
    "unit_laplace": unit_laplace,
    "unit_t5": unit_t5,
    "rademacher10": rademacher10,
}
