"""Host-side inputs of the library, computed from a noise schedule or an energy: the per-transition
coefficients (a_k, c_k, sigma_k) of the affine transition means, the per-step scalars of the mixture
denoiser, the deterministic sampler the Picard drafter iterates, and an orthonormal basis for the
projected accept test. These are caller inputs of the C ABI (sds_schedule, sds_set_projection); the
library copies them and never recomputes them. NumPy only, no device work.
"""
from __future__ import annotations

import math

import numpy as np


def ddpm_schedule(beta: np.ndarray):
    """Ancestral-sampler coefficients for an x0-predicting denoiser. Transition k moves noise level
    t = K - k to t - 1: mean = a_k x_t + c_k x0_hat, std = sqrt(beta_t). Returns float32 (a, c, sigma)
    and float64 abar[k] = abar_{K-k}."""
    beta = np.asarray(beta, dtype=np.float64)
    K = len(beta)
    abar_full = np.concatenate([[1.0], np.cumprod(1.0 - beta)])
    t = K - np.arange(K)
    ab_t, ab_p, b_t = abar_full[t], abar_full[t - 1], beta[t - 1]
    a = np.sqrt(1.0 - b_t) * (1.0 - ab_p) / (1.0 - ab_t)
    c = np.sqrt(ab_p) * b_t / (1.0 - ab_t)
    return a.astype(np.float32), c.astype(np.float32), np.sqrt(b_t).astype(np.float32), ab_t


def ddim_schedule(beta: np.ndarray):
    """Coefficients (a_det, c_det) of the deterministic counterpart of ddpm_schedule, the sampler the
    Picard drafter iterates: x_{t-1} = sqrt(abar_{t-1}) D + sqrt(1 - abar_{t-1}) (x_t - sqrt(abar_t) D)/sqrt(1 - abar_t)."""
    beta = np.asarray(beta, dtype=np.float64)
    K = len(beta)
    abar_full = np.concatenate([[1.0], np.cumprod(1.0 - beta)])
    t = K - np.arange(K)
    ab_t, ab_p = abar_full[t], abar_full[t - 1]
    a_det = np.sqrt((1.0 - ab_p) / (1.0 - ab_t))
    c_det = np.sqrt(ab_p) - a_det * np.sqrt(ab_t)
    return a_det.astype(np.float32), c_det.astype(np.float32)


def gmm_tcond_posterior_mean(abar: np.ndarray, comp_std: float) -> np.ndarray:
    """(A, Bq, C, E) per step for E[x0 | x_t] of a mixture with shared std s under x_t = al x0 + sqrt(1-al^2) eps:
    v = al^2 s^2 + 1 - al^2;  A = al/v, Bq = -al^2/(2v), C = (1-al^2)/v, E = al s^2/v."""
    abar = np.asarray(abar, dtype=np.float64)
    al = np.sqrt(abar)
    v = abar * comp_std ** 2 + 1.0 - abar
    return np.stack([al / v, -abar / (2 * v), (1.0 - abar) / v, al * comp_std ** 2 / v], axis=1)


def ula_schedule(K: int, gamma: float):
    """Unadjusted Langevin: mean = x - gamma grad E(x), std = sqrt(2 gamma)."""
    return (np.ones(K, np.float32), np.full(K, -gamma, np.float32), np.full(K, math.sqrt(2 * gamma), np.float32))


def gmm_tcond_grad_energy(K: int, comp_std: float) -> np.ndarray:
    """(A, Bq, C, E) for grad E of E = -log sum_c w_c N(x; mu_c, s^2 I): (1/s^2, -1/(2 s^2), -1/s^2, 1/s^2)."""
    s2 = comp_std ** 2
    return np.tile(np.array([1 / s2, -0.5 / s2, -1 / s2, 1 / s2], dtype=np.float64), (K, 1))


def projection_basis(A: np.ndarray, rtol: float = 1e-10) -> np.ndarray:
    """Orthonormal rows [r, d] spanning the row space of A (from its singular value decomposition),
    the form sds_set_projection takes: Q^T Q = A^+ A."""
    A = np.atleast_2d(np.asarray(A, dtype=np.float64))
    _, sv, Vt = np.linalg.svd(A, full_matrices=False)
    r = int(np.sum(sv > rtol * sv.max())) if sv.size else 0
    return np.ascontiguousarray(Vt[:r], dtype=np.float32)
