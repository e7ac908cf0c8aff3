"""CPU oracle for the draft-then-verify window of speculative sampling for diffusion models
(arxiv 2501.05370). TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by
the benchmark's CPU-baseline leg; the product path never calls it.

Plain, slow, fp64 NumPy, one chain at a time, the paper's steps in the paper's order and
notation (draft density p, target density q). It shares no code with the CUDA path.

What each function follows:
  philox4x32_10 / uniform01 / normals  counter-based generator (published Philox-4x32-10 definition)
  ddpm_affine, ula_affine              transition mean written as a_k*y + c_k*D, std sigma_k
                                       (Eq. 3 target transition; Langevin Eq. 13)
  gmm_posterior_mean, gmm_grad_energy  exact denoiser / score of a Gaussian mixture (Tweedie)
  mlp_forward                          bf16-operand MLP denoiser
  phi4_energy, phi4_grad_energy        the lattice energy of the Langevin experiment (Appendix K)
  rejection_discrete                   Algorithm 2 (generic maximal coupling), finite space
  rejection_reflection                 Algorithm 3 (reflection maximal coupling)
  rejection_incorrect                  the biased rule of Appendix "need for adjusted rejection"
  log_ratio                            log of the acceptance ratio, both printed forms
  verify_window                        the accept/reflect loop of Algorithm 4 on given arrays
  rejection_reflection_projected       the rule of Appendix F for a matrix A, in the original space
  ddim_affine, picard_trajectory       deterministic sampler and its Picard iterates (Appendix C)
  speculative_chain                    Algorithm 4 (detailed speculative sampling for DDM) and
                                       Algorithm 5 (Langevin) through the affine form
  plain_chain                          the target chain itself (Eq. 3), no speculation

Pins (tests/test_oracle_*.py): Philox known-answer vectors; acceptance frequency against the
closed form 2 - 2*Phi(|m^p - m^q| / (2 sigma)) (Proposition 2) on the two worked Gaussian pairs
the paper draws; output law of the reflection step by KS at d = 1, 2 (and the incorrect rule
failing it); the discrete worked example; E[log a] = -|Delta|^2/2; mean window advance against
the geometric sum; speculative vs plain chain in law; mixture denoiser against brute force and
finite differences; DDPM coefficient identities; the projected rule against Algorithm 3 (invertible
matrix), the whitened-image identity and the image's law; the Picard iterates against the sequential
deterministic chain, window 1 against the plain chain, and the chain's law.
Parity unpinned: agreement of the NFE counters with the paper's tables (the paper does not say
which frozen-drafter variant or call count produced them).
"""
from __future__ import annotations

import math

import numpy as np

# ----------------------------------------------------------------------------------------
# Philox-4x32-10 (Salmon et al., SC'11), counters -> 4 x uint32
# ----------------------------------------------------------------------------------------

_M0 = np.uint64(0xD2511F53)
_M1 = np.uint64(0xCD9E8D57)
_W0 = 0x9E3779B9
_W1 = 0xBB67AE85
_MASK = np.uint64(0xFFFFFFFF)
_SH = np.uint64(32)

STREAM_DRAFT = 0      # draft noise xi_{b,k}
STREAM_ACCEPT = 1     # accept uniform U_{b,k}
STREAM_INIT = 2       # initial state Y_0


def philox4x32_10(c0, c1, c2, c3, k0, k1):
    """Ten Philox rounds on arrays (or scalars) of 32-bit counter words; returns 4 uint32 arrays."""
    c0 = np.asarray(c0, dtype=np.uint64) & _MASK
    c1 = np.asarray(c1, dtype=np.uint64) & _MASK
    c2 = np.asarray(c2, dtype=np.uint64) & _MASK
    c3 = np.asarray(c3, dtype=np.uint64) & _MASK
    c0, c1, c2, c3 = np.broadcast_arrays(c0, c1, c2, c3)
    k0 = int(k0) & 0xFFFFFFFF
    k1 = int(k1) & 0xFFFFFFFF
    for _ in range(10):
        p0 = _M0 * c0                      # 32x32 -> 64
        p1 = _M1 * c2
        hi0, lo0 = p0 >> _SH, p0 & _MASK
        hi1, lo1 = p1 >> _SH, p1 & _MASK
        c0, c1, c2, c3 = (hi1 ^ c1 ^ np.uint64(k0)), lo1, (hi0 ^ c3 ^ np.uint64(k1)), lo0
        k0 = (k0 + _W0) & 0xFFFFFFFF
        k1 = (k1 + _W1) & 0xFFFFFFFF
    return (c0.astype(np.uint32), c1.astype(np.uint32), c2.astype(np.uint32), c3.astype(np.uint32))


def _counter(q, k, b, stream):
    """Counter words (q, k, b_lo, stream + 256*b_hi): q = element index // 4 (0 for the uniform),
    k = absolute transition index, b = global chain id."""
    b = int(b)
    return q, int(k), b & 0xFFFFFFFF, (int(stream) + 256 * (b >> 32)) & 0xFFFFFFFF


def uniform01(seed: int, b: int, k: int) -> float:
    """U_{b,k} in (0, 1]: ((x >> 8) + 1) * 2^-24 from word 0 of the accept stream."""
    c = _counter(0, k, b, STREAM_ACCEPT)
    x0, _, _, _ = philox4x32_10(*c, seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF)
    return (float(int(x0) >> 8) + 1.0) * 2.0 ** -24


def normals(seed: int, stream: int, b: int, k: int, d: int) -> np.ndarray:
    """d standard normals for (chain b, step k): Box-Muller on the word pairs (x0,x1), (x2,x3) of
    the block q = i // 4; both uniforms use 24 bits so that they are exact in single precision:
    u1 = ((x_even >> 8) + 1) 2^-24 in (0,1], u2 = (x_odd >> 8) 2^-24 in [0,1)."""
    nq = (d + 3) // 4
    q = np.arange(nq, dtype=np.uint64)
    c = _counter(q, k, b, stream)
    x = philox4x32_10(*c, seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF)
    z = np.empty((nq, 4), dtype=np.float64)
    for pair in range(2):
        xe = x[2 * pair].astype(np.float64)
        xo = x[2 * pair + 1].astype(np.float64)
        u1 = (np.floor(xe / 256.0) + 1.0) * 2.0 ** -24
        u2 = np.floor(xo / 256.0) * 2.0 ** -24
        r = np.sqrt(-2.0 * np.log(u1))
        z[:, 2 * pair] = r * np.cos(2.0 * math.pi * u2)
        z[:, 2 * pair + 1] = r * np.sin(2.0 * math.pi * u2)
    return z.reshape(-1)[:d]


# ----------------------------------------------------------------------------------------
# transition coefficients: mean m_k(y, D) = a_k*y + c_k*D, std sigma_k
# ----------------------------------------------------------------------------------------


def ddpm_affine(beta: np.ndarray):
    """Ancestral DDPM posterior written for an x0-predicting denoiser D.

    Transition k (k = 0..K-1) goes from noise level t = K-k to t-1. With alpha_t = 1-beta_t,
    abar_t = prod alpha, abar_0 = 1:
        a_k = sqrt(alpha_t) (1 - abar_{t-1}) / (1 - abar_t)
        c_k = sqrt(abar_{t-1}) beta_t / (1 - abar_t)
        sigma_k = sqrt(beta_t)                      (noise kept at every step, also the last)
    Returns (a, c, sigma, abar_at_step) with abar_at_step[k] = abar_{K-k} (what D is conditioned on).
    The target transition N(m^q_k, sigma_k^2 I) is the paper's Eq. 3 with this mean.
    """
    beta = np.asarray(beta, dtype=np.float64)
    K = beta.shape[0]
    alpha = 1.0 - beta
    abar = np.concatenate([[1.0], np.cumprod(alpha)])        # abar[t], t = 0..K
    a = np.empty(K)
    c = np.empty(K)
    sig = np.empty(K)
    abar_step = np.empty(K)
    for k in range(K):
        t = K - k
        a[k] = math.sqrt(alpha[t - 1]) * (1.0 - abar[t - 1]) / (1.0 - abar[t])
        c[k] = math.sqrt(abar[t - 1]) * beta[t - 1] / (1.0 - abar[t])
        sig[k] = math.sqrt(beta[t - 1])
        abar_step[k] = abar[t]
    return a, c, sig, abar_step


def ddim_affine(beta: np.ndarray):
    """Deterministic counterpart of ddpm_affine (the sampler without noise the Picard drafter
    iterates, Appendix C "parallel sampling"): with the denoiser output D read as x0 and the noise
    direction (x_t - sqrt(abar_t) D)/sqrt(1 - abar_t) kept,
        x_{t-1} = sqrt(abar_{t-1}) D + sqrt(1 - abar_{t-1}) (x_t - sqrt(abar_t) D)/sqrt(1 - abar_t)
                = abar_det_k x_t + cbar_det_k D,
        abar_det_k = sqrt((1 - abar_{t-1})/(1 - abar_t)),  cbar_det_k = sqrt(abar_{t-1}) - abar_det_k sqrt(abar_t),
    t = K - k. Returns (a_det, c_det)."""
    beta = np.asarray(beta, dtype=np.float64)
    K = beta.shape[0]
    abar = np.concatenate([[1.0], np.cumprod(1.0 - beta)])
    a_det = np.empty(K)
    c_det = np.empty(K)
    for k in range(K):
        t = K - k
        a_det[k] = math.sqrt((1.0 - abar[t - 1]) / (1.0 - abar[t]))
        c_det[k] = math.sqrt(abar[t - 1]) - a_det[k] * math.sqrt(abar[t])
    return a_det, c_det


def ula_affine(K: int, gamma: float):
    """Unadjusted Langevin X_{k+1} = X_k - gamma grad E(X_k) + sqrt(2 gamma) W_k (Eq. 13):
    a = 1, c = -gamma, sigma = sqrt(2 gamma), D = grad E."""
    return np.ones(K), np.full(K, -gamma), np.full(K, math.sqrt(2.0 * gamma))


# ----------------------------------------------------------------------------------------
# denoisers
# ----------------------------------------------------------------------------------------


def bf16_round(x: np.ndarray) -> np.ndarray:
    """Round to the nearest bfloat16 (ties to even), returned in float64."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + np.uint64(0x7FFF) + ((u >> np.uint64(16)) & np.uint64(1))) >> np.uint64(16)
    return (u.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def _log_softmax_weights(logit: np.ndarray) -> np.ndarray:
    m = np.max(logit)
    e = np.exp(logit - m)
    return e / np.sum(e)


def gmm_posterior_mean(x, abar_t, means, logw, s, bf16_operands=False):
    """E[x_0 | x_t = x] for x_0 ~ sum_c w_c N(mu_c, s^2 I), x_t = sqrt(abar) x_0 + sqrt(1-abar) eps.

    Written from the definition: x_t | c ~ N(alpha mu_c, v I), v = alpha^2 s^2 + 1 - alpha^2;
    responsibilities r_c ~ w_c N(x; alpha mu_c, v I); within a component x_0 | x_t, c has mean
    mu_c + (alpha s^2 / v)(x - alpha mu_c).
    bf16_operands: the inner products x.mu_c and the mixing sum_c r_c mu_c take x, mu, r rounded
    to bfloat16 (the large-component tensor-core setting); everything else stays in double.
    """
    x = np.asarray(x, dtype=np.float64)
    mu = np.asarray(means, dtype=np.float64)
    al = math.sqrt(abar_t)
    v = al * al * s * s + 1.0 - al * al
    if not bf16_operands:
        diff = x[None, :] - al * mu
        logit = np.asarray(logw, dtype=np.float64) - 0.5 * np.sum(diff * diff, axis=1) / v
        r = _log_softmax_weights(logit)
        comp_mean = mu + (al * s * s / v) * diff
        return r @ comp_mean
    xb = bf16_round(x)
    mub = bf16_round(mu)
    # |x - al mu|^2 = |x|^2 - 2 al x.mu + al^2 |mu|^2 ; |x|^2 is common to all components
    logit = np.asarray(logw, dtype=np.float64) + (al / v) * (mub @ xb) - 0.5 * al * al * np.sum(mub * mub, axis=1) / v
    r = _log_softmax_weights(logit)
    rb = bf16_round(r)
    mix = rb @ mub
    # sum_c r_c (mu_c + g (x - al mu_c)) with g = al s^2 / v and sum r = 1
    g = al * s * s / v
    return (1.0 - al * g) * mix + g * x


def gmm_grad_energy(x, means, logw, s):
    """grad E(x) for E = -log sum_c w_c N(x; mu_c, s^2 I): sum_c r_c (x - mu_c) / s^2."""
    x = np.asarray(x, dtype=np.float64)
    mu = np.asarray(means, dtype=np.float64)
    diff = x[None, :] - mu
    logit = np.asarray(logw, dtype=np.float64) - 0.5 * np.sum(diff * diff, axis=1) / (s * s)
    r = _log_softmax_weights(logit)
    return (r @ diff) / (s * s)


def phi4_energy(x, side, beta, periodic=False):
    """E(x) = beta/2 sum_{|i-j|=1} (x_i - x_j)^2 + sum_i (x_i^2 - 1)^2 on a side x side grid
    (Appendix K; each neighbouring pair counted once; free boundaries unless periodic)."""
    g = np.asarray(x, dtype=np.float64).reshape(side, side)
    e = np.sum((g * g - 1.0) ** 2)
    for axis in (0, 1):
        if periodic:
            dif = g - np.roll(g, -1, axis=axis)
        else:
            dif = np.diff(g, axis=axis)
        e += 0.5 * beta * np.sum(dif * dif)
    return float(e)


def phi4_grad_energy(x, side, beta, periodic=False):
    """Gradient of phi4_energy: beta * sum over neighbours (x_i - x_j) + 4 x_i (x_i^2 - 1)."""
    g = np.asarray(x, dtype=np.float64).reshape(side, side)
    grad = 4.0 * g * (g * g - 1.0)
    for axis in (0, 1):
        if periodic:
            grad += beta * (2.0 * g - np.roll(g, 1, axis=axis) - np.roll(g, -1, axis=axis))
        else:
            fwd = np.zeros_like(g)
            bwd = np.zeros_like(g)
            sl_a = [slice(None)] * 2
            sl_b = [slice(None)] * 2
            sl_a[axis] = slice(0, -1)
            sl_b[axis] = slice(1, None)
            fwd[tuple(sl_a)] = g[tuple(sl_a)] - g[tuple(sl_b)]      # pair (i, i+1) seen from i
            bwd[tuple(sl_b)] = g[tuple(sl_b)] - g[tuple(sl_a)]      # same pair seen from i+1
            grad += beta * (fwd + bwd)
    return grad.reshape(-1)


def silu(x):
    return x / (1.0 + np.exp(-x))


def mlp_forward(x, k, weights, bias, temb):
    """bf16-operand MLP: h_l = SiLU(W_l h_{l-1} + b_l + E_l[k]) for hidden layers, last layer linear.
    weights[l], temb[l][k] are bfloat16-representable values; the input and every stored hidden
    activation are rounded to bfloat16; sums, bias/embedding add and SiLU are in double."""
    h = bf16_round(np.asarray(x, dtype=np.float64))
    nl = len(weights)
    for l in range(nl):
        y = np.asarray(weights[l], dtype=np.float64) @ h + np.asarray(bias[l], dtype=np.float64)
        if l < nl - 1:
            y = y + np.asarray(temb[l][k], dtype=np.float64)
            h = bf16_round(silu(y))
        else:
            h = y
    return h


# ----------------------------------------------------------------------------------------
# rejection mechanisms
# ----------------------------------------------------------------------------------------


def rejection_discrete(p: np.ndarray, q: np.ndarray, x_tilde: int, rng: np.random.Generator):
    """Algorithm 2 on a finite space: accept x_tilde ~ p w.p. min(1, q/p); else draw from
    r ~ max(0, q - p)."""
    u = rng.random()
    if u <= min(1.0, q[x_tilde] / p[x_tilde]):
        return x_tilde, True
    r = np.maximum(0.0, q - p)
    r = r / r.sum()
    return int(rng.choice(len(q), p=r)), False


def rejection_incorrect_discrete(p, q, x_tilde, rng):
    """The biased variant: on rejection draw from q itself (kept only to show the law test fails)."""
    u = rng.random()
    if u <= min(1.0, q[x_tilde] / p[x_tilde]):
        return x_tilde, True
    return int(rng.choice(len(q), p=q)), False


def log_ratio(Z: np.ndarray, Delta: np.ndarray) -> float:
    """log[N(Z + Delta; 0, I) / N(Z; 0, I)] = -|Z + Delta|^2/2 + |Z|^2/2 (Appendix F)."""
    return float(-0.5 * np.dot(Z + Delta, Z + Delta) + 0.5 * np.dot(Z, Z))


def log_ratio_expanded(Z: np.ndarray, Delta: np.ndarray) -> float:
    """The same quantity as -(Delta + 2 Z).Delta / 2 (Algorithm 8 with A = I)."""
    return float(-0.5 * np.dot(Delta + 2.0 * Z, Delta))


def rejection_reflection(m_p, m_q, sigma, y_tilde, U, tau=1.0):
    """Algorithm 3: reflection maximal coupling of N(m^p, sigma^2 I) and N(m^q, sigma^2 I).
    Returns (Y, accept, log_ratio). Delta = 0 accepts (ratio 1; e is never needed).
    tau != 1 is the temperature variant (Algorithm 6): the accept test compares U with
    N(Z + Delta; 0, tau I) / N(Z; 0, tau I) = ratio^(1/tau); the reflection is unchanged and the
    output law is no longer exactly the target's. The returned log ratio is the tempered one."""
    m_p = np.asarray(m_p, dtype=np.float64)
    m_q = np.asarray(m_q, dtype=np.float64)
    y_tilde = np.asarray(y_tilde, dtype=np.float64)
    Delta = (m_p - m_q) / sigma
    Z = (y_tilde - m_p) / sigma
    ell = log_ratio_expanded(Z, Delta) / tau
    nrm2 = float(np.dot(Delta, Delta))
    accept = (nrm2 < 1e-30) or (math.log(U) <= min(0.0, ell))
    if accept:
        return y_tilde.copy(), True, ell
    e = Delta / math.sqrt(nrm2)
    Y = m_q + sigma * (Z - 2.0 * e * np.dot(e, Z))
    return Y, False, ell


def rejection_reflection_projected(m_p, m_q, sigma, y_tilde, U, A):
    """Reflection coupling decided in the image of a matrix A, written in the original space
    (Appendix F, the algorithm for a full matrix A): with P = A^+ A (the orthogonal projector onto
    the row space of A), accept iff U <= min(1, exp(-(Delta + 2 Z)^T P Delta / 2)); a rejected draft
    becomes m^q + sigma (Z - 2 (Z^T P Delta)/(Delta^T P Delta) Delta). For invertible A, P = I and
    this is Algorithm 3; otherwise the output law is not the target's, but (A Y~, A Y) are maximally
    coupled. Returns (Y, accept, log_ratio). P Delta = 0 accepts."""
    m_p = np.asarray(m_p, dtype=np.float64)
    m_q = np.asarray(m_q, dtype=np.float64)
    y_tilde = np.asarray(y_tilde, dtype=np.float64)
    A = np.atleast_2d(np.asarray(A, dtype=np.float64))
    P = np.linalg.pinv(A) @ A
    Delta = (m_p - m_q) / sigma
    Z = (y_tilde - m_p) / sigma
    PD = P @ Delta
    ell = -0.5 * float(np.dot(Delta + 2.0 * Z, PD))
    dPd = float(np.dot(Delta, PD))
    accept = (dPd < 1e-30) or (math.log(U) <= min(0.0, ell))
    if accept:
        return y_tilde.copy(), True, ell
    Y = m_q + sigma * (Z - 2.0 * (float(np.dot(Z, PD)) / dPd) * Delta)
    return Y, False, ell


def rejection_incorrect_gaussian(m_p, m_q, sigma, y_tilde, U, fresh_normal):
    """Same accept test, but on rejection a fresh draw from N(m^q, sigma^2 I) (biased)."""
    Y, acc, ell = rejection_reflection(m_p, m_q, sigma, y_tilde, U)
    if acc:
        return Y, True, ell
    return np.asarray(m_q, dtype=np.float64) + sigma * np.asarray(fresh_normal, dtype=np.float64), False, ell


# ----------------------------------------------------------------------------------------
# the window
# ----------------------------------------------------------------------------------------


def verify_window(W, Dq, D_c, a, c, sigma, n, logU, decide_f32=True, tau=1.0, proj=None, M_p=None):
    """The verification loop of Algorithm 4 for one chain on given arrays.

    W   [Lt+1, d]  W[0] = Y_n, W[j] = drafted state for transition k = n+j-1
    Dq  [Lt, d]    target denoiser outputs, Dq[j-1] = D(W[j-1], k)
    D_c [d]        the frozen (carried) denoiser output the drafter used, or [Lt, d]: the draft
                   model's own output per position (independent drafter)
    logU[Lt]       log of the accept uniforms
    Draft mean m^p = a_k W[j-1] + c_k D_c, target mean m^q = a_k W[j-1] + c_k Dq[j-1].
    decide_f32: compare log U and the log-ratio after rounding both to single precision
    (the precision in which the GPU path stores and compares them).
    M_p [Lt, d]    explicit draft means (drafters whose mean is not a_k W[j-1] + c_k D, such as the
                   Picard drafter); D_c is then ignored
    proj: a matrix A [r, d]; the test and the reflection coefficient then use P = A^+ A as in
    rejection_reflection_projected, and S1 = Delta^T P Delta, S2 = Z^T P Delta.
    Returns dict(S1, S2, ell, acc, jstar, Y_reflect) with jstar in 1..Lt+1 (Lt+1 = all accepted).
    """
    W = np.asarray(W, dtype=np.float64)
    Dq = np.asarray(Dq, dtype=np.float64)
    Lt = Dq.shape[0]
    D_c = np.zeros(Dq.shape[1]) if D_c is None else np.asarray(D_c, dtype=np.float64)
    if D_c.ndim == 1:                      # frozen drafter: one output for the whole window
        D_c = np.broadcast_to(D_c, Dq.shape)
    S1 = np.zeros(Lt)
    S2 = np.zeros(Lt)
    ell = np.zeros(Lt)
    acc = np.zeros(Lt, dtype=bool)
    jstar = Lt + 1
    Y_reflect = None
    P = None
    if proj is not None:
        Amat = np.atleast_2d(np.asarray(proj, dtype=np.float64))
        P = np.linalg.pinv(Amat) @ Amat
    for j in range(1, Lt + 1):
        k = n + j - 1
        m_p = a[k] * W[j - 1] + c[k] * D_c[j - 1] if M_p is None else np.asarray(M_p[j - 1], dtype=np.float64)
        m_q = a[k] * W[j - 1] + c[k] * Dq[j - 1]
        Delta = (m_p - m_q) / sigma[k]
        Z = (W[j] - m_p) / sigma[k]
        if P is not None:                                        # ratio decided in the image of A
            PD = P @ Delta
            S1[j - 1] = np.dot(Delta, PD)
            S2[j - 1] = np.dot(Z, PD)
            ell[j - 1] = -0.5 * np.dot(Delta + 2.0 * Z, PD) / tau
            if decide_f32:
                ok = np.float32(logU[j - 1]) <= np.float32(ell[j - 1])
            else:
                ok = logU[j - 1] <= ell[j - 1]
            acc[j - 1] = bool(ok) or S1[j - 1] < 1e-30
            if not acc[j - 1] and jstar == Lt + 1:
                jstar = j
                Y_reflect = m_q + sigma[k] * (Z - 2.0 * (S2[j - 1] / S1[j - 1]) * Delta)
            continue
        S1[j - 1] = np.dot(Delta, Delta)
        S2[j - 1] = np.dot(Delta, Z)
        ell[j - 1] = log_ratio_expanded(Z, Delta) / tau          # tau = 1: the exact method
        if decide_f32:
            ok = np.float32(logU[j - 1]) <= np.float32(ell[j - 1])
        else:
            ok = logU[j - 1] <= ell[j - 1]
        acc[j - 1] = bool(ok) or S1[j - 1] < 1e-30
        if not acc[j - 1] and jstar == Lt + 1:
            jstar = j
            e = Delta / math.sqrt(S1[j - 1])
            Y_reflect = m_q + sigma[k] * (Z - 2.0 * e * np.dot(e, Z))
    return dict(S1=S1, S2=S2, ell=ell, acc=acc, jstar=jstar, Y_reflect=Y_reflect)


FROZEN_PREV = 0     # carry the latest target output on the accepted trajectory (no extra call)
FROZEN_EXACT = 1    # evaluate the target at Y_n before drafting (main-text frozen drafter)
INDEPENDENT = 2     # a second, cheaper model proposes every draft step (Eq. 5)
PICARD = 3          # draft means from Picard iterations of the deterministic sampler (Appendix C)


def picard_trajectory(denoise, a_det, c_det, Y, D_c, n, Lt, iters):
    """Picard iterates of the deterministic sampler over one window (Appendix C, parallel sampling
    as drafting). Points F_0 .. F_{Lt-1}, F_0 = Y_n throughout. Start: the deterministic rollout
    with the carried output frozen, F^0_{j+1} = a_det F^0_j + c_det D_c (the paper leaves the
    deterministic start free). Each iteration evaluates the target at all points of the previous
    iterate in one batch and shifts: F^m_{j+1} = a_det_k F^{m-1}_j + c_det_k D(F^{m-1}_j, k),
    k = n + j. After m iterations the first m+1 points equal the sequential deterministic chain.
    Returns F [Lt, d]."""
    Y = np.asarray(Y, dtype=np.float64)
    F = np.empty((Lt, Y.shape[0]))
    F[0] = Y
    for j in range(Lt - 1):
        F[j + 1] = a_det[n + j] * F[j] + c_det[n + j] * D_c
    for _ in range(iters):
        D = [denoise(F[j], n + j) for j in range(Lt - 1)]          # one batched target call
        Fn = F.copy()
        for j in range(Lt - 1):
            Fn[j + 1] = a_det[n + j] * F[j] + c_det[n + j] * D[j]
        F = Fn
    return F


def speculative_chain(denoise, a, c, sigma, L, seed, b, d, mode=FROZEN_PREV, Y0=None,
                      record=False, decide_f32=True, draft_denoise=None, tau=1.0, proj=None, picard=None, stage=None):
    """Algorithm 4 for chain b with the frozen-target drafter, or (mode INDEPENDENT) with the draft
    model draft_denoise(x, k): m^p_k(y) = a_k y + c_k D^p(y, k) evaluated at every drafted state.

    mode PICARD with picard = (p, a_det, c_det): p >= 1 parallel target calls per window build the
    draft. p - 1 Picard iterations (picard_trajectory) give points F_0..F_{Lt-1}; the last call
    evaluates the target there and the draft mean of position j is the stochastic sampler's step
    from F_{j-1}: m^p_j = a_k F_{j-1} + c_k D(F_{j-1}, k), k = n+j-1, independent of the earlier
    drafted states. Since F_0 = Y_n, position 1 is drafted from the target itself and its target
    output is already known; the verify call evaluates positions 2..Lt. The carried output (start
    of the next window's Picard sequence) follows the FROZEN_PREV rule.

    stage (FROZEN_PREV only; None = the algorithm as printed): the window of Algorithm 4 evaluated lazily, at
    most `stage` positions per target call. The accept tests of a window use only the window's frozen output,
    the drafted states and the draws keyed by (chain, step), so a window whose first `stage` positions were all
    accepted can draft, evaluate and test its next positions afterwards with the same frozen output: the same
    states and decisions as the one batched call, fewer rows evaluated after a rejection (nfe_rows), one more
    sequential call for each stage passed (nfe_calls). `adv` then lists the advance of each call.

    denoise(x, k) -> D; transition means are a_k y + c_k D, std sigma_k.
    Returns dict(Y, nfe_calls, nfe_rows, adv (list), windows (list of per-window records if record)).
    """
    if stage is not None and (mode != FROZEN_PREV or stage < 1):
        raise ValueError("staged evaluation is defined for the carried-output drafter")
    K = len(a)
    Y = normals(seed, STREAM_INIT, b, 0, d) if Y0 is None else np.asarray(Y0, dtype=np.float64).copy()
    n = 0
    nfe_calls = 0
    nfe_rows = 0
    D_c = None
    if mode in (FROZEN_PREV, PICARD):
        D_c = denoise(Y, 0)               # the one initial call
        nfe_calls += 1
        nfe_rows += 1
    advs = []
    windows = []
    left = 0                               # staged evaluation: positions of the current window not yet tested
    while n < K:
        Lt = min(L, K - n)
        if stage is not None:
            if left == 0:
                left = Lt                  # a new window
            Lt = min(left, stage)
        W = np.empty((Lt + 1, d))
        W[0] = Y
        Dq = np.empty((Lt, d))
        first = 1
        if mode == FROZEN_EXACT:
            D_c = denoise(Y, n)           # frozen output at (Y_n, t_n); it is also row 1 of the batch
            Dq[0] = D_c
            nfe_calls += 1
            nfe_rows += 1
            first = 2
        xi = np.empty((Lt, d))
        Dp = np.empty((Lt, d)) if mode == INDEPENDENT else None
        Mp = None
        if mode == PICARD:
            p_calls, a_det, c_det = picard
            F = picard_trajectory(denoise, a_det, c_det, Y, D_c, n, Lt, p_calls - 1)
            if Lt >= 2:
                nfe_calls += p_calls - 1
                nfe_rows += (p_calls - 1) * (Lt - 1)
            Mp = np.empty((Lt, d))
            for j in range(1, Lt + 1):     # last parallel call: the target at every Picard point
                k = n + j - 1
                DF = denoise(F[j - 1], k)
                if j == 1:
                    Dq[0] = DF             # F_0 = Y_n = W_0: this is the target output of position 1
                Mp[j - 1] = a[k] * F[j - 1] + c[k] * DF
            nfe_calls += 1
            nfe_rows += Lt
            first = 2
        for j in range(1, Lt + 1):         # sequential draft
            k = n + j - 1
            xi[j - 1] = normals(seed, STREAM_DRAFT, b, k, d)
            if mode == PICARD:
                W[j] = Mp[j - 1] + sigma[k] * xi[j - 1]
            elif mode == INDEPENDENT:
                Dp[j - 1] = draft_denoise(W[j - 1], k)
                W[j] = a[k] * W[j - 1] + c[k] * Dp[j - 1] + sigma[k] * xi[j - 1]
            else:
                W[j] = a[k] * W[j - 1] + c[k] * D_c + sigma[k] * xi[j - 1]
        for j in range(first, Lt + 1):     # one batched target call on the drafted states
            Dq[j - 1] = denoise(W[j - 1], n + j - 1)
        if Lt >= first:
            nfe_calls += 1
            nfe_rows += Lt - first + 1
        logU = np.array([math.log(uniform01(seed, b, n + j - 1)) for j in range(1, Lt + 1)])
        v = verify_window(W, Dq, Dp if mode == INDEPENDENT else D_c, a, c, sigma, n, logU, decide_f32=decide_f32,
                          tau=tau, proj=proj, M_p=Mp)
        adv = min(v["jstar"], Lt)
        if v["jstar"] <= Lt:
            W[adv] = v["Y_reflect"]
        if record:
            windows.append(dict(n=n, W=W.copy(), Dq=Dq.copy(), D_c=(Dp if mode == INDEPENDENT else D_c).copy(),
                                logU=logU, xi=xi, M_p=None if Mp is None else Mp.copy(), **v))
        Y = W[adv].copy()
        if stage is not None and v["jstar"] > Lt and Lt < left:
            left -= Lt                     # every position of the stage accepted: the window goes on, output frozen
        else:
            left = 0
            D_c = Dq[adv - 1].copy()
        n += adv
        advs.append(adv)
    return dict(Y=Y, nfe_calls=nfe_calls, nfe_rows=nfe_rows, adv=advs, windows=windows)


def plain_chain(denoise, a, c, sigma, seed, b, d, Y0=None, stream=STREAM_DRAFT):
    """The target chain itself: Y_{k+1} = a_k Y_k + c_k D(Y_k, k) + sigma_k xi_k."""
    K = len(a)
    Y = normals(seed, STREAM_INIT, b, 0, d) if Y0 is None else np.asarray(Y0, dtype=np.float64).copy()
    for k in range(K):
        Y = a[k] * Y + c[k] * denoise(Y, k) + sigma[k] * normals(seed, stream, b, k, d)
    return Y


def expected_advance(alpha: float, L: int) -> float:
    """sum_{l<L} (l+1) alpha^l (1-alpha) + L alpha^L, the mean window advance when every draft is
    accepted independently with probability alpha (Section 4.1; summed form)."""
    return sum((l + 1) * alpha ** l * (1 - alpha) for l in range(L)) + L * alpha ** L
