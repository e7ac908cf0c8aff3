"""Seeded synthetic inputs for the speculative-sampling window (arxiv 2501.05370).

This module only *generates inputs*: noise-schedule tables (beta_t), Gaussian-mixture
parameters, random-init MLP weights and the five workload descriptions. It holds none of
the sampler's arithmetic (no transition means, no denoiser, no accept test), so both the
CPU oracle's tests and the CUDA path's tests may draw their inputs from it without sharing
any of the method between them.

The paper's experiments run on CIFAR-10 / LSUN / PushT data with trained networks
(Section 7, Appendix I); none of that is available offline, so inputs of the same *shapes*
stand in: exact Gaussian-mixture denoisers (the paper's low-dimensional study uses
16-component mixtures, Section 7 "Low dimensional experiments") and a random-init MLP with
the CIFAR-10 pixel dimension d = 3*32*32.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

# ----------------------------------------------------------------------------------------
# noise schedules (published definitions; no sampler arithmetic)
# ----------------------------------------------------------------------------------------


def beta_linear(T: int, beta_1: float = 1e-4, beta_T: float = 0.02) -> np.ndarray:
    """beta_t, t = 1..T, linear from beta_1 to beta_T (returned array index t-1)."""
    if T == 1:
        return np.array([beta_1], dtype=np.float64)
    t = np.arange(1, T + 1, dtype=np.float64)
    return beta_1 + (beta_T - beta_1) * (t - 1.0) / (T - 1.0)


def beta_cosine(T: int, s: float = 0.008, beta_max: float = 0.999) -> np.ndarray:
    """beta_t, t = 1..T, of the cosine schedule: abar_t = f(t)/f(0),
    f(t) = cos^2(((t/T + s)/(1 + s)) * pi/2), beta_t = min(1 - abar_t/abar_{t-1}, beta_max)."""
    t = np.arange(0, T + 1, dtype=np.float64)
    f = np.cos(((t / T + s) / (1.0 + s)) * (math.pi / 2.0)) ** 2
    abar = f / f[0]
    beta = 1.0 - abar[1:] / abar[:-1]
    return np.minimum(beta, beta_max)


# ----------------------------------------------------------------------------------------
# bf16 helpers (format conversion only)
# ----------------------------------------------------------------------------------------


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even float32 -> bfloat16, returned as uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    lsb = (u >> np.uint64(16)) & np.uint64(1)
    u = u + np.uint64(0x7FFF) + lsb
    return (u >> np.uint64(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


# ----------------------------------------------------------------------------------------
# mixture / MLP parameters
# ----------------------------------------------------------------------------------------


@dataclass
class GmmParams:
    means: np.ndarray        # [ncomp, d] float32 (bf16-representable when means_bf16)
    logw: np.ndarray         # [ncomp] float32, log mixture weights
    comp_std: float          # shared isotropic component std s
    means_bf16: bool = False


def gmm_params(seed: int, ncomp: int, d: int, mean_scale: float, comp_std: float,
               unit_norm: bool = False, means_bf16: bool = False) -> GmmParams:
    """Equal-weight mixture; means ~ N(0, mean_scale^2 I), or mean_scale * g/|g| when unit_norm."""
    rng = np.random.default_rng(seed)
    g = rng.standard_normal((ncomp, d))
    if unit_norm:
        g = g / np.linalg.norm(g, axis=1, keepdims=True)
    means = (mean_scale * g).astype(np.float32)
    if means_bf16:
        means = bf16_bits_to_f32(f32_to_bf16_bits(means))
    logw = np.full((ncomp,), -math.log(ncomp), dtype=np.float32)
    return GmmParams(means=means, logw=logw, comp_std=float(comp_std), means_bf16=means_bf16)


@dataclass
class MlpParams:
    """Random-init MLP denoiser: dims[0] -> dims[1] -> ... -> dims[-1].

    weights[l]: [dims[l+1], dims[l]] as bf16 bit patterns (uint16), Kaiming-normal N(0, 2/fan_in)
    bias[l]   : [dims[l+1]] float32 (zeros)
    temb[l]   : [K, dims[l+1]] bf16 bits, the per-step embedding row added before the activation
                of hidden layer l (l < nlayer-1): P_l @ tau(k), tau = 64 sin + 64 cos features of
                the integer step k at frequencies 10000^(-i/64), P_l ~ N(0, 2/128).
    """
    dims: list
    weights: list
    bias: list
    temb: list
    K: int


def time_features(K: int, dim: int = 128) -> np.ndarray:
    half = dim // 2
    freq = 10000.0 ** (-np.arange(half, dtype=np.float64) / half)
    ang = np.arange(K, dtype=np.float64)[:, None] * freq[None, :]
    return np.concatenate([np.sin(ang), np.cos(ang)], axis=1)          # [K, dim]


def mlp_params(seed: int, dims: list, K: int, temb_dim: int = 128) -> MlpParams:
    rng = np.random.default_rng(seed)
    tau = time_features(K, temb_dim)
    weights, bias, temb = [], [], []
    nlayer = len(dims) - 1
    for l in range(nlayer):
        fan_in, fan_out = dims[l], dims[l + 1]
        W = rng.standard_normal((fan_out, fan_in)) * math.sqrt(2.0 / fan_in)
        weights.append(f32_to_bf16_bits(W.astype(np.float32)))
        bias.append(np.zeros((fan_out,), dtype=np.float32))
        if l < nlayer - 1:
            P = rng.standard_normal((fan_out, temb_dim)) * math.sqrt(2.0 / temb_dim)
            temb.append(f32_to_bf16_bits((tau @ P.T).astype(np.float32)))
        else:
            temb.append(None)
    return MlpParams(dims=list(dims), weights=weights, bias=bias, temb=temb, K=K)


# ----------------------------------------------------------------------------------------
# the five workloads
# ----------------------------------------------------------------------------------------


@dataclass
class Workload:
    name: str
    B: int                      # chains
    d: int                      # state dimension
    L: int                      # window (lookahead)
    K: int                      # number of transitions
    sampler: str                # "ddpm" | "ula"
    schedule: str = ""          # "linear" | "cosine" (ddpm)
    ula_gamma: float = 0.0
    denoiser: str = "gmm"       # "gmm" | "mlp"
    gmm: dict = field(default_factory=dict)
    mlp_dims: list = field(default_factory=list)
    phi4: dict = field(default_factory=dict)     # side, beta, periodic (lattice energy workload)
    drafter_mode: int = 0                        # 0: carried target output, 1: target evaluated at Y_n
    param_seed: int = 0
    sample_seed: int = 2025
    dtype: str = "f32"

    def beta(self) -> np.ndarray:
        if self.sampler != "ddpm":
            raise ValueError("beta is defined for ddpm workloads only")
        return beta_linear(self.K) if self.schedule == "linear" else beta_cosine(self.K)

    def gmm_params(self, d: int | None = None, ncomp: int | None = None) -> GmmParams:
        g = dict(self.gmm)
        return gmm_params(self.param_seed, ncomp or g["ncomp"], d or self.d, g["mean_scale"],
                          g["comp_std"], g.get("unit_norm", False), g.get("means_bf16", False))

    def mlp_params(self, dims: list | None = None, K: int | None = None) -> MlpParams:
        return mlp_params(self.param_seed, dims or self.mlp_dims, K or self.K)

    def scaled(self, **kw) -> "Workload":
        """A smaller instance of the same recipe (for parity tests the oracle can finish)."""
        import copy
        w = copy.deepcopy(self)
        for k, v in kw.items():
            setattr(w, k, v)
        return w


WORKLOADS = {
    # 2-D mixture, K_mix = 4, means ~ N(0, 4 I), s = 0.3; linear beta, T = 100
    "cfg1": Workload("cfg1", B=64, d=2, L=4, K=100, sampler="ddpm", schedule="linear",
                     gmm=dict(ncomp=4, mean_scale=2.0, comp_std=0.3), param_seed=1001, sample_seed=2025),
    # d = 64, 16 components, means ~ N(0, 9 I), s = 0.5; cosine, T = 200
    "cfg2": Workload("cfg2", B=4096, d=64, L=8, K=200, sampler="ddpm", schedule="cosine",
                     gmm=dict(ncomp=16, mean_scale=3.0, comp_std=0.5), param_seed=1002, sample_seed=2026),
    # image-shaped state with a random-init bf16 MLP denoiser; linear beta, T = 250
    "cfg3": Workload("cfg3", B=2048, d=3072, L=8, K=250, sampler="ddpm", schedule="linear",
                     denoiser="mlp", mlp_dims=[3072, 2048, 2048, 2048, 3072], param_seed=1003,
                     sample_seed=2027, dtype="bf16"),
    # large-K mixture: d = 16384, 1024 unit-norm means scaled by 8, s = 0.2; cosine, T = 500
    "cfg4": Workload("cfg4", B=1024, d=16384, L=16, K=500, sampler="ddpm", schedule="cosine",
                     gmm=dict(ncomp=1024, mean_scale=8.0, comp_std=0.2, unit_norm=True, means_bf16=True),
                     param_seed=1004, sample_seed=2028, dtype="bf16"),
    # unadjusted Langevin on a mixture energy: d = 1024, 256 comps, means ~ N(0, 16 I), s = 1
    "cfg5": Workload("cfg5", B=8192, d=1024, L=32, K=2000, sampler="ula", ula_gamma=1e-3,
                     gmm=dict(ncomp=256, mean_scale=4.0, comp_std=1.0), param_seed=1005, sample_seed=2029),
    # Langevin chains on the phi^4 lattice energy (Appendix K): 8x8 grid, beta = 100, step 1e-3,
    # 100000 iterations, window 20, 500 runs, frozen drafter evaluated at Y_n
    "phi4": Workload("phi4", B=500, d=64, L=20, K=100000, sampler="ula", ula_gamma=1e-3, denoiser="phi4",
                     phi4=dict(side=8, beta=100.0, periodic=False), drafter_mode=1, sample_seed=2030),
}
