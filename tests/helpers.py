"""Shared test helpers: oracle-side closures for a workload and comparison utilities."""
import math

import numpy as np

from oracle import sds_oracle as o


def oracle_setup(w, gmm=None, mlp=None):
    """(denoise(x, k), a, c, sigma) in double for workload w, all from the oracle's own formulas."""
    if w.sampler == "ddpm":
        a, c, sig, abar = o.ddpm_affine(w.beta())
    else:
        a, c, sig = o.ula_affine(w.K, w.ula_gamma)
        abar = None
    if w.denoiser == "gmm":
        gp = gmm if gmm is not None else w.gmm_params()
        if w.sampler == "ddpm":
            den = lambda x, k: o.gmm_posterior_mean(x, abar[k], gp.means, gp.logw, gp.comp_std,
                                                    bf16_operands=gp.means_bf16)
        else:
            den = lambda x, k: o.gmm_grad_energy(x, gp.means, gp.logw, gp.comp_std)
    elif w.denoiser == "phi4":
        p4 = w.phi4
        den = lambda x, k: o.phi4_grad_energy(x, p4["side"], p4["beta"], p4.get("periodic", False))
    else:
        import workloads as wl
        mp = mlp if mlp is not None else w.mlp_params()
        W = [wl.bf16_bits_to_f32(x).astype(np.float64) for x in mp.weights]
        T = [wl.bf16_bits_to_f32(x).astype(np.float64) if x is not None else None for x in mp.temb]
        den = lambda x, k: o.mlp_forward(x, k, W, mp.bias, T)
    return den, a, c, sig


def rel_l2(got, want, floor=1e-6):
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    return np.linalg.norm(got - want) / max(np.linalg.norm(want), floor)


def ell_close(g, w):
    """|l_gpu - l_oracle| <= 1e-4 where the oracle's value is in [-20, 0.5], else 1e-5 relative."""
    tol = 1e-4 if -20.0 <= w <= 0.5 else 1e-5 * abs(w)
    return abs(g - w) <= tol


BAND = 2e-4   # |log ratio - log U| below this: either decision is a correct rounding
