"""Builds a Sampler for a workload description (any object with the fields of workloads.Workload)."""
from __future__ import annotations

import numpy as np

from . import binding as sb
from . import schedules as sc


def schedule_for(w):
    """float32 (a, c, sigma) and the mixture conditioning table for workload w (None for non-mixtures)."""
    if w.sampler == "ddpm":
        a, c, sigma, abar = sc.ddpm_schedule(w.beta())
        tcond = sc.gmm_tcond_posterior_mean(abar, w.gmm["comp_std"]) if w.denoiser == "gmm" else None
    elif w.sampler == "ula":
        a, c, sigma = sc.ula_schedule(w.K, w.ula_gamma)
        tcond = sc.gmm_tcond_grad_energy(w.K, w.gmm["comp_std"]) if w.denoiser == "gmm" else None
    else:
        raise ValueError(w.sampler)
    return a, c, sigma, tcond


def drafter_for(w, *, gmm=None, mlp=None):
    """Description of an independent draft model for workload w: a (smaller) mixture or MLP."""
    if gmm is not None:
        if w.sampler == "ddpm":
            tc = sc.gmm_tcond_posterior_mean(sc.ddpm_schedule(w.beta())[3], gmm.comp_std)
        else:
            tc = sc.gmm_tcond_grad_energy(w.K, gmm.comp_std)
        return dict(gmm_means=gmm.means, gmm_logw=gmm.logw, tcond=tc, gmm_bf16=bool(getattr(gmm, "means_bf16", False)))
    if mlp is not None:
        return dict(mlp=mlp)
    raise ValueError("a draft model is required")


def picard_for(w, calls: int):
    """(calls, a_det, c_det) for Sampler(picard=...): the deterministic sampler that goes with the
    workload's schedule (noise-free ancestral step for ddpm, gradient step for Langevin)."""
    if w.sampler == "ddpm":
        a_det, c_det = sc.ddim_schedule(w.beta())
    else:
        a_det, c_det, _ = sc.ula_schedule(w.K, w.ula_gamma)
    return (int(calls), a_det, c_det)


def sampler_for(w, *, seed=None, chain_id_offset=0, B=None, device="cuda:0", gmm=None, mlp=None, drafter_mode=None,
                drafter=None, picard=None):
    a, c, sigma, tcond = schedule_for(w)
    if drafter_mode is None:
        drafter_mode = getattr(w, "drafter_mode", 0)
    seed = w.sample_seed if seed is None else seed
    B = w.B if B is None else B
    if w.denoiser == "gmm":
        gp = gmm if gmm is not None else w.gmm_params()
        return sb.Sampler(a, c, sigma, B, w.d, w.L, gmm_means=gp.means, gmm_logw=gp.logw, tcond=tcond,
                          gmm_bf16=bool(getattr(gp, "means_bf16", False)), seed=seed,
                          chain_id_offset=chain_id_offset, drafter_mode=drafter_mode, drafter=drafter, picard=picard, device=device)
    if w.denoiser == "mlp":
        mp = mlp if mlp is not None else w.mlp_params()
        return sb.Sampler(a, c, sigma, B, w.d, w.L, mlp=mp, seed=seed, chain_id_offset=chain_id_offset, drafter_mode=drafter_mode, drafter=drafter, picard=picard, device=device)
    if w.denoiser == "phi4":
        p4 = w.phi4
        return sb.Sampler(a, c, sigma, B, w.d, w.L, phi4=(p4["side"], p4["beta"], p4.get("periodic", False)), seed=seed,
                          chain_id_offset=chain_id_offset, drafter_mode=drafter_mode, drafter=drafter, picard=picard, device=device)
    raise NotImplementedError(w.denoiser)
