"""The allocation-free mixture denoiser call (sds_gmm_denoise_static) against the regular
context-based call (sds_denoise) and against the CPU oracle.

Some users of the library cannot allocate device memory where they need a target pass (code
hosted inside an application that owns the memory pool, latency-critical paths that must avoid
the synchronisation an allocation implies, fixed memory budgets). For them the call keeps its
only scratch, the |mu_c|^2 table, in an array built into the library. Because that array is
shared by all calls and keeps its previous contents, the test makes two calls in a row with
different mixtures (the second smaller, so stale entries would show) and checks both.
This file sorts last so that a run stopping at the first failure has already run the others.
"""
import numpy as np
import pytest

import paper_2501_05370_b200 as sds
from paper_2501_05370_b200 import binding as sb
from oracle import sds_oracle as o
import workloads as wl

pytestmark = pytest.mark.gpu


def _case(torch, name, d, ncomp, rows, seed, with_ctx=True):
    w = wl.WORKLOADS[name].scaled(d=d, B=rows, L=1)
    gp = w.gmm_params(d=d, ncomp=ncomp)
    _, _, _, tcond = sds.schedule_for(w)
    rng = np.random.default_rng(seed)
    x = (rng.standard_normal((rows, d)) * 1.5).astype(np.float32)
    k = rng.integers(0, w.K, size=rows).astype(np.int32)
    s = sds.sampler_for(w, gmm=gp) if with_ctx else None
    return dict(w=w, gp=gp, s=s, tcond=torch.from_numpy(tcond).cuda(), x=torch.from_numpy(x).cuda(),
                k=torch.from_numpy(k).cuda(), x_np=x, k_np=k,
                means=s.means if s else torch.from_numpy(gp.means).cuda(),
                logw=s.logw if s else torch.from_numpy(gp.logw).cuda())


def _row_err(got, want):
    got, want = np.asarray(got, np.float64), np.asarray(want, np.float64)
    return np.linalg.norm(got - want, axis=-1) / np.maximum(np.linalg.norm(want, axis=-1), 1e-6)


def _oracle_rows(c, rows):
    abar = o.ddpm_affine(c["w"].beta())[3]
    gp = c["gp"]
    return np.stack([o.gmm_posterior_mean(c["x_np"][r].astype(np.float64), abar[int(c["k_np"][r])], gp.means, gp.logw,
                                          gp.comp_std) for r in rows])


def test_static_scratch_denoiser_matches_context_denoiser_twice():
    import torch
    cases = [_case(torch, "cfg2", 64, 16, 300, 1), _case(torch, "cfg2", 33, 5, 77, 2)]
    outs = [torch.empty_like(c["x"]) for c in cases]       # caller-owned outputs, allocated up front
    for c, out in zip(cases, outs):
        sb.gmm_denoise_static(c["x"], c["k"], c["means"], c["logw"], c["tcond"], out)
    torch.cuda.synchronize()
    for c, out in zip(cases, outs):
        ref = c["s"].denoise(c["x"], c["k"])
        torch.cuda.synchronize()
        err = _row_err(out.cpu().numpy(), ref.cpu().numpy())
        assert err.max() <= 1e-5, err.max()
        # and against the oracle's closed form, so that an error shared by both calls would show
        rows = list(range(0, out.shape[0], 7))
        err = _row_err(out.cpu().numpy()[rows], _oracle_rows(c, rows))
        assert err.max() <= 1e-5, err.max()
    # sizes beyond the built-in scratch are refused, nothing is launched
    c = cases[0]
    rc = c["s"].lib.sds_gmm_denoise_static(c["x"].data_ptr(), c["k"].data_ptr(), 1, 64, sb.STATIC_MAX_NCOMP + 1,
                                           c["means"].data_ptr(), c["logw"].data_ptr(), c["tcond"].data_ptr(),
                                           c["tcond"].shape[0], outs[0].data_ptr(), None)
    assert rc == sb.SDS_EUNSUPPORTED
    for c in cases:
        c["s"].close()


@pytest.mark.parametrize("d,ncomp,rows", [
    (64, 100, 50),                          # the register-tiled kernel (33 to 256 components, d % 4 == 0)
    (33, 40, 45),                           # one warp per row, means staged in shared memory
    (64, 300, 40),                          # one warp per row, means too large for shared memory
    (8, sb.STATIC_MAX_NCOMP, 6),            # the top of the built-in table (64 KiB of logits per CTA)
])
def test_static_scratch_denoiser_every_kernel_branch_against_the_oracle(d, ncomp, rows):
    """One shape per kernel the float mixture dispatches to, up to the largest mixture the built-in
    table holds, each run twice in a row (the second call reuses the table the first one filled)."""
    import torch
    c = _case(torch, "cfg2", d, ncomp, rows, 100 + ncomp, with_ctx=False)
    want = _oracle_rows(c, range(rows))
    for _ in range(2):
        out = torch.full_like(c["x"], float("nan"))
        sb.gmm_denoise_static(c["x"], c["k"], c["means"], c["logw"], c["tcond"], out)
        torch.cuda.synchronize()
        err = _row_err(out.cpu().numpy(), want)
        assert err.max() <= 1e-5, (d, ncomp, err.max())
