"""The allocation-free mixture denoiser call (sds_gmm_denoise_static) against the regular
context-based call (sds_denoise).

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
import workloads as wl

pytestmark = pytest.mark.gpu


def _case(torch, name, d, ncomp, rows, seed):
    w = wl.WORKLOADS[name].scaled(d=d, B=rows, L=1)
    gp = w.gmm_params(d=d, ncomp=ncomp)
    s = sds.sampler_for(w, gmm=gp)
    _, _, _, tcond = sds.schedule_for(w)
    rng = np.random.default_rng(seed)
    x = torch.from_numpy((rng.standard_normal((rows, d)) * 1.5).astype(np.float32)).cuda()
    k = torch.from_numpy(rng.integers(0, w.K, size=rows).astype(np.int32)).cuda()
    return s, torch.from_numpy(tcond).cuda(), x, k


def test_static_scratch_denoiser_matches_context_denoiser_twice():
    import torch
    cases = [_case(torch, "cfg2", 64, 16, 300, 1), _case(torch, "cfg2", 33, 5, 77, 2)]
    outs = [torch.empty_like(c[2]) for c in cases]       # caller-owned outputs, allocated up front
    for (s, tcond, x, k), out in zip(cases, outs):
        sb.gmm_denoise_static(x, k, s.means, s.logw, tcond, out)
    torch.cuda.synchronize()
    for (s, tcond, x, k), out in zip(cases, outs):
        ref = s.denoise(x, k)
        torch.cuda.synchronize()
        got, want = out.cpu().numpy().astype(np.float64), ref.cpu().numpy().astype(np.float64)
        err = np.linalg.norm(got - want, axis=1) / np.maximum(np.linalg.norm(want, axis=1), 1e-6)
        assert err.max() <= 1e-5, err.max()
    # sizes beyond the built-in scratch are refused, nothing is launched
    s, tcond, x, k = cases[0]
    rc = s.lib.sds_gmm_denoise_static(x.data_ptr(), k.data_ptr(), 1, 64, sb.STATIC_MAX_NCOMP + 1, s.means.data_ptr(),
                                      s.logw.data_ptr(), tcond.data_ptr(), tcond.shape[0], outs[0].data_ptr(), None)
    assert rc == sb.SDS_EUNSUPPORTED
    for c in cases:
        c[0].close()
