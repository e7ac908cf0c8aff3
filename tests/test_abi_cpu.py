"""CPU-side checks of the boundary: the library loads, exports every call the header declares,
validates arguments on the host, and the binding's schedule helpers agree with the oracle's."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import paper_2501_05370_b200 as sds
from paper_2501_05370_b200 import binding as sb
from paper_2501_05370_b200 import schedules as sc
from oracle import sds_oracle as o
import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    names = set()
    for f in os.listdir(os.path.join(ROOT, "include")):
        if f.endswith(".h"):
            txt = open(os.path.join(ROOT, "include", f)).read()
            txt = re.sub(r"/\*.*?\*/", "", txt, flags=re.S)
            names |= set(re.findall(r"\b(sds_[a-z_0-9]+)\s*\(", txt))
    return names


def test_library_exports_every_declared_symbol():
    lib = sds.load()
    declared = _declared()
    assert len(declared) >= 18
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(sb.EXPORTS), declared ^ set(sb.EXPORTS)


def _sched(K=5, sigma0=0.1):
    a = np.full(K, 0.9, np.float32)
    c = np.full(K, 0.1, np.float32)
    s = np.full(K, sigma0, np.float32)
    t = np.zeros((K, 4), np.float64)
    sch = sb.SdsSchedule(K, a.ctypes.data, c.ctypes.data, s.ctypes.data, t.ctypes.data, 4)
    return sch, (a, c, s, t)


def _gmm_den():
    den = sb.SdsDenoiser()
    den.kind, den.ncomp, den.means_dev, den.logw_dev, den.means_dtype = sb.SDS_DEN_GMM, 4, 256, 512, sb.SDS_F32
    return den


def test_host_side_argument_validation():
    lib = sds.load()
    n = C.c_size_t(0)
    sch, keep = _sched()
    den = _gmm_den()
    ok = lib.sds_workspace_bytes(C.byref(sch), C.byref(den), 8, 6, 4, C.byref(n))
    assert ok == sb.SDS_OK and n.value > 8 * 4 * 6 * 4 * 2 and n.value % 256 == 0
    assert lib.sds_workspace_bytes(None, C.byref(den), 8, 6, 4, C.byref(n)) == sb.SDS_EINVAL
    assert lib.sds_workspace_bytes(C.byref(sch), C.byref(den), 0, 6, 4, C.byref(n)) == sb.SDS_EINVAL
    assert lib.sds_workspace_bytes(C.byref(sch), C.byref(den), 8, 0, 4, C.byref(n)) == sb.SDS_EINVAL
    assert lib.sds_workspace_bytes(C.byref(sch), C.byref(den), 8, 6, 0, C.byref(n)) == sb.SDS_EINVAL
    assert lib.sds_workspace_bytes(C.byref(sch), C.byref(den), 8, 6, 33, C.byref(n)) == sb.SDS_EINVAL
    bad, keep2 = _sched(sigma0=0.0)          # sigma must be positive (equal, proper Gaussians)
    assert lib.sds_workspace_bytes(C.byref(bad), C.byref(den), 8, 6, 4, C.byref(n)) == sb.SDS_EINVAL
    keep[0][2] = np.nan
    assert lib.sds_workspace_bytes(C.byref(sch), C.byref(den), 8, 6, 4, C.byref(n)) == sb.SDS_EINVAL
    keep[0][2] = 0.9
    den.kind = 99
    assert lib.sds_workspace_bytes(C.byref(sch), C.byref(den), 8, 6, 4, C.byref(n)) == sb.SDS_EUNSUPPORTED
    h = C.c_void_p()
    assert lib.sds_create(C.byref(sch), C.byref(den), 8, 6, 4, C.byref(h)) == sb.SDS_EUNSUPPORTED and not h.value
    assert lib.sds_reset(None) == sb.SDS_EINVAL
    assert lib.sds_strerror(sb.SDS_ESTATE) == b"call out of order"


@pytest.mark.parametrize("name", ["cfg1", "cfg2", "cfg3", "cfg4"])
def test_ddpm_schedule_helper_matches_oracle(name):
    w = wl.WORKLOADS[name]
    a, c, s, abar = sc.ddpm_schedule(w.beta())
    ao, co, so, abo = o.ddpm_affine(w.beta())
    assert a.dtype == np.float32
    for x, y in ((a, ao), (c, co), (s, so)):
        assert np.all(np.abs(x.astype(np.float64) - y) <= 2e-7 * np.maximum(np.abs(y), 1e-30) + 1e-12)
    assert np.allclose(abar, abo, rtol=1e-14)


def test_gmm_conditioning_table_reproduces_oracle_denoiser():
    """The (A, Bq, C, E) form the kernels evaluate, computed in double from the helper's table,
    equals the oracle's definition-level posterior mean / energy gradient."""
    w = wl.WORKLOADS["cfg2"]
    gp = w.gmm_params()
    a, c, s, abar = sc.ddpm_schedule(w.beta())
    tc = sc.gmm_tcond_posterior_mean(abar, gp.comp_std).astype(np.float64)
    rng = np.random.default_rng(0)
    mu = gp.means.astype(np.float64)
    for k in (0, 57, 150, 199):
        x = rng.standard_normal(w.d) * 1.5
        A, Bq, Cc, E = tc[k]
        lg = gp.logw + A * (mu @ x) + Bq * np.sum(mu * mu, axis=1)
        r = np.exp(lg - lg.max()); r /= r.sum()
        got = Cc * (r @ mu) + E * x
        want = o.gmm_posterior_mean(x, abar[k], gp.means, gp.logw, gp.comp_std)
        assert np.allclose(got, want, rtol=2e-5, atol=2e-5)
    w5 = wl.WORKLOADS["cfg5"]
    gp5 = w5.gmm_params(d=32, ncomp=8)
    tc5 = sc.gmm_tcond_grad_energy(3, gp5.comp_std).astype(np.float64)
    x = rng.standard_normal(32) * 4
    mu = gp5.means.astype(np.float64)
    A, Bq, Cc, E = tc5[0]
    lg = gp5.logw + A * (mu @ x) + Bq * np.sum(mu * mu, axis=1)
    r = np.exp(lg - lg.max()); r /= r.sum()
    assert np.allclose(Cc * (r @ mu) + E * x, o.gmm_grad_energy(x, gp5.means, gp5.logw, gp5.comp_std), rtol=1e-6, atol=1e-6)
    a5, c5, s5 = sc.ula_schedule(3, 1e-3)
    ao, co, so = o.ula_affine(3, 1e-3)
    assert np.allclose(a5, ao) and np.allclose(c5, co, rtol=1e-7) and np.allclose(s5, so, rtol=1e-7)


def test_sampler_refuses_to_run_without_cuda():
    import torch
    if torch.cuda.is_available():
        pytest.skip("CUDA present")
    w = wl.WORKLOADS["cfg1"]
    with pytest.raises(RuntimeError):
        sds.sampler_for(w)


def test_binding_constants_equal_the_header_macros():
    """Every SDS_OPT_* / SDS_GET_* / SDS_PROF_* macro and status code the binding names has the header's value."""
    txt = open(os.path.join(ROOT, "include", "sds.h")).read()
    macros = {m.group(1): int(m.group(2), 0) for m in re.finditer(r"#define\s+(SDS_[A-Z0-9_]+)\s+\(?(-?\d+)\)?", txt)}
    assert macros["SDS_OPT_STAGED_WINDOWS"] == sb.Sampler.OPT_STAGED_WINDOWS
    assert macros["SDS_STAGED_ADAPTIVE"] == sb.Sampler.STAGED_ADAPTIVE
    checked = 0
    for name, val in macros.items():
        if name.startswith("SDS_OPT_"):
            assert getattr(sb.Sampler, name[4:]) == val, name
            checked += 1
        elif name.startswith("SDS_GET_") and hasattr(sb, name[4:]):
            assert getattr(sb, name[4:]) == val, name
            checked += 1
        elif hasattr(sb, name):
            assert getattr(sb, name) == val, name
            checked += 1
    assert checked >= 25
    assert len(sb.Sampler.PROF_KINDS) == macros["SDS_PROF_KINDS"]
