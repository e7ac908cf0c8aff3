"""GPU parity of the Picard drafter (Appendix C: parallel sampling as drafting) with the oracle."""
import math

import numpy as np
import pytest

import paper_2501_05370_b200 as sds
from paper_2501_05370_b200 import binding as sb
from oracle import sds_oracle as o
import workloads as wl
from helpers import BAND, assert_rows_close, chain_matches_or_band, ell_close, oracle_setup, rel_l2

pytestmark = pytest.mark.gpu


def _det_coeffs(w):
    if w.sampler == "ddpm":
        return o.ddim_affine(w.beta())
    a, c, _ = o.ula_affine(w.K, w.ula_gamma)
    return a, c


def _picard_window(s, w, den, a, c, sig, a_det, c_det, calls, seed, chains, stats, tol=1e-5):
    """One window on the GPU (draft, verify, advance), replayed by the oracle: the Picard points and
    draft means from the oracle's own trajectory, the verification on the GPU's arrays."""
    s.set_option(s.OPT_VERIFY_EARLY_EXIT, 0)      # these checks look at every position of the window
    B, L, d, K = s.B, s.L, s.d, s.K
    na = int(s.get(sb.GET_CTL)[0])
    act, rowoff, n = s.get(sb.GET_ACT)[:na], s.get(sb.GET_ROWOFF)[:na + 1], s.get(sb.GET_N)
    Y, Dc = s.get(sb.GET_Y), s.get(sb.GET_DC)
    s.draft()
    X, T, Mp, rowk = s.get(sb.GET_X), s.get(sb.GET_TAIL), s.get(sb.GET_DP), s.get(sb.GET_ROWK)
    s.verify_window()
    Dq, X2, T2 = s.get(sb.GET_DQ), s.get(sb.GET_X), s.get(sb.GET_TAIL)
    S1, ell, logU = s.get(sb.GET_S1), s.get(sb.GET_ELL), s.get(sb.GET_LOGU)
    accmask, jstar = s.get(sb.GET_ACCMASK), s.get(sb.GET_JSTAR)
    for si, b in enumerate(act):
        if int(b) not in chains:
            continue
        nb = int(n[b]); Lt = min(L, K - nb); r0 = int(rowoff[si])
        assert np.array_equal(rowk[r0:r0 + Lt], nb + np.arange(Lt))
        assert np.array_equal(X[r0], Y[b])
        F = o.picard_trajectory(den, a_det, c_det, Y[b].astype(np.float64), Dc[b].astype(np.float64), nb, Lt, calls - 1)
        W = np.concatenate([X[r0:r0 + Lt], T[b:b + 1]]).astype(np.float64)
        for j in range(1, Lt + 1):
            k = nb + j - 1
            want_mp = a[k] * F[j - 1] + c[k] * den(F[j - 1], k)
            assert_rows_close(Mp[r0 + j - 1], want_mp, tol, (b, j))
            xi = o.normals(seed, o.STREAM_DRAFT, int(b), k, d)
            assert_rows_close(W[j], Mp[r0 + j - 1].astype(np.float64) + sig[k] * xi, 1e-5, (b, j))
            assert_rows_close(Dq[r0 + j - 1], den(W[j - 1], k), tol, (b, j))
        v = o.verify_window(W, Dq[r0:r0 + Lt], None, a, c, sig, nb, logU[b, :Lt].astype(np.float64),
                            M_p=Mp[r0:r0 + Lt])
        assert S1[b, 0] < 1e-20 and (int(accmask[b]) & 1)          # position 1 is drafted from the target itself
        amb = np.abs(v["ell"] - logU[b, :Lt]) < BAND
        for j in range(Lt):
            assert ell_close(float(ell[b, j]), float(v["ell"][j])), (b, j, ell[b, j], v["ell"][j])
            stats["tests"] += 1
            if amb[j]:
                stats["band"] += 1
            else:
                assert bool((int(accmask[b]) >> j) & 1) == bool(v["acc"][j]), (b, j)
        js = int(jstar[b])
        if not amb.any():
            assert js == v["jstar"]
        if js <= Lt and js == v["jstar"]:
            got = X2[r0 + js] if js < Lt else T2[b]
            assert_rows_close(got, v["Y_reflect"], 1e-5, (b, js))
            stats["reflected"] += 1
    s.advance()
    n2, Y2, Dc2 = s.get(sb.GET_N), s.get(sb.GET_Y), s.get(sb.GET_DC)
    for si, b in enumerate(act):
        nb = int(n[b]); Lt = min(L, K - nb); r0 = int(rowoff[si])
        adv = min(int(jstar[b]), Lt)
        assert n2[b] == nb + adv
        assert np.array_equal(Y2[b], X2[r0 + adv] if adv < Lt else T2[b])
        assert np.array_equal(Dc2[b], Dq[r0 + adv - 1])


@pytest.mark.parametrize("calls,d", [(1, 64), (3, 64), (2, 1030)])
def test_picard_window_and_free_run_match_oracle(calls, d):
    w = wl.WORKLOADS["cfg2"].scaled(B=20, d=d, K=30, L=6)
    gp = w.gmm_params(d=d)
    den, a, c, sig = oracle_setup(w, gmm=gp)
    a_det, c_det = _det_coeffs(w)
    s = sds.sampler_for(w, gmm=gp, seed=51, picard=sds.picard_for(w, calls))
    s.reset()
    stats = dict(tests=0, band=0, reflected=0)
    for _ in range(4):
        _picard_window(s, w, den, a, c, sig, a_det, c_det, calls, 51, set(range(6)), stats)
    assert stats["reflected"] >= 1 and stats["band"] <= 2
    out, ncalls, nrows = [x.cpu().numpy() for x in s.sample_all()]
    bad = 0
    for b in range(6):
        r = o.speculative_chain(den, a, c, sig, w.L, 51, b, d, mode=o.PICARD, picard=(calls, a_det, c_det), record=True)
        bad += not chain_matches_or_band(r, ncalls[b], nrows[b], out[b])
    assert bad <= 1
    assert np.array_equal(s.get(sb.GET_N), np.full(w.B, w.K))
    s.close()


def test_picard_langevin_chain():
    w = wl.WORKLOADS["cfg5"].scaled(B=16, d=96, K=40, L=8)
    gp = w.gmm_params(d=96, ncomp=12)
    den, a, c, sig = oracle_setup(w, gmm=gp)
    a_det, c_det = _det_coeffs(w)
    s = sds.sampler_for(w, gmm=gp, seed=52, picard=sds.picard_for(w, 2))
    s.reset()
    stats = dict(tests=0, band=0, reflected=0)
    for _ in range(3):
        _picard_window(s, w, den, a, c, sig, a_det, c_det, 2, 52, set(range(5)), stats)
    out, ncalls, nrows = [x.cpu().numpy() for x in s.sample_all()]
    bad = 0
    for b in range(5):
        r = o.speculative_chain(den, a, c, sig, w.L, 52, b, w.d, mode=o.PICARD, picard=(2, a_det, c_det), record=True)
        bad += not chain_matches_or_band(r, ncalls[b], nrows[b], out[b])
    assert bad <= 1
    s.close()


def test_picard_with_tensor_core_mlp():
    dims = [256, 384, 256]
    w = wl.WORKLOADS["cfg3"].scaled(d=256, B=40, L=6, K=24, mlp_dims=dims)
    mp = w.mlp_params()
    den, a, c, sig = oracle_setup(w, mlp=mp)
    a_det, c_det = _det_coeffs(w)
    s = sds.sampler_for(w, mlp=mp, seed=53, picard=sds.picard_for(w, 2))
    s.reset()
    stats = dict(tests=0, band=0, reflected=0)
    for _ in range(3):
        _picard_window(s, w, den, a, c, sig, a_det, c_det, 2, 53, set(range(4)), stats, tol=2e-2)
    out, ncalls, nrows = [x.cpu().numpy() for x in s.sample_all()]
    assert np.all(np.isfinite(out)) and np.array_equal(s.get(sb.GET_N), np.full(w.B, w.K))
    assert np.array_equal(out, s.sample_all()[0].cpu().numpy())      # deterministic
    s.close()


def test_picard_context_and_mode_go_together():
    w = wl.WORKLOADS["cfg1"]
    gp = w.gmm_params()
    with pytest.raises(sb.SdsError):
        sds.sampler_for(w, gmm=gp, drafter_mode=sb.SDS_PICARD)          # plain context, Picard mode
    with pytest.raises(sb.SdsError):
        sds.sampler_for(w, gmm=gp, picard=(0,) + sds.picard_for(w, 1)[1:])   # at least one call
