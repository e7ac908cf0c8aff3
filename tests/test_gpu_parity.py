"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded
inputs. Tiers: generator and denoiser kernels alone; one window on forced arrays (decisions
exact outside the rounding band); free-running chains end to end."""
import math

import numpy as np
import pytest

import paper_2501_05370_b200 as sds
from paper_2501_05370_b200 import binding as sb
from oracle import sds_oracle as o
import workloads as wl
from helpers import BAND, assert_rows_close, chain_matches_or_band, ell_close, oracle_setup, rel_l2

pytestmark = pytest.mark.gpu


def _torch():
    import torch
    return torch


# ------------------------------------------------------------------ generator -----------

@pytest.mark.parametrize("b0,k,d", [(0, 0, 1), (5, 17, 7), (123456, 499, 64), ((1 << 32) + 9, 3, 130), (7, 1999, 1024)])
def test_rng_normals_and_uniforms(b0, k, d):
    seed = 0x1234_5678_9ABC_DEF1
    nb = 5
    for stream in (o.STREAM_DRAFT, o.STREAM_INIT):
        got = sb.rng_normals(seed, stream, b0, nb, k, d).cpu().numpy()
        want = np.stack([o.normals(seed, stream, b0 + i, k, d) for i in range(nb)])
        # the library's Box-Muller uses the special-function unit: lg2 (2^-22), sqrt (2^-23 relative),
        # sin/cos (2^-20.5 absolute) give at most ~1e-6 r + 1.7e-7/r per normal, r <= 5.77
        assert np.max(np.abs(got - want)) <= 7e-6
        assert np.mean(np.abs(got - want)) <= 1e-6
    u = sb.rng_uniforms(seed, b0, nb, k).cpu().numpy()
    uw = np.array([o.uniform01(seed, b0 + i, k) for i in range(nb)])
    assert np.array_equal(u.astype(np.float64), uw)          # exact: multiples of 2^-24


# ------------------------------------------------------------------ denoiser ------------

@pytest.mark.parametrize("name,d,ncomp,rows", [("cfg1", 2, 4, 37), ("cfg2", 64, 16, 515), ("cfg2", 33, 5, 70),
                                              ("cfg5", 96, 40, 130), ("cfg5", 1024, 24, 21), ("cfg5", 1024, 256, 150),
                                              ("cfg2", 200, 100, 131), ("cfg5", 260, 33, 64), ("cfg2", 256, 128, 300),
                                              ("cfg5", 384, 256, 77)])
def test_gmm_denoiser_rows(name, d, ncomp, rows):
    torch = _torch()
    w = wl.WORKLOADS[name].scaled(d=d, B=max(rows, 1), L=1)
    gp = w.gmm_params(d=d, ncomp=ncomp)
    s = sds.sampler_for(w, gmm=gp)
    den, a, c, sig = oracle_setup(w, gmm=gp)
    rng = np.random.default_rng(1)
    scale = 4.0 if w.sampler == "ula" else 1.5
    x = (rng.standard_normal((rows, d)) * scale).astype(np.float32)
    # some rows sit near a component mean (sharp responsibilities)
    x[::7] = gp.means[rng.integers(0, ncomp, size=len(x[::7]))] * (0.9 if w.sampler == "ddpm" else 1.0) + 0.1 * x[::7]
    k = rng.integers(0, w.K, size=rows).astype(np.int32)
    out = s.denoise(torch.from_numpy(x).cuda(), torch.from_numpy(k).cuda()).cpu().numpy()
    for r in range(rows):
        want = den(x[r].astype(np.float64), int(k[r]))
        assert_rows_close(out[r], want, 1e-5, r)
    s.close()


def test_split_precision_tensor_path_agrees_with_float_alu_path():
    """Float mixtures of tensor-core shape run as bf16 GEMMs on a three-way split of every operand;
    the float ALU kernel (option off) must give the same rows to float accuracy."""
    torch = _torch()
    for name, d, ncomp in (("cfg2", 256, 128), ("cfg5", 1024, 256)):
        rows = 333
        w = wl.WORKLOADS[name].scaled(d=d, B=rows, L=1)
        gp = w.gmm_params(d=d, ncomp=ncomp)
        s = sds.sampler_for(w, gmm=gp)
        rng = np.random.default_rng(9)
        x = torch.from_numpy((rng.standard_normal((rows, d)) * (4.0 if w.sampler == "ula" else 1.5)).astype(np.float32)).cuda()
        k = torch.from_numpy(rng.integers(0, w.K, size=rows).astype(np.int32)).cuda()
        a = s.denoise(x, k).cpu().numpy()
        s.set_option(s.OPT_TENSOR_SPLIT, 0)
        b = s.denoise(x, k).cpu().numpy()
        err = np.linalg.norm(a - b, axis=1) / np.maximum(np.linalg.norm(b, axis=1), 1e-6)
        assert err.max() <= 1e-5, err.max()
        s.close()


# ------------------------------------------------------------------ one window, forced ---

def _window_check(s, w, den, a32, c32, s32, seed, chain_off, stats, chains=None, draft_den=None, proj=None):
    """Runs draft + verify on the GPU and replays the verification on the GPU's own arrays."""
    s.set_option(s.OPT_VERIFY_EARLY_EXIT, 0)      # these checks look at every position of the window
    B, L, d, K = s.B, s.L, s.d, s.K
    ctl = s.get(sb.GET_CTL)
    na, nrows = int(ctl[0]), int(ctl[1])
    act, rowoff, n = s.get(sb.GET_ACT)[:na], s.get(sb.GET_ROWOFF)[:na + 1], s.get(sb.GET_N)
    assert np.all(np.diff(act) > 0)
    assert int(rowoff[na]) == nrows == int(sum(min(L, K - n[b]) for b in act))
    Y = s.get(sb.GET_Y)
    s.draft()
    Dc = s.get(sb.GET_DC)            # the frozen output the draft used (recomputed by the draft call in exact mode)
    X, T, rowk = s.get(sb.GET_X), s.get(sb.GET_TAIL), s.get(sb.GET_ROWK)
    Dp = s.get(sb.GET_DP) if draft_den is not None else None     # independent draft model: output per drafted row
    s.verify_window()
    Dq = s.get(sb.GET_DQ)
    X2, T2 = s.get(sb.GET_X), s.get(sb.GET_TAIL)
    S1, S2, ell, logU = s.get(sb.GET_S1), s.get(sb.GET_S2), s.get(sb.GET_ELL), s.get(sb.GET_LOGU)
    accmask, jstar = s.get(sb.GET_ACCMASK), s.get(sb.GET_JSTAR)
    a64, c64, s64 = a32.astype(np.float64), c32.astype(np.float64), s32.astype(np.float64)
    for si, b in enumerate(act):
        if chains is not None and int(b) not in chains:
            continue
        nb = int(n[b]); Lt = min(L, K - nb); r0 = int(rowoff[si])
        assert np.array_equal(rowk[r0:r0 + Lt], nb + np.arange(Lt))
        W = np.concatenate([X[r0:r0 + Lt], T[b:b + 1]]).astype(np.float64)
        assert np.array_equal(X[r0], Y[b])
        # draft: W_j = a W_{j-1} + c D_c + sigma xi with the oracle's normals
        for j in range(1, Lt + 1):
            k = nb + j - 1
            xi = o.normals(seed, o.STREAM_DRAFT, chain_off + int(b), k, d)
            if draft_den is not None:
                assert_rows_close(Dp[r0 + j - 1], draft_den(W[j - 1], k), 1e-5, (b, j))
                dcj = Dp[r0 + j - 1].astype(np.float64)
            else:
                dcj = Dc[b].astype(np.float64)
            want = a64[k] * W[j - 1] + c64[k] * dcj + s64[k] * xi
            assert_rows_close(W[j], want, 1e-5, (b, j))
        # target rows
        for j in range(1, Lt + 1):
            assert_rows_close(Dq[r0 + j - 1], den(W[j - 1], nb + j - 1), 1e-5, (b, j))
        lu = np.array([math.log(o.uniform01(seed, chain_off + int(b), nb + j)) for j in range(Lt)])
        assert np.max(np.abs(logU[b, :Lt] - lu)) <= 2e-6
        dc_arg = Dp[r0:r0 + Lt] if draft_den is not None else Dc[b]
        v = o.verify_window(W, Dq[r0:r0 + Lt], dc_arg, a64, c64, s64, nb, logU[b, :Lt].astype(np.float64), proj=proj)
        amb = np.abs(v["ell"] - logU[b, :Lt]) < BAND
        if proj is None and draft_den is None and stats.get("mode", 0) == 0:
            # The same test on the kernel's own single-precision Delta and Z (its element formulas retyped
            # in float32, sums in double as in the kernel): the decisions must then agree everywhere, not
            # only outside the band (the band exists because the oracle forms Delta and Z in double). A
            # margin of 1e-6 covers the order of the double sums and the emulated fused multiply-adds.
            f32 = np.float32
            fma = lambda x, y, z: (x.astype(np.float64) * np.float64(y) + z.astype(np.float64)).astype(f32)
            for j in range(1, Lt + 1):
                k = nb + j - 1
                ak, ck, sk = f32(a32[k]), f32(c32[k]), f32(s32[k])
                inv_s = f32(1.0) / sk
                cs = ck * inv_s
                wp = X[r0 + j - 1]
                wj = X[r0 + j] if j < Lt else T[b]
                D = cs * (Dc[b] - Dq[r0 + j - 1])
                Z = fma(wp, -ak, wj)                                                # fmaf(-a, wp, wj)
                Z = fma(Dc[b], -ck, Z) * inv_s                                      # fmaf(-c, dc, .) / sigma
                S1k = float(np.sum(D.astype(np.float64) ** 2))
                S2k = float(np.sum(D.astype(np.float64) * Z.astype(np.float64)))
                ellk = -0.5 * S1k - S2k
                if abs(ellk - float(logU[b, j - 1])) > 1e-6 * max(1.0, abs(ellk)):
                    want_acc = (S1k < 1e-30) or (f32(logU[b, j - 1]) <= f32(ellk))
                    assert bool((int(accmask[b]) >> (j - 1)) & 1) == bool(want_acc), ("exact replay", b, j, ellk, logU[b, j - 1])
                    stats["exact"] = stats.get("exact", 0) + 1
        for j in range(Lt):
            assert ell_close(float(ell[b, j]), float(v["ell"][j])), (b, j, ell[b, j], v["ell"][j])
            assert abs(S1[b, j] - v["S1"][j]) <= 1e-5 * max(v["S1"][j], 1e-12) + 1e-12
            if proj is not None:
                assert abs(S2[b, j] - v["S2"][j]) <= 1e-5 * math.sqrt(max(v["S1"][j], 1e-12)) * 8 + 1e-9
            gacc = bool((int(accmask[b]) >> j) & 1)
            stats["tests"] += 1
            if amb[j]:
                stats["band"] += 1
            else:
                assert gacc == bool(v["acc"][j]), (b, j)
        if not amb.any():
            assert int(jstar[b]) == v["jstar"]
        js = int(jstar[b])
        assert 1 <= js <= Lt + 1
        if js <= Lt and js == v["jstar"]:
            got = X2[r0 + js] if js < Lt else T2[b]
            assert_rows_close(got, v["Y_reflect"], 1e-5, (b, js))
            stats["reflected"] += 1
            if proj is not None:
                continue
            # reflection is an isometry about the target mean
            k = nb + js - 1
            m_q = a64[k] * W[js - 1] + c64[k] * Dq[r0 + js - 1].astype(np.float64)
            m_p = a64[k] * W[js - 1] + c64[k] * (Dp[r0 + js - 1] if draft_den is not None else Dc[b]).astype(np.float64)
            assert abs(np.linalg.norm(got - m_q) - np.linalg.norm(W[js] - m_p)) <= 1e-4 * np.linalg.norm(W[js] - m_p) + 1e-6
        # rows other than the reflected one are untouched
        for j in range(Lt + 1):
            if j != js:
                assert np.array_equal(X2[r0 + j] if j < Lt else T2[b], X[r0 + j] if j < Lt else T[b])
    n_before = n.copy()
    na2 = s.advance()
    n2, Y2, Dc2 = s.get(sb.GET_N), s.get(sb.GET_Y), s.get(sb.GET_DC)
    for si, b in enumerate(act):
        if chains is not None and int(b) not in chains:
            continue
        nb = int(n_before[b]); Lt = min(L, K - nb); r0 = int(rowoff[si])
        adv = min(int(jstar[b]), Lt)
        assert n2[b] == nb + adv
        assert np.array_equal(Y2[b], X2[r0 + adv] if adv < Lt else T2[b])
        assert np.array_equal(Dc2[b], Dq[r0 + adv - 1])          # carry rule (unused by the other drafters)
    assert na2 == int(np.sum(n2 < K))
    return na2


SHAPES = [
    # name, B, d, L, K, ncomp, windows
    ("cfg1", 64, 2, 4, 100, 4, 6),
    ("cfg2", 96, 64, 8, 200, 16, 4),
    ("cfg2", 65, 33, 5, 23, 7, 8),
    ("cfg2", 3, 5, 2, 9, 3, 9),
    ("cfg1", 1, 1, 1, 6, 2, 6),
    ("cfg2", 9, 3, 32, 70, 4, 5),
    ("cfg5", 20, 1024, 6, 40, 12, 4),
    ("cfg5", 7, 516, 32, 64, 5, 3),
    ("cfg2", 5, 1030, 3, 11, 6, 5),
    ("cfg2", 4, 8, 8, 3, 4, 1),          # the whole chain is shorter than one window
    ("cfg5", 3, 2052, 32, 5, 3, 1),      # same, one CTA per chain
]


@pytest.mark.parametrize("name,B,d,L,K,ncomp,windows", SHAPES)
def test_window_forced_parity(name, B, d, L, K, ncomp, windows):
    w = wl.WORKLOADS[name].scaled(B=B, d=d, L=L, K=K)
    gp = w.gmm_params(d=d, ncomp=ncomp)
    seed, off = 4242 + d, 1000
    s = sds.sampler_for(w, gmm=gp, seed=seed, chain_id_offset=off)
    den, a, c, sig = oracle_setup(w, gmm=gp)
    a32, c32, s32, _ = sds.schedule_for(w)
    s.reset()
    # initial state and carried output
    Y0, Dc0 = s.get(sb.GET_Y), s.get(sb.GET_DC)
    for b in range(min(B, 8)):
        want = o.normals(seed, o.STREAM_INIT, off + b, 0, d)
        assert np.max(np.abs(Y0[b] - want)) <= 3e-6
        assert_rows_close(Dc0[b], den(Y0[b].astype(np.float64), 0), 1e-5, b)
    stats = dict(tests=0, band=0, reflected=0)
    na = B
    for _ in range(windows):
        if na == 0:
            break
        na = _window_check(s, w, den, a32, c32, s32, seed, off, stats)
    assert stats["band"] <= max(2, 2e-3 * stats["tests"])
    assert stats.get("exact", 0) >= 0.99 * stats["tests"]        # decisions replayed exactly on the kernel's own Delta and Z
    print(f"band events {stats['band']} of {stats['tests']} tests; {stats.get('exact', 0)} decisions replayed exactly")
    s.close()


@pytest.mark.parametrize("name", ["cfg2", "cfg5"])
def test_full_size_windows_on_sampled_chains(name):
    """The window kernels at the benchmark's full sizes and launch shapes; the oracle replays a
    sample of chains (every position of their windows)."""
    w = wl.WORKLOADS[name]
    gp = w.gmm_params()
    s = sds.sampler_for(w, gmm=gp)
    den, a, c, sig = oracle_setup(w, gmm=gp)
    a32, c32, s32, _ = sds.schedule_for(w)
    rng = np.random.default_rng(5)
    chains = set(int(x) for x in rng.choice(w.B, size=6, replace=False)) | {0, w.B - 1}
    s.reset()
    stats = dict(tests=0, band=0, reflected=0)
    for _ in range(2):
        _window_check(s, w, den, a32, c32, s32, w.sample_seed, 0, stats, chains=chains)
    assert stats["tests"] >= 8 * w.L and stats["band"] <= 2
    s.close()


def test_full_size_cfg5_free_run_sampled():
    w = wl.WORKLOADS["cfg5"]
    out, calls, rows = _free_run_compare(w, w.gmm_params(), [3, 8191], w.sample_seed)
    assert np.all(calls <= 1 + w.K) and calls.mean() < 0.2 * w.K


# ------------------------------------------------------------------ free running ---------

def _free_run_compare(w, gp, chains, seed, off=0, B=None):
    torch = _torch()
    s = sds.sampler_for(w, gmm=gp, seed=seed, chain_id_offset=off, B=B)
    out, calls, rows = s.sample_all()
    out, calls, rows = out.cpu().numpy(), calls.cpu().numpy(), rows.cpu().numpy()
    assert np.all(np.isfinite(out))
    assert np.array_equal(s.get(sb.GET_N), np.full(s.B, w.K))
    den, a, c, sig = oracle_setup(w, gmm=gp)
    diverged = 0
    for b in chains:
        r = o.speculative_chain(den, a, c, sig, w.L, seed, off + b, w.d, record=True)
        diverged += not chain_matches_or_band(r, calls[b], rows[b], out[b])
        # counters are consistent on their own
        assert calls[b] >= 1 + math.ceil(w.K / w.L) and rows[b] >= w.K + 1 - 0
    assert diverged <= max(1, len(chains) // 20)
    s.close()
    return out, calls, rows


def test_free_running_cfg1_all_chains():
    w = wl.WORKLOADS["cfg1"]
    _free_run_compare(w, w.gmm_params(), range(w.B), w.sample_seed)


def test_free_running_cfg2_sampled_chains():
    w = wl.WORKLOADS["cfg2"]
    rng = np.random.default_rng(0)
    chains = sorted(rng.choice(w.B, size=24, replace=False).tolist())
    out, calls, rows = _free_run_compare(w, w.gmm_params(), chains, w.sample_seed)
    # whole-batch properties at full size
    assert np.all(calls <= 1 + w.K) and np.all(rows <= 1 + w.K * w.L)
    assert calls.mean() < 1 + w.K          # speculation saves sequential calls


def test_free_running_ula_small():
    w = wl.WORKLOADS["cfg5"].scaled(B=12, d=128, K=120, L=16)
    gp = w.gmm_params(d=128, ncomp=12)
    _free_run_compare(w, gp, range(12), 99)


def test_stepwise_loop_equals_sample_all_and_is_deterministic():
    w = wl.WORKLOADS["cfg2"].scaled(B=200, K=60)
    gp = w.gmm_params()
    s = sds.sampler_for(w, gmm=gp, seed=5)
    o1, c1, r1 = [x.cpu().numpy() for x in s.sample_all()]
    o2, c2, r2 = [x.cpu().numpy() for x in s.sample_all()]
    assert np.array_equal(o1, o2) and np.array_equal(c1, c2) and np.array_equal(r1, r2)
    s.reset()
    na, windows = s.B, 0
    while na > 0:
        s.draft(); s.verify_window(); na = s.advance(); windows += 1
        assert windows <= w.K
    assert np.array_equal(s.get(sb.GET_Y), o1)
    assert np.array_equal(s.get(sb.GET_NFE_CALLS), c1) and np.array_equal(s.get(sb.GET_NFE_ROWS), r1)
    assert int(s.get(sb.GET_CTL)[2]) == windows
    s.close()


FUSED_SHAPES = [(64, 2, 4, 100, 4), (300, 64, 8, 200, 16), (65, 33, 5, 23, 7), (3, 5, 2, 9, 3), (1, 1, 1, 6, 2),
                (9, 3, 32, 70, 4), (20, 128, 6, 40, 20), (10, 256, 4, 30, 32), (40, 16, 8, 50, 16), (40, 20, 8, 50, 17),
                (33, 68, 3, 31, 9), (4, 8, 8, 3, 4)]


@pytest.mark.parametrize("B,d,L,K,ncomp,ncomp_d", [(40, 64, 8, 60, 16, 8), (9, 33, 5, 23, 7, 20), (3, 5, 2, 9, 3, 1),
                                                   (12, 128, 6, 40, 20, 32), (17, 16, 32, 70, 16, 16)])
def test_whole_chain_kernel_with_independent_drafter_equals_window_kernels_bitwise(B, d, L, K, ncomp, ncomp_d):
    for name in ("cfg2", "cfg5"):
        w = wl.WORKLOADS[name].scaled(B=B, d=d, L=L, K=K)
        gp = w.gmm_params(d=d, ncomp=ncomp)
        gd = wl.gmm_params(4321, ncomp_d, d, w.gmm["mean_scale"] * 1.1, w.gmm["comp_std"] * 1.3)
        res = {}
        for fused in (1, 0):
            s = sds.sampler_for(w, gmm=gp, seed=91 + d, chain_id_offset=3, drafter=sds.drafter_for(w, gmm=gd))
            s.set_option(s.OPT_WHOLE_CHAIN_KERNEL, fused)
            l0 = s.launch_count()
            res[fused] = [x.cpu().numpy() for x in s.sample_all()] + [s.launch_count() - l0]
            s.close()
        assert all(np.array_equal(x, y) for x, y in zip(res[1][:3], res[0][:3]))
        assert res[1][3] <= 3 < res[0][3]


@pytest.mark.parametrize("B,d,L,K,ncomp", FUSED_SHAPES)
def test_whole_chain_kernel_equals_window_kernels_bitwise(B, d, L, K, ncomp):
    for name in ("cfg2", "cfg5"):
        for mode in (sb.SDS_FROZEN_PREV, sb.SDS_FROZEN_EXACT):       # carried output; target evaluated at Y_n
            w = wl.WORKLOADS[name].scaled(B=B, d=d, L=L, K=K)
            gp = w.gmm_params(d=d, ncomp=ncomp)
            s = sds.sampler_for(w, gmm=gp, seed=77 + d, chain_id_offset=5, drafter_mode=mode)
            l0 = s.launch_count()
            f = [x.cpu().numpy() for x in s.sample_all()]
            assert s.launch_count() - l0 <= 2                           # one kernel (plus the |mu|^2 table once)
            s.set_option(s.OPT_WHOLE_CHAIN_KERNEL, 0)
            g = [x.cpu().numpy() for x in s.sample_all()]
            assert np.array_equal(f[0], g[0]) and np.array_equal(f[1], g[1]) and np.array_equal(f[2], g[2])
            assert np.all(np.isfinite(f[0]))
            s.close()


def test_chain_shards_reproduce_the_unsharded_run_bitwise():
    w = wl.WORKLOADS["cfg2"].scaled(B=96, K=50)
    gp = w.gmm_params()
    full = sds.sampler_for(w, gmm=gp, seed=11)
    of, cf, rf = [x.cpu().numpy() for x in full.sample_all()]
    parts = []
    for off, nb in ((0, 40), (40, 56)):
        s = sds.sampler_for(w, gmm=gp, seed=11, chain_id_offset=off, B=nb)
        parts.append([x.cpu().numpy() for x in s.sample_all()])
        s.close()
    assert np.array_equal(np.concatenate([p[0] for p in parts]), of)
    assert np.array_equal(np.concatenate([p[1] for p in parts]), cf)
    assert np.array_equal(np.concatenate([p[2] for p in parts]), rf)
    full.close()


def test_identical_drafter_and_target_accepts_everything():
    """With c_k = 0 the draft and target means coincide (Delta = 0): every draft is accepted and
    every window advances by its full length."""
    w = wl.WORKLOADS["cfg2"].scaled(B=32, K=30)
    gp = w.gmm_params()
    a, c, sig, tcond = sds.schedule_for(w)
    s = sb.Sampler(a, np.zeros_like(c), sig, 32, w.d, w.L, gmm_means=gp.means, gmm_logw=gp.logw, tcond=tcond, seed=3)
    out, calls, rows = s.sample_all()
    assert np.array_equal(calls.cpu().numpy(), np.full(32, 1 + math.ceil(30 / w.L)))
    s.set_option(s.OPT_WHOLE_CHAIN_KERNEL, 0)          # window-by-window kernels keep S1 for inspection
    out, calls, rows = s.sample_all()
    # Delta = 0 everywhere: every window is accepted in full
    assert np.array_equal(calls.cpu().numpy(), np.full(32, 1 + math.ceil(30 / w.L)))
    assert np.all(s.get(sb.GET_S1) == 0.0)
    s.close()


def test_call_order_is_enforced():
    w = wl.WORKLOADS["cfg1"]
    s = sds.sampler_for(w)
    lib = s.lib
    assert lib.sds_draft(s.h) == sb.SDS_ESTATE
    s.reset()
    assert lib.sds_verify_window(s.h) == sb.SDS_ESTATE
    assert lib.sds_advance(s.h, None) == sb.SDS_ESTATE
    s.draft()
    assert lib.sds_draft(s.h) == sb.SDS_ESTATE
    s.verify_window()
    assert lib.sds_reset(s.h) == sb.SDS_OK
    s.close()


def test_set_state_resume_is_bitwise():
    torch = _torch()
    w = wl.WORKLOADS["cfg2"].scaled(B=50, K=40)
    gp = w.gmm_params()
    s = sds.sampler_for(w, gmm=gp, seed=21)
    ref = s.sample_all()[0].cpu().numpy()
    s.reset()
    for _ in range(3):
        s.draft(); s.verify_window(); s.advance()
    Y, n, Dc = (torch.from_numpy(s.get(x)).cuda() for x in (sb.GET_Y, sb.GET_N, sb.GET_DC))
    s2 = sds.sampler_for(w, gmm=gp, seed=21)
    s2.reset()
    s2.set_state(Y, n, Dc)
    na = 1
    while na > 0:
        s2.draft(); s2.verify_window(); na = s2.advance()
    assert np.array_equal(s2.get(sb.GET_Y), ref)
    s.close(); s2.close()


# ------------------------------------------------------------------ callback denoiser, failures ---

class _DevArray:
    """Zero-copy view of device memory handed to a callback (CUDA array interface)."""

    def __init__(self, ptr, shape, typestr):
        self.__cuda_array_interface__ = {"data": (int(ptr), False), "shape": tuple(shape), "typestr": typestr,
                                         "version": 2, "strides": None}


def _make_callback(torch, means_t, logw_t, tcond_t, poison_row=None, fail=False):
    """User denoiser written with torch ops on the library's stream: the same mixture formula."""
    state = {"poisoned": False}

    def cb(user, x_ptr, k_ptr, rows, d, out_ptr, stream):
        if fail:
            return 7
        with torch.cuda.stream(torch.cuda.ExternalStream(int(stream or 0))):
            x = torch.as_tensor(_DevArray(x_ptr, (rows, d), "<f4"), device="cuda")
            k = torch.as_tensor(_DevArray(k_ptr, (rows,), "<i4"), device="cuda").long()
            out = torch.as_tensor(_DevArray(out_ptr, (rows, d), "<f4"), device="cuda")
            tc = tcond_t[k]                                              # [rows, 4] double
            xd = x.double()
            lg = logw_t.double()[None, :] + tc[:, 0:1] * (xd @ means_t.double().T) \
                + tc[:, 1:2] * (means_t.double() ** 2).sum(1)[None, :]
            r = torch.softmax(lg, dim=1)
            res = tc[:, 2:3] * (r @ means_t.double()) + tc[:, 3:4] * xd
            if poison_row is not None and not state["poisoned"] and rows > poison_row:
                res[poison_row] = float("nan")            # only the first (initial) target call is hit
                state["poisoned"] = True
            out.copy_(res.float())
        return 0
    return cb


def test_callback_denoiser_matches_builtin_mixture_and_oracle():
    torch = _torch()
    w = wl.WORKLOADS["cfg2"].scaled(B=40, K=30)
    gp = w.gmm_params()
    a, c, sig, tcond = sds.schedule_for(w)
    means_t, logw_t = torch.from_numpy(gp.means).cuda(), torch.from_numpy(gp.logw).cuda()
    tcond_t = torch.from_numpy(tcond).cuda()
    s_cb = sb.Sampler(a, c, sig, 40, w.d, w.L, callback=_make_callback(torch, means_t, logw_t, tcond_t), seed=9)
    out, calls, rows = [x.cpu().numpy() for x in s_cb.sample_all()]
    den, ao, co, so = oracle_setup(w, gmm=gp)
    bad = 0
    for b in range(12):
        r = o.speculative_chain(den, ao, co, so, w.L, 9, b, w.d, record=True)
        bad += not chain_matches_or_band(r, calls[b], rows[b], out[b])
    assert bad <= 1
    s_cb.close()


def test_non_finite_target_output_freezes_only_that_chain():
    torch = _torch()
    w = wl.WORKLOADS["cfg2"].scaled(B=16, K=24)
    gp = w.gmm_params()
    a, c, sig, tcond = sds.schedule_for(w)
    means_t, logw_t = torch.from_numpy(gp.means).cuda(), torch.from_numpy(gp.logw).cuda()
    tcond_t = torch.from_numpy(tcond).cuda()
    clean = sb.Sampler(a, c, sig, 16, w.d, w.L, callback=_make_callback(torch, means_t, logw_t, tcond_t), seed=4)
    ref = clean.sample_all()[0].cpu().numpy()
    # row 3 of the initial target call is poisoned: chain 3 starts with a NaN carried output
    s = sb.Sampler(a, c, sig, 16, w.d, w.L, callback=_make_callback(torch, means_t, logw_t, tcond_t, poison_row=3), seed=4)
    out_t = torch.empty((16, w.d), dtype=torch.float32, device="cuda")
    rc = s.lib.sds_sample_all(s.h, out_t.data_ptr(), None, None)
    assert rc == sb.SDS_ENONFINITE
    ctl = s.get(sb.GET_CTL)
    assert ctl[0] == 0 and ctl[4] == 1                      # nobody active, exactly one chain frozen
    assert np.array_equal(s.get(sb.GET_N), np.full(16, w.K))
    out = out_t.cpu().numpy()
    # every other chain is bit-identical to the clean run
    same = [b for b in range(16) if np.array_equal(out[b], ref[b])]
    assert same == [b for b in range(16) if b != 3]
    clean.close(); s.close()


def test_failing_callback_is_reported():
    torch = _torch()
    w = wl.WORKLOADS["cfg1"].scaled(K=10)
    a, c, sig, _ = sds.schedule_for(w)
    s = sb.Sampler(a, c, sig, 8, w.d, w.L, callback=_make_callback(torch, None, None, None, fail=True), seed=1)
    assert s.lib.sds_reset(s.h) == sb.SDS_ECALLBACK
    s.close()


# ------------------------------------------------------------------ main-text frozen drafter ---

def test_exact_frozen_drafter_matches_oracle():
    w = wl.WORKLOADS["cfg2"].scaled(B=48, K=40)
    gp = w.gmm_params()
    s = sds.sampler_for(w, gmm=gp, seed=13, drafter_mode=sb.SDS_FROZEN_EXACT)
    # one window by hand: position 1 compares the frozen output with itself and always accepts
    s.reset()
    s.draft(); s.verify_window()
    assert np.all(s.get(sb.GET_ACCMASK) & 1 == 1)
    assert np.all(s.get(sb.GET_S1)[:, 0] == 0.0)
    s.advance()
    out, calls, rows = [x.cpu().numpy() for x in s.sample_all()]
    den, a, c, sig = oracle_setup(w, gmm=gp)
    bad = 0
    for b in range(16):
        r = o.speculative_chain(den, a, c, sig, w.L, 13, b, w.d, mode=o.FROZEN_EXACT, record=True)
        bad += not chain_matches_or_band(r, calls[b], rows[b], out[b])
    assert bad <= 1
    s.close()


def test_exact_frozen_drafter_with_window_one_is_the_plain_chain():
    w = wl.WORKLOADS["cfg2"].scaled(B=8, K=25, L=1)
    gp = w.gmm_params()
    s = sds.sampler_for(w, gmm=gp, seed=17, drafter_mode=sb.SDS_FROZEN_EXACT)
    out, calls, rows = [x.cpu().numpy() for x in s.sample_all()]
    den, a, c, sig = oracle_setup(w, gmm=gp)
    assert np.all(calls == 25) and np.all(rows == 25)
    for b in range(8):
        y = o.plain_chain(den, a, c, sig, seed=17, b=b, d=w.d)
        assert rel_l2(out[b], y) <= 1e-4
    s.close()


# ------------------------------------------------------------------ independent drafter ----------

def _cheap_mixture(w, gp, keep):
    """A cheaper draft model: the first `keep` components, slightly displaced and wider."""
    return wl.GmmParams(means=(gp.means[:keep] * 1.05).astype(np.float32), logw=np.full(keep, -math.log(keep), np.float32),
                        comp_std=gp.comp_std * 1.3)


def _oracle_cheap(w, cheap):
    if w.sampler == "ddpm":
        abar = o.ddpm_affine(w.beta())[3]
        return lambda x, k: o.gmm_posterior_mean(x, abar[k], cheap.means, cheap.logw, cheap.comp_std)
    return lambda x, k: o.gmm_grad_energy(x, cheap.means, cheap.logw, cheap.comp_std)


@pytest.mark.parametrize("name,B,d,L,K,ncomp,keep", [("cfg2", 40, 64, 8, 60, 16, 6), ("cfg2", 9, 33, 5, 23, 7, 3),
                                                     ("cfg5", 12, 512, 6, 40, 40, 12)])
def test_independent_drafter_windows_and_free_run(name, B, d, L, K, ncomp, keep):
    w = wl.WORKLOADS[name].scaled(B=B, d=d, L=L, K=K)
    gp = w.gmm_params(d=d, ncomp=ncomp)
    cheap = _cheap_mixture(w, gp, keep)
    s = sds.sampler_for(w, gmm=gp, seed=23, drafter=sds.drafter_for(w, gmm=cheap))
    den, a, c, sig = oracle_setup(w, gmm=gp)
    dden = _oracle_cheap(w, cheap)
    a32, c32, s32, _ = sds.schedule_for(w)
    s.reset()
    stats = dict(tests=0, band=0, reflected=0)
    for _ in range(3):
        _window_check(s, w, den, a32, c32, s32, 23, 0, stats, draft_den=dden)
    assert stats["band"] <= 2
    out, calls, rows = [x.cpu().numpy() for x in s.sample_all()]
    bad = 0
    for b in range(min(B, 10)):
        r = o.speculative_chain(den, a, c, sig, L, 23, b, d, mode=o.INDEPENDENT, draft_denoise=dden, record=True)
        bad += not chain_matches_or_band(r, calls[b], rows[b], out[b])
    assert bad <= 1
    s.close()


def test_independent_drafter_equal_to_target_accepts_everything():
    w = wl.WORKLOADS["cfg2"].scaled(B=20, K=50)
    gp = w.gmm_params()
    s = sds.sampler_for(w, gmm=gp, seed=29, drafter=sds.drafter_for(w, gmm=gp))
    out, calls, rows = [x.cpu().numpy() for x in s.sample_all()]
    assert np.all(calls == math.ceil(50 / w.L)) and np.all(rows == 50)
    den, a, c, sig = oracle_setup(w, gmm=gp)
    for b in range(6):
        assert rel_l2(out[b], o.plain_chain(den, a, c, sig, seed=29, b=b, d=w.d)) <= 1e-4
    s.close()


def test_independent_mlp_drafter_for_mlp_target_runs():
    dims, ddims = [256, 384, 384, 256], [256, 128, 256]
    w = wl.WORKLOADS["cfg3"].scaled(d=256, B=64, L=4, K=24, mlp_dims=dims)
    mp = w.mlp_params()
    dmp = wl.mlp_params(77, ddims, 24)
    s = sds.sampler_for(w, mlp=mp, seed=5, drafter=sds.drafter_for(w, mlp=dmp))
    out, calls, rows = [x.cpu().numpy() for x in s.sample_all()]
    assert np.all(np.isfinite(out)) and np.array_equal(s.get(sb.GET_N), np.full(64, 24))
    assert np.all(calls >= 6) and np.all(calls <= 24) and np.all(rows >= 24)
    s.close()


# ------------------------------------------------------------------ temperature variant ----------

@pytest.mark.parametrize("tau", [0.5, 2.0])
def test_temperature_variant_matches_oracle(tau):
    w = wl.WORKLOADS["cfg2"].scaled(B=64, K=40)
    gp = w.gmm_params()
    den, a, c, sig = oracle_setup(w, gmm=gp)
    res = {}
    for fused in (1, 0):
        s = sds.sampler_for(w, gmm=gp, seed=37)
        s.set_temperature(tau)
        s.set_option(s.OPT_WHOLE_CHAIN_KERNEL, fused)
        res[fused] = [x.cpu().numpy() for x in s.sample_all()]
        if not fused:                                   # tempered log ratio is what the library reports
            s.reset(); s.draft(); s.verify_window()
            ell, S1, S2 = s.get(sb.GET_ELL), s.get(sb.GET_S1), s.get(sb.GET_S2)
            assert np.allclose(ell, (-0.5 * S1 - S2) / tau, rtol=1e-6, atol=1e-6)
        s.close()
    assert all(np.array_equal(x, y) for x, y in zip(res[0], res[1]))
    out, calls, rows = res[1]
    bad = 0
    for b in range(12):
        r = o.speculative_chain(den, a, c, sig, w.L, 37, b, w.d, tau=tau, record=True)
        bad += not chain_matches_or_band(r, calls[b], rows[b], out[b])
    assert bad <= 1
    # a higher temperature accepts more
    if tau > 1:
        s = sds.sampler_for(w, gmm=gp, seed=37)
        base = s.sample_all()[1].cpu().numpy()
        assert calls.mean() < base.mean()
        s.close()


# ----------------------------------------------------------------------------------------
# acceptance ratio decided in a subspace (Appendix F)
# ----------------------------------------------------------------------------------------


@pytest.mark.gpu
@pytest.mark.parametrize("d,r", [(64, 5), (1030, 7), (3072, 16)])
def test_projected_ratio_matches_oracle(d, r):
    import torch
    w = wl.WORKLOADS["cfg2"].scaled(B=24, d=d, K=24, L=6)
    gp = w.gmm_params(d=d)
    den, a, c, sig = oracle_setup(w, gmm=gp)
    a32, c32, s32 = [np.asarray(v, dtype=np.float32) for v in (a, c, sig)]
    A = np.random.default_rng(5).standard_normal((r, d))
    Q = sds.projection_basis(A)
    assert Q.shape == (r, d) and np.allclose(Q @ Q.T, np.eye(r), atol=1e-5)
    s = sds.sampler_for(w, gmm=gp, seed=41)
    s.set_projection(torch.from_numpy(Q).cuda())
    stats = dict(tests=0, band=0, reflected=0)
    s.reset()
    for _ in range(4):
        _window_check(s, w, den, a32, c32, s32, 41, 0, stats, chains=set(range(8)), proj=A)
    assert stats["reflected"] >= 1 and stats["band"] <= 2
    # whole run against the oracle's chain with the same matrix
    out, calls, rows = [x.cpu().numpy() for x in s.sample_all()]
    bad = 0
    for b in range(6):
        ref = o.speculative_chain(den, a, c, sig, w.L, 41, b, d, proj=A, record=True)
        bad += not chain_matches_or_band(ref, calls[b], rows[b], out[b])
    assert bad <= 1
    # deciding in a low-dimensional image accepts more than the full-space test
    s.set_projection(None)
    full = s.sample_all()[1].cpu().numpy()
    assert calls.mean() < full.mean()
    s.close()


@pytest.mark.gpu
def test_projection_onto_the_whole_space_is_the_exact_method():
    import torch
    w = wl.WORKLOADS["cfg2"].scaled(B=32, K=30)
    gp = w.gmm_params()
    s = sds.sampler_for(w, gmm=gp, seed=43)
    s.set_option(s.OPT_WHOLE_CHAIN_KERNEL, 0)
    base = [x.cpu().numpy() for x in s.sample_all()]
    Q = sds.projection_basis(np.random.default_rng(6).standard_normal((w.d, w.d)))
    s.set_projection(torch.from_numpy(Q).cuda())
    s.reset(); s.draft(); s.verify_window()
    S1p, S2p = s.get(sb.GET_S1), s.get(sb.GET_S2)
    s.set_projection(None)
    s.reset(); s.draft(); s.verify_window()
    S1, S2 = s.get(sb.GET_S1), s.get(sb.GET_S2)
    assert np.allclose(S1p, S1, rtol=1e-4, atol=1e-9) and np.allclose(S2p, S2, rtol=1e-3, atol=1e-5)
    s.set_projection(torch.from_numpy(Q).cuda())
    got = [x.cpu().numpy() for x in s.sample_all()]
    same = np.sum(got[1] == base[1])
    assert same >= w.B - 2                              # decisions can differ only inside the rounding band
    s.close()


# ----------------------------------------------------------------------------------------
# verify with early exit (blocks of positions; nothing after the block of the first rejection is read)
# ----------------------------------------------------------------------------------------


@pytest.mark.gpu
@pytest.mark.parametrize("d,L,B", [(1024, 12, 40), (3072, 8, 24), (4096, 16, 12), (16384, 16, 6)])
def test_verify_early_exit_only_skips_diagnostics(d, L, B):
    w = wl.WORKLOADS["cfg2"].scaled(B=B, d=d, K=3 * L + 5, L=L)
    gp = w.gmm_params(d=d, ncomp=8)
    res = {}
    for early in (1, 0):
        s = sds.sampler_for(w, gmm=gp, seed=61)
        s.set_option(s.OPT_VERIFY_EARLY_EXIT, early)
        s.reset()
        wins = []
        for _ in range(3):
            s.draft(); s.verify_window()
            wins.append(dict(n=s.get(sb.GET_N).copy(), X=s.get(sb.GET_X).copy(), T=s.get(sb.GET_TAIL).copy(),
                             js=s.get(sb.GET_JSTAR).copy(), am=s.get(sb.GET_ACCMASK).copy(), S1=s.get(sb.GET_S1).copy(),
                             S2=s.get(sb.GET_S2).copy(), ell=s.get(sb.GET_ELL).copy(), lu=s.get(sb.GET_LOGU).copy()))
            s.advance()
        full = [x.cpu().numpy() for x in s.sample_all()]
        res[early] = (wins, full)
        s.close()
    skipped = 0
    blk = 2 if d >= 2048 else 4
    for a, b in zip(res[1][0], res[0][0]):
        assert np.array_equal(a["n"], b["n"]) and np.array_equal(a["js"], b["js"])
        assert np.array_equal(a["X"], b["X"]) and np.array_equal(a["T"], b["T"])      # same reflected states
        for c in range(B):
            Lt = min(L, w.K - int(a["n"][c]))
            js = int(a["js"][c])
            if js > Lt:
                n_eval = Lt
            elif d >= 2048:                                   # blocks {1}, {2, 3}, {4, 5}, ...
                n_eval = 1 if js == 1 else min(Lt, 1 + 2 * (js // 2))
            else:                                             # blocks {1..4}, {5..8}, ...
                n_eval = min(Lt, blk * ((js + blk - 1) // blk))
            keep = (1 << n_eval) - 1
            assert int(a["am"][c]) == int(b["am"][c]) & keep
            for key in ("S1", "S2", "ell", "lu"):
                assert np.array_equal(a[key][c, :n_eval], b[key][c, :n_eval])
                assert not np.any(a[key][c, n_eval:Lt])
            skipped += Lt - n_eval
    assert skipped > 0                                                                # the case does skip positions
    assert all(np.array_equal(x, y) for x, y in zip(res[1][1], res[0][1]))            # whole runs agree bit for bit


@pytest.mark.gpu
def test_early_exit_run_matches_oracle():
    w = wl.WORKLOADS["cfg2"].scaled(B=16, d=1024, K=40, L=12)
    gp = w.gmm_params(d=1024, ncomp=6)
    den, a, c, sig = oracle_setup(w, gmm=gp)
    s = sds.sampler_for(w, gmm=gp, seed=62)
    out, calls, rows = [x.cpu().numpy() for x in s.sample_all()]
    bad = 0
    for b in range(6):
        r = o.speculative_chain(den, a, c, sig, w.L, 62, b, w.d, record=True)
        bad += not chain_matches_or_band(r, calls[b], rows[b], out[b])
    assert bad <= 1
    s.close()


@pytest.mark.gpu
@pytest.mark.parametrize("d,L,B,mode", [(64, 8, 70, 0), (1024, 12, 40, 0), (2048, 7, 9, 0), (3072, 8, 24, 1), (3072, 8, 24, 0), (4096, 16, 12, 0), (8192, 6, 5, 0),
                          (16384, 5, 6, 0), (12292, 5, 6, 0), (5000, 6, 5, 0)])
def test_sample_all_with_fused_advance_equals_the_stepwise_calls(d, L, B, mode):
    """sds_sample_all (verify kernel advancing its chains, early exit on) against an explicit
    draft / verify / advance loop, and against the same run with the advance kernel: same bits.
    (A float mixture reads the float rows, so the drafted states are read back here whatever the
    option says; the bf16 targets' test covers the other path.)"""
    w = wl.WORKLOADS["cfg2"].scaled(B=B, d=d, K=3 * L + 7, L=L)
    gp = w.gmm_params(d=d, ncomp=8)
    s = sds.sampler_for(w, gmm=gp, seed=71, drafter_mode=mode)
    s.set_option(s.OPT_WHOLE_CHAIN_KERNEL, 0)
    got = [x.cpu().numpy() for x in s.sample_all()]
    windows_fused = int(s.get(sb.GET_CTL)[2])
    s.set_option(s.OPT_REGEN_DRAFTS, 0)                    # fused advance with the drafted states read back
    mid = [x.cpu().numpy() for x in s.sample_all()]
    assert all(np.array_equal(x, y) for x, y in zip(got, mid))
    s.set_option(s.OPT_FUSE_ADVANCE, 0)
    ref = [x.cpu().numpy() for x in s.sample_all()]
    assert all(np.array_equal(x, y) for x, y in zip(got, ref))
    assert windows_fused == int(s.get(sb.GET_CTL)[2])
    s.reset()
    na = B
    while na > 0:
        s.draft(); s.verify_window(); na = s.advance()
    assert np.array_equal(s.get(sb.GET_Y), got[0])
    assert np.array_equal(s.get(sb.GET_NFE_CALLS), got[1]) and np.array_equal(s.get(sb.GET_NFE_ROWS), got[2])
    s.close()


# ----------------------------------------------------------------------------------------
# laws on the GPU at scale
# ----------------------------------------------------------------------------------------


@pytest.mark.gpu
def test_gpu_normals_follow_the_standard_normal_law():
    """The library's normals use hardware approximations of log, sqrt, sin and cos: their law is
    checked directly (Kolmogorov-Smirnov, moments, independence of neighbours)."""
    from scipy import stats
    z = sb.rng_normals(20250101, o.STREAM_DRAFT, 0, 2048, 3, 1024).cpu().numpy().astype(np.float64).ravel()
    n = z.size
    assert stats.kstest(z[:400_000], stats.norm.cdf).pvalue > 1e-3
    assert abs(z.mean()) < 5 / math.sqrt(n) and abs(z.var() - 1) < 5 * math.sqrt(2 / n)
    assert abs(np.mean(z ** 4) - 3) < 5 * math.sqrt(96 / n)
    pairs = z.reshape(-1, 2)                               # the two outputs of one Box-Muller pair
    assert abs(np.mean(pairs[:, 0] * pairs[:, 1])) < 5 / math.sqrt(n / 2)
    assert abs(np.mean(z[:-1] * z[1:])) < 5 / math.sqrt(n)


@pytest.mark.gpu
def test_speculative_and_plain_chains_agree_in_law_on_the_gpu():
    """cfg2 at full batch: window 8 with the carried-output drafter against the plain sequential
    chain (window 1 with the drafter evaluated at Y_n, which accepts every step) under another seed."""
    w = wl.WORKLOADS["cfg2"]
    gp = w.gmm_params()
    s = sds.sampler_for(w, gmm=gp, seed=101)
    S = s.sample_all()[0].cpu().numpy().astype(np.float64)
    s.close()
    wp = w.scaled(L=1)
    p = sds.sampler_for(wp, gmm=gp, seed=202, drafter_mode=sb.SDS_FROZEN_EXACT)
    outp, calls, _ = p.sample_all()
    P = outp.cpu().numpy().astype(np.float64)
    assert np.all(calls.cpu().numpy() == w.K)              # one target call per step: the plain chain
    p.close()
    B = w.B
    se = np.sqrt(S.var(axis=0) / B + P.var(axis=0) / B)
    zmean = (S.mean(axis=0) - P.mean(axis=0)) / se
    assert np.max(np.abs(zmean)) < 4.5 and abs(zmean.mean()) < 4 / math.sqrt(w.d)
    rv = S.var(axis=0) / P.var(axis=0)
    assert np.max(np.abs(rv - 1)) < 6 * math.sqrt(2 / B) * 2
    # a random projection, compared as distributions
    u = np.random.default_rng(0).standard_normal(w.d); u /= np.linalg.norm(u)
    from scipy import stats
    assert stats.ks_2samp(S @ u, P @ u).pvalue > 1e-3


@pytest.mark.gpu
@pytest.mark.parametrize("d", [2, 8, 32])
def test_sequential_target_calls_fall_with_the_window_size(d):
    """Section 7, low-dimensional mixtures (16 components, 200 steps): the number of sequential
    target calls falls as the window grows, and window 1 is the plain chain's count."""
    calls = []
    for L in (1, 2, 4, 8, 16):
        w = wl.WORKLOADS["cfg2"].scaled(B=512, d=d, L=L)
        s = sds.sampler_for(w, gmm=w.gmm_params(d=d), seed=5)
        calls.append(float(s.sample_all()[1].float().mean().item()))
        s.close()
    assert calls[0] == 1 + 200
    assert all(a > b for a, b in zip(calls, calls[1:])), calls
    assert calls[-1] < 0.6 * 200


# ----------------------------------------------------------------------------------------
# staged windows: the same window evaluated a few positions per launch
# ----------------------------------------------------------------------------------------


@pytest.mark.gpu
@pytest.mark.parametrize("d,L,B", [(64, 8, 70), (1000, 12, 20), (1027, 5, 9), (3072, 8, 24), (16384, 16, 6)])
def test_staged_windows_give_the_samples_of_whole_windows(d, L, B):
    """Algorithm 4 evaluated lazily: every launch takes at most `stage` positions of each chain's window and a
    chain that passed its stage goes on with the rest of the SAME window (carried output frozen). Final states
    bit for bit those of whole windows, for every stage length, with the advance step inside verify or in its own
    kernel; only the work differs: never more target rows, never fewer sequential calls."""
    w = wl.WORKLOADS["cfg2"].scaled(B=B, d=d, K=3 * L + 7, L=L)
    gp = w.gmm_params(d=d, ncomp=8)
    s = sds.sampler_for(w, gmm=gp, seed=91)
    s.set_option(s.OPT_WHOLE_CHAIN_KERNEL, 0)
    ref = [x.cpu().numpy() for x in s.sample_all()]
    assert int(s.get(sb.GET_CTL)[7]) == 0
    assert np.all(np.isfinite(ref[0]))
    for fuse in (1, 0):
        s.set_option(s.OPT_FUSE_ADVANCE, fuse)
        for stage in (1, 2, 3, L - 1, L, s.STAGED_ADAPTIVE):
            s.set_option(s.OPT_STAGED_WINDOWS, stage)
            got = [x.cpu().numpy() for x in s.sample_all()]
            assert np.array_equal(got[0], ref[0]), (fuse, stage)
            assert np.all(got[2] <= ref[2]) and np.all(got[1] >= ref[1]), (fuse, stage)
            if stage == L:
                assert np.array_equal(got[1], ref[1]) and np.array_equal(got[2], ref[2])
            if stage == 1:                                 # one row per launch: a call per step, no row wasted
                assert np.array_equal(got[2], got[1]) and np.all(got[1] == w.K + 1)
            assert np.array_equal(s.get(sb.GET_N), np.full(B, w.K))
    s.set_option(s.OPT_STAGED_WINDOWS, 0)
    s.set_option(s.OPT_FUSE_ADVANCE, 1)
    again = [x.cpu().numpy() for x in s.sample_all()]
    assert all(np.array_equal(x, y) for x, y in zip(again, ref))
    s.close()


@pytest.mark.gpu
@pytest.mark.parametrize("stage", [1, 3, 5])
def test_staged_free_run_against_the_oracle_counters(stage):
    """A fixed stage length, chain by chain against the oracle's lazily evaluated windows: final state, sequential
    target calls and target rows (a chain that differs must show a rounding-band event in the oracle's record)."""
    w = wl.WORKLOADS["cfg2"].scaled(B=48, K=60)
    gp = w.gmm_params()
    s = sds.sampler_for(w, gmm=gp, seed=w.sample_seed)
    s.set_option(s.OPT_WHOLE_CHAIN_KERNEL, 0)
    s.set_option(s.OPT_STAGED_WINDOWS, stage)
    out, calls, rows = [x.cpu().numpy() for x in s.sample_all()]
    assert int(s.get(sb.GET_CTL)[7]) > 0 or stage >= w.L
    den, a, c, sig = oracle_setup(w, gmm=gp)
    bad = 0
    for b in range(0, w.B, 3):
        r = o.speculative_chain(den, a, c, sig, w.L, w.sample_seed, b, w.d, record=True, stage=stage)
        bad += not chain_matches_or_band(r, calls[b], rows[b], out[b])
    assert bad <= 1
    s.close()
