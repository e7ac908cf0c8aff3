"""Pins for the CPU oracle: each test checks oracle/sds_oracle.py against something the paper or
the mathematics fixes (closed forms, worked examples, invariants, brute force), never against
itself or the CUDA path."""
import json
import math
import os

import numpy as np
import pytest
from scipy import stats

from oracle import sds_oracle as o
import workloads as wl

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "worked_examples.json")))


# ------------------------------------------------------------------ RNG ----------------

def test_philox_known_answer_vectors():
    for v in GOLD["philox4x32_10_kat"]["vectors"]:
        ctr = [int(x, 16) for x in v["ctr"]]
        key = [int(x, 16) for x in v["key"]]
        out = o.philox4x32_10(*ctr, *key)
        assert [format(int(x), "08x") for x in out] == v["out"]


def test_uniform_range_and_law():
    u = np.array([o.uniform01(7, b, k) for b in range(200) for k in range(100)])
    assert u.min() > 0.0 and u.max() <= 1.0
    assert len(np.unique(u)) > 0.999 * len(u)
    assert stats.kstest(u, stats.uniform().cdf).pvalue > 1e-3
    assert abs(u.mean() - 0.5) < 4 * math.sqrt(1 / 12 / len(u))


def test_normals_moments_ks_and_stream_independence():
    z0 = np.concatenate([o.normals(11, o.STREAM_DRAFT, b, k, 64) for b in range(40) for k in range(50)])
    z2 = np.concatenate([o.normals(11, o.STREAM_INIT, b, k, 64) for b in range(40) for k in range(50)])
    n = len(z0)
    assert abs(z0.mean()) < 4 / math.sqrt(n)
    assert abs(z0.var() - 1) < 4 * math.sqrt(2 / n)
    assert abs(np.mean(z0 ** 3)) < 4 * math.sqrt(15 / n)
    assert abs(np.mean(z0 ** 4) - 3) < 4 * math.sqrt(96 / n)
    assert stats.kstest(z0, stats.norm().cdf).pvalue > 1e-3
    assert abs(np.corrcoef(z0, z2)[0, 1]) < 4 / math.sqrt(n)
    # neighbouring elements (same Philox block, cos/sin pair) are uncorrelated
    assert abs(np.corrcoef(z0[0::2], z0[1::2])[0, 1]) < 4 / math.sqrt(n / 2)
    # a prefix of a longer draw is the shorter draw (element i depends on (b, k, i) only)
    assert np.array_equal(o.normals(3, 0, 5, 9, 7), o.normals(3, 0, 5, 9, 64)[:7])
    # distinct (b, k) give distinct draws; 64-bit chain ids reach the last counter word
    assert not np.allclose(o.normals(3, 0, 5, 9, 8), o.normals(3, 0, 6, 9, 8))
    assert not np.allclose(o.normals(3, 0, 5, 9, 8), o.normals(3, 0, 5 + (1 << 32), 9, 8))


# ------------------------------------------------------------------ accept probability --

def _mc_reject_freq(m_p, m_q, sigma, N, seed):
    rng = np.random.default_rng(seed)
    m_p = np.atleast_1d(np.asarray(m_p, float))
    m_q = np.atleast_1d(np.asarray(m_q, float))
    rej = 0
    for _ in range(N):
        y = m_p + sigma * rng.standard_normal(m_p.shape)
        _, acc, _ = o.rejection_reflection(m_p, m_q, sigma, y, 1.0 - rng.random())
        rej += (not acc)
    return rej / N


@pytest.mark.parametrize("name", ["fig_couplings", "fig_temperature"])
def test_reject_probability_worked_pairs(name):
    g = GOLD[name]
    closed = 2 * stats.norm.cdf(abs(g["m_p"] - g["m_q"]) / (2 * g["sigma"])) - 1
    assert abs(closed - g["reject_prob"]) < 1e-12
    N = 120_000
    f = _mc_reject_freq(g["m_p"], g["m_q"], g["sigma"], N, 1)
    assert abs(f - closed) < 4 * math.sqrt(closed * (1 - closed) / N)


@pytest.mark.parametrize("d", [2, 64])
def test_reject_probability_depends_on_distance_only(d):
    rng = np.random.default_rng(d)
    m_p = rng.standard_normal(d)
    u = rng.standard_normal(d)
    u /= np.linalg.norm(u)
    sigma, dist = 0.7, 1.3
    m_q = m_p + dist * u
    closed = 2 * stats.norm.cdf(dist / (2 * sigma)) - 1
    N = 60_000
    f = _mc_reject_freq(m_p, m_q, sigma, N, 2)
    assert abs(f - closed) < 4 * math.sqrt(closed * (1 - closed) / N)


def test_identical_means_always_accept():
    rng = np.random.default_rng(0)
    m = rng.standard_normal(5)
    for _ in range(200):
        y = m + 0.3 * rng.standard_normal(5)
        Y, acc, ell = o.rejection_reflection(m, m, 0.3, y, 1e-300)
        assert acc and ell == 0.0 and np.array_equal(Y, y)


# ------------------------------------------------------------------ log ratio ----------

def test_log_ratio_forms_and_density_definition():
    rng = np.random.default_rng(3)
    for d in (1, 3, 64):
        m_p, m_q = rng.standard_normal(d), rng.standard_normal(d)
        sigma = 0.45
        y = m_p + sigma * rng.standard_normal(d)
        Delta, Z = (m_p - m_q) / sigma, (y - m_p) / sigma
        l1, l2 = o.log_ratio(Z, Delta), o.log_ratio_expanded(Z, Delta)
        ref = (stats.multivariate_normal.logpdf(y, m_q, sigma ** 2 * np.eye(d))
               - stats.multivariate_normal.logpdf(y, m_p, sigma ** 2 * np.eye(d)))
        assert abs(l1 - l2) < 1e-11 * max(1, abs(l1))
        assert abs(l1 - ref) < 1e-9 * max(1, abs(ref))
        assert abs(o.rejection_reflection(m_p, m_q, sigma, y, 0.5)[2] - ref) < 1e-9 * max(1, abs(ref))


def test_mean_log_ratio_is_minus_half_delta_sq():
    rng = np.random.default_rng(4)
    Delta = rng.standard_normal(8) * 0.6
    N = 100_000
    Z = rng.standard_normal((N, 8))
    vals = np.array([o.log_ratio_expanded(z, Delta) for z in Z])
    want = -0.5 * Delta @ Delta
    # Var[ell] = |Delta|^2
    assert abs(vals.mean() - want) < 4 * math.sqrt(Delta @ Delta / N)


# ------------------------------------------------------------------ reflection ---------

def test_reflection_isometry_involution_and_axis():
    rng = np.random.default_rng(5)
    d, sigma = 6, 0.8
    m_p, m_q = rng.standard_normal(d), rng.standard_normal(d)
    e = (m_p - m_q) / np.linalg.norm(m_p - m_q)
    seen = 0
    for _ in range(300):
        y = m_p + sigma * rng.standard_normal(d)
        Y, acc, _ = o.rejection_reflection(m_p, m_q, sigma, y, 1.0)   # log U = 0: rejects unless ratio >= 1
        if acc:
            continue
        seen += 1
        r_in, r_out = y - m_p, Y - m_q
        assert abs(np.linalg.norm(r_in) - np.linalg.norm(r_out)) < 1e-12
        diff = r_out - r_in
        assert np.linalg.norm(diff - e * (e @ diff)) < 1e-12          # they differ along e only
        assert abs(e @ r_out + e @ r_in) < 1e-12                       # component along e flips sign
        # reflecting twice gives back the residual
        back = r_out - 2 * e * (e @ r_out)
        assert np.allclose(back, r_in, atol=1e-12)
    assert seen > 50


def _outputs(rule, m_p, m_q, sigma, N, seed):
    rng = np.random.default_rng(seed)
    out = np.empty((N, len(m_p)))
    for i in range(N):
        y = m_p + sigma * rng.standard_normal(len(m_p))
        U = 1.0 - rng.random()
        if rule == "reflection":
            out[i] = o.rejection_reflection(m_p, m_q, sigma, y, U)[0]
        else:
            out[i] = o.rejection_incorrect_gaussian(m_p, m_q, sigma, y, U, rng.standard_normal(len(m_p)))[0]
    return out


def test_reflection_output_law_d1_and_incorrect_rule_fails():
    g = GOLD["fig_couplings"]
    m_p, m_q, s = np.array([g["m_p"]]), np.array([g["m_q"]]), g["sigma"]
    N = 60_000
    good = _outputs("reflection", m_p, m_q, s, N, 6)[:, 0]
    bad = _outputs("incorrect", m_p, m_q, s, N, 6)[:, 0]
    assert stats.kstest(good, stats.norm(m_q[0], s).cdf).pvalue > 1e-3
    assert stats.kstest(bad, stats.norm(m_q[0], s).cdf).pvalue < 1e-6


def test_reflection_output_law_d2():
    m_p, m_q, s = np.array([0.2, -0.4]), np.array([0.9, 0.3]), 0.6
    N = 60_000
    Y = _outputs("reflection", m_p, m_q, s, N, 7)
    R = (Y - m_q) / s
    e = (m_p - m_q) / np.linalg.norm(m_p - m_q)
    f = np.array([-e[1], e[0]])
    for proj in (R[:, 0], R[:, 1], R @ e, R @ f, R @ (e + f) / math.sqrt(2)):
        assert stats.kstest(proj, stats.norm().cdf).pvalue > 1e-3
    assert abs(np.corrcoef(R @ e, R @ f)[0, 1]) < 4 / math.sqrt(N)
    # radial law: |R|^2 ~ chi2(2)
    assert stats.kstest(np.sum(R * R, axis=1), stats.chi2(2).cdf).pvalue > 1e-3


def test_discrete_worked_example():
    g = GOLD["discrete_example"]
    p, q = np.array(g["p"]), np.array(g["q"])
    rng = np.random.default_rng(8)
    N = 80_000
    good = np.zeros(4)
    bad = np.zeros(4)
    nacc = 0
    for _ in range(N):
        xt = int(rng.choice(4, p=p))
        x, acc = o.rejection_discrete(p, q, xt, rng)
        good[x] += 1
        nacc += acc
        x2, _ = o.rejection_incorrect_discrete(p, q, xt, rng)
        bad[x2] += 1
    tol = 4 * math.sqrt(0.25 / N)
    assert abs(nacc / N - g["accept_prob"]) < tol
    assert np.all(np.abs(good / N - np.array(g["law_correct"])) < tol)
    assert np.all(np.abs(bad / N - np.array(g["law_incorrect"])) < tol)


# ------------------------------------------------------------------ window logic -------

def test_window_advance_matches_geometric_sum():
    rng = np.random.default_rng(9)
    d, L, K = 5, 6, 6
    a = np.full(K, 0.97)
    c = np.full(K, 0.05)
    sig = np.full(K, 0.2)
    delta = 0.9
    alpha = 2 - 2 * stats.norm.cdf(delta / 2)
    N = 30_000
    tot = 0
    first_counts = np.zeros(L + 2)
    for _ in range(N):
        D_c = rng.standard_normal(d)
        W = np.empty((L + 1, d))
        W[0] = rng.standard_normal(d)
        Dq = np.empty((L, d))
        for j in range(1, L + 1):
            W[j] = a[j - 1] * W[j - 1] + c[j - 1] * D_c + sig[j - 1] * rng.standard_normal(d)
            u = rng.standard_normal(d)
            u /= np.linalg.norm(u)
            Dq[j - 1] = D_c - (sig[j - 1] * delta / c[j - 1]) * u       # |Delta| = delta at every position
        logU = np.log(1.0 - rng.random(L))
        v = o.verify_window(W, Dq, D_c, a, c, sig, 0, logU)
        assert np.allclose(v["S1"], delta ** 2, rtol=1e-9)
        tot += min(v["jstar"], L)
        first_counts[v["jstar"]] += 1
    want = o.expected_advance(alpha, L)
    assert abs(want - (1 - alpha ** L) / (1 - alpha)) < 1e-12          # closed form of the printed sum
    assert abs(tot / N - want) < 4 * L / math.sqrt(N)
    # P(first rejection at j) = alpha^(j-1)(1-alpha)
    for j in range(1, L + 1):
        pj = alpha ** (j - 1) * (1 - alpha)
        assert abs(first_counts[j] / N - pj) < 4 * math.sqrt(pj * (1 - pj) / N) + 1e-9


def _cfg1_denoiser(K=40):
    w = wl.WORKLOADS["cfg1"]
    gp = w.gmm_params()
    a, c, sig, abar = o.ddpm_affine(wl.beta_linear(K))
    den = lambda x, k: o.gmm_posterior_mean(x, abar[k], gp.means, gp.logw, gp.comp_std)
    return den, a, c, sig


def test_chain_bookkeeping_and_counters():
    den, a, c, sig = _cfg1_denoiser(K=37)
    for mode in (o.FROZEN_PREV, o.FROZEN_EXACT):
        for b in range(6):
            r = o.speculative_chain(den, a, c, sig, L=4, seed=123, b=b, d=2, mode=mode, record=True)
            assert sum(r["adv"]) == 37
            assert all(1 <= x <= 4 for x in r["adv"])
            nwin = len(r["adv"])
            rows = sum(min(4, 37 - w_["n"]) for w_ in r["windows"])
            if mode == o.FROZEN_PREV:
                assert r["nfe_calls"] == 1 + nwin and r["nfe_rows"] == 1 + rows
                # first position of the first window: drafter == target
                assert r["windows"][0]["S1"][0] == 0.0 and r["windows"][0]["acc"][0]
            else:
                # position 1 always accepts; windows of length 1 make one call, others two
                assert all(w_["acc"][0] for w_ in r["windows"])
                assert r["nfe_rows"] == rows
                assert r["nfe_calls"] == sum(1 if min(4, 37 - w_["n"]) == 1 else 2 for w_ in r["windows"])


def test_exact_frozen_window_one_is_the_plain_chain_bitwise():
    den, a, c, sig = _cfg1_denoiser(K=25)
    for b in range(4):
        r = o.speculative_chain(den, a, c, sig, L=1, seed=77, b=b, d=2, mode=o.FROZEN_EXACT)
        y = o.plain_chain(den, a, c, sig, seed=77, b=b, d=2)
        assert np.array_equal(r["Y"], y)
        assert r["adv"] == [1] * 25


def _mmd_perm_pvalue(X, Y, rng, nperm=200):
    Z = np.concatenate([X, Y])
    D2 = np.sum((Z[:, None, :] - Z[None, :, :]) ** 2, axis=2)
    bw = np.median(D2[D2 > 0])
    Kmat = np.exp(-D2 / bw)
    n = len(X)

    def mmd(idx):
        i, j = idx[:n], idx[n:]
        return Kmat[np.ix_(i, i)].mean() + Kmat[np.ix_(j, j)].mean() - 2 * Kmat[np.ix_(i, j)].mean()

    base = mmd(np.arange(len(Z)))
    cnt = sum(mmd(rng.permutation(len(Z))) >= base for _ in range(nperm))
    return (cnt + 1) / (nperm + 1)


@pytest.mark.parametrize("mode", [o.FROZEN_PREV, o.FROZEN_EXACT])
def test_speculative_chain_matches_plain_chain_in_law(mode):
    den, a, c, sig = _cfg1_denoiser(K=40)
    N = 400
    S = np.array([o.speculative_chain(den, a, c, sig, L=4, seed=1, b=b, d=2, mode=mode)["Y"] for b in range(N)])
    P = np.array([o.plain_chain(den, a, c, sig, seed=2, b=b, d=2) for b in range(N)])
    for i in range(2):
        se = math.sqrt(S[:, i].var() / N + P[:, i].var() / N)
        assert abs(S[:, i].mean() - P[:, i].mean()) < 4 * se
        # variance comparison through the F-like ratio, generous (multi-modal law)
        assert 0.6 < S[:, i].var() / P[:, i].var() < 1.6
    assert _mmd_perm_pvalue(S, P, np.random.default_rng(0)) > 0.01


def test_incorrect_rule_in_chain_breaks_the_law():
    """Planted mistake (on the CPU): replacing the reflection by a fresh target draw changes
    the one-step output law enough for the d=1 KS test used above to see it; the chain-level
    test above would therefore not pass by accident."""
    m_p, m_q, s = np.array([0.0]), np.array([0.8]), 0.5
    bad = _outputs("incorrect", m_p, m_q, s, 40_000, 10)[:, 0]
    assert stats.kstest(bad, stats.norm(m_q[0], s).cdf).pvalue < 1e-4


# ------------------------------------------------------------------ denoisers ----------

def test_gmm_single_component_is_gaussian_posterior_mean():
    rng = np.random.default_rng(11)
    d, s, abar = 4, 0.7, 0.35
    mu = rng.standard_normal((1, d))
    x = rng.standard_normal(d)
    al = math.sqrt(abar)
    # x0 ~ N(mu, s^2 I), x | x0 ~ N(al x0, (1-abar) I): textbook conjugate update
    prec = 1 / s ** 2 + abar / (1 - abar)
    want = (mu[0] / s ** 2 + al * x / (1 - abar)) / prec
    got = o.gmm_posterior_mean(x, abar, mu, np.zeros(1), s)
    assert np.allclose(got, want, rtol=1e-12, atol=1e-12)


def _log_pt(x, abar, means, logw, s):
    al = math.sqrt(abar)
    v = abar * s * s + 1 - abar
    d = len(x)
    comp = logw - 0.5 * np.sum((x[None] - al * means) ** 2, axis=1) / v - 0.5 * d * math.log(2 * math.pi * v)
    m = comp.max()
    return m + math.log(np.exp(comp - m).sum())


def test_gmm_posterior_mean_is_tweedie_of_finite_difference_score():
    rng = np.random.default_rng(12)
    d, ncomp, s = 3, 5, 0.4
    means = rng.standard_normal((ncomp, d)) * 1.5
    logw = np.log(rng.dirichlet(np.ones(ncomp)))
    for abar in (0.05, 0.5, 0.95):
        x = rng.standard_normal(d)
        h = 1e-5
        grad = np.array([(_log_pt(x + h * np.eye(d)[i], abar, means, logw, s)
                          - _log_pt(x - h * np.eye(d)[i], abar, means, logw, s)) / (2 * h) for i in range(d)])
        want = (x + (1 - abar) * grad) / math.sqrt(abar)          # Tweedie
        got = o.gmm_posterior_mean(x, abar, means, logw, s)
        assert np.allclose(got, want, rtol=1e-6, atol=1e-6)
        # responsibilities do not change if all log-weights shift by a constant
        assert np.allclose(got, o.gmm_posterior_mean(x, abar, means, logw + 3.7, s), rtol=1e-12)


def test_gmm_posterior_mean_brute_force_importance_sampling():
    rng = np.random.default_rng(13)
    d, ncomp, s, abar = 2, 3, 0.5, 0.6
    means = rng.standard_normal((ncomp, d)) * 1.2
    logw = np.log(np.array([0.2, 0.5, 0.3]))
    x = np.array([0.4, -0.3])
    N = 400_000
    comp = rng.choice(ncomp, size=N, p=np.exp(logw))
    x0 = means[comp] + s * rng.standard_normal((N, d))
    lw = -0.5 * np.sum((x[None] - math.sqrt(abar) * x0) ** 2, axis=1) / (1 - abar)
    wgt = np.exp(lw - lw.max())
    want = (wgt[:, None] * x0).sum(0) / wgt.sum()
    got = o.gmm_posterior_mean(x, abar, means, logw, s)
    assert np.allclose(got, want, atol=1e-2)


def test_gmm_bf16_operand_variant_is_close_to_exact():
    w = wl.WORKLOADS["cfg4"]
    gp = w.gmm_params(d=256, ncomp=32)
    rng = np.random.default_rng(14)
    x = rng.standard_normal(256)
    for abar in (0.02, 0.5):
        e = o.gmm_posterior_mean(x, abar, gp.means, gp.logw, gp.comp_std)
        b = o.gmm_posterior_mean(x, abar, gp.means, gp.logw, gp.comp_std, bf16_operands=True)
        assert np.linalg.norm(e - b) <= 3e-2 * np.linalg.norm(e) + 1e-3


def _bf16_grid(rng, shape, scale=2.0):
    """Random values that bfloat16 holds exactly: multiples of 1/16 below 8 in size (at most 7 significant bits)."""
    return np.round(rng.uniform(-scale, scale, size=shape) * 16.0) / 16.0


def test_gmm_bf16_operand_variant_equals_the_definition_on_representable_inputs():
    """The bf16-operand branch expands |x - al mu|^2 and drops the |x|^2 term that all components
    share, rounds x, mu and the responsibilities to bfloat16, and writes the mixing step as
    (1 - al g) r.mu + g x. When x and mu are bfloat16 values and the responsibilities are too, no
    rounding happens anywhere, so the branch must reproduce the definition (the exact branch) to
    double precision: a wrong sign or factor in the expanded logit, in the |mu|^2 term or in the
    mixing step would show at once."""
    rng = np.random.default_rng(21)
    # (a) one component far ahead: responsibilities (1, 0, ..., 0) up to e^-60
    d, ncomp, s = 16, 6, 0.25
    means = _bf16_grid(rng, (ncomp, d), 4.0)
    logw = np.log(np.full(ncomp, 1.0 / ncomp))
    for abar in (0.9, 0.5):
        x = np.round(math.sqrt(abar) * means[2] * 16.0) / 16.0        # next to component 2, on the bf16 grid
        e = o.gmm_posterior_mean(x, abar, means, logw, s)
        b = o.gmm_posterior_mean(x, abar, means, logw, s, bf16_operands=True)
        assert np.allclose(b, e, rtol=0, atol=1e-12 * np.linalg.norm(e)), np.abs(b - e).max()
    # (b) two components of different norm whose responsibilities are exactly (3/4, 1/4) and (1/2, 1/2):
    # mu_2 is mu_1 with two coordinates swapped and x is symmetric under the swap, so both are equally far
    # from x and the log-weights alone decide
    mu = np.array([[1.0, 2.0, 0.5, -1.0, 3.0], [2.0, 1.0, 0.5, -1.0, 3.0]])
    x = np.array([0.75, 0.75, -0.25, 1.5, 0.125])
    for wts in ((0.75, 0.25), (0.5, 0.5)):
        for abar, s_ in ((0.64, 0.5), (0.09, 1.5)):
            e = o.gmm_posterior_mean(x, abar, mu, np.log(np.array(wts)), s_)
            b = o.gmm_posterior_mean(x, abar, mu, np.log(np.array(wts)), s_, bf16_operands=True)
            assert np.allclose(b, e, rtol=0, atol=1e-12), (wts, abar, np.abs(b - e).max())
    # (c) different norms AND different distances (the |mu|^2 term matters), one component dominant
    mu = np.array([[2.0, 0.0, 1.0], [0.0, 0.5, 0.0], [-1.0, -1.0, 4.0]])
    x = np.array([1.75, 0.0, 0.875])
    # (abar = 0.99, s = 1/8: v = 0.0255, the nearest competitor is 78 below in the logit)
    e = o.gmm_posterior_mean(x, 0.99, mu, np.log(np.full(3, 1 / 3)), 0.125)
    b = o.gmm_posterior_mean(x, 0.99, mu, np.log(np.full(3, 1 / 3)), 0.125, bf16_operands=True)
    assert np.allclose(b, e, rtol=0, atol=1e-12), np.abs(b - e).max()


def test_gmm_bf16_operand_variant_hand_computed_value():
    """d = 2, two components, every number worked out by hand. abar = 1/4 (al = 1/2), s = 1, so
    v = al^2 s^2 + 1 - al^2 = 1 and g = al s^2 / v = 1/2. mu_1 = (2, 0), mu_2 = (0, 1), equal weights,
    x = (1, 1). Distances: |x - al mu_1|^2 = |(0, 1)|^2 = 1, |x - al mu_2|^2 = |(1, 1/2)|^2 = 5/4, so the
    logits differ by (5/4 - 1)/2 = 1/8 and r = (1/(1 + e^(-1/8)), 1/(1 + e^(1/8))) = (0.531209..., 0.468790...).
    In bfloat16 (8 significant bits): 0.531209 = 1.0624 / 2 -> 1.0625 / 2 = 0.53125 (17/32) and
    0.468790 = 1.87516 / 4 -> 1.875 / 4 = 0.46875 (15/32). Mixing sum 17/32 (2, 0) + 15/32 (0, 1) = (1.0625, 0.46875);
    output (1 - al g) mix + g x = 0.75 (1.0625, 0.46875) + 0.5 (1, 1) = (1.296875, 0.8515625).
    The exact branch keeps r unrounded: 0.75 (2 r_1, r_2) + 0.5 (1, 1)."""
    mu = np.array([[2.0, 0.0], [0.0, 1.0]])
    x = np.array([1.0, 1.0])
    logw = np.log(np.array([0.5, 0.5]))
    b = o.gmm_posterior_mean(x, 0.25, mu, logw, 1.0, bf16_operands=True)
    assert np.allclose(b, [1.296875, 0.8515625], rtol=0, atol=1e-14), b
    r1 = 1.0 / (1.0 + math.exp(-0.125))
    e = o.gmm_posterior_mean(x, 0.25, mu, logw, 1.0)
    assert np.allclose(e, [0.75 * 2 * r1 + 0.5, 0.75 * (1 - r1) + 0.5], rtol=0, atol=1e-14), e


def test_gmm_grad_energy_finite_difference():
    rng = np.random.default_rng(15)
    d, ncomp, s = 4, 6, 0.9
    means = rng.standard_normal((ncomp, d)) * 2
    logw = np.log(rng.dirichlet(np.ones(ncomp)))

    def E(x):
        comp = logw - 0.5 * np.sum((x[None] - means) ** 2, axis=1) / s ** 2
        m = comp.max()
        return -(m + math.log(np.exp(comp - m).sum()))

    x = rng.standard_normal(d)
    h = 1e-5
    want = np.array([(E(x + h * np.eye(d)[i]) - E(x - h * np.eye(d)[i])) / (2 * h) for i in range(d)])
    assert np.allclose(o.gmm_grad_energy(x, means, logw, s), want, rtol=1e-6, atol=1e-7)


def test_mlp_layer_and_silu():
    assert np.allclose(o.silu(np.array([0.0, 1.0, -1.0, 20.0, -20.0])),
                       [0.0, 0.7310585786300049, -0.2689414213699951, 20.0 / (1 + math.exp(-20.0)), -20.0 / (1 + math.exp(20.0))])
    mp = wl.mlp_params(5, [12, 9, 7], K=6)
    W = [wl.bf16_bits_to_f32(x) for x in mp.weights]
    T = [wl.bf16_bits_to_f32(x) if x is not None else None for x in mp.temb]
    rng = np.random.default_rng(16)
    x = rng.standard_normal(12)
    xb = wl.bf16_bits_to_f32(wl.f32_to_bf16_bits(x.astype(np.float32))).astype(np.float64)
    pre = W[0].astype(np.float64) @ xb + T[0][3].astype(np.float64)
    h = pre / (1 + np.exp(-pre))
    hb = wl.bf16_bits_to_f32(wl.f32_to_bf16_bits(h.astype(np.float32))).astype(np.float64)
    want = W[1].astype(np.float64) @ hb
    got = o.mlp_forward(x, 3, W, mp.bias, T)
    assert np.allclose(got, want, rtol=1e-12, atol=1e-12)
    # bf16 rounding helper agrees with the independent converter of the input module, ties to even
    v = np.array([1.0, 1.00390625, 1.01171875, -3.1415926, 1e-20, 65504.0], dtype=np.float32)
    assert np.array_equal(o.bf16_round(v), wl.bf16_bits_to_f32(wl.f32_to_bf16_bits(v)).astype(np.float64))
    assert o.bf16_round(np.array([1.00390625]))[0] == 1.0 and o.bf16_round(np.array([1.01171875]))[0] == 1.015625


# ------------------------------------------------------------------ schedules ----------

@pytest.mark.parametrize("sched", ["linear", "cosine"])
def test_ddpm_affine_identities(sched):
    K = 50
    beta = wl.beta_linear(K) if sched == "linear" else wl.beta_cosine(K)
    assert np.all(beta > 0) and np.all(beta <= 0.999)
    a, c, sig, abar_step = o.ddpm_affine(beta)
    abar = np.concatenate([[1.0], np.cumprod(1 - beta)])
    assert np.all(np.diff(abar) < 0)
    assert np.all(sig > 0)
    # noise-free consistency: with x_t = sqrt(abar_t) x0 and D = x0 the mean is sqrt(abar_{t-1}) x0
    for k in range(K):
        t = K - k
        assert abs(a[k] * math.sqrt(abar[t]) + c[k] - math.sqrt(abar[t - 1])) < 1e-12
        assert abar_step[k] == abar[t]
        assert abs(sig[k] ** 2 - beta[t - 1]) < 1e-15
    # last transition (t = 1): the mean is the denoiser output itself
    assert abs(a[K - 1]) < 1e-12 and abs(c[K - 1] - 1) < 1e-12
    # posterior-mean identity of the forward process: one ancestral step from the exact posterior
    # keeps the marginal variance: for x0 fixed, Var = a^2 (1-abar_t) + sigma_post^2 where the DDPM
    # posterior variance is beta_t (1-abar_{t-1})/(1-abar_t) <= beta_t
    for k in range(K):
        t = K - k
        post_var = beta[t - 1] * (1 - abar[t - 1]) / (1 - abar[t])
        assert abs(a[k] ** 2 * (1 - abar[t]) + post_var - (1 - abar[t - 1])) < 1e-12


def test_ula_affine():
    a, c, s = o.ula_affine(7, 1e-3)
    assert np.all(a == 1) and np.allclose(c, -1e-3) and np.allclose(s, math.sqrt(2e-3))
    # Delta of the Langevin listing: sqrt(gamma/2) (grad E - grad E_hat) equals (m^p - m^q)/sigma
    g, gh = np.array([0.3, -1.0]), np.array([0.1, 0.4])
    x = np.array([1.0, 2.0])
    m_p, m_q = a[0] * x + c[0] * gh, a[0] * x + c[0] * g
    assert np.allclose((m_p - m_q) / s[0], math.sqrt(1e-3 / 2) * (g - gh))


# ------------------------------------------------------------------ phi^4 Langevin experiment ----

def test_phi4_gradient_is_the_gradient_of_the_energy():
    rng = np.random.default_rng(21)
    for periodic in (False, True):
        x = rng.standard_normal(36)
        h = 1e-6
        fd = np.array([(o.phi4_energy(x + h * np.eye(36)[i], 6, 7.5, periodic)
                        - o.phi4_energy(x - h * np.eye(36)[i], 6, 7.5, periodic)) / (2 * h) for i in range(36)])
        assert np.allclose(o.phi4_grad_energy(x, 6, 7.5, periodic), fd, rtol=1e-6, atol=1e-6)
    # a constant field at a minimum of the site potential has zero energy and zero gradient
    assert o.phi4_energy(np.ones(64), 8, 100.0) == 0.0
    assert np.all(o.phi4_grad_energy(-np.ones(64), 8, 100.0) == 0.0)
    # 2x1 lattice by hand: E = beta/2 (a-b)^2 + (a^2-1)^2 + (b^2-1)^2 on the pair, second row independent
    x = np.array([0.5, -0.25, 0.0, 0.0])
    e_pairs = 0.5 * 3.0 * ((0.5 + 0.25) ** 2 + 0.5 ** 2 + 0.25 ** 2 + 0.0)
    e_site = (0.25 - 1) ** 2 + (0.0625 - 1) ** 2 + 2.0
    assert abs(o.phi4_energy(x, 2, 3.0) - (e_pairs + e_site)) < 1e-12


def _phi4_windows_per_step(beta, periodic, K, chains, g):
    a, c, sig = o.ula_affine(K, g["gamma"])
    den = lambda x, k: o.phi4_grad_energy(x, g["side"], beta, periodic)
    ratios, advs = [], []
    for b in range(chains):
        r = o.speculative_chain(den, a, c, sig, g["window"], 5, b, g["side"] ** 2, mode=o.FROZEN_EXACT)
        ratios.append(len(r["adv"]) / K)
        advs += r["adv"]
        assert 2 * len(r["adv"]) - 1 <= r["nfe_calls"] <= 2 * len(r["adv"])   # the oracle counts both sequential calls
    adv = np.array(advs, dtype=np.float64)
    # standard error of windows/steps = 1/mean(adv) from the spread of the advances (delta method)
    se = (adv.std() / adv.mean()) / math.sqrt(len(adv)) / adv.mean()
    return float(np.mean(ratios)), float(se)


def test_phi4_speculative_langevin_reproduces_the_papers_nfe():
    """The one experiment with printed numbers that needs no data: 100000 Langevin steps cost 48564
    target calls with window 20 and the frozen drafter (Appendix K). With the target evaluated at
    Y_n before drafting and one call counted per window, windows per step must come out at 0.4856.
    The advance per window hardly varies (2 or 3 steps, standard deviation 0.25), so two chains of
    7000 steps fix the ratio to about 0.0007: enough to tell the readings of the energy apart.
    Free boundaries with every neighbouring pair counted once give the paper's figure; periodic
    boundaries give 0.491 and pairs counted twice (the same as doubling beta) 0.500, both rejected."""
    g = GOLD["phi4_table"]
    got, se = _phi4_windows_per_step(g["beta"], False, 7000, 2, g)
    assert se < 1.2e-3
    assert abs(got - g["nfe_per_step"]) < 3e-3, (got, se)
    periodic, _ = _phi4_windows_per_step(g["beta"], True, 5000, 1, g)
    assert periodic - g["nfe_per_step"] > 4e-3, periodic
    twice, _ = _phi4_windows_per_step(2 * g["beta"], False, 3000, 1, g)
    assert twice - g["nfe_per_step"] > 8e-3, twice


# ------------------------------------------------------------------ independent drafter ----------

def test_independent_drafter_equal_to_target_is_the_plain_chain():
    den, a, c, sig = _cfg1_denoiser(K=30)
    for b in range(3):
        r = o.speculative_chain(den, a, c, sig, L=4, seed=31, b=b, d=2, mode=o.INDEPENDENT, draft_denoise=den)
        assert r["adv"] == [4] * 7 + [2]                      # every draft accepted
        assert r["nfe_calls"] == 8 and r["nfe_rows"] == 30    # one batched target call per window, no initial call
        assert np.array_equal(r["Y"], o.plain_chain(den, a, c, sig, seed=31, b=b, d=2))


def test_independent_drafter_keeps_the_target_law():
    den, a, c, sig = _cfg1_denoiser(K=40)
    w = wl.WORKLOADS["cfg1"]
    gp = w.gmm_params()
    abar = o.ddpm_affine(wl.beta_linear(40))[3]
    # the cheaper model knows only two of the four components, and those slightly displaced
    cheap = lambda x, k: o.gmm_posterior_mean(x, abar[k], gp.means[:2] * 1.1, gp.logw[:2], gp.comp_std * 1.5)
    N = 400
    S = np.array([o.speculative_chain(den, a, c, sig, L=4, seed=3, b=b, d=2, mode=o.INDEPENDENT, draft_denoise=cheap)["Y"]
                  for b in range(N)])
    P = np.array([o.plain_chain(den, a, c, sig, seed=4, b=b, d=2) for b in range(N)])
    for i in range(2):
        se = math.sqrt(S[:, i].var() / N + P[:, i].var() / N)
        assert abs(S[:, i].mean() - P[:, i].mean()) < 4 * se
    assert _mmd_perm_pvalue(S, P, np.random.default_rng(1)) > 0.01
    # and the draft model alone does NOT have that law (the test above is not vacuous)
    Q = np.array([o.plain_chain(cheap, a, c, sig, seed=5, b=b, d=2) for b in range(N)])
    assert _mmd_perm_pvalue(Q, P, np.random.default_rng(2)) < 0.01


# ------------------------------------------------------------------ temperature variant ----------

def _tempered_accept_prob(delta, tau):
    """E[min(1, exp(l / tau))] for l ~ N(-delta^2/2, delta^2): X = l/tau ~ N(mu, s^2),
    P = Phi(mu/s) + exp(mu + s^2/2) Phi(-(mu + s^2)/s)."""
    mu, s = -delta ** 2 / (2 * tau), delta / tau
    return stats.norm.cdf(mu / s) + math.exp(mu + s * s / 2) * stats.norm.cdf(-(mu + s * s) / s)


@pytest.mark.parametrize("tau", [0.5, 2.0, 8.0])
def test_temperature_accept_probability_and_mean_shift(tau):
    g = GOLD["fig_temperature"]                       # draft mean 1, target mean 3, std 0.5
    m_p, m_q, s = np.array([g["m_p"]]), np.array([g["m_q"]]), g["sigma"]
    delta = abs(g["m_p"] - g["m_q"]) / s
    assert abs(_tempered_accept_prob(delta, 1.0) - (2 - 2 * stats.norm.cdf(delta / 2))) < 1e-12
    rng = np.random.default_rng(int(tau * 10))
    N = 80_000
    acc = 0
    ys = np.empty(N)
    for i in range(N):
        y = m_p + s * rng.standard_normal(1)
        Y, a_, _ = o.rejection_reflection(m_p, m_q, s, y, 1.0 - rng.random(), tau=tau)
        acc += a_
        ys[i] = Y[0]
    p = _tempered_accept_prob(delta, tau)
    assert abs(acc / N - p) < 4 * math.sqrt(p * (1 - p) / N) + 1e-4
    # Proposition "link with guidance": the output mean moves toward the draft mean for tau > 1
    # and away from it for tau < 1 (target mean 3 > draft mean 1)
    shift = ys.mean() - m_q[0]
    se = ys.std() / math.sqrt(N)
    assert (shift < -3 * se) if tau > 1 else (shift > 3 * se)


def test_temperature_one_is_the_exact_method_and_large_tau_accepts_the_draft():
    den, a, c, sig = _cfg1_denoiser(K=20)
    r1 = o.speculative_chain(den, a, c, sig, L=4, seed=8, b=0, d=2)
    r2 = o.speculative_chain(den, a, c, sig, L=4, seed=8, b=0, d=2, tau=1.0)
    assert np.array_equal(r1["Y"], r2["Y"]) and r1["adv"] == r2["adv"]
    r3 = o.speculative_chain(den, a, c, sig, L=4, seed=8, b=0, d=2, tau=1e9)
    assert r3["adv"] == [4] * 5                        # every draft accepted


# ----------------------------------------------------------------------------------------
# projected acceptance ratio (Appendix F: the rule for a full matrix A, in the original space)
# ----------------------------------------------------------------------------------------


def test_projected_rule_with_invertible_matrix_is_algorithm_3():
    rng = np.random.default_rng(77)
    for _ in range(50):
        d = 3
        A = rng.standard_normal((d, d)) + 2 * np.eye(d)
        m_p, m_q = rng.standard_normal(d), rng.standard_normal(d)
        s = 0.7
        y = m_p + s * rng.standard_normal(d)
        U = 1.0 - rng.random()
        Y1, a1, l1 = o.rejection_reflection(m_p, m_q, s, y, U)
        Y2, a2, l2 = o.rejection_reflection_projected(m_p, m_q, s, y, U, A)
        assert a1 == a2 and abs(l1 - l2) < 1e-10 and np.allclose(Y1, Y2, atol=1e-10)


def test_projected_log_ratio_equals_the_whitened_image_form():
    # (Delta + 2Z)^T A^+ A Delta = |Z_A + Delta_A|^2 - |Z_A|^2 with v_A = (A A^T)^(-1/2) A v
    rng = np.random.default_rng(78)
    A = rng.standard_normal((2, 5))
    w, V = np.linalg.eigh(A @ A.T)
    Wh = V @ np.diag(w ** -0.5) @ V.T @ A
    m_p, m_q = rng.standard_normal(5), rng.standard_normal(5)
    s = 1.3
    y = m_p + s * rng.standard_normal(5)
    _, _, ell = o.rejection_reflection_projected(m_p, m_q, s, y, 0.5, A)
    Z, D = (y - m_p) / s, (m_p - m_q) / s
    ZA, DA = Wh @ Z, Wh @ D
    assert abs(ell - (-0.5) * (np.dot(ZA + DA, ZA + DA) - np.dot(ZA, ZA))) < 1e-10


def test_projected_rule_couples_the_images_maximally():
    # accept frequency = 2 - 2 Phi(|Delta_A| / 2) with |Delta_A|^2 = Delta^T A^+ A Delta, and the image
    # A Y has the image of the target law although Y itself does not follow the target law
    rng = np.random.default_rng(79)
    A = np.array([[0.6, 0.8]])                        # one orthonormal row: A Y is a scalar
    m_p, m_q, s = np.array([0.0, 0.0]), np.array([2.0, -0.5]), 1.0
    dA = abs((A @ (m_p - m_q))[0]) / s
    N = 60_000
    acc = 0
    img = np.empty(N)
    for i in range(N):
        y = m_p + s * rng.standard_normal(2)
        Y, a_, _ = o.rejection_reflection_projected(m_p, m_q, s, y, 1.0 - rng.random(), A)
        acc += a_
        img[i] = (A @ Y)[0]
    p = 2 - 2 * stats.norm.cdf(dA / 2)
    assert abs(acc / N - p) < 4 * math.sqrt(p * (1 - p) / N)
    assert abs(p - (2 - 2 * stats.norm.cdf(np.linalg.norm(m_p - m_q) / 2))) > 0.02   # not the full-space rate
    assert stats.kstest(img, stats.norm(loc=(A @ m_q)[0], scale=s).cdf).pvalue > 1e-3


def test_window_with_projection_follows_the_single_step_rule():
    rng = np.random.default_rng(80)
    d, Lt, n = 6, 4, 3
    K = 12
    a, c, sig = 0.9 + 0.01 * np.arange(K), 0.05 + 0.01 * np.arange(K), 0.3 + 0.02 * np.arange(K)
    A = rng.standard_normal((2, d))
    W = rng.standard_normal((Lt + 1, d))
    Dq = rng.standard_normal((Lt, d))
    Dc = rng.standard_normal(d)
    logU = np.log(1.0 - rng.random(Lt))
    v = o.verify_window(W, Dq, Dc, a, c, sig, n, logU, decide_f32=False, proj=A)
    first = None
    for j in range(1, Lt + 1):
        k = n + j - 1
        m_p, m_q = a[k] * W[j - 1] + c[k] * Dc, a[k] * W[j - 1] + c[k] * Dq[j - 1]
        Y, ok, ell = o.rejection_reflection_projected(m_p, m_q, sig[k], W[j], math.exp(logU[j - 1]), A)
        assert abs(ell - v["ell"][j - 1]) < 1e-10 and ok == bool(v["acc"][j - 1])
        if not ok and first is None:
            first = j
            assert np.allclose(Y, v["Y_reflect"], atol=1e-10)
    assert v["jstar"] == (first if first is not None else Lt + 1)
    # a square invertible matrix changes nothing
    v0 = o.verify_window(W, Dq, Dc, a, c, sig, n, logU, decide_f32=False)
    v1 = o.verify_window(W, Dq, Dc, a, c, sig, n, logU, decide_f32=False, proj=rng.standard_normal((d, d)) + 3 * np.eye(d))
    assert np.allclose(v0["ell"], v1["ell"], atol=1e-9) and v0["jstar"] == v1["jstar"]


# ----------------------------------------------------------------------------------------
# Picard drafter (Appendix C: parallel sampling as drafting)
# ----------------------------------------------------------------------------------------


def test_deterministic_sampler_keeps_the_noise_direction():
    # if x_t = sqrt(abar_t) x0 + sqrt(1 - abar_t) eps and the denoiser returns x0, one deterministic
    # step lands on sqrt(abar_{t-1}) x0 + sqrt(1 - abar_{t-1}) eps with the same eps
    K = 25
    beta = wl.beta_cosine(K)
    a_det, c_det = o.ddim_affine(beta)
    abar = np.concatenate([[1.0], np.cumprod(1 - beta)])
    rng = np.random.default_rng(3)
    x0, eps = rng.standard_normal(4), rng.standard_normal(4)
    for k in range(K):
        t = K - k
        xt = math.sqrt(abar[t]) * x0 + math.sqrt(1 - abar[t]) * eps
        want = math.sqrt(abar[t - 1]) * x0 + math.sqrt(1 - abar[t - 1]) * eps
        assert np.allclose(a_det[k] * xt + c_det[k] * x0, want, atol=1e-12)


def test_picard_iterates_reach_the_sequential_deterministic_chain():
    den, a, c, sig = _cfg1_denoiser(K=30)
    a_det, c_det = o.ddim_affine(wl.beta_linear(30))
    rng = np.random.default_rng(4)
    Y, Dc, n, Lt = rng.standard_normal(2), rng.standard_normal(2), 5, 6
    seq = np.empty((Lt, 2))
    seq[0] = Y
    for j in range(Lt - 1):
        seq[j + 1] = a_det[n + j] * seq[j] + c_det[n + j] * den(seq[j], n + j)
    for m in range(Lt):
        F = o.picard_trajectory(den, a_det, c_det, Y, Dc, n, Lt, m)
        assert np.allclose(F[:m + 1], seq[:m + 1], atol=1e-12)       # m iterations fix the first m+1 points
        if m < Lt - 1:
            assert not np.allclose(F[m + 1], seq[m + 1], atol=1e-6)  # and not yet the next one
    # no iteration: the rollout with the carried output frozen
    F0 = o.picard_trajectory(den, a_det, c_det, Y, Dc, n, Lt, 0)
    assert np.allclose(F0[2], a_det[n + 1] * (a_det[n] * Y + c_det[n] * Dc) + c_det[n + 1] * Dc)


def test_picard_drafter_with_window_one_is_the_plain_chain():
    den, a, c, sig = _cfg1_denoiser(K=20)
    a_det, c_det = o.ddim_affine(wl.beta_linear(20))
    for p in (1, 3):
        r = o.speculative_chain(den, a, c, sig, L=1, seed=17, b=2, d=2, mode=o.PICARD, picard=(p, a_det, c_det))
        assert r["adv"] == [1] * 20
        assert r["nfe_calls"] == 1 + 20 and r["nfe_rows"] == 1 + 20   # initial call + one target row per step
        assert np.array_equal(r["Y"], o.plain_chain(den, a, c, sig, seed=17, b=2, d=2))


def test_picard_drafter_counters_and_first_position():
    den, a, c, sig = _cfg1_denoiser(K=23)
    a_det, c_det = o.ddim_affine(wl.beta_linear(23))
    for p in (1, 2, 4):
        r = o.speculative_chain(den, a, c, sig, L=4, seed=19, b=1, d=2, mode=o.PICARD, picard=(p, a_det, c_det),
                                record=True)
        assert sum(r["adv"]) == 23
        calls, rows = 1, 1
        for wd in r["windows"]:
            Lt = wd["Dq"].shape[0]
            calls += (p - 1 if Lt >= 2 else 0) + 1 + (1 if Lt >= 2 else 0)
            rows += (p - 1) * (Lt - 1) + Lt + (Lt - 1)
            assert wd["S1"][0] < 1e-24 and wd["acc"][0]              # position 1 is drafted from the target itself
        assert (r["nfe_calls"], r["nfe_rows"]) == (calls, rows)


def test_picard_drafter_keeps_the_target_law():
    den, a, c, sig = _cfg1_denoiser(K=40)
    a_det, c_det = o.ddim_affine(wl.beta_linear(40))
    N = 400
    S = np.array([o.speculative_chain(den, a, c, sig, L=4, seed=6, b=b, d=2, mode=o.PICARD, picard=(2, a_det, c_det))["Y"]
                  for b in range(N)])
    P = np.array([o.plain_chain(den, a, c, sig, seed=7, b=b, d=2) for b in range(N)])
    for i in range(2):
        se = math.sqrt(S[:, i].var() / N + P[:, i].var() / N)
        assert abs(S[:, i].mean() - P[:, i].mean()) < 4 * se
    assert _mmd_perm_pvalue(S, P, np.random.default_rng(3)) > 0.01


def test_staged_evaluation_of_a_window_changes_no_state_and_no_decision():
    """Algorithm 4 with its window evaluated a few positions per target call: the final state and the sequence of
    accepted steps are those of the one batched call, exactly (fp64, same operations); only the counters move:
    never more rows, never fewer calls; stage >= L is the algorithm as printed; stage 1 is one row per step."""
    d, K, L = 6, 60, 7
    rng = np.random.default_rng(11)
    means = rng.normal(0, 2.0, size=(5, d))
    logw = np.log(np.full(5, 0.2))
    beta = np.linspace(1e-4, 0.05, K)
    a, c, sig, abar = o.ddpm_affine(beta)
    den = lambda x, k: o.gmm_posterior_mean(x, abar[k], means, logw, 0.4)
    for b in range(6):
        ref = o.speculative_chain(den, a, c, sig, L, 123, b, d, record=True)
        steps_ref = np.cumsum(ref["adv"])
        for stage in (1, 2, 3, L - 1, L, L + 5):
            r = o.speculative_chain(den, a, c, sig, L, 123, b, d, stage=stage, record=True)
            assert np.array_equal(r["Y"], ref["Y"]), (b, stage)
            assert r["nfe_rows"] <= ref["nfe_rows"] and r["nfe_calls"] >= ref["nfe_calls"]
            # every state the whole-window run passed through is passed through by the staged run
            assert set(steps_ref.tolist()) <= set(np.cumsum(r["adv"]).tolist())
            if stage >= L:
                assert r["nfe_rows"] == ref["nfe_rows"] and r["nfe_calls"] == ref["nfe_calls"] and r["adv"] == ref["adv"]
            if stage == 1:
                assert r["nfe_calls"] == K + 1 and r["nfe_rows"] == K + 1
        # rows saved are exactly the positions behind a rejection that the batched call evaluated for nothing
        r2 = o.speculative_chain(den, a, c, sig, L, 123, b, d, stage=2)
        assert r2["nfe_rows"] < ref["nfe_rows"]
    with pytest.raises(ValueError):
        o.speculative_chain(den, a, c, sig, L, 123, 0, d, mode=o.FROZEN_EXACT, stage=2)
