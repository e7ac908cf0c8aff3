"""GPU parity and the paper's printed figure for the phi^4 Langevin workload (Appendix K)."""
import json
import os

import numpy as np
import pytest

import paper_2501_05370_b200 as sds
from paper_2501_05370_b200 import binding as sb
from oracle import sds_oracle as o
import workloads as wl
from helpers import assert_rows_close, chain_matches_or_band, oracle_setup, rel_l2
from test_gpu_parity import _window_check

pytestmark = pytest.mark.gpu
GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "worked_examples.json")))


@pytest.mark.parametrize("side,beta,periodic,rows", [(8, 100.0, False, 300), (5, 7.5, True, 77), (2, 3.0, False, 9),
                                                     (16, 40.0, False, 50)])
def test_phi4_gradient_rows(side, beta, periodic, rows):
    import torch
    w = wl.WORKLOADS["phi4"].scaled(d=side * side, B=rows, L=1, K=4, phi4=dict(side=side, beta=beta, periodic=periodic))
    s = sds.sampler_for(w)
    rng = np.random.default_rng(side)
    x = (1.0 + 0.3 * rng.standard_normal((rows, side * side))).astype(np.float32)
    k = np.zeros(rows, np.int32)
    out = s.denoise(torch.from_numpy(x).cuda(), torch.from_numpy(k).cuda()).cpu().numpy()
    for r in range(rows):
        assert_rows_close(out[r], o.phi4_grad_energy(x[r].astype(np.float64), side, beta, periodic), 1e-5, r)
    s.close()


def test_phi4_windows_and_free_run_against_oracle():
    w = wl.WORKLOADS["phi4"].scaled(B=24, K=600)
    s = sds.sampler_for(w, seed=3)
    den, a, c, sig = oracle_setup(w)
    a32, c32, s32, _ = sds.schedule_for(w)
    s.reset()
    stats = dict(tests=0, band=0, reflected=0)
    for _ in range(3):
        _window_check(s, w, den, a32, c32, s32, 3, 0, stats)
    assert stats["band"] <= 2 and stats["reflected"] > 0
    out, calls, rows = [x.cpu().numpy() for x in s.sample_all()]
    diverged = 0
    for b in range(8):
        r = o.speculative_chain(den, a, c, sig, w.L, 3, b, w.d, mode=o.FROZEN_EXACT, record=True)
        diverged += not chain_matches_or_band(r, calls[b], rows[b], out[b])
    assert diverged <= 1
    s.close()


def test_phi4_full_run_reproduces_the_papers_nfe():
    """500 chains x 100000 Langevin steps, window 20: the paper reports 48564 target calls per
    100000 steps. One call per window is what it counts, i.e. windows per step = 0.4856."""
    g = GOLD["phi4_table"]
    w = wl.WORKLOADS["phi4"]
    assert (w.K, w.L, w.phi4["side"], w.phi4["beta"], w.ula_gamma) == (g["steps"], g["window"], g["side"], g["beta"], g["gamma"])
    s = sds.sampler_for(w)
    out, calls, rows = [x.cpu().numpy().astype(np.float64) for x in s.sample_all()]
    assert np.all(np.isfinite(out)) and np.array_equal(s.get(sb.GET_N), np.full(w.B, w.K))
    windows_per_step = (calls / 2.0).mean() / w.K           # two sequential calls per window in this mode
    assert abs(windows_per_step - g["nfe_per_step"]) < 0.004, windows_per_step
    energies = np.array([o.phi4_energy(x, g["side"], g["beta"]) for x in out])
    print(f"windows per step {windows_per_step:.5f} (paper {g['nfe_per_step']}), "
          f"final energy {energies.mean():.2f} +- {energies.std():.2f}")
    s.close()


@pytest.mark.parametrize("side,L,periodic", [(8, 20, False), (6, 7, True), (5, 4, False)])
def test_phi4_whole_chain_kernel_equals_window_kernels(side, L, periodic):
    """The one-launch path and the window-by-window path give the same bits (states and counters)."""
    w = wl.WORKLOADS["phi4"].scaled(B=40, K=257, L=L, d=side * side,
                                    phi4=dict(side=side, beta=100.0, periodic=periodic))
    res = {}
    for fused in (1, 0):
        s = sds.sampler_for(w, seed=9)
        s.set_option(s.OPT_WHOLE_CHAIN_KERNEL, fused)
        res[fused] = [x.cpu().numpy() for x in s.sample_all()] + [s.launch_count()]
        s.close()
    for x, y in zip(res[1][:3], res[0][:3]):
        assert np.array_equal(x, y)
    assert res[1][3] < 10 < res[0][3]                       # one launch against hundreds


def test_phi4_energy_of_the_last_samples_plain_and_speculative_agree():
    """Appendix K reports the energy over the last samples of every run for the plain Langevin chain
    and for speculative sampling. Both sample the same chain in law, so their energies must agree
    within the statistical error (samples of one chain are correlated: the error is bounded by the
    pooled standard deviation over the square root of the number of chains). The statistic itself is
    the one bench.py prints for the lattice workload; the energies are checked against the oracle's."""
    import bench
    w = wl.WORKLOADS["phi4"].scaled(B=128, K=3000)
    res = bench.phi4_energy_statistic(sds, w, "cuda:0", last=100)
    sp, pl = res["speculative"], res["plain"]
    assert sp["samples"] == pl["samples"] == 128 * 100          # every one of the last 100 states of every chain
    tol = 4.0 * max(sp["std_pairs_once"], pl["std_pairs_once"]) * np.sqrt(2.0 / 128)
    assert abs(sp["mean_pairs_once"] - pl["mean_pairs_once"]) <= tol
    assert 0.5 * 64 < sp["mean_pairs_once"] < 2.0 * 64          # about d/2 at unit temperature plus the quartic part
    x = np.random.default_rng(3).standard_normal((5, 64))
    once, twice = bench.phi4_energies(x, 8, 100.0)
    for r in range(5):
        assert abs(once[r] - o.phi4_energy(x[r], 8, 100.0)) <= 1e-9 * once[r]
        assert abs(twice[r] - (2 * o.phi4_energy(x[r], 8, 100.0) - np.sum((x[r] ** 2 - 1) ** 2))) <= 1e-9 * twice[r]
