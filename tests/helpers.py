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


ELEM_FACTOR = 8.0   # element-wise bound = ELEM_FACTOR * tol * rms(want)


def elem_err(got, want, floor=1e-6):
    """Largest element-wise difference in units of the row's root mean square: a row-L2 bound alone
    lets a single wrong element of a long row pass (one element of a d = 3072 row that is off by its
    own size moves the row norm by 1.8 %), so every row comparison also bounds each element."""
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    rms = max(float(np.sqrt(np.mean(want * want))) if want.size else 0.0, floor)
    return float(np.max(np.abs(got - want))) / rms if want.size else 0.0


def rows_close(got, want, tol, floor=1e-6):
    """Row comparison used for states and denoiser rows: relative row-L2 error <= tol AND every
    element within ELEM_FACTOR * tol of the row's rms. Returns (ok, l2 error, element error)."""
    r, e = rel_l2(got, want, floor), elem_err(got, want, floor)
    return (r <= tol and e <= ELEM_FACTOR * tol), r, e


def assert_rows_close(got, want, tol, what=""):
    ok, r, e = rows_close(got, want, tol)
    assert ok, (what, "row L2", r, "largest element error / rms", e, "tol", tol)


def ell_close(g, w):
    """|l_gpu - l_oracle| <= 1e-4 where the oracle's value is in [-20, 0.5], else 1e-5 relative."""
    tol = 1e-4 if -20.0 <= w <= 0.5 else 1e-5 * abs(w)
    return abs(g - w) <= tol


BAND = 2e-4   # |log ratio - log U| below this: either decision is a correct rounding


def chain_matches_or_band(r, calls_b, rows_b, out_b, tol=1e-4):
    """A free-running chain against the oracle's chain `r` (speculative_chain(..., record=True)).
    True when the counters are identical and the final state agrees (row L2 and element-wise).
    A chain that differs is accepted only with proof that a rounding-band event sent the two runs
    apart: some position of some window of the oracle's record has |log ratio - log U| < BAND, where
    either decision is a correct rounding. Without such a position the assertion fails."""
    same = (int(r["nfe_calls"]) == int(calls_b) and int(r["nfe_rows"]) == int(rows_b)
            and rows_close(out_b, r["Y"], tol)[0])
    if same:
        return True
    gaps = [float(np.min(np.abs(np.asarray(win["ell"]) - np.asarray(win["logU"])))) for win in r["windows"]]
    assert gaps and min(gaps) < BAND, ("chain differs from the oracle's with no rounding-band event",
                                       min(gaps) if gaps else None, r["nfe_calls"], calls_b, r["nfe_rows"], rows_b)
    return False
