#!/usr/bin/env python
"""Benchmark of the speculative-sampling hot path.

One "step" is one full sds_sample_all over a batch of chains of the chosen workload: initial
state and target call, then draft / batched target / verify / advance windows until every chain
has made its K transitions. The metric is accepted chain-steps per second (B*K per run; both
accepted and reflected steps are valid target steps).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg4] [--impl reference]

Prints one JSON line (rank 0). The default workload is the largest single-GPU configuration (cfg4:
1024 chains of dimension 16384, 1024-component mixture on the tensor cores). N > 1: chains are sharded
across ranks by global chain id, no collective on the data path (weak scaling: B chains per rank);
started without a launcher, the script starts its own N ranks under torch.distributed.run. After the
timed region the ranks gather the final samples and sum the counters (NCCL, off the timed path).
--impl reference times the CPU oracle, as it stands, on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import workloads as wl  # noqa: E402

METRIC = "accepted_chain_steps_per_sec"
UNIT = "chain-steps/s"
FP32_LANES_PER_SM, SMS = 128, 148
DEFAULT_WORKLOAD = "cfg4"
CSRC = os.path.join(ROOT, "paper_2501_05370_b200", "csrc")
TRAFFIC_TABLE = os.path.join(ROOT, "profiles", "dram_traffic.md")


def measured_traffic():
    """DRAM bytes (read + written) and warp instructions per launch from the profiler captures listed
    in the traffic table: rows `| workload | kernel kind | chains | DRAM bytes per launch | warp
    instructions per launch | source file:hash | note |`. A capture is taken at a reduced number of
    chains; every chain moves the same bytes, so a launch at B chains moves B / chains times as much.
    A row whose source file no longer has the recorded hash describes a kernel that has changed since:
    it is ignored (the figure is then null). Returns {(workload, kind): (chains, bytes, inst)}."""
    out = {}
    if not os.path.exists(TRAFFIC_TABLE):
        return out
    for ln in open(TRAFFIC_TABLE):
        f = [x.strip() for x in ln.strip().strip("|").split("|")]
        if len(f) < 6 or not f[2].isdigit():
            continue
        src, _, want = f[5].partition(":")
        path = os.path.join(CSRC, src)
        if not os.path.exists(path) or hashlib.sha256(open(path, "rb").read()).hexdigest()[:12] != want:
            continue
        num = lambda x: float(x) if x not in ("", "-") else None
        out[(f[0], f[1])] = (int(f[2]), num(f[3]), num(f[4]))
    return out


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"], bf16_sustained=d["bf16_tflops_sustained"],
                    sm_max_mhz=d.get("sm_max_mhz", 1965.0), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_sustained=1400.0, sm_max_mhz=1965.0, source="fallback")


# --------------------------------------------------------------------------------------------
# CPU oracle legs
# --------------------------------------------------------------------------------------------

def oracle_closure(w):
    from oracle import sds_oracle as o
    if w.sampler == "ddpm":
        a, c, sig, abar = o.ddpm_affine(w.beta())
    else:
        a, c, sig = o.ula_affine(w.K, w.ula_gamma)
    if w.denoiser == "phi4":
        p4 = w.phi4
        den = lambda x, k: o.phi4_grad_energy(x, p4["side"], p4["beta"], p4.get("periodic", False))
    elif w.denoiser == "mlp":
        mp = w.mlp_params()
        W = [wl.bf16_bits_to_f32(x).astype(np.float64) for x in mp.weights]
        T = [wl.bf16_bits_to_f32(x).astype(np.float64) if x is not None else None for x in mp.temb]
        den = lambda x, k: o.mlp_forward(x, k, W, mp.bias, T)
    else:
        gp = w.gmm_params()
        if w.sampler == "ddpm":
            den = lambda x, k: o.gmm_posterior_mean(x, abar[k], gp.means, gp.logw, gp.comp_std,
                                                    bf16_operands=gp.means_bf16)
        else:
            den = lambda x, k: o.gmm_grad_energy(x, gp.means, gp.logw, gp.comp_std)
    return o, den, a, c, sig


VARIANTS = ("default", "exact", "independent", "picard2", "tau2", "proj16")


def draft_mixture(w):
    """The cheaper draft model of the `independent` variant: the first half of the mixture's components."""
    gp = w.gmm_params()
    half = max(1, w.gmm["ncomp"] // 2)
    return wl.GmmParams(means=gp.means[:half].copy(), logw=np.full((half,), -np.log(half), dtype=np.float32),
                        comp_std=gp.comp_std, means_bf16=gp.means_bf16)


def proj_matrix(w, r: int = 16):
    return np.random.default_rng(1234).standard_normal((r, w.d))


def gpu_sampler(sds, w, variant: str, **kw):
    """The sampler of a bench variant: the default drafter, or one of the other drafters / accept tests."""
    import torch
    from paper_2501_05370_b200 import binding as sb
    if variant == "exact":
        s = sds.sampler_for(w, drafter_mode=sb.SDS_FROZEN_EXACT, **kw)
    elif variant == "independent":
        if w.denoiser != "gmm":
            raise SystemExit("--variant independent is defined for the mixture workloads")
        s = sds.sampler_for(w, drafter=sds.drafter_for(w, gmm=draft_mixture(w)), **kw)
    elif variant == "picard2":
        s = sds.sampler_for(w, picard=sds.picard_for(w, 2), **kw)
    else:
        s = sds.sampler_for(w, **kw)
    if variant == "tau2":
        s.set_temperature(2.0)
    if variant == "proj16":
        s.set_projection(torch.from_numpy(sds.projection_basis(proj_matrix(w))).to(kw.get("device", "cuda:0")))
    return s


def oracle_chain_kwargs(w, variant: str, o, a, c, sig):
    """Keyword arguments that make the oracle's chain follow the same variant."""
    if variant == "exact":
        return dict(mode=o.FROZEN_EXACT)
    if variant == "independent":
        gp = draft_mixture(w)
        if w.sampler == "ddpm":
            abar = o.ddpm_affine(w.beta())[3]
            dd = lambda x, k: o.gmm_posterior_mean(x, abar[k], gp.means, gp.logw, gp.comp_std, bf16_operands=gp.means_bf16)
        else:
            dd = lambda x, k: o.gmm_grad_energy(x, gp.means, gp.logw, gp.comp_std)
        return dict(mode=o.INDEPENDENT, draft_denoise=dd)
    if variant == "picard2":
        ad, cd = o.ddim_affine(w.beta()) if w.sampler == "ddpm" else o.ula_affine(w.K, w.ula_gamma)[:2]
        return dict(mode=o.PICARD, picard=(2, ad, cd))
    if variant == "tau2":
        return dict(mode=getattr(w, "drafter_mode", 0), tau=2.0)
    if variant == "proj16":
        return dict(mode=getattr(w, "drafter_mode", 0), proj=proj_matrix(w))
    return dict(mode=getattr(w, "drafter_mode", 0))


def oracle_time(w, budget_s: float, min_chains: int = 1, first_chain: int = 0, variant: str = "default"):
    """Runs oracle chains one after another for about budget_s seconds of CPU work.

    Heavy workloads cannot finish even one chain in the budget, so a chain is run over the first
    Kp transitions only (Kp starts small and grows while chains stay cheap); the sample is then a
    prefix of the chain, which the returned description says. Returns (chain_steps, seconds, text)."""
    o, den, a, c, sig = oracle_closure(w)
    t0 = time.perf_counter()
    n, steps, Kp = 0, 0, min(w.K, w.L)           # at least one full window per chain
    prefix = False
    while True:
        t1 = time.perf_counter()
        okw = oracle_chain_kwargs(w, variant, o, a, c, sig)
        if "picard" in okw:
            okw["picard"] = (okw["picard"][0], okw["picard"][1][:Kp], okw["picard"][2][:Kp])
        o.speculative_chain(den, a[:Kp], c[:Kp], sig[:Kp], w.L, w.sample_seed, first_chain + n, w.d, **okw)
        dt = time.perf_counter() - t1
        n += 1
        steps += Kp
        prefix |= Kp < w.K
        el = time.perf_counter() - t0
        if (n >= min_chains and el >= budget_s) or n >= w.B:
            break
        if Kp < w.K and dt < budget_s / 8:
            Kp = min(w.K, Kp * 4)
    what = (f"{n} chains of {w.name}, {steps} chain-steps" + (" (chains cut to their first transitions)" if prefix else "")
            + f" in {el:.1f} s, one NumPy thread")
    return steps, el, what


def oracle_plain_time(w, budget_s: float):
    """The oracle's plain (non-speculative) chain, same sampling rule as oracle_time: the context
    for the saving in sequential target calls. Returns (chain_steps, seconds)."""
    o, den, a, c, sig = oracle_closure(w)
    t0 = time.perf_counter()
    n, steps, Kp = 0, 0, min(w.K, w.L)
    while True:
        t1 = time.perf_counter()
        o.plain_chain(den, a[:Kp], c[:Kp], sig[:Kp], w.sample_seed, n, w.d)
        dt = time.perf_counter() - t1
        n += 1
        steps += Kp
        el = time.perf_counter() - t0
        if el >= budget_s or n >= w.B:
            break
        if Kp < w.K and dt < budget_s / 8:
            Kp = min(w.K, Kp * 4)
    return steps, el


def run_reference(args, w):
    """--impl reference: the oracle on the host cores, same metric, bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    per_step_budget = max(1.0, min(8.0, 60.0 / max(1, args.steps + args.warmup)))
    for _ in range(args.warmup):
        oracle_time(w, per_step_budget / 2, variant=args.variant)
    tot_steps, tot_s, what = 0, 0.0, ""
    for i in range(args.steps):
        n, s, what = oracle_time(w, per_step_budget, first_chain=i * 16, variant=args.variant)
        tot_steps += n
        tot_s += s
    value = tot_steps / tot_s
    sample = f"{args.steps} steps, each: {what}"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * tot_s / max(1, args.steps),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(w, args),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def workload_config(w, args):
    return {"workload": f"{w.name}: B={w.B} chains/GPU, d={w.d}, L={w.L}, K={w.K}, {w.sampler} "
                        f"{w.schedule or 'gamma=%g' % w.ula_gamma}, {w.denoiser} denoiser"
                        + (f" ncomp={w.gmm['ncomp']}" if w.denoiser == 'gmm' else ""),
            "drafter": {"exact": "frozen target output evaluated at Y_n",
                        "independent": "independent draft model: the first half of the mixture's components",
                        "picard2": "Picard drafter, 2 parallel target calls per window"}.get(
                            getattr(args, "variant", "default"),
                            "frozen target output " + ("evaluated at Y_n" if getattr(w, "drafter_mode", 0) else "(carried)")),
            "accept_test": {"tau2": "temperature 2 (inexact)", "proj16": "decided in the image of a 16 x d matrix (inexact)"}.get(
                getattr(args, "variant", "default"), "exact"),
            "seed": w.sample_seed,
            "l2": "256 MiB buffer written between timed steps (working set may fit L2)",
            "sharding": "chains by global id, no data-path collective"}


# --------------------------------------------------------------------------------------------
# clocks
# --------------------------------------------------------------------------------------------

class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.path = tempfile.mktemp(prefix="sds_clocks_", suffix=".csv")
        self.proc = None
        self.idx = gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.idx), "-lms", "100"], stdout=open(self.path, "w"),
                                         stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def mark(self):
        """Samples taken before this call are ignored by stop()."""
        try:
            self.skip = sum(1 for _ in open(self.path))
        except Exception:
            self.skip = 0

    def count(self) -> int:
        """Samples taken since mark()."""
        try:
            return max(0, sum(1 for _ in open(self.path)) - getattr(self, "skip", 0))
        except Exception:
            return 0

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for i, ln in enumerate(open(self.path)):
                if i < getattr(self, "skip", 0):
                    continue
                f = [x.strip() for x in ln.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1])); mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


# --------------------------------------------------------------------------------------------
# GPU arm
# --------------------------------------------------------------------------------------------

def run_counts(w, variant, calls_np, rows_np):
    """(target rows of the windows, chain-windows) of one run, from the per-chain counters."""
    B = len(calls_np)
    if getattr(w, "drafter_mode", 0) == 1 or variant == "exact":
        # drafter evaluated at Y_n: no initial call, two sequential calls per window (one for a last window of one row)
        return float(rows_np.sum()), float(np.ceil(calls_np / 2.0).sum())
    if variant == "independent":                       # no initial call, one target call per window
        return float(rows_np.sum()), float(calls_np.sum())
    if variant == "picard2":                           # initial call, then 2 draft calls + 1 verify call per window
        cw = float(np.ceil((calls_np - 1) / 3.0).sum())
        return float(w.L * cw), cw                     # rows of the verify calls (full windows assumed)
    return float(rows_np.sum() - B), float(calls_np.sum() - B)   # the initial call is not a window


def tensor_mixture(w):
    return w.denoiser == "gmm" and (w.gmm.get("means_bf16") or
                                    (32 < w.gmm["ncomp"] <= 1024 and w.gmm["ncomp"] % 128 == 0 and w.d % 128 == 0))


def kernel_rooflines(w, variant, prof, steps, rows, cw, positions, pk, ctl, traffic, launch_shape):
    """One roofline entry per kernel kind that ran in the timed region.

    rows: target rows of the windows per run (sum of window lengths over chains and windows);
    cw: chain-windows per run; positions: window positions whose accept test verify evaluated per run
    (fewer than rows when it stops reading after the first rejection). Algorithmic bytes / flops are the
    per-unit figures of the method (what any implementation must move or compute); `requested` is what
    this implementation's kernels ask memory for."""
    d, B = w.d, w.B
    hbm, tens = pk["hbm_gbs"], pk["bf16_sustained"]
    alu_peak = SMS * FP32_LANES_PER_SM * 2 * pk["sm_max_mhz"] * 1e6 / 1e12
    kinds = {k: v for k, v in prof.items() if v[1] > 0 and v[0] > 0}
    total_ms = sum(v[0] for v in kinds.values())
    bf16_rows = w.denoiser == "mlp" or (w.denoiser == "gmm" and w.gmm.get("means_bf16"))
    split = tensor_mixture(w) and not w.gmm.get("means_bf16")
    regen = launch_shape.get("regen", False)
    out = []
    for kind, (ms, n) in sorted(kinds.items(), key=lambda kv: -kv[1][0]):
        if kind in ("init", "aux"):
            continue
        per_run_launches = n / steps
        avg_s = ms / n * 1e-3
        e = {"kernel": kind, "launches_per_step": per_run_launches, "avg_launch_us": avg_s * 1e6,
             "ms_per_step": ms / steps, "share_of_kernel_time": ms / max(total_ms, 1e-9)}
        if kind in ("denoise", "fused", "draft_model", "mix"):
            if w.denoiser == "phi4":
                bound, per_run = "alu", 12.0 * d * (rows + B)
            elif w.denoiser == "mlp":
                bound, per_run = "tensor", 2.0 * sum(w.mlp_dims[i] * w.mlp_dims[i + 1] for i in range(len(w.mlp_dims) - 1)) * (rows + B)
            elif tensor_mixture(w) and kind in ("denoise", "mix"):
                # two contractions of 2 ncomp d flop per row each: "denoise" times the logits GEMM, "mix" the mixing
                # GEMM, whose tiles are not computed where every row of a block is one-hot (a row of the means table
                # is read instead): only the contraction work that ran counts as achieved
                bound, per_run = "tensor", 2.0 * w.gmm["ncomp"] * d * (rows + B)
                if kind == "mix":
                    ran, skipped = int(ctl[8]) + int(ctl[9]), int(ctl[10])
                    per_run *= ran / max(1, ran + skipped)
                    e["mixing_tiles_skipped_frac"] = skipped / max(1, ran + skipped)
            else:
                bound, per_run = "alu", 4.0 * w.gmm["ncomp"] * d * (rows + B)
            if kind == "draft_model":
                bound, per_run = "alu", 4.0 * max(1, w.gmm["ncomp"] // 2) * d * rows
            peak, unit, src = (tens, "TFLOP/s", pk["source"] + " (sustained bf16 GEMM)") if bound == "tensor" else \
                              (alu_peak, "TFLOP/s", "derived: 148 SMs x 128 fp32 lanes x 2 x max SM clock")
            if bound == "tensor" and split:
                # float operands as bf16 planes: 3 bf16 products per float product in the logits, 6 in the mixing
                # (3 for tiles whose responsibilities need only their first plane; the library counts both)
                t_full, t_brief = int(ctl[8]), int(ctl[9])
                products = 3.0 if kind == "denoise" else (6.0 * t_full + 3.0 * t_brief) / max(1, t_full + t_brief)
                peak = tens / products
                src = pk["source"] + f" (sustained bf16 GEMM / {products:.2f} bf16 products per float product)"
            ach = per_run / (ms / steps * 1e-3) / 1e12
            e.update(bound=bound, achieved=ach, peak=peak, unit=unit, frac=ach / peak, peak_source=src,
                     algorithmic_per_launch=per_run / per_run_launches)
        else:
            if kind == "verify":
                per_run = 8.0 * d * rows                         # two float streams per window position
                # requested: per evaluated position the target row (and the drafted state unless it is made
                # again in registers), per chain-window the state, the carried output, the reflected row's
                # inputs again and the two rows the advance step writes
                pos_regen = min(positions, float(int(ctl[13]) & 0x7fffffff))   # positions verified with the states made again
                req = 8.0 * d * (positions - pos_regen) + 4.0 * d * pos_regen + (8.0 * d + 4.0 * d + 8.0 * d) * cw
                e["positions_with_states_made_again"] = pos_regen
                e.update(positions_evaluated_per_step=positions, requested_bytes_per_launch=req / per_run_launches,
                         requested_achieved=req / (ms / steps * 1e-3) / 1e9,
                         requested_frac=req / (ms / steps * 1e-3) / 1e9 / hbm)
            elif kind == "draft":
                rows_w = 4.0 * d * rows + (2.0 * d * rows if bf16_rows else 0.0) + (4.0 * d * rows if split else 0.0)
                per_run = 8.0 * d * cw + rows_w
                # stored by this implementation: the float rows are skipped where nothing reads them
                rows_float = min(rows, float(int(ctl[14]) & 0x7fffffff))       # drafted rows also stored as floats
                moved = (8.0 * d * cw + rows_w - 4.0 * d * (rows - rows_float)) if bf16_rows else (8.0 * d * cw + rows_w)
                e.update(requested_bytes_per_launch=moved / per_run_launches,
                         requested_achieved=moved / (ms / steps * 1e-3) / 1e9,
                         requested_frac=moved / (ms / steps * 1e-3) / 1e9 / hbm)
                # the generator, not memory, bounds this kernel. Philox-4x32-10 takes twenty high-half and twenty
                # low-half 32 x 32-bit multiplies per four normals; measured unit rates on this part: 32 high-half
                # and 128 low-half multiplies per clock and SM, so one block keeps an SM's multiplier busy for
                # 20/32 + 20/128 = 0.78 clocks; and the kernel issues 32 instructions per lane and normal (profiler),
                # 128 lanes per clock and SM: one clock per block. The slower of the two bounds the kernel.
                drawn = d * (rows - (cw if regen else 0.0))                         # normals per run (about: the last row of a
                                                                                    # window is not drafted where verify makes it)
                sm_hz = SMS * pk["sm_max_mhz"] * 1e6
                mult_bound = 4.0 * sm_hz / (20.0 / 32.0 + 20.0 / 128.0)
                issue_bound = 4.0 * sm_hz / (4.0 * 32.0 / 128.0)
                rate = drawn / (ms / steps * 1e-3)
                e["generator"] = {"normals_per_launch": drawn / per_run_launches, "achieved_normals_per_s": rate,
                                  "multiplier_bound_normals_per_s": mult_bound, "issue_bound_normals_per_s": issue_bound,
                                  "frac_of_multiplier_bound": rate / mult_bound, "frac_of_issue_bound": rate / issue_bound}
            elif kind == "advance":
                per_run = 16.0 * d * cw
            elif kind == "softmax":
                nc = w.gmm["ncomp"] if w.denoiser == "gmm" else 0
                per_run = (4.0 + (6.0 if split else 2.0)) * nc * (rows + B)   # logits in, responsibilities out
            else:
                per_run = 0.0
            ach = per_run / (ms / steps * 1e-3) / 1e9
            e.update(bound="hbm", achieved=ach, peak=hbm, unit="GB/s", frac=ach / hbm, peak_source=pk["source"] + " (copy)",
                     algorithmic_per_launch=per_run / per_run_launches)
        t = traffic.get((w.name, kind))
        e["traffic"] = None
        if t is not None and t[1] is not None:
            e["traffic"] = t[1] * B / t[0]                       # captured at t[0] chains; traffic grows with the chains
            e["traffic_over_algorithmic"] = e["traffic"] / max(e["algorithmic_per_launch"], 1.0) if e["bound"] == "hbm" else None
        if t is not None and t[2] is not None:
            # issue bound: warp instructions per launch against one instruction per cycle and scheduler
            inst = t[2] * B / t[0]
            slots = SMS * 4 * pk["sm_max_mhz"] * 1e6
            e["issue"] = {"warp_instructions_per_launch": inst, "issue_slots_per_s": slots,
                          "frac_of_issue_peak": inst / avg_s / slots}
        out.append(e)
    return out


def acceptance_by_step(sds, w, dev, variant: str = "default", chains: int = 64, bins: int = 10):
    """Acceptance rate of the drafted steps by position in the chain (ten equal ranges of the step
    index), from a window-by-window run of a few chains outside the timed region: a draft tested
    at step k counts once, as accepted or rejected; drafts after a window's first rejection are
    never tested."""
    from paper_2501_05370_b200 import binding as sb
    B = min(chains, w.B)
    s = gpu_sampler(sds, w, variant, B=B, device=dev)
    s.set_option(s.OPT_VERIFY_EARLY_EXIT, 0)
    s.reset()
    tested, accepted = np.zeros(bins), np.zeros(bins)
    na, windows, cap = B, 0, 800                        # very long chains: the first 800 windows only
    while na > 0 and windows < cap:
        n = s.get(sb.GET_N).astype(np.int64)
        s.draft(); s.verify_window()
        js, am = s.get(sb.GET_JSTAR).astype(np.int64), s.get(sb.GET_ACCMASK).astype(np.int64)
        live = (n < w.K) & (js >= 1)
        Lt = np.minimum(w.L, w.K - n)
        last = np.minimum(js, Lt)                           # positions 1..last were tested
        for j in range(1, w.L + 1):
            m = live & (j <= last)
            if not m.any():
                break
            bi = np.minimum(bins - 1, (n[m] + j - 1) * bins // w.K)
            np.add.at(tested, bi, 1)
            np.add.at(accepted, bi, (am[m] >> (j - 1)) & 1)
        na = s.advance()
        windows += 1
    s.close()
    return {"chains": B, "bins": bins, "windows": windows,
            "rate": [round(float(a / t), 4) if t > 0 else None for a, t in zip(accepted, tested)]}


def staged_run(s, w, out, calls, rows, ref_out, steps: int):
    """ms per run and counters of sds_sample_all with SDS_OPT_STAGED_WINDOWS adaptive on an existing sampler; the
    final states must equal ref_out (the whole-window run's) bit for bit."""
    import torch
    st = torch.cuda.current_stream()
    s.set_option(s.OPT_STAGED_WINDOWS, s.STAGED_ADAPTIVE)
    for _ in range(2):
        s.sample_all(out, calls, rows)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(st)
    for _ in range(steps):
        s.sample_all(out, calls, rows)
    e1.record(st)
    e1.synchronize()
    s.set_option(s.OPT_STAGED_WINDOWS, 0)
    ms = e0.elapsed_time(e1) / steps
    c, r = calls.cpu().numpy().astype(np.int64), rows.cpu().numpy().astype(np.int64)
    return {"ms_per_run": ms, "chain_steps_per_s": w.B * w.K / (ms * 1e-3), "mean_target_calls": float(c.mean()),
            "mean_target_rows": float(r.mean()), "same_samples": bool(torch.equal(out, ref_out)), "steps_timed": steps,
            "stage": "adaptive"}


def quick_config(sds, name, dev, steps: int = 5, warmup: int = 2):
    """ms per run, chain-steps/s and the counters of another workload, in the same process."""
    import torch
    w = wl.WORKLOADS[name]
    s = gpu_sampler(sds, w, "default", device=dev)
    out = torch.empty((w.B, w.d), dtype=torch.float32, device=dev)
    calls = torch.empty((w.B,), dtype=torch.int32, device=dev)
    rows = torch.empty((w.B,), dtype=torch.int32, device=dev)
    st = torch.cuda.current_stream()
    for _ in range(warmup):
        s.sample_all(out, calls, rows)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(st)
    for _ in range(steps):
        s.sample_all(out, calls, rows)
    e1.record(st)
    e1.synchronize()
    ms = e0.elapsed_time(e1) / steps
    c, r = calls.cpu().numpy().astype(np.int64), rows.cpu().numpy().astype(np.int64)
    rws, cw = run_counts(w, "default", c, r)
    res = {"B": w.B, "d": w.d, "L": w.L, "K": w.K, "ms_per_run": ms, "chain_steps_per_s": w.B * w.K / (ms * 1e-3),
           "mean_target_calls": float(c.mean()), "mean_target_rows": float(r.mean()),
           "mean_advance": float(w.K * w.B / max(cw, 1.0)), "steps_timed": steps}
    if name in ("cfg3", "cfg4", "cfg5"):                   # (cfg1, cfg2 run as one whole-chain launch)
        res["staged_windows"] = staged_run(s, w, out, calls, rows, out.clone(), steps)
    s.close()
    del out
    torch.cuda.empty_cache()
    return res


def phi4_energies(x, side, beta):
    """Lattice energy of each row of x [n, side*side] with every neighbouring pair counted once
    (free boundaries), and the same with each pair counted from both of its sites (twice)."""
    g = np.asarray(x, np.float64).reshape(-1, side, side)
    site = ((g * g - 1.0) ** 2).sum(axis=(1, 2))
    pairs = (np.diff(g, axis=1) ** 2).sum(axis=(1, 2)) + (np.diff(g, axis=2) ** 2).sum(axis=(1, 2))
    return 0.5 * beta * pairs + site, beta * pairs + site


def phi4_energy_statistic(sds, w, dev, last: int = 500):
    """Appendix K reports the mean and standard deviation of the energy over the last 500 simulated
    samples of 500 runs, for the plain Langevin chain and for speculative sampling. Here: every chain is
    run to step K - last, then stepped window by window to the end while every accepted state (the
    samples X_{K-last+1} .. X_K) is read back; the plain chain is the same with window 1. Both energy
    conventions are reported (the sampler itself uses each pair once)."""
    import torch
    from paper_2501_05370_b200 import binding as sb
    res = {}
    for label, L in (("speculative", w.L), ("plain", 1)):
        head = w.scaled(K=w.K - last, L=L)
        s = gpu_sampler(sds, head, "default", device=dev)
        Y = s.sample_all()[0].clone()
        s.close()
        full = w.scaled(L=L)
        s = gpu_sampler(sds, full, "default", device=dev)
        s.reset()
        s.set_state(Y=Y, n=torch.full((w.B,), w.K - last, dtype=torch.int32, device=dev))
        e1, e2, na = [], [], w.B
        while na > 0:
            n0 = s.get(sb.GET_N).astype(np.int64)
            act, rowoff = s.get(sb.GET_ACT), s.get(sb.GET_ROWOFF)
            nact = int(s.get(sb.GET_CTL)[0])
            s.draft(); s.verify_window()
            X, T, js = s.get(sb.GET_X), s.get(sb.GET_TAIL), s.get(sb.GET_JSTAR).astype(np.int64)
            for si in range(nact):
                b = int(act[si]); r0 = int(rowoff[si]); Lt = min(L, w.K - int(n0[b]))
                adv = min(int(js[b]), Lt)
                states = [X[r0 + j] if j < Lt else T[b] for j in range(1, adv + 1)]   # W_1 .. W_adv (the last one reflected or accepted)
                a, b2 = phi4_energies(np.stack(states), w.phi4["side"], w.phi4["beta"])
                e1 += a.tolist(); e2 += b2.tolist()
            na = s.advance()
        s.close()
        e1, e2 = np.array(e1), np.array(e2)
        res[label] = {"samples": int(e1.size), "mean_pairs_once": float(e1.mean()), "std_pairs_once": float(e1.std()),
                      "mean_pairs_twice": float(e2.mean()), "std_pairs_twice": float(e2.std())}
    res["paper"] = {"plain": [62.27, 13.32], "speculative": [65.90, 12.48],
                    "note": "Appendix K table; the paper does not say how the pairs of its reported energy are counted"}
    return res


def independent_cost_ratio(sds, w, dev, prof, steps, rows, cw, ms_per_step):
    """Section 4.1, proposition on the average cost ratio: with C_p the cost of one draft-model call
    (one position of all chains) and C_q the cost of one batched target call, the original sampler
    costs K C_q and the speculative one (K / E[adv]) (L C_p + C_q): ratio E[adv] / (1 + L C_p / C_q).
    C_p and C_q are the measured kernel times per call; the measured ratio is the plain chain's time
    (window 1, target at every step: one call on B rows per step) over the speculative run's."""
    import torch
    dm, dn = prof.get("draft_model", (0.0, 0)), prof.get("denoise", (0.0, 0))
    sm = prof.get("softmax", (0.0, 0))
    if dm[1] == 0 or dn[1] == 0:
        return None
    windows = cw / w.B                                   # windows per run (every chain takes part in each)
    calls_q = max(1.0, float(np.ceil(dn[1] / steps / max(1.0, (dn[1] / steps) / max(windows, 1.0)))))
    c_p = dm[0] / steps / (windows * w.L)                # ms per draft-model call
    c_q = (dn[0] + sm[0]) / steps / windows              # ms per batched target call
    adv = w.K * w.B / max(cw, 1.0)
    from paper_2501_05370_b200 import binding as sb
    plain = sds.sampler_for(w.scaled(L=1), drafter_mode=sb.SDS_FROZEN_EXACT, device=dev)
    plain.set_option(plain.OPT_WHOLE_CHAIN_KERNEL, 0)
    plain.sample_all()
    st = torch.cuda.current_stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(st); plain.sample_all(); e1.record(st); e1.synchronize()
    ms_plain = e0.elapsed_time(e1)
    plain.close()
    return {"C_p_ms_per_draft_call": c_p, "C_q_ms_per_target_call": c_q, "C_p_over_C_q": c_p / c_q, "L": w.L,
            "mean_advance": adv, "predicted_cost_ratio": adv / (1.0 + w.L * c_p / c_q),
            "plain_chain_ms": ms_plain, "speculative_ms": ms_per_step, "measured_cost_ratio": ms_plain / ms_per_step,
            "note": "window kernels on both sides; the proposition counts a batched call as one unit whatever its "
                    "row count, while on the GPU a call on B*L rows costs more than a call on B rows"}


def run_gpu(args, w):
    import torch
    import paper_2501_05370_b200 as sds
    from paper_2501_05370_b200 import binding as sb
    from paper_2501_05370_b200 import sharding

    rank, local, world = sharding.dist_env()
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (no CPU fallback); use --impl reference for the oracle")
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    dist = sharding.init_process_group("nccl", dev)

    def barrier():
        sharding.barrier(dist)
        torch.cuda.synchronize()

    s = gpu_sampler(sds, w, args.variant, chain_id_offset=sharding.weak_offset(rank, w.B), device=dev)
    if args.variant == "independent":
        s.set_option(s.OPT_WHOLE_CHAIN_KERNEL, 0)      # the cost ratio is about the draft-model and target kernels
    if args.staged:
        s.set_option(s.OPT_STAGED_WINDOWS, s.STAGED_ADAPTIVE if args.staged == "adaptive" else int(args.staged))
    B, d, K = w.B, w.d, w.K
    out = torch.empty((B, d), dtype=torch.float32, device=dev)
    calls = torch.empty((B,), dtype=torch.int32, device=dev)
    rows = torch.empty((B,), dtype=torch.int32, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    if w.denoiser == "gmm":
        gp = w.gmm_params()
        if gp.means_bf16:
            means_h = torch.from_numpy((gp.means.view(np.uint32) >> np.uint32(16)).astype(np.uint16).view(np.int16)).pin_memory()
        else:
            means_h = torch.from_numpy(gp.means).pin_memory()
        logw_h = torch.from_numpy(gp.logw).pin_memory()
    else:
        means_h = logw_h = None      # network weights stay resident on the device
    out_h = torch.empty((B, d), dtype=torch.float32).pin_memory()
    calls_h = torch.empty((B,), dtype=torch.int32).pin_memory()
    rows_h = torch.empty((B,), dtype=torch.int32).pin_memory()
    stream = torch.cuda.current_stream()

    def timed(fn, steps):
        tot = 0.0
        for _ in range(steps):
            flush.fill_(1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            fn()
            e1.record(stream)
            e1.synchronize()
            tot += e0.elapsed_time(e1)
        return tot

    dev_step = lambda: s.sample_all(out, calls, rows)
    e2e_step = lambda: s.sample_all_host(means_h, logw_h, out_h, calls_h, rows_h)

    clocks = ClockSampler(local)
    if rank == 0:
        clocks.start()
        time.sleep(0.5)                 # let the sampler come up before any timed work
    for _ in range(args.warmup):
        dev_step()
    barrier()
    if rank == 0:
        clocks.mark()
    l0 = s.launch_count()
    s.profile(True)
    s.profile_read(reset=True)
    ms_total = timed(dev_step, args.steps)
    barrier()
    prof = s.profile_read(reset=True)
    s.profile(False)
    launches = s.launch_count() - l0
    clk_source = "timed region"
    if rank == 0 and clocks.proc is not None and clocks.count() < 3:
        # the timed region was shorter than the sampling period: repeat the same step, untimed, long
        # enough for the sampler to see the clocks this workload runs at
        clk_source = "the same step repeated for 0.8 s right after the timed region (it was shorter than the sampling period)"
        t_end = time.time() + 0.8
        while time.time() < t_end:
            dev_step()
        torch.cuda.synchronize()
    clk = clocks.stop() if rank == 0 else None
    if clk is not None:
        clk["source"] = clk_source
    calls_np, rows_np = calls.cpu().numpy().astype(np.int64), rows.cpu().numpy().astype(np.int64)
    ctl = s.get(sb.GET_CTL)

    # the same metric through the host-buffer entry point
    for _ in range(min(args.warmup, 3)):
        e2e_step()
    barrier()
    ms_e2e = timed(e2e_step, args.steps)
    barrier()

    # end of the run: every rank's samples in global chain order and the counters summed (off the timed path)
    all_samples, tot_calls, tot_rows = sharding.gather_results(out, calls, rows, dist)
    gathered = {"samples_shape": list(all_samples.shape), "all_finite": bool(torch.isfinite(all_samples).all().item()),
                "target_calls_all_chains": tot_calls, "target_rows_all_chains": tot_rows,
                "collectives": "none" if world == 1 else "one all-gather of the [B, d] samples, one all-reduce of the counters (NCCL)"}
    del all_samples

    ms_total, ms_e2e = sharding.max_over_ranks([ms_total, ms_e2e], dist, dev)
    if rank != 0:
        s.close()
        if dist is not None:
            dist.destroy_process_group()
        return

    pk = peaks()
    steps = args.steps
    ms_per_step = ms_total / steps
    value = world * B * K / (ms_per_step * 1e-3)
    e2e_value = world * B * K / (ms_e2e / steps * 1e-3)
    rows_per_step, windows_chains = run_counts(w, args.variant, calls_np, rows_np)
    positions = float(int(ctl[12]) & 0x7fffffff) if prof.get("verify", (0, 0))[1] > 0 else 0.0   # of the last run
    launch_shape = {"regen": bool(int(ctl[11]) & 1), "indexed_one_hot_rows": bool(int(ctl[11]) & 4)}
    traffic = measured_traffic()                        # captured at a reduced batch, scaled to this one by the chains
    rl = kernel_rooflines(w, args.variant, prof, steps, rows_per_step, windows_chains, positions, pk, ctl, traffic, launch_shape)
    if not rl:
        raise RuntimeError("no kernel of the library ran inside the timed region")
    dom = rl[0]
    roofline = {k: dom.get(k) for k in ("kernel", "bound", "achieved", "peak", "unit", "frac", "traffic", "peak_source",
                                        "avg_launch_us", "launches_per_step", "share_of_kernel_time")}
    roofline["kernel_ms_per_step"] = {k: v[0] / steps for k, v in prof.items() if v[1] > 0}

    acc_profile = acceptance_by_step(sds, w, dev, args.variant)
    extra = {}
    if prof.get("verify", (0, 0))[1] > 0 and args.variant == "default" and not args.no_extras:
        # the streaming kernels with every position of every window evaluated and the drafted rows read back
        # (options off, outside the timed region): the two-stream reduction of the verify step as such
        s.set_option(s.OPT_VERIFY_EARLY_EXIT, 0); s.set_option(s.OPT_REGEN_DRAFTS, 0)
        dev_step()
        s.profile(True); s.profile_read(reset=True)
        for _ in range(3):
            dev_step()
        prof_all = s.profile_read(reset=True)
        s.profile(False)
        ctl_all = s.get(sb.GET_CTL)
        rl_all = kernel_rooflines(w, args.variant, prof_all, 3, rows_per_step, windows_chains, float(int(ctl_all[12]) & 0x7fffffff),
                                  pk, ctl_all, {}, {"regen": False})
        extra["rooflines_every_position"] = [e for e in rl_all if e["kernel"] in ("verify", "draft", "advance")]
        s.set_option(s.OPT_VERIFY_EARLY_EXIT, 1); s.set_option(s.OPT_REGEN_DRAFTS, 1)
    if prof.get("verify", (0, 0))[1] > 0 and args.variant == "default" and not args.no_extras and not args.staged:
        # the same run with every window evaluated in stages (same samples, checked here against the timed run's):
        # reported beside the headline, which stays on whole windows as the paper states the method
        ref_out = out.clone()
        extra["staged_windows"] = staged_run(s, w, out, calls, rows, ref_out, min(steps, 5))
    if w.denoiser == "phi4" and not args.no_extras:
        extra["phi4_energy"] = phi4_energy_statistic(sds, w, dev)
    if args.variant == "independent":
        extra["cost_ratio"] = independent_cost_ratio(sds, w, dev, prof, steps, rows_per_step, windows_chains, ms_per_step)
    s.close()
    del out, flush
    torch.cuda.empty_cache()
    if world == 1 and not args.no_extras and args.variant == "default" and not args.chains:
        extra["per_config"] = {w.name: {"B": B, "d": d, "L": w.L, "K": K, "ms_per_run": ms_per_step, "chain_steps_per_s": value,
                                        "mean_target_calls": float(calls_np.mean()), "mean_target_rows": float(rows_np.mean()),
                                        "mean_advance": float(K * B / max(windows_chains, 1)), "steps_timed": steps}}
        for name in ("cfg1", "cfg2", "cfg3", "cfg4", "cfg5"):
            if name != w.name:
                extra["per_config"][name] = quick_config(sds, name, dev)

    osteps, sec, what = oracle_time(w, args.cpu_seconds, variant=args.variant)
    cpu = {"value": osteps / sec, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": what}
    psteps, psec = oracle_plain_time(w, max(1.0, args.cpu_seconds / 5))
    cpu["plain_chain_value"] = psteps / psec          # the oracle's plain sequential chain, same unit, for context

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": ("bf16" if w.dtype == "bf16" else "f32"), "data": "synthetic", "config": workload_config(w, args),
        "nfe": {"K": K, "mean_target_calls": float(calls_np.mean()), "mean_target_rows": float(rows_np.mean()),
                "mean_advance": float(K * B / max(windows_chains, 1)), "calls_saved_frac": float(1 - calls_np.mean() / K),
                "acceptance_by_step": acc_profile},
        "e2e": {"value": e2e_value, "unit": UNIT, "ms_per_step": ms_e2e / steps,
                "h2d_bytes_per_step": int(means_h.numel() * means_h.element_size() + logw_h.numel() * 4) if means_h is not None else 0,
                "d2h_bytes_per_step": int(out_h.numel() * 4 + calls_h.numel() * 4 + rows_h.numel() * 4)},
        "gpu_launches": int(launches),
        "roofline": roofline, "rooflines": rl, "gathered": gathered, "cpu_baseline": cpu, "clocks": clk,
    }
    line.update(extra)
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="sds", choices=["sds", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(wl.WORKLOADS))
    ap.add_argument("--cpu-seconds", type=float, default=15.0, help="budget of the cpu_baseline leg")
    ap.add_argument("--chains", type=int, default=0, help="chains per GPU (default: the workload's own B)")
    ap.add_argument("--variant", default="default", choices=VARIANTS,
                    help="another drafter or accept test on the same workload (default: the workload's own)")
    ap.add_argument("--staged", default="", help="evaluate every window in stages: a stage length, or 'adaptive' "
                    "(same samples; default: whole windows, as the paper states the method)")
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the per-workload table and the lattice energy statistic (profiler captures)")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "sds":
        args.warmup = 3
    w = wl.WORKLOADS[args.workload]
    if args.chains > 0:
        w = w.scaled(B=args.chains)
    if args.impl == "reference":
        run_reference(args, w)
        return
    from paper_2501_05370_b200 import sharding
    if args.gpus > 1 and not sharding.under_launcher():
        # started as `python bench.py --gpus N`: become N ranks, one per GPU
        sys.exit(sharding.launch_ranks(args.gpus, os.path.abspath(__file__), sys.argv[1:]))
    run_gpu(args, w)


if __name__ == "__main__":
    main()
