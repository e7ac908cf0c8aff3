#!/usr/bin/env python
"""Benchmark of the speculative-sampling hot path.

One "step" is one full sds_sample_all over a batch of chains of the chosen workload: initial
state and target call, then draft / batched target / verify / advance windows until every chain
has made its K transitions. The metric is accepted chain-steps per second (B*K per run; both
accepted and reflected steps are valid target steps).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2] [--impl reference]

Prints one JSON line (rank 0). N > 1 (under torch.distributed.run): chains are sharded across
ranks by global chain id, no collective on the data path (weak scaling: B chains per rank).
--impl reference times the CPU oracle, as it stands, on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
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
# DRAM bytes (read + written) of one launch of the dominant kernel, from the profiler's counters of that
# kernel as it stands, at the workload's own size (profiles/k_fused_small_cfg2.md). An entry goes back to
# None when its kernel's source changes. Keyed by (workload, variant, kernel kind).
CAPTURED_TRAFFIC = {("cfg2", "default", "fused"): 82176.0}


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
        s.set_projection(torch.from_numpy(sb.projection_basis(proj_matrix(w))).to(kw.get("device", "cuda:0")))
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
    n, steps, Kp = 0, 0, min(w.K, 2 * w.L)
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
    n, steps, Kp = 0, 0, min(w.K, 2 * w.L)
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

def algorithmic(kind: str, w, rows_per_step: float, windows_chains: float, launches: float):
    """Algorithmic bytes or flops one average launch of `kind` must move / compute.
    rows_per_step: target rows verified per step (sum of window lengths); windows_chains: chain-windows."""
    d = w.d
    if kind == "verify":        # two fp32 streams per verified chain-step (target output + drafted state)
        return "hbm", 8.0 * d * rows_per_step / launches
    if kind == "draft":         # read state + carried output, write the drafted rows
        return "hbm", (8.0 * d * windows_chains + 4.0 * d * rows_per_step) / launches
    if kind == "advance":
        return "hbm", 16.0 * d * windows_chains / launches
    if kind in ("denoise", "fused"):
        if w.denoiser == "phi4":    # four neighbour differences, the site term, one fma per site
            return "alu", 12.0 * d * (rows_per_step + w.B) / launches
        if w.denoiser == "mlp":     # 2 * sum of layer products per row, bf16 tensor cores
            per_row = 2.0 * sum(w.mlp_dims[i] * w.mlp_dims[i + 1] for i in range(len(w.mlp_dims) - 1))
            return "tensor", per_row * (rows_per_step + w.B) / launches
        per_row = 4.0 * w.gmm["ncomp"] * d      # logits + mixing contractions
        if w.gmm.get("means_bf16"):
            bound = "tensor"
        elif kind == "denoise" and 32 < w.gmm["ncomp"] <= 1024 and w.gmm["ncomp"] % 128 == 0 and d % 128 == 0:
            bound = "tensor_split"              # float operands as bf16 planes: 3 products (logits) + 6 (mixing)
        else:
            bound = "alu"
        return bound, per_row * (rows_per_step + w.B) / launches
    return "hbm", 0.0


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


def run_gpu(args, w):
    import torch
    import torch.distributed as dist
    import paper_2501_05370_b200 as sds

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (no CPU fallback); use --impl reference for the oracle")
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(dev))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    from paper_2501_05370_b200 import sharding
    s = gpu_sampler(sds, w, args.variant, chain_id_offset=sharding.weak_offset(rank, w.B), device=dev)
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

    # the same metric through the host-buffer entry point
    for _ in range(min(args.warmup, 3)):
        e2e_step()
    barrier()
    ms_e2e = timed(e2e_step, args.steps)
    barrier()

    ms_total, ms_e2e = sharding.max_over_ranks([ms_total, ms_e2e], dist if world > 1 else None, dev)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    pk = peaks()
    steps = args.steps
    ms_per_step = ms_total / steps
    value = world * B * K / (ms_per_step * 1e-3)
    e2e_value = world * B * K / (ms_e2e / steps * 1e-3)
    if getattr(w, "drafter_mode", 0) == 1 or args.variant == "exact":
        # drafter evaluated at Y_n: no initial call, two sequential calls per window (one for a last window of one row)
        rows_per_step = float(rows_np.sum())
        windows_chains = float(np.ceil(calls_np / 2.0).sum())
    elif args.variant == "independent":                       # no initial call, one target call per window
        rows_per_step = float(rows_np.sum())
        windows_chains = float(calls_np.sum())
    elif args.variant == "picard2":                           # initial call, then 2 draft calls + 1 verify call per window
        windows_chains = float(np.ceil((calls_np - 1) / 3.0).sum())
        rows_per_step = float(w.L * windows_chains)           # rows of the verify calls (full windows assumed)
    else:
        rows_per_step = float(rows_np.sum() - B)              # rows verified (the initial call is not a window)
        windows_chains = float(calls_np.sum() - B)
    kinds = {k: v for k, v in prof.items() if v[1] > 0}
    dom = max(kinds, key=lambda k: kinds[k][0]) if kinds else "fused"
    dom_ms, dom_n = kinds.get(dom, (ms_total, steps))
    denoise_launch_groups = {"mlp": len(w.mlp_dims) - 1}.get(w.denoiser, 3 if (w.denoiser == "gmm" and w.gmm.get("means_bf16")) else 1)
    from paper_2501_05370_b200 import binding as sb
    split_products, t_full, t_brief = 4.5, 0, 0
    bound, per_launch = algorithmic(dom, w, rows_per_step, windows_chains, dom_n / steps)
    avg_s = dom_ms / max(dom_n, 1) * 1e-3
    if bound == "hbm":
        achieved, peak, unit = per_launch / avg_s / 1e9, pk["hbm_gbs"], "GB/s"
    elif bound == "tensor":
        achieved, peak, unit = per_launch / avg_s / 1e12, pk["bf16_sustained"], "TFLOP/s"
    elif bound == "tensor_split":
        # float-equivalent flops: the logits contraction costs 3 bf16 products per float product, the
        # mixing contraction 6 (or 3, see below), and the two contractions are the same size
        # where a tile of responsibilities needs only its first plane (one-hot rows) the mixing contraction
        # runs 3 products instead of 6; the library counts both kinds of tile
        ctl = s.get(sb.GET_CTL)
        t_full, t_brief = int(ctl[8]), int(ctl[9])
        mix_products = (6.0 * t_full + 3.0 * t_brief) / max(1, t_full + t_brief)
        split_products = (3.0 + mix_products) / 2.0
        achieved, peak, unit = per_launch / avg_s / 1e12, pk["bf16_sustained"] / split_products, "TFLOP/s"
    else:
        peak = SMS * FP32_LANES_PER_SM * 2 * pk["sm_max_mhz"] * 1e6 / 1e12
        achieved, unit = per_launch / avg_s / 1e12, "TFLOP/s"
    roofline = {"kernel": dom, "bound": "tensor" if bound == "tensor_split" else bound, "achieved": achieved, "peak": peak, "unit": unit,
                "frac": achieved / peak,
                "traffic": CAPTURED_TRAFFIC.get((w.name, args.variant, dom)) if not args.chains else None,
                "peak_source": (pk["source"] + {"tensor": " (sustained bf16 GEMM)", "tensor_split": f" (sustained bf16 GEMM / {split_products:.2f}: 3 bf16 products per float product in the logits, 6 in the mixing, 3 for tiles of one-hot rows: {t_brief} of {t_full + t_brief} tiles)"}.get(bound, " (copy)")) if bound != "alu"
                else "derived: 148 SMs x 128 fp32 lanes x 2 x max SM clock",
                "avg_launch_us": avg_s * 1e6, "launches_per_step": dom_n / steps,
                "share_of_kernel_time": dom_ms / max(sum(v[0] for v in kinds.values()), 1e-9),
                "kernel_ms_per_step": {k: v[0] / steps for k, v in kinds.items()}}

    acc_profile = acceptance_by_step(sds, w, dev, args.variant)

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
        "roofline": roofline, "cpu_baseline": cpu, "clocks": clk,
    }
    print(json.dumps(line), flush=True)
    s.close()
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="sds", choices=["sds", "reference"])
    ap.add_argument("--workload", default="cfg2", choices=sorted(wl.WORKLOADS))
    ap.add_argument("--cpu-seconds", type=float, default=15.0, help="budget of the cpu_baseline leg")
    ap.add_argument("--chains", type=int, default=0, help="chains per GPU (default: the workload's own B)")
    ap.add_argument("--variant", default="default", choices=VARIANTS,
                    help="another drafter or accept test on the same workload (default: the workload's own)")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "sds":
        args.warmup = 3
    w = wl.WORKLOADS[args.workload]
    if args.chains > 0:
        w = w.scaled(B=args.chains)
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_gpu(args, w)


if __name__ == "__main__":
    main()
