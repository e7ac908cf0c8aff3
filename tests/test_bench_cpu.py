"""Host-side logic of bench.py that needs no GPU: the counters-to-units arithmetic, the per-kernel
roofline entries built from event times, and the reader of the profiler-traffic table (rows whose
kernel source has changed since the capture are dropped)."""
import hashlib
import os

import numpy as np

import bench
import workloads as wl

PK = dict(hbm_gbs=6500.0, bf16_tflops=1600.0, bf16_sustained=1400.0, sm_max_mhz=1965.0, source="measured")


def test_run_counts_follow_the_counters_of_each_drafter():
    w = wl.WORKLOADS["cfg4"]
    calls = np.array([5, 7], dtype=np.int64)           # 1 initial call + windows
    rows = np.array([1 + 4 * 16, 1 + 6 * 16], dtype=np.int64)
    assert bench.run_counts(w, "default", calls, rows) == (160.0, 10.0)
    # drafter evaluated at Y_n: two calls per window, no initial call
    assert bench.run_counts(w, "exact", np.array([8, 9]), np.array([64, 70])) == (134.0, 9.0)
    assert bench.run_counts(w, "independent", np.array([4, 6]), np.array([64, 96])) == (160.0, 10.0)


def test_kernel_rooflines_from_event_times():
    w = wl.WORKLOADS["cfg4"]
    steps, rows, cw = 2, 1.8e6, 1.2e5
    ctl = np.zeros(16, dtype=np.int64)
    ctl[8], ctl[10], ctl[13], ctl[14] = 1000, 3000, 4.0e5, 3.0e5       # a quarter of the mixing tiles ran
    prof = {"denoise": (100.0, 276), "mix": (20.0, 276), "draft": (80.0, 276), "verify": (60.0, 276), "softmax": (8.0, 276),
            "init": (0.1, 2), "aux": (0.1, 4), "advance": (0.0, 0)}
    rl = bench.kernel_rooflines(w, "default", prof, steps, rows, cw, 5.0e5, PK, ctl, {("cfg4", "denoise"): (256, 1.7e8, 1.7e7)},
                                {"regen": True})
    by = {e["kernel"]: e for e in rl}
    assert [e["kernel"] for e in rl][0] == "denoise" and set(by) == {"denoise", "mix", "draft", "verify", "softmax"}
    d = by["denoise"]
    flops = 2.0 * 1024 * 16384 * (rows + w.B)
    assert d["bound"] == "tensor" and abs(d["achieved"] - flops / 0.050 / 1e12) < 1e-6 * d["achieved"]
    assert abs(d["frac"] - d["achieved"] / PK["bf16_sustained"]) < 1e-12
    assert abs(d["traffic"] - 1.7e8 * w.B / 256) < 1.0                  # captured at 256 chains, scaled by the chains
    assert abs(d["issue"]["warp_instructions_per_launch"] - 1.7e7 * 4) < 1.0
    m = by["mix"]
    assert abs(m["mixing_tiles_skipped_frac"] - 0.75) < 1e-12
    assert abs(m["achieved"] - 0.25 * flops / 0.010 / 1e12) < 1e-6 * m["achieved"]
    v = by["verify"]
    assert v["bound"] == "hbm" and abs(v["algorithmic_per_launch"] - 8.0 * w.d * rows / 138) < 1.0
    req = 8.0 * w.d * (5.0e5 - 4.0e5) + 4.0 * w.d * 4.0e5 + 20.0 * w.d * cw
    assert abs(v["requested_bytes_per_launch"] - req / 138) < 1.0
    dr = by["draft"]
    assert abs(dr["generator"]["issue_bound_normals_per_s"] - 4.0 * 148 * 1965.0e6) < 1.0
    assert dr["generator"]["multiplier_bound_normals_per_s"] > dr["generator"]["issue_bound_normals_per_s"]
    assert dr["requested_bytes_per_launch"] < dr["algorithmic_per_launch"]   # float rows skipped in most windows


def test_traffic_table_rows_are_dropped_when_the_kernel_source_has_changed(tmp_path, monkeypatch):
    src = os.path.join(bench.CSRC, "sds_tc.cu")
    good = hashlib.sha256(open(src, "rb").read()).hexdigest()[:12]
    table = tmp_path / "dram_traffic.md"
    table.write_text("\n".join([
        "| workload | kernel kind | chains | DRAM bytes per launch | warp instructions per launch | source file:hash | note |",
        "|---|---|---|---|---|---|---|",
        f"| cfg4 | denoise | 256 | 1.7e8 | 1.6e7 | sds_tc.cu:{good} | logits GEMM |",
        "| cfg4 | mix | 256 | 3.0e8 | - | sds_tc.cu:000000000000 | stale: the hash is not the file's |",
        f"| cfg4 | softmax | 256 | 1.6e7 | 5.6e6 | no_such_file.cu:{good} | unknown file |",
    ]))
    monkeypatch.setattr(bench, "TRAFFIC_TABLE", str(table))
    t = bench.measured_traffic()
    assert t == {("cfg4", "denoise"): (256, 1.7e8, 1.6e7)}


def test_lattice_energy_conventions():
    x = np.array([[0.5, -0.25, 0.0, 0.0]])
    once, twice = bench.phi4_energies(x, 2, 3.0)
    pairs = (0.5 + 0.25) ** 2 + 0.5 ** 2 + 0.25 ** 2
    site = (0.25 - 1) ** 2 + (0.0625 - 1) ** 2 + 2.0
    assert abs(once[0] - (1.5 * pairs + site)) < 1e-12 and abs(twice[0] - (3.0 * pairs + site)) < 1e-12


def test_bench_started_without_a_launcher_becomes_n_ranks(monkeypatch):
    """`python bench.py --gpus 4` with no launcher around it re-executes itself as four ranks through
    sharding.launch_ranks (one per GPU, loopback rendezvous) and exits with the launcher's code; under a
    launcher (WORLD_SIZE and RANK set) it does not launch again."""
    import sys
    from paper_2501_05370_b200 import sharding
    calls = []
    monkeypatch.setattr(sharding, "launch_ranks", lambda n, script, argv, **kw: calls.append((n, script, list(argv))) or 7)
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "4", "--steps", "2"])
    monkeypatch.delenv("WORLD_SIZE", raising=False)
    monkeypatch.delenv("RANK", raising=False)
    try:
        bench.main()
        raise AssertionError("bench.main() should have exited with the launcher's code")
    except SystemExit as e:
        assert e.code == 7
    assert calls == [(4, os.path.abspath(bench.__file__), ["--gpus", "4", "--steps", "2"])]
    # inside a rank: no second launch (run_gpu is reached instead)
    reached = []
    monkeypatch.setattr(bench, "run_gpu", lambda args, w: reached.append((args.gpus, w.name)))
    monkeypatch.setenv("WORLD_SIZE", "4")
    monkeypatch.setenv("RANK", "1")
    bench.main()
    assert reached == [(4, "cfg4")] and len(calls) == 1
