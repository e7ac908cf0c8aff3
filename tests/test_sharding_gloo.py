"""World-size-2 check (gloo, CPU) of the multi-rank host logic, through the launcher bench.py uses:
sharding.launch_ranks starts two ranks of tests/rank_stub.py under torch.distributed.run; each runs
its shard of chains (the oracle's chains stand in for the GPU step) and the ranks finish exactly as
bench.py does: all-gather of the final samples, all-reduce of the counters, maximum of the timings.
The gathered result must equal the unsharded run bit for bit (the random numbers are keyed by
global chain id). The GPU shard test in test_gpu_parity.py covers the CUDA path."""
import json
import os
import sys

import numpy as np
import pytest

from paper_2501_05370_b200 import sharding as sh
from oracle import sds_oracle as o
import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
B, SEED = 3, 77


def _unsharded(total):
    w = wl.WORKLOADS["cfg1"].scaled(K=20)
    gp = w.gmm_params()
    a, c, sig, abar = o.ddpm_affine(wl.beta_linear(w.K))
    den = lambda x, k: o.gmm_posterior_mean(x, abar[k], gp.means, gp.logw, gp.comp_std)
    res = [o.speculative_chain(den, a, c, sig, w.L, SEED, b, w.d) for b in range(total)]
    return (np.array([r["Y"] for r in res]).reshape(total, w.d), sum(r["nfe_calls"] for r in res),
            sum(r["nfe_rows"] for r in res))


def test_chain_range_tiles_the_batch():
    for world in (1, 2, 3, 8):
        for total in (0, 1, 7, 64, 4097):
            r = [sh.chain_range(k, world, total) for k in range(world)]
            assert r[0][0] == 0 and r[-1][1] == total
            assert all(r[i][1] == r[i + 1][0] for i in range(world - 1))
            sizes = [e - b for b, e in r]
            assert max(sizes) - min(sizes) <= 1
    assert sh.weak_offset(3, 4096) == 12288
    with pytest.raises(ValueError):
        sh.chain_range(2, 2, 5)
    assert sh.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]


def test_single_rank_helpers_are_the_identity():
    import torch
    x = torch.arange(6.0).reshape(3, 2)
    assert sh.all_gather_rows(x) is x and sh.sum_over_ranks(x) is x
    s, c, r = sh.gather_results(x, torch.tensor([1, 2, 3], dtype=torch.int32), torch.tensor([4, 5, 6], dtype=torch.int32))
    assert s is x and (c, r) == (6, 15)
    assert sh.dist_env()[2] >= 1


def test_launcher_command_names_one_rank_per_gpu_on_the_loopback_address():
    cmd = sh.torchrun_command(4, "bench.py", ["--gpus", "4"], port=29511)
    assert cmd[0] == sys.executable and cmd[1:3] == ["-m", "torch.distributed.run"]
    assert "--nproc-per-node=4" in cmd and "--nnodes=1" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[cmd.index("--master-port") + 1] == "29511"
    assert cmd[-3:] == ["bench.py", "--gpus", "4"]
    with pytest.raises(ValueError):
        sh.torchrun_command(0, "bench.py", [])


def test_two_ranks_started_by_the_launcher_reproduce_the_unsharded_run(tmp_path):
    out = str(tmp_path / "ranks.json")
    env = dict(os.environ)
    env["PYTHONPATH"] = ROOT + os.pathsep + env.get("PYTHONPATH", "")
    env.pop("WORLD_SIZE", None); env.pop("RANK", None)
    rc = sh.launch_ranks(2, os.path.join(ROOT, "tests", "rank_stub.py"), [out, str(B), str(SEED)], env=env, timeout=600)
    assert rc == 0
    info = json.load(open(out))
    got = np.load(out + ".npy")
    want, calls, rows = _unsharded(2 * B)
    assert info["world"] == 2 and info["n_gpus"] == 2
    assert got.shape == want.shape and np.array_equal(got, want)      # rank order = global chain order, bit for bit
    assert (info["calls"], info["rows"]) == (calls, rows)
    assert info["tmax"][1] == 101.0 and info["tmax"][0] >= info["ms_rank0"]
