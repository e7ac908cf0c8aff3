"""World-size-2 check (gloo, CPU) of the multi-rank host logic: id ranges tile the batch, the
per-rank results stacked in rank order equal the unsharded run bit for bit (the random numbers are
keyed by global chain id), and the timing reduction takes the maximum over ranks. The per-rank
work here is the oracle's chain; the GPU shard test in test_gpu_parity.py covers the CUDA path."""
import os
import socket

import numpy as np
import pytest
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2501_05370_b200 import sharding as sh
from oracle import sds_oracle as o
import workloads as wl

TOTAL, SEED = 7, 77


def _setup():
    w = wl.WORKLOADS["cfg1"].scaled(K=20)
    gp = w.gmm_params()
    a, c, sig, abar = o.ddpm_affine(wl.beta_linear(w.K))
    den = lambda x, k: o.gmm_posterior_mean(x, abar[k], gp.means, gp.logw, gp.comp_std)
    return w, den, a, c, sig


def _run_range(begin, end):
    w, den, a, c, sig = _setup()
    ys, calls = [], []
    for b in range(begin, end):
        r = o.speculative_chain(den, a, c, sig, w.L, SEED, b, w.d)
        ys.append(r["Y"]); calls.append(r["nfe_calls"])
    return np.array(ys).reshape(-1, w.d), np.array(calls)


def _worker(rank, world, port, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        b, e = sh.chain_range(rank, world, TOTAL)
        y, calls = _run_range(b, e)
        full = sh.gather_rows(y, dist)
        allcalls = sh.gather_rows(calls.reshape(-1, 1), dist)
        tmax = sh.max_over_ranks([10.0 + rank, 5.0 - rank], dist)
        if rank == 0:
            q.put((full, allcalls[:, 0], tmax, (b, e)))
        dist.barrier()
    finally:
        dist.destroy_process_group()


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


def test_two_ranks_reproduce_the_unsharded_run():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    full, calls, tmax, rng0 = q.get(timeout=180)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    ref_y, ref_calls = _run_range(0, TOTAL)
    assert rng0 == (0, 4)
    assert np.array_equal(full, ref_y) and np.array_equal(calls, ref_calls)
    assert tmax == [11.0, 5.0]
