"""One rank of the launcher test (run by torch.distributed.run, gloo, CPU). The step is a stand-in
for the GPU run: the oracle's chains of this rank's shard (global chain ids rank * B ...), as CPU
tensors. Everything around the step is what bench.py does on GPUs: the environment of the launcher,
the process group, the shard offset, the gather of the final samples, the sum of the counters and
the maximum of the timings. Rank 0 writes the gathered result to the file named on the command line."""
import json
import sys
import time

import numpy as np
import torch

from paper_2501_05370_b200 import sharding as sh
from oracle import sds_oracle as o
import workloads as wl


def main():
    out_path, B, seed = sys.argv[1], int(sys.argv[2]), int(sys.argv[3])
    rank, local, world = sh.dist_env()
    dist = sh.init_process_group("gloo")
    w = wl.WORKLOADS["cfg1"].scaled(K=20)
    gp = w.gmm_params()
    a, c, sig, abar = o.ddpm_affine(wl.beta_linear(w.K))
    den = lambda x, k: o.gmm_posterior_mean(x, abar[k], gp.means, gp.logw, gp.comp_std)
    off = sh.weak_offset(rank, B)
    t0 = time.perf_counter()
    res = [o.speculative_chain(den, a, c, sig, w.L, seed, off + b, w.d) for b in range(B)]
    ms = 1e3 * (time.perf_counter() - t0)
    sh.barrier(dist)
    samples = torch.from_numpy(np.array([r["Y"] for r in res]).reshape(B, w.d))
    calls = torch.tensor([r["nfe_calls"] for r in res], dtype=torch.int32)
    rows = torch.tensor([r["nfe_rows"] for r in res], dtype=torch.int32)
    all_samples, tot_calls, tot_rows = sh.gather_results(samples, calls, rows, dist)
    tmax = sh.max_over_ranks([ms, 100.0 + rank], dist)
    if rank == 0:
        np.save(out_path + ".npy", all_samples.numpy())
        json.dump({"world": world, "n_gpus": world, "calls": tot_calls, "rows": tot_rows, "tmax": tmax,
                   "ms_rank0": ms}, open(out_path, "w"))
    sh.barrier(dist)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
