"""Chain sharding across ranks: chains are independent and the generator is keyed by the global
chain id, so a rank needs only its id range. No collective touches the data path; after the timed
region the ranks gather the final samples and sum the counters (one all-gather, one all-reduce)
and exchange the timing maximum.

This module also starts the ranks: one process per GPU under torch.distributed.run, rendezvous on
127.0.0.1. The same helpers run on CPU tensors with the gloo backend.
"""
from __future__ import annotations

import os
import socket
import subprocess
import sys


def chain_range(rank: int, world: int, total_chains: int):
    """Contiguous [begin, end) of global chain ids for `rank` when `total_chains` are split as
    evenly as possible (the first total % world ranks get one more)."""
    if not (0 <= rank < world) or total_chains < 0:
        raise ValueError("bad rank/world/total")
    base, extra = divmod(total_chains, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def weak_offset(rank: int, chains_per_rank: int) -> int:
    """Global id of a rank's first chain when every rank runs the same number of chains."""
    return rank * chains_per_rank


# ---------------------------------------------------------------------------------------------
# starting the ranks
# ---------------------------------------------------------------------------------------------

def free_port() -> int:
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def torchrun_command(nproc: int, script: str, script_args, port: int | None = None):
    """The command that runs `script` as nproc ranks on this node (one per GPU)."""
    if nproc < 1:
        raise ValueError("nproc must be positive")
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={nproc}",
            "--master-addr", "127.0.0.1", "--master-port", str(port or free_port()), script] + list(script_args)


def launch_ranks(nproc: int, script: str, script_args, env=None, timeout=None) -> int:
    """Runs `script` as nproc ranks and returns the launcher's exit code (output is inherited)."""
    return subprocess.run(torchrun_command(nproc, script, script_args), env=env, timeout=timeout).returncode


def under_launcher() -> bool:
    return "WORLD_SIZE" in os.environ and "RANK" in os.environ


def dist_env():
    """(rank, local_rank, world_size) from the launcher's environment (0, 0, 1 without one)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init_process_group(backend: str, device=None):
    """Joins the process group of the launcher (nccl on GPUs, gloo on CPU); returns torch.distributed,
    or None when there is only one rank."""
    rank, local, world = dist_env()
    if world <= 1:
        return None
    import torch.distributed as dist
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    kw = {}
    if backend == "nccl" and device is not None:
        import torch
        kw["device_id"] = torch.device(device)
    dist.init_process_group(backend, **kw)
    return dist


# ---------------------------------------------------------------------------------------------
# what the ranks exchange (all off the timed path)
# ---------------------------------------------------------------------------------------------

def max_over_ranks(values, dist=None, device=None):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return [float(v) for v in values]
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def all_gather_rows(local, dist=None):
    """All ranks' [n, d] tensors (same shape on every rank) stacked in rank order, i.e. in global chain
    order for weak_offset shards: one all-gather on the tensors' own device."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return local
    import torch
    world = dist.get_world_size()
    out = torch.empty((world * local.shape[0],) + tuple(local.shape[1:]), dtype=local.dtype, device=local.device)
    dist.all_gather_into_tensor(out, local.contiguous())
    return out


def sum_over_ranks(local, dist=None):
    """Element-wise sum of a tensor over all ranks (one all-reduce); the input is left untouched."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return local
    t = local.clone()
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return t


def barrier(dist=None):
    if dist is not None and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()


def gather_results(samples, nfe_calls, nfe_rows, dist=None):
    """End of a sharded run: every rank's final samples [B, d] stacked in global chain order (one
    all-gather) and the counters summed over all chains of all ranks (one all-reduce).
    Returns (all_samples [world * B, d], total target calls, total target rows)."""
    import torch
    all_samples = all_gather_rows(samples, dist)
    local = torch.stack([nfe_calls.sum(dtype=torch.int64), nfe_rows.sum(dtype=torch.int64)])
    totals = sum_over_ranks(local, dist)
    return all_samples, int(totals[0]), int(totals[1])
