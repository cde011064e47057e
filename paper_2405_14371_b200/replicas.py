"""Replicas: the path does not shard across GPUs (one shard is one device's work), so N GPUs run N
independent copies of the workload, one process per GPU.  This module holds the little that the
copies share: the process-group set-up, a barrier, and the reduction that turns per-rank times into
the job's figure (units of all ranks over the SLOWEST rank's time).  No data-path collective exists.
The same code runs over NCCL on GPUs and over gloo on CPUs (tests)."""
from __future__ import annotations

import os

import torch


def launch_plan(n_gpus: int, environ, argv):
    """How a benchmark asked for `n_gpus` replicas should start them.  None: run in this process (one GPU, or
    this process already is a rank of a running job: WORLD_SIZE is set).  Otherwise the command line that
    starts the same script with the same arguments as `n_gpus` ranks of one node under torch.distributed.run
    (rendezvous on 127.0.0.1: the host name of a container may not resolve)."""
    import sys

    if n_gpus <= 1 or "WORLD_SIZE" in environ:
        return None
    return [sys.executable, "-m", "torch.distributed.run", "--standalone", "--nnodes=1", f"--nproc-per-node={n_gpus}",
            "--local-addr", "127.0.0.1"] + list(argv)


def setup(backend: str | None = None):
    """(rank, local_rank, world_size); initialises torch.distributed when WORLD_SIZE > 1."""
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if backend is None:
        backend = "nccl" if torch.cuda.is_available() else "gloo"
    if backend == "nccl":
        torch.cuda.set_device(local if world > 1 else 0)
    if world > 1:
        import torch.distributed as dist

        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        if not dist.is_initialized():
            if backend == "nccl":
                dist.init_process_group("nccl", device_id=torch.device("cuda", local))
            else:
                dist.init_process_group(backend)
    return rank, local, world


def _device():
    import torch.distributed as dist

    return torch.device("cuda", torch.cuda.current_device()) if dist.get_backend() == "nccl" else torch.device("cpu")


def barrier(world: int) -> None:
    if world > 1:
        import torch.distributed as dist

        dist.barrier()
    if torch.cuda.is_available():
        torch.cuda.synchronize()


def max_over_ranks(x: float, world: int) -> float:
    """The slowest rank's figure: a job of replicas ends when its last replica does."""
    if world <= 1:
        return x
    import torch.distributed as dist

    t = torch.tensor([x], dtype=torch.float64, device=_device())
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t[0])


def job_throughput(units_per_rank: float, ms_this_rank: float, world: int) -> float:
    """Units per second of the whole job: every rank processed `units_per_rank`, the job took as long
    as its slowest rank."""
    return units_per_rank * world / (max_over_ranks(ms_this_rank, world) / 1e3)
