"""Multi-GPU plumbing.  The compression pass shards by worker: every data-parallel worker owns its
gradients, its EF21 state, its budget and its DP, so ranks exchange nothing on the data path.  What
ranks do share is the clock: a barrier around the timed region and a max-reduction of the measured
time.  Works with NCCL (one process per GPU) and with gloo (CPU tests)."""
from __future__ import annotations

import os


def world():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def init_distributed(backend="nccl"):
    """Joins the process group described by RANK / WORLD_SIZE / MASTER_* when WORLD_SIZE > 1."""
    rank, size = world()
    if size <= 1:
        return rank, size
    import torch.distributed as dist

    if not dist.is_initialized():
        if backend == "nccl":
            import torch

            torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", 0)))
        dist.init_process_group(backend=backend, rank=rank, world_size=size)
    return rank, size


def _active():
    try:
        import torch.distributed as dist

        return dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1
    except Exception:
        return False


def barrier():
    if _active():
        import torch.distributed as dist

        dist.barrier()


def max_over_ranks(x: float) -> float:
    """Largest value of `x` over all ranks (the job is as slow as its slowest rank)."""
    if not _active():
        return float(x)
    import torch
    import torch.distributed as dist

    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([float(x)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def shard_workers(n_workers_total: int, rank: int, size: int):
    """Contiguous block of global worker ids owned by `rank` when a job of n_workers_total simulated
    workers is spread over `size` GPUs (sizes differ by at most one)."""
    base, rem = divmod(n_workers_total, size)
    lo = rank * base + min(rank, rem)
    return list(range(lo, lo + base + (1 if rank < rem else 0)))
