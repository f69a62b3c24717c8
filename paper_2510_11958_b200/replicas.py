"""Multi-GPU form of the decode benchmark: independent replicas, one process per GPU.

The decode path does not shard: sequences are independent and the passes of one sequence are
strictly sequential, so N GPUs run N copies of the workload with no data-path collective.  The
only communication is the timing protocol below (a barrier on both sides of the timed region
and a max over ranks of the device-measured time).
"""
import torch
import torch.distributed as dist


def init_from_env(backend: str):
    """Join the process group torchrun set up; returns (rank, world_size)."""
    if not dist.is_initialized():
        dist.init_process_group(backend=backend)
    return dist.get_rank(), dist.get_world_size()


def barrier():
    if dist.is_initialized():
        dist.barrier()


def aggregate(elapsed_ms: float, units: float, device="cpu"):
    """Whole-job figures from per-rank ones: (max elapsed ms over ranks, total units).

    `units` is what this rank processed in the timed region (tokens).  Throughput of the job
    is total units / max time, the definition used for every multi-GPU number.
    """
    if not dist.is_initialized():
        return float(elapsed_ms), float(units)
    t = torch.tensor([float(elapsed_ms)], dtype=torch.float64, device=device)
    u = torch.tensor([float(units)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return t.item(), u.item()
