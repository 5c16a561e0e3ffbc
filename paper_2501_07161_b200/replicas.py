"""Multi-GPU: the sweep of one model never exchanges data between GPUs, so several GPUs run
independent replicas (one process per GPU, a different model instance each).  The only
cross-rank traffic is the bookkeeping below: a barrier, the slowest rank's time and the total
amount of work.  The tensors live on the CPU for a gloo group and on the GPU for NCCL."""
from __future__ import annotations

import torch
import torch.distributed as dist


def _dev():
    if dist.is_initialized() and dist.get_backend() == "nccl":
        return torch.device("cuda", torch.cuda.current_device())
    return torch.device("cpu")


def world() -> int:
    return dist.get_world_size() if dist.is_initialized() else 1


def rank() -> int:
    return dist.get_rank() if dist.is_initialized() else 0


def barrier():
    if dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float) -> float:
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=_dev())
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float) -> float:
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=_dev())
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def replica_seed(base_seed: int, rank_: int) -> int:
    """Every replica sweeps its own model instance."""
    return base_seed + 1000003 * rank_


def whole_job_throughput(units_local: float, elapsed_local_s: float) -> tuple:
    """(units per second over all ranks, slowest rank's seconds): total work of all replicas
    divided by the maximum time over ranks."""
    total = sum_over_ranks(units_local)
    slowest = max_over_ranks(elapsed_local_s)
    return (total / slowest if slowest > 0 else 0.0), slowest
