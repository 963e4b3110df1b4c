"""Multi-GPU driver logic: the DMA hot path has no exchange step, so N GPUs run N independent replicas
(one process per GPU). The only cross-rank operations are a barrier and the max-over-ranks of the step time."""
import torch
import torch.distributed as dist


def max_over_ranks(value: float, device="cpu") -> float:
    """Largest `value` over all ranks of the default process group (identity without one)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: float, step_ms_max: float) -> float:
    """Aggregate rate of N replicas that each process `units_per_rank` per step: N * units / slowest step."""
    n = dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1
    return n * units_per_rank / (step_ms_max * 1e-3)
