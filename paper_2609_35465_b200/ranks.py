"""Multi-process plumbing of the benchmark: the path does not shard (one GPU,
batch 1 in the paper), so N ranks are N independent replicas of the same pass.
The only collectives are a barrier and the maximum of the per-rank time; the
aggregate rate is (work of all ranks) / (slowest rank's time)."""
import torch
import torch.distributed as dist


def max_over_ranks(value: float, device="cpu") -> float:
    """Maximum of a per-rank scalar over the default process group (identity without one)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_rate(units_per_rank: float, seconds_this_rank: float, device="cpu") -> float:
    """Whole-job rate of a weak-scaling run: every rank processed units_per_rank
    units; the job took as long as its slowest rank."""
    world = dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1
    return world * units_per_rank / max_over_ranks(seconds_this_rank, device)
