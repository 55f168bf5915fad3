"""Host-side logic of the multi-GPU benchmark: the path shards by data only, so N GPUs run N
independent replicas (own model copy, own batch, no collective on the data path).  The only
exchange is the timing itself: the slowest rank's device time decides the whole-job rate."""
import torch
import torch.distributed as dist


def rank_seeds(base_model_seed, base_token_seed, rank):
    """Every replica draws its own weights and its own batch."""
    return base_model_seed + rank, base_token_seed + rank


def max_over_ranks(value, device="cpu"):
    """Largest `value` (a float, e.g. elapsed ms) over all ranks; the value itself without a group."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(steps_per_rank, world, elapsed_ms):
    """Steps per second of the whole job: every rank did `steps_per_rank` steps within `elapsed_ms`
    (the maximum over ranks)."""
    return world * steps_per_rank / (elapsed_ms / 1000.0)
