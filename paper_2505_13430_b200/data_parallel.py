"""Data-parallel QZO step: every rank holds the same int4 weights and scales and its own part of
the batch.  Because z is a pure function of (seed, scale index), the only exchange per step is
one all-reduce of four floats (sum of token losses and number of kept tokens, for each
perturbation sign); every rank then applies the identical seeded update, so the scales stay
bit-identical without any parameter traffic (the seed trick of Sec. 3.1 taken across ranks;
Algorithm 1 otherwise unchanged).

Nothing of the method is computed here: the forwards, d, d' (Eq. 6) and the update run in the
library (qzo_step_begin / qzo_step_finish); this module only places the collective between them.
"""
import torch.distributed as dist


def all_reduce_sums(sums):
    """Element-wise sum of the four loss sums over all ranks, in place (a no-op without a group)."""
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(sums, op=dist.ReduceOp.SUM)
    return sums


def dp_step(model, tokens, labels, seed, eps, lr, clip, read_back=True):
    """One QZO step on this rank's part of the batch; returns (l+, l-, d, d') of the whole batch
    (None without read_back).  `model` offers qzo_step_begin / qzo_step_finish (a qzo.Model);
    tokens / labels are this rank's int32 [B][S] device tensors.  seed, eps, lr and clip must be the
    same on every rank."""
    sums = model.qzo_step_begin(tokens, labels, seed, eps)
    all_reduce_sums(sums)
    return model.qzo_step_finish(sums, seed, eps, lr, clip, read_back=read_back)


def all_gather_sums(sums):
    """The four loss sums of every rank, in rank order: a [world][4] tensor (just [1][4] without a group)."""
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        parts = [sums.new_empty(sums.shape) for _ in range(dist.get_world_size())]
        dist.all_gather(parts, sums)
        return parts
    return [sums]


def dp_step_seed_per_rank(model, tokens, labels, seed_base, eps, lr_per_seed, clip, read_back=True):
    """One step with one perturbation direction PER RANK (n-SPSA: the average of n independent
    zeroth-order estimates; a variant the paper does not run, listed as optional): rank r perturbs with
    seed_base + r on its own part of the batch; the ranks exchange their four loss sums (an all-gather of
    4 n floats), and every rank then applies the n seeded updates in rank order, each with step size
    lr_per_seed (the caller divides its learning rate by the number of ranks).  Every update is the
    library's: d and d' (Eq. 6) from that rank's sums, then the seeded update with that rank's seed, so all
    ranks end with bit-identical scales.  Returns the list of (l+, l-, d, d') per rank (None without
    read_back)."""
    rank = dist.get_rank() if dist.is_available() and dist.is_initialized() else 0
    sums = model.qzo_step_begin(tokens, labels, seed_base + rank, eps)
    outs = []
    for r, part in enumerate(all_gather_sums(sums)):
        outs.append(model.qzo_step_finish(part, seed_base + r, eps, lr_per_seed, clip, read_back=read_back))
    return outs if read_back else None
