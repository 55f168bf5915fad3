"""Data-parallel QZO step: every rank holds the same int4 weights and scales and its own part of
the batch.  Because z is a pure function of (seed, scale index), the only exchange per step is
an all-reduce of two scalars per perturbation sign (sum of token losses, number of kept tokens);
every rank then applies the identical seeded update, so the scales stay bit-identical without any
parameter traffic (the seed trick of Sec. 3.1 taken across ranks; Algorithm 1 otherwise unchanged).
"""
import numpy as np
import torch
import torch.distributed as dist


def kept_tokens(labels):
    """Number of positions that count in the loss (label != -100 and not negative)."""
    return int((labels >= 0).sum().item())


def global_mean_loss(local_mean, local_count, device="cpu"):
    """Mean loss over the tokens of all ranks from each rank's mean and token count."""
    t = torch.tensor([float(local_mean) * float(local_count), float(local_count)], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t[0].item() / max(t[1].item(), 1.0))


def directional_derivative(loss_plus, loss_minus, eps, clip):
    """d = (l+ - l-) / (2 eps) and d' = clip(d, -C, C) (Eq. 6), in fp32 like the device kernel."""
    d = (np.float32(loss_plus) - np.float32(loss_minus)) / (np.float32(2.0) * np.float32(eps))
    dc = np.float32(min(max(d, np.float32(-clip)), np.float32(clip)))
    return float(d), float(dc)


def dp_step(model, tokens, labels, seed, eps, lr, clip, device="cuda"):
    """One QZO step on this rank's part of the batch; returns (l+, l-, d, d') of the whole batch.
    `model` is a qzo.Model; tokens / labels are this rank's int32 [B][S] CUDA tensors."""
    n = kept_tokens(labels)
    lp = float(model.qzo_forward_loss(tokens, labels, seed, +1, eps).cpu()[0])
    lm = float(model.qzo_forward_loss(tokens, labels, seed, -1, eps).cpu()[0])
    lp, lm = global_mean_loss(lp, n, device), global_mean_loss(lm, n, device)
    d, dc = directional_derivative(lp, lm, eps, clip)
    if np.isfinite(lp) and np.isfinite(lm):
        model.qzo_update_scales(seed, lr, d, clip)         # clips d itself; same seed on every rank
    return lp, lm, d, dc
