"""One QZO step (oracle): Algorithm 1, Eq. 5 (Q-SPSA) and Eq. 6 (DDC).

`step_functional` evaluates both losses from the untouched scales,
Delta' = Delta + sign*eps*z (Eq. 5), then d, d' (Eq. 6) and the seeded update
with max(., 0) (Algorithm 1's last loop); this is also what the library does.
Algorithm 1 itself moves the scales in place (by +eps z, then -2 eps z, then
+eps z to restore them); `perturb_scales_in_place` is that single operation,
kept so that the tests can pin the equivalence of the two readings: a forward
on scales moved in place equals the forward with the matching sign, and the
three moves return the scales to where they started.

Storage rounding of the updated scale (bf16, ties to even) is a reading: the
paper does not fix the dtype of Delta.  `lr * d'` is formed once in fp32 and
the update s - (lr d') z is evaluated in fp32 before rounding, the precision
the library uses, so that the rounding decision is taken alike on both sides.
"""
import numpy as np
from . import philox
from .int4 import bf16_round
from .model import (forward_loss, scale_index_bases, dense_index_bases, dense_tensor_names, dense_tensor,
                    LINEAR_ORDER)


def ddc_clip(d, C):
    """Eq. 6: d' = C if d > C; d if -C <= d <= C; -C if d < -C  (C >= 0)."""
    assert C >= 0
    if d > C:
        return float(C)
    if d < -C:
        return float(-C)
    return float(d)


def directional_derivative(loss_plus, loss_minus, eps):
    """d = (l+ - l-) / (2 eps), Algorithm 1."""
    return (loss_plus - loss_minus) / (2.0 * eps)


def update_scales_flat(s, seed, index_base, lr, d_clipped):
    """s_i <- bf16(max(s_i - (lr d') z_i, 0)), fp32 arithmetic (Algorithm 1, last loop)."""
    s = np.asarray(s, dtype=np.float32)
    z = philox.normal_range(seed, index_base, s.size).reshape(s.shape)
    coef = np.float32(np.float32(lr) * np.float32(d_clipped))
    prod = (coef * z).astype(np.float32)
    new = np.maximum((s - prod).astype(np.float32), np.float32(0.0))
    return bf16_round(new)


def update_model_scales(model, seed, lr, d_clipped):
    """Apply the seeded update to every int4 linear of the model, in place."""
    cfg = model["cfg"]
    bases, _ = scale_index_bases(cfg)
    for li, layer in enumerate(model["layers"]):
        for name in LINEAR_ORDER[cfg["arch"]]:
            p = layer["lin"][name]
            p["s"] = update_scales_flat(p["s"], seed, bases[li][name], lr, d_clipped)


def spsa_perturbed(theta, seed, index_base, sign, eps):
    """Def. 3.1: theta + sign*eps*z for an un-quantised tensor, z_i = z(seed, index_base + i) in the
    tensor's row-major order, fp64."""
    t = np.asarray(theta, dtype=np.float64)
    if sign == 0:
        return t.copy()
    z = philox.normal_range(seed, index_base, t.size).astype(np.float64).reshape(t.shape)
    return t + float(sign) * float(eps) * z


def update_dense_flat(theta, seed, index_base, lr, d_clipped, storage):
    """ZO-SGD on an un-quantised tensor (Def. 3.2, Eq. 2 with the SPSA estimate d' z of Def. 3.1):
    theta_i <- theta_i - (lr d') z_i, fp32 arithmetic; no max(., 0) (that belongs to the scales).
    storage: 'bf16' (rounded to bf16, ties to even) or 'f32'."""
    t = np.asarray(theta, dtype=np.float32)
    z = philox.normal_range(seed, index_base, t.size).reshape(t.shape)
    coef = np.float32(np.float32(lr) * np.float32(d_clipped))
    new = (t - (coef * z).astype(np.float32)).astype(np.float32)
    return bf16_round(new) if storage == "bf16" else new


def update_model_dense(model, seed, lr_dense, d_clipped):
    """Joint mode: the seeded update of every un-quantised tensor of dense_tensor_names, in place.
    Embedding and lm_head matrices are stored in bf16, norm gains and biases in fp32."""
    cfg = model["cfg"]
    dbases, _ = dense_index_bases(cfg)
    for key, layer in dense_tensor_names(cfg):
        storage = "bf16" if key in ("embed", "lm_head") else "f32"
        new = update_dense_flat(dense_tensor(model, key, layer), seed, dbases[(key, layer)], lr_dense, d_clipped, storage)
        if layer is None:
            model[key] = new
        else:
            model["layers"][layer][key] = new


def step_functional(model, tokens, labels, seed, eps, lr, C, update=True, joint=False, lr_dense=None):
    """One step from the untouched parameters; returns (l+, l-, d, d').
    joint: Q-SPSA on the scales combined with SPSA on the un-quantised tensors (one z stream, one d')."""
    lp = forward_loss(model, tokens, labels, seed, +1, eps, perturb_dense=joint)
    lm = forward_loss(model, tokens, labels, seed, -1, eps, perturb_dense=joint)
    d = directional_derivative(lp, lm, eps)
    dc = ddc_clip(d, C)
    if update:
        update_model_scales(model, seed, lr, dc)
        if joint:
            update_model_dense(model, seed, lr if lr_dense is None else lr_dense, dc)
    return lp, lm, d, dc


def perturb_scales_in_place(model, scale, seed):
    """Delta_i += scale * z_i(seed) for every scale of the model, in fp64, without clamping
    (the in-place perturbation of Algorithm 1; the scales become fp64 arrays)."""
    cfg = model["cfg"]
    bases, _ = scale_index_bases(cfg)
    for li, layer in enumerate(model["layers"]):
        for name in LINEAR_ORDER[cfg["arch"]]:
            p = layer["lin"][name]
            s = np.asarray(p["s"], dtype=np.float64)
            z = philox.normal_range(seed, bases[li][name], s.size).astype(np.float64)
            p["s"] = s + scale * z.reshape(s.shape)
