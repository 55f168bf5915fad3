"""Perturbed de-quantised linear layer (oracle, fp64).

Eq. 5 perturbs only the scales: Delta' = Delta + sign * eps * z, the integer
weights stay fixed; Eq. 4 then gives the weight Delta' * w_bar that the normal
forward uses.  No clamp is applied to Delta' (Algorithm 1, PERTURB_SCALES).
"""
import numpy as np
from . import philox
from .int4 import GROUP


def perturbed_scales(s, seed, index_base, sign, eps):
    """fp64 s' = s + sign*eps*z, z_i for i = index_base + g*N + n (row-major)."""
    s = np.asarray(s, dtype=np.float64)
    if sign == 0:
        return s.copy()
    z = philox.normal_range(seed, index_base, s.size).astype(np.float64).reshape(s.shape)
    return s + float(sign) * float(eps) * z


def perturbed_linear(x, q, s, seed, index_base, sign, eps, bias=None):
    """Y[t][n] = sum_k X[t][k] * s'[k // 128][n] * q[k][n]  (+ bias[n])."""
    x = np.asarray(x, dtype=np.float64)
    q = np.asarray(q)
    K = q.shape[0]
    sp = perturbed_scales(s, seed, index_base, sign, eps)
    w = sp[np.arange(K) // GROUP] * q.astype(np.float64)
    y = x @ w
    if bias is not None:
        y = y + np.asarray(bias, dtype=np.float64)[None, :]
    return y
