"""Perturbed de-quantised linear layer (oracle, fp64).

Eq. 5 perturbs only the scales: Delta' = Delta + sign * eps * z, the integer
weights stay fixed; Eq. 4 then gives the weight Delta' * w_bar that the normal
forward uses.  No clamp is applied to Delta' (Algorithm 1, PERTURB_SCALES).

The same estimator applies to block-scaled codebook formats (the paper's NF4
experiment, appendix "Results with Stable Diffusion": the continuous scales of a
4-bit codebook quantiser are what QZO perturbs and updates): there the fixed part
of a weight is a table entry instead of an integer, see perturbed_linear_table16.
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


def perturbed_linear_samples(x_rows, q_cols, s_cols, cols, N, seed, index_base, sign, eps, bias_cols=None):
    """The same Y (Eq. 4 inside Eq. 5) for a few columns `cols` of a layer with N output features.

    x_rows [R][K], q_cols [K][C] and s_cols [G][C] hold the sampled rows / columns only; the
    logical index of scale (g, cols[c]) is still index_base + g*N + cols[c].  Returns [R][C].
    """
    x = np.asarray(x_rows, dtype=np.float64)
    q = np.asarray(q_cols)
    sp = np.asarray(s_cols, dtype=np.float64).copy()
    cols = np.asarray(cols, dtype=np.uint64)
    K, G = q.shape[0], sp.shape[0]
    if sign != 0:
        idx = np.uint64(index_base) + np.arange(G, dtype=np.uint64)[:, None] * np.uint64(N) + cols[None, :]
        z = philox.normal_from_index(seed, idx).astype(np.float64)
        sp = sp + float(sign) * float(eps) * z
    w = sp[np.arange(K) // GROUP] * q.astype(np.float64)
    y = x @ w
    if bias_cols is not None:
        y = y + np.asarray(bias_cols, dtype=np.float64)[None, :]
    return y


TABLE_BLOCK = 64


def perturbed_linear_table16(x, codes, s, table, seed, index_base, sign, eps, bias=None, channelwise=False):
    """Block-scaled 16-entry codebook weights (NF4-style storage): w[k][n] = s'[k // 64][n] * table[codes[k][n]],
    codes in [0, 15], one scale per block of 64 consecutive input rows of an output column, and
    s' = s + sign*eps*z with z at index index_base + b*N + n for scale [b][n] (Eq. 5 on the format's
    continuous scales; the codes and the table stay fixed).  Y = X W (+ bias), fp64.

    channelwise: s is [1][N], one scale per output channel (the codebook setting of Sec. 4.1, where the
    channel-wise scales are what QZO tunes): w[k][n] = s'[n] * table[codes[k][n]], z at index_base + n."""
    x = np.asarray(x, dtype=np.float64)
    codes = np.asarray(codes)
    table = np.asarray(table, dtype=np.float64)
    assert table.shape == (16,) and codes.min() >= 0 and codes.max() <= 15
    K = codes.shape[0]
    sp = perturbed_scales(s, seed, index_base, sign, eps)
    if channelwise:
        assert sp.shape[0] == 1
        w = sp[np.zeros(K, dtype=np.int64)] * table[codes]
    else:
        assert sp.shape[0] == (K + TABLE_BLOCK - 1) // TABLE_BLOCK
        w = sp[np.arange(K) // TABLE_BLOCK] * table[codes]
    y = x @ w
    if bias is not None:
        y = y + np.asarray(bias, dtype=np.float64)[None, :]
    return y
