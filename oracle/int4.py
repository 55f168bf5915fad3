"""int4 storage and the symmetric group quantiser (oracle).

Eq. 3: w_bar = round(w / Delta);  Eq. 4: w = Delta * w_bar;  the standard
k-bit choice Delta = absmax(W) / (2**(k-1) - 1) with k = 4, one Delta per
group of 128 consecutive input rows of one output column (the paper's GPTQ
setting: group 128).

Storage layout shared with the library boundary:
  q[k][n] in [-8, 7], stored nibble u = q + 8;
  packed uint32[K/8][N], nibble j (bits 4j..4j+3) of word [kw][n] is u[8 kw + j][n];
  scales bf16[G][N], G = ceil(K / 128), group g covers rows 128 g .. 128 g + 127.
"""
import numpy as np

GROUP = 128


def bf16_round(x):
    """Round fp32 values to the nearest bf16 (ties to even); result kept as fp32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    bits = x.view(np.uint32).astype(np.uint64)
    lsb = (bits >> np.uint64(16)) & np.uint64(1)
    rounded = (bits + np.uint64(0x7FFF) + lsb) & np.uint64(0xFFFF0000)
    out = rounded.astype(np.uint32).view(np.float32).copy()
    nan = np.isnan(x)
    out[nan] = np.nan
    return out.reshape(x.shape)


def pack_int4(q):
    """q int[K][N] in [-8,7], K % 8 == 0  ->  uint32[K/8][N]."""
    q = np.asarray(q)
    K, N = q.shape
    assert K % 8 == 0 and q.min() >= -8 and q.max() <= 7
    u = (q.astype(np.int64) + 8).astype(np.uint32).reshape(K // 8, 8, N)
    word = np.zeros((K // 8, N), dtype=np.uint32)
    for j in range(8):
        word |= u[:, j, :] << np.uint32(4 * j)
    return word


def unpack_int4(packed):
    """uint32[K/8][N] -> int8 q[K][N] in [-8,7]."""
    packed = np.asarray(packed, dtype=np.uint32)
    KW, N = packed.shape
    q = np.empty((KW, 8, N), dtype=np.int8)
    for j in range(8):
        q[:, j, :] = ((packed >> np.uint32(4 * j)) & np.uint32(0xF)).astype(np.int8) - 8
    return q.reshape(KW * 8, N)


def num_groups(K):
    return (K + GROUP - 1) // GROUP


def quantize_int4(w):
    """fp32 w[K][N] -> (q int8[K][N], scales fp32-held-bf16 [G][N]).

    Delta32 = absmax / 7 in fp32, s = bf16(Delta32); q = clamp(rne(w / s), -8, 7),
    the division done in fp32 (the decision precision both sides share);
    a group whose scale rounds to zero gets q = 0.
    """
    w = np.asarray(w, dtype=np.float32)
    K, N = w.shape
    G = num_groups(K)
    q = np.zeros((K, N), dtype=np.int8)
    s = np.zeros((G, N), dtype=np.float32)
    for g in range(G):
        blk = w[g * GROUP:(g + 1) * GROUP]
        absmax = np.max(np.abs(blk), axis=0).astype(np.float32)
        sg = bf16_round(absmax / np.float32(7.0))
        s[g] = sg
        safe = np.where(sg == 0, np.float32(1.0), sg)
        ratio = (blk / safe[None, :]).astype(np.float32)
        qg = np.clip(np.rint(ratio), -8, 7).astype(np.int8)   # rint = ties to even
        qg[:, sg == 0] = 0
        q[g * GROUP:(g + 1) * GROUP] = qg
    return q, s


def dequantize(q, s):
    """Eq. 4 in fp64: w[k][n] = s[k // 128][n] * q[k][n]."""
    q = np.asarray(q)
    K = q.shape[0]
    gidx = np.arange(K) // GROUP
    return np.asarray(s, dtype=np.float64)[gidx] * q.astype(np.float64)
