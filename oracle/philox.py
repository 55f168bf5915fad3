"""Philox4x32-10 counter RNG and the z(seed, index) map (oracle, fp64).

The paper only says that a random seed is stored and the Gaussian direction z
is regenerated from it when needed (Sec. 3.1, MeZO seed trick; Algorithm 1
re-seeds its generator before every sweep over the scales).  The generator used here is the
published Philox4x32-10 (Salmon et al., SC'11) keyed on the 64-bit seed, with
the logical scale index as the counter, so that z_i is a pure function of
(seed, i) and can be regenerated in any order.

Mapping (a reading of the paper, which leaves the generator open):
  key      = (seed & 0xffffffff, seed >> 32)
  counter  = (lo32(i >> 2), hi32(i >> 2), 0, 0),  lane = i & 3
  uniform  U(x) = ((x >> 9) + 0.5) * 2**-23            (exact in fp32)
  normals  rho0 = sqrt(-2 ln U(r0)), rho1 = sqrt(-2 ln U(r2))
           lane 0: rho0 cos(2 pi U(r1))   lane 1: rho0 sin(2 pi U(r1))
           lane 2: rho1 cos(2 pi U(r3))   lane 3: rho1 sin(2 pi U(r3))
  evaluated in fp64 and rounded once to fp32.
"""
import numpy as np

PHILOX_M0 = 0xD2511F53
PHILOX_M1 = 0xCD9E8D57
PHILOX_W0 = 0x9E3779B9
PHILOX_W1 = 0xBB67AE85
_MASK32 = np.uint64(0xFFFFFFFF)


def philox4x32_10(c0, c1, c2, c3, k0, k1):
    """Ten Philox rounds on arrays of 32-bit words (held in uint64)."""
    c0 = np.asarray(c0, dtype=np.uint64) & _MASK32
    c1 = np.asarray(c1, dtype=np.uint64) & _MASK32
    c2 = np.asarray(c2, dtype=np.uint64) & _MASK32
    c3 = np.asarray(c3, dtype=np.uint64) & _MASK32
    k0 = np.uint64(int(k0) & 0xFFFFFFFF)
    k1 = np.uint64(int(k1) & 0xFFFFFFFF)
    for r in range(10):
        p0 = np.uint64(PHILOX_M0) * c0          # 32x32 -> 64, no overflow
        p1 = np.uint64(PHILOX_M1) * c2
        hi0, lo0 = p0 >> np.uint64(32), p0 & _MASK32
        hi1, lo1 = p1 >> np.uint64(32), p1 & _MASK32
        c0, c1, c2, c3 = hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0
        if r != 9:
            k0 = (k0 + np.uint64(PHILOX_W0)) & _MASK32
            k1 = (k1 + np.uint64(PHILOX_W1)) & _MASK32
    return c0, c1, c2, c3


def philox_words(seed, index):
    """The four output words of the counter block that holds scale `index`."""
    idx = np.asarray(index, dtype=np.uint64)
    blk = idx >> np.uint64(2)
    seed = int(seed) & 0xFFFFFFFFFFFFFFFF
    zeros = np.zeros_like(blk)
    return philox4x32_10(blk & _MASK32, blk >> np.uint64(32), zeros, zeros,
                         seed & 0xFFFFFFFF, seed >> 32)


def uniform_from_word(x):
    """U(x) in (0, 1): 23 random bits plus a half, exactly representable in fp32."""
    x = np.asarray(x, dtype=np.uint64)
    return ((x >> np.uint64(9)).astype(np.float64) + 0.5) * 2.0 ** -23


def normal_from_index(seed, index):
    """z_i ~ N(0,1) for logical scale index i, fp64 math rounded to fp32."""
    idx = np.asarray(index, dtype=np.uint64)
    r0, r1, r2, r3 = philox_words(seed, idx)
    lane = idx & np.uint64(3)
    radial = np.where(lane < 2, uniform_from_word(r0), uniform_from_word(r2))
    angle = np.where(lane < 2, uniform_from_word(r1), uniform_from_word(r3))
    rho = np.sqrt(-2.0 * np.log(radial))
    phi = 2.0 * np.pi * angle
    z = np.where((lane & np.uint64(1)) == 0, rho * np.cos(phi), rho * np.sin(phi))
    return z.astype(np.float32)


def normal_range(seed, base, count):
    """z for indices base .. base+count-1."""
    return normal_from_index(seed, np.uint64(base) + np.arange(count, dtype=np.uint64))
