"""Pins for oracle/philox.py: published known answers, counter-mode properties,
closed-form ranges and the statistics of the normals."""
import os

import numpy as np
from scipy import stats

from oracle import philox

GOLD = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def _kat_rows():
    rows = []
    with open(GOLD) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            rows.append([int(t, 16) for t in line.split()])
    return rows


def test_known_answer_vectors():
    rows = _kat_rows()
    assert len(rows) == 3
    for c0, c1, c2, c3, k0, k1, r0, r1, r2, r3 in rows:
        out = philox.philox4x32_10([c0], [c1], [c2], [c3], k0, k1)
        assert [int(o[0]) for o in out] == [r0, r1, r2, r3]


def test_words_keyed_on_seed_and_block():
    # seed 0, indices 0..3 share counter block 0 -> first KAT row.
    w = philox.philox_words(0, np.arange(4))
    assert [int(x[0]) for x in w] == [0x6627e8d5, 0xe169c58d, 0xbc57ac4c, 0x9b00dbd8]
    for lane in range(4):
        assert [int(x[lane]) for x in w] == [int(x[0]) for x in w]
    # all-ones key and a counter block whose low two words are all ones would need c2,c3 = ones;
    # instead check the 64-bit block split: index 4*(2**32) has counter (0, 1, 0, 0).
    hi = philox.philox_words(5, np.array([4 * 2 ** 32], dtype=np.uint64))
    ref = philox.philox4x32_10([0], [1], [0], [0], 5, 0)
    assert [int(a[0]) for a in hi] == [int(b[0]) for b in ref]
    k = philox.philox_words((7 << 32) | 9, np.array([0], dtype=np.uint64))
    ref = philox.philox4x32_10([0], [0], [0], [0], 9, 7)
    assert [int(a[0]) for a in k] == [int(b[0]) for b in ref]


def test_counter_mode_order_independence_and_regeneration():
    idx = np.arange(10_000, dtype=np.uint64)
    z = philox.normal_from_index(1234, idx)
    perm = np.random.default_rng(0).permutation(idx.size)
    z_perm = philox.normal_from_index(1234, idx[perm])
    assert np.array_equal(z[perm].view(np.uint32), z_perm.view(np.uint32))
    assert np.array_equal(philox.normal_range(1234, 0, 10_000).view(np.uint32), z.view(np.uint32))
    # one at a time == batch
    for i in (0, 1, 2, 3, 4, 4097, 9999):
        assert philox.normal_from_index(1234, np.array([i]))[0] == z[i]
    assert not np.array_equal(philox.normal_range(1235, 0, 10_000), z)


def test_uniform_range_and_exactness():
    assert philox.uniform_from_word(0) == 2.0 ** -24
    assert philox.uniform_from_word(0xFFFFFFFF) == 1.0 - 2.0 ** -24
    x = np.random.default_rng(1).integers(0, 2 ** 32, size=100_000, dtype=np.uint64)
    u = philox.uniform_from_word(x)
    assert np.array_equal(u.astype(np.float32).astype(np.float64), u)   # exact in fp32
    assert u.min() >= 2.0 ** -24 and u.max() <= 1.0 - 2.0 ** -24
    # the nine low bits of the word do not matter
    assert philox.uniform_from_word(0x1FF) == philox.uniform_from_word(0)


def test_box_muller_identity_pairs_lanes():
    # z(4j)^2 + z(4j+1)^2 = -2 ln U(r0), z(4j+2)^2 + z(4j+3)^2 = -2 ln U(r2)
    n = 4096
    z = philox.normal_range(99, 0, 4 * n).astype(np.float64).reshape(n, 4)
    r0, r1, r2, r3 = philox.philox_words(99, np.arange(0, 4 * n, 4, dtype=np.uint64))
    np.testing.assert_allclose(z[:, 0] ** 2 + z[:, 1] ** 2,
                               -2 * np.log(philox.uniform_from_word(r0)), rtol=1e-5)
    np.testing.assert_allclose(z[:, 2] ** 2 + z[:, 3] ** 2,
                               -2 * np.log(philox.uniform_from_word(r2)), rtol=1e-5)
    # angle of the pair is 2 pi U(r1): atan2(lane1, lane0)
    ang = np.mod(np.arctan2(z[:, 1], z[:, 0]), 2 * np.pi)
    np.testing.assert_allclose(ang, 2 * np.pi * philox.uniform_from_word(r1), atol=1e-5)
    ang = np.mod(np.arctan2(z[:, 3], z[:, 2]), 2 * np.pi)
    np.testing.assert_allclose(ang, 2 * np.pi * philox.uniform_from_word(r3), atol=1e-5)


def test_normal_statistics():
    n = 4_000_000
    z = philox.normal_range(2024, 0, n).astype(np.float64)
    assert np.abs(z).max() <= np.sqrt(48 * np.log(2)) + 1e-6
    assert abs(z.mean()) < 2e-3
    assert abs(z.var() - 1.0) < 4e-3
    assert abs(stats.skew(z)) < 5e-3
    assert abs(stats.kurtosis(z)) < 1e-2
    ks = stats.kstest(z[:400_000], "norm")
    assert ks.pvalue > 1e-3
    zz = z.reshape(-1, 4)
    c = np.corrcoef(zz.T)
    assert np.abs(c - np.eye(4)).max() < 3e-3
    # neighbouring counter blocks are uncorrelated too
    assert abs(np.corrcoef(zz[:-1, 0], zz[1:, 0])[0, 1]) < 3e-3
