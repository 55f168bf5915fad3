"""Pins for oracle/int4.py: the storage layout and Eq. 3 / Eq. 4."""
import numpy as np

from oracle import int4


def test_pack_word_by_hand():
    # q = -8..-1 down a column -> nibbles 0..7 -> word 0x76543210
    q = np.arange(-8, 0).reshape(8, 1)
    assert int(int4.pack_int4(q)[0, 0]) == 0x76543210
    q = np.arange(0, 8).reshape(8, 1)
    assert int(int4.pack_int4(q)[0, 0]) == 0xFEDCBA98


def test_pack_unpack_roundtrip_all_values_all_positions():
    for pos in range(8):
        for val in range(-8, 8):
            q = np.zeros((8, 3), dtype=np.int8)
            q[pos, 1] = val
            w = int4.pack_int4(q)
            assert int(w[0, 1]) == (0x88888888 & ~(0xF << 4 * pos)) | ((val + 8) << 4 * pos)
            assert int(w[0, 0]) == 0x88888888
            assert np.array_equal(int4.unpack_int4(w), q)
    rng = np.random.default_rng(0)
    q = rng.integers(-8, 8, size=(256, 40)).astype(np.int8)
    assert np.array_equal(int4.unpack_int4(int4.pack_int4(q)), q)


def test_bf16_round_matches_torch():
    import torch
    rng = np.random.default_rng(3)
    x = np.concatenate([rng.standard_normal(100_000).astype(np.float32) * 0.02,
                        np.array([0.0, 1.0, 1.00390625, 1.01171875, 3.0e38, -1e-40], np.float32)])
    ref = torch.from_numpy(x).bfloat16().float().numpy()
    assert np.array_equal(int4.bf16_round(x), ref)


def test_quantiser_eq3_eq4_bounds():
    rng = np.random.default_rng(1)
    w = (rng.standard_normal((688, 96)) * 0.02).astype(np.float32)
    w[128:256, 5] = 0.0                                # an all-zero group
    q, s = int4.quantize_int4(w)
    G = int4.num_groups(688)
    assert s.shape == (G, 96) and G == 6
    assert np.array_equal(int4.bf16_round(s), s)
    assert s[1, 5] == 0 and np.all(q[128:256, 5] == 0)
    deq = int4.dequantize(q, s)
    gidx = np.arange(688) // 128
    # |w - s q| <= s/2 wherever the clamp is not hit; the clamp is hit only when
    # bf16(absmax/7) rounded down, by at most 2**-9 relative of 7 steps.
    err = np.abs(w.astype(np.float64) - deq)
    bound = s[gidx].astype(np.float64) * (0.5 + 7 * 2.0 ** -8)
    assert np.all(err <= bound + 1e-12)
    # symmetric range: max |q| is 7 in every non-zero group, never 8 on the positive side
    for g in range(G):
        blk = np.abs(q[g * 128:(g + 1) * 128]).max(axis=0)
        nz = s[g] != 0
        assert np.all(blk[nz] == 7)
    assert q.min() >= -8 and q.max() <= 7
    # scale is absmax/7 up to bf16 rounding
    am = np.abs(w[:128]).max(axis=0)
    np.testing.assert_allclose(s[0], am / 7, rtol=2.0 ** -8)


def test_quantiser_rounds_half_to_even():
    # scale exactly 1 (absmax 7): w = 0.5, 1.5, 2.5 -> 0, 2, 2
    w = np.zeros((128, 1), dtype=np.float32)
    w[0, 0] = 7.0
    w[1:4, 0] = [0.5, 1.5, 2.5]
    w[4:7, 0] = [-0.5, -1.5, -2.5]
    q, s = int4.quantize_int4(w)
    assert s[0, 0] == 1.0
    assert list(q[:7, 0]) == [7, 0, 2, 2, 0, -2, -2]
