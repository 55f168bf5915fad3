"""Pins for oracle/linear.py: brute force, the unperturbed special case, linearity in eps."""
import numpy as np

from oracle import int4, linear, philox


def _case(M=5, K=272, N=12, seed=0):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((M, K))
    q = rng.integers(-8, 8, size=(K, N)).astype(np.int8)
    s = int4.bf16_round(rng.uniform(0.005, 0.02, size=(int4.num_groups(K), N)).astype(np.float32))
    return x, q, s


def test_brute_force_tiny():
    x, q, s = _case(M=3, K=136, N=4)
    seed, base, eps = 77, 40, 1e-3
    y = linear.perturbed_linear(x, q, s, seed, base, -1, eps)
    G, N = s.shape
    for t in range(3):
        for n in range(N):
            acc = 0.0
            for k in range(136):
                g = k // 128
                z = float(philox.normal_from_index(seed, np.array([base + g * N + n]))[0])
                acc += x[t, k] * (float(s[g, n]) - eps * z) * int(q[k, n])
            assert abs(acc - y[t, n]) <= 1e-12 * max(1.0, abs(acc))


def test_sign_zero_is_textbook_dequant_gemm():
    x, q, s = _case()
    y0 = linear.perturbed_linear(x, q, s, 1, 0, 0, 1e-3)
    np.testing.assert_allclose(y0, x @ int4.dequantize(q, s), rtol=1e-13, atol=1e-13)
    b = np.linspace(-1, 1, q.shape[1])
    yb = linear.perturbed_linear(x, q, s, 1, 0, 0, 1e-3, bias=b)
    np.testing.assert_allclose(yb - y0, np.broadcast_to(b, y0.shape), atol=1e-12)


def test_linearity_in_the_perturbation():
    x, q, s = _case(seed=2)
    seed, base, eps = 5, 8, 1e-3
    yp = linear.perturbed_linear(x, q, s, seed, base, +1, eps)
    ym = linear.perturbed_linear(x, q, s, seed, base, -1, eps)
    y0 = linear.perturbed_linear(x, q, s, seed, base, 0, eps)
    np.testing.assert_allclose(yp + ym, 2 * y0, rtol=1e-12, atol=1e-12)
    z = philox.normal_range(seed, base, s.size).astype(np.float64).reshape(s.shape)
    zq = z[np.arange(q.shape[0]) // 128] * q
    np.testing.assert_allclose(yp - ym, 2 * eps * (x @ zq), rtol=1e-9, atol=1e-12)
    # a different index base draws different noise
    yp2 = linear.perturbed_linear(x, q, s, seed, base + 8, +1, eps)
    assert np.abs(yp2 - yp).max() > 0


def test_no_clamp_on_perturbed_scales():
    s = np.full((1, 8), 1e-6, dtype=np.float32)
    sp = linear.perturbed_scales(s, 3, 0, +1, 1e-3)
    assert (sp < 0).any()          # Algorithm 1's PERTURB_SCALES has no max(., 0)


def test_sampled_columns_equal_the_full_layer():
    # perturbed_linear_samples must give the very entries of the full result, with the scale index of
    # column n still index_base + g*N + n (a shifted or compacted index would draw other z)
    x, q, s = _case(M=6, K=400, N=24, seed=3)
    seed, base, eps = 5, 16, 2e-3
    rows, cols = [0, 3, 5], [0, 7, 23, 11]
    for sign in (+1, -1, 0):
        full = linear.perturbed_linear(x, q, s, seed, base, sign, eps)
        part = linear.perturbed_linear_samples(x[rows], q[:, cols], s[:, cols], cols, 24, seed, base, sign, eps)
        np.testing.assert_allclose(part, full[np.ix_(rows, cols)], rtol=1e-13, atol=1e-13)
    # and by brute force for one entry
    t, n = 3, 23
    acc = 0.0
    for k in range(400):
        g = k // 128
        z = float(philox.normal_from_index(seed, np.array([base + g * 24 + n]))[0])
        acc += x[t, k] * (float(s[g, n]) + eps * z) * int(q[k, n])
    got = linear.perturbed_linear_samples(x[[t]], q[:, [n]], s[:, [n]], [n], 24, seed, base, +1, eps)[0, 0]
    assert abs(acc - got) <= 1e-12 * max(1.0, abs(acc))


def test_table16_linear_brute_force_and_special_cases():
    # block-scaled 16-entry codebook weights: triple loop on a small case, sign 0 = plain de-quantised GEMM,
    # the two linearity identities of the perturbation, and the reduction to the int4 routine
    from paper_2505_13430_b200 import inputs
    x, codes, s, table = inputs.table16_case(3, 136, 16, seed=2)
    x, codes, s, table = x.float().numpy(), codes.numpy(), s.float().numpy(), table.numpy()
    seed, base, eps = 5, 32, 2e-3
    z = philox.normal_range(seed, base, s.size).astype(np.float64).reshape(s.shape)
    for sign in (+1, -1, 0):
        got = linear.perturbed_linear_table16(x, codes, s, table, seed, base, sign, eps)
        want = np.zeros((3, 16))
        for t in range(3):
            for n in range(16):
                for k in range(136):
                    want[t, n] += float(x[t, k]) * (float(s[k // 64, n]) + sign * eps * z[k // 64, n]) * float(table[codes[k, n]])
        assert np.abs(got - want).max() <= 1e-12 * np.abs(want).max()
    y0 = linear.perturbed_linear_table16(x, codes, s, table, seed, base, 0, eps)
    yp = linear.perturbed_linear_table16(x, codes, s, table, seed, base, +1, eps)
    ym = linear.perturbed_linear_table16(x, codes, s, table, seed, base, -1, eps)
    assert np.abs(yp + ym - 2 * y0).max() <= 1e-12 * np.abs(y0).max()
    zt = z[np.arange(136) // 64] * table.astype(np.float64)[codes]
    assert np.abs((yp - ym) - 2 * eps * (x.astype(np.float64) @ zt)).max() <= 1e-12 * np.abs(yp - ym).max()
    # with the affine table c - 8 and equal scales in the two blocks of every group it IS the int4 linear
    K, N = 256, 8
    rng = np.random.default_rng(3)
    xx = rng.standard_normal((4, K))
    q = rng.integers(-8, 8, size=(K, N)).astype(np.int8)
    s128 = int4.bf16_round(rng.uniform(0.005, 0.02, size=(2, N)).astype(np.float32))
    a = linear.perturbed_linear(xx, q, s128, 1, 0, 0, 1e-3)
    b = linear.perturbed_linear_table16(xx, q + 8, np.repeat(s128, 2, axis=0), np.arange(16) - 8.0, 1, 0, 0, 1e-3)
    assert np.abs(a - b).max() <= 1e-13 * np.abs(a).max()


def test_channelwise_codebook_linear_factors_out_of_the_contraction():
    # One scale per output channel (the codebook setting of Sec. 4.1): the perturbed scale multiplies the whole
    # column, so Y = (X table[codes]) * s' column by column -- a closed form the routine must reproduce --,
    # z is indexed by the channel alone, and at sign 0 it is the block-scaled routine with equal scales in
    # every block.
    from paper_2505_13430_b200 import inputs
    x, codes, s, table = inputs.table16_case(3, 200, 16, seed=4)
    x, codes, table = x.float().numpy().astype(np.float64), codes.numpy(), table.numpy().astype(np.float64)
    s1 = s.float().numpy()[:1]                                   # [1][N]
    seed, base, eps = 9, 24, 3e-3
    z = philox.normal_range(seed, base, 16).astype(np.float64)
    plain = x @ table[codes]                                     # the contraction without any scale
    for sign in (+1, -1, 0):
        got = linear.perturbed_linear_table16(x, codes, s1, table, seed, base, sign, eps, channelwise=True)
        want = plain * (s1[0].astype(np.float64) + sign * eps * z)[None, :]
        assert np.abs(got - want).max() <= 1e-12 * np.abs(want).max()
        brute = sum(float(x[1, k]) * (float(s1[0, 5]) + sign * eps * z[5]) * float(table[codes[k, 5]]) for k in range(200))
        assert abs(got[1, 5] - brute) <= 1e-12 * abs(brute)
    blocks = np.repeat(s1, 4, axis=0)                            # ceil(200 / 64) = 4 equal rows
    a = linear.perturbed_linear_table16(x, codes, s1, table, seed, base, 0, eps, channelwise=True)
    b = linear.perturbed_linear_table16(x, codes, blocks, table, seed, base, 0, eps)
    assert np.abs(a - b).max() <= 1e-13 * np.abs(a).max()
    # a different channel's z must not leak in: shifting the base by one channel shifts which z a column gets
    c = linear.perturbed_linear_table16(x, codes, s1, table, seed, base + 4, +1, eps, channelwise=True)
    z4 = philox.normal_range(seed, base + 4, 16).astype(np.float64)
    assert np.abs(c - plain * (s1[0] + eps * z4)[None, :]).max() <= 1e-12 * np.abs(c).max()
