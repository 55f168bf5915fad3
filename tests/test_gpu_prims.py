"""GPU parity of the small steps against the oracle: Philox words / uniforms and int4 unpacking
bit-exact, the quantiser's integer decisions bit-exact, normals and the seeded update within fp32 /
one bf16 ulp."""
import numpy as np
import pytest
import torch

from oracle import int4, philox, qzo as oqzo
from paper_2505_13430_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def lib():
    from paper_2505_13430_b200 import qzo
    return qzo


def _bf16_ulp_diff(a, b):
    """distance in bf16 ulps between two bf16 torch tensors (monotone integer mapping)."""
    def key(t):
        i = t.view(torch.int16).to(torch.int32) & 0xFFFF
        return torch.where(i >= 0x8000, 0x8000 - i, i)
    return (key(a) - key(b)).abs()


def test_philox_words_and_uniforms_bit_exact(lib):
    for seed, base, n in ((0, 0, 1), (42, 0, 5000), ((7 << 32) | 9, 2 ** 32 - 10, 64), (2 ** 64 - 1, 123456789, 1000)):
        words, uni = lib.qzo_philox_words(seed, base, n)
        w = words.cpu().numpy().view(np.uint32)
        blocks = np.uint64(base) + np.arange(n, dtype=np.uint64)
        ref = philox.philox_words(seed, blocks * np.uint64(4))
        ref = np.stack([r.astype(np.uint32) for r in ref], axis=1)
        assert np.array_equal(w, ref)
        uref = philox.uniform_from_word(ref.astype(np.uint64)).astype(np.float32)
        assert np.array_equal(uni.cpu().numpy().view(np.uint32), uref.view(np.uint32))
    words, _ = lib.qzo_philox_words(0, 0, 1)
    assert [int(x) for x in words.cpu().numpy().view(np.uint32)[0]] == [0x6627e8d5, 0xe169c58d, 0xbc57ac4c, 0x9b00dbd8]


def test_normals_match_oracle_and_regenerate_bit_identically(lib):
    for seed, base, n in ((42, 0, 100_003), (5, 12_672 - 8, 4099), (99, 2 ** 34 + 4, 1001), (3, 6, 9)):
        z = lib.qzo_normals(seed, base, n).cpu().numpy()
        ref = philox.normal_range(seed, base, n)
        np.testing.assert_allclose(z, ref, rtol=5e-6, atol=5e-6)
        z2 = lib.qzo_normals(seed, base, n).cpu().numpy()
        assert np.array_equal(z.view(np.uint32), z2.view(np.uint32))
        # a sub-range regenerates the same values (counter mode)
        sub = lib.qzo_normals(seed, base + 3, max(n - 5, 1)).cpu().numpy()
        assert np.array_equal(sub.view(np.uint32), z[3:3 + sub.size].view(np.uint32))


def test_unpack_and_repack_bit_exact(lib):
    rng = np.random.default_rng(0)
    for K, N in ((8, 8), (256, 128), (688, 256), (256, 688), (1024, 1000)):
        q = rng.integers(-8, 8, size=(K, N)).astype(np.int8)
        words = int4.pack_int4(q)
        dev = torch.from_numpy(words.view(np.int32)).cuda()
        assert np.array_equal(lib.qzo_unpack_int4(dev, K, N).cpu().numpy(), q)
        wq = lib.qzo_repack_int4(dev, K, N)
        assert wq.numel() == lib.qzo_repacked_bytes(K, N)
        assert np.array_equal(lib.qzo_unpack_kernel_layout(wq, K, N).cpu().numpy(), q)


def test_quantiser_bit_exact(lib):
    for K, N, seed in ((256, 256, 1), (688, 256, 2), (256, 688, 3)):
        w = inputs.normal_fp32((K, N), 0.02, seed)
        w[0:128, 3] = 0.0
        q_ref, s_ref = int4.quantize_int4(w.numpy())
        words, scales = lib.qzo_quantize_int4(w.cuda())
        assert np.array_equal(scales.float().cpu().numpy(), s_ref)
        assert np.array_equal(lib.qzo_unpack_int4(words, K, N).cpu().numpy(), q_ref)
        assert np.array_equal(words.cpu().numpy().view(np.uint32), int4.pack_int4(q_ref))


def test_seeded_update_within_one_bf16_ulp(lib):
    g = torch.Generator().manual_seed(0)
    for count, base, lr, gval, clip in ((12_672, 0, 1e-5, 37.5, 100.0), (1001, 8, 1e-5, -250.0, 100.0),
                                        (4096, 2 ** 33, 1e-2, 100.0, 100.0), (515, 4, 1e-5, 3.0, 0.0)):
        s = (torch.rand((count,), generator=g) * 0.015 + 0.005).bfloat16()
        dc = oqzo.ddc_clip(gval, clip)
        ref = oqzo.update_scales_flat(s.float().numpy(), 77, base, lr, dc)
        dev = s.clone().cuda()
        lib.qzo_update_scales_flat(dev, 77, base, lr, gval, clip)
        got = dev.cpu()
        ulps = _bf16_ulp_diff(got, torch.from_numpy(ref).bfloat16())
        assert int(ulps.max()) <= 1
        assert float((ulps > 0).float().mean()) < 0.01          # ulp flips are rare rounding ties
        assert (got.float() >= 0).all()
        if clip == 0.0:
            assert torch.equal(got.view(torch.int16), s.view(torch.int16))     # d' = 0: bit-unchanged
    # g = 0: bit-unchanged; non-finite g: rejected, no write
    dev = s.clone().cuda()
    lib.qzo_update_scales_flat(dev, 1, 0, 1e-5, 0.0, 100.0)
    assert torch.equal(dev.cpu().view(torch.int16), s.view(torch.int16))
    with pytest.raises(lib.QzoError) as e:
        lib.qzo_update_scales_flat(dev, 1, 0, 1e-5, float("nan"), 100.0)
    assert e.value.status == lib.ERR_NONFINITE
    assert torch.equal(dev.cpu().view(torch.int16), s.view(torch.int16))
