"""GPU parity of the block-scaled 16-entry-codebook GEMM (NF4-style storage; the format's continuous scales
are what QZO perturbs) against the oracle, element by element, on shapes with several tiles, ragged tails in
M, K and N (K = 688: eleven blocks of 64, an odd number of k-blocks), split-K, both signs; and the seeded
update of such scales."""
import numpy as np
import pytest
import torch

from oracle import int4, linear as olinear, qzo as oqzo
from paper_2505_13430_b200 import inputs

pytestmark = pytest.mark.gpu

CASES = [(16, 256, 128), (40, 688, 688), (300, 1024, 384), (1, 512, 256), (128, 4096, 512), (257, 2048, 1024)]


def _relerr(got, ref):
    got = got.float().cpu().numpy().astype(np.float64)
    return np.abs(got - ref).max() / np.abs(ref).max()


@pytest.mark.parametrize("M,K,N", CASES)
def test_table16_gemm_matches_oracle(M, K, N):
    from paper_2505_13430_b200 import qzo as lib
    x, codes, s, table = inputs.table16_case(M, K, N, seed=M + K + N)
    words = torch.from_numpy(int4.pack_int4(codes.numpy().astype(np.int64) - 8).view(np.int32)).cuda()   # nibble = code
    wq = lib.qzo_repack_int4(words, K, N)
    assert np.array_equal(lib.qzo_unpack_kernel_layout(wq, K, N).cpu().numpy().astype(np.int64) + 8, codes.numpy())
    status = torch.zeros((1,), dtype=torch.int32, device="cuda")
    seed, base, eps = 77 + M, 8 * (N % 3), 2e-3
    outs = {}
    for sign in (+1, -1, 0):
        y = lib.qzo_perturbed_gemm_table16(x.cuda(), wq, s.cuda(), table.tolist(), M, K, N, seed, base, sign, eps, status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        ref = olinear.perturbed_linear_table16(x.float().numpy(), codes.numpy(), s.float().numpy(), table.numpy(),
                                               seed, base, sign, eps)
        assert _relerr(y, ref) <= 2e-2, (M, K, N, sign, _relerr(y, ref))
        outs[sign] = (y.float().cpu().numpy().astype(np.float64), ref)
    # the perturbation is the oracle's: Y+ - Y- against 2 eps X (z (.) table[c]), element by element
    d_got, d_ref = outs[+1][0] - outs[-1][0], outs[+1][1] - outs[-1][1]
    assert np.abs(d_got - d_ref).max() <= 3e-2 * np.abs(d_ref).max() + 2.0 ** -7 * np.abs(outs[+1][1]).max()
    # deterministic
    again = lib.qzo_perturbed_gemm_table16(x.cuda(), wq, s.cuda(), table.tolist(), M, K, N, seed, base, +1, eps, status=status)
    first = lib.qzo_perturbed_gemm_table16(x.cuda(), wq, s.cuda(), table.tolist(), M, K, N, seed, base, +1, eps, status=status)
    assert torch.equal(again.view(torch.int16), first.view(torch.int16))


def test_table16_scales_take_the_seeded_update():
    from paper_2505_13430_b200 import qzo as lib
    _, _, s, _ = inputs.table16_case(4, 640, 256, seed=3)
    dev = s.cuda().reshape(-1).clone()
    lib.qzo_update_scales_flat(dev, 11, 64, 1e-3, 250.0, 100.0)            # clipped to 100 (Eq. 6)
    ref = oqzo.update_scales_flat(s.float().numpy().reshape(-1), 11, 64, 1e-3, oqzo.ddc_clip(250.0, 100.0))
    got = dev.float().cpu().numpy()
    assert np.abs(got - ref).max() <= 2.0 ** -7 * np.abs(ref).max() and not np.array_equal(got, s.float().numpy().reshape(-1))


@pytest.mark.parametrize("M,K,N", [(16, 256, 128), (40, 688, 688), (300, 1024, 384), (128, 4096, 512), (257, 2048, 1024)])
def test_channelwise_codebook_gemm_matches_oracle(M, K, N):
    # one scale per output channel (the codebook setting of Sec. 4.1): same codes, same table, scales [N]
    from paper_2505_13430_b200 import qzo as lib
    x, codes, s, table = inputs.table16_case(M, K, N, seed=M + K + N + 1)
    s1 = s[:1].contiguous()
    words = torch.from_numpy(int4.pack_int4(codes.numpy().astype(np.int64) - 8).view(np.int32)).cuda()
    wq = lib.qzo_repack_int4(words, K, N)
    status = torch.zeros((1,), dtype=torch.int32, device="cuda")
    seed, base, eps = 31 + M, 8 * (N % 5), 2e-3
    outs = {}
    for sign in (+1, -1, 0):
        y = lib.qzo_perturbed_gemm_codebook16_channelwise(x.cuda(), wq, s1.cuda().reshape(-1), table.tolist(), M, K, N, seed, base,
                                                          sign, eps, status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        ref = olinear.perturbed_linear_table16(x.float().numpy(), codes.numpy(), s1.float().numpy(), table.numpy(),
                                               seed, base, sign, eps, channelwise=True)
        assert _relerr(y, ref) <= 2e-2, (M, K, N, sign, _relerr(y, ref))
        outs[sign] = (y.float().cpu().numpy().astype(np.float64), ref)
    d_got, d_ref = outs[+1][0] - outs[-1][0], outs[+1][1] - outs[-1][1]
    assert np.abs(d_got - d_ref).max() <= 3e-2 * np.abs(d_ref).max() + 2.0 ** -7 * np.abs(outs[+1][1]).max()
    # it is NOT the block-scaled call on the same memory: there the rows below the first would be read as scales
    if K > 64:
        blk = lib.qzo_perturbed_gemm_table16(x.cuda(), wq, s.cuda(), table.tolist(), M, K, N, seed, base, +1, eps, status=status)
        assert not torch.equal(blk.view(torch.int16), torch.from_numpy(outs[+1][0]).bfloat16().cuda().view(torch.int16))
