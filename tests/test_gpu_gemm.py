"""GPU parity of the perturbed W4A16 GEMM against the oracle (element by element), on shapes that
span several tiles, ragged tails in M, K and N, split-K, and both perturbation signs."""
import numpy as np
import pytest
import torch

from oracle import int4, linear as olinear
from paper_2505_13430_b200 import inputs

pytestmark = pytest.mark.gpu

TOL = 2e-2       # max |a - b| / max |b| per tensor (bf16 outputs)


@pytest.fixture(scope="module")
def lib():
    from paper_2505_13430_b200 import qzo
    return qzo


def _run(lib, x, q, s, seed, base, sign, eps, bias=None):
    M, K = x.shape
    N = q.shape[1]
    words = torch.from_numpy(int4.pack_int4(q.numpy()).view(np.int32)).cuda()
    wq = lib.qzo_repack_int4(words, K, N)
    status = torch.zeros((1,), dtype=torch.int32, device="cuda")
    y = lib.qzo_perturbed_gemm(x.cuda(), wq, s.cuda(), M, K, N, seed, base, sign, eps,
                               bias=None if bias is None else bias.cuda(), status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0, "a bounded device-side wait expired"
    return y


def _ref(x, q, s, seed, base, sign, eps, bias=None):
    return olinear.perturbed_linear(x.float().numpy(), q.numpy(), s.float().numpy(), seed, base, sign, eps,
                                    None if bias is None else bias.numpy())


def _relerr(got, ref):
    got = got.float().cpu().numpy().astype(np.float64)
    return np.abs(got - ref).max() / np.abs(ref).max()


def _floored_relerr(got, ref):
    """Element-wise |a - b| / max(|b|, 1e-2 rms(b)): reported beside the per-tensor figure."""
    got = got.float().cpu().numpy().astype(np.float64)
    floor = 1e-2 * np.sqrt(np.mean(ref * ref))
    return (np.abs(got - ref) / np.maximum(np.abs(ref), floor)).max()


def _rounding_units(got, ref, x, q, s_pert):
    """Element-wise error in units of what the arithmetic allows: every weight s' q is rounded once to
    bf16 (relative 2^-9 at most, independent from weight to weight) and the result once more, so the
    error of Y[t][n] has a standard deviation below 2^-9 sqrt(sum_k (x w)^2 / 3) plus half an ulp of
    the result.  A wrong value in a small-magnitude column shows here, where max|a-b| / max|b| hides it."""
    got = got.float().cpu().numpy().astype(np.float64)
    K = q.shape[0]
    w = s_pert[np.arange(K) // 128] * q.astype(np.float64)
    spread = np.sqrt((x.astype(np.float64) ** 2) @ (w ** 2))
    return (np.abs(got - ref) / (2.0 ** -9 * spread + 2.0 ** -8 * np.abs(ref) + 1e-30)).max()


ELEMENT_UNITS = 5.0     # about 9 standard deviations of the weight-rounding term (3.5 observed)


CASES = [
    # M, K, N
    (16, 256, 128),        # one tile, two groups
    (16, 128, 8),          # single group, N far below a tile
    (40, 688, 688),        # K tail (last group of 48 rows, odd number of k-blocks) and N tail (48)
    (300, 1024, 384),      # two token tiles, ragged M
    (1, 512, 256),         # single token
    (130, 384, 1000),      # N tail 104, 3 groups
    (8, 1024, 384),        # streaming kernel, one token tile of 8
    (5, 688, 688),         # streaming kernel: K tail, N tail, ragged M
    (9, 11008, 192),       # streaming kernel: 86 groups, CTAs share every output block
    (16, 4096, 4096),      # streaming kernel at a sweep size
    (128, 4096, 512),      # split-K with M = 128
    (257, 2048, 1024),     # 256-token tile + 1
]


@pytest.mark.parametrize("M,K,N", CASES)
def test_perturbed_gemm_matches_oracle(lib, M, K, N):
    x, q, s = inputs.gemm_case(M, K, N, seed=M + K + N)
    seed, base, eps = 1234 + M, 8 * (N % 5), 1e-3
    for sign in (+1, -1, 0):
        got = _run(lib, x, q, s, seed, base, sign, eps)
        ref = _ref(x, q, s, seed, base, sign, eps)
        sp = olinear.perturbed_scales(s.float().numpy(), seed, base, sign, eps)
        units = _rounding_units(got, ref, x.float().numpy(), q.numpy(), sp)
        print(f"M={M} K={K} N={N} sign={sign:+d}: max-rel {_relerr(got, ref):.2e}, element-wise with floor "
              f"{_floored_relerr(got, ref):.2e}, {units:.2f} rounding units")
        assert _relerr(got, ref) <= TOL, (M, K, N, sign)
        assert units <= ELEMENT_UNITS, (M, K, N, sign, units)


def test_perturbation_signal_is_resolved(lib):
    # Y+ - Y- = 2 eps X (z (.) q): the difference of the two GPU outputs must follow the oracle's
    # difference, i.e. the prologue really applies sign*eps*z with the oracle's z.
    M, K, N = 64, 1024, 256
    x, q, s = inputs.gemm_case(M, K, N, seed=5)
    eps = 4e-3
    yp = _run(lib, x, q, s, 9, 16, +1, eps).float().cpu().numpy().astype(np.float64)
    ym = _run(lib, x, q, s, 9, 16, -1, eps).float().cpu().numpy().astype(np.float64)
    dref = _ref(x, q, s, 9, 16, +1, eps) - _ref(x, q, s, 9, 16, -1, eps)
    # element by element, against the size of the signal 2 eps X (z (.) q) itself: each of the two bf16
    # outputs carries half an ulp of its own value, the weight rounding is common to both
    assert np.abs((yp - ym) - dref).max() <= 2e-2 * np.abs(dref).max()
    cos = np.sum((yp - ym) * dref) / (np.linalg.norm(yp - ym) * np.linalg.norm(dref))
    assert cos > 0.999
    # a different seed or index base draws different noise
    other = _run(lib, x, q, s, 10, 16, +1, eps).float().cpu().numpy()
    assert np.abs(other - yp).max() > 0
    shifted = _run(lib, x, q, s, 9, 24, +1, eps).float().cpu().numpy()
    assert np.abs(shifted - yp).max() > 0


def test_bias_and_determinism(lib):
    M, K, N = 48, 512, 640
    x, q, s = inputs.gemm_case(M, K, N, seed=11)
    bias = inputs.normal_fp32((N,), 0.5, 3)
    got = _run(lib, x, q, s, 7, 0, +1, 1e-3, bias=bias)
    ref = _ref(x, q, s, 7, 0, +1, 1e-3, bias=bias)
    assert _relerr(got, ref) <= TOL
    again = _run(lib, x, q, s, 7, 0, +1, 1e-3, bias=bias)
    assert torch.equal(got.view(torch.int16), again.view(torch.int16))
    # split-K path is deterministic too
    x, q, s = inputs.gemm_case(16, 4096, 1024, seed=12)
    a = _run(lib, x, q, s, 7, 0, -1, 1e-3)
    b = _run(lib, x, q, s, 7, 0, -1, 1e-3)
    assert torch.equal(a.view(torch.int16), b.view(torch.int16))


def test_bad_arguments_are_rejected(lib):
    x, q, s = inputs.gemm_case(16, 256, 128, seed=1)
    words = torch.from_numpy(int4.pack_int4(q.numpy()).view(np.int32)).cuda()
    wq = lib.qzo_repack_int4(words, 256, 128)
    for kwargs in (dict(sign=2), dict(eps=0.0), dict(base=2)):
        with pytest.raises(lib.QzoError) as e:
            lib.qzo_perturbed_gemm(x.cuda(), wq, s.cuda(), 16, 256, 128, 1, kwargs.get("base", 0),
                                   kwargs.get("sign", 1), kwargs.get("eps", 1e-3))
        assert e.value.status == lib.ERR_BAD_ARG
    # undersized split-K workspace
    x, q, s = inputs.gemm_case(16, 4096, 512, seed=2)
    words = torch.from_numpy(int4.pack_int4(q.numpy()).view(np.int32)).cuda()
    wq = lib.qzo_repack_int4(words, 4096, 512)
    assert lib.qzo_gemm_workspace_bytes(16, 4096, 512) > 0
    small = torch.empty((256,), dtype=torch.uint8, device="cuda")
    with pytest.raises(lib.QzoError) as e:
        lib.qzo_perturbed_gemm(x.cuda(), wq, s.cuda(), 16, 4096, 512, 1, 0, 1, 1e-3, workspace=small)
    assert e.value.status == lib.ERR_WORKSPACE
