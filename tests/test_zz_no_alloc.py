"""The allocation-free GEMM entry point (for callers that cannot call cudaMalloc and own no
workspace: all device memory already belongs to their pool, or an allocation's device-wide
synchronisation has no place in their loop) gives the same output as qzo_perturbed_gemm.

Collected last on purpose: a run that stops at the first failure has then run every other test."""
import pytest
import torch

from oracle import int4
from paper_2505_13430_b200 import inputs

pytestmark = pytest.mark.gpu


def _case(lib, M, K, N, seed):
    import numpy as np
    x, q, s = inputs.gemm_case(M, K, N, seed=seed)
    words = torch.from_numpy(int4.pack_int4(q.numpy()).view(np.int32)).cuda()
    return x.cuda(), lib.qzo_repack_int4(words, K, N), s.cuda()


def test_noalloc_entry_matches_workspace_entry_twice_in_a_row():
    from paper_2505_13430_b200 import qzo as lib
    M, K, N = 16, 4096, 1024                       # split-K: the partial sums need scratch memory
    assert 0 < lib.qzo_gemm_workspace_bytes(M, K, N) <= lib.NOALLOC_SCRATCH_BYTES
    status = torch.zeros((1,), dtype=torch.int32, device="cuda")
    y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    # two calls in a row on different inputs: the second one finds the first one's partial sums
    # in the shared scratch array and must not be affected by them
    for call, (seed, sign) in enumerate(((21, +1), (22, -1))):
        x, wq, s = _case(lib, M, K, N, seed)
        ref = lib.qzo_perturbed_gemm(x, wq, s, M, K, N, 1000 + call, 8 * call, sign, 1e-3, status=status)
        y.fill_(float("nan"))
        torch.cuda.synchronize()
        free0, held0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
        lib.qzo_perturbed_gemm_noalloc(x, wq, s, y, M, K, N, 1000 + call, 8 * call, sign, 1e-3, status=status)
        torch.cuda.synchronize()
        if call > 0:        # after the first call on the device (module load, address look-up) nothing is taken
            assert torch.cuda.mem_get_info()[0] >= free0 and torch.cuda.memory_allocated() == held0
        assert int(status.item()) == 0
        # same kernels, same fixed summation order: the outputs are bit-identical (the parity tests
        # of qzo_perturbed_gemm against the oracle allow 2e-2; this is stricter)
        assert torch.equal(y.view(torch.int16), ref.view(torch.int16)), call
    # a problem without split-K (no scratch needed) goes through the same entry point
    M2, K2, N2 = 300, 1024, 384
    x, wq, s = _case(lib, M2, K2, N2, 23)
    y2 = torch.empty((M2, N2), dtype=torch.bfloat16, device="cuda")
    lib.qzo_perturbed_gemm_noalloc(x, wq, s, y2, M2, K2, N2, 5, 0, +1, 1e-3, status=status)
    ref2 = lib.qzo_perturbed_gemm(x, wq, s, M2, K2, N2, 5, 0, +1, 1e-3, status=status)
    torch.cuda.synchronize()
    assert torch.equal(y2.view(torch.int16), ref2.view(torch.int16))


def test_noalloc_entry_rejects_problems_beyond_its_scratch():
    from paper_2505_13430_b200 import qzo as lib
    M, K, N = 128, 8192, 12288                     # split-K partial sums of 18.9 MB exceed the 16 MiB array
    assert lib.qzo_gemm_workspace_bytes(M, K, N) > lib.NOALLOC_SCRATCH_BYTES
    x = torch.zeros((M, K), dtype=torch.bfloat16, device="cuda")
    wq = torch.zeros((lib.qzo_repacked_bytes(K, N),), dtype=torch.uint8, device="cuda")
    s = torch.zeros(((K + 127) // 128, N), dtype=torch.bfloat16, device="cuda")
    y = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(lib.QzoError) as e:
        lib.qzo_perturbed_gemm_noalloc(x, wq, s, y, M, K, N, 1, 0, +1, 1e-3)
    assert e.value.status == lib.ERR_WORKSPACE
