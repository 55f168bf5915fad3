"""The bounded device-side waits of the GEMM kernel, tested without a fault: a test entry withholds the
copies of one quantisation group and shortens the wait limit, so the waits that depend on those copies run
out.  The kernel must RETURN (every role gives up, the CTA drains what it did issue and frees its tensor
memory), report through the status word, and leave later launches unaffected."""
import time

import numpy as np
import pytest
import torch

from oracle import int4
from paper_2505_13430_b200 import inputs

pytestmark = pytest.mark.gpu


def test_expired_wait_is_reported_and_the_next_launch_is_unaffected():
    from paper_2505_13430_b200 import qzo as lib
    M, K, N = 16, 512, 128                                   # one CTA, one work unit of four groups
    x, q, s = inputs.gemm_case(M, K, N, seed=4)
    words = torch.from_numpy(int4.pack_int4(q.numpy()).view(np.int32)).cuda()
    wq = lib.qzo_repack_int4(words, K, N)
    x_d, s_d = x.cuda(), s.cuda()
    status = torch.zeros((1,), dtype=torch.int32, device="cuda")
    before = lib.qzo_perturbed_gemm(x_d, wq, s_d, M, K, N, 1, 0, +1, 1e-3, status=status).clone()
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    y = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    t0 = time.perf_counter()
    lib.qzo_debug_gemm_wait_expiry(x_d, wq, s_d, y, M, K, N, skip_group=1, wait_limit_cycles=2_000_000, status=status)
    torch.cuda.synchronize()                                 # the kernel came back by itself
    elapsed = time.perf_counter() - t0
    assert int(status.item()) == 1
    assert elapsed < 1.0, elapsed                            # a millisecond or so per expired wait, not the two-second limit
    # the context is intact, tensor memory was freed (the next launch allocates all of it) and the result is
    # bit for bit what it was
    status.zero_()
    after = lib.qzo_perturbed_gemm(x_d, wq, s_d, M, K, N, 1, 0, +1, 1e-3, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(after.view(torch.int16), before.view(torch.int16))
    # the same through a larger launch: every CTA of a 3-tile, split-free problem loses its second group
    M2, K2, N2 = 300, 1024, 384
    x2, q2, s2 = inputs.gemm_case(M2, K2, N2, seed=5)
    wq2 = lib.qzo_repack_int4(torch.from_numpy(int4.pack_int4(q2.numpy()).view(np.int32)).cuda(), K2, N2)
    ref2 = lib.qzo_perturbed_gemm(x2.cuda(), wq2, s2.cuda(), M2, K2, N2, 1, 0, +1, 1e-3, status=status).clone()
    y2 = torch.zeros((M2, N2), dtype=torch.bfloat16, device="cuda")
    lib.qzo_debug_gemm_wait_expiry(x2.cuda(), wq2, s2.cuda(), y2, M2, K2, N2, skip_group=1, wait_limit_cycles=2_000_000,
                                   status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 1
    status.zero_()
    again2 = lib.qzo_perturbed_gemm(x2.cuda(), wq2, s2.cuda(), M2, K2, N2, 1, 0, +1, 1e-3, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and torch.equal(again2.view(torch.int16), ref2.view(torch.int16))
