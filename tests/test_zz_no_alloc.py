"""awq_linear_gemv_static: the matrix-vector kernel for callers that cannot allocate.

A serving process whose memory pool owns the whole GPU (or that forbids allocations after
start-up) cannot hand the library a workspace.  This entry point keeps the kernel's scratch
in an array inside the library's device image instead.  The test calls it through the C ABI
twice in a row - the array keeps the first call's contents, so the second call checks that
what must start at zero is cleared - and compares with the regular entry point.

This file is collected last on purpose: a run that stops at the first failure has then
already run every other test.
"""
import numpy as np
import pytest

from tests.util import Case, MAX_ABS_TOL, REL_L2_TOL, oracle_packed_to_cuda, to_cuda

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("N,K,M,G", [(1024, 1408, 1, 128), (512, 2048, 8, 64), (4096, 4096, 3, 128)])
def test_static_scratch_matches_regular_entry_point(N, K, M, G):
    import torch
    from oracle import awq_oracle as orc
    from paper_2306_00978_b200 import binding

    case = Case(7000 + N + K + M, N, K, M, G, 0.5)
    qw, sc, zp = oracle_packed_to_cuda(case)
    x = to_cuda(case.x)
    want = binding.linear(x, qw, sc, zp, N, K, G, path=binding.PATH_GEMV_SPLITK)
    binding.poll_status()
    want = want.cpu().numpy().astype(np.float64)

    mem_before = torch.cuda.memory_allocated()
    out = torch.empty((M, N), dtype=torch.float16, device="cuda")
    mem_with_out = torch.cuda.memory_allocated()
    for call in range(2):                                   # two calls in a row on one stream
        out.fill_(float("nan"))
        binding.linear_gemv_static(x, qw, sc, zp, N, K, G, out)
        binding.poll_status()
        assert torch.cuda.memory_allocated() == mem_with_out >= mem_before
        got = out.cpu().numpy().astype(np.float64)
        rel, mx = orc.parity_errors(got, want)
        assert rel <= REL_L2_TOL and mx <= MAX_ABS_TOL, (call, rel, mx)


def test_static_scratch_rejects_what_does_not_fit():
    import torch
    from paper_2306_00978_b200 import binding
    L = binding.lib()
    case = Case(7100, 128, 128, 1, 128, 0.0)
    qw, sc, zp = oracle_packed_to_cuda(case)
    x9 = torch.zeros((9, 128), dtype=torch.float16, device="cuda")
    y9 = torch.zeros((9, 128), dtype=torch.float16, device="cuda")
    rc = L.awq_linear_gemv_static(x9.data_ptr(), qw.data_ptr(), sc.data_ptr(), zp.data_ptr(), y9.data_ptr(),
                                  9, 128, 128, 128, None)
    assert rc == 11 and b"built-in scratch" in L.awq_status_string(rc)
    torch.cuda.synchronize()
    assert not y9.any()                                     # nothing ran
