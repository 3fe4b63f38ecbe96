"""awq_linear_gemv_static: the matrix-vector kernel for callers that cannot allocate.

A serving process whose memory pool owns the whole GPU (or that forbids allocations after
start-up) cannot hand the library a workspace.  This entry point keeps the kernel's scratch
in an array inside the library's device image instead.  The test calls it through the C ABI
twice in a row on one stream and checks, each time,
  - the output against the CPU oracle at the layer's tolerance,
  - that it is bit-identical to the regular entry point with the same kernel (the header says so),
  - that the device's free memory does not move (the driver's own figure, which would also show
    an allocation made behind torch's back),
after the arrival counters at the head of the shared array were overwritten with garbage, as a
call that was cut short would leave them: what must start at zero is cleared by the call itself.

This file is collected last on purpose: a run that stops at the first failure has then
already run every other test.
"""
import numpy as np
import pytest

from tests.util import Case, assert_parity, oracle_packed_to_cuda, to_cuda

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("N,K,M,G", [(1024, 1408, 1, 128), (512, 2048, 8, 64), (4096, 4096, 3, 128)])
def test_static_scratch_matches_oracle_and_regular_entry_point(N, K, M, G):
    import torch
    from paper_2306_00978_b200 import binding

    case = Case(7000 + N + K + M, N, K, M, G, 0.5)
    y_ref = case.y_ref()
    qw, sc, zp = oracle_packed_to_cuda(case)
    x = to_cuda(case.x)
    want = binding.linear(x, qw, sc, zp, N, K, G, path=binding.PATH_GEMV_SPLITK)
    binding.poll_status()
    assert_parity(want.cpu().numpy(), y_ref, "split-K path")

    out = torch.empty((M, N), dtype=torch.float16, device="cuda")
    # warm-up: the first call on a device looks up the array's address (and may load device code)
    binding.linear_gemv_static(x, qw, sc, zp, N, K, G, out)
    binding.poll_status()
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    for call in range(2):                                   # two calls in a row on one stream
        out.fill_(float("nan"))
        binding.static_scratch_fill(0xA5 if call == 0 else 0xFF)
        binding.linear_gemv_static(x, qw, sc, zp, N, K, G, out)
        binding.poll_status()
        assert torch.cuda.mem_get_info()[0] == free_before, "device memory was allocated or freed"
        assert torch.equal(out, want), f"call {call}: not bit-identical to AWQ_PATH_GEMV_SPLITK"
        assert_parity(out.cpu().numpy(), y_ref, f"static scratch, call {call}")


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
