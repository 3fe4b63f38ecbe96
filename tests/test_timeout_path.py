"""The bounded device-side waits: one is made to run out, on purpose and harmlessly.

Every wait of the kernels (on a copy's arrival, on another block's partial sums) has a time limit;
a wait that runs out records a code that awq_poll_status reports as AWQ_ERR_TIMEOUT, and the kernel
still runs to its end by itself.  Here the limit is lowered to a few milliseconds and one launch of
the split-K matrix-vector kernel announces 16 bytes more on its copy barriers than its copies
deliver (awq_test_stall_next_gemv), so its first wait can never complete.  Nothing faults, traps or
spins without bound: the data copies themselves are correct and complete, only the byte count is
off.  Afterwards the status is clean again, the arrival counters are reset, and the same call gives
bit for bit what it gave before.
"""
import time

import numpy as np
import pytest

from tests.util import Case, assert_parity, oracle_packed_to_cuda, to_cuda


def test_timeout_status_text_needs_no_gpu():
    from paper_2306_00978_b200 import binding
    L = binding.lib()
    assert b"wait ran out" in L.awq_status_string(9)
    for name in ("awq_set_wait_limit_us", "awq_test_stall_next_gemv", "awq_poll_status"):
        assert hasattr(L, name)


@pytest.mark.gpu
def test_wait_runs_out_kernel_returns_and_library_recovers():
    import torch
    from paper_2306_00978_b200 import binding
    L = binding.lib()
    case = Case(8100, 512, 1024, 2, 128, 0.5)
    qw, sc, zp = oracle_packed_to_cuda(case)
    x = to_cuda(case.x)
    run = lambda: binding.linear(x, qw, sc, zp, case.N, case.K, case.group, path=binding.PATH_GEMV_SPLITK)
    good = run()
    binding.poll_status()
    assert_parity(good.cpu().numpy(), case.y_ref(), "before the time-out")

    binding.set_wait_limit_us(3000)
    try:
        assert L.awq_test_stall_next_gemv() == 0
        t0 = time.time()
        run()                                              # output undefined; the kernel must end by itself
        with pytest.raises(binding.AwqError, match="status 9"):
            binding.poll_status()
        assert time.time() - t0 < 5.0
        binding.poll_status()                              # the report cleared the status word
        # the stall was for one launch only: the next one is normal even with the short limit
        again = run()
        binding.poll_status()
        assert torch.equal(again, good)
    finally:
        binding.set_wait_limit_us(0)
    final = run()
    binding.poll_status()
    assert torch.equal(final, good)
    # a path that uses the (reset) arrival counters of the workspace as well
    y8 = binding.linear(to_cuda(np.tile(case.x, (4, 1))), qw, sc, zp, case.N, case.K, case.group,
                        path=binding.PATH_GEMV_SPLITK)
    binding.poll_status()
    assert_parity(y8.cpu().numpy(), np.tile(case.y_ref(), (4, 1)), "after the time-out, 8 tokens")
