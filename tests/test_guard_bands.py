"""Out-of-bounds writes: every output of the library sits between two guard bands filled with a
sentinel, the call runs, the bands must be untouched and the output fully written.

This stands in for a memory checker on the outputs (the kernels write y, the packed arrays and the
workspace through bulk copies, tensor-map stores and plain stores whose extents are computed per
kernel): a store past the end of an array, or in front of it, lands in a band.  Reads are not
covered.  The calls go through the C ABI with raw pointers into one larger allocation."""
import ctypes

import numpy as np
import pytest

from tests.util import Case, oracle_packed_to_cuda, to_cuda

pytestmark = pytest.mark.gpu

GUARD = 4096          # bytes on each side
SENTINEL = 0xA5


def _guarded(nbytes):
    """A uint8 buffer [guard | payload | guard], payload 256-byte aligned and pre-filled with 0x5A."""
    import torch
    pad = (-nbytes) % 256
    buf = torch.full((GUARD + nbytes + pad + GUARD,), SENTINEL, dtype=torch.uint8, device="cuda")
    buf[GUARD:GUARD + nbytes] = 0x5A
    assert buf.data_ptr() % 256 == 0
    return buf, buf.data_ptr() + GUARD


def _check(buf, nbytes, what):
    import torch
    torch.cuda.synchronize()
    head, tail = buf[:GUARD], buf[GUARD + nbytes:]
    assert bool((head == SENTINEL).all()), f"{what}: bytes in front of the array were written"
    assert bool((tail == SENTINEL).all()), f"{what}: bytes behind the array were written"


@pytest.mark.parametrize("N,K,M,G,path", [
    (2432, 4096, 1, 128, 1),      # band kernel, x in registers
    (2432, 1152, 3, 64, 1),       # band kernel, x through the stages
    (2432, 8320, 2, 128, 1),      # band kernel, x resident
    (512, 1408, 9, 128, 3),       # split-K matrix-vector kernel
    (1024, 1408, 13, 128, 5),     # chunked matrix-vector kernel
    (768, 2304, 24, 64, 5),
    (1024, 1408, 33, 128, 6),     # chunked tensor-core kernel
    (256, 640, 17, 64, 6),
    (384, 640, 100, 64, 4),       # one-SM prefill kernel, ragged token tile
    (512, 1024, 300, 128, 2),     # SM-pair prefill kernel, ragged token tile
    (1024, 2048, 5, 256, 0),      # automatic, coarse group
])
def test_linear_outputs_stay_inside_their_arrays(N, K, M, G, path):
    import torch
    from paper_2306_00978_b200 import binding
    L = binding.lib()
    case = Case(7700 + N + K + M, N, K, M, G, 0.5)
    qw, sc, zp = oracle_packed_to_cuda(case)
    x = to_cuda(case.x)
    binding.ensure_workspace(binding.workspace_bytes(M, N, K, G))
    ybytes = M * N * 2
    buf, yptr = _guarded(ybytes)
    rc = L.awq_linear_path(x.data_ptr(), qw.data_ptr(), sc.data_ptr(), zp.data_ptr(), yptr, M, N, K, G, path, None)
    assert rc == 0
    binding.poll_status()
    _check(buf, ybytes, f"y, path {path}")
    y = buf[GUARD:GUARD + ybytes].view(torch.float16).reshape(M, N)
    ref = binding.linear(x, qw, sc, zp, N, K, G, path=path)
    assert torch.equal(y, ref)                       # fully written, and the same as into a plain tensor


@pytest.mark.parametrize("N,K,G,bits", [(256, 512, 128, 4), (384, 640, 64, 4), (128, 2048, 1024, 3), (1024, 1408, 128, 4)])
def test_quantizer_outputs_stay_inside_their_arrays(N, K, G, bits):
    import torch
    from paper_2306_00978_b200 import binding
    L = binding.lib()
    case = Case(7800 + N + K, N, K, 1, G, 0.5)
    W, a = to_cuda(case.W), to_cuda(case.a)
    qb, sb, zb = binding.packed_sizes(N, K, G)
    bq, pq = _guarded(qb)
    bs, ps = _guarded(sb)
    bz, pz = _guarded(zb)
    rc = L.awq_quantize_pack_ex(W.data_ptr(), a.data_ptr(), 0.5, G, bits, 0, None, pq, ps, pz, N, K, None)
    assert rc == 0
    for buf, n, what in ((bq, qb, "qweight"), (bs, sb, "scales"), (bz, zb, "zeros")):
        _check(buf, n, what)
    ref = binding.quantize_pack(W, a, 0.5, G, bits=bits)
    assert torch.equal(bq[GUARD:GUARD + qb], ref[0].reshape(-1))
    assert torch.equal(bs[GUARD:GUARD + sb].view(torch.float16), ref[1].reshape(-1))
    assert torch.equal(bz[GUARD:GUARD + zb], ref[2].reshape(-1))
    # the 3-bit storage and back
    q3 = int(L.awq_qweight_bytes_int3(N, K))
    b3, p3 = _guarded(q3)
    assert L.awq_pack_int3(pq, p3, N, K, None) == 0
    _check(b3, q3, "3-bit storage")
    b4, p4 = _guarded(qb)
    assert L.awq_unpack_int3(p3, p4, N, K, None) == 0
    _check(b4, qb, "unpacked 4-bit array")


def test_workspace_is_not_overrun():
    """The kernels that use the workspace (split-K, chunked matrix-vector, chunked tensor-core, the
    prefill kernels' split-K / stream-K) with a workspace of exactly awq_workspace_bytes."""
    import torch
    from paper_2306_00978_b200 import binding
    L = binding.lib()
    torch.cuda.synchronize()
    dev = torch.cuda.current_device()
    saved = binding._workspace.pop(dev, None)
    try:
        for (N, K, M, G, path) in ((512, 1408, 9, 128, 3), (2432, 4096, 13, 128, 5), (1024, 1408, 24, 128, 5),
                                   (4096, 4096, 32, 128, 6), (1024, 1408, 64, 64, 6), (384, 4096, 100, 128, 4),
                                   (512, 4096, 300, 128, 2)):
            case = Case(7900 + N + K + M, N, K, M, G, 0.5)
            qw, sc, zp = oracle_packed_to_cuda(case)
            x = to_cuda(case.x)
            need = int(L.awq_workspace_bytes(M, N, K, G))
            assert need > 0
            buf, wptr = _guarded(need)
            assert L.awq_set_workspace(ctypes.c_void_p(wptr), need) == 0
            y = torch.empty((M, N), dtype=torch.float16, device="cuda")
            for _ in range(2):
                rc = L.awq_linear_path(x.data_ptr(), qw.data_ptr(), sc.data_ptr(), zp.data_ptr(), y.data_ptr(),
                                       M, N, K, G, path, None)
                assert rc == 0
            binding.poll_status()
            _check(buf, need, f"workspace, path {path}, M={M}")
            assert L.awq_set_workspace(None, 0) == 0
    finally:
        if saved is not None:
            assert L.awq_set_workspace(saved.data_ptr(), saved.numel()) == 0
            binding._workspace[dev] = saved
