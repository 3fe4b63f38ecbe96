"""GPU parity of awq_linear (matrix-vector and tcgen05 paths) against the fp64 oracle:
relative L2 error <= 1e-3 and max abs error <= 5e-3 * max|y_ref| on the same seeded inputs."""
import numpy as np
import pytest

from tests.util import Case, assert_parity, oracle_packed_to_cuda, to_cuda

pytestmark = pytest.mark.gpu


def _run(case, path, packed=None):
    import torch
    from paper_2306_00978_b200 import binding
    qw, sc, zp = packed if packed is not None else oracle_packed_to_cuda(case)
    y = binding.linear(to_cuda(case.x), qw, sc, zp, case.N, case.K, case.group, path=path)
    binding.poll_status()
    return y.cpu().numpy()


GEMV_CASES = [
    # N, K, M, G, alpha  - several tiles, ragged k-tile counts, both groups, all token counts.
    # PATH_GEMV picks the band kernel for the large-N, M <= 8 cases and the split-K kernel for
    # the others; PATH_GEMV_SPLITK forces the split-K kernel on all of them.
    (128, 128, 1, 128, 0.5), (128, 384, 1, 64, 0.5), (256, 640, 3, 128, 0.0), (384, 1152, 8, 64, 1.0),
    (1024, 1408, 5, 128, 0.5), (512, 2048, 16, 128, 0.5), (256, 896, 9, 64, 0.5),
    (4096, 4096, 1, 128, 0.5), (4096, 4096, 2, 64, 0.5), (4096, 4096, 4, 128, 0.0),
    (2048, 1152, 3, 64, 0.5), (2432, 8320, 1, 128, 0.5), (11008, 4096, 1, 128, 0.5),
    # band kernel with 5..8 tokens: x in registers (K = 4096) and x through the stages
    (4096, 4096, 8, 128, 0.5), (4096, 4096, 5, 64, 0.5), (11008, 4096, 6, 128, 0.5),
    (2432, 8320, 7, 128, 0.5), (2432, 1152, 8, 64, 0.5),
]


@pytest.mark.parametrize("forced", [False, True])
@pytest.mark.parametrize("N,K,M,G,alpha", GEMV_CASES)
def test_gemv_parity(N, K, M, G, alpha, forced):
    from paper_2306_00978_b200 import binding
    path = binding.PATH_GEMV_SPLITK if forced else binding.PATH_GEMV
    case = Case(2000 + N + K + M, N, K, M, G, alpha)
    y = _run(case, path)
    assert_parity(y, case.y_ref(), f"gemv N={N} K={K} M={M} G={G} path={path}")
    y2 = _run(case, path)
    assert np.array_equal(y.view(np.uint16), y2.view(np.uint16))       # bit-reproducible


GEMM_CASES = [
    (128, 128, 16, 128, 0.5), (128, 256, 32, 64, 0.5), (256, 384, 17, 128, 0.0), (384, 640, 100, 64, 1.0),
    (256, 1024, 128, 128, 0.5), (512, 512, 300, 128, 0.5), (1024, 1408, 257, 64, 0.5),
    (2048, 2048, 1000, 128, 0.5), (128, 128, 1, 128, 0.5),
    # more tiles than SM pairs (each pair takes a second tile), ragged last token tile
    (2560, 256, 2100, 128, 0.5), (2560, 384, 2100, 64, 0.5),
    # long K loops: with stream-K most pairs start or end inside a tile, some tiles are cut twice
    (512, 8192, 520, 128, 0.5), (1280, 6144, 1300, 64, 0.5),
    # M <= 128 with a workspace: split-K of the one-SM kernel (several splits per tile, ragged
    # group counts per split, more items than SMs)
    (4096, 4096, 64, 128, 0.5), (1024, 2816, 33, 64, 0.5), (11008, 1408, 128, 128, 0.5), (2560, 1152, 20, 128, 0.5),
    # wide matrices at 33 .. 128 tokens: the SM-pair kernel with half-empty token tiles
    (8192, 512, 100, 128, 0.5), (16384, 256, 40, 64, 0.5), (8192, 384, 64, 128, 0.5),
]


def _run_gemm_without_workspace(case):
    """The tensor-core path with no workspace registered: whole tiles round-robin over the SM pairs."""
    import torch
    from paper_2306_00978_b200 import binding
    L = binding.lib()
    qw, sc, zp = oracle_packed_to_cuda(case)
    x = to_cuda(case.x)
    y = torch.empty((case.M, case.N), dtype=torch.float16, device="cuda")
    torch.cuda.synchronize()
    saved = binding._workspace.pop(torch.cuda.current_device(), None)
    assert L.awq_set_workspace(None, 0) == 0
    try:
        rc = L.awq_linear_path(x.data_ptr(), qw.data_ptr(), sc.data_ptr(), zp.data_ptr(), y.data_ptr(),
                               case.M, case.N, case.K, case.group, binding.PATH_GEMM, None)
        assert rc == 0
        binding.poll_status()
    finally:
        if saved is not None:
            assert L.awq_set_workspace(saved.data_ptr(), saved.numel()) == 0
            binding._workspace[torch.cuda.current_device()] = saved
    return y.cpu().numpy()


@pytest.mark.parametrize("mode", ["auto", "one-sm", "no-workspace"])
@pytest.mark.parametrize("N,K,M,G,alpha", GEMM_CASES)
def test_gemm_parity(N, K, M, G, alpha, mode):
    """PATH_GEMM runs SM pairs when N % 256 == 0 and M > 128, or less on wide matrices (stream-K over the registered
    workspace, or whole tiles round-robin without one) and one SM per tile otherwise;
    PATH_GEMM_1SM forces the latter on every case."""
    from paper_2306_00978_b200 import binding
    case = Case(3000 + N + K + M, N, K, M, G, alpha)
    if mode == "no-workspace":
        run = lambda: _run_gemm_without_workspace(case)
    else:
        path = binding.PATH_GEMM_1SM if mode == "one-sm" else binding.PATH_GEMM
        run = lambda: _run(case, path)
    y = run()
    assert_parity(y, case.y_ref(), f"gemm N={N} K={K} M={M} G={G} {mode}")
    y2 = run()
    assert np.array_equal(y.view(np.uint16), y2.view(np.uint16))


def zero_point_cancellation_bound(x, scales, group):
    """Largest |y| the matrix-vector kernels may return where every code equals its zero point.

    They form  Delta * (2^24 * D - z * X)  per group, D = sum over the group's columns of
    (byte * 2^-24) * x with byte = q_g + 16 * q_{g+8} <= 255 in the tensor-core product (exact
    products, fp32 accumulation in steps of 16 columns), X = sum of x in fp32.  In exact arithmetic
    the terms cancel; what is left is fp32 rounding.  Every partial result is bounded by
    255 * S, S = sum |x| over the group, and at most c = 2 * (group / 16) + 8 roundings of unit
    round-off u = 2^-24 act on such values (two per 16-column accumulation step, then the lower-row
    subtraction, the zero-point and scale multiply-adds, the sum of x and the sums across warps):
        |y[m][n]| <= c * u * sum_g Delta[n][g] * 255 * S[m][g]  +  2^-24   (fp16 output granularity).
    Returned per (m, n)."""
    M, K = x.shape
    S = np.abs(x.astype(np.float64)).reshape(M, K // group, group).sum(axis=2)          # [M][ng]
    c = 2 * (group // 16) + 8
    return c * 2.0 ** -24 * 255.0 * (S @ scales.astype(np.float64).T) + 2.0 ** -24


def test_auto_dispatch_and_special_values():
    """All codes equal to the zero point give y = 0 - exactly on the tensor-core path, up to the
    fp32 rounding bound above on the matrix-vector path; a single non-zero (q - z) gives
    x * (q - z) * Delta."""
    import torch
    from oracle import awq_oracle as orc
    from paper_2306_00978_b200 import binding
    rng = np.random.default_rng(4)
    N, K, G = 256, 512, 128
    zeros = rng.integers(0, 16, size=(N, K // G), dtype=np.uint8)
    scales = (rng.random((N, K // G)) * 0.01 + 0.001).astype(np.float16)
    codes = np.repeat(zeros, G, axis=1)
    codes[200, 300] = (int(zeros[200, 2]) + 3) % 16
    packed = (to_cuda(orc.pack_qweight(codes).view(np.uint8)), to_cuda(orc.pack_scales(scales)),
              to_cuda(orc.pack_zeros(zeros)))
    for M in (1, 8, 40):
        x = rng.standard_normal((M, K)).astype(np.float16)
        y = binding.linear(to_cuda(x), *packed, N, K, G).cpu().numpy().astype(np.float64)
        binding.poll_status()
        ref = orc.linear(x, orc.dequantize(codes, zeros, scales, G))
        mask = np.ones(N, bool)
        mask[200] = False
        if M > 16:
            assert not y[:, mask].any()                      # (q - z) * Delta is formed first: exact zeros
        else:
            bound = zero_point_cancellation_bound(x, scales, G)
            assert (np.abs(y[:, mask]) <= bound[:, mask]).all(), float((np.abs(y) / bound)[:, mask].max())
        slack = bound[:, 200] if M <= 16 else 1e-5
        assert (np.abs(y[:, 200] - ref[:, 200]) <= 2e-3 * np.abs(ref[:, 200]) + slack).all()


def test_quantize_then_linear_back_to_back_on_one_stream():
    """The band kernel copies weights before its stream dependency resolves.  The library must
    cover its own quantizer: awq_quantize_pack followed directly by awq_linear on the same stream,
    x already on the device and nothing in between, gives bit for bit what the same two calls give
    with a synchronize between them - on fresh weights every time, so that a read of the packed
    arrays ahead of the quantizer would show."""
    import torch
    from paper_2306_00978_b200 import binding, synth
    L = binding.lib()
    for (N, K) in ((1792, 4096), (2048, 11008)):
        G, M = 128, 1
        qb, sb, zb = binding.packed_sizes(N, K, G)
        qw = torch.empty(qb, dtype=torch.uint8, device="cuda")
        sc = torch.empty(sb // 2, dtype=torch.float16, device="cuda")
        zp = torch.empty(zb, dtype=torch.uint8, device="cuda")
        x = to_cuda(synth.activations(91, M, K))
        a = to_cuda(synth.act_mean_abs(91, K))
        y = torch.empty((M, N), dtype=torch.float16, device="cuda")
        y_sync = torch.empty_like(y)
        Ws = [to_cuda(synth.weight(9100 + i, N, K)) for i in range(4)]
        stream = torch.cuda.current_stream().cuda_stream
        before = binding.launch_count()
        for it in range(20):
            W = Ws[it % 4] if it < 4 else (Ws[it % 4] * float(1 + it % 3)).contiguous()
            torch.cuda.synchronize()
            # back to back: nothing between the two calls
            assert L.awq_quantize_pack(W.data_ptr(), a.data_ptr(), 0.5, G, qw.data_ptr(), sc.data_ptr(),
                                       zp.data_ptr(), N, K, stream) == 0
            assert L.awq_linear(x.data_ptr(), qw.data_ptr(), sc.data_ptr(), zp.data_ptr(), y.data_ptr(),
                                M, N, K, G, stream) == 0
            torch.cuda.synchronize()
            got = y.clone()
            # the same with the packed arrays complete before the layer is enqueued
            qw.zero_(); sc.zero_(); zp.zero_()
            assert L.awq_quantize_pack(W.data_ptr(), a.data_ptr(), 0.5, G, qw.data_ptr(), sc.data_ptr(),
                                       zp.data_ptr(), N, K, stream) == 0
            torch.cuda.synchronize()
            assert L.awq_linear(x.data_ptr(), qw.data_ptr(), sc.data_ptr(), zp.data_ptr(), y_sync.data_ptr(),
                                M, N, K, G, stream) == 0
            torch.cuda.synchronize()
            assert torch.equal(got, y_sync), (N, K, it)
            qw.zero_(); sc.zero_(); zp.zero_()              # the next round must not find old weights
        assert binding.launch_count() - before == 20 * 4
        binding.poll_status()


def test_auto_dispatch_between_9_and_16_tokens():
    """awq_linear with 9..16 tokens: the chunked matrix-vector kernel when a workspace is registered
    (the binding registers one), the tensor-core kernel otherwise.  Each result is bit-equal to its
    forced path."""
    import torch
    from paper_2306_00978_b200 import binding
    L = binding.lib()
    for (N, K) in ((1024, 1408), (1024, 4096)):
        case = Case(77 + K, N, K, 12, 128, 0.5)
        qw, sc, zp = oracle_packed_to_cuda(case)
        x = to_cuda(case.x)
        auto = binding.linear(x, qw, sc, zp, case.N, case.K, case.group)
        assert torch.equal(auto, binding.linear(x, qw, sc, zp, case.N, case.K, case.group, path=binding.PATH_GEMV_MID))
        assert_parity(auto.cpu().numpy(), case.y_ref(), f"auto M=12, chunked kernel, K={K}")
    # a large matrix (random packed arrays: only the choice of kernel is checked here; parity at
    # this size is covered by the 70B sweep)
    N, K, G, M = 16384, 8192, 128, 12
    qw = torch.randint(0, 256, (N * K // 2,), dtype=torch.uint8, device="cuda")
    sc = (torch.rand((N // 16, K // G, 16), device="cuda") * 0.01 + 0.001).half()
    zp = torch.randint(0, 256, (N // 32, K // G, 16), dtype=torch.uint8, device="cuda")
    x = torch.randn((M, K), device="cuda").half()
    with_ws = binding.linear(x, qw, sc, zp, N, K, G)                       # binding registers a workspace
    assert torch.equal(with_ws, binding.linear(x, qw, sc, zp, N, K, G, path=binding.PATH_GEMV_MID))
    y = torch.empty_like(with_ws)
    ref = torch.empty_like(with_ws)
    torch.cuda.synchronize()
    saved = binding._workspace.pop(torch.cuda.current_device(), None)
    assert L.awq_set_workspace(None, 0) == 0
    try:
        args = (x.data_ptr(), qw.data_ptr(), sc.data_ptr(), zp.data_ptr())
        assert L.awq_linear(*args, y.data_ptr(), M, N, K, G, None) == 0
        assert L.awq_linear_path(*args, ref.data_ptr(), M, N, K, G, binding.PATH_GEMM, None) == 0
        binding.poll_status()
    finally:
        if saved is not None:
            assert L.awq_set_workspace(saved.data_ptr(), saved.numel()) == 0
            binding._workspace[torch.cuda.current_device()] = saved
    assert torch.equal(y, ref)                                              # no workspace: tensor-core kernel
    assert not torch.equal(y, with_ws)


@pytest.mark.parametrize("M,G", [(1, 128), (3, 64), (7, 128)])
def test_multi_matrix_call(M, G):
    """awq_linear_multi: three matrices reading the same x in one launch; each output against
    the oracle, and bit-equal to the single call where that also runs the band kernel."""
    import torch
    from paper_2306_00978_b200 import binding
    K = 1152
    cases = [Case(6000 + i, N, K, M, G, 0.5) for i, N in enumerate((1024, 2432, 1280))]
    x = cases[0].x                                    # one shared activation
    mats = []
    for c in cases:
        qw, sc, zp = oracle_packed_to_cuda(c)
        mats.append((qw, sc, zp, c.N))
    ys = binding.linear_multi(to_cuda(x), mats, K, G)
    binding.poll_status()
    from oracle import awq_oracle as orc
    for c, y, m in zip(cases, ys, mats):
        ref = orc.linear(x, orc.dequantize(c.codes, c.zeros, c.scales, G))
        assert_parity(y.cpu().numpy(), ref, f"multi N={c.N}")
    single = binding.linear(to_cuda(x), *mats[1][:3], mats[1][3], K, G, path=binding.PATH_GEMV)
    assert torch.equal(single, ys[1])                 # N = 2432 runs the band kernel on its own too


def test_end_to_end_quantize_then_linear():
    """The product path end to end: GPU quantize+pack feeding the GPU linear layer."""
    from paper_2306_00978_b200 import binding
    for M, path in ((1, 0), (64, 0)):
        case = Case(4100 + M, 1024, 1024, M, 128, 0.5)
        packed = binding.quantize_pack(to_cuda(case.W), to_cuda(case.a), case.alpha, case.group)
        y = _run(case, path, packed=packed)
        assert_parity(y, case.y_ref(), f"e2e M={M}")


def test_missing_workspace_is_reported():
    import torch
    from paper_2306_00978_b200 import binding
    L = binding.lib()
    case = Case(5, 128, 512, 1, 128, 0.0)
    qw, sc, zp = oracle_packed_to_cuda(case)
    x, y = to_cuda(case.x), torch.empty((1, 128), dtype=torch.float16, device="cuda")
    torch.cuda.synchronize()
    saved = binding._workspace.pop(torch.cuda.current_device(), None)
    assert L.awq_set_workspace(None, 0) == 0
    rc = L.awq_linear(x.data_ptr(), qw.data_ptr(), sc.data_ptr(), zp.data_ptr(), y.data_ptr(),
                      1, 128, 512, 128, None)
    assert rc == 6
    if saved is not None:
        assert L.awq_set_workspace(saved.data_ptr(), saved.numel()) == 0
        binding._workspace[torch.cuda.current_device()] = saved


@pytest.mark.parametrize("N,K,M,G", [
    (512, 1024, 9, 128),      # one chunk
    (1024, 1408, 16, 128),    # ragged second chunk (6 k-tiles)
    (768, 4096, 17, 64),      # three token fragments, four chunks
    (512, 2304, 32, 128),     # four token fragments, ragged last chunk
    (640, 2048, 24, 64),      # 40 bands: a last unit of 8 bands
    (2432, 4096, 13, 128),    # more units than blocks
    (128, 8192, 10, 128),     # one unit of 8 bands per chunk
    (4224, 1152, 9, 128),     # units crossing from one chunk to the next inside a block
])
def test_chunked_matrix_vector_kernel(N, K, M, G):
    """AWQ_PATH_GEMV_MID: units of 16 bands x 1024 input channels, one band per warp; partial sums
    per chunk, added by a second kernel.  Parity with the oracle and bit-reproducibility."""
    from paper_2306_00978_b200 import binding
    case = Case(600 + N + K + M + G, N, K, M, G, 0.5)
    y = _run(case, binding.PATH_GEMV_MID)
    assert_parity(y, case.y_ref(), f"chunked N={N} K={K} M={M} G={G}")
    y2 = _run(case, binding.PATH_GEMV_MID)
    assert np.array_equal(y.view(np.uint16), y2.view(np.uint16))


@pytest.mark.parametrize("N,K,M,G,alpha", [
    (128, 128, 17, 128, 0.5),     # one slab, one stage
    (256, 256, 20, 128, 0.5),
    (512, 1024, 17, 128, 0.0),    # 16-token tile does not fit: 32-token tile
    (1024, 1408, 33, 128, 0.5),   # 64-token tile; 11 stages per unit: the warps' stage parity crosses units
    (768, 4096, 64, 64, 1.0),     # full 64-token tile, group 64, four chunks
    (1280, 2048, 9, 128, 0.5),    # 16-token tile
    (2048, 5120, 48, 64, 0.5),
    (4096, 4096, 32, 128, 0.5),   # more units than blocks: ranges that cross from one chunk to the next
    (19072, 384, 25, 128, 0.5),   # 149 slabs, one short chunk of 3 stages per unit
    (128, 8192, 40, 128, 0.5),    # one slab, many chunks
    (256, 640, 1, 64, 0.5),       # a single token
])
def test_chunked_tensor_core_kernel(N, K, M, G, alpha):
    """AWQ_PATH_GEMM_SKINNY: units of 128 channels x a chunk of K on tcgen05, the chunk's slice of x
    resident in shared memory; partial sums per chunk, added by a second kernel.  Parity with the
    oracle and bit-reproducibility."""
    from paper_2306_00978_b200 import binding
    case = Case(900 + N + K + M + G, N, K, M, G, alpha)
    y = _run(case, binding.PATH_GEMM_SKINNY)
    assert_parity(y, case.y_ref(), f"chunked tensor-core N={N} K={K} M={M} G={G}")
    y2 = _run(case, binding.PATH_GEMM_SKINNY)
    assert np.array_equal(y.view(np.uint16), y2.view(np.uint16))


def test_auto_dispatch_between_17_and_64_tokens():
    """awq_linear with 17..64 tokens and a registered workspace: the chunked matrix-vector kernel up
    to 24 tokens on matrices of at least 2^25 weights, else the chunked tensor-core kernel; above 64
    tokens, or where N is not a multiple of 128, the prefill kernels.  Each result is bit-equal to
    its forced path."""
    import torch
    from paper_2306_00978_b200 import binding
    for (N, K, M, want) in ((1024, 1408, 20, binding.PATH_GEMM_SKINNY), (1024, 1408, 64, binding.PATH_GEMM_SKINNY),
                            (1024, 1408, 65, binding.PATH_GEMM), (8192, 4096, 24, binding.PATH_GEMV_MID),
                            (8192, 4096, 25, binding.PATH_GEMM_SKINNY)):
        if N * K >= 1 << 24:
            qw = torch.randint(0, 256, (N * K // 2,), dtype=torch.uint8, device="cuda")
            sc = (torch.rand((N // 16, K // 128, 16), device="cuda") * 0.01 + 0.001).half()
            zp = torch.randint(0, 256, (N // 32, K // 128, 16), dtype=torch.uint8, device="cuda")
            x = torch.randn((M, K), device="cuda").half()
        else:
            case = Case(31 + M, N, K, M, 128, 0.5)
            qw, sc, zp = oracle_packed_to_cuda(case)
            x = to_cuda(case.x)
        auto = binding.linear(x, qw, sc, zp, N, K, 128)
        forced = binding.linear(x, qw, sc, zp, N, K, 128, path=want)
        binding.poll_status()
        assert torch.equal(auto, forced), (N, K, M)
        if N * K < 1 << 24:
            assert_parity(auto.cpu().numpy(), case.y_ref(), f"auto M={M}")
