"""Group sizes above 128 (256, 512, 1024 input channels per scale and zero point).

The quantizer takes the group's min / max over all its columns; the packed scale and zero-point
arrays hold one entry per 128 columns (each group's entry group / 128 times in a row), so the layer
kernels run unchanged.  CPU part: the oracle's storage rule against hand-derived positions and
against its own per-group quantization.  GPU part: packed arrays bit-identical to the oracle
(plain, clipped, 3-bit, symmetric), the layer within tolerance on every kernel, the canonical
unpacking, and what the searches answer."""
import numpy as np
import pytest

from oracle import awq_oracle as orc
from paper_2306_00978_b200 import synth
from tests.util import Case, assert_parity, oracle_packed_to_cuda, to_cuda


def test_stored_groups_positions_by_hand():
    # N = 32, K = 512, group 256: two groups per row, four stored entries per row.
    # scales [band][stored group][16]: row n, group gi -> elements ((n/16)*4 + 2*gi)*16 + n%16 and the
    # next stored group, 16 elements on.  Row 17, group 1: band 1 -> (4 + 2)*16 + 1 = 97 and 113.
    N, K, G = 32, 512, 256
    scales = (np.arange(N * 2, dtype=np.float32).reshape(N, 2) + 1).astype(np.float16)
    zeros = (np.arange(N * 2).reshape(N, 2) % 16).astype(np.uint8)
    sc = orc.pack_scales(orc.stored_groups(scales, G)).reshape(-1)
    assert sc.size == N * K // 128
    assert sc[97] == scales[17, 1] and sc[113] == scales[17, 1]
    assert sc[0] == scales[0, 0] and sc[16] == scales[0, 0] and sc[32] == scales[0, 1] and sc[48] == scales[0, 1]
    # zero bytes [band pair][stored group][16]: row 25 (band 1 of pair 0, r = 9: byte 8 + 1, high
    # nibble), group 1 -> stored groups 2 and 3 -> bytes 2*16 + 9 = 41 and 3*16 + 9 = 57
    zp = orc.pack_zeros(orc.stored_groups(zeros, G)).reshape(-1)
    assert zp.size == N * K // 128 // 2
    assert zp[41] >> 4 == zeros[25, 1] and zp[57] >> 4 == zeros[25, 1]
    assert zp[41] & 0xF == zeros[17, 1]
    # groups up to 128 are stored as they are
    assert orc.stored_groups(scales, 128) is not None and orc.stored_groups(scales, 128).shape == (N, 2)


@pytest.mark.parametrize("G", [256, 512, 1024])
def test_oracle_coarse_group_is_the_group_min_max(G):
    """The oracle's quantizer with a coarse group against the definition written out for one row:
    Delta = fp16((max - min) / 15) over the group's G columns, z = clamp(rne(-min / Delta))."""
    N, K = 32, 2048
    W = synth.weight(31 + G, N, K)
    s = orc.channel_scale(synth.act_mean_abs(31 + G, K), 0.5)
    codes, zeros, scales = orc.quantize(W, s, G)
    assert zeros.shape == (N, K // G) and scales.shape == (N, K // G)
    n, gi = 5, 1
    wp = (W[n, gi * G:(gi + 1) * G].astype(np.float32) * s[gi * G:(gi + 1) * G]).astype(np.float32)
    d = np.float16((wp.max() - wp.min()) / np.float32(15))
    assert scales[n, gi] == d
    z = int(np.clip(np.rint(np.float32(-wp.min()) / np.float32(d)), 0, 15))
    assert zeros[n, gi] == z
    q = np.clip(np.rint(wp / np.float32(d)) + z, 0, 15).astype(np.uint8)
    assert np.array_equal(codes[n, gi * G:(gi + 1) * G], q)
    # and the product from the packed arrays (stored per 128 columns) equals the product from the
    # per-group arrays
    x = synth.activations(3, 2, K)
    qw, sc, zp = orc.pack_qweight(codes), orc.pack_scales(orc.stored_groups(scales, G)), orc.pack_zeros(orc.stored_groups(zeros, G))
    y1 = orc.linear_from_packed(x, qw, sc, zp, N, K, G)
    y2 = orc.linear(x, orc.dequantize(codes, zeros, scales, G))
    assert np.array_equal(y1, y2)


def test_sizes_and_rejections_need_no_gpu():
    from paper_2306_00978_b200 import binding
    L = binding.lib()
    for G in (256, 512, 1024):
        assert L.awq_scales_bytes(256, 2048, G) == L.awq_scales_bytes(256, 2048, 128) == 256 * 16 * 2
        assert L.awq_zeros_bytes(256, 2048, G) == L.awq_zeros_bytes(256, 2048, 128)
    assert L.awq_scales_bytes(256, 1152, 256) == 0          # K not a multiple of the group
    assert L.awq_scales_bytes(256, 2048, 32) == 0 and L.awq_scales_bytes(256, 2048, 2048) == 0
    assert L.awq_search_scratch_bytes(16, 256, 2048, 256) == 0


def _packed_equal(got, want):
    qw, sc, zp = got
    assert np.array_equal(qw.cpu().numpy().view(np.uint32).reshape(-1), want[0].reshape(-1))
    assert np.array_equal(sc.cpu().numpy().view(np.uint16).reshape(-1), want[1].view(np.uint16).reshape(-1))
    assert np.array_equal(zp.cpu().numpy().reshape(-1), want[2].reshape(-1))


@pytest.mark.gpu
@pytest.mark.parametrize("N,K,G,alpha,bits,symmetric,clipped", [
    (128, 256, 256, 0.5, 4, False, False), (256, 1024, 512, 0.0, 4, False, False),
    (384, 2048, 1024, 1.0, 4, False, False), (1024, 4096, 256, 0.5, 4, False, False),
    (4096, 4096, 512, 0.5, 4, False, False), (512, 2048, 256, 0.5, 4, False, True),
    (256, 1024, 256, 0.35, 3, False, False), (256, 2048, 1024, 0.5, 3, False, True),
    (384, 1536, 512, 0.5, 4, True, False), (384, 1536, 256, 0.5, 3, True, True),
])
def test_quantize_pack_coarse_groups_bit_exact(N, K, G, alpha, bits, symmetric, clipped):
    import torch
    from paper_2306_00978_b200 import binding
    seed = 4100 + N + K + G + bits
    W, a = synth.weight(seed, N, K), synth.act_mean_abs(seed, K)
    alpha = float(np.float32(alpha))
    clip = None
    if clipped:
        rng = np.random.default_rng(seed)
        clip = rng.choice(np.asarray([1.0, 0.95, 0.9, 0.8, 0.7], dtype=np.float32), size=(N, K // G)).astype(np.float32)
    got = binding.quantize_pack(to_cuda(W), to_cuda(a), alpha, G, bits=bits, symmetric=symmetric,
                                clip_ratio=None if clip is None else to_cuda(clip))
    torch.cuda.synchronize()
    want = orc.quantize_pack(W, a, alpha, G, clip=clip, bits=bits, symmetric=symmetric)
    _packed_equal(got, want)
    again = binding.quantize_pack(to_cuda(W), to_cuda(a), alpha, G, bits=bits, symmetric=symmetric,
                                  clip_ratio=None if clip is None else to_cuda(clip))
    assert all(torch.equal(p, q) for p, q in zip(got, again))


@pytest.mark.gpu
@pytest.mark.parametrize("N,K,M,G", [
    (2432, 4096, 1, 256), (2432, 2048, 6, 512), (512, 1024, 3, 1024), (1024, 2048, 12, 256),
    (768, 4096, 40, 512), (512, 1024, 100, 256), (512, 2048, 300, 1024),
])
def test_layer_on_coarse_groups(N, K, M, G):
    """Every kernel family of awq_linear (band and split-K matrix-vector, chunked matrix-vector,
    chunked tensor-core, one-SM and SM-pair prefill kernels) on arrays quantized with a coarse group,
    quantized on the GPU and by the oracle."""
    import torch
    from paper_2306_00978_b200 import binding
    case = Case(5200 + N + K + M + G, N, K, M, G, 0.5)
    x = to_cuda(case.x)
    packed = oracle_packed_to_cuda(case)
    y = binding.linear(x, *packed, N, K, G)
    binding.poll_status()
    assert_parity(y.cpu().numpy(), case.y_ref(), f"coarse group {G}, M={M}")
    # the same call told the stored group size gives the same bits
    assert torch.equal(y, binding.linear(x, *packed, N, K, 128))
    gq = binding.quantize_pack(to_cuda(case.W), to_cuda(case.a), 0.5, G)
    assert torch.equal(y, binding.linear(x, *gq, N, K, G))
    if M <= 16:
        ys = binding.linear(x, *packed, N, K, G, path=binding.PATH_GEMV_SPLITK)
        binding.poll_status()
        assert_parity(ys.cpu().numpy(), case.y_ref(), f"coarse group {G}, split-K, M={M}")


@pytest.mark.gpu
def test_unpack_canonical_and_searches_on_coarse_groups():
    import torch
    from paper_2306_00978_b200 import binding
    case = Case(5300, 384, 2048, 1, 512, 0.5)
    qw, sc, zp = binding.quantize_pack(to_cuda(case.W), to_cuda(case.a), 0.5, 512)
    codes, scales, zeros = binding.unpack_canonical(qw, sc, zp, case.N, case.K, 512)
    assert np.array_equal(codes.cpu().numpy(), case.codes)
    assert np.array_equal(zeros.cpu().numpy(), case.zeros)
    assert np.array_equal(scales.cpu().numpy().view(np.uint16), case.scales.view(np.uint16))
    L = binding.lib()
    one = torch.zeros(1024, dtype=torch.float32, device="cuda")
    assert L.awq_search_clip(one.data_ptr(), one.data_ptr(), 0.5, 256, 4, None, 1, one.data_ptr(), 384, 2048, None) == 3
