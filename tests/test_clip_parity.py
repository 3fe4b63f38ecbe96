"""GPU parity of weight clipping and of the 3-bit grid against the oracle: the chosen ratios,
the packed words, zero points and fp16 scales must all be bit-identical (each is an encoding or
an argmin taken in the same fp32 arithmetic on both sides), and the layer on the result must
meet the usual tolerance."""
import numpy as np
import pytest

from oracle import awq_oracle as orc
from paper_2306_00978_b200 import synth
from tests.util import assert_parity, to_cuda

pytestmark = pytest.mark.gpu

RATIOS = [float(r) for r in np.linspace(1.0, 0.5, 20).astype(np.float32)]


def _inputs(seed, N, K):
    W = synth.weight(seed, N, K).copy()
    rng = np.random.default_rng(seed)
    # sparse large weights so that clipping pays for a good share of the groups
    hot = rng.random((N, K)) < 0.002
    W[hot] = (W[hot].astype(np.float32) * 5.0).astype(np.float16)
    return W, synth.act_mean_abs(seed, K)


def _packed_equal(got, want):
    qw, sc, zp = got
    assert np.array_equal(qw.cpu().numpy().view(np.uint32).reshape(-1), want[0].reshape(-1))
    assert np.array_equal(sc.cpu().numpy().view(np.uint16).reshape(-1), want[1].view(np.uint16).reshape(-1))
    assert np.array_equal(zp.cpu().numpy().reshape(-1), want[2].reshape(-1))


@pytest.mark.parametrize("N,K,G,alpha,bits", [
    (128, 128, 128, 0.0, 4), (256, 640, 64, 0.5, 4), (384, 2304, 128, 0.5, 4),     # 2304: a ragged second chunk
    (1024, 4096, 128, 0.5, 4), (256, 1152, 64, 1.0, 3), (512, 2048, 128, 0.35, 3),
])
def test_clip_search_and_clipped_quantizer_bit_exact(N, K, G, alpha, bits):
    import torch
    from paper_2306_00978_b200 import binding
    W, a = _inputs(500 + N + K, N, K)
    alpha = float(np.float32(alpha))                            # alpha is an fp32 argument of the library
    s = orc.channel_scale(a, alpha)
    want_r = orc.search_clip(W, s, G, RATIOS, bits=bits)
    Wd, ad = to_cuda(W), to_cuda(a)
    got_r = binding.search_clip(Wd, ad, alpha, G, RATIOS, bits=bits)
    torch.cuda.synchronize()
    assert np.array_equal(got_r.cpu().numpy().view(np.uint32), want_r.view(np.uint32))
    assert (want_r < 1.0).mean() > 0.1                          # the case does exercise clipping
    got = binding.quantize_pack(Wd, ad, alpha, G, clip_ratio=got_r, bits=bits)
    want = orc.quantize_pack(W, a, alpha, G, clip=want_r, bits=bits)
    _packed_equal(got, want)
    # reproducible
    again = binding.search_clip(Wd, ad, alpha, G, RATIOS, bits=bits)
    assert torch.equal(again, got_r)


@pytest.mark.parametrize("N,K,G", [(256, 512, 128), (384, 640, 64), (4096, 4096, 128)])
def test_int3_quantizer_bit_exact_and_layer_parity(N, K, G):
    from paper_2306_00978_b200 import binding
    seed = 900 + N + K
    W, a = synth.weight(seed, N, K), synth.act_mean_abs(seed, K)
    got = binding.quantize_pack(to_cuda(W), to_cuda(a), 0.5, G, bits=3)
    want = orc.quantize_pack(W, a, 0.5, G, bits=3)
    _packed_equal(got, want)
    # the layer on 3-bit codes: same kernels, same tolerance (both matrix-vector and tensor-core paths)
    s = orc.channel_scale(a, 0.5)
    codes, zeros, scales = orc.quantize(W, s, G, bits=3)
    Wdq = orc.dequantize(codes, zeros, scales, G)
    for M in (1, 40):
        x = (synth.activations(seed, M, K).astype(np.float32) / s[None, :]).astype(np.float16)
        y = binding.linear(to_cuda(x), *got, N, K, G)
        binding.poll_status()
        assert_parity(y.cpu().numpy(), orc.linear(x, Wdq), f"int3 N={N} K={K} M={M}")


def test_clipping_lowers_the_layer_error_on_weights_with_outliers():
    """End to end on the device: search, clipped quantization, layer; the output error against
    the fp16 layer is lower than without clipping (what the step is for)."""
    from paper_2306_00978_b200 import binding
    N, K, G, M = 512, 1024, 128, 64
    W, a = _inputs(4242, N, K)
    ones = np.ones(K, np.float32)
    x = synth.activations(4242, M, K)
    Wd, xd = to_cuda(W), to_cuda(x)
    r = binding.search_clip(Wd, None, 0.0, G, RATIOS)
    y_ref = x.astype(np.float64) @ W.astype(np.float64).T
    errs = []
    for clip in (None, r):
        packed = binding.quantize_pack(Wd, None, 0.0, G, clip_ratio=clip)
        y = binding.linear(xd, *packed, N, K, G).cpu().numpy().astype(np.float64)
        errs.append(float(((y - y_ref) ** 2).mean()))
    assert errs[1] < 0.9 * errs[0]


@pytest.mark.parametrize("N,K,G,bits,clipped", [(256, 512, 128, 4, False), (384, 640, 64, 4, True),
                                               (1024, 4096, 128, 3, False), (4096, 4096, 128, 4, False)])
def test_symmetric_quantizer_bit_exact_and_layer_parity(N, K, G, bits, clipped):
    """The symmetric grid of Eq. 2 (zero point fixed at 2^(bits-1)): packed arrays bit-identical to
    the oracle, with and without clipping ratios; the layer kernels on them within tolerance."""
    from paper_2306_00978_b200 import binding
    seed = 1300 + N + K + bits
    W, a = _inputs(seed, N, K)
    clip = None
    if clipped:
        rng = np.random.default_rng(seed)
        clip = rng.choice(np.asarray(RATIOS, dtype=np.float32), size=(N, K // G)).astype(np.float32)
    got = binding.quantize_pack(to_cuda(W), to_cuda(a), 0.5, G, bits=bits, symmetric=True,
                                clip_ratio=None if clip is None else to_cuda(clip))
    want = orc.quantize_pack(W, a, 0.5, G, clip=clip, bits=bits, symmetric=True)
    _packed_equal(got, want)
    if N <= 1024:
        s = orc.channel_scale(a, 0.5)
        codes, zeros, scales = orc.quantize(W, s, G, clip=clip, bits=bits, symmetric=True)
        assert (zeros == (1 << (bits - 1))).all()
        Wdq = orc.dequantize(codes, zeros, scales, G)
        for M in (2, 33):
            x = (synth.activations(seed, M, K).astype(np.float32) / s[None, :]).astype(np.float16)
            y = binding.linear(to_cuda(x), *got, N, K, G)
            binding.poll_status()
            assert_parity(y.cpu().numpy(), orc.linear(x, Wdq), f"symmetric N={N} K={K} M={M}")
