"""GPU parity of awq_quantize_pack against the oracle: packed words, zero points and fp16
scales must be bit-identical (the quantizer is an encoding: exactly one result is right)."""
import numpy as np
import pytest

from oracle import awq_oracle as orc
from paper_2306_00978_b200 import synth
from tests.util import Case, to_cuda

pytestmark = pytest.mark.gpu


def _gpu_quantize(case, a_override="case"):
    import torch
    from paper_2306_00978_b200 import binding
    a = None if a_override is None else to_cuda(case.a)
    qw, sc, zp = binding.quantize_pack(to_cuda(case.W), a, case.alpha, case.group)
    torch.cuda.synchronize()
    return qw, sc, zp


def _assert_bit_exact(case, qw, sc, zp):
    got_q = qw.cpu().numpy().view(np.uint32).reshape(-1)
    got_s = sc.cpu().numpy().view(np.uint16).reshape(-1)
    got_z = zp.cpu().numpy().reshape(-1)
    bad_s = int((got_s != case.scales_gn.view(np.uint16).reshape(-1)).sum())
    bad_z = int((got_z != case.zeros_packed.reshape(-1)).sum())
    bad_q = int((got_q != case.qweight.reshape(-1)).sum())
    assert (bad_s, bad_z, bad_q) == (0, 0, 0), f"mismatching scales/zeros/words: {bad_s}/{bad_z}/{bad_q}"


@pytest.mark.parametrize("N,K,G,alpha", [
    (128, 128, 128, 0.0), (128, 128, 64, 0.5), (256, 512, 64, 0.5), (384, 640, 128, 1.0),
    (1024, 1408, 128, 0.5), (4096, 4096, 128, 0.0), (4096, 4096, 128, 0.5), (4096, 4096, 64, 1.0),
])
def test_quantize_pack_bit_exact(N, K, G, alpha):
    case = Case(1000 + N + K, N, K, 1, G, alpha)
    qw, sc, zp = _gpu_quantize(case)
    _assert_bit_exact(case, qw, sc, zp)
    # and twice: the result is a pure function of the inputs
    qw2, sc2, zp2 = _gpu_quantize(case)
    import torch
    assert torch.equal(qw, qw2) and torch.equal(sc, sc2) and torch.equal(zp, zp2)


def test_alpha_zero_accepts_null_statistics():
    case = Case(77, 256, 256, 1, 128, 0.0)
    qw, sc, zp = _gpu_quantize(case, a_override=None)
    _assert_bit_exact(case, qw, sc, zp)


def test_unpack_canonical_matches_oracle_codes():
    from paper_2306_00978_b200 import binding
    case = Case(78, 384, 512, 1, 64, 0.5)
    qw, sc, zp = _gpu_quantize(case)
    codes, scales, zeros = binding.unpack_canonical(qw, sc, zp, case.N, case.K, case.group)
    assert np.array_equal(codes.cpu().numpy(), case.codes)
    assert np.array_equal(zeros.cpu().numpy(), case.zeros)
    assert np.array_equal(scales.cpu().numpy().view(np.uint16), case.scales.view(np.uint16))


def test_channel_scale_matches_oracle():
    from paper_2306_00978_b200 import binding
    K = 4096
    a = synth.act_mean_abs(5, K)
    a[:4] = [0.0, -1.0, np.inf, np.nan]
    for alpha in (0.0, 0.5, 1.0):
        s = binding.channel_scale(to_cuda(a), alpha, K).cpu().numpy()
        assert np.array_equal(s.view(np.uint32), orc.channel_scale(a, alpha).view(np.uint32))
    # a general exponent goes through pow in fp64 on both sides: allow one fp32 ulp
    s = binding.channel_scale(to_cuda(a), 0.3, K).cpu().numpy()
    ref = orc.channel_scale(a, 0.3)
    assert np.all(np.abs(s.view(np.int32).astype(np.int64) - ref.view(np.int32).astype(np.int64)) <= 1)


def test_degenerate_and_grid_aligned_groups():
    """All-zero groups take Delta = 1, z = q = 0; grid-aligned weights come back exactly."""
    import torch
    from paper_2306_00978_b200 import binding
    rng = np.random.default_rng(9)
    N, K, G = 128, 256, 128
    q = rng.integers(0, 16, size=(N, K // G, G))
    q[:, :, 0], q[:, :, 1] = 0, 15
    z = rng.integers(0, 16, size=(N, K // G))
    W = ((q - z[:, :, None]) * 2.0**-7).reshape(N, K).astype(np.float16)
    W[5, :G] = 0                                                    # a degenerate group
    qw, sc, zp = binding.quantize_pack(to_cuda(W), None, 0.0, G)
    codes, scales, zeros = (t.cpu().numpy() for t in binding.unpack_canonical(qw, sc, zp, N, K, G))
    want_c, want_z, want_s = orc.quantize(W, np.ones(K, np.float32), G)
    assert np.array_equal(codes, want_c) and np.array_equal(zeros, want_z)
    assert np.array_equal(scales.view(np.uint16), want_s.view(np.uint16))
    assert float(scales[5, 0]) == 1.0 and not codes[5, :G].any() and zeros[5, 0] == 0
    back = orc.dequantize(codes, zeros, scales, G)
    assert np.array_equal(back, W.astype(np.float64))


def test_rounding_boundaries_bit_exact():
    """Weights whose quotient w / Delta sits exactly on, one fp16 step below and one above a
    half-integer (where round-to-nearest-even decides the code), and groups whose range is tiny
    against their magnitude (quotients in the thousands): the kernel replaces the per-weight
    division by a multiplication only away from such points, so these exercise its exact path."""
    import torch
    from paper_2306_00978_b200 import binding
    N, K, G = 128, 256, 128
    rng = np.random.default_rng(11)
    W = np.zeros((N, K), dtype=np.float16)
    delta = np.float16(2.0 ** -6)
    for n in range(N):
        for gi in range(K // G):
            k = rng.integers(0, 15, size=G).astype(np.float32)
            base = (k + 0.5) * np.float32(delta)                   # exact in fp16: quotient k + 0.5
            w = base.astype(np.float16)
            step = np.spacing(w)                                   # one fp16 step at each value
            choice = rng.integers(0, 3, size=G)
            w = np.where(choice == 1, w - step, np.where(choice == 2, w + step, w)).astype(np.float16)
            w[0], w[1] = np.float16(0.0), np.float16(15.0 * float(delta))   # min and max fix Delta = 2^-6
            if n % 4 == 3:                                         # tiny range on a large offset
                w = (np.float16(8.0) + (k * np.float32(2.0 ** -7)).astype(np.float16)).astype(np.float16)
            W[n, gi * G:(gi + 1) * G] = w
    s = np.ones(K, dtype=np.float32)                               # alpha = 0
    codes, zeros, scales = orc.quantize(W, s, G)
    qw, sc, zp = binding.quantize_pack(to_cuda(W), None, 0.0, G)
    torch.cuda.synchronize()
    assert np.array_equal(qw.cpu().numpy().view(np.uint32).reshape(-1), orc.pack_qweight(codes).reshape(-1))
    assert np.array_equal(sc.cpu().numpy().view(np.uint16).reshape(-1), orc.pack_scales(scales).view(np.uint16).reshape(-1))
    assert np.array_equal(zp.cpu().numpy().reshape(-1), orc.pack_zeros(zeros).reshape(-1))
