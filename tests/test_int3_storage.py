"""The 3-bit storage (INT3-g128 setting of the paper's accuracy tables): packed words bit-exact
against the oracle's layout, the round trip through awq_unpack_int3, and the layer on the dense
3-bit array against the oracle's fp64 product, on every variant of the band kernel and through the
expansion path of the other kernels."""
import numpy as np
import pytest

from tests.util import assert_parity, to_cuda
from paper_2306_00978_b200 import synth

pytestmark = pytest.mark.gpu


class Case3:
    def __init__(self, seed, N, K, M, G):
        from oracle import awq_oracle as orc
        self.N, self.K, self.M, self.G = N, K, M, G
        W = synth.weight(seed, N, K)
        a = synth.act_mean_abs(seed, K)
        s = orc.channel_scale(a, 0.5)
        x = synth.activations(seed, M, K)
        self.W, self.a = W, a
        self.x = (x.astype(np.float32) / s[None, :]).astype(np.float16)
        self.codes, self.zeros, self.scales = orc.quantize(W, s, G, bits=3)
        self.q3 = orc.pack_qweight_int3(self.codes)
        self.y_ref = orc.linear(self.x, orc.dequantize(self.codes, self.zeros, self.scales, G))


@pytest.mark.parametrize("N,K,M,G", [
    (2432, 4096, 1, 128),    # band kernel: x in registers, ring known at compile time
    (2432, 4096, 3, 64),
    (2432, 4096, 7, 128),    # x in registers, generic loop
    (2432, 1408, 1, 128),    # x resident in shared memory, ragged last stage
    (2432, 2304, 2, 64),
    (2432, 1152, 5, 128),    # x through the stages
    (512, 1024, 2, 128),     # split-K kernel through the expansion
    (384, 1024, 40, 64),     # tensor-core kernel through the expansion
])
def test_int3_storage_pack_and_layer(N, K, M, G):
    import torch
    from oracle import awq_oracle as orc
    from paper_2306_00978_b200 import binding
    c = Case3(3300 + N + K + M + G, N, K, M, G)
    qw4, sc, zp = binding.quantize_pack(to_cuda(c.W), to_cuda(c.a), 0.5, G, bits=3)
    q3 = binding.pack_int3(qw4, N, K)
    assert q3.numel() == N * K * 3 // 8 == binding.lib().awq_qweight_bytes_int3(N, K)
    assert np.array_equal(q3.cpu().numpy().view(np.uint32), c.q3)
    assert torch.equal(binding.unpack_int3(q3, N, K), qw4)
    y = binding.linear_int3(to_cuda(c.x), q3, sc, zp, N, K, G)
    binding.poll_status()
    assert_parity(y.cpu().numpy(), c.y_ref, f"int3 N={N} K={K} M={M} G={G}")
    # the same kernel on the 4-bit layout holding the same codes gives the same bits
    y4 = binding.linear(to_cuda(c.x), qw4, sc, zp, N, K, G)
    assert torch.equal(y, y4)
