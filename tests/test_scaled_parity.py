"""awq_linear_scaled / awq_linear_multi_scaled: diag(s)^-1 (Sec. 3.2: it goes into a neighbouring
operator) folded into the layer call.  The GPU receives the UNSCALED x and inv_s = fp32(1 / s); the
oracle receives x' = fp16(fp32(x) * inv_s), formed here in numpy.  Checked: parity with the oracle at
the layer's tolerance, bit-identity with the plain call on that x', and that the library's
reciprocal is the correctly rounded one."""
import numpy as np
import pytest

from tests.util import Case, assert_parity, oracle_packed_to_cuda, to_cuda
from paper_2306_00978_b200 import synth

pytestmark = pytest.mark.gpu

CASES = [
    # N, K, M, G            kernel that serves the call
    (2432, 4096, 1, 128),   # band kernel, x in registers
    (2432, 4096, 3, 64),
    (2432, 4096, 8, 128),
    (2432, 1408, 1, 128),   # band kernel, x resident in shared memory, ragged last stage
    (2560, 11008, 1, 128),
    (2432, 2304, 2, 64),
    (2432, 1152, 4, 128),   # band kernel that cannot fold (x through the stages): divide kernel + scratch
    (2432, 2048, 6, 128),   # band kernel that cannot fold: divide kernel + scratch
    (512, 1024, 2, 128),    # split-K kernel: divide kernel + scratch
    (384, 1024, 40, 128),   # tensor-core kernel: divide kernel + scratch
]


@pytest.mark.parametrize("N,K,M,G", CASES)
def test_scaled_call_matches_oracle_and_plain_call(N, K, M, G):
    import torch
    from paper_2306_00978_b200 import binding
    case = Case(9000 + N + K + M + G, N, K, M, G, 0.5)
    qw, sc, zp = oracle_packed_to_cuda(case)
    x_raw = synth.activations(case.seed, M, K)                     # what Case divided by s
    inv_s = (np.float32(1.0) / case.s).astype(np.float32)          # IEEE division: correctly rounded
    inv_gpu = binding.inverse_channel_scale(to_cuda(case.a), 0.5, K)
    assert np.array_equal(inv_gpu.cpu().numpy().view(np.uint32), inv_s.view(np.uint32))
    xs = (x_raw.astype(np.float32) * inv_s[None, :]).astype(np.float16)
    # x * (1 / s) is x / s up to the last bit of a few elements
    assert np.mean(xs.view(np.uint16) != case.x.view(np.uint16)) < 0.02
    case.x = xs                                                    # the oracle's input from here on
    plain = binding.linear(to_cuda(xs), qw, sc, zp, N, K, G)
    (y,) = binding.linear_multi_scaled(to_cuda(x_raw), inv_gpu, [(qw, sc, zp, N)], K, G)
    binding.poll_status()
    assert_parity(y.cpu().numpy(), case.y_ref(), f"scaled N={N} K={K} M={M} G={G}")
    assert torch.equal(y, plain)


def test_scaled_multi_call_is_one_launch_where_it_folds():
    import torch
    from paper_2306_00978_b200 import binding
    L = binding.lib()
    K, G, M = 4096, 128, 1
    cases = [Case(9500 + i, n, K, M, G, 0.5) for i, n in enumerate((1024, 1024, 2048))]
    # the three matrices read the same activation: one s, one x
    base = cases[0]
    x_raw = synth.activations(base.seed, M, K)
    inv_s = (np.float32(1.0) / base.s).astype(np.float32)
    base.x = (x_raw.astype(np.float32) * inv_s[None, :]).astype(np.float16)
    mats, refs = [], []
    from oracle import awq_oracle as orc
    for c in cases:
        codes, zeros, scales = orc.quantize(c.W, base.s, G)
        mats.append((to_cuda(orc.pack_qweight(codes).view(np.uint8)), to_cuda(orc.pack_scales(scales)),
                     to_cuda(orc.pack_zeros(zeros)), c.N))
        refs.append(orc.linear(base.x, orc.dequantize(codes, zeros, scales, G)))
    assert L.awq_linear_scaled_needs_scratch(M, sum(c.N for c in cases), K, G) == 0
    n0 = binding.launch_count()
    outs = binding.linear_multi_scaled(to_cuda(x_raw), to_cuda(inv_s), mats, K, G)
    assert binding.launch_count() - n0 == 1
    binding.poll_status()
    for y, ref in zip(outs, refs):
        assert_parity(y.cpu().numpy(), ref, "fused q/k/v with the division folded in")
    # without scratch where one is needed: refused, nothing launched
    x40 = torch.zeros((40, K), dtype=torch.float16, device="cuda")
    y40 = torch.zeros((40, 1024), dtype=torch.float16, device="cuda")
    assert L.awq_linear_scaled_needs_scratch(40, 1024, K, G) == 1
    rc = L.awq_linear_scaled(x40.data_ptr(), to_cuda(inv_s).data_ptr(), None, mats[0][0].data_ptr(),
                             mats[0][1].data_ptr(), mats[0][2].data_ptr(), y40.data_ptr(), 40, 1024, K, G, None)
    assert rc == 1
