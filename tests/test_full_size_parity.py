"""Parity at the full benchmark sizes, in the launch configuration bench.py times, on sampled
output channels: the oracle quantizes and multiplies only the sampled rows of W (quantization is
independent per row and group), the library quantizes the whole matrix and runs the whole layer."""
import numpy as np
import pytest

from oracle import awq_oracle as orc
from paper_2306_00978_b200 import synth
from tests.util import assert_parity, to_cuda

pytestmark = pytest.mark.gpu

ALPHA, GROUP = 0.5, 128


def _layer(seed, N, K):
    W = synth.weight(seed, N, K)
    a = synth.act_mean_abs(seed, K)
    s = orc.channel_scale(a, ALPHA)
    return W, a, s


def _oracle_rows(W, s, x_scaled, rows):
    codes, zeros, scales = orc.quantize(W[rows], s, GROUP)
    return orc.linear(x_scaled, orc.dequantize(codes, zeros, scales, GROUP))


def _sample_rows(rng, N, count=96):
    # every 128-row slab boundary region and random rows in between
    rows = np.unique(np.concatenate([rng.choice(N, size=count, replace=False), [0, 127, 128, N - 129, N - 1]]))
    return rows


@pytest.mark.parametrize("name,K,N", list(synth.LLAMA2_13B_MLP))
def test_prefill_gemm_13b_m2048_sampled(name, K, N):
    """configs[2]: M = 2048 on the 13B MLP shapes through awq_linear (SM-pair kernel; stream-K on
    the down projection with the registered workspace)."""
    from paper_2306_00978_b200 import binding
    M = 2048
    seed = 4100 + (0 if name == "up_proj" else 1)
    W, a, s = _layer(seed, N, K)
    x = synth.activations(seed, M, K)
    xs = (x.astype(np.float32) / s[None, :]).astype(np.float16)
    qw, sc, zp = binding.quantize_pack(to_cuda(W), to_cuda(a), ALPHA, GROUP)
    y = binding.linear(to_cuda(xs), qw, sc, zp, N, K, GROUP)
    binding.poll_status()
    rows = _sample_rows(np.random.default_rng(seed), N)
    y_ref = _oracle_rows(W, s, xs, rows)
    assert_parity(y.cpu().numpy()[:, rows], y_ref, f"13B {name} M=2048, {len(rows)} sampled channels")


def test_decode_layer_7b_m1_sampled():
    """configs[1]: the 7 linears of a Llama-2-7B-shaped layer at M = 1, issued as bench.py issues
    them (fused q/k/v and gate/up calls), sampled channels of every output."""
    import torch
    from paper_2306_00978_b200 import binding
    shapes = {name: (K, N) for name, K, N in synth.LLAMA2_7B_LAYER}
    packed, ref = {}, {}
    xs_by_k = {}
    for idx, (name, K, N) in enumerate(synth.LLAMA2_7B_LAYER):
        seed = 4200 + idx
        W, a, s = _layer(seed, N, K)
        if K not in xs_by_k:
            x = synth.activations(4200 + K, 1, K)
            xs_by_k[K] = x
        # the fused calls share one x; it is taken as already divided by s (the layer's precondition)
        # and the same x goes to the oracle, whatever s each matrix was quantized with
        packed[name] = (binding.quantize_pack(to_cuda(W), to_cuda(a), ALPHA, GROUP), N, K)
        rows = _sample_rows(np.random.default_rng(seed), N, count=64)
        codes, zeros, scales = orc.quantize(W[rows], s, GROUP)
        ref[name] = (rows, orc.dequantize(codes, zeros, scales, GROUP))
    x4 = xs_by_k[4096]
    x11 = xs_by_k[11008]
    def mats(names):
        return [(*packed[n][0], packed[n][1]) for n in names]
    outs = {}
    q, k, v = binding.linear_multi(to_cuda(x4), mats(["q_proj", "k_proj", "v_proj"]), 4096, GROUP)
    outs.update(q_proj=q, k_proj=k, v_proj=v)
    (qw, sc, zp), N, K = packed["o_proj"]
    outs["o_proj"] = binding.linear(to_cuda(x4), qw, sc, zp, N, K, GROUP)
    g, u = binding.linear_multi(to_cuda(x4), mats(["gate_proj", "up_proj"]), 4096, GROUP)
    outs.update(gate_proj=g, up_proj=u)
    (qw, sc, zp), N, K = packed["down_proj"]
    outs["down_proj"] = binding.linear(to_cuda(x11), qw, sc, zp, N, K, GROUP)
    binding.poll_status()
    torch.cuda.synchronize()
    for name, (K, N) in shapes.items():
        rows, Wd = ref[name]
        x = x4 if K == 4096 else x11
        assert_parity(outs[name].cpu().numpy()[:, rows], orc.linear(x, Wd), f"7B {name} M=1")


@pytest.mark.parametrize("name,K,N", list(synth.LLAMA2_70B_MLP))
def test_70b_mlp_batch_sweep_sampled(name, K, N):
    """configs[3]: the 70B MLP shapes over the small-batch sweep M in {1, 4, 8, 16} through
    awq_linear's own dispatch (band kernel, split-K kernel, tensor-core kernel)."""
    from paper_2306_00978_b200 import binding
    seed = 4300 + (0 if name == "up_proj" else 1)
    W, a, s = _layer(seed, N, K)
    qw, sc, zp = binding.quantize_pack(to_cuda(W), to_cuda(a), ALPHA, GROUP)
    rows = _sample_rows(np.random.default_rng(seed), N, count=48)
    codes, zeros, scales = orc.quantize(W[rows], s, GROUP)
    Wd = orc.dequantize(codes, zeros, scales, GROUP)
    del W
    x_all = synth.activations(seed, 16, K)
    xs_all = (x_all.astype(np.float32) / s[None, :]).astype(np.float16)
    for M in (1, 4, 8, 16):
        xs = np.ascontiguousarray(xs_all[:M])
        y = binding.linear(to_cuda(xs), qw, sc, zp, N, K, GROUP)
        binding.poll_status()
        assert_parity(y.cpu().numpy()[:, rows], orc.linear(xs, Wd), f"70B {name} M={M}")


SWEEP_SHAPES = [("q_proj", 4096, 4096), ("up_proj", 4096, 11008), ("down_proj", 11008, 4096)]


@pytest.mark.parametrize("G,alpha", [(128, 0.5), (64, 1.0), (128, 0.0)])
@pytest.mark.parametrize("name,K,N", SWEEP_SHAPES)
def test_7b_shape_sweep_sampled(name, K, N, G, alpha):
    """The full-shape sweep: the three distinct 7B layer shapes over the token counts
    1 .. 8192 (every kernel and every dispatch branch), both group sizes and the three exact
    alphas, through awq_linear; sampled channels, for large M sampled tokens as well."""
    from paper_2306_00978_b200 import binding
    seed = 7000 + K // 64 + N // 64 + G
    W = synth.weight(seed, N, K)
    a = synth.act_mean_abs(seed, K)
    s = orc.channel_scale(a, alpha)
    qw, sc, zp = binding.quantize_pack(to_cuda(W), to_cuda(a), alpha, G)
    rng = np.random.default_rng(seed)
    rows = _sample_rows(rng, N, count=40)
    codes, zeros, scales = orc.quantize(W[rows], s, G)
    Wdq = orc.dequantize(codes, zeros, scales, G)
    Ms = (1, 2, 4, 8, 16, 32, 64, 128, 512, 2048, 8192)
    x_all = synth.activations(seed, max(Ms), K)
    xs_all = (x_all.astype(np.float32) / s[None, :]).astype(np.float16)
    for M in Ms:
        xs = xs_all[:M]
        y = binding.linear(to_cuda(xs), qw, sc, zp, N, K, G)
        binding.poll_status()
        y = y.cpu().numpy()
        toks = np.arange(M) if M <= 128 else np.unique(np.concatenate(
            [rng.choice(M, size=64, replace=False), [0, 127, 128, 255, 256, M - 1]]))
        y_ref = orc.linear(xs[toks], Wdq)
        assert_parity(y[np.ix_(toks, rows)], y_ref, f"sweep {name} G={G} alpha={alpha} M={M}")
