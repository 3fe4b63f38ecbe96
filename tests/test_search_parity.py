"""GPU parity of awq_search_alpha (Sec. 3.2, Eq. 4-5) against the oracle's search: the loss of
every grid point within 0.5 %, and the same choice of alpha wherever the oracle's choice is
clear (otherwise a choice whose oracle loss is within 1 % of the least)."""
import numpy as np
import pytest

from oracle import awq_oracle as orc
from tests.util import to_cuda

pytestmark = pytest.mark.gpu


def _inputs(seed, N, K, M):
    rng = np.random.default_rng(seed)
    W = (rng.standard_normal((N, K)) * 0.04).astype(np.float16)
    X = rng.standard_normal((M, K)).astype(np.float32)
    X[:, rng.choice(K, size=max(2, K // 128), replace=False)] *= 25.0      # activation outlier channels
    X = X.astype(np.float16)
    a = np.abs(X.astype(np.float32)).mean(axis=0).astype(np.float32)
    return W, a, X


@pytest.mark.parametrize("N,K,M,G", [(256, 512, 48, 128), (512, 512, 200, 64), (1024, 1024, 256, 128)])
def test_search_alpha_parity(N, K, M, G):
    from paper_2306_00978_b200 import binding
    W, a, X = _inputs(900 + N + M, N, K, M)
    alphas = [float(np.float32(i / 20)) for i in range(20)]                 # the paper's grid size
    ref_losses, ref_best = orc.search_alpha(W, a, X, G, alphas)
    losses, best = binding.search_alpha(to_cuda(W), to_cuda(a), to_cuda(X), G, alphas)
    binding.poll_status()
    losses = np.asarray(losses, dtype=np.float64)
    assert np.allclose(losses, ref_losses, rtol=5e-3), (losses / ref_losses).round(4)
    order = np.sort(ref_losses)
    if order[1] > order[0] * 1.01:
        assert best == ref_best
    else:
        assert ref_losses[best] <= order[0] * 1.01
    assert best > 0 and losses[best] < losses[0]                            # scaling helps here
    # and the same answer twice
    losses2, best2 = binding.search_alpha(to_cuda(W), to_cuda(a), to_cuda(X), G, alphas)
    assert best2 == best and np.array_equal(np.asarray(losses2), np.asarray(losses, dtype=np.float32).astype(np.float64))


def test_search_alpha_argument_errors():
    from paper_2306_00978_b200 import binding
    W, a, X = _inputs(5, 128, 128, 16)
    with pytest.raises(binding.AwqError):
        binding.search_alpha(to_cuda(W), to_cuda(a), to_cuda(X), 128, [0.5, 1.5])
    with pytest.raises(binding.AwqError):
        binding.search_alpha(to_cuda(W), to_cuda(a), to_cuda(X), 128, [0.0] * 65)
