"""Shared helpers of the parity tests: one seeded case -> oracle results and device tensors."""
from __future__ import annotations

import numpy as np

from oracle import awq_oracle as orc
from paper_2306_00978_b200 import synth

REL_L2_TOL = 1e-3        # relative L2 error of y against the fp64 oracle
MAX_ABS_TOL = 5e-3       # max |y - y_ref| / max |y_ref|


class Case:
    """Inputs of one (seed, N, K, M, group, alpha) point and the oracle's quantization of them."""

    def __init__(self, seed, N, K, M, group, alpha):
        self.seed, self.N, self.K, self.M, self.group, self.alpha = seed, N, K, M, group, alpha
        self.W = synth.weight(seed, N, K)
        self.a = synth.act_mean_abs(seed, K)
        self.s = orc.channel_scale(self.a, alpha)
        x = synth.activations(seed, M, K)
        # the caller's side of Eq. 4: x / s, rounded once to fp16; the same x' goes to both sides
        self.x = (x.astype(np.float32) / self.s[None, :]).astype(np.float16)
        self.codes, self.zeros, self.scales = orc.quantize(self.W, self.s, group)
        self.qweight = orc.pack_qweight(self.codes)
        self.scales_gn = orc.pack_scales(orc.stored_groups(self.scales, group))
        self.zeros_packed = orc.pack_zeros(orc.stored_groups(self.zeros, group))

    def y_ref(self, rows=None, tokens=None):
        x = self.x if tokens is None else self.x[tokens]
        c, z, s = self.codes, self.zeros, self.scales
        if rows is not None:
            c, z, s = c[rows], z[rows], s[rows]
        return orc.linear(x, orc.dequantize(c, z, s, self.group))


def to_cuda(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def oracle_packed_to_cuda(case):
    import torch
    qw = torch.from_numpy(case.qweight.view(np.uint8).copy()).cuda()
    sc = torch.from_numpy(case.scales_gn.copy()).cuda()
    zp = torch.from_numpy(case.zeros_packed.copy()).cuda()
    return qw, sc, zp


def assert_parity(y_gpu, y_ref, what=""):
    rel, mx = orc.parity_errors(np.asarray(y_gpu, dtype=np.float64), y_ref)
    assert rel <= REL_L2_TOL, f"{what}: rel-L2 {rel:.3e} > {REL_L2_TOL}"
    assert mx <= MAX_ABS_TOL, f"{what}: max-abs/max|y| {mx:.3e} > {MAX_ABS_TOL}"
    return rel, mx
