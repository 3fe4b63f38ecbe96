"""Pins for the CPU oracle: each test checks oracle/awq_oracle.py against something fixed
by the paper or by mathematics (closed forms, exact special cases, brute force), never
against the oracle's own formula retyped and never against the CUDA path."""
import itertools
import os
import struct
from fractions import Fraction

import numpy as np
import pytest

from oracle import awq_oracle as orc
from paper_2306_00978_b200 import synth


# ----------------------------------------------------------------------------- helpers
def _f16_rne_bits(x: float) -> int:
    """Independent fp32 -> fp16 round-to-nearest-even on the bit patterns (no numpy cast)."""
    b = struct.unpack("<I", struct.pack("<f", x))[0]
    sign = (b >> 16) & 0x8000
    exp = (b >> 23) & 0xFF
    man = b & 0x7FFFFF
    if exp == 0xFF:
        return sign | 0x7C00 | (0x200 if man else 0)
    e = exp - 127
    if e > 15:
        return sign | 0x7C00
    if e >= -14:
        m = man | 0x800000
        shift = 13
        he = e + 15
    else:
        if e < -25:
            return sign
        m = man | 0x800000
        shift = 13 + (-14 - e)
        he = 0
    q, r = m >> shift, m & ((1 << shift) - 1)
    half = 1 << (shift - 1)
    if r > half or (r == half and (q & 1)):
        q += 1
    if he == 0:
        return sign | q                       # a carry into bit 10 becomes the smallest normal
    q -= 0x400
    out = (he << 10) + q                      # a mantissa carry increments the exponent
    return sign | min(out, 0x7C00)


def _golden(path):
    rows = {}
    with open(path) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                k, *v = line.split()
                rows[k] = v
    return rows


def _grid_aligned(rng, N, K, G, exps=(-6, -9)):
    """W = (q - z) * 2^-e with codes 0 and 15 present in every group: exactly representable."""
    ng = K // G
    q = rng.integers(0, 16, size=(N, ng, G), dtype=np.int64)
    q[:, :, 0], q[:, :, 1] = 0, 15
    q = rng.permuted(q, axis=2)
    z = rng.integers(0, 16, size=(N, ng), dtype=np.int64)
    e = rng.integers(exps[1], exps[0] + 1, size=(N, ng))
    d = np.ldexp(1.0, e)
    W = ((q - z[:, :, None]) * d[:, :, None]).reshape(N, K)
    W16 = W.astype(np.float16)
    assert np.array_equal(W16.astype(np.float64), W)
    return W16, q.reshape(N, K).astype(np.uint8), z.astype(np.uint8), d.astype(np.float16)


# ------------------------------------------------------------------- rounding primitives
def test_round_half_to_even_table():
    # the quantizer's Round(.) must be half-to-even (np.rint), not half-away (np.round is
    # also half-to-even in numpy, so pin the values themselves)
    x = np.array([0.5, 1.5, 2.5, -0.5, -1.5, 3.5, 6.5, 7.5], dtype=np.float32)
    assert np.rint(x).tolist() == [0.0, 2.0, 2.0, -0.0, -2.0, 4.0, 6.0, 8.0]
    # observable through the oracle: Delta = 1, min = -7 -> z = 7; w = 0.5, 1.5, 2.5 -> 0, 2, 2
    W = np.array([[-7, 8, 0.5, 1.5, 2.5, -0.5, -1.5, 3.5]], dtype=np.float16)
    codes, zeros, scales = orc.quantize(W, np.ones(8, np.float32), 8)
    assert float(scales[0, 0]) == 1.0 and int(zeros[0, 0]) == 7
    assert codes[0].tolist() == [0, 15, 7, 9, 9, 7, 5, 11]


def test_fp16_rounding_matches_bit_level_definition():
    rng = np.random.default_rng(1)
    bits = rng.integers(0, 2**32, size=200_000, dtype=np.uint64).astype(np.uint32)
    specials = np.array([0x33000000, 0x33000001, 0x33800000, 0x387FC000, 0x387FE000, 0x387FF000,
                         0x477FE000, 0x477FEFFF, 0x477FF000, 0x3F801000, 0x3F803000, 0x3F802FFF,
                         0x38800000, 0x00000001, 0x80000000], dtype=np.uint32)
    bits = np.concatenate([bits, specials])
    x = bits.view(np.float32)
    x = x[np.isfinite(x)]
    with np.errstate(over="ignore"):
        got = x.astype(np.float16).view(np.uint16)
    sample = np.concatenate([np.arange(0, 2000), np.arange(x.size - specials.size, x.size)])
    for i in sample:
        assert int(got[i]) == _f16_rne_bits(float(x[i])), hex(int(x[i:i + 1].view(np.uint32)[0]))


# ------------------------------------------------------------------------ Eq. 5: s = s_X^a
def test_channel_scale_special_cases():
    a = np.array([1.0, 4.0, 16.0, 0.25, 0.0, -3.0, np.inf, np.nan, 2.0], dtype=np.float32)
    assert orc.channel_scale(a, 0.0).tolist() == [1.0] * 9            # 0 = "do not scale"
    s1 = orc.channel_scale(a, 1.0)
    assert s1[:4].tolist() == [1.0, 4.0, 16.0, 0.25] and s1[4:8].tolist() == [1.0] * 4
    sh = orc.channel_scale(a, 0.5)
    assert sh[:4].tolist() == [1.0, 2.0, 4.0, 0.5] and sh[4:8].tolist() == [1.0] * 4
    assert sh[8] == np.float32(np.sqrt(2.0))
    # general alpha: exact powers of two, and agreement with exact rational roots
    sq = orc.channel_scale(np.array([16.0, 81.0], np.float32), 0.25)
    assert sq.tolist() == [2.0, 3.0]
    with pytest.raises(ValueError):
        orc.channel_scale(a, 1.5)


# ---------------------------------------------------- Eq. 2: grid-aligned weights round-trip
@pytest.mark.parametrize("G", [64, 128])
def test_grid_aligned_round_trip(G):
    rng = np.random.default_rng(7)
    N, K = 128, 4 * G
    W, q, z, d = _grid_aligned(rng, N, K, G)
    codes, zeros, scales = orc.quantize(W, orc.channel_scale(np.ones(K, np.float32), 0.0), G)
    assert np.array_equal(codes, q)
    assert np.array_equal(zeros, z)
    assert np.array_equal(scales.view(np.uint16), d.view(np.uint16))
    back = orc.dequantize(codes, zeros, scales, G)
    assert np.array_equal(back, W.astype(np.float64))                   # bit-for-bit


# ------------------------------------- Eq. 3/4: Q(W diag(s)) (diag(s)^-1 x) = W x when exact
def test_scaling_equivalence_exact_case():
    rng = np.random.default_rng(11)
    N, K, G, M = 128, 256, 128, 3
    Ws, _, _, _ = _grid_aligned(rng, N, K, G, exps=(-5, -7))             # this is W * s
    a = rng.choice(np.array([1.0, 4.0, 16.0], np.float32), size=K)
    s = orc.channel_scale(a, 0.5)
    assert set(np.unique(s).tolist()) <= {1.0, 2.0, 4.0}
    W = (Ws.astype(np.float64) / s).astype(np.float16)                   # exact: powers of two
    assert np.array_equal(W.astype(np.float64) * s, Ws.astype(np.float64))
    x = (rng.integers(-64, 65, size=(M, K)) / 8.0).astype(np.float16)
    xs = (x.astype(np.float32) / s[None, :]).astype(np.float16)
    assert np.array_equal(xs.astype(np.float64) * s, x.astype(np.float64))
    codes, zeros, scales = orc.quantize(W, s, G)
    y = orc.linear(xs, orc.dequantize(codes, zeros, scales, G))
    y_fp = x.astype(np.float64) @ W.astype(np.float64).T                 # the unquantized layer
    assert np.abs(y - y_fp).max() <= 1e-13 * np.abs(y_fp).max()
    # and the scale really matters: quantizing the *unscaled* W is not on its grid any more
    c2, z2, s2 = orc.quantize(W, np.ones(K, np.float32), G)
    assert np.abs(orc.dequantize(c2, z2, s2, G) - W.astype(np.float64)).max() > 0


# ----------------------------------------------------------------- Sec. 4.2: the pack order
def test_pack_order_worked_example(golden_dir):
    g = _golden(os.path.join(golden_dir, "pack_order.txt"))
    order = [int(v) for v in g["order"]]
    want = int(g["word_for_codes_0_to_7"][0], 16)
    # the slot stored at nibble p is order[p]
    assert [orc.NIBBLE_OF_SLOT.index(p) for p in range(8)] == order
    codes = np.zeros((128, 64), np.uint8)
    # the eight slots of word 0 are rows 0 and 8, columns 0..3 of the first piece of band 0
    slots = [(0, 0), (0, 1), (8, 0), (8, 1), (0, 2), (0, 3), (8, 2), (8, 3)]
    for v, (n, k) in enumerate(slots):
        codes[n, k] = v
    words = orc.pack_qweight(codes)
    assert int(words[0]) == want == 0x75316420
    assert not words[1:].any()
    # the two-at-a-time register conversion that motivates the order: masking the low
    # nibble of each 16-bit half yields slots (0,1); shifting by 4, 8, 12 yields (2,3), (4,5), (6,7)
    w = int(words[0])
    pairs = [((w >> sh) & 0xF, (w >> (sh + 16)) & 0xF) for sh in (0, 4, 8, 12)]
    assert pairs == [(0, 1), (2, 3), (4, 5), (6, 7)]


def test_pack_matches_location_formula_and_round_trips():
    rng = np.random.default_rng(3)
    for N, K in [(128, 64), (256, 192)]:
        codes = rng.integers(0, 16, size=(N, K), dtype=np.uint8)
        words = orc.pack_qweight(codes)
        ref = [0] * (N * K // 8)
        seen = set()
        for n in range(N):
            for k in range(K):
                wi, p = orc.qweight_location(n, k, K)
                assert (wi, p) not in seen
                seen.add((wi, p))
                ref[wi] |= int(codes[n, k]) << (4 * p)
        assert words.tolist() == ref
        assert np.array_equal(orc.unpack_qweight(words, N, K), codes)
    # a block is 512 contiguous bytes and the blocks of one 16-row band follow each other along K
    assert orc.qweight_location(15, 63, 192)[0] == 127
    assert orc.qweight_location(0, 64, 192)[0] == 128
    assert orc.qweight_location(16, 0, 192)[0] == 3 * 128


def _layout_table(golden_dir):
    rows = {"qweight": [], "zeros": [], "scales": [], "int3": []}
    with open(os.path.join(golden_dir, "packed_layout.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            kind, *vals = line.split()
            rows[kind].append(tuple(int(v) for v in vals))
    return rows


def test_packed_layout_against_hand_derived_table(golden_dir):
    """The layout is a free choice, so what pins it is its written definition: the table was worked
    out by hand from the prose of the public header, entry by entry, and covers every index of the
    formula (row in band, upper / lower row, column inside a word, word in piece, piece in block,
    block along K, band): a swapped pair of indices or a wrong nibble table fails here."""
    t = _layout_table(golden_dir)
    assert len(t["qweight"]) >= 12
    nib_seen = set()
    for (n, k, K, byte, half) in t["qweight"]:
        wi, p = orc.qweight_location(n, k, K)
        assert (4 * wi + p // 2, p % 2) == (byte, half), (n, k)
        nib_seen.add(p)
        # the same through the array routine: a single non-zero code lands in that nibble only
        N = 16 * (n // 16 + 1)
        N += (-N) % 16
        codes = np.zeros((N, K), np.uint8)
        codes[n, k] = 0xF
        raw = orc.pack_qweight(codes).astype("<u4").view(np.uint8)
        want = np.zeros_like(raw)
        want[byte] = 0xF0 if half else 0x0F
        assert np.array_equal(raw, want), (n, k)
        # and the closed form printed in the header
        closed = ((n // 16) * (K // 64) + k // 64) * 512 + 16 * (4 * (n % 8) + (k % 16) // 4) \
            + 4 * ((k % 64) // 16) + (0, 2, 1, 3)[k % 4]
        assert closed == byte and (n % 16 >= 8) == bool(half)
    assert nib_seen == set(range(8))                     # every entry of the nibble table is exercised
    for (n, gi, ng, byte, half) in t["zeros"]:
        assert orc.zeros_location(n, gi, ng) == (byte, half), (n, gi)
        N = 32 * (n // 32 + 1)
        z = np.zeros((N, ng), np.uint8)
        z[n, gi] = 0xF
        raw = orc.pack_zeros(z).reshape(-1)
        want = np.zeros_like(raw)
        want[byte] = 0xF0 if half else 0x0F
        assert np.array_equal(raw, want), (n, gi)
    for (n, gi, ng, idx) in t["scales"]:
        assert orc.scales_location(n, gi, ng) == idx, (n, gi)
        N = 16 * (n // 16 + 1)
        sc = np.zeros((N, ng), np.float16)
        sc[n, gi] = 1.0
        raw = orc.pack_scales(sc).reshape(-1)
        assert raw[idx] == 1.0 and np.count_nonzero(raw) == 1, (n, gi)


def test_int3_storage_against_hand_derived_table_and_round_trip(golden_dir):
    t = _layout_table(golden_dir)
    assert len(t["int3"]) >= 10
    for (n, k, K, *pos) in t["int3"]:
        want = [(pos[2 * b], pos[2 * b + 1]) for b in range(3)]              # (byte, bit in byte)
        got = [(4 * w + bit // 8, bit % 8) for (w, bit) in orc.int3_location(n, k, K)]
        assert got == want, (n, k)
        N = 16 * (n // 16 + 1)
        for b in range(3):                                                   # one code bit at a time
            codes = np.zeros((N, K), np.uint8)
            codes[n, k] = 1 << b
            raw = orc.pack_qweight_int3(codes).astype("<u4").view(np.uint8)
            expect = np.zeros_like(raw)
            expect[want[b][0]] = 1 << want[b][1]
            assert np.array_equal(raw, expect), (n, k, b)
    rng = np.random.default_rng(11)
    for N, K in [(128, 64), (256, 192)]:
        codes = rng.integers(0, 8, size=(N, K), dtype=np.uint8)
        words = orc.pack_qweight_int3(codes)
        assert words.size == N * K * 3 // 32                                 # 3/8 byte per weight
        assert np.array_equal(orc.unpack_qweight_int3(words, N, K), codes)
        ref = [0] * words.size
        seen = set()
        for n in range(N):
            for k in range(K):
                for b, (w, bit) in enumerate(orc.int3_location(n, k, K)):
                    assert (w, bit) not in seen
                    seen.add((w, bit))
                    ref[w] |= ((int(codes[n, k]) >> b) & 1) << bit
        assert words.tolist() == ref


def test_zero_and_scale_packing():
    rng = np.random.default_rng(5)
    N, ng = 256, 3
    zeros = rng.integers(0, 16, size=(N, ng), dtype=np.uint8)
    packed = orc.pack_zeros(zeros)
    assert packed.shape == (N // 32, ng, 16)
    flat = packed.reshape(-1)
    seen = set()
    for n in range(N):
        for gi in range(ng):
            b, nib = orc.zeros_location(n, gi, ng)
            assert (b, nib) not in seen
            seen.add((b, nib))
            assert (int(flat[b]) >> (4 * nib)) & 0xF == int(zeros[n, gi])
    assert np.array_equal(orc.unpack_zeros(packed, N, ng), zeros)
    sc = rng.standard_normal((N, ng)).astype(np.float16)
    ps = orc.pack_scales(sc)
    assert ps.shape == (N // 16, ng, 16)
    for n in (0, 5, 15, 16, 127, 128, 255):
        for gi in range(ng):
            assert ps.reshape(-1)[orc.scales_location(n, gi, ng)] == sc[n, gi]
    assert np.array_equal(orc.unpack_scales(ps, N, ng), sc)
    # parameters of consecutive groups are contiguous: 32 bytes of scales per band, 16 bytes of
    # zero points per pair of bands
    assert orc.scales_location(0, 1, ng) - orc.scales_location(0, 0, ng) == 16
    assert orc.zeros_location(0, 1, ng)[0] - orc.zeros_location(0, 0, ng)[0] == 16
    assert orc.zeros_location(16, 0, ng)[0] - orc.zeros_location(0, 0, ng)[0] == 8


# ------------------------------------------------------- dequantize-then-multiply, exactly
def test_linear_special_cases():
    rng = np.random.default_rng(13)
    N, K, G, M = 128, 256, 128, 4
    zeros = rng.integers(0, 16, size=(N, K // G), dtype=np.uint8)
    scales = (rng.random((N, K // G)) * 0.01 + 0.001).astype(np.float16)
    x = rng.standard_normal((M, K)).astype(np.float16)
    codes = np.repeat(zeros, G, axis=1)                                  # every code = its zero point
    y0 = orc.linear(x, orc.dequantize(codes, zeros, scales, G))
    assert not y0.any()
    n, k = 77, 200
    codes2 = codes.copy()
    codes2[n, k] = (int(zeros[n, 1]) + 5) % 16
    diff = int(codes2[n, k]) - int(zeros[n, 1])
    y1 = orc.linear(x, orc.dequantize(codes2, zeros, scales, G))
    want = x[:, k].astype(np.float64) * diff * float(scales[n, 1])
    assert np.array_equal(y1[:, n], want)
    y1[:, n] = 0
    assert not y1.any()
    # linear in x
    codes3 = rng.integers(0, 16, size=(N, K), dtype=np.uint8)
    Wdq = orc.dequantize(codes3, zeros, scales, G)
    xa = (rng.integers(-8, 9, size=(M, K))).astype(np.float16)
    xb = (rng.integers(-8, 9, size=(M, K))).astype(np.float16)
    lhs = orc.linear((xa + xb).astype(np.float16), Wdq)
    assert np.allclose(lhs, orc.linear(xa, Wdq) + orc.linear(xb, Wdq), rtol=1e-12, atol=1e-12)


def test_linear_against_explicit_sum():
    rng = np.random.default_rng(17)
    N, K, G, M = 128, 128, 64, 2
    codes = rng.integers(0, 16, size=(N, K), dtype=np.uint8)
    zeros = rng.integers(0, 16, size=(N, K // G), dtype=np.uint8)
    scales = (rng.random((N, K // G)) * 0.01 + 0.001).astype(np.float16)
    x = rng.standard_normal((M, K)).astype(np.float16)
    y = orc.linear(x, orc.dequantize(codes, zeros, scales, G))
    for m in range(M):
        for n in range(0, N, 9):
            acc = Fraction(0)
            for k in range(K):
                w = Fraction(int(codes[n, k]) - int(zeros[n, k // G])) * Fraction(float(scales[n, k // G]))
                acc += Fraction(float(x[m, k])) * w
            assert abs(y[m, n] - float(acc)) <= 1e-12 * max(1.0, abs(float(acc)))
    # the packed entry point agrees, also on a subset of rows
    qw, sc, zp = orc.pack_qweight(codes), orc.pack_scales(scales), orc.pack_zeros(zeros)
    assert np.array_equal(orc.linear_from_packed(x, qw, sc, zp, N, K, G), y)
    rows = np.array([3, 64, 127])
    assert np.array_equal(orc.linear_from_packed(x, qw, sc, zp, N, K, G, rows=rows), y[:, rows])


# --------------------------------------------------------------- brute force on tiny groups
@pytest.mark.parametrize("G", [2, 3, 4])
def test_brute_force_tiny_groups(G):
    """For the oracle's own (Delta, z) the chosen codes must minimise the squared error over
    all 16^G code vectors (exact rational arithmetic)."""
    rng = np.random.default_rng(100 + G)
    vals = (rng.integers(-40, 41, size=(40, G)) / 64.0).astype(np.float16)
    vals = vals[(vals.max(axis=1) > 0) & (vals.min(axis=1) < 0)]
    codes, zeros, scales = orc.quantize(vals, np.ones(G, np.float32), G)
    for r in range(vals.shape[0]):
        d, z = Fraction(float(scales[r, 0])), int(zeros[r, 0])
        w = [Fraction(float(v)) for v in vals[r]]
        err = lambda qs: sum((wi - (qi - z) * d) ** 2 for wi, qi in zip(w, qs))
        best = min(err(qs) for qs in itertools.product(range(16), repeat=G))
        assert err([int(c) for c in codes[r]]) <= best * (1 + Fraction(1, 2**20))


# ------------------------------------------------------------ closed-form error invariants
def _gaussian_case(seed, N, K):
    return synth.weight(seed, N, K), synth.act_mean_abs(seed, K)


@pytest.mark.parametrize("alpha,G", [(0.0, 128), (0.5, 128), (1.0, 64)])
def test_error_bound_invariants(alpha, G):
    N, K = 256, 1024
    W, a = _gaussian_case(21, N, K)
    s = orc.channel_scale(a, alpha)
    codes, zeros, scales = orc.quantize(W, s, G)
    wp = W.astype(np.float64) * s.astype(np.float64)
    wg = wp.reshape(N, K // G, G)
    d = scales.astype(np.float64)[:, :, None]
    back = orc.dequantize(codes, zeros, scales, G).reshape(N, K // G, G)
    straddle = (wg.min(axis=2) <= 0) & (wg.max(axis=2) >= 0)
    assert straddle.all()                                  # Gaussian groups always straddle 0
    bound = (0.5 + 15 * 2.0**-11) * d + 2.0**-22 * np.abs(wg) + 1e-12
    assert (np.abs(wg - back) <= bound).all()
    cg = codes.reshape(N, K // G, G)
    imin, imax = wg.argmin(axis=2), wg.argmax(axis=2)
    qmin = np.take_along_axis(cg, imin[:, :, None], axis=2)
    qmax = np.take_along_axis(cg, imax[:, :, None], axis=2)
    assert (qmin == 0).all()
    assert np.isin(qmax, (14, 15)).all() and (qmax == 15).mean() > 0.9
    # Delta is the fp16 rounding of range / 15
    rng_ = (wg.max(axis=2) - wg.min(axis=2)) / 15.0
    assert (np.abs(scales.astype(np.float64) - rng_) <= 2.0**-11 * rng_ * 1.0001).all()


def test_round_error_statistics(golden_dir):
    """Sec. 3.2: the rounding error is roughly uniform on [0, 0.5] with mean 0.25."""
    g = _golden(os.path.join(golden_dir, "round_error_model.txt"))
    N, K, G = 512, 1024, 128
    W, a = _gaussian_case(22, N, K)
    for alpha in (0.0, 0.5):
        s = orc.channel_scale(a, alpha)
        codes, zeros, scales = orc.quantize(W, s, G)
        wp = (W.astype(np.float64) * s).reshape(N, K // G, G)
        d = scales.astype(np.float64)[:, :, None]
        back = orc.dequantize(codes, zeros, scales, G).reshape(N, K // G, G)
        err = np.abs(wp - back) / d
        inside = (codes.reshape(err.shape) > 0) & (codes.reshape(err.shape) < 15)
        e = err[inside]
        assert e.min() >= float(g["round_err_min"][0])
        assert e.max() <= float(g["round_err_max"][0]) + 1e-6
        assert abs(e.mean() - float(g["round_err_mean"][0])) < 0.01
        hist, _ = np.histogram(e, bins=5, range=(0, 0.5))
        assert hist.min() / hist.max() > 0.9                # flat


def test_salient_channel_scaling_trend(golden_dir):
    """Sec. 3.2 / Table 2: multiplying 1 % of the channels by s > 1 leaves most group
    Deltas unchanged and shrinks those channels' error by (Delta'/Delta) / s."""
    rows = []
    with open(os.path.join(golden_dir, "scale_study_table2.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                rows.append([float(v) for v in line.split()])
    for s_, _, ratio, ratio_over_s in rows:                # the table's own identity
        assert abs(ratio / s_ - ratio_over_s) < 2e-3
    N, K, G = 512, 2048, 128
    W = synth.weight(23, N, K)
    sal = synth.outlier_channels(23, K)
    base_codes, base_z, base_d = orc.quantize(W, np.ones(K, np.float32), G)
    base_err = np.abs(orc.dequantize(base_codes, base_z, base_d, G) - W.astype(np.float64))
    prev_changed, prev_rel = -1.0, 2.0
    for s_, *_ in rows[1:]:
        s = np.ones(K, np.float32)
        s[sal] = s_
        c, z, d = orc.quantize(W, s, G)
        changed = (d.view(np.uint16) != base_d.view(np.uint16)).mean()
        ratio = (d.astype(np.float64) / base_d.astype(np.float64)).mean()
        err = np.abs(orc.dequantize(c, z, d, G) / s.astype(np.float64) - W.astype(np.float64))
        rel = err[:, sal].mean() / base_err[:, sal].mean()
        assert changed > prev_changed and changed < 0.5     # a minority, growing with s
        assert 1.0 <= ratio < 1.5
        assert rel < prev_rel                               # salient error keeps falling
        assert abs(rel - ratio / s_) < 0.15 * ratio / s_ + 0.05   # ~ (Delta'/Delta) / s
        prev_changed, prev_rel = changed, rel


def test_alpha_zero_ignores_statistics_and_output_bound():
    N, K, G, M = 256, 1024, 128, 2
    seed = 24
    W, a = _gaussian_case(seed, N, K)
    q0 = orc.quantize_pack(W, a, 0.0, G)
    q1 = orc.quantize_pack(W, a * 7 + 1, 0.0, G)
    q2 = orc.quantize_pack(W, None, 0.0, G)
    for u, v, w in zip(q0, q1, q2):
        assert np.array_equal(u, v) and np.array_equal(u, w)
    for alpha in (0.0, 0.5, 1.0):
        s = orc.channel_scale(a, alpha)
        x = synth.activations(seed, M, K)
        xs = (x.astype(np.float32) / s[None, :]).astype(np.float16)
        codes, zeros, scales = orc.quantize(W, s, G)
        y = orc.linear(xs, orc.dequantize(codes, zeros, scales, G))
        y_fp = xs.astype(np.float64) @ (W.astype(np.float64) * s).T
        dk = np.repeat(scales.astype(np.float64), G, axis=1)             # [N][K]
        bound = np.abs(xs.astype(np.float64)) @ (0.508 * dk).T
        assert (np.abs(y - y_fp) <= bound + 1e-9).all()
        rel = np.linalg.norm(y - y_fp) / np.linalg.norm(y_fp)
        assert rel < 0.2


def test_activation_aware_scaling_reduces_output_error():
    """The paper's claim in Sec. 3.2: scaling salient channels lowers the layer's output error
    on activations with outlier channels (alpha = 0.5 beats plain round-to-nearest)."""
    N, K, G, M = 512, 2048, 128, 16
    seed = 25
    W, a = _gaussian_case(seed, N, K)
    x = synth.activations(seed, M, K)
    y_fp = x.astype(np.float64) @ W.astype(np.float64).T
    errs = {}
    for alpha in (0.0, 0.5):
        s = orc.channel_scale(a, alpha)
        xs = (x.astype(np.float32) / s[None, :]).astype(np.float16)
        codes, zeros, scales = orc.quantize(W, s, G)
        y = orc.linear(xs, orc.dequantize(codes, zeros, scales, G))
        errs[alpha] = np.linalg.norm(y - y_fp) / np.linalg.norm(y_fp)
    assert errs[0.5] < 0.7 * errs[0.0]


def test_parity_error_helper():
    y_ref = np.array([[3.0, 4.0]])
    rel, mx = orc.parity_errors(np.array([[3.0, 4.5]]), y_ref)
    assert abs(rel - 0.1) < 1e-12 and abs(mx - 0.125) < 1e-12


# ----------------------------------------------------------------- scale search (Eq. 4, Eq. 5)
def _search_inputs(seed, N=64, K=256, M=48, outliers=True):
    rng = np.random.default_rng(seed)
    W = (rng.standard_normal((N, K)) * 0.05).astype(np.float16)
    X = rng.standard_normal((M, K)).astype(np.float32)
    if outliers:                      # a few input channels carry activations ~30x larger (Sec. 3.1)
        X[:, rng.choice(K, size=4, replace=False)] *= 30.0
    X = X.astype(np.float16)
    a = np.abs(X.astype(np.float32)).mean(axis=0).astype(np.float32)
    return W, a, X


def test_search_alpha_zero_is_plain_rtn_loss():
    """alpha = 0 is "do not scale" (Sec. 3.2): its loss is the round-to-nearest layer's output
    error, written out here without the search routine."""
    W, a, X = _search_inputs(1)
    losses, _ = orc.search_alpha(W, a, X, 128, [0.0])
    codes, zeros, scales = orc.quantize(W, np.ones(W.shape[1], dtype=np.float32), 128)
    Wd = orc.dequantize(codes, zeros, scales, 128)
    direct = np.mean((X.astype(np.float64) @ (Wd - W.astype(np.float64)).T) ** 2)
    assert np.isclose(losses[0], direct, rtol=1e-12)


def test_search_alpha_brute_force_tiny():
    """A tiny case evaluated element by element with Python loops (Eq. 4 as printed)."""
    rng = np.random.default_rng(2)
    N, K, M, G = 2, 64, 3, 64
    W = (rng.standard_normal((N, K)) * 0.1).astype(np.float16)
    X = rng.standard_normal((M, K)).astype(np.float16)
    a = np.abs(X.astype(np.float32)).mean(axis=0).astype(np.float32)
    alphas = [0.0, 0.5, 1.0]
    losses, best = orc.search_alpha(W, a, X, G, alphas)
    for i, alpha in enumerate(alphas):
        s = orc.channel_scale(a, alpha)
        codes, zeros, scales = orc.quantize(W, s, G)
        total = 0.0
        for m in range(M):
            for n in range(N):
                yq = 0.0
                yr = 0.0
                for k in range(K):
                    wq = (float(codes[n, k]) - float(zeros[n, k // G])) * float(scales[n, k // G])
                    xs = float(np.float16(np.float32(X[m, k]) / s[k]))
                    yq += wq * xs
                    yr += float(W[n, k]) * float(X[m, k])
                total += (yq - yr) ** 2
        assert np.isclose(losses[i], total / (M * N), rtol=1e-9)
    assert best == int(np.argmin(losses))


def test_search_alpha_loss_scales_with_the_square_of_x():
    """Multiplying the calibration activations by 2 (exact in fp16) with the statistic s_X held
    fixed multiplies every output difference by 2, hence the loss by 4."""
    W, a, X = _search_inputs(3)
    alphas = [0.0, 0.25, 0.5, 1.0]
    l1, b1 = orc.search_alpha(W, a, X, 128, alphas)
    l2, b2 = orc.search_alpha(W, a, (X.astype(np.float32) * 2).astype(np.float16), 128, alphas)
    assert np.allclose(l2, 4.0 * l1, rtol=1e-12) and b1 == b2


def test_search_alpha_prefers_scaling_when_activations_have_outliers():
    """Sec. 3.1-3.2: protecting the weight channels that meet large activations lowers the
    output error, so with outlier channels some alpha > 0 beats alpha = 0; without outliers and
    with a flat statistic every alpha gives s = 1 and the same loss."""
    W, a, X = _search_inputs(4, outliers=True)
    alphas = [i / 20 for i in range(20)]
    losses, best = orc.search_alpha(W, a, X, 128, alphas)
    assert best > 0 and losses[best] < 0.9 * losses[0]
    flat = np.ones_like(a)
    lf, _ = orc.search_alpha(W, flat, X, 128, [0.0, 0.5, 1.0])
    assert lf[0] == lf[1] == lf[2]


# ----------------------------------------------------------- weight clipping, 3-bit grid
def _clip_example(sign):
    """One group of 128 whose best clipping ratio and codes follow by hand: delta = 2^-6; the
    values are 0, an outlier 20 delta and 126 values in {2, 6, 10, 14} delta.  On the full range
    Delta = 20 delta / 15 = 4 delta / 3 and every v in {2, 6, 10, 14} sits half-way between two
    levels (0.75 v = 1.5, 4.5, 7.5, 10.5): error (2 delta / 3)^2 each, 126 * 4/9 = 56 delta^2 in
    all.  With ratio 0.75 the range is 15 delta, Delta = delta, every value but the outlier is a
    level and the outlier saturates: error (5 delta)^2 = 25 delta^2 < 56 delta^2."""
    delta = 2.0**-6
    v = np.array([0] + [2, 6, 10, 14] * 31 + [2, 6, 20], dtype=np.float64)
    assert v.size == 128
    return (sign * v * delta).astype(np.float16)[None, :], v.astype(np.int64)


@pytest.mark.parametrize("sign", [1, -1])
def test_clip_worked_example(sign):
    W, v = _clip_example(sign)
    ones = np.ones(128, np.float32)
    r = orc.search_clip(W, ones, 128, [1.0, 0.75])
    assert r.shape == (1, 1) and r[0, 0] == np.float32(0.75)
    codes, zeros, scales = orc.quantize(W, ones, 128, clip=r)
    assert float(scales[0, 0]) == 2.0**-6
    if sign > 0:
        assert zeros[0, 0] == 0 and np.array_equal(codes[0], np.minimum(v, 15))
    else:
        assert zeros[0, 0] == 15 and np.array_equal(codes[0], 15 - np.minimum(v, 15))
    # the other order of the list: same ratio
    assert orc.search_clip(W, ones, 128, [0.75, 1.0])[0, 0] == np.float32(0.75)
    # the clipped reconstruction misses only the outlier: 25 delta^2
    back = orc.dequantize(codes, zeros, scales, 128)
    assert np.isclose(((back - W.astype(np.float64)) ** 2).sum(), 25 * 2.0**-12, rtol=1e-12)


def test_clip_ratio_one_is_the_plain_quantizer_and_ties_keep_the_first():
    W, a = _gaussian_case(31, 64, 512)
    s = orc.channel_scale(a, 0.5)
    r = orc.search_clip(W, s, 128, [1.0])
    assert (r == 1.0).all()
    plain = orc.quantize(W, s, 128)
    clipped = orc.quantize(W, s, 128, clip=r)
    assert all(np.array_equal(p, c) for p, c in zip(plain, clipped))
    # a list that repeats a ratio has equal errors for both copies: the choice must not change
    r2 = orc.search_clip(W, s, 128, [0.9, 0.8, 0.9, 0.8])
    r1 = orc.search_clip(W, s, 128, [0.9, 0.8])
    assert np.array_equal(r1, r2)


@pytest.mark.parametrize("bits,G", [(4, 128), (3, 64)])
def test_clip_choice_is_the_least_error_through_an_independent_route(bits, G):
    """The chosen ratio's error, recomputed in fp64 through quantize + dequantize (functions
    pinned above), is the least over the list up to fp32 summation error, and never above the
    unclipped error."""
    N, K = 32, 512
    W, a = _gaussian_case(33, N, K)
    W = W.copy()
    W[::3, ::37] *= np.float16(6.0)                         # a few outliers so that clipping pays
    s = orc.channel_scale(a, 0.5)
    ratios = np.linspace(1.0, 0.5, 11).astype(np.float32)
    chosen = orc.search_clip(W, s, G, ratios, bits=bits)
    assert np.isin(chosen, ratios).all()
    wp = (W.astype(np.float32) * s[None, :]).astype(np.float64).reshape(N, K // G, G)
    errs = []
    for r in ratios:
        clip = np.full((N, K // G), r, np.float32)
        back = orc.dequantize(*orc.quantize(W, s, G, clip=clip, bits=bits), G).reshape(N, K // G, G)
        errs.append(((back - wp) ** 2).sum(axis=2))
    errs = np.stack(errs)                                    # [ratio][N][groups]
    idx = np.argmax(ratios[:, None, None] == chosen[None], axis=0)
    picked = np.take_along_axis(errs, idx[None], axis=0)[0]
    assert (picked <= errs.min(axis=0) * (1 + 1e-4)).all()
    assert (picked <= errs[0] * (1 + 1e-4)).all()
    assert (idx > 0).mean() > 0.2                            # clipping is chosen for many groups


def test_int3_grid_invariants_and_brute_force():
    """bits = 3: codes and zero points stay in [0, 7], Delta is the fp16 rounding of range / 7,
    the reconstruction error is at most half a step, and on tiny groups the codes minimise the
    squared error over all 8^G code vectors for the oracle's own (Delta, z)."""
    N, K, G = 64, 512, 128
    W, a = _gaussian_case(35, N, K)
    s = orc.channel_scale(a, 0.5)
    codes, zeros, scales = orc.quantize(W, s, G, bits=3)
    assert codes.max() == 7 and zeros.max() <= 7
    wg = (W.astype(np.float64) * s.astype(np.float64)).reshape(N, K // G, G)
    rng_ = (wg.max(axis=2) - wg.min(axis=2)) / 7.0
    assert (np.abs(scales.astype(np.float64) - rng_) <= 2.0**-11 * rng_ * 1.0001).all()
    back = orc.dequantize(codes, zeros, scales, G).reshape(N, K // G, G)
    d = scales.astype(np.float64)[:, :, None]
    assert (np.abs(wg - back) <= (0.5 + 7 * 2.0**-11) * d + 2.0**-22 * np.abs(wg) + 1e-12).all()
    # a grid-aligned group round-trips exactly: levels {-3..4} * 2^-5
    lv = (np.arange(-3, 5) * 2.0**-5).astype(np.float16)
    Wg = np.tile(lv, 16)[None, :]
    c, z, sc = orc.quantize(Wg, np.ones(128, np.float32), 128, bits=3)
    assert z[0, 0] == 3 and float(sc[0, 0]) == 2.0**-5 and np.array_equal(c[0, :8], np.arange(8))
    rng = np.random.default_rng(7)
    vals = (rng.integers(-40, 41, size=(30, 3)) / 64.0).astype(np.float16)
    vals = vals[(vals.max(axis=1) > 0) & (vals.min(axis=1) < 0)]
    c, z, sc = orc.quantize(vals, np.ones(3, np.float32), 3, bits=3)
    for r in range(vals.shape[0]):
        dd, zz = Fraction(float(sc[r, 0])), int(z[r, 0])
        w = [Fraction(float(v)) for v in vals[r]]
        err = lambda qs: sum((wi - (qi - zz) * dd) ** 2 for wi, qi in zip(w, qs))
        best = min(err(qs) for qs in itertools.product(range(8), repeat=3))
        assert err([int(x) for x in c[r]]) <= best * (1 + Fraction(1, 2**20))


# ------------------------------------------------------------------- symmetric grid (Eq. 2)
def test_symmetric_grid_is_eq2():
    """Eq. 2 as printed: Q(w) = Delta * Round(w / Delta), Delta = max|w| / 2^(N-1).  Pinned by a
    grid-aligned group (codes known by hand), by exact zeros, by odd symmetry and by the half-step
    error bound; the one level the 4-bit code cannot hold (+8) saturates."""
    d = 2.0 ** -5
    lv = np.arange(-8, 8)                                            # -8 .. 7: max|w| = 8 d, so Delta = d
    Wg = (np.tile(lv, 8) * d).astype(np.float16)[None, :]
    ones = np.ones(128, np.float32)
    c, z, sc = orc.quantize(Wg, ones, 128, symmetric=True)
    assert z[0, 0] == 8 and float(sc[0, 0]) == d
    assert np.array_equal(c[0, :16], lv + 8)                         # code = Round(w / Delta) + 8
    assert np.array_equal(orc.dequantize(c, z, sc, 128), Wg.astype(np.float64))      # round trip exact
    # mirrored group: max at +8 d: that single element saturates at code 15 (value 7 d), the rest mirror
    c2, z2, sc2 = orc.quantize((-Wg).astype(np.float16), ones, 128, symmetric=True)
    assert float(sc2[0, 0]) == d and c2[0, 0] == 15
    assert np.array_equal(c2[0, 1:16], 16 - c[0, 1:16])
    # random groups: zero stays zero, |error| <= Delta / 2 (+ fp16 rounding of Delta) away from the top level
    W, a = _gaussian_case(41, 64, 512)
    W = W.copy()
    W[:, ::17] = np.float16(0.0)
    s = orc.channel_scale(a, 0.5)
    c, z, sc = orc.quantize(W, s, 128, symmetric=True)
    assert (z == 8).all()
    back = orc.dequantize(c, z, sc, 128)
    assert (back[:, ::17] == 0.0).all()
    wp = W.astype(np.float64) * s.astype(np.float64)
    dd = np.repeat(sc.astype(np.float64), 128, axis=1)
    top_level = wp >= 7.5 * dd
    assert (np.abs(wp - back)[~top_level] <= (0.5 + 8 * 2.0**-11) * dd[~top_level] + 1e-12).all()
    assert (np.abs(wp - back)[top_level] <= (1.0 + 8 * 2.0**-11) * dd[top_level]).all()
    amax = np.abs(wp).reshape(64, 4, 128).max(axis=2)
    assert (np.abs(sc.astype(np.float64) - amax / 8.0) <= 2.0**-11 * amax / 8.0 * 1.0001).all()
    # 3 bits: zero point 4, codes 0 .. 7
    c3, z3, sc3 = orc.quantize(W, s, 128, bits=3, symmetric=True)
    assert (z3 == 4).all() and c3.max() <= 7
