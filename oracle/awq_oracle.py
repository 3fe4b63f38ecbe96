"""CPU oracle for the W4A16 group-wise linear layer.  TEST INFRASTRUCTURE ONLY.

Nothing in the product path may import this module: it exists so that the CUDA kernels
can be checked against a plain, slow, independent statement of what they must compute.
It shares no code with the CUDA path (no headers, tables, helpers or constants); it is
written in numpy, every fp32 step being a single IEEE-754 binary32 operation (numpy
ufuncs on float32 arrays do not contract into fused multiply-adds) and the linear layer
being evaluated in fp64.

What is computed, and where it comes from
-----------------------------------------
* channel_scale      s = s_X ** alpha, per input channel                     (Eq. 5)
* quantize           w' = w * s folded into the weight (Eq. 3, Eq. 4), then the
                     group-wise round-to-nearest grid Delta * Round(w'/Delta)   (Eq. 2),
                     in the asymmetric min/max form with an integer zero point in
                     [0, 15] and Delta stored in fp16 (Sec. 3.2 keeps Delta and the
                     activations in half precision).
* search_clip        weight clipping (Sec. 3.2): per group, the range ratio of a given list that
                     minimizes the squared quantization error of the group.
* pack_* / unpack_*  eight 4-bit codes per 32-bit word in the order
                     w{0,2,4,6,1,3,5,7} (Sec. 4.2, SIMD-aware weight packing), inside
                     512-byte blocks (16 rows x 64 columns) whose 16-byte pieces are ordered
                     for a warp-wide register fragment; see `qweight_location`.
* dequantize         (q - z) * Delta, exact in fp64.
* linear             y = x . dequant(Wq)^T in fp64 (Sec. 4.2, on-the-fly weight
                     dequantization followed by the matrix product; here unfused).
* search_alpha       the scale search of Sec. 3.2: L(s) = || Q(W diag(s)) (diag(s)^-1 X) - W X ||
                     (Eq. 4) evaluated for s = s_X ** alpha over a given list of alpha (Eq. 5),
                     and the first alpha of least loss.

Readings adopted where the paper is silent
------------------------------------------
The paper's Eq. 2 is the symmetric abs-max grid.  The deployed form asked for here is
asymmetric: Delta = (max - min) / 15, z = Round(-min / Delta) clamped to [0, 15],
q = clamp(Round(w'/Delta) + z, 0, 15).  Round is round-half-to-even in fp32; Delta is
rounded to fp16 *before* it is used, so that quantize and dequantize use the same grid; the
group's raw min and max are used (the range is not widened to contain 0); a degenerate
group (Delta rounds to 0 or is not finite) takes Delta = 1.  w * s stays in fp32.
The search's norm is not named in the paper: the mean of the squared differences is used (any
monotone function of the Frobenius norm has the same minimizer); diag(s)^-1 X is rounded to fp16
once, because that is what the layer is given; the grid of alpha is an argument (Sec. 3.2 searches
20 grid points over [0, 1] and does not say whether 1 is one of them).
Weight clipping is one sentence in the paper (the appendix it may have been detailed in is not
part of the text): the reading here shrinks a group's [min, max] by a common ratio taken from a
caller-given list, measures the error in the scaled weight space w' = w * s (the tensor that is
actually quantized), unweighted, in fp32 in a fixed order so that the choice is reproducible bit
for bit, and keeps the first best ratio.  INT3 (the paper's INT3-g128 tables) is the same
quantizer on 8 levels (Delta = (max - min) / 7, z and q in [0, 7]); how the paper's kernels would
store 3-bit codes is not described, here they occupy the 4-bit fields of the INT4 layout.
The symmetric grid is Eq. 2 as printed; since Round(w / Delta) then spans 2**bits + 1 values
(-2**(bits-1) .. +2**(bits-1)), the single level +2**(bits-1) - reached only by a group's largest
positive element - saturates at the top code.
Parity for these asymmetric details is unpinned by the paper (it prints no worked numeric
example of Q); they are pinned by closed-form invariants, grid-aligned round trips and
brute-force enumeration in tests/test_oracle_pins.py.
"""
from __future__ import annotations

import numpy as np

BAND_ROWS = 16           # output channels per band (one packed block holds a band x 64 columns)
TILE_COLS = 64           # input channels per packed block
WORDS_PER_BLOCK = BAND_ROWS * TILE_COLS // 8
# Nibble position (bits 4p..4p+3) of element slot e inside a word: slot order read from
# the low nibble upwards is {0,2,4,6,1,3,5,7} (Sec. 4.2).
NIBBLE_OF_SLOT = (0, 4, 1, 5, 2, 6, 3, 7)


# --------------------------------------------------------------------------- Eq. 5
def channel_scale(act_mean_abs, alpha: float) -> np.ndarray:
    """s_k = a_k ** alpha as fp32 [K]  (Eq. 5: s = s_X^alpha).

    alpha = 0 means "do not scale" (s = 1).  A statistic that is not finite or not
    positive gives s_k = 1.  alpha = 1 is the identity and alpha = 0.5 the correctly
    rounded fp32 square root; any other alpha is the fp64 power rounded once to fp32.
    """
    alpha = float(alpha)
    if not (0.0 <= alpha <= 1.0):
        raise ValueError("alpha must lie in [0, 1]")
    a = np.asarray(act_mean_abs, dtype=np.float32)
    if alpha == 0.0:
        return np.ones(a.shape, dtype=np.float32)
    ok = np.isfinite(a) & (a > 0)
    safe = np.where(ok, a, np.float32(1.0)).astype(np.float32)
    if alpha == 1.0:
        s = safe
    elif alpha == 0.5:
        s = np.sqrt(safe, dtype=np.float32)
    else:
        s = np.power(safe.astype(np.float64), alpha).astype(np.float32)
    return np.where(ok, s, np.float32(1.0)).astype(np.float32)


# --------------------------------------------------------------------- Eq. 2 - Eq. 4
def quantize(W, s, group: int, clip=None, bits: int = 4, symmetric: bool = False):
    """Group-wise round-to-nearest of W * diag(s) on a grid of 2**bits levels: asymmetric (min / max
    with a zero point), or symmetric (Eq. 2 as printed: Delta = max|w'| / 2**(bits-1), no offset;
    stored with the fixed zero point 2**(bits-1), the level +2**(bits-1) saturating at the top code).

    W fp16 [N][K]; s fp32 [K]; groups are `group` consecutive input channels of one
    output row.  clip: None, or fp32 [N][K/group] of range ratios (Sec. 3.2, weight clipping):
    a group's range becomes [r * min, r * max] (one fp32 multiply each) and values outside it
    saturate at codes 0 and 2**bits - 1.  bits is 4 (INT4) or 3 (INT3).
    Returns (codes u8 [N][K], zeros u8 [N][K/group], scales fp16 [N][K/group]).
    """
    W = np.asarray(W)
    assert W.dtype == np.float16 and W.ndim == 2
    N, K = W.shape
    assert K % group == 0
    assert bits in (3, 4)
    ng = K // group
    s = np.asarray(s, dtype=np.float32)
    assert s.shape == (K,)
    if clip is not None:
        clip = np.asarray(clip)
        assert clip.dtype == np.float32 and clip.shape == (N, ng)

    codes = np.empty((N, K), dtype=np.uint8)
    zeros = np.empty((N, ng), dtype=np.uint8)
    scales = np.empty((N, ng), dtype=np.float16)
    rows = max(1, (1 << 23) // K)                       # bound the fp32 temporaries
    f15, f0 = np.float32((1 << bits) - 1), np.float32(0.0)    # top code: 15 (INT4) or 7 (INT3)
    for r0 in range(0, N, rows):
        r1 = min(N, r0 + rows)
        wp = W[r0:r1].astype(np.float32) * s[None, :]   # Eq. 3: w * s, one fp32 multiply
        wg = wp.reshape(r1 - r0, ng, group)
        mn = wg.min(axis=2)
        mx = wg.max(axis=2)
        if clip is not None:
            mn = mn * clip[r0:r1]
            mx = mx * clip[r0:r1]
        if symmetric:
            half = np.float32(1 << (bits - 1))
            amax = np.maximum(np.abs(mn), np.abs(mx))
            with np.errstate(over="ignore", invalid="ignore", divide="ignore"):
                d16 = (amax / half).astype(np.float16)               # Eq. 2: Delta = max|w| / 2^(N-1)
                bad = ~np.isfinite(d16) | (d16 == 0)
                d16 = np.where(bad, np.float16(1.0), d16).astype(np.float16)
                d = d16.astype(np.float32)
                z = np.full_like(d, half)
                q = np.clip(np.rint(wg / d[:, :, None]) + half, f0, f15)   # Eq. 2: Round(w / Delta)
            codes[r0:r1] = q.reshape(r1 - r0, K).astype(np.uint8)
            zeros[r0:r1] = z.astype(np.uint8)
            scales[r0:r1] = d16
            continue
        with np.errstate(over="ignore", invalid="ignore", divide="ignore"):
            d16 = ((mx - mn) / f15).astype(np.float16)  # Delta, stored in fp16
            bad = ~np.isfinite(d16) | (d16 == 0)
            d16 = np.where(bad, np.float16(1.0), d16).astype(np.float16)
            d = d16.astype(np.float32)
            z = np.clip(np.rint((-mn) / d), f0, f15)    # zero point, half-to-even
            q = np.rint(wg / d[:, :, None]) + z[:, :, None]   # Eq. 2: Round(w / Delta)
            q = np.clip(q, f0, f15)
        codes[r0:r1] = q.reshape(r1 - r0, K).astype(np.uint8)
        zeros[r0:r1] = z.astype(np.uint8)
        scales[r0:r1] = d16
    return codes, zeros, scales


# ------------------------------------------------------------------- packed layout
def qweight_location(n: int, k: int, K: int):
    """(word index, nibble position) of code (n, k) in the packed weight array.

    Rows are taken in bands of 16; everything a band needs is contiguous along K.  Block
    (band, k // 64) is 512 bytes (128 words) at word (band * (K // 64) + k // 64) * 128.  A
    block is 32 pieces of 16 bytes; piece (g, t), g = 0..7, t = 0..3, holds rows g and g+8 of
    the band.  Word j of a piece holds columns 16j+4t .. 16j+4t+3 of the block for both rows
    (so the four pieces of a row pair interleave along K in runs of four columns), in the
    slot order (g,c0) (g,c1) (g+8,c0) (g+8,c1) (g,c2) (g,c3) (g+8,c2) (g+8,c3), and slot e
    sits at nibble NIBBLE_OF_SLOT[e].
    """
    band, rr = n // BAND_ROWS, n % BAND_ROWS
    block = band * (K // TILE_COLS) + k // TILE_COLS
    c = k % TILE_COLS
    g, h = rr % 8, rr // 8
    j, t, i = c // 16, (c % 16) // 4, c % 4
    word = block * WORDS_PER_BLOCK + (g * 4 + t) * 4 + j
    slot = (i // 2) * 4 + h * 2 + (i % 2)
    return word, NIBBLE_OF_SLOT[slot]


def zeros_location(n: int, gi: int, ng: int):
    """(byte index, nibble position) of the zero point of row n, group gi (ng groups per row).

    Two bands (32 rows) share a 16-byte block per group: [N/32][ng][16].  Bytes 0-7 belong to
    the even band, 8-15 to the odd band; byte g of a band holds the zero points of its rows g
    (low nibble) and g+8 (high nibble).
    """
    band, rr = n // BAND_ROWS, n % BAND_ROWS
    return ((band // 2) * ng + gi) * 16 + (band % 2) * 8 + rr % 8, rr // 8


def scales_location(n: int, gi: int, ng: int) -> int:
    """Element index of Delta of row n, group gi: fp16 [N/16][ng][16] (band, group, row)."""
    return ((n // BAND_ROWS) * ng + gi) * BAND_ROWS + n % BAND_ROWS


def pack_qweight(codes) -> np.ndarray:
    """codes u8 [N][K] -> uint32 [N*K/8] in the layout of `qweight_location`."""
    codes = np.asarray(codes, dtype=np.uint8)
    N, K = codes.shape
    assert N % BAND_ROWS == 0 and K % TILE_COLS == 0
    # axes: band, h, g, C, j, t, ihi, ilo      (column in block = 16 j + 4 t + 2 ihi + ilo)
    a = codes.reshape(N // 16, 2, 8, K // 64, 4, 4, 2, 2)
    # -> band, C, g, t, j, ihi, h, ilo   (the last three are the slot bits, high to low)
    a = a.transpose(0, 3, 2, 5, 4, 6, 1, 7).reshape(-1, 8).astype(np.uint32)
    words = np.zeros(a.shape[0], dtype=np.uint32)
    for slot in range(8):
        words |= a[:, slot] << np.uint32(4 * NIBBLE_OF_SLOT[slot])
    return words


def unpack_qweight(words, N: int, K: int) -> np.ndarray:
    """Inverse of pack_qweight."""
    words = np.asarray(words, dtype=np.uint32).reshape(-1)
    assert words.size == N * K // 8
    a = np.empty((words.size, 8), dtype=np.uint8)
    for slot in range(8):
        a[:, slot] = (words >> np.uint32(4 * NIBBLE_OF_SLOT[slot])) & np.uint32(0xF)
    a = a.reshape(N // 16, K // 64, 8, 4, 4, 2, 2, 2)   # band, C, g, t, j, ihi, h, ilo
    return a.transpose(0, 6, 2, 1, 4, 3, 5, 7).reshape(N, K)


# ------------------------------------------------------------- 3-bit storage (INT3-g128 setting)
def int3_location(n: int, k: int, K: int):
    """Where the three bits of code (n, k) sit in the 3-bit array: [(word index, bit), ...] for
    bit 0, 1, 2 of the code.

    The paper's INT3 tables need codes of 3 bits; it does not describe a storage, this is the
    layout used.  Blocks, bands and pieces are those of the 4-bit layout, but a piece is three
    words instead of four: block (band, k // 64) is 96 words at (band * (K // 64) + k // 64) * 96,
    piece (g, t) at word 3 * (4 g + t) of it.  With (j, p) the word and nibble that
    `qweight_location` gives inside the piece: for j < 3 the code keeps its place, bits
    4p .. 4p+2 of word j; for j = 3 (columns 48 .. 63 of the block) bit b of the code sits in the
    spare top bit of nibble p of word b, i.e. bit 4p+3 of word b.
    """
    word4, p = qweight_location(n, k, K)
    block, in_block = divmod(word4, WORDS_PER_BLOCK)
    piece, j = divmod(in_block, 4)
    base = block * 96 + piece * 3
    if j < 3:
        return [(base + j, 4 * p + b) for b in range(3)]
    return [(base + b, 4 * p + 3) for b in range(3)]


def pack_qweight_int3(codes) -> np.ndarray:
    """codes u8 [N][K], all < 8 -> uint32 [N*K*3/32] in the layout of `int3_location`: of the four
    nibble words w0 .. w3 of every 16-byte piece of the 4-bit layout, word b (b = 0, 1, 2) takes
    bit b of w3's nibbles into the spare top bits of its own."""
    codes = np.asarray(codes, dtype=np.uint8)
    assert codes.max(initial=0) < 8
    w = pack_qweight(codes).reshape(-1, 4)
    out = np.empty((w.shape[0], 3), dtype=np.uint32)
    ones = np.uint32(0x11111111)
    for b in range(3):
        out[:, b] = w[:, b] | (((w[:, 3] >> np.uint32(b)) & ones) << np.uint32(3))
    return out.reshape(-1)


def unpack_qweight_int3(words3, N: int, K: int) -> np.ndarray:
    """Inverse of pack_qweight_int3."""
    u = np.asarray(words3, dtype=np.uint32).reshape(-1, 3)
    assert u.size == N * K * 3 // 32
    w = np.empty((u.shape[0], 4), dtype=np.uint32)
    ones, low = np.uint32(0x11111111), np.uint32(0x77777777)
    w[:, 3] = 0
    for b in range(3):
        w[:, b] = u[:, b] & low
        w[:, 3] |= ((u[:, b] >> np.uint32(3)) & ones) << np.uint32(b)
    return unpack_qweight(w.reshape(-1), N, K)


def stored_groups(per_group, group: int) -> np.ndarray:
    """[N][K/group] -> [N][K/min(group, 128)]: the packed scale and zero-point arrays hold one entry
    per group up to 128 input channels and one per 128 input channels above (each group's entry
    group / 128 times), so that a kernel never meets more than two 64-column blocks per entry.  The
    paper does not say how other group sizes are stored; this is a choice of the layout."""
    a = np.asarray(per_group)
    return np.repeat(a, group // 128, axis=1) if group > 128 else a


def pack_zeros(zeros) -> np.ndarray:
    """zeros u8 [N][ng] -> u8 [N/32][ng][16] in the layout of `zeros_location`."""
    zeros = np.asarray(zeros, dtype=np.uint8)
    N, ng = zeros.shape
    assert N % 32 == 0
    a = zeros.reshape(N // 32, 2, 2, 8, ng)             # pair, band-in-pair, h, g, gi
    a = a.transpose(0, 4, 1, 3, 2)                      # pair, gi, band-in-pair, g, h
    return (a[..., 0] | (a[..., 1] << 4)).reshape(N // 32, ng, 16).astype(np.uint8)


def unpack_zeros(packed, N: int, ng: int) -> np.ndarray:
    p = np.asarray(packed, dtype=np.uint8).reshape(N // 32, ng, 2, 8)    # pair, gi, band-in-pair, g
    a = np.stack([p & 0xF, p >> 4], axis=-1)            # pair, gi, band-in-pair, g, h
    return a.transpose(0, 2, 4, 3, 1).reshape(N, ng).copy()


def pack_scales(scales) -> np.ndarray:
    """scales fp16 [N][ng] -> fp16 [N/16][ng][16] (band, group, row)."""
    sc = np.asarray(scales, dtype=np.float16)
    N, ng = sc.shape
    return np.ascontiguousarray(sc.reshape(N // 16, 16, ng).transpose(0, 2, 1))


def unpack_scales(packed, N: int, ng: int) -> np.ndarray:
    p = np.asarray(packed, dtype=np.float16).reshape(N // 16, ng, 16)
    return np.ascontiguousarray(p.transpose(0, 2, 1).reshape(N, ng))


def search_clip(W, s, group: int, ratios, bits: int = 4) -> np.ndarray:
    """Weight clipping (Sec. 3.2: clipping that minimizes the squared error of quantization).

    For every group and every ratio r of `ratios` the group of w' = W * diag(s) is quantized on
    the range [r * min, r * max] and the squared error of the group is summed,
        err(r) = sum over k ascending of (dequant(q_k) - w'_k) ** 2,
    every step a single fp32 operation: dequant = (q - z) * Delta (one multiply), the difference,
    its square, and the running sum.  The first ratio of least error is taken (a NaN error counts
    as +inf).  Returns fp32 [N][K/group], each entry one of `ratios`.
    """
    W = np.asarray(W)
    assert W.dtype == np.float16 and W.ndim == 2 and bits in (3, 4)
    N, K = W.shape
    ng = K // group
    s = np.asarray(s, dtype=np.float32)
    ratios = np.asarray(ratios, dtype=np.float32)
    top, f0 = np.float32((1 << bits) - 1), np.float32(0.0)
    wg = (W.astype(np.float32) * s[None, :]).reshape(N, ng, group)
    mn0 = wg.min(axis=2)
    mx0 = wg.max(axis=2)
    best_err = np.full((N, ng), np.inf, dtype=np.float32)
    best = np.zeros((N, ng), dtype=np.int64)
    for i, r in enumerate(ratios):
        mn = mn0 * r
        mx = mx0 * r
        with np.errstate(over="ignore", invalid="ignore", divide="ignore"):
            d16 = ((mx - mn) / top).astype(np.float16)
            bad = ~np.isfinite(d16) | (d16 == 0)
            d = np.where(bad, np.float16(1.0), d16).astype(np.float16).astype(np.float32)
            z = np.clip(np.rint((-mn) / d), f0, top)
            err = np.zeros((N, ng), dtype=np.float32)
            for k in range(group):                      # ascending k, fp32 running sum
                w = wg[:, :, k]
                q = np.clip(np.rint(w / d) + z, f0, top)
                e = (q - z) * d - w
                err = err + e * e
        err = np.where(np.isnan(err), np.float32(np.inf), err)
        if i == 0:
            best_err = err
        else:
            better = err < best_err                     # strict: the first of equal errors stays
            best = np.where(better, i, best)
            best_err = np.where(better, err, best_err)
    return ratios[best].astype(np.float32)


def quantize_pack(W, act_mean_abs, alpha: float, group: int, clip=None, bits: int = 4, symmetric: bool = False):
    """The whole offline step: returns (qweight u32, scales fp16 [N/16][ng][16], zeros u8 [N/32][ng][16]),
    ng = K / min(group, 128) stored entries per row (stored_groups).  3-bit codes (bits = 3) are stored
    in the same 4-bit fields."""
    K = W.shape[1]
    a = np.ones(K, np.float32) if act_mean_abs is None else act_mean_abs
    codes, zeros, scales = quantize(W, channel_scale(a, alpha), group, clip=clip, bits=bits, symmetric=symmetric)
    return pack_qweight(codes), pack_scales(stored_groups(scales, group)), pack_zeros(stored_groups(zeros, group))


# ----------------------------------------------------------------- dequantize, multiply
def dequantize(codes, zeros, scales, group: int) -> np.ndarray:
    """Wdq[n][k] = (q - z) * Delta in fp64 (exact: a 5-bit integer times an fp16 value)."""
    N, K = codes.shape
    ng = K // group
    q = codes.reshape(N, ng, group).astype(np.float64)
    z = np.asarray(zeros, dtype=np.float64)[:, :, None]
    d = np.asarray(scales, dtype=np.float16).astype(np.float64)[:, :, None]
    return ((q - z) * d).reshape(N, K)


def linear(x, Wdq) -> np.ndarray:
    """y[m][n] = sum_k x[m][k] * Wdq[n][k] in fp64; x is fp16 and already divided by s."""
    x = np.asarray(x)
    assert x.dtype == np.float16
    return x.astype(np.float64) @ np.asarray(Wdq, dtype=np.float64).T


def linear_from_packed(x, qweight, scales_gn, zeros_packed, N: int, K: int, group: int,
                       rows=None) -> np.ndarray:
    """Dequantize-then-multiply starting from the packed arrays (optionally only the
    output channels listed in `rows`, for sampled checks at sizes where the full product
    is too slow)."""
    nsg, rep = K // min(group, 128), max(group // 128, 1)       # stored entries per row; see stored_groups
    codes = unpack_qweight(qweight, N, K)
    zeros = unpack_zeros(zeros_packed, N, nsg)[:, ::rep]
    scales = unpack_scales(scales_gn, N, nsg)[:, ::rep]
    if rows is not None:
        codes, zeros, scales = codes[rows], zeros[rows], scales[rows]
    return linear(x, dequantize(codes, zeros, scales, group))


def search_alpha(W, act_mean_abs, X, group: int, alphas):
    """Eq. 4 and Eq. 5: for every alpha, s = s_X ** alpha, quantize W diag(s), and measure the
    layer-output error on the calibration activations X (fp16 [M][K]) against the fp16 layer:
        loss(alpha) = mean over (m, n) of ( sum_k dequant(Q(W s))[n][k] * fp16(X[m][k] / s[k])
                                            - sum_k W[n][k] * X[m][k] ) ** 2,        all in fp64.
    Returns (losses fp64 [len(alphas)], index of the first least loss)."""
    W = np.asarray(W)
    X = np.asarray(X)
    assert W.dtype == np.float16 and X.dtype == np.float16
    y_ref = X.astype(np.float64) @ W.astype(np.float64).T
    losses = np.zeros(len(alphas), dtype=np.float64)
    for i, alpha in enumerate(alphas):
        s = channel_scale(act_mean_abs, float(np.float32(alpha)))      # alpha is an fp32 argument
        codes, zeros, scales = quantize(W, s, group)
        xs = (X.astype(np.float32) / s[None, :]).astype(np.float16)
        y = linear(xs, dequantize(codes, zeros, scales, group))
        losses[i] = np.mean((y - y_ref) ** 2)
    return losses, int(np.argmin(losses))


def parity_errors(y, y_ref):
    """(relative L2 error, max abs error / max |y_ref|) of y against the fp64 reference."""
    y = np.asarray(y, dtype=np.float64)
    y_ref = np.asarray(y_ref, dtype=np.float64)
    den = np.linalg.norm(y_ref)
    amax = np.abs(y_ref).max() if y_ref.size else 0.0
    rel = np.linalg.norm(y - y_ref) / den if den > 0 else float(np.linalg.norm(y - y_ref))
    mx = np.abs(y - y_ref).max() / amax if amax > 0 else float(np.abs(y - y_ref).max(initial=0.0))
    return float(rel), float(mx)
