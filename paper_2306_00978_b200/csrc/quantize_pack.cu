// Offline step of the layer: channel scale (Eq. 5), fold into W (Eq. 3), group-wise
// asymmetric 4-bit round-to-nearest (Eq. 2) and the packed tile layout (Sec. 4.2).
//
// HBM-bound: 2 bytes read and ~0.52 bytes written per weight.  One warp owns a band of 16
// rows x 128 columns; lane (g, t) loads rows g and g+8, columns 16j+4t..+3 (j = 0..3) of both
// 64-column tiles (sixteen 8-byte loads in flight per thread; the four lanes of a row read 32
// contiguous bytes), which is exactly the data of the two 16-byte packed pieces it writes, so
// no shared-memory transpose is needed.  Every
// rounding point is an explicit IEEE operation (no contraction); the per-weight division is
// replaced by a multiplication only where that provably rounds to the same integer.
#include <type_traits>

#include "common.cuh"

namespace awq {

__device__ __forceinline__ float channel_scale_one(float a, float alpha, int mode) {
    if (mode == kAlphaZero) return 1.0f;
    const bool ok = isfinite(a) && a > 0.0f;
    if (!ok) return 1.0f;
    if (mode == kAlphaOne) return a;
    if (mode == kAlphaHalf) return __fsqrt_rn(a);
    return (float)pow((double)a, (double)alpha);
}

__global__ void channel_scale_kernel(const float* __restrict__ a, float alpha, int mode,
                                     float* __restrict__ s, int K) {
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k < K) s[k] = channel_scale_one(mode == kAlphaZero ? 1.0f : a[k], alpha, mode);
}

__device__ __forceinline__ uint2 ldg_stream(const uint2* p) {
    uint2 v;
    asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
    return v;
}

// Delta (fp16) and zero point of a group from its min and max; `top` is the largest code
// (15 for 4-bit, 7 for 3-bit grids).
__device__ __forceinline__ void group_params(float mn, float mx, float top, __half& d16, float& d, float& z) {
    const float d32 = __fdiv_rn(__fsub_rn(mx, mn), top);
    d16 = __float2half_rn(d32);
    const unsigned short bits = __half_as_ushort(d16);
    if ((bits & 0x7FFFu) == 0u || (bits & 0x7C00u) == 0x7C00u) d16 = __ushort_as_half(0x3C00u);
    d = __half2float(d16);
    z = fminf(fmaxf(rintf(__fdiv_rn(-mn, d)), 0.0f), top);
}

// q = clamp(rne(w / d) + z, 0, 15) with w / d the IEEE-rounded fp32 quotient.  `rd` = 1 / d
// (rounded).  w * rd is within 2.5e-7 |w / d| of the quotient, so it rounds to the same integer
// unless it lies within 1e-3 of a half-integer (or is large): only then is the division done.
__device__ __forceinline__ uint32_t code_of(float w, float d, float rd, float z, float top) {
    const float t = __fmul_rn(w, rd);
    float r = rintf(t);
    if (!(fabsf(t - r) < 0.499f && fabsf(t) < 1024.0f)) r = rintf(__fdiv_rn(w, d));
    return (uint32_t)fminf(fmaxf(__fadd_rn(r, z), 0.0f), top);
}
// four codes (exact small integers held in floats) as four nibbles: q0 + 16 q1 + 256 q2 + 4096 q3 is
// exact in fp32, so three FFMAs and one conversion replace four conversions and the shifts and ORs
__device__ __forceinline__ uint32_t pack4(float q0, float q1, float q2, float q3) {
    return (uint32_t)fmaf(q3, 4096.0f, fmaf(q2, 256.0f, fmaf(q1, 16.0f, q0)));
}

// grid = (K/128, N/32), block = 128: warp w takes band w % 2 of the block's 32 rows and block w / 2 of
// the 128 columns, a lane 2 rows x 16 columns - exactly the data of the 16-byte packed piece it writes.
// The products w' = w * s stay in registers (32), formed once (64 registers, 32 warps per SM).  For
// G = 128 the two warps that share a group exchange their min / max through shared memory.  The
// division w' / Delta is done only where it can matter: w' * (1 / Delta) rounds to the same integer
// unless it lies within the group's own error bound of a half-integer; that test is taken per
// packed word and row (the largest distance of the word's products from their rounded values), so
// there is no branch per element, and a word that fails is redone element by element with the
// division (code_of).  Rounding is by adding 1.5 * 2^23 (the zero point rides in the subtraction
// that follows), group min / max take three-input min / max instructions, clamping to [0, top] is
// compiled in only for the warps one of whose groups can leave the range, the nibbles of four codes
// are assembled by FFMA and converted once.
// What bounds it (measured on 4096 -> 11008, 113.6 MB): a block loads, computes and stores in
// phases, and the blocks of an SM run in step, so the loads overlap the arithmetic only as far as
// the blocks drift apart.  With 512-thread blocks (two per SM) 45.4 us, whatever the instruction
// count (a form with a third more instructions and half the warps: 45 us; a third fewer
// integer-pipe instructions: 44.3 us); 256-thread blocks 41.6 us, 128-thread blocks 37.9 us, 64-thread
// blocks 41.0 us (the 128 channel scales are then formed per 64 threads).  A persistent form whose
// producer warp keeps six 32 KB tiles in flight by tensor-map copies for sixteen quantizing warps
// measured 58 us: the arithmetic needs the 32 warps.  The same 128-thread blocks made persistent
// (eight per SM, each walking the tiles): 44.0 us - blocks that never leave stay in step.
__device__ __forceinline__ float min3(float a, float b, float c) {
    float d; asm("min.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c)); return d;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d; asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c)); return d;
}
// code (still a float) = clamp(rne(w * rd) + z): zc = 1.5 * 2^23 - z, so that (w * rd + 1.5 * 2^23) - zc
// is the rounded product plus the zero point, exactly (the product enters the sum unrounded, by a
// fused multiply-add: 4 instead of 5 instructions per weight, 38.0 -> 35.7 us on 4096 -> 11008)
// `dev` receives |t - rne(t)|, the distance that decides whether the product may stand for the
// quotient; CLAMP = false where the group's smallest and largest element are known to stay in range.
template <bool CLAMP>
__device__ __forceinline__ float level_fast2(float w, float rd, float zc, float top, float& dev) {
    // one rounding to the integer grid (the product is not rounded first), and the distance of the
    // exact product from that integer, by one fused multiply-add each
    const float u = __fmaf_rn(w, rd, 12582912.0f);
    const float r = __fsub_rn(u, 12582912.0f);
    dev = fabsf(__fmaf_rn(w, rd, -r));
    const float q = __fsub_rn(u, zc);
    return CLAMP ? fminf(fmaxf(q, 0.0f), top) : q;
}

// One warp per band (16 rows) and 64-column block.  A thread block covers one group of columns (two
// groups for G = 64) so that the group's min / max meet in shared memory: 2 bands x 2 blocks up to
// G = 128, 1 band x G / 64 blocks above.  Scales and zero points are stored per 128 columns for
// G > 128 (each group's entry G / 128 times), so that the layer kernels need no variant for them.
template <int G> struct QCfg {
    static constexpr int kBlocks = G < 128 ? 2 : G / 64;            // 64-column blocks per thread block
    static constexpr int kBands = kBlocks <= 4 ? 4 / kBlocks : 1;   // bands per thread block
    static constexpr int kThreads = kBlocks * kBands * 32;
    static constexpr int kStored = G < 128 ? G : 128;               // columns per stored scale / zero point
};

template <int G, int BITS, bool CLIP, bool SYM>
__global__ void __launch_bounds__(QCfg<G>::kThreads, 1024 / QCfg<G>::kThreads)
quantize_pack_tile_kernel(const __half* __restrict__ W, const float* __restrict__ a, float alpha,
                          int mode, const float* __restrict__ clip,
                          uint32_t* __restrict__ qweight, __half* __restrict__ scales,
                          uint8_t* __restrict__ zeros, int N, int K) {
    constexpr float top = (float)((1 << BITS) - 1);       // largest code
    constexpr int kQBands = QCfg<G>::kBands, kQBlocks = QCfg<G>::kBlocks, kQThreads = QCfg<G>::kThreads;
    __shared__ __align__(16) float s_sm[kQBlocks * 64];
    __shared__ float2 s_mm[kQBlocks][kQBands * 16];        // G >= 128: [64-column block][row] (min, max)
    const int kblk = blockIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int bw = warp % kQBands, ti = warp / kQBands;
    const int g = lane >> 2, t = lane & 3;
    const int n0 = (blockIdx.y * kQBands + bw) * 16 + g;   // this lane's upper row; lower = n0 + 8
    const int kbase = kblk * (kQBlocks * 64);

    uint2 raw[2][4];                                       // [row h][word j] = columns 16j + 4t .. +3 of the block
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int j = 0; j < 4; ++j)
            raw[h][j] = ldg_stream(reinterpret_cast<const uint2*>(
                W + (size_t)(n0 + 8 * h) * K + kbase + ti * 64 + 16 * j + 4 * t));
    for (int i = threadIdx.x; i < kQBlocks * 64; i += kQThreads) {
        const int k = kbase + i;
        s_sm[i] = channel_scale_one(mode == kAlphaZero ? 1.0f : a[k], alpha, mode);
    }
    __syncthreads();

    // w' = fp32(w) * s  (Eq. 3), once, and the min / max of this lane's 16 columns of each row
    float wp[2][4][4];
    float mn[2], mx[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) { mn[h] = INFINITY; mx[h] = -INFINITY; }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const float4 s4 = *reinterpret_cast<const float4*>(&s_sm[ti * 64 + 16 * j + 4 * t]);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const float2 f01 = __half22float2(*reinterpret_cast<const __half2*>(&raw[h][j].x));
            const float2 f23 = __half22float2(*reinterpret_cast<const __half2*>(&raw[h][j].y));
            wp[h][j][0] = __fmul_rn(f01.x, s4.x);
            wp[h][j][1] = __fmul_rn(f01.y, s4.y);
            wp[h][j][2] = __fmul_rn(f23.x, s4.z);
            wp[h][j][3] = __fmul_rn(f23.y, s4.w);
            mn[h] = min3(mn[h], wp[h][j][0], wp[h][j][1]);
            mn[h] = min3(mn[h], wp[h][j][2], wp[h][j][3]);
            mx[h] = max3(mx[h], wp[h][j][0], wp[h][j][1]);
            mx[h] = max3(mx[h], wp[h][j][2], wp[h][j][3]);
        }
    }
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int off = 1; off <= 2; off <<= 1) {
            mn[h] = fminf(mn[h], __shfl_xor_sync(0xFFFFFFFFu, mn[h], off));
            mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xFFFFFFFFu, mx[h], off));
        }
    if (G >= 128) {
        // the group spans all 64-column blocks of the thread block: the others' min / max through shared memory
        if (t == 0) {
            s_mm[ti][bw * 16 + g] = make_float2(mn[0], mx[0]);
            s_mm[ti][bw * 16 + g + 8] = make_float2(mn[1], mx[1]);
        }
        __syncthreads();
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int o = 1; o < kQBlocks; ++o) {
                const float2 v = s_mm[(ti + o) % kQBlocks][bw * 16 + g + 8 * h];
                mn[h] = fminf(mn[h], v.x);
                mx[h] = fmaxf(mx[h], v.y);
            }
    }
    float wabs[2];                                          // largest |w'| of each group (before clipping)
#pragma unroll
    for (int h = 0; h < 2; ++h) wabs[h] = fmaxf(fabsf(mn[h]), fabsf(mx[h]));
    const int gi = (G == 64) ? kblk * 2 + ti : kblk;
    const int ng = K / G;
    if (CLIP) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const float r = __ldg(clip + (size_t)(n0 + 8 * h) * ng + gi);
            mn[h] = __fmul_rn(mn[h], r);
            mx[h] = __fmul_rn(mx[h], r);
        }
    }
    __half d16[2]; float d[2], z[2], rd[2], thr[2], zc[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        if (SYM) {
            constexpr float half_levels = (float)(1 << (BITS - 1));
            const float d32 = __fdiv_rn(fmaxf(fabsf(mn[h]), fabsf(mx[h])), half_levels);
            d16[h] = __float2half_rn(d32);
            const unsigned short bits = __half_as_ushort(d16[h]);
            if ((bits & 0x7FFFu) == 0u || (bits & 0x7C00u) == 0x7C00u) d16[h] = __ushort_as_half(0x3C00u);
            d[h] = __half2float(d16[h]);
            z[h] = half_levels;
        } else {
            group_params(mn[h], mx[h], top, d16[h], d[h], z[h]);
        }
        rd[h] = __frcp_rn(d[h]);
        zc[h] = 12582912.0f - z[h];                          // exact: z is a small integer
        // |w * rd - w / d| <= 1.8e-7 |w / d| (three roundings); the group's largest |w / d|
        // bounds it for every element; quotients beyond 1024 always take the division
        const float tmax = __fmul_rn(wabs[h], rd[h]);
        thr[h] = tmax < 1024.0f ? 0.5f - fmaf(tmax, 4e-7f, 1e-6f) : -1.0f;
    }
    // Clamping to [0, top] can only matter where the group's smallest or largest element leaves the
    // range (the level is monotone in w'): rare without clipping - rne(max / Delta) + rne(-min / Delta)
    // exceeds top only when both quotients sit on a tie - so the warp takes the clamped code only if one
    // of its lanes needs it.
    bool need_clamp = CLIP || SYM;
    if (!need_clamp) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            float dummy;
            const float qlo = level_fast2<false>(mn[h], rd[h], zc[h], top, dummy);
            const float qhi = level_fast2<false>(mx[h], rd[h], zc[h], top, dummy);
            need_clamp = need_clamp || !(qlo >= 0.0f && qhi <= top);
        }
        need_clamp = __any_sync(0xFFFFFFFFu, need_clamp);
    }
    uint32_t words[4];
    auto quantize_words = [&](auto clamp_tag) {
        constexpr bool CL = decltype(clamp_tag)::value;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            float qu[4], ql[4], du[4], dl[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                qu[e] = level_fast2<CL>(wp[0][j][e], rd[0], zc[0], top, du[e]);
                ql[e] = level_fast2<CL>(wp[1][j][e], rd[1], zc[1], top, dl[e]);
            }
            // the word's largest distance from the rounded value, per row, decides
            const float dmu = max3(max3(du[0], du[1], du[2]), du[3], 0.0f);
            const float dml = max3(max3(dl[0], dl[1], dl[2]), dl[3], 0.0f);
            const bool bad = !(dmu < thr[0]) || !(dml < thr[1]);
            // nibbles 0 .. 3 = (g,c) (g+8,c) (g,c+2) (g+8,c+2), nibbles 4 .. 7 the same for c+1, c+3
            words[j] = pack4(qu[0], ql[0], qu[2], ql[2]) | (pack4(qu[1], ql[1], qu[3], ql[3]) << 16);
            if (bad)                                               // rare: the word again, element by element
                words[j] = (code_of(wp[0][j][0], d[0], rd[0], z[0], top) << 0) | (code_of(wp[0][j][1], d[0], rd[0], z[0], top) << 16) |
                           (code_of(wp[1][j][0], d[1], rd[1], z[1], top) << 4) | (code_of(wp[1][j][1], d[1], rd[1], z[1], top) << 20) |
                           (code_of(wp[0][j][2], d[0], rd[0], z[0], top) << 8) | (code_of(wp[0][j][3], d[0], rd[0], z[0], top) << 24) |
                           (code_of(wp[1][j][2], d[1], rd[1], z[1], top) << 12) | (code_of(wp[1][j][3], d[1], rd[1], z[1], top) << 28);
        }
    };
    if (need_clamp) quantize_words(std::true_type{}); else quantize_words(std::false_type{});
    // band-major: block (band, k-tile) is 512 bytes, a band's blocks are contiguous along K
    const size_t band = (size_t)blockIdx.y * kQBands + bw;
    const size_t block = band * (K / 64) + (size_t)kblk * kQBlocks + ti;
    uint4* dst = reinterpret_cast<uint4*>(qweight) + block * 32 + lane;
    *dst = make_uint4(words[0], words[1], words[2], words[3]);
    if (t == 0 && (G == 64 || (ti & 1) == 0)) {
        // scales: [band][stored group][16]; zero bytes: [band pair][stored group][16], 8 per band; a
        // stored group is the group itself up to 128 columns, else each of its runs of 128 columns
        const size_t nsg = K / QCfg<G>::kStored;
        const size_t sgi = (G == 64) ? (size_t)gi : (size_t)kblk * (kQBlocks / 2) + ti / 2;
        scales[(band * nsg + sgi) * 16 + g] = d16[0];
        scales[(band * nsg + sgi) * 16 + g + 8] = d16[1];
        zeros[((band >> 1) * nsg + sgi) * 16 + (band & 1) * 8 + g] =
            (uint8_t)((uint32_t)z[0] | ((uint32_t)z[1] << 4));
    }
}

// Weight clipping (Sec. 3.2).  For every group of w' = w * s and every ratio r of the list, the
// group is quantized on [r * min, r * max] and its squared error summed; the first ratio of least
// error is written to clip[n][group].  The choice decides integer codes downstream, so the error
// is defined operation by operation: dequant = (q - z) * Delta (one fp32 multiply), e = dequant -
// w', err += e * e in fp32 over ascending k (no contraction), a NaN error counts as +inf.
// grid = (ceil(K / 2048), N), block = 256: one row's chunk of w' in shared memory; a thread takes
// one (group, ratio) pair at a time and walks the group's elements in order.
constexpr int kClipChunk = 2048;
struct ClipGrid {
    float r[kMaxClipRatios];
    int n;
};

template <int G>
__global__ void __launch_bounds__(256)
clip_search_kernel(const __half* __restrict__ W, const float* __restrict__ a, float alpha, int mode,
                   const ClipGrid ratios, float top, float* __restrict__ clip, int N, int K) {
    constexpr int kGroups = kClipChunk / G;
    __shared__ float w_sm[kClipChunk];
    __shared__ float mn_sm[kGroups], mx_sm[kGroups];
    __shared__ float err_sm[kGroups * kMaxClipRatios];
    const int n = blockIdx.y, k0 = blockIdx.x * kClipChunk;
    const int cols = min(kClipChunk, K - k0);              // a multiple of 128: whole groups
    const int ngr = cols / G;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    for (int i = threadIdx.x; i < cols; i += 256) {
        const float sk = channel_scale_one(mode == kAlphaZero ? 1.0f : a[k0 + i], alpha, mode);
        w_sm[i] = __fmul_rn(__half2float(W[(size_t)n * K + k0 + i]), sk);          // Eq. 3
    }
    __syncthreads();
    for (int gi = warp; gi < ngr; gi += 8) {
        float mn = INFINITY, mx = -INFINITY;
#pragma unroll
        for (int e = 0; e < G / 32; ++e) {
            const float w = w_sm[gi * G + e * 32 + lane];
            mn = fminf(mn, w);
            mx = fmaxf(mx, w);
        }
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) {
            mn = fminf(mn, __shfl_xor_sync(0xFFFFFFFFu, mn, off));
            mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, off));
        }
        if (lane == 0) { mn_sm[gi] = mn; mx_sm[gi] = mx; }
    }
    __syncthreads();
    const int nr = ratios.n;
    for (int item = threadIdx.x; item < ngr * nr; item += 256) {
        const int gi = item / nr, i = item - gi * nr;
        const float r = ratios.r[i];
        __half d16;
        float d, z;
        group_params(__fmul_rn(mn_sm[gi], r), __fmul_rn(mx_sm[gi], r), top, d16, d, z);
        const float* wg = w_sm + gi * G;
        float err = 0.0f;
#pragma unroll 4
        for (int k = 0; k < G; ++k) {
            const float w = wg[k];
            const float q = fminf(fmaxf(__fadd_rn(rintf(__fdiv_rn(w, d)), z), 0.0f), top);
            const float e = __fsub_rn(__fmul_rn(__fsub_rn(q, z), d), w);
            err = __fadd_rn(err, __fmul_rn(e, e));
        }
        err_sm[gi * kMaxClipRatios + i] = (err != err) ? INFINITY : err;
    }
    __syncthreads();
    if ((int)threadIdx.x < ngr) {
        const float* e = err_sm + threadIdx.x * kMaxClipRatios;
        int best = 0;
        for (int i = 1; i < nr; ++i)
            if (e[i] < e[best]) best = i;
        clip[(size_t)n * (K / G) + k0 / G + threadIdx.x] = ratios.r[best];
    }
}

// One thread per (row, 8 columns): expands the packed arrays (test / debug path).
__global__ void unpack_kernel(const uint32_t* __restrict__ qweight, const __half* __restrict__ scales,
                              const uint8_t* __restrict__ zeros, int N, int K, int group,
                              uint8_t* __restrict__ codes, uint16_t* __restrict__ scales_nk,
                              uint8_t* __restrict__ zeros_nk) {
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t total = (size_t)N * K;
    if (idx >= total) return;
    const int n = (int)(idx / K), k = (int)(idx % K);
    const int band = n / 16, rr = n % 16, g = rr % 8, h = rr / 8;
    const size_t block = (size_t)band * (K / 64) + k / 64;
    const int c = k % 64;
    const int j = c / 16, t = (c % 16) / 4, i = c % 4;
    const uint32_t w = qweight[block * 128 + (g * 4 + t) * 4 + j];
    const int slot = (i / 2) * 4 + h * 2 + (i % 2);
    const int nib = (slot % 2) * 4 + slot / 2;
    codes[idx] = (uint8_t)((w >> (4 * nib)) & 0xFu);
    if (k % group == 0) {
        // the group's first stored entry (groups above 128 columns are stored once per 128 columns)
        const int gi = k / group, ng = K / group;
        const int stored = group < 128 ? group : 128;
        const size_t sgi = k / stored, nsg = K / stored;
        scales_nk[(size_t)n * ng + gi] = __half_as_ushort(scales[((size_t)band * nsg + sgi) * 16 + rr]);
        const uint8_t zb = zeros[((size_t)(band >> 1) * nsg + sgi) * 16 + (band & 1) * 8 + g];
        zeros_nk[(size_t)n * ng + gi] = (uint8_t)((zb >> (4 * h)) & 0xFu);
    }
}

cudaError_t launch_channel_scale(const float* a, float alpha, float* s, int K, cudaStream_t st) {
    channel_scale_kernel<<<(K + 255) / 256, 256, 0, st>>>(a, alpha, (int)alpha_mode(alpha), s, K);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_quantize_pack(const __half* W, const float* a, float alpha, int group, int bits,
                                 bool symmetric, const float* clip, uint32_t* qweight, __half* scales, uint8_t* zeros,
                                 int N, int K, cudaStream_t st) {
    const int mode = (int)alpha_mode(alpha);
#define AWQ_QP_LAUNCH(GG, BB, CC, SS)                                                                           \
    quantize_pack_tile_kernel<GG, BB, CC, SS><<<dim3(K / (QCfg<GG>::kBlocks * 64), N / (16 * QCfg<GG>::kBands)), \
                                                QCfg<GG>::kThreads, 0, st>>>(W, a, alpha, mode, clip, qweight, scales, zeros, N, K)
#define AWQ_QP_PICK2(GG, SS)                                             \
    do {                                                                 \
        if (bits == 4 && !clip) AWQ_QP_LAUNCH(GG, 4, false, SS);         \
        else if (bits == 4) AWQ_QP_LAUNCH(GG, 4, true, SS);              \
        else if (!clip) AWQ_QP_LAUNCH(GG, 3, false, SS);                 \
        else AWQ_QP_LAUNCH(GG, 3, true, SS);                             \
    } while (0)
#define AWQ_QP_PICK(GG)                                                  \
    do {                                                                 \
        if (symmetric) AWQ_QP_PICK2(GG, true); else AWQ_QP_PICK2(GG, false); \
    } while (0)
    switch (group) {
        case 64: AWQ_QP_PICK(64); break;
        case 128: AWQ_QP_PICK(128); break;
        case 256: AWQ_QP_PICK(256); break;
        case 512: AWQ_QP_PICK(512); break;
        default: AWQ_QP_PICK(1024); break;
    }
#undef AWQ_QP_PICK
#undef AWQ_QP_PICK2
#undef AWQ_QP_LAUNCH
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_clip_search(const __half* W, const float* a, float alpha, int group, int bits,
                               const float* ratios, int n_ratios, float* clip, int N, int K,
                               cudaStream_t st) {
    ClipGrid grid_r;
    grid_r.n = n_ratios;
    for (int i = 0; i < kMaxClipRatios; ++i) grid_r.r[i] = i < n_ratios ? ratios[i] : 1.0f;
    const dim3 grid((K + kClipChunk - 1) / kClipChunk, N);
    const int mode = (int)alpha_mode(alpha);
    const float top = (float)((1 << bits) - 1);
    if (group == 128)
        clip_search_kernel<128><<<grid, 256, 0, st>>>(W, a, alpha, mode, grid_r, top, clip, N, K);
    else
        clip_search_kernel<64><<<grid, 256, 0, st>>>(W, a, alpha, mode, grid_r, top, clip, N, K);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_unpack(const uint32_t* qweight, const __half* scales, const uint8_t* zeros,
                          int N, int K, int group, uint8_t* codes, uint16_t* scales_nk,
                          uint8_t* zeros_nk, cudaStream_t st) {
    const size_t total = (size_t)N * K;
    unpack_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(qweight, scales, zeros, N, K, group,
                                                                    codes, scales_nk, zeros_nk);
    count_launch();
    return cudaGetLastError();
}

// ---- 3-bit storage: four nibble words of a piece (codes < 8) <-> three words.  One thread per piece.
__global__ void pack_int3_kernel(const uint4* __restrict__ q4, uint32_t* __restrict__ q3, size_t pieces) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= pieces) return;
    const uint4 w = q4[i];
    q3[3 * i + 0] = (w.x & 0x77777777u) | ((w.w & 0x11111111u) << 3);
    q3[3 * i + 1] = (w.y & 0x77777777u) | (((w.w >> 1) & 0x11111111u) << 3);
    q3[3 * i + 2] = (w.z & 0x77777777u) | (((w.w >> 2) & 0x11111111u) << 3);
}
__global__ void unpack_int3_kernel(const uint32_t* __restrict__ q3, uint4* __restrict__ q4, size_t pieces) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= pieces) return;
    const uint32_t u0 = q3[3 * i], u1 = q3[3 * i + 1], u2 = q3[3 * i + 2];
    uint4 w;
    w.x = u0 & 0x77777777u;
    w.y = u1 & 0x77777777u;
    w.z = u2 & 0x77777777u;
    w.w = ((u0 >> 3) & 0x11111111u) | ((u1 >> 2) & 0x22222222u) | ((u2 >> 1) & 0x44444444u);
    q4[i] = w;
}

cudaError_t launch_pack_int3(const void* q4, void* q3, int N, int K, cudaStream_t st) {
    const size_t pieces = (size_t)N * K / 32;
    pack_int3_kernel<<<(unsigned)((pieces + 255) / 256), 256, 0, st>>>(
        reinterpret_cast<const uint4*>(q4), reinterpret_cast<uint32_t*>(q3), pieces);
    count_launch();
    return cudaGetLastError();
}
cudaError_t launch_unpack_int3(const void* q3, void* q4, int N, int K, cudaStream_t st) {
    const size_t pieces = (size_t)N * K / 32;
    unpack_int3_kernel<<<(unsigned)((pieces + 255) / 256), 256, 0, st>>>(
        reinterpret_cast<const uint32_t*>(q3), reinterpret_cast<uint4*>(q4), pieces);
    count_launch();
    return cudaGetLastError();
}

}  // namespace awq
