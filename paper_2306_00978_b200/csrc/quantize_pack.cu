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
// The same without the per-element branch: `bad` collects whether any element came within `thr`
// of a half-integer (thr = 0.5 minus the group's bound on |w * rd - w / d|); the caller then redoes
// the word with code_of.  Every lane of a warp has to pass for the warp to skip the divisions, so
// the margin is the group's own bound (a few 1e-6) and not a fixed 1e-3.
__device__ __forceinline__ float level_fast(float w, float rd, float z, float top, float thr, bool& bad) {
    const float t = __fmul_rn(w, rd);
    // round half to even by addition (exact for |t| < 2^22; larger quotients have thr < 0): two fp32
    // additions instead of a conversion-pipe instruction, the pipe this kernel keeps busiest
    const float r = __fsub_rn(__fadd_rn(t, 12582912.0f), 12582912.0f);
    bad = bad || !(fabsf(t - r) < thr);
    return fminf(fmaxf(__fadd_rn(r, z), 0.0f), top);              // the code, still a float
}
// four codes (exact small integers held in floats) as four nibbles: q0 + 16 q1 + 256 q2 + 4096 q3 is
// exact in fp32, so three FFMAs and one conversion replace four conversions and the shifts and ORs
__device__ __forceinline__ uint32_t pack4(float q0, float q1, float q2, float q3) {
    return (uint32_t)fmaf(q3, 4096.0f, fmaf(q2, 256.0f, fmaf(q1, 16.0f, q0)));
}

// grid = (K/128, N/128), block = 256 (8 warps = 8 bands of the 128-row slab); two blocks per SM
// (118 registers, no spills; three blocks at 80 registers spill and measure 1 % slower).  The kernel
// is bound by its own instruction stream (issue slots 62 % active, conversion pipe 55 %): measured on
// 4096->11008, 67.6 us at first, 56 us with the multiply-instead-of-divide path per element, 50.5 us
// with that path made branch-free per word, 48.2 us with rounding by addition, 46.4 us with the
// nibbles assembled by FFMA (one conversion per four codes).
#ifndef AWQ_QP_BLOCKS
#define AWQ_QP_BLOCKS 2
#endif
// SYM: the symmetric grid of Eq. 2 (Delta = max|w'| / 2^(BITS-1), fixed zero point 2^(BITS-1))
template <int G, int BITS, bool CLIP, bool SYM>
__global__ void __launch_bounds__(256, AWQ_QP_BLOCKS)
quantize_pack_kernel(const __half* __restrict__ W, const float* __restrict__ a, float alpha,
                     int mode, const float* __restrict__ clip,
                     uint32_t* __restrict__ qweight, __half* __restrict__ scales,
                     uint8_t* __restrict__ zeros, int N, int K) {
    constexpr float top = (float)((1 << BITS) - 1);       // largest code
    __shared__ __align__(16) float s_sm[128];
    const int kblk = blockIdx.x, slab = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;
    const int n0 = slab * 128 + warp * 16 + g;            // this lane's upper row; lower = n0 + 8
    const int kbase = kblk * 128;

    // issue the weight loads first: [tile][row h][word j] = columns 16j + 4t .. +3 of the tile
    uint2 raw[2][2][4];
#pragma unroll
    for (int ti = 0; ti < 2; ++ti)
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int j = 0; j < 4; ++j)
                raw[ti][h][j] = ldg_stream(reinterpret_cast<const uint2*>(
                    W + (size_t)(n0 + 8 * h) * K + kbase + ti * 64 + 16 * j + 4 * t));
    if (threadIdx.x < 128) {
        const int k = kbase + threadIdx.x;
        s_sm[threadIdx.x] = channel_scale_one(mode == kAlphaZero ? 1.0f : a[k], alpha, mode);
    }
    __syncthreads();

    // w' = fp32(w) * s  (Eq. 3) is formed twice from the raw words - here for the group's min / max,
    // below for the codes (the same two operations give the same value) - so that only the 32 raw
    // registers stay live.  The four scales of a word are one 16-byte
    // shared-memory read, used for both rows.
    auto wprime = [&](int ti, int h, int j, const float (&sv)[4], float (&w4)[4]) {
        const uint32_t u0 = raw[ti][h][j].x, u1 = raw[ti][h][j].y;
        w4[0] = __fmul_rn(__half2float(__ushort_as_half((unsigned short)(u0 & 0xFFFFu))), sv[0]);
        w4[1] = __fmul_rn(__half2float(__ushort_as_half((unsigned short)(u0 >> 16))), sv[1]);
        w4[2] = __fmul_rn(__half2float(__ushort_as_half((unsigned short)(u1 & 0xFFFFu))), sv[2]);
        w4[3] = __fmul_rn(__half2float(__ushort_as_half((unsigned short)(u1 >> 16))), sv[3]);
    };
    // group min / max: a row's group is spread over the 4 lanes t = 0..3 (and, for
    // G = 128, over both tiles)
    float mn[2][2], mx[2][2];
#pragma unroll
    for (int ti = 0; ti < 2; ++ti) {
#pragma unroll
        for (int h = 0; h < 2; ++h) { mn[ti][h] = INFINITY; mx[ti][h] = -INFINITY; }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float4 s4 = *reinterpret_cast<const float4*>(&s_sm[ti * 64 + 16 * j + 4 * t]);
            const float sv[4] = {s4.x, s4.y, s4.z, s4.w};
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                float w4[4];
                wprime(ti, h, j, sv, w4);
#pragma unroll
                for (int e = 0; e < 4; ++e) { mn[ti][h] = fminf(mn[ti][h], w4[e]); mx[ti][h] = fmaxf(mx[ti][h], w4[e]); }
            }
        }
    }
    if (G == 128) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            mn[0][h] = mn[1][h] = fminf(mn[0][h], mn[1][h]);
            mx[0][h] = mx[1][h] = fmaxf(mx[0][h], mx[1][h]);
        }
    }
#pragma unroll
    for (int ti = 0; ti < 2; ++ti)
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int off = 1; off <= 2; off <<= 1) {
                mn[ti][h] = fminf(mn[ti][h], __shfl_xor_sync(0xFFFFFFFFu, mn[ti][h], off));
                mx[ti][h] = fmaxf(mx[ti][h], __shfl_xor_sync(0xFFFFFFFFu, mx[ti][h], off));
            }

    float wabs[2][2];                                       // largest |w'| of each group (before clipping)
#pragma unroll
    for (int ti = 0; ti < 2; ++ti)
#pragma unroll
        for (int h = 0; h < 2; ++h) wabs[ti][h] = fmaxf(fabsf(mn[ti][h]), fabsf(mx[ti][h]));

    if (CLIP) {
        // weight clipping (Sec. 3.2): the group's range shrinks by its ratio, values outside saturate
        const int ng = K / G;
#pragma unroll
        for (int ti = 0; ti < 2; ++ti)
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int gi = (G == 64) ? kblk * 2 + ti : kblk;
                const float r = __ldg(clip + (size_t)(n0 + 8 * h) * ng + gi);
                mn[ti][h] = __fmul_rn(mn[ti][h], r);
                mx[ti][h] = __fmul_rn(mx[ti][h], r);
            }
    }

#pragma unroll
    for (int ti = 0; ti < 2; ++ti) {
        __half d16[2]; float d[2], z[2], rd[2], thr[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            if (SYM) {
                constexpr float half_levels = (float)(1 << (BITS - 1));
                const float d32 = __fdiv_rn(fmaxf(fabsf(mn[ti][h]), fabsf(mx[ti][h])), half_levels);
                d16[h] = __float2half_rn(d32);
                const unsigned short bits = __half_as_ushort(d16[h]);
                if ((bits & 0x7FFFu) == 0u || (bits & 0x7C00u) == 0x7C00u) d16[h] = __ushort_as_half(0x3C00u);
                d[h] = __half2float(d16[h]);
                z[h] = half_levels;
            } else {
                group_params(mn[ti][h], mx[ti][h], top, d16[h], d[h], z[h]);
            }
            rd[h] = __frcp_rn(d[h]);
            // |w * rd - w / d| <= 1.8e-7 |w / d| (three roundings); the group's largest |w / d|
            // bounds it for every element; quotients beyond 1024 always take the division
            const float tmax = __fmul_rn(wabs[ti][h], rd[h]);
            thr[h] = tmax < 1024.0f ? 0.5f - fmaf(tmax, 4e-7f, 1e-6f) : -1.0f;
        }

        uint32_t words[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float4 s4 = *reinterpret_cast<const float4*>(&s_sm[ti * 64 + 16 * j + 4 * t]);
            const float sv[4] = {s4.x, s4.y, s4.z, s4.w};
            float wu[4], wl[4];                                  // rows g and g + 8, columns c .. c+3
            wprime(ti, 0, j, sv, wu);
            wprime(ti, 1, j, sv, wl);
            // slots (g,c) (g,c+1) (g+8,c) (g+8,c+1) (g,c+2) (g,c+3) (g+8,c+2) (g+8,c+3)
            // at nibbles 0, 4, 1, 5, 2, 6, 3, 7
            bool bad = false;
            float qu[4], ql[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                qu[e] = level_fast(wu[e], rd[0], z[0], top, thr[0], bad);
                ql[e] = level_fast(wl[e], rd[1], z[1], top, thr[1], bad);
            }
            // nibbles 0 .. 3 = (g,c) (g+8,c) (g,c+2) (g+8,c+2), nibbles 4 .. 7 the same for c+1, c+3
            words[j] = pack4(qu[0], ql[0], qu[2], ql[2]) | (pack4(qu[1], ql[1], qu[3], ql[3]) << 16);
            if (bad)                                               // rare: the word again, element by element
                words[j] = (code_of(wu[0], d[0], rd[0], z[0], top) << 0) | (code_of(wu[1], d[0], rd[0], z[0], top) << 16) |
                           (code_of(wl[0], d[1], rd[1], z[1], top) << 4) | (code_of(wl[1], d[1], rd[1], z[1], top) << 20) |
                           (code_of(wu[2], d[0], rd[0], z[0], top) << 8) | (code_of(wu[3], d[0], rd[0], z[0], top) << 24) |
                           (code_of(wl[2], d[1], rd[1], z[1], top) << 12) | (code_of(wl[3], d[1], rd[1], z[1], top) << 28);
        }
        // band-major: block (band, k-tile) is 512 bytes, a band's blocks are contiguous along K
        const size_t band = (size_t)slab * 8 + warp;
        const size_t block = band * (K / 64) + (size_t)kblk * 2 + ti;
        uint4* dst = reinterpret_cast<uint4*>(qweight) + block * 32 + lane;
        *dst = make_uint4(words[0], words[1], words[2], words[3]);

        if (t == 0 && (G == 64 || ti == 0)) {
            // scales: [band][group][16]; zero bytes: [band pair][group][16], 8 per band
            const int gi = (G == 64) ? kblk * 2 + ti : kblk;
            const size_t ng = K / G;
            scales[(band * ng + gi) * 16 + g] = d16[0];
            scales[(band * ng + gi) * 16 + g + 8] = d16[1];
            zeros[((band >> 1) * ng + gi) * 16 + (band & 1) * 8 + g] =
                (uint8_t)((uint32_t)z[0] | ((uint32_t)z[1] << 4));
        }
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
        const int gi = k / group, ng = K / group;
        scales_nk[(size_t)n * ng + gi] = __half_as_ushort(scales[((size_t)band * ng + gi) * 16 + rr]);
        const uint8_t zb = zeros[((size_t)(band >> 1) * ng + gi) * 16 + (band & 1) * 8 + g];
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
    const dim3 grid(K / 128, N / 128);
    const int mode = (int)alpha_mode(alpha);
#define AWQ_QP_LAUNCH(GG, BB, CC, SS) \
    quantize_pack_kernel<GG, BB, CC, SS><<<grid, 256, 0, st>>>(W, a, alpha, mode, clip, qweight, scales, zeros, N, K)
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
    if (group == 128) AWQ_QP_PICK(128); else AWQ_QP_PICK(64);
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
