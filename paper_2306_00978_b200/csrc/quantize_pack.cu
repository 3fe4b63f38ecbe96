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

// Delta (fp16) and zero point of a group from its min and max.
__device__ __forceinline__ void group_params(float mn, float mx, __half& d16, float& d, float& z) {
    const float d32 = __fdiv_rn(__fsub_rn(mx, mn), 15.0f);
    d16 = __float2half_rn(d32);
    const unsigned short bits = __half_as_ushort(d16);
    if ((bits & 0x7FFFu) == 0u || (bits & 0x7C00u) == 0x7C00u) d16 = __ushort_as_half(0x3C00u);
    d = __half2float(d16);
    z = fminf(fmaxf(rintf(__fdiv_rn(-mn, d)), 0.0f), 15.0f);
}

// q = clamp(rne(w / d) + z, 0, 15) with w / d the IEEE-rounded fp32 quotient.  `rd` = 1 / d
// (rounded).  w * rd is within 2.5e-7 |w / d| of the quotient, so it rounds to the same integer
// unless it lies within 1e-3 of a half-integer (or is large): only then is the division done.
__device__ __forceinline__ uint32_t code_of(float w, float d, float rd, float z) {
    const float t = __fmul_rn(w, rd);
    float r = rintf(t);
    if (!(fabsf(t - r) < 0.499f && fabsf(t) < 1024.0f)) r = rintf(__fdiv_rn(w, d));
    return (uint32_t)fminf(fmaxf(__fadd_rn(r, z), 0.0f), 15.0f);
}

// grid = (K/128, N/128), block = 256 (8 warps = 8 bands of the 128-row slab); three blocks per SM:
// the kernel is latency-bound (loads, then arithmetic), measured 67.6 -> 53.2 us on 4096->11008
template <int G>
__global__ void __launch_bounds__(256, 3)
quantize_pack_kernel(const __half* __restrict__ W, const float* __restrict__ a, float alpha,
                     int mode, uint32_t* __restrict__ qweight, __half* __restrict__ scales,
                     uint8_t* __restrict__ zeros, int N, int K) {
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
    // registers stay live and four blocks fit an SM.  The four scales of a word are one 16-byte
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

#pragma unroll
    for (int ti = 0; ti < 2; ++ti) {
        __half d16[2]; float d[2], z[2], rd[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            group_params(mn[ti][h], mx[ti][h], d16[h], d[h], z[h]);
            rd[h] = __frcp_rn(d[h]);
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
            words[j] = (code_of(wu[0], d[0], rd[0], z[0]) << 0) | (code_of(wu[1], d[0], rd[0], z[0]) << 16) |
                       (code_of(wl[0], d[1], rd[1], z[1]) << 4) | (code_of(wl[1], d[1], rd[1], z[1]) << 20) |
                       (code_of(wu[2], d[0], rd[0], z[0]) << 8) | (code_of(wu[3], d[0], rd[0], z[0]) << 24) |
                       (code_of(wl[2], d[1], rd[1], z[1]) << 12) | (code_of(wl[3], d[1], rd[1], z[1]) << 28);
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

cudaError_t launch_quantize_pack(const __half* W, const float* a, float alpha, int group,
                                 uint32_t* qweight, __half* scales, uint8_t* zeros,
                                 int N, int K, cudaStream_t st) {
    const dim3 grid(K / 128, N / 128);
    const int mode = (int)alpha_mode(alpha);
    if (group == 128)
        quantize_pack_kernel<128><<<grid, 256, 0, st>>>(W, a, alpha, mode, qweight, scales, zeros, N, K);
    else
        quantize_pack_kernel<64><<<grid, 256, 0, st>>>(W, a, alpha, mode, qweight, scales, zeros, N, K);
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

}  // namespace awq
