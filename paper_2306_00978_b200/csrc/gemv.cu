// Decode path of the layer (Sec. 4.2: fused dequantize + matrix-vector product), M <= 16.
//
// HBM-bound: the packed weights (0.5 byte per weight) are streamed once with coalesced
// 128-bit loads; a warp's 32 loads cover one contiguous 512-byte band piece (16 rows x 64
// columns).  The 16 bytes a lane receives are, after the two-at-a-time int4 -> fp16
// register conversion that the w{0,2,4,6,1,3,5,7} nibble order makes cheap, exactly the
// four A-operand fragments of four warp-level m16n8k16 tensor-core products: (q - z) enters
// as exact fp16 integers, the activations (up to 8 tokens per product) as the B operand,
// and the accumulation is fp32.  Delta is applied in fp32 once per group.  ALU cost is
// about 9 lane-operations per 8 codes, inside the ~2.5 op/code budget HBM allows.
//
// K is split across thread blocks; partial sums go to an fp32 workspace and the last
// block to arrive for a 128-row slab adds them in split order (deterministic, no float
// atomics, nobody waits).
#include "common.cuh"

namespace awq {

namespace {

constexpr int kGemvThreads = 256;
constexpr int kBatch = 4;                // k-tiles fetched per thread before computing

__device__ __forceinline__ uint4 ldg_stream_v4(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__device__ __forceinline__ void mma_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                          uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t hsub2_u32(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("sub.rn.f16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ uint32_t hfma2_u32(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t d;
    asm("fma.rn.f16x2 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

// One packed word -> the four fp16x2 A fragments holding exact (q - z).
//   zlo = fp16x2(1024 + z_upper), zhi = fp16x2(-(64 + z_lower))
__device__ __forceinline__ void dequant_word(uint32_t w, uint32_t zlo, uint32_t zhi,
                                             uint32_t& a0, uint32_t& a1, uint32_t& a2, uint32_t& a3) {
    constexpr uint32_t kMagic = 0x64006400u;       // fp16 1024.0 in both halves
    constexpr uint32_t kSixteenth = 0x2C002C00u;   // fp16 1/16 in both halves
    const uint32_t w8 = w >> 8;
    a0 = hsub2_u32((w & 0x000F000Fu) | kMagic, zlo);               // 1024 + q  - (1024 + z)
    a1 = hfma2_u32((w & 0x00F000F0u) | kMagic, kSixteenth, zhi);   // (1024 + 16q)/16 - (64 + z)
    a2 = hsub2_u32((w8 & 0x000F000Fu) | kMagic, zlo);
    a3 = hfma2_u32((w8 & 0x00F000F0u) | kMagic, kSixteenth, zhi);
}

// grid.x = slabs * splits (slab-major); block = 256 = 8 warps = the 8 bands of a slab.
// MT = number of 8-token column tiles (1: M <= 8, 2: M <= 16).
template <int G, int MT>
__global__ void __launch_bounds__(kGemvThreads, (MT == 1 ? 3 : 2))
gemv_kernel(const uint4* __restrict__ qweight, const __half* __restrict__ scales,
            const uint8_t* __restrict__ zeros, const __half* __restrict__ x,
            __half* __restrict__ y, float* __restrict__ partial, unsigned int* __restrict__ counters,
            int M, int N, int K, int splits, int ktiles_per_split) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __half* xs = reinterpret_cast<__half*>(smem_raw);
    __shared__ unsigned int s_last;

    constexpr int TPG = G / 64;                       // k-tiles per group
    const int slab = blockIdx.x / splits, sp = blockIdx.x % splits;
    const int ktiles = K / 64;
    const int kt0 = sp * ktiles_per_split;
    const int kt1 = min(kt0 + ktiles_per_split, ktiles);
    const int nkt = kt1 - kt0;                        // a whole number of groups
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;
    const int n0 = slab * 128 + warp * 16 + g;        // rows n0 and n0 + 8
    const int ldx = ktiles_per_split * 64 + 8;        // padded row of the x stage (halfs)

    const uint4* wp = qweight + ((size_t)slab * ktiles + kt0) * 256 + warp * 32 + lane;

    // start the weight stream before anything else
    uint4 pk[kBatch];
#pragma unroll
    for (int u = 0; u < kBatch; ++u)
        pk[u] = (u < nkt) ? ldg_stream_v4(wp + (size_t)u * 256) : make_uint4(0u, 0u, 0u, 0u);

    // stage this block's slice of x: xs[m][k - kt0*64]
    {
        const int kspan = nkt * 64;
        const int chunks_per_row = kspan / 8;         // 16-byte chunks
        for (int i = threadIdx.x; i < M * chunks_per_row; i += kGemvThreads) {
            const int m = i / chunks_per_row, c = i % chunks_per_row;
            const uint4 v = *reinterpret_cast<const uint4*>(x + (size_t)m * K + (size_t)kt0 * 64 + c * 8);
            *reinterpret_cast<uint4*>(xs + m * ldx + c * 8) = v;
        }
    }
    __syncthreads();

    float acc[MT][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[mt][i] = 0.0f;

    const __half* sc_p = scales + (size_t)(kt0 / TPG) * N + n0;
    const uint8_t* z_p = zeros + (size_t)(kt0 / TPG) * (N / 2) + (n0 >> 4) * 8 + g;
    bool tok_ok[MT];
    const __half* xrow[MT];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
        tok_ok[mt] = (mt * 8 + g) < M;
        xrow[mt] = xs + (tok_ok[mt] ? (mt * 8 + g) : 0) * ldx + 16 * t;
    }

    for (int kb = 0; kb < nkt; kb += kBatch) {
        // group parameters of this batch (kBatch / TPG groups)
        constexpr int NG = kBatch / TPG;
        float d_up[NG], d_lo[NG];
        uint32_t zlo[NG], zhi[NG];
#pragma unroll
        for (int q = 0; q < NG; ++q) {
            const int gi = min(kb / TPG + q, nkt / TPG - 1);      // ragged last batch: clamp
            d_up[q] = __half2float(sc_p[(size_t)gi * N]);
            d_lo[q] = __half2float(sc_p[(size_t)gi * N + 8]);
            const uint32_t zb = z_p[(size_t)gi * (N / 2)];
            const uint32_t zu = 0x6400u + (zb & 0xFu);            // fp16(1024 + z_upper)
            const uint32_t zl = 0xD400u + ((zb >> 4) << 4);       // fp16(-(64 + z_lower))
            zlo[q] = zu | (zu << 16);
            zhi[q] = zl | (zl << 16);
        }
        uint4 cur[kBatch];
#pragma unroll
        for (int u = 0; u < kBatch; ++u) cur[u] = pk[u];
#pragma unroll
        for (int u = 0; u < kBatch; ++u)
            if (kb + kBatch + u < nkt) pk[u] = ldg_stream_v4(wp + (size_t)(kb + kBatch + u) * 256);

#pragma unroll
        for (int q = 0; q < NG; ++q) {
            if (kb + q * TPG >= nkt) break;                       // ragged last batch
            float accg[MT][4];
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                for (int i = 0; i < 4; ++i) accg[mt][i] = 0.0f;
#pragma unroll
            for (int v = 0; v < TPG; ++v) {
                const int u = q * TPG + v;
                const uint32_t wds[4] = {cur[u].x, cur[u].y, cur[u].z, cur[u].w};
                uint4 xa[MT], xb[MT];
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) {
                    if (tok_ok[mt]) {
                        const uint4* xp = reinterpret_cast<const uint4*>(xrow[mt] + (kb + u) * 64);
                        xa[mt] = xp[0];
                        xb[mt] = xp[1];
                    } else {
                        xa[mt] = make_uint4(0u, 0u, 0u, 0u);
                        xb[mt] = make_uint4(0u, 0u, 0u, 0u);
                    }
                }
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    uint32_t a0, a1, a2, a3;
                    dequant_word(wds[j], zlo[q], zhi[q], a0, a1, a2, a3);
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt) {
                        const uint32_t b0 = (j == 0) ? xa[mt].x : (j == 1) ? xa[mt].z : (j == 2) ? xb[mt].x : xb[mt].z;
                        const uint32_t b1 = (j == 0) ? xa[mt].y : (j == 1) ? xa[mt].w : (j == 2) ? xb[mt].y : xb[mt].w;
                        mma_16816(accg[mt], a0, a1, a2, a3, b0, b1);
                    }
                }
            }
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
                acc[mt][0] = fmaf(d_up[q], accg[mt][0], acc[mt][0]);
                acc[mt][1] = fmaf(d_up[q], accg[mt][1], acc[mt][1]);
                acc[mt][2] = fmaf(d_lo[q], accg[mt][2], acc[mt][2]);
                acc[mt][3] = fmaf(d_lo[q], accg[mt][3], acc[mt][3]);
            }
        }
    }

    // acc[mt][0..1]: row n0, tokens mt*8 + 2t, +1; acc[mt][2..3]: row n0 + 8, same tokens
    if (splits == 1) {
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int m = mt * 8 + 2 * t + (i & 1);
                if (m < M) y[(size_t)m * N + n0 + (i >> 1) * 8] = __float2half_rn(acc[mt][i]);
            }
        return;
    }

    float* mine = partial + (size_t)sp * M * N;
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int m = mt * 8 + 2 * t + (i & 1);
            if (m < M) __stcg(mine + (size_t)m * N + n0 + (i >> 1) * 8, acc[mt][i]);
        }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned int prev = atomicAdd(counters + slab, 1u);
        s_last = (prev == (unsigned int)(splits - 1)) ? 1u : 0u;
    }
    __syncthreads();
    if (s_last == 0u) return;
    __threadfence();
    // last block of this slab: add the partial sums in split order
    for (int i = threadIdx.x; i < M * 128; i += kGemvThreads) {
        const int m = i >> 7, n = slab * 128 + (i & 127);
        float s = 0.0f;
        for (int q = 0; q < splits; ++q) s += __ldcg(partial + ((size_t)q * M + m) * N + n);
        y[(size_t)m * N + n] = __float2half_rn(s);
    }
    if (threadIdx.x == 0) counters[slab] = 0u;        // ready for the next call
}

}  // namespace

GemvPlan gemv_plan(int M, int N, int K, int group) {
    (void)group;
    GemvPlan p;
    const int slabs = N / 128, ktiles = K / 64;
    // k-tiles per block: a multiple of the batch, at most 16 (1024 input channels), chosen so
    // that the grid has a few thousand warps' worth of independent streams
    int kps = 16;
    while (kps > kBatch && (long long)slabs * ((ktiles + kps - 1) / kps) < 148LL * 6) kps -= kBatch;
    p.ktiles_per_split = kps;
    p.splits = (ktiles + kps - 1) / kps;
    p.workspace_bytes = p.splits > 1 ? kCounterBytes + (size_t)p.splits * M * N * sizeof(float) : 0;
    return p;
}

cudaError_t launch_gemv(const void* x, const void* qweight, const void* scales, const void* zeros,
                        void* y, int M, int N, int K, int group, const GemvPlan& plan,
                        void* workspace, cudaStream_t st) {
    const int slabs = N / 128;
    unsigned int* counters = reinterpret_cast<unsigned int*>(workspace);
    float* partial = workspace
        ? reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(workspace) + kCounterBytes) : nullptr;
    const size_t smem = (size_t)M * (plan.ktiles_per_split * 64 + 8) * sizeof(__half);
    const dim3 grid((unsigned)(slabs * plan.splits));
#define AWQ_GEMV_LAUNCH(GG, MTT)                                                                   \
    gemv_kernel<GG, MTT><<<grid, kGemvThreads, smem, st>>>(                                        \
        reinterpret_cast<const uint4*>(qweight), reinterpret_cast<const __half*>(scales),          \
        reinterpret_cast<const uint8_t*>(zeros), reinterpret_cast<const __half*>(x),               \
        reinterpret_cast<__half*>(y), partial, counters, M, N, K, plan.splits, plan.ktiles_per_split)
    if (group == 128) { if (M <= 8) AWQ_GEMV_LAUNCH(128, 1); else AWQ_GEMV_LAUNCH(128, 2); }
    else              { if (M <= 8) AWQ_GEMV_LAUNCH(64, 1);  else AWQ_GEMV_LAUNCH(64, 2); }
#undef AWQ_GEMV_LAUNCH
    count_launch();
    return cudaGetLastError();
}

}  // namespace awq
