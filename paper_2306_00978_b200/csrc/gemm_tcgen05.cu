// Prefill path of the layer (Sec. 4.2: fused dequantize + matrix-matrix product), sm_100a.
//
// The weights are the MMA's A operand (128 output channels = 128 TMEM lanes), the tokens
// its N side (BN = 32..256 columns of the fp32 accumulator in tensor memory), so
// D[n][m] = sum_k dequant(Wq)[n][k] * x[m][k] and the epilogue writes y[m][n] = D[n][m].
//
// Shared-memory bandwidth, not the tensor pipe, is what a dequantizing GEMM runs out of first
// (per 64-wide k-block the x tile is written once and read once, 64 KB at BN = 256).  So the
// dequantized weights never touch shared memory: they go from registers straight into tensor
// memory (tcgen05.st) and the MMA takes its A operand from there.
//
// One persistent thread block per SM, warp-specialised:
//   warp 0       producer: per k-block two TMA tensor copies into a ring of stages - the x tile
//                (BN x 64 fp16, 128-byte swizzle) and the packed weights of the slab's 8 bands
//                (8 x 512 bytes, one box of the band-major weight array) - completion counted
//                on an mbarrier.
//   warps 8-15   dequantizers, one per 16-row band.  Lane (g, t) reads its 16-byte packed piece
//                (rows g, g+8; columns 16j+4t..+3), converts two codes at a time to exact fp16
//                (q - z) with the magic-number trick that the w{0,2,4,6,1,3,5,7} nibble order
//                allows, multiplies by Delta (one fp16 rounding) and stores its 16 registers
//                with one tcgen05.st: the piece layout is exactly the 16x256b register layout,
//                so the band's 16 lanes x 32 columns of A land in the stage's slot of tensor
//                memory without any shuffle.  Scales and zero points (32 + 8 bytes per band
//                and group) are read straight from global memory two groups ahead.
//   warp 1       one thread issues tcgen05.mma (kind::f16, M = 128, N = BN, K = 16, four per
//                k-block, A from tensor memory, B through a shared-memory descriptor), commits
//                to the stage's "empty" barrier and, after the last k-block, to the
//                accumulator's "full" barrier.
//   warps 4-7    epilogue: tcgen05.ld 32 columns at a time, convert to fp16, transpose through a
//                2 KB shared-memory block to [token][channel] and store it with one TMA tensor
//                store (two-byte global stores were an order of magnitude slower).
//                BN <= 128 keeps two accumulators so that the epilogue overlaps the next tile.
//
// Tensor-memory columns: accumulators first (BN or 2 BN), then 32 columns per stage for A.
// Every wait is bounded (about two seconds of wall clock): a wait that runs out writes a code to
// the status word, raises a block-wide flag, and every role leaves its loop; the block
// then waits (bounded) for its own copies in flight, frees its tensor memory and returns.
#include "tcgen05.cuh"

namespace awq {

namespace {

constexpr int kGemmThreads = 512;
constexpr int kMaxSplits = 16;                  // split-K factor of a tile (M <= 128)
constexpr int kDequantUnroll = 2;               // k-blocks a dequantizer warp handles per iteration

template <int BN> struct GemmCfg {
    static constexpr int kXTileBytes = BN * kBK * 2;
    static constexpr int kStageBytes = kXTileBytes + kTileBytes;          // x tile + packed weights
    static constexpr int kNumAcc = BN <= 128 ? 2 : 1;                      // accumulators in TMEM
    static constexpr int kOutBytes = 4 * 2 * 2048;                         // 4 epilogue warps x 2 staging buffers
    static constexpr int kStagesSmem = (216 * 1024 - kOutBytes) / kStageBytes;
    static constexpr int kStagesTmem = (512 - kNumAcc * BN) / 32;          // 32 columns of A per stage
    static constexpr int kStagesMin = kStagesSmem < kStagesTmem ? kStagesSmem : kStagesTmem;
    static constexpr int kStages = kStagesMin > 8 ? 8 : kStagesMin;
    static constexpr int kAColumn0 = kNumAcc * BN;                         // first A column
    static constexpr int kTmemCols = 512;
    static constexpr int kSmemBytes = kStages * kStageBytes + kOutBytes + 1024 /*align*/ + 256 /*barriers*/;
    static constexpr uint32_t kTxBytes = kXTileBytes + kTileBytes;
};

// ------------------------------------------------------------------------- the kernel
template <int G, int BN>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap x_map, const __grid_constant__ CUtensorMap w_map,
            const __grid_constant__ CUtensorMap y_map,
            const __half* __restrict__ scales, const unsigned char* __restrict__ zeros,
            int M, int N, int K, int splits, float* __restrict__ partials,
            unsigned int* __restrict__ counters, unsigned int* status_word) {
    using Cfg = GemmCfg<BN>;
    constexpr int S = Cfg::kStages;
    constexpr int NACC = Cfg::kNumAcc;
    extern __shared__ unsigned char smem_dyn[];
    __shared__ unsigned int s_abort;
    __shared__ uint32_t s_tmem_base;

    const uint32_t dyn = smem_u32(smem_dyn);
    const uint32_t base = (dyn + 1023u) & ~1023u;                    // 1024-byte aligned stage ring
    unsigned char* base_ptr = smem_dyn + (base - dyn);
    // stage layout: [x tile | packed weights (8 bands x 512 bytes)]
    auto x_addr = [&](int s) { return base + (uint32_t)s * Cfg::kStageBytes; };
    auto w_ptr = [&](int s) { return base_ptr + (size_t)s * Cfg::kStageBytes + Cfg::kXTileBytes; };
    const uint32_t out_base = base + (uint32_t)S * Cfg::kStageBytes;   // epilogue staging, then 8-byte barriers
    const uint32_t bars = out_base + (uint32_t)Cfg::kOutBytes;
    auto raw_full = [&](int s) { return bars + 8u * (uint32_t)s; };
    auto a_full = [&](int s) { return bars + 8u * (uint32_t)(S + s); };
    auto empty = [&](int s) { return bars + 8u * (uint32_t)(2 * S + s); };
    auto acc_full = [&](int b) { return bars + 8u * (uint32_t)(3 * S + b); };
    auto acc_empty = [&](int b) { return bars + 8u * (uint32_t)(3 * S + 2 + b); };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m_tiles = (M + BN - 1) / BN;
    const int total_tiles = (N / 128) * m_tiles;
    // split-K: a work item is (tile, split); split sp of a tile covers the groups
    // [sp * ng / splits, (sp + 1) * ng / splits), i.e. whole groups and at least one
    constexpr int KPG = G / kBK;                    // k-blocks per group
    const int ng = K / G;
    const int total_items = total_tiles * splits;
    auto kb_begin = [&](int sp) { return (int)(((long long)sp * ng) / splits) * KPG; };

    if (threadIdx.x == 0) {
        s_abort = 0u;
        for (int s = 0; s < S; ++s) { mbar_init(raw_full(s), 1); mbar_init(a_full(s), 8); mbar_init(empty(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(acc_full(b), 1); mbar_init(acc_empty(b), 4); }
        mbar_fence_init();
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&s_tmem_base)), "r"((uint32_t)Cfg::kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = s_tmem_base;
    const WaitCtl ctl{status_word, &s_abort};

    if (warp == 0) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            unsigned int issued = 0;
            bool ok = true;
            for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x) {
                const int tile = item / splits, sp = item - tile * splits;
                const int slab = tile / m_tiles, mt = tile % m_tiles;
                const int kb1 = kb_begin(sp + 1);
                for (int kb = kb_begin(sp); kb < kb1; ++kb) {
                    if (!mbar_wait(empty(stage), phase ^ 1u, ctl)) { ok = false; break; }
                    const uint32_t bar = raw_full(stage);
                    mbar_arrive_expect_tx(bar, Cfg::kTxBytes);
                    tma_load_2d(x_addr(stage), &x_map, kb * kBK, mt * BN, bar);
                    // weights: box of 8 bands x 512 bytes (128 words) at (k-block, first band)
                    tma_load_2d(x_addr(stage) + Cfg::kXTileBytes, &w_map, kb * 128, slab * 8, bar);
                    ++issued;
                    if (++stage == S) { stage = 0; phase ^= 1u; }
                }
            }
            if (!ok) {
                // giving up: let the copies already issued land before the block exits
                const unsigned int pending = issued < (unsigned)S ? issued : (unsigned)S;
                uint32_t st = stage, ph = phase;
                for (unsigned int i = 0; i < pending; ++i) {
                    if (st == 0) { st = S - 1; ph ^= 1u; } else { --st; }
                    const unsigned long long t0 = global_ns();
                    while (!mbar_try_wait(raw_full(st), ph) && global_ns() - t0 < 100000000ull) {}
                }
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc(BN);
            uint32_t stage = 0, phase = 0;
            int local = 0;
            bool ok = true;
            for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x, ++local) {
                const int sp = item % splits;
                const int kb0 = kb_begin(sp), kb1 = kb_begin(sp + 1);
                const int b = local % NACC;
                const uint32_t use = (uint32_t)(local / NACC) & 1u;
                if (!mbar_wait(acc_empty(b), use ^ 1u, ctl)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(b * BN);
                for (int kb = kb0; kb < kb1; ++kb) {
                    if (!mbar_wait(raw_full(stage), phase, ctl) || !mbar_wait(a_full(stage), phase, ctl)) {
                        ok = false; break;
                    }
                    tc_fence_after();
                    const uint32_t a_tmem = tmem_base + (uint32_t)(Cfg::kAColumn0 + stage * 32);
                    const uint64_t bdesc = smem_desc_sw128(x_addr(stage));
#pragma unroll
                    for (int k = 0; k < kBK / 16; ++k)       // A: +8 columns, B: +32 bytes per K = 16 step
                        umma_f16_a_tmem(d_tmem, a_tmem + (uint32_t)(8 * k), bdesc + (uint64_t)(2 * k), idesc,
                                        (kb != kb0 || k != 0) ? 1u : 0u);
                    umma_commit(empty(stage));
                    if (++stage == S) { stage = 0; phase ^= 1u; }
                }
                if (ok) umma_commit(acc_full(b));
            }
        }
    } else if (warp >= 8) {
        // -------------------------------------------------------------- dequantizers
        // one warp per 16-row band; lane (g, t) holds the band's piece (rows g and g+8, columns
        // 16j + 4t .. +3 for j = 0..3), which is exactly its share of a 16-lane x 32-column
        // tensor-memory store in the 16x256b register layout (four columns blocks of 8)
        const int wi = warp - 8, quad = wi & 3, hsel = wi >> 2;
        const int band = 2 * quad + hsel;               // bands 0..7 <-> TMEM lanes 16*band .. +15
        const int g = lane >> 2;
        const uint32_t taddr_band = tmem_base + ((uint32_t)(quad * 32 + hsel * 16) << 16) + (uint32_t)Cfg::kAColumn0;
        uint32_t stage = 0, phase = 0;
        bool ok = true;
        for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x) {
            const int tile = item / splits, sp = item - tile * splits;
            const int slab = tile / m_tiles;
            const int kb0 = kb_begin(sp), kb1 = kb_begin(sp + 1);
            // this lane's rows' parameters: scales [band][group][16], zero bytes [band pair][group][16]
            const unsigned short* sc_g = reinterpret_cast<const unsigned short*>(scales) +
                                         (size_t)(slab * 8 + band) * ng * 16 + g;
            const unsigned char* z_g = zeros + (size_t)(slab * 4 + (band >> 1)) * ng * 16 + (band & 1) * 8 + g;
            // U k-blocks per iteration, so that their shared-memory reads, conversions and
            // tensor-memory stores overlap (one k-block at a time is a chain of latencies: measured
            // ~860 cycles per k-block).  The scales and zero points of an iteration's groups are
            // fetched two iterations ahead.
            constexpr int U = kDequantUnroll;
            constexpr int GPI = U / KPG;                // groups per iteration
            uint32_t du[GPI], dl[GPI], zb[GPI], du1[GPI], dl1[GPI], zb1[GPI], du2[GPI], dl2[GPI], zb2[GPI];
            const int g0 = kb0 / KPG;
#pragma unroll
            for (int q = 0; q < GPI; ++q) {
                const int ga = min(g0 + q, ng - 1), gb = min(g0 + GPI + q, ng - 1);
                du[q] = dl[q] = zb[q] = 0u;
                du1[q] = __ldg(sc_g + ga * 16); dl1[q] = __ldg(sc_g + ga * 16 + 8); zb1[q] = __ldg(z_g + ga * 16);
                du2[q] = __ldg(sc_g + gb * 16); dl2[q] = __ldg(sc_g + gb * 16 + 8); zb2[q] = __ldg(z_g + gb * 16);
            }
            for (int kb = kb0; kb < kb1; kb += U) {
                const int n = min(U, kb1 - kb);                    // k-blocks of this iteration
#pragma unroll
                for (int q = 0; q < GPI; ++q) {
                    du[q] = du1[q]; dl[q] = dl1[q]; zb[q] = zb1[q];
                    du1[q] = du2[q]; dl1[q] = dl2[q]; zb1[q] = zb2[q];
                    const int gc = min(kb / KPG + 2 * GPI + q, ng - 1);
                    du2[q] = __ldg(sc_g + gc * 16); dl2[q] = __ldg(sc_g + gc * 16 + 8); zb2[q] = __ldg(z_g + gc * 16);
                }
                uint32_t stg[U];
                uint4 pk[U];
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    stg[u] = stage;
                    if (u < n) {
                        ok = ok && mbar_wait(raw_full(stage), phase, ctl);
                        if (++stage == S) { stage = 0; phase ^= 1u; }
                    }
                }
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
#pragma unroll
                for (int u = 0; u < U; ++u)
                    if (u < n) pk[u] = *reinterpret_cast<const uint4*>(w_ptr(stg[u]) + band * 512 + lane * 16);
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    if (u < n) {
                        const int q = u / KPG;
                        const uint32_t d_up = du[q] | (du[q] << 16), d_lo = dl[q] | (dl[q] << 16);
                        const uint32_t zu = 0x6400u + (zb[q] & 0xFu), zl = 0xD400u + ((zb[q] >> 4) << 4);
                        const uint32_t zlo = zu | (zu << 16), zhi = zl | (zl << 16);
                        const uint32_t wds[4] = {pk[u].x, pk[u].y, pk[u].z, pk[u].w};
                        // per word j: (row g: c, c+1) (row g: c+2, c+3) (row g+8: c, c+1) (row g+8: c+2, c+3)
                        uint32_t v[16];
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            constexpr uint32_t kMagic = 0x64006400u, kSixteenth = 0x2C002C00u;
                            const uint32_t w = wds[j], w8 = w >> 8;
                            v[4 * j + 0] = hmul2_u32(hsub2_u32((w & 0x000F000Fu) | kMagic, zlo), d_up);
                            v[4 * j + 1] = hmul2_u32(hsub2_u32((w8 & 0x000F000Fu) | kMagic, zlo), d_up);
                            v[4 * j + 2] = hmul2_u32(hfma2_u32((w & 0x00F000F0u) | kMagic, kSixteenth, zhi), d_lo);
                            v[4 * j + 3] = hmul2_u32(hfma2_u32((w8 & 0x00F000F0u) | kMagic, kSixteenth, zhi), d_lo);
                        }
                        tmem_st_16x32cols(taddr_band + stg[u] * 32u, v);
                    }
                }
                tmem_st_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
#pragma unroll
                    for (int u = 0; u < U; ++u)
                        if (u < n) mbar_arrive(a_full(stg[u]));
                }
            }
        }
    } else if (warp >= 4) {
        // ------------------------------------------------------------------ epilogue
        const int quad = warp & 3;                     // TMEM lanes 32*quad .. +31
        int local = 0;
        int obuf = 0;
        bool ok = true;
        for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x, ++local) {
            const int tile = item / splits, sp = item - tile * splits;
            const int slab = tile / m_tiles, mt = tile % m_tiles;
            const int b = local % NACC;
            const uint32_t use = (uint32_t)(local / NACC) & 1u;
            ok = mbar_wait(acc_full(b), use, ctl);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            tc_fence_after();
            const int n0 = slab * 128 + quad * 32;
            const int m0 = mt * BN;
            const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(b * BN);
            bool finish = true;                 // this warp writes its 32 channels of y
            if (splits > 1) {
                // split-K: the partial sums go to the workspace as fp32 [tile][split][token][channel];
                // the warp whose arrival completes the (tile, quad) count adds all splits in split
                // order - whichever arrives last, the sum is formed the same way - and nobody waits
                float* mine = partials + ((size_t)(tile * splits + sp) * BN) * 128 + quad * 32 + lane;
#pragma unroll 1
                for (int c = 0; c < BN; c += 32) {
                    uint32_t r[32];
                    tmem_ld_32cols(taddr + (uint32_t)c, r);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 32; ++i) mine[(size_t)(c + i) * 128] = __uint_as_float(r[i]);
                }
                tc_fence_before();
                __threadfence();
                __syncwarp();
                unsigned int old = 0;
                if (lane == 0) {
                    mbar_arrive(acc_empty(b));
                    old = atomicAdd(counters + tile * 4 + quad, 1u);
                }
                old = __shfl_sync(0xFFFFFFFFu, old, 0);
                finish = old == (unsigned int)(splits - 1);
                if (finish) {
                    __threadfence();
                    if (lane == 0) counters[tile * 4 + quad] = 0u;      // ready for the next call
                }
            }
            if (!finish) continue;
#pragma unroll 1
            for (int c = 0; c < BN; c += 32) {
                uint32_t r[32];
                if (splits > 1) {
                    const float* all = partials + ((size_t)tile * splits * BN + c) * 128 + quad * 32 + lane;
#pragma unroll
                    for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__ldcg(all + (size_t)i * 128));
#pragma unroll 1
                    for (int q = 1; q < splits; ++q) {
                        const float* p = all + (size_t)q * BN * 128;
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            r[i] = __float_as_uint(__uint_as_float(r[i]) + __ldcg(p + (size_t)i * 128));
                    }
                } else {
                    tmem_ld_32cols(taddr + (uint32_t)c, r);
                    tmem_ld_wait();
                    if (c + 32 >= BN) {
                        // the accumulator is in registers: the MMA thread may start the next tile
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(acc_empty(b));
                    }
                }
                // stage the 32 x 32 block as [token][channel] fp16 and hand it to the copy engine:
                // one tensor store per block instead of 32 two-byte stores per thread (rows past
                // M are clipped by the tensor map)
                if (lane == 0) bulk_wait_read_1();                  // the store that last used this buffer
                __syncwarp();
                const uint32_t tb = out_base + (uint32_t)((quad * 2 + obuf) * 2048);
                unsigned char* tp = base_ptr + (tb - base);
#pragma unroll
                for (int i = 0; i < 32; ++i)
                    *reinterpret_cast<__half*>(tp + i * 64 + lane * 2) = __float2half_rn(__uint_as_float(r[i]));
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    tma_store_2d(&y_map, n0, m0 + c, tb);
                    bulk_commit_group();
                }
                obuf ^= 1;
            }
        }
        if (lane == 0) bulk_wait_all();                             // all of y written before exit
    }

    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;"
                     ::"r"(tmem_base), "r"((uint32_t)Cfg::kTmemCols) : "memory");
    }
}

// ------------------------------------------------------------------------------ host
template <int G, int BN>
cudaError_t launch_one(const CUtensorMap& map, const CUtensorMap& wmap, const CUtensorMap& ymap,
                       const void* scales, const void* zeros,
                       int M, int N, int K, int splits, void* workspace,
                       unsigned int* status_word, int sms, cudaStream_t st) {
    using Cfg = GemmCfg<BN>;
    static bool attr_done[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (!attr_done[dev & 63]) {
        cudaError_t e = cudaFuncSetAttribute(gemm_kernel<G, BN>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             Cfg::kSmemBytes);
        if (e != cudaSuccess) return e;
        attr_done[dev & 63] = true;
    }
    const int items = (N / 128) * ((M + BN - 1) / BN) * splits;
    const int grid = items < sms ? items : sms;
    unsigned char* ws = static_cast<unsigned char*>(workspace);
    gemm_kernel<G, BN><<<grid, kGemmThreads, Cfg::kSmemBytes, st>>>(
        map, wmap, ymap, reinterpret_cast<const __half*>(scales),
        reinterpret_cast<const unsigned char*>(zeros), M, N, K, splits,
        reinterpret_cast<float*>(ws + kCounterBytes), reinterpret_cast<unsigned int*>(ws), status_word);
    count_launch();
    return cudaGetLastError();
}

// Split-K factor of the one-SM kernel for M <= 128 (one token tile): with few 128-channel tiles
// most SMs would idle and the busy ones would each dequantize a whole 128 x K slab.  The factor
// minimizes rounds / splits, rounds = ceil(tiles * splits / SMs), with a small charge per split for
// the fp32 partial sums (written and read once), within: at least four k-blocks per split, the
// workspace at hand, one arrival counter per (tile, 32-channel quarter).
int gemm_splits(int M, int N, int K, int group, int bn, int sms, size_t workspace_bytes) {
    if (M > 128 || workspace_bytes <= kCounterBytes) return 1;
    const int tiles = N / 128;
    if (tiles * 4 > kMaxSlabs) return 1;
    const int ng = K / group, nkb = K / kBK;
    int best = 1;
    double best_cost = 1e30;
    for (int sp = 1; sp <= kMaxSplits; ++sp) {
        if (sp > ng || nkb / sp < 4) break;
        const size_t need = kCounterBytes + (size_t)tiles * sp * 128 * bn * sizeof(float);
        if (sp > 1 && need > workspace_bytes) break;
        const int rounds = (tiles * sp + sms - 1) / sms;
        const double cost = (double)rounds / sp + (sp > 1 ? 0.02 * sp : 0.0);
        if (cost < best_cost - 1e-9) { best_cost = cost; best = sp; }
    }
    return best;
}

}  // namespace

cudaError_t launch_gemm(const void* x, const void* qweight, const void* scales, const void* zeros,
                        void* y, int M, int N, int K, int group, bool path_pair_allowed,
                        void* workspace, size_t workspace_bytes,
                        unsigned int* status_word, cudaStream_t st) {
    EncodeTiledFn enc = encode_fn();
    if (!enc) return cudaErrorNotSupported;
    const int bn = M > 128 ? 256 : M > 64 ? 128 : M > 32 ? 64 : 32;
    const cuuint32_t estr[2] = {1, 1};
    // x as [M][K] fp16 in boxes of `tokens` rows x one k-block, 128-byte swizzle
    auto make_x_map = [&](CUtensorMap* map, int tokens) {
        const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)M};
        const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
        const cuuint32_t box[2] = {(cuuint32_t)kBK, (cuuint32_t)tokens};
        return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(x), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    };
    // packed weights as a 2-D array of 32-bit words, one row per 16-row band (K * 8 bytes):
    // boxes of 8 bands x `words` (128 words = one 64-wide k-tile of a band)
    auto make_w_map = [&](CUtensorMap* map, int words) {
        const cuuint64_t wdims[2] = {(cuuint64_t)K * 2, (cuuint64_t)(N / 16)};
        const cuuint64_t wstrides[1] = {(cuuint64_t)K * 8};
        const cuuint32_t wbox[2] = {(cuuint32_t)words, 8};
        return enc(map, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<void*>(qweight), wdims, wstrides, wbox,
                   estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    };
    // y as [M][N] fp16, stored in boxes of 32 tokens x 32 channels
    CUtensorMap ymap;
    const cuuint64_t ydims[2] = {(cuuint64_t)N, (cuuint64_t)M};
    const cuuint64_t ystrides[1] = {(cuuint64_t)N * 2};
    const cuuint32_t ybox[2] = {32, 32};
    const CUresult ry = enc(&ymap, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, y, ydims, ystrides, ybox, estr,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                            CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (ry != CUDA_SUCCESS) return cudaErrorInvalidValue;
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    CUtensorMap map, wmap;
    if (path_pair_allowed && gemm_pair_applies(M, N)) {
        if (!make_x_map(&map, 128) || !make_w_map(&wmap, 256)) return cudaErrorInvalidValue;
        bool launched = false;
        e = launch_gemm_pair(map, wmap, ymap, scales, zeros, M, N, K, group, workspace, workspace_bytes,
                             status_word, sms, st, &launched);
        if (e != cudaSuccess || launched) return e;
    }
    if (!make_x_map(&map, bn) || !make_w_map(&wmap, 128)) return cudaErrorInvalidValue;
    const int splits = gemm_splits(M, N, K, group, bn, sms, workspace ? workspace_bytes : 0);
#define AWQ_GEMM_CASE(GG, BNN) \
    return launch_one<GG, BNN>(map, wmap, ymap, scales, zeros, M, N, K, splits, workspace, status_word, sms, st)
    if (group == 128) {
        switch (bn) { case 256: AWQ_GEMM_CASE(128, 256); case 128: AWQ_GEMM_CASE(128, 128);
                      case 64: AWQ_GEMM_CASE(128, 64); default: AWQ_GEMM_CASE(128, 32); }
    } else {
        switch (bn) { case 256: AWQ_GEMM_CASE(64, 256); case 128: AWQ_GEMM_CASE(64, 128);
                      case 64: AWQ_GEMM_CASE(64, 64); default: AWQ_GEMM_CASE(64, 32); }
    }
#undef AWQ_GEMM_CASE
}

size_t gemm_workspace_bytes(int M, int N, int sms) {
    if (gemm_pair_applies(M, N)) return gemm_pair_workspace_bytes(sms);
    if (M > 128) return 0;
    // split-K of the one-SM kernel: the most it can use for this M and N (any K)
    const int bn = M > 64 ? 128 : M > 32 ? 64 : 32;
    const int tiles = N / 128;
    if (tiles * 4 > kMaxSlabs) return 0;
    return kCounterBytes + (size_t)tiles * kMaxSplits * 128 * bn * sizeof(float);
}

}  // namespace awq
