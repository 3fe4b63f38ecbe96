// The layer for 17 .. 64 tokens (Sec. 4.2: fused dequantize + product) on the tensor cores, where
// the weights still set the time: every packed byte should cross HBM once and nothing else should
// be slower than that.
//
// The prefill kernels (gemm_tcgen05*.cu) are built for many tokens: per 64-wide k-block a tile
// fetches its x tile again, eight warps dequantize, one thread polls two barriers for four
// products, and split-K meets through counters and a fix-up pass - about 780 cycles per 4 KB of
// packed weights and 9 us per launch, whatever the number of tokens.  This kernel keeps their
// arithmetic (weights -> exact fp16 (q - z), times Delta in fp16, straight into tensor memory as
// the A operand of tcgen05.mma; tokens on the N side, fp32 accumulator in tensor memory) and
// changes the decomposition, like the chunked matrix-vector kernel:
//   * a work unit is one 128-channel slab x one chunk of K; a block takes a contiguous range of
//     units that stay in one chunk as long as possible, so the chunk's slice of x (BN tokens x up
//     to 128 KB / BN columns, 128-byte swizzle, one tensor-map copy per 64 columns) is fetched
//     once per chunk and stays in shared memory as the B operand of every slab;
//   * a stage of the weight ring is 8 bands x 128 input channels = 8 KB (one tensor-map copy);
//     sixteen dequantizer warps (band, every second stage) fill 64 columns of tensor memory per
//     stage; two threads issue the stage's eight products (one k-block each, into accumulators of
//     their own), and the slots of tensor memory are released in two groups per turn of the ring;
//   * a unit's sums over ONE chunk are partial: four epilogue warps move them from tensor memory to
//     the fp32 workspace [chunk][token][channel] (coalesced, 128 bytes per warp and token), and the
//     chunked matrix-vector kernel's reduce kernel adds the chunks in ascending order and rounds
//     to fp16 once - deterministic, no counters, no waiting between blocks.
// Every wait is bounded as in the other kernels.
//
// Measured on 8192 -> 28672 at 16 tokens (cycle counters per role, then taken out again), in the
// order the changes were made: as first built, with the prefill kernel's way of fetching scales and
// zero points (global loads, two iterations ahead) 80 us; those parameters by tensor-map copies into
// shared memory, one box per unit, 75 us (an iteration no longer ends on a load that left two
// iterations earlier but whose register is moved one iteration earlier); a second issuing thread
// 65 us (one thread issued a product per ~105 cycles, 850 per stage; alone on the SM it issues one
// per ~80); dequantizer warps that own every second stage instead of half of every stage 63 us.
// A deeper ring of packed weights (10 stages instead of 6) and fewer commits (two per turn of the
// ring instead of one per stage) changed nothing by themselves.  What is left is the issue rate of
// the four schedulers: a dequantizer warp spends about 100 instructions on 8 packed words (13 per
// word are the conversion itself), four such warps and a share of the issuing, copying and epilogue
// warps per scheduler make about 600 cycles per 8 KB stage, against 350 at the HBM rate.
#include "tcgen05.cuh"

namespace awq {

namespace {

constexpr int kSkThreads = 768;                  // warp 0 weight copies, 1 and 3 products, 2 x copies, 4-7 epilogue, 8-23 dequantizers
constexpr int kSkStageBytes = 2 * kTileBytes;    // 8 bands x 2 k-blocks x 512 bytes
constexpr int kSkRing = 10;                      // stages of packed weights in shared memory (80 KB in flight per SM)
constexpr int kSkXBytes = 128 * 1024;            // the chunk's slice of x
// tensor memory: four accumulators of BN columns (two units in flight x the two halves of a stage,
// one issuing thread each), then 64 columns of dequantized weights per stage
template <int BN> struct SkCfg {
    static constexpr int kAColumn0 = 4 * BN <= 128 ? 128 : 256;
    static constexpr int kStages = (512 - kAColumn0) / 64;
};
constexpr int kSkTmemCols = 512;
constexpr int kSkMaxGroups = 16;                 // groups per chunk (one tensor-map box of scales / zero points)
constexpr int kSkParBytes = kSkMaxGroups * (8 * 32 + 4 * 16);   // a unit's scales [8 bands][groups][16] fp16 + zero bytes [4][groups][16]
constexpr int kSkSmem = kSkRing * kSkStageBytes + kSkXBytes + 2 * kSkParBytes + 1024 /*align*/ + 512 /*barriers*/;

__device__ __forceinline__ void tmem_ld_16cols(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
}

template <int G, int BN>
__global__ void __launch_bounds__(kSkThreads, 1)
gemm_skinny_kernel(const __grid_constant__ CUtensorMap x_map, const __grid_constant__ CUtensorMap w_map,
                   const __grid_constant__ CUtensorMap sc_map, const __grid_constant__ CUtensorMap z_map,
                   float* __restrict__ partial, int M, int N, int K, int CK,
                   const __grid_constant__ UnitStarts starts, unsigned int* status_word) {
    constexpr int S = SkCfg<BN>::kStages, R = kSkRing, A0 = SkCfg<BN>::kAColumn0;
    constexpr int GS = S / 2;                        // the A slots are released in two groups per turn of the ring
    constexpr int KPG = G / kBK;                     // k-blocks per group
    extern __shared__ unsigned char smem_dyn[];
    __shared__ unsigned int s_abort;
    __shared__ uint32_t s_tmem_base;

    const uint32_t dyn = smem_u32(smem_dyn);
    const uint32_t base = (dyn + 1023u) & ~1023u;
    unsigned char* base_ptr = smem_dyn + (base - dyn);
    // [x slice: CK tiles of BN rows x 128 bytes | ring of weight stages | two parameter buffers | barriers]
    const uint32_t x_base = base;
    const uint32_t w_base = base + (uint32_t)kSkXBytes;
    const uint32_t par_base = w_base + (uint32_t)(R * kSkStageBytes);
    const uint32_t bars = par_base + 2u * (uint32_t)kSkParBytes;
    // the packed weights' ring (raw_*: filled by the copy engine, released by the dequantizers as soon
    // as the words are in registers) is deeper than the ring of A slots in tensor memory (a_*:
    // filled by the dequantizers, released by the products' completion)
    auto raw_full = [&](uint32_t r) { return bars + 8u * r; };
    auto raw_empty = [&](uint32_t r) { return bars + 8u * (uint32_t)(R + r); };
    auto a_full = [&](uint32_t s) { return bars + 8u * (uint32_t)(2 * R + s); };
    auto a_empty = [&](uint32_t s) { return bars + 8u * (uint32_t)(2 * R + S + s); };
    auto acc_full = [&](int b) { return bars + 8u * (uint32_t)(2 * R + 2 * S + b); };
    auto acc_empty = [&](int b) { return bars + 8u * (uint32_t)(2 * R + 2 * S + 2 + b); };
    const uint32_t x_full = bars + 8u * (uint32_t)(2 * R + 2 * S + 4), x_empty = bars + 8u * (uint32_t)(2 * R + 2 * S + 5);
    auto par_full = [&](uint32_t b) { return bars + 8u * (uint32_t)(2 * R + 2 * S + 6) + 8u * b; };
    auto par_empty = [&](uint32_t b) { return bars + 8u * (uint32_t)(2 * R + 2 * S + 8) + 8u * b; };
    const int gpc = CK / KPG;                        // groups per chunk (<= kSkMaxGroups)
    const uint32_t z_in_par = (uint32_t)(gpc * 8 * 32), par_bytes = (uint32_t)(gpc * (8 * 32 + 4 * 16));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nslabs = N / 128, nkb = K / kBK;
    const int nchunks = (nkb + CK - 1) / CK;
    const int units = nchunks * nslabs;
    const int u0 = starts.v[blockIdx.x], u1 = starts.v[blockIdx.x + 1];
    (void)units;
    // unit u = chunk * nslabs + slab; a chunk has nt k-blocks = nt / 2 stages (K is a multiple of 128)
    auto chunk_of = [&](int u) { return u / nslabs; };
    auto tiles_of = [&](int c) { return min(CK, nkb - c * CK); };

    if (threadIdx.x == 0) {
        s_abort = 0u;
        for (int r = 0; r < R; ++r) { mbar_init(raw_full(r), 1); mbar_init(raw_empty(r), 8); }
        for (int s = 0; s < S; ++s) { mbar_init(a_full(s), 8); if (s < 2) mbar_init(a_empty(s), 2); }
        for (int b = 0; b < 2; ++b) { mbar_init(acc_full(b), 2); mbar_init(acc_empty(b), 4); }
        mbar_init(x_full, 1);
        mbar_init(x_empty, 2);
        for (uint32_t b = 0; b < 2; ++b) { mbar_init(par_full(b), 1); mbar_init(par_empty(b), 16); }
        mbar_fence_init();
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&s_tmem_base)), "r"((uint32_t)kSkTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = s_tmem_base;
    const WaitCtl ctl{status_word, &s_abort};
    // programmatic dependent launch: the packed arrays are constants of the layer and are copied
    // before the work in front of this launch has completed; x and the workspace are touched after it
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    if (warp == 0) {
        // ------------------------------------------------------------ weight copies
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            unsigned int issued = 0, par_issued = 0;
            bool ok = true;
            for (int u = u0; u < u1 && ok; ++u) {
                const int c = chunk_of(u), slab = u - c * nslabs;
                const int kb0 = c * CK, nt = tiles_of(c);
                // the unit's scales and zero points: boxes of 8 bands (4 band pairs) x the chunk's groups
                const uint32_t pb = (uint32_t)(u - u0) & 1u, puse = ((uint32_t)(u - u0) >> 1) & 1u;
                if (!mbar_wait(par_empty(pb), puse ^ 1u, ctl)) { ok = false; break; }
                mbar_arrive_expect_tx(par_full(pb), par_bytes);
                tma_load_2d(par_base + pb * (uint32_t)kSkParBytes, &sc_map, (kb0 / KPG) * 16, slab * 8, par_full(pb));
                tma_load_2d(par_base + pb * (uint32_t)kSkParBytes + z_in_par, &z_map, (kb0 / KPG) * 16, slab * 4, par_full(pb));
                ++par_issued;
                for (int j = 0; j < nt; j += 2) {
                    if (!mbar_wait(raw_empty(stage), phase ^ 1u, ctl)) { ok = false; break; }
                    mbar_arrive_expect_tx(raw_full(stage), kSkStageBytes);
                    // 8 bands x 2 k-blocks (256 words) at (word kb * 128 of the band's run, first band)
                    tma_load_2d(w_base + stage * kSkStageBytes, &w_map, (kb0 + j) * 128, slab * 8, raw_full(stage));
                    ++issued;
                    if (++stage == R) { stage = 0; phase ^= 1u; }
                }
            }
            if (!ok) {
                // giving up: let the copies already issued land before the block exits
                const unsigned int pending = issued < (unsigned)R ? issued : (unsigned)R;
                uint32_t st = stage, ph = phase;
                for (unsigned int i = 0; i < pending; ++i) {
                    if (st == 0) { st = R - 1; ph ^= 1u; } else { --st; }
                    const unsigned long long t0 = global_ns();
                    while (!mbar_try_wait(raw_full(st), ph) && global_ns() - t0 < drain_limit_ns(ctl)) {}
                }
                for (unsigned int i = 0; i < 2u && i < par_issued; ++i) {
                    const unsigned int k = par_issued - 1u - i;          // the k-th parameter copy: buffer k & 1, use k >> 1
                    const unsigned long long t0 = global_ns();
                    while (!mbar_try_wait(par_full(k & 1u), (k >> 1) & 1u) && global_ns() - t0 < drain_limit_ns(ctl)) {}
                }
            }
        }
    } else if (warp == 2) {
        // ------------------------------------------------------------ x copies, one slice per chunk
        if (lane == 0) {
            asm volatile("griddepcontrol.wait;" ::: "memory");
            int cur = -1;
            uint32_t n = 0;
            for (int u = u0; u < u1; ++u) {
                const int c = chunk_of(u);
                if (c == cur) continue;
                // the products that read the previous slice have completed
                if (n > 0 && !mbar_wait_relaxed(x_empty, (n - 1u) & 1u, ctl)) break;
                const int nt = tiles_of(c);
                mbar_arrive_expect_tx(x_full, (uint32_t)(nt * BN * 128));
                for (int kb = 0; kb < nt; ++kb)
                    tma_load_2d(x_base + (uint32_t)(kb * BN * 128), &x_map, (c * CK + kb) * kBK, 0, x_full);
                cur = c;
                ++n;
            }
            if (s_abort && n > 0) {
                // giving up: the last slice's copies must have landed before the block exits
                const unsigned long long t0 = global_ns();
                while (!mbar_try_wait(x_full, (n - 1u) & 1u) && global_ns() - t0 < drain_limit_ns(ctl)) {}
            }
        }
    } else if (warp == 1 || warp == 3) {
        // ------------------------------------------------------------ products
        // Two issuing threads: a thread cannot issue these small products faster than one per
        // ~50 - 100 cycles, which alone would cap the kernel below the HBM rate.  Thread h takes
        // k-block h of every stage into an accumulator of its own; the epilogue adds the two.
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc(BN);
            const int h = warp >> 1;
            uint32_t stage = 0, phase = 0, xn = 0;
            int local = 0, cur = -1;
            bool ok = true;
            for (int u = u0; u < u1 && ok; ++u, ++local) {
                const int c = chunk_of(u);
                const int nt = tiles_of(c);
                if (c != cur) {
                    if (!mbar_wait(x_full, xn & 1u, ctl)) break;
                    ++xn;
                    cur = c;
                }
                const int b = local & 1;
                const uint32_t use = (uint32_t)(local >> 1) & 1u;
                if (!mbar_wait(acc_empty(b), use ^ 1u, ctl)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)((2 * b + h) * BN);
                uint64_t bdesc = smem_desc_sw128(x_base + (uint32_t)(h * BN * 128));
                for (int j = 0; j < nt; j += 2) {
                    if (!mbar_wait(a_full(stage), phase, ctl)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_tmem = tmem_base + (uint32_t)(A0 + stage * 64 + 32 * h);
#pragma unroll
                    for (int k = 0; k < kBK / 16; ++k)           // A: +8 columns, B: +32 bytes per K = 16 step
                        umma_f16_a_tmem(d_tmem, a_tmem + (uint32_t)(8 * k), bdesc + (uint64_t)(2 * k), idesc,
                                        (j != 0 || k != 0) ? 1u : 0u);
                    if (stage % GS == GS - 1) umma_commit(a_empty(stage / GS));
                    bdesc += (uint64_t)((2 * BN * 128) >> 4);   // two k-blocks further in the slice of x
                    if (++stage == S) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                umma_commit(acc_full(b));
                // the slice of x may be replaced once the products of its last unit have completed
                if (u + 1 < u1 && chunk_of(u + 1) != c) umma_commit(x_empty);
            }
        }
    } else if (warp >= 8) {
        // ------------------------------------------------------------ dequantizers
        // warp (band, parity): the band's 16 rows, both k-blocks of every second stage (stages are
        // counted through the whole range of units), so that a warp pays its barrier polls,
        // parameter reads and arrivals once per 8 packed words.  Lane (g, t) holds, per k-block,
        // the piece (rows g and g+8, columns 16j + 4t .. +3 for j = 0..3), which is exactly its
        // share of a 16-lane x 32-column tensor-memory store in the 16x256b register layout.
        const int wi = warp - 8, quad = wi & 3, hsel = (wi >> 2) & 1, par2 = wi >> 3;
        const int band = 2 * quad + hsel;               // bands 0..7 <-> TMEM lanes 16 * band .. +15
        const int g = lane >> 2;
        const uint32_t taddr_band = tmem_base + ((uint32_t)(quad * 32 + hsel * 16) << 16) + (uint32_t)A0;
        const unsigned char* w_lane = base_ptr + kSkXBytes + band * 1024 + lane * 16;
        uint32_t stage = (uint32_t)par2, phase = 0;     // slot of A in tensor memory (this warp's next)
        uint32_t rstage = (uint32_t)par2, rphase = 0;   // stage of the packed weights' ring
        int first = par2;                               // this warp's first stage inside the next unit
        bool ok = true;
        for (int u = u0; u < u1 && ok; ++u) {
            const int c = chunk_of(u);
            const int nst = tiles_of(c) / 2;
            const uint32_t pb = (uint32_t)(u - u0) & 1u, puse = ((uint32_t)(u - u0) >> 1) & 1u;
            ok = mbar_wait(par_full(pb), puse, ctl);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            // this lane's rows' parameters: scales [band][group][16], zero bytes [band pair][group][16]
            const unsigned char* par = base_ptr + (par_base - base) + pb * kSkParBytes;
            const unsigned char* psc = par + band * (gpc * 32) + g * 2;
            const unsigned char* pz = par + z_in_par + (band >> 1) * (gpc * 16) + (band & 1) * 8 + g;
            int j = first;
            for (; j < nst; j += 2) {
                ok = mbar_wait(raw_full(rstage), rphase, ctl) && mbar_wait(a_empty(stage / GS), phase ^ 1u, ctl);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
                tc_fence_after();
                uint4 pk[2];
#pragma unroll
                for (int h = 0; h < 2; ++h)
                    pk[h] = *reinterpret_cast<const uint4*>(w_lane + rstage * kSkStageBytes + h * 512);
                // the words are in registers: the copy engine may refill the stage
                __syncwarp();
                if (lane == 0) mbar_arrive(raw_empty(rstage));
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int gi = (2 * j + h) / KPG;                 // group inside the chunk
                    const uint32_t du = *reinterpret_cast<const unsigned short*>(psc + gi * 32);
                    const uint32_t dl = *reinterpret_cast<const unsigned short*>(psc + gi * 32 + 16);
                    const uint32_t zb = pz[gi * 16];
                    const uint32_t d_up = du | (du << 16), d_lo = dl | (dl << 16);
                    const uint32_t zu = 0x6400u + (zb & 0xFu), zl = 0xD400u + ((zb >> 4) << 4);
                    const uint32_t zlo = zu | (zu << 16), zhi = zl | (zl << 16);
                    const uint32_t wds[4] = {pk[h].x, pk[h].y, pk[h].z, pk[h].w};
                    // per word j: (row g: c, c+1) (row g: c+2, c+3) (row g+8: c, c+1) (row g+8: c+2, c+3)
                    uint32_t v[16];
#pragma unroll
                    for (int jw = 0; jw < 4; ++jw) {
                        constexpr uint32_t kMagic = 0x64006400u, kSixteenth = 0x2C002C00u;
                        const uint32_t w = wds[jw], w8 = w >> 8;
                        v[4 * jw + 0] = hmul2_u32(hsub2_u32((w & 0x000F000Fu) | kMagic, zlo), d_up);
                        v[4 * jw + 1] = hmul2_u32(hsub2_u32((w8 & 0x000F000Fu) | kMagic, zlo), d_up);
                        v[4 * jw + 2] = hmul2_u32(hfma2_u32((w & 0x00F000F0u) | kMagic, kSixteenth, zhi), d_lo);
                        v[4 * jw + 3] = hmul2_u32(hfma2_u32((w8 & 0x00F000F0u) | kMagic, kSixteenth, zhi), d_lo);
                    }
                    tmem_st_16x32cols(taddr_band + stage * 64u + (uint32_t)(32 * h), v);
                }
                tmem_st_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(a_full(stage));
                stage += 2;
                if (stage >= (uint32_t)S) { stage -= S; phase ^= 1u; }
                rstage += 2;
                if (rstage >= (uint32_t)R) { rstage -= R; rphase ^= 1u; }
            }
            first = j - nst;                             // 0 or 1: where this warp's stages resume
            __syncwarp();
            if (lane == 0) mbar_arrive(par_empty(pb));               // the unit's parameters may be replaced
        }
    } else if (warp >= 4) {
        // ------------------------------------------------------------ epilogue
        asm volatile("griddepcontrol.wait;" ::: "memory");
        const int quad = warp & 3;                     // TMEM lanes 32 * quad .. +31
        int local = 0;
        for (int u = u0; u < u1; ++u, ++local) {
            const int c = chunk_of(u), slab = u - c * nslabs;
            const int b = local & 1;
            const uint32_t use = (uint32_t)(local >> 1) & 1u;
            bool ok = mbar_wait(acc_full(b), use, ctl);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(2 * b * BN);
            float* out = partial + (size_t)c * M * N + slab * 128 + quad * 32 + lane;
#pragma unroll 1
            for (int c0 = 0; c0 < BN; c0 += 16) {
                uint32_t r0[16], r1[16];
                tmem_ld_16cols(taddr + (uint32_t)c0, r0);
                tmem_ld_16cols(taddr + (uint32_t)(BN + c0), r1);
                tmem_ld_wait();
                if (c0 + 16 >= BN) {
                    // both accumulators are in registers: the next unit's products may overwrite them
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(acc_empty(b));
                }
#pragma unroll
                for (int i = 0; i < 16; ++i)
                    if (c0 + i < M) out[(size_t)(c0 + i) * N] = __uint_as_float(r0[i]) + __uint_as_float(r1[i]);
            }
        }
    }

    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;"
                     ::"r"(tmem_base), "r"((uint32_t)kSkTmemCols) : "memory");
    }
}

int skinny_bn(int M) { return M <= 16 ? 16 : M <= 32 ? 32 : 64; }

// k-blocks per chunk: the slice of x must fit (128 KB / BN / 128 bytes), the units (chunks x slabs)
// should fill the blocks' equal shares, and every chunk costs one fp32 [M][N] array written and
// read once (M / (4 CK) of the weight bytes).
int skinny_chunk_kb(int M, int N, int K, int group, int sms) {
    const int bn = skinny_bn(M), nkb = K / kBK, nslabs = N / 128;
    int best = 4;
    double best_cost = 1e30;
    for (int ck = 4; ck <= kSkXBytes / (bn * 128) && ck <= kSkMaxGroups * (group / kBK); ck *= 2) {
        const int units = ((nkb + ck - 1) / ck) * nslabs;
        const int blocks = units < sms ? units : sms;
        const int worst = (units + blocks - 1) / blocks;
        const double eff = (double)units / ((double)worst * sms);
        const double cost = (1.0 + (double)M / (4.0 * ck)) / eff;
        if (cost < best_cost - 1e-9) { best_cost = cost; best = ck; }
        if (ck >= nkb) break;
    }
    return best;
}

}  // namespace

bool gemm_skinny_applies(int M, int N, int K, int group) {
    return M >= 1 && M <= 64 && N % 128 == 0 && K % 128 == 0 && (group == 64 || group == 128) &&
           encode_fn() != nullptr;
}

size_t gemm_skinny_workspace_bytes(int M, int N, int K, int group, int sms) {
    const int ck = skinny_chunk_kb(M, N, K, group, sms);
    return kCounterBytes + (size_t)((K / kBK + ck - 1) / ck) * M * N * sizeof(float);
}

cudaError_t launch_gemm_skinny(const void* x, const void* qweight, const void* scales, const void* zeros, void* y,
                               int M, int N, int K, int group, void* workspace, unsigned int* status_word, int sms,
                               bool serialize, cudaStream_t st) {
    EncodeTiledFn enc = encode_fn();
    if (!enc) return cudaErrorNotSupported;
    const int bn = skinny_bn(M), ck = skinny_chunk_kb(M, N, K, group, sms);
    const int ng = K / group, gpc = ck / (group / kBK);
    const cuuint32_t estr[2] = {1, 1};
    CUtensorMap xmap, wmap, scmap, zmap;
    {
        // x as [M][K] fp16 in boxes of BN tokens x one k-block, 128-byte swizzle; rows past M read as zeros
        const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)M};
        const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
        const cuuint32_t box[2] = {(cuuint32_t)kBK, (cuuint32_t)bn};
        if (enc(&xmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(x), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    {
        // packed weights: one row of K * 2 words per band; boxes of 8 bands x 2 k-tiles (256 words)
        const cuuint64_t dims[2] = {(cuuint64_t)K * 2, (cuuint64_t)(N / 16)};
        const cuuint64_t strides[1] = {(cuuint64_t)K * 8};
        const cuuint32_t box[2] = {256, 8};
        if (enc(&wmap, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<void*>(qweight), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    {
        // scales: fp16 [band][group][16]; boxes of 8 bands x a chunk's groups
        const cuuint64_t dims[2] = {(cuuint64_t)ng * 16, (cuuint64_t)(N / 16)};
        const cuuint64_t strides[1] = {(cuuint64_t)ng * 32};
        const cuuint32_t box[2] = {(cuuint32_t)(gpc * 16), 8};
        if (enc(&scmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(scales), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    {
        // zero points: bytes [band pair][group][16]; boxes of 4 pairs x a chunk's groups
        const cuuint64_t dims[2] = {(cuuint64_t)ng * 16, (cuuint64_t)(N / 32)};
        const cuuint64_t strides[1] = {(cuuint64_t)ng * 16};
        const cuuint32_t box[2] = {(cuuint32_t)(gpc * 16), 4};
        if (enc(&zmap, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(zeros), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    float* partial = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(workspace) + kCounterBytes);
    const int chunks = (K / kBK + ck - 1) / ck;
    const int units = chunks * (N / 128);
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    int blocks = units < sms ? units : sms;
    if (blocks > kUnitMaxBlocks) blocks = kUnitMaxBlocks;
    const UnitStarts starts = unit_starts(units, N / 128, blocks);
    cfg.gridDim = dim3((unsigned)blocks);
    cfg.blockDim = dim3(kSkThreads);
    cfg.dynamicSmemBytes = kSkSmem;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = serialize ? 0 : 1;
    cudaError_t e;
#define AWQ_SK_LAUNCH(GG, BNN)                                                                      \
    do {                                                                                            \
        static bool done[64] = {};                                                                  \
        int dev = 0;                                                                                \
        e = cudaGetDevice(&dev);                                                                    \
        if (e != cudaSuccess) return e;                                                             \
        if (!done[dev & 63]) {                                                                      \
            e = cudaFuncSetAttribute(gemm_skinny_kernel<GG, BNN>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSkSmem); \
            if (e != cudaSuccess) return e;                                                         \
            done[dev & 63] = true;                                                                  \
        }                                                                                           \
        e = cudaLaunchKernelEx(&cfg, gemm_skinny_kernel<GG, BNN>, xmap, wmap, scmap, zmap,          \
                               partial, M, N, K, ck, starts, status_word);                          \
        if (e != cudaSuccess) return e;                                                             \
    } while (0)
#define AWQ_SK_PICK(GG)                                                                             \
    do {                                                                                            \
        if (bn == 16) AWQ_SK_LAUNCH(GG, 16);                                                        \
        else if (bn == 32) AWQ_SK_LAUNCH(GG, 32);                                                   \
        else AWQ_SK_LAUNCH(GG, 64);                                                                 \
    } while (0)
    if (group == 128) AWQ_SK_PICK(128); else AWQ_SK_PICK(64);
#undef AWQ_SK_PICK
#undef AWQ_SK_LAUNCH
    count_launch();
    e = launch_chunk_reduce(partial, y, chunks, (size_t)M * N, st);
    if (e != cudaSuccess) return e;
    return cudaGetLastError();
}

}  // namespace awq
