// Decode path of the layer (Sec. 4.2: fused dequantize + matrix-vector product), M <= 16.
//
// HBM-bound: the packed weights (0.5 byte per weight) are streamed exactly once.  One
// persistent thread block per SM takes a contiguous range of the (128-row slab, 512-column)
// work units.  A copy warp keeps a ring of shared-memory stages full with bulk asynchronous
// copies - 32 KB of packed weight tiles, the units' fp16 scales and zero points, and the
// matching slice of x - so that well over 100 KB per SM is always in flight, independent of
// registers and of what the math warps are doing.
//
// Sixteen math warps each own one 16-row band of four 64-column tiles per stage.  The 16
// bytes a lane reads from the stage are already the A fragments of four warp-level m16n8k16
// tensor-core products: thanks to the w{0,2,4,6,1,3,5,7} nibble order, masking a packed word
// with 0x000F000F / 0x00F000F0 (before and after one shift by 8) leaves two codes in the
// mantissa bits of an fp16x2 register, i.e. the exact values q * 2^-24 (upper row) and
// q * 2^-20 (lower row) as fp16 subnormals.  Five logic operations and one MMA per eight
// weights - the paper counts a shift, an AND and an FMA per single weight.  x (up to 8 tokens
// per product) is the B operand, accumulation is fp32.  The zero point is applied once per
// group in fp32:  sum (q - z) x = 2^24 * D - z * X,  X = sum of x over the group (the same
// for every output row: each block sums it once, in fp32, while its first weight stages are
// in flight); Delta is applied in the same step.  Nothing is rounded to fp16 before the output.
//
// A block's range may begin or end inside a slab.  At the end of each slab segment the math
// warps hand their fp32 sums to two flush warps through shared memory and go on streaming;
// the flush warps write y, or publish a partial sum in an fp32 workspace slot owned by the
// block, and the last block to arrive for that slab (an atomic counter; nobody waits) adds
// the slots in block order: deterministic, no float atomics.
//
// All mbarrier waits are bounded; a wait that runs out records a time-out in the status
// word, after which every wait of the block returns at once and the block runs to its end
// (its output is then undefined, the status word says so).
#include <mutex>

#include "async_copy.cuh"
#include "common.cuh"

namespace awq {

namespace {

constexpr int kMathWarps = 16;
constexpr int kMathThreads = kMathWarps * 32;
constexpr int kFlushThreads = 64;
constexpr int kGemvThreads = kMathThreads + 32 + kFlushThreads;   // + copy warp, two flush warps
constexpr int kUT = 8;                                 // k-tiles per work unit (512 input channels)
constexpr int kWT = kUT / 2;                           // k-tiles per math warp and stage
constexpr int kWBytes = kUT * kTileBytes;              // 32 KB of packed weights per stage
constexpr int kScaleBytes = kUT * 256;                 // up to kUT groups x 128 rows x fp16
constexpr int kZeroBytes = kUT * 64;                   // up to kUT groups x 64 bytes
constexpr int kXRowBytes = kUT * 128 + 16;             // one token's slice, padded against bank conflicts
constexpr int kXOff = kWBytes + kScaleBytes + kZeroBytes;
constexpr int kZeroRowBytes = 1024;                    // a row of zeros read by lanes without a token
constexpr int kSmemBudget = 200 * 1024;

// Shared-memory layout, computed once on the host and passed to the kernel.
struct GemvLayout {
    int stage_bytes, stages, zero_off, xsum_off, red_off, bar_off, total;
};
inline GemvLayout gemv_layout(int M, int K, int group) {
    GemvLayout l;
    const int mtok = M <= 8 ? 8 : 16;
    l.stage_bytes = kXOff + ((M * kXRowBytes + 127) / 128) * 128;
    const int red = 2 * (2 * mtok * 128 * 4);            // two buffers of [k-half][token][row] fp32
    const int xsum = (K / group) * mtok * 4;             // [group][token] fp32 sums of x
    int s = (kSmemBudget - red - xsum - kZeroRowBytes - 256) / l.stage_bytes;
    l.stages = s > 8 ? 8 : s;
    l.zero_off = l.stages * l.stage_bytes;
    l.xsum_off = l.zero_off + kZeroRowBytes;
    l.red_off = l.xsum_off + xsum;
    l.bar_off = l.red_off + red;
    l.total = l.bar_off + 256;
    return l;
}

__device__ __forceinline__ void mma_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                          uint32_t a3, uint32_t b0, uint32_t b1) {
    asm(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// the same product starting a new accumulation (C = 0)
__device__ __forceinline__ void mma_16816_first(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                                uint32_t a3, uint32_t b0, uint32_t b1) {
    asm(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
        : "=f"(c[0]), "=f"(c[1]), "=f"(c[2]), "=f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(0.0f));
}
// Work decomposition shared by the producer and the math warps.
struct Range {
    int ups;        // units per slab
    int U;          // units in total
    int P;          // blocks
    // U * P < 2^31 for every accepted shape (U <= 1024 slabs * 64 units, P <= 256 blocks)
    __device__ __forceinline__ int start(int c) const { return (int)(((unsigned)U * (unsigned)c) / (unsigned)P); }
    __device__ __forceinline__ int block_of(int u) const {
        return (int)((((unsigned)u + 1u) * (unsigned)P - 1u) / (unsigned)U);
    }
};

// One math warp's share of one stage: NT tiles (4, or 2 for a ragged last unit of a slab).
// The accumulation chains are independent (one or two per tile), and the activations are
// fetched 8 bytes at a time right before the product that uses them.
template <int G, int MT, int NT>
__device__ __forceinline__ void math_stage(const unsigned char* st, const unsigned char* const (&xp)[MT],
                                           int w_off, int sc_off, int z_off, const float* xs,
                                           float (&acc)[MT][4]) {
    constexpr int TPG = G / 64, NG = NT / TPG, NCH = (MT == 1) ? 2 : 1;
    // all shared-memory reads of the stage first, then one straight run of logic + MMA work
    uint4 pk[NT];
    uint4 xv[MT][NT][2];
#pragma unroll
    for (int tile = 0; tile < NT; ++tile)
        pk[tile] = *reinterpret_cast<const uint4*>(st + w_off + tile * kTileBytes);
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int tile = 0; tile < NT; ++tile) {
            xv[mt][tile][0] = *reinterpret_cast<const uint4*>(xp[mt] + tile * 128);
            xv[mt][tile][1] = *reinterpret_cast<const uint4*>(xp[mt] + tile * 128 + 16);
        }
    // group parameters, folded with the power-of-two scales of the subnormal codes
    float su[NG], sl[NG], zu[NG], zl[NG];
#pragma unroll
    for (int q = 0; q < NG; ++q) {
        const float d_up = __half2float(*reinterpret_cast<const __half*>(st + sc_off + q * 256));
        const float d_lo = __half2float(*reinterpret_cast<const __half*>(st + sc_off + q * 256 + 16));
        const uint32_t zb = st[z_off + q * 64];
        su[q] = d_up * 16777216.0f;
        sl[q] = d_lo * 1048576.0f;
        zu[q] = -d_up * (float)(zb & 0xFu);
        zl[q] = -d_lo * (float)(zb >> 4);
    }
    float c[NT][MT][NCH][4];
#pragma unroll
    for (int jw = 0; jw < 4; ++jw) {
#pragma unroll
        for (int tile = 0; tile < NT; ++tile) {
            // codes as fp16 subnormals: q * 2^-24 (upper row), q * 2^-20 (lower row)
            const uint32_t w = (jw == 0) ? pk[tile].x : (jw == 1) ? pk[tile].y : (jw == 2) ? pk[tile].z : pk[tile].w;
            const uint32_t w8 = w >> 8;
            const uint32_t a0 = w & 0x000F000Fu, a1 = w & 0x00F000F0u;
            const uint32_t a2 = w8 & 0x000F000Fu, a3 = w8 & 0x00F000F0u;
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
                const uint4 xq = xv[mt][tile][jw >> 1];
                const uint32_t b0 = (jw & 1) ? xq.z : xq.x, b1 = (jw & 1) ? xq.w : xq.y;
                if (jw < NCH) mma_16816_first(c[tile][mt][jw % NCH], a0, a1, a2, a3, b0, b1);
                else mma_16816(c[tile][mt][jw % NCH], a0, a1, a2, a3, b0, b1);
            }
        }
    }
    // per group: sum (q - z) x = 2^24 * D - z * X (upper row; 2^20 for the lower row), times Delta
#pragma unroll
    for (int q = 0; q < NG; ++q) {
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
            const float2 X = *reinterpret_cast<const float2*>(xs + q * (MT * 8) + mt * 8);
            float d[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
            for (int v = 0; v < TPG; ++v)
#pragma unroll
                for (int ch = 0; ch < NCH; ++ch)
#pragma unroll
                    for (int i = 0; i < 4; ++i) d[i] += c[q * TPG + v][mt][ch][i];
            acc[mt][0] = fmaf(su[q], d[0], fmaf(zu[q], X.x, acc[mt][0]));
            acc[mt][1] = fmaf(su[q], d[1], fmaf(zu[q], X.y, acc[mt][1]));
            acc[mt][2] = fmaf(sl[q], d[2], fmaf(zl[q], X.x, acc[mt][2]));
            acc[mt][3] = fmaf(sl[q], d[3], fmaf(zl[q], X.y, acc[mt][3]));
        }
    }
}

#ifdef AWQ_DBG_TS
__device__ unsigned long long g_dbg_ts[256 * 16];
#define DBG_TS(i) do { if (threadIdx.x == 0) g_dbg_ts[blockIdx.x * 16 + (i)] = global_ns(); } while (0)
#define DBG_TS_ANY(i) do { g_dbg_ts[blockIdx.x * 16 + (i)] = global_ns(); } while (0)
#define DBG_CLK(v) const long long v = clock64()
#define DBG_ACC(i, a, b) do { dbg_acc[i] += (b) - (a); } while (0)
#define DBG_ACC_DECL long long dbg_acc[4] = {0, 0, 0, 0}
#define DBG_ACC_STORE(base) do { for (int _i = 0; _i < 4; ++_i) g_dbg_ts[blockIdx.x * 16 + (base) + _i] = (unsigned long long)dbg_acc[_i]; } while (0)
#else
#define DBG_CLK(v) do {} while (0)
#define DBG_ACC(i, a, b) do {} while (0)
#define DBG_ACC_DECL do {} while (0)
#define DBG_ACC_STORE(base) do {} while (0)
#define DBG_TS(i) do {} while (0)
#define DBG_TS_ANY(i) do {} while (0)
#endif

// MT = number of 8-token column tiles (1: M <= 8, 2: M <= 16).
template <int G, int MT>
__global__ void __launch_bounds__(kGemvThreads, 1)
gemv_kernel(const unsigned char* __restrict__ qweight, const __half* __restrict__ scales,
            const unsigned char* __restrict__ zeros, const __half* __restrict__ x,
            __half* __restrict__ y, float* __restrict__ partial, unsigned int* __restrict__ counters,
            int M, int N, int K, const GemvLayout lay, unsigned int* status_word) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ unsigned int s_abort;
    __shared__ unsigned int s_last;

    DBG_TS(0);
    const int S = lay.stages;
    const uint32_t sbase = smem_u32(smem);
    // barriers: full[s] at 8s (copies landed), empty[s] at 64 + 8s (math warps done)
    const uint32_t bars = sbase + (uint32_t)lay.bar_off;

    const int ktiles = K / 64;
    Range rg;
    rg.ups = (ktiles + kUT - 1) / kUT;
    rg.U = (N / 128) * rg.ups;
    rg.P = gridDim.x;
    const int u0 = rg.start(blockIdx.x), u1 = rg.start(blockIdx.x + 1);
    const int slab0 = u0 / rg.ups;
    // Visiting order: the block's last slab segment first (it is the one most likely shared
    // with the next block, so its cross-block sum is out of the way early), then the rest in
    // natural order.  Position p -> unit u.
    const int nu = u1 - u0;
    const int ul = max(u0, ((u1 - 1) / rg.ups) * rg.ups);     // first unit of the last segment
    const int nl = (ul == u0) ? 0 : u1 - ul;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;
    // barriers also at 192 + 8b: flush_req[b] (math warps handed over buffer b) and
    // 208 + 8b: red_free[b] (flush warps are done with buffer b)
    if (threadIdx.x < (unsigned)S) {
        mbar_init(bars + 8u * threadIdx.x, 1);
        mbar_init(bars + 64u + 8u * threadIdx.x, kMathWarps);
        mbar_fence_init();
    } else if (threadIdx.x >= 32 && threadIdx.x < 34) {
        mbar_init(bars + 192u + 8u * (threadIdx.x - 32), kMathWarps);
        mbar_init(bars + 208u + 8u * (threadIdx.x - 32), 1);
        mbar_fence_init();
        if (threadIdx.x == 32) s_abort = 0u;
    }
    if (threadIdx.x < kZeroRowBytes / 4) reinterpret_cast<uint32_t*>(smem + lay.zero_off)[threadIdx.x] = 0u;
    __syncthreads();
    DBG_TS(1);
    const WaitCtl ctl{status_word, &s_abort};
    const unsigned char* zero_row = smem + lay.zero_off;

    if (warp == kMathWarps) {
        // ------------------------------------------------------------------ copy warp
        // lane 0 posts the byte count, then lanes 0 .. 2+M-1 each issue one bulk copy
        // (weights, scales, zero points, one x row per token)
        {
            DBG_ACC_DECL;
            uint32_t stage = 0, phase = 0;
            const int ng = K / G;
            for (int p = 0; p < nu; ++p) {
                const int u = (p < nl) ? ul + p : u0 + (p - nl);
                const int slab = u / rg.ups, j = u - slab * rg.ups;
                const int kt = j * kUT;
                const int nt = min(kUT, ktiles - kt);
                const int ngr = nt * 64 / G;
                const uint32_t dst = sbase + stage * (uint32_t)lay.stage_bytes;
                const uint32_t bar = bars + 8u * stage;
                if (lane == 0) {
                    DBG_CLK(tc0);
                    mbar_wait(bars + 64u + 8u * stage, phase ^ 1u, ctl);
                    DBG_CLK(tc1);
                    DBG_ACC(0, tc0, tc1);
                    mbar_arrive_expect_tx(bar, (uint32_t)(nt * kTileBytes + ngr * (256 + 64) + M * nt * 128));
                }
                __syncwarp();
                const size_t sg = (size_t)slab * ng + (size_t)(kt * 64 / G);
                if (lane == 0)
                    bulk_load(dst, qweight + ((size_t)slab * ktiles + kt) * kTileBytes, (uint32_t)(nt * kTileBytes), bar);
                else if (lane == 1)
                    bulk_load(dst + kWBytes, scales + sg * 128, (uint32_t)(ngr * 256), bar);
                else if (lane == 2)
                    bulk_load(dst + kWBytes + kScaleBytes, zeros + sg * 64, (uint32_t)(ngr * 64), bar);
                else if (lane - 3 < M)
                    bulk_load(dst + kXOff + (lane - 3) * kXRowBytes, x + (size_t)(lane - 3) * K + (size_t)kt * 64,
                              (uint32_t)(nt * 128), bar);
                if (++stage == (uint32_t)S) { stage = 0; phase ^= 1u; }
            }
            if (lane != 0) return;
            DBG_ACC_STORE(9);   // [9] = copy warp cycles waiting for an empty stage
            // every copy issued above must have landed before the block may exit
            const int issued = nu;
            const int pending = issued < S ? issued : S;
            for (int i = 0; i < pending; ++i) {
                if (stage == 0) { stage = S - 1; phase ^= 1u; } else { --stage; }
                const unsigned long long t0 = global_ns();
                while (!mbar_try_wait(bars + 8u * stage, phase) && global_ns() - t0 < 200000000ull) {}
            }
        }
        return;
    }

    constexpr int MTOK = MT * 8;
    constexpr int TPG = G / 64;                        // tiles per group

    // ---------------------------------------------------------- x sums (all but the copy warp)
    // X[group][token] = sum of x over the group's input channels, in fp32, one warp per sum.
    {
        float* xsum = reinterpret_cast<float*>(smem + lay.xsum_off);
        const int w = warp < kMathWarps ? warp : warp - 1;          // 0 .. 17
        constexpr int NW = kMathWarps + kFlushThreads / 32;
        constexpr int LPS = G / 4;                                  // lanes per sum, 4 halfs each
        constexpr int SPW = 32 / LPS;                               // sums per warp and pass
        const int nsum = (K / G) * M;
        const int sub = lane / LPS, l = lane % LPS;
        for (int s0 = w * SPW; s0 < nsum; s0 += NW * SPW) {
            const int sidx = s0 + sub;
            float v = 0.0f;
            if (sidx < nsum) {
                const int gi = sidx / M, m = sidx - gi * M;
                const uint2 h = __ldg(reinterpret_cast<const uint2*>(x + (size_t)m * K + (size_t)gi * G) + l);
                const float2 f0 = __half22float2(*reinterpret_cast<const __half2*>(&h.x));
                const float2 f1 = __half22float2(*reinterpret_cast<const __half2*>(&h.y));
                v = (f0.x + f0.y) + (f1.x + f1.y);
            }
#pragma unroll
            for (int off = LPS / 2; off >= 1; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
            if (l == 0 && sidx < nsum) {
                const int gi = sidx / M, m = sidx - gi * M;
                xsum[gi * MTOK + m] = v;
            }
        }
        named_barrier_sync(3, kGemvThreads - 32);
    }

    if (warp >= kMathWarps + 1) {
        // --------------------------------------------------------------- flush warps
        const int ft = threadIdx.x - (kMathThreads + 32);          // 0 .. kFlushThreads-1
        const float* red = reinterpret_cast<const float*>(smem + lay.red_off);
        int nflush = 0;
        for (int p = 0; p < nu; ++p) {
            const int u = (p < nl) ? ul + p : u0 + (p - nl);
            const int slab = u / rg.ups, j = u - slab * rg.ups;
            if (j == rg.ups - 1 || u == u1 - 1) {
                const bool whole = (u - j >= u0) && (j == rg.ups - 1);
                const uint32_t b = (uint32_t)nflush & 1u, use = ((uint32_t)nflush >> 1) & 1u;
                if (ft == 0) DBG_TS_ANY(3 + 2 * min(nflush, 5));
                mbar_wait(bars + 192u + 8u * b, use, ctl);
                const float* rb = red + b * (2 * MTOK * 128);
                const int slot = (slab == slab0) ? 0 : 1;
                float* mine = partial + (size_t)(blockIdx.x * 2 + slot) * M * 128;
                for (int idx = ft; idx < M * 128; idx += kFlushThreads) {
                    const int m = idx >> 7, r = idx & 127;
                    const float v = rb[m * 128 + r] + rb[(MTOK + m) * 128 + r];
                    if (whole) y[(size_t)m * N + slab * 128 + r] = __float2half_rn(v);
                    else __stcg(mine + idx, v);
                }
                named_barrier_sync(2, kFlushThreads);               // red[b] has been read
                if (ft == 0) mbar_arrive(bars + 208u + 8u * b);
                if (!whole) {
                    const int c_first = rg.block_of(slab * rg.ups), c_last = rg.block_of(slab * rg.ups + rg.ups - 1);
                    if (ft == 0) {
                        __threadfence();                            // cumulative over the barrier above
                        const unsigned int prev = atomicAdd(counters + slab, 1u);
                        s_last = (prev == (unsigned int)(c_last - c_first)) ? 1u : 0u;
                    }
                    named_barrier_sync(2, kFlushThreads);
                    if (s_last != 0u) {
                        __threadfence();
                        for (int idx = ft; idx < M * 128; idx += kFlushThreads) {
                            const int m = idx >> 7, r = idx & 127;
                            float sum = 0.0f;
                            for (int c = c_first; c <= c_last; ++c) {
                                const int cslot = (rg.start(c) / rg.ups == slab) ? 0 : 1;
                                sum += __ldcg(partial + (size_t)(c * 2 + cslot) * M * 128 + idx);
                            }
                            y[(size_t)m * N + slab * 128 + r] = __float2half_rn(sum);
                        }
                        if (ft == 0) counters[slab] = 0u;           // ready for the next call
                    }
                    named_barrier_sync(2, kFlushThreads);           // s_last may be rewritten
                }
                if (ft == 0) DBG_TS_ANY(4 + 2 * min(nflush, 5));
                ++nflush;
            }
        }
        if (ft == 0) DBG_TS_ANY(15);
        return;
    }

    // -------------------------------------------------------------------- math warps
    // warp = (half, band): tiles kWT*half .. +kWT-1 of each stage, rows 16*band .. +15
    const int half = warp >> 3, band = warp & 7;
    constexpr int GPW = kWT * 64 / G;                  // groups per warp and stage
    float* red = reinterpret_cast<float*>(smem + lay.red_off);

    // stage-relative byte offsets of this lane's pieces
    const int w_off = (kWT * half) * kTileBytes + band * 512 + lane * 16;
    const int sc_off = kWBytes + ((GPW * half) * 128 + band * 16 + g) * 2;
    const int z_off = kWBytes + kScaleBytes + (GPW * half) * 64 + band * 8 + g;
    const float* xsum = reinterpret_cast<const float*>(smem + lay.xsum_off);
    int x_off[MT];
    bool tok_ok[MT];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
        tok_ok[mt] = (mt * 8 + g) < M;
        x_off[mt] = kXOff + (mt * 8 + g) * kXRowBytes + (kWT * half) * 128 + t * 32;
    }

    float acc[MT][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[mt][i] = 0.0f;

    uint32_t stage = 0, phase = 0;
    int nflush = 0;
    DBG_ACC_DECL;
    for (int p = 0; p < nu; ++p) {
        const int u = (p < nl) ? ul + p : u0 + (p - nl);
        const int slab = u / rg.ups, j = u - slab * rg.ups;
        const int ntw = min(kUT, ktiles - j * kUT) - kWT * half;      // tiles of this warp: <= 0, 2 or 4
        DBG_CLK(tm0);
        mbar_wait(bars + 8u * stage, phase, ctl);
        DBG_CLK(tm1);
        DBG_ACC(0, tm0, tm1);
        if (p == 0) DBG_TS(2);
        const unsigned char* st = smem + (size_t)stage * lay.stage_bytes;
        const unsigned char* xp[MT];
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) xp[mt] = tok_ok[mt] ? st + x_off[mt] : zero_row;
        // this warp's first group of the unit, and its tokens 2t, 2t+1 (+ 8 per column tile)
        const float* xs = xsum + ((j * kUT + kWT * half) * 64 / G) * MTOK + 2 * t;
        if (ntw >= kWT) math_stage<G, MT, kWT>(st, xp, w_off, sc_off, z_off, xs, acc);
        else if (ntw >= 2) math_stage<G, MT, 2>(st, xp, w_off, sc_off, z_off, xs, acc);
        DBG_CLK(tm3);
        DBG_ACC(1, tm1, tm3);
        __syncwarp();
        if (lane == 0) mbar_arrive(bars + 64u + 8u * stage);
        if (++stage == (uint32_t)S) { stage = 0; phase ^= 1u; }
        DBG_CLK(tm4);
        DBG_ACC(3, tm3, tm4);

        if (j == rg.ups - 1 || u == u1 - 1) {
            // end of this block's segment of the slab: hand the sums to the flush warps
            const uint32_t b = (uint32_t)nflush & 1u, use = ((uint32_t)nflush >> 1) & 1u;
            mbar_wait(bars + 208u + 8u * b, use ^ 1u, ctl);
            float* rb = red + b * (2 * MTOK * 128);
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int m = mt * 8 + 2 * t + (i & 1), r = band * 16 + g + (i >> 1) * 8;
                    rb[(half * MTOK + m) * 128 + r] = acc[mt][i];
                    acc[mt][i] = 0.0f;
                }
            __syncwarp();
            if (lane == 0) mbar_arrive(bars + 192u + 8u * b);
            ++nflush;
        }
    }
    DBG_TS(14);
    if (threadIdx.x == 0) DBG_ACC_STORE(10);   // [10..13] math warp 0: full wait, mma, ready wait, finalize
}

}  // namespace

#ifdef AWQ_DBG_TS
extern "C" __attribute__((visibility("default"))) int awq_dbg_read_ts(unsigned long long* dst) {
    return (int)cudaMemcpyFromSymbol(dst, g_dbg_ts, sizeof(g_dbg_ts));
}
#endif

GemvPlan gemv_plan(int M, int N, int K, int group) {
    (void)group; (void)N; (void)K;
    GemvPlan p;
    p.max_blocks = kGemvMaxBlocks;
    p.workspace_bytes = kCounterBytes + (size_t)kGemvMaxBlocks * 2 * M * 128 * sizeof(float);
    return p;
}

// Built-in scratch of awq_linear_gemv_static: arrival counters followed by the partial-sum
// slots of up to kStaticMaxM tokens.  Every GPU that loads the library holds it until exit.
constexpr int kStaticMaxM = 8;
constexpr size_t kStaticScratchBytes = kCounterBytes + (size_t)kGemvMaxBlocks * 2 * kStaticMaxM * 128 * sizeof(float);
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

int gemv_static_max_m() { return kStaticMaxM; }

// Device address of the built-in scratch on the current device, looked up once per device
// (in host code the array's name is only a handle; kernels need the address from the runtime).
cudaError_t gemv_static_scratch(void** out) {
    static void* s_ptr[64] = {};
    static std::mutex s_mutex;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(s_mutex);
    if (!s_ptr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return e;
        s_ptr[dev] = p;
    }
    *out = s_ptr[dev];
    return cudaSuccess;
}

cudaError_t launch_gemv(const void* x, const void* qweight, const void* scales, const void* zeros,
                        void* y, int M, int N, int K, int group, void* workspace,
                        unsigned int* status_word, int sms, cudaStream_t st) {
    const int ktiles = K / 64;
    const int units = (N / 128) * ((ktiles + kUT - 1) / kUT);
    int blocks = sms < kGemvMaxBlocks ? sms : kGemvMaxBlocks;
    if (units < blocks) blocks = units;
    {
        // Prefer a slightly smaller grid whose equal shares line up with slab boundaries
        // (every block then ends exactly one segment, and fewer partial sums are exchanged).
        const int ups = (ktiles + kUT - 1) / kUT;
        for (int b = blocks; b * 20 >= blocks * 17; --b) {
            if (units % b != 0) continue;
            const int share = units / b;
            if (share % ups == 0 || ups % share == 0) { blocks = b; break; }
        }
    }
    unsigned int* counters = reinterpret_cast<unsigned int*>(workspace);
    float* partial = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(workspace) + kCounterBytes);
    const GemvLayout lay = gemv_layout(M, K, group);
    if (lay.stages < 2) return cudaErrorInvalidValue;      // K too large for the x-sum table
    cudaError_t e = cudaSuccess;
#define AWQ_GEMV_LAUNCH(GG, MTT)                                                                     \
    do {                                                                                             \
        static bool attr_done[64] = {};                                                              \
        int dev = 0;                                                                                 \
        cudaGetDevice(&dev);                                                                         \
        if (!attr_done[dev & 63]) {                                                                  \
            e = cudaFuncSetAttribute(gemv_kernel<GG, MTT>, cudaFuncAttributeMaxDynamicSharedMemorySize, \
                                     kSmemBudget);                                                   \
            if (e != cudaSuccess) return e;                                                          \
            attr_done[dev & 63] = true;                                                              \
        }                                                                                            \
        gemv_kernel<GG, MTT><<<blocks, kGemvThreads, lay.total, st>>>(                               \
            reinterpret_cast<const unsigned char*>(qweight), reinterpret_cast<const __half*>(scales), \
            reinterpret_cast<const unsigned char*>(zeros), reinterpret_cast<const __half*>(x),       \
            reinterpret_cast<__half*>(y), partial, counters, M, N, K, lay, status_word);                  \
    } while (0)
    if (group == 128) { if (M <= 8) AWQ_GEMV_LAUNCH(128, 1); else AWQ_GEMV_LAUNCH(128, 2); }
    else              { if (M <= 8) AWQ_GEMV_LAUNCH(64, 1);  else AWQ_GEMV_LAUNCH(64, 2); }
#undef AWQ_GEMV_LAUNCH
    count_launch();
    return cudaGetLastError();
}

}  // namespace awq
