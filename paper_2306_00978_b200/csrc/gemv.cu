// Decode path of the layer (Sec. 4.2: fused dequantize + matrix-vector product), M <= 16.
//
// HBM-bound: the packed weights (0.5 byte per weight) are streamed exactly once by persistent
// thread blocks, one per SM.  A copy warp keeps a ring of shared-memory stages full with bulk
// asynchronous copies (packed weights, fp16 scales, zero points and the matching slice of x,
// completion counted in bytes on an mbarrier), so that well over 100 KB per SM is always in
// flight, independent of registers and of what the math warps are doing.
//
// Math (both kernels).  Sixteen math warps.  The 16 bytes a lane reads from a stage are already
// the A fragments of four warp-level m16n8k16 tensor-core products: thanks to the
// w{0,2,4,6,1,3,5,7} nibble order, every byte of a packed word holds the codes of rows g (low
// nibble) and g+8 (high nibble) of one column, and bytes 0 / 2 and 1 / 3 line up with the two
// halves of an fp16x2 register.  A byte in the mantissa bits of an fp16 is the exact subnormal
// (q_g + 16 q_{g+8}) * 2^-24: the upper rows' operands are the bytes as they are (mask 0x00FF00FF,
// or one byte permute for the odd bytes), the lower rows' operands the high nibbles alone (mask
// 0x00F000F0 = 16 q_{g+8} * 2^-24), and the lower rows' sums are taken off the upper rows' once per
// group.  Four integer-pipe operations and one MMA per eight weights - the paper counts a shift, an
// AND and an FMA per single weight; the count matters because integer-pipe instructions dispatch at
// half the fp32 rate and the stage time follows them.  x (up to 8 tokens per product) is the B
// operand, accumulation is fp32.  Zero point and scale are applied once per group in fp32:
//   sum (q - z) x = 2^24 * D - z * X,   X = sum of x over the group's columns,
// where X is the same for every output row, so each block sums it once, in fp32, while its
// first weight stages are in flight.  Nothing is rounded to fp16 before the output.
//
// Two work decompositions:
//   gemv_band_kernel    M <= 8, N/16 not much smaller than the SM count.  A task is one 16-row
//                       band over all of K (contiguous in the band-major weight layout); the 16
//                       math warps split the columns of each stage and their sums meet in
//                       shared memory - no traffic between blocks, no workspace.
//   gemv_splitk_kernel  everything else (M <= 16, small N).  Work units are (128-row slab,
//                       512 columns); each block takes a contiguous range of units, so a slab
//                       can be shared by several blocks: such partial sums go to an fp32
//                       workspace slot owned by the block, and the last block to arrive for the
//                       slab (an atomic counter; nobody waits) adds the slots in block order:
//                       deterministic, no float atomics.
// In both, finished sums are handed through shared memory to separate flush warps, so the math
// warps go straight on to the next stage.
//
// All mbarrier waits are bounded; a wait that runs out records a time-out in the status word,
// after which every wait of the block returns at once and the block runs to its end (its
// output is then undefined, the status word says so).
#include <mutex>

#include "async_copy.cuh"
#include "common.cuh"

namespace awq {

namespace {

constexpr int kMathWarps = 16;
constexpr int kMathThreads = kMathWarps * 32;
constexpr int kZeroRowBytes = 1024;                    // a row of zeros read by lanes without a token
constexpr int kSmemBudget = 216 * 1024;

__device__ __forceinline__ void mma_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                          uint32_t a3, uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// the same product starting a new accumulation (C = 0)
__device__ __forceinline__ void mma_16816_first(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                                uint32_t a3, uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
        : "=f"(c[0]), "=f"(c[1]), "=f"(c[2]), "=f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(0.0f));
}

// One 16-row x 64-column packed block (this lane's 16 bytes `pk`) times the matching 64
// activations of MT*8 tokens (this lane's 4 x 8 bytes per token tile: word j of the piece
// multiplies x[16j + 4t .. +3]):
// c[mt][chain] receive D = sum (q_g + 16 q_{g+8}) * 2^-24 x (rows g: the whole byte is the
// operand, see band_full_stage) and sum q_{g+8} * 2^-20 x (rows g+8); the caller subtracts.
template <int MT, int NCH, bool FIRST = true>
__device__ __forceinline__ void block_mma(const uint4& pk, const uint2 (&xq)[MT][4],
                                          float (&c)[MT][NCH][4]) {
    const uint32_t wds[4] = {pk.x, pk.y, pk.z, pk.w};
#pragma unroll
    for (int jw = 0; jw < 4; ++jw) {
        const uint32_t w = wds[jw], w8 = __byte_perm(w, 0u, 0x4341u);     // bytes 1 and 3 of w
        const uint32_t a0 = w & 0x00FF00FFu, a1 = w & 0x00F000F0u;
        const uint32_t a2 = w8, a3 = w8 & 0x00F000F0u;
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
            const uint32_t b0 = xq[mt][jw].x, b1 = xq[mt][jw].y;
            if (FIRST && jw < NCH) mma_16816_first(c[mt][jw % NCH], a0, a1, a2, a3, b0, b1);
            else mma_16816(c[mt][jw % NCH], a0, a1, a2, a3, b0, b1);
        }
    }
}

// X[k-tile][token] = sum of x over the 64 columns of the k-tile, in fp32.  A warp takes 256
// consecutive activations of one token per item (8 halfs per lane, 8 lanes per k-tile) and
// keeps four items' loads in flight.  Called by `nwarps` warps (index w) of the block.
__device__ __forceinline__ void tile_sums_of_x(const __half* __restrict__ x, float* xsum, int M, int K,
                                               int mtok, int w, int nwarps, int lane) {
    const int cpr = K / 256;                       // whole 256-column chunks per token row
    const int items = M * cpr;
    const float inv_cpr = 1.0f / (float)cpr;
    for (int i0 = w; i0 < items; i0 += 4 * nwarps) {
        uint4 h[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int it = i0 + q * nwarps;
            h[q] = make_uint4(0u, 0u, 0u, 0u);
            if (it < items) {
                const int m = (int)(((float)it + 0.5f) * inv_cpr), c = it - m * cpr;   // items <= 4096: exact
                h[q] = __ldg(reinterpret_cast<const uint4*>(x + (size_t)m * K + (size_t)c * 256) + lane);
            }
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int it = i0 + q * nwarps;
            const uint32_t u[4] = {h[q].x, h[q].y, h[q].z, h[q].w};
            float v = 0.0f;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&u[e]));
                v += f.x + f.y;
            }
#pragma unroll
            for (int off = 4; off >= 1; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
            if ((lane & 7) == 0 && it < items) {
                const int m = (int)(((float)it + 0.5f) * inv_cpr), c = it - m * cpr;
                xsum[(c * 4 + (lane >> 3)) * mtok + m] = v;
            }
        }
    }
    // K is a multiple of 128: a last half chunk of 128 columns (2 k-tiles) may remain
    if ((K & 255) != 0) {
        for (int m = w; m < M; m += nwarps) {
            const uint2 h2 = __ldg(reinterpret_cast<const uint2*>(x + (size_t)m * K + (size_t)cpr * 256) + lane);
            const float2 f0 = __half22float2(*reinterpret_cast<const __half2*>(&h2.x));
            const float2 f1 = __half22float2(*reinterpret_cast<const __half2*>(&h2.y));
            float v = (f0.x + f0.y) + (f1.x + f1.y);
#pragma unroll
            for (int off = 8; off >= 1; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
            if ((lane & 15) == 0) xsum[(cpr * 4 + (lane >> 4)) * mtok + m] = v;
        }
    }
}

// =========================================================================== band kernel
constexpr int kBandThreads = kMathThreads + 96;        // + weight-copy warp + flush warp + x-copy warp

// Stage layout of the band kernel, fixed at compile time by TPW (k-tiles per math warp and
// stage) and the group size, so that every shared-memory read is base + immediate.
// TB: bytes of a packed block (16 rows x 64 columns): 512 for 4-bit codes, 384 for the 3-bit storage.
template <int G, int TPW, int TB = 512> struct BandStage {
    static constexpr int kUT = 16 * TPW;                // k-tiles per stage
    static constexpr int kGroups = kUT * 64 / G;
    static constexpr int kScOff = kUT * TB;             // [group][16] fp16
    static constexpr int kZOff = kScOff + kGroups * 32; // [group][16] bytes (a pair of bands)
    static constexpr int kXOff = kZOff + kGroups * 16;  // [token][kXRow]
    static constexpr int kXRow = kUT * 128 + 16;        // padded against bank conflicts
};

struct BandLayout {
    int stage_bytes, stages, xsum_off, red_off, bar_off, total;
    int red_tokens;                  // tokens per reduction buffer row block: 4 (M <= 4) or 8
    int x_row, xg_off;               // x resident in shared memory: bytes per token row; offset of the
                                     // per-group sums of x, fp32 [K / G][4 tokens], behind the rows
};

// Up to four weight matrices that share x, K and the group size (fused q/k/v or gate/up
// projections): their 16-row bands form one task list for one launch.
struct BandProblems {
    const unsigned char* qweight[kMaxMulti];
    const __half* scales[kMaxMulti];
    const unsigned char* zeros[kMaxMulti];
    __half* y[kMaxMulti];
    int n[kMaxMulti];            // output channels of each matrix
    int first_band[kMaxMulti + 1];
    int count;
};
struct BandRef {                 // one task: matrix, band inside it
    const unsigned char* qweight;
    const __half* scales;
    const unsigned char* zeros;
    __half* y;
    int n, band;
};
__device__ __forceinline__ BandRef band_ref(const BandProblems& pr, int task) {
    int p = 0;
#pragma unroll
    for (int i = 1; i < kMaxMulti; ++i)
        if (i < pr.count && task >= pr.first_band[i]) p = i;
    BandRef r;
    r.qweight = pr.qweight[0]; r.scales = pr.scales[0]; r.zeros = pr.zeros[0]; r.y = pr.y[0]; r.n = pr.n[0];
#pragma unroll
    for (int i = 1; i < kMaxMulti; ++i)
        if (p == i) { r.qweight = pr.qweight[i]; r.scales = pr.scales[i]; r.zeros = pr.zeros[i]; r.y = pr.y[i]; r.n = pr.n[i]; }
    r.band = task - pr.first_band[p];
    return r;
}
template <int G, int TPW, int TB = 512>
inline BandLayout band_layout(int M, int K, bool x_in_registers, bool x_resident = false) {
    using St = BandStage<G, TPW, TB>;
    BandLayout l;
    l.stage_bytes = ((St::kXOff + ((x_in_registers || x_resident) ? 0 : M * St::kXRow) + 127) / 128) * 128;
    // per-k-tile sums of x (+ one stage of slack for ragged reads); with x in registers the region
    // is the math warps' staging block for x instead (16 warps x 512 bytes); with x resident in
    // shared memory it holds the M rows of x (padded against bank conflicts) and the group sums
    l.x_row = K * 2 + 32;
    l.xg_off = ((M * l.x_row + 127) / 128) * 128;
    const int xsum = x_resident ? l.xg_off + (K / G) * 16
                                : (x_in_registers ? kMathWarps * 512 : (K / 64 + St::kUT) * 8 * 4);
    l.red_tokens = M <= 4 ? 4 : 8;
    const int red = 6 * kMathWarps * l.red_tokens * 16 * 4;   // one buffer per stage of [warp][token][row] fp32
    int s = (kSmemBudget - xsum - red - 256 - 128) / l.stage_bytes;
    l.stages = s > 6 ? 6 : s;
    l.xsum_off = l.stages * l.stage_bytes;
    l.red_off = ((l.xsum_off + xsum + 127) / 128) * 128;
    l.bar_off = l.red_off + red;
    l.total = l.bar_off + 256;
    l.xg_off += l.xsum_off;
    return l;
}

// A read-only 16-byte load that stays where it is written (the compiler may otherwise sink a plain
// load below the dependency wait, towards its first use).
__device__ __forceinline__ float4 ld_const_f4(const float* p) {
    float4 v;
    asm volatile("ld.global.nc.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
    return v;
}

// Eight activations times their inverse channel scales: fp16_rne(fp32(x) * inv_s), one fp32
// multiply and one rounding per element (the caller's side of Eq. 4, folded into the fetch of x).
__device__ __forceinline__ uint4 scale8(const uint4& h, const float4& s0, const float4& s1) {
    const float sv[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
    const uint32_t w[4] = {h.x, h.y, h.z, h.w};
    uint32_t o[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w[e]));
        const __half2 r = __floats2half2_rn(__fmul_rn(f.x, sv[2 * e]), __fmul_rn(f.y, sv[2 * e + 1]));
        o[e] = *reinterpret_cast<const uint32_t*>(&r);
    }
    return make_uint4(o[0], o[1], o[2], o[3]);
}

// A lane's packed piece of one block as the four nibble words of the 4-bit layout.  3-bit storage
// (TB = 384): three words per piece, the fourth word's bits ride in the spare top bits of the
// nibbles of the other three.
template <int TB>
__device__ __forceinline__ uint4 load_piece(const unsigned char* p) {
    if constexpr (TB == 512) {
        return *reinterpret_cast<const uint4*>(p);
    } else {
        const uint32_t u0 = *reinterpret_cast<const uint32_t*>(p), u1 = *reinterpret_cast<const uint32_t*>(p + 4),
                       u2 = *reinterpret_cast<const uint32_t*>(p + 8);
        uint4 w;
        w.x = u0 & 0x77777777u;
        w.y = u1 & 0x77777777u;
        w.z = u2 & 0x77777777u;
        w.w = ((u0 >> 3) & 0x11111111u) | ((u1 >> 2) & 0x22222222u) | ((u2 >> 1) & 0x44444444u);
        return w;
    }
}

// One full stage of one math warp: the warp's TPW k-tiles (GPW whole groups) of the band's 16
// rows times x, added to acc.  Straight-line code, one accumulation chain per group, the groups'
// products interleaved word by word so that no MMA waits for the one before it.  Kx / Ky are
// 2^-24 times the sums of x over each group for the lane's two accumulator columns (tokens 2t
// and 2t+1).
template <int G, int TPW, bool ONE, int TB = 512>
__device__ __forceinline__ void band_full_stage(const unsigned char* st, int o_w, int o_sc, int o_z,
                                                const uint2 (&xr)[TPW][4],
                                                const float (&Kx)[(TPW + G / 64 - 1) / (G / 64)],
                                                const float (&Ky)[(TPW + G / 64 - 1) / (G / 64)],
                                                float (&acc)[4]) {
    constexpr int TPG = G / 64;
    constexpr int GPW = (TPW + TPG - 1) / TPG;
    float c[GPW][4];
    uint4 pk[TPW];
#pragma unroll
    for (int v = 0; v < TPW; ++v) pk[v] = load_piece<TB>(st + o_w + v * TB);
#pragma unroll
    for (int v = 0; v < TPG; ++v)
#pragma unroll
        for (int jw = 0; jw < 4; ++jw)
#pragma unroll
            for (int q = 0; q < GPW; ++q) {
                const int tile = q * TPG + v;
                const uint32_t w = (jw == 0) ? pk[tile].x : (jw == 1) ? pk[tile].y : (jw == 2) ? pk[tile].z : pk[tile].w;
                // Integer and logic instructions issue at half the rate of fp32 ones and four masks
                // plus a shift per word were the largest item of the stage, so the upper rows'
                // operands keep their whole byte - the row-g code plus 16 times the row-(g+8) code of
                // the same column, still an exact fp16 subnormal - and the lower rows' share is
                // taken off once per group below; the byte permute replaces shift and mask.
                const uint32_t w8 = __byte_perm(w, 0u, 0x4341u);            // bytes 1 and 3 of w
                const uint32_t bb0 = xr[tile][jw].x, bb1 = xr[tile][jw].y;
                if (v == 0 && jw == 0)
                    mma_16816_first(c[q], w & 0x00FF00FFu, w & 0x00F000F0u, w8, w8 & 0x00F000F0u, bb0, bb1);
                else
                    mma_16816(c[q], w & 0x00FF00FFu, w & 0x00F000F0u, w8, w8 & 0x00F000F0u, bb0, bb1);
            }
    // per group: Delta * (2^24 D - z X); integers below 2^23 become floats without a conversion
    // instruction; the lower rows' codes entered the product 16 times too large (mask 0xF0) and
    // their zero point is read 16 times too large as well, so one factor serves both
#pragma unroll
    for (int q = 0; q < GPW; ++q) {
        const float d_up = __half2float(*reinterpret_cast<const __half*>(st + o_sc + q * 32));
        const float d_lo = __half2float(*reinterpret_cast<const __half*>(st + o_sc + q * 32 + 16));
        const uint32_t zb = st[o_z + q * 16];
        const float z_up = __uint_as_float(0x4B000000u | (zb & 0xFu)) - 8388608.0f;
        const float z_lo16 = __uint_as_float(0x4B000000u | (zb & 0xF0u)) - 8388608.0f;   // 16 * z
        const float su = d_up * 16777216.0f, sl = d_lo * 1048576.0f;
        const float kx = Kx[q];
        // c[q][0] holds sum (q_g + 16 q_{g+8}) x, c[q][2] holds sum 16 q_{g+8} x (both times 2^-24)
        acc[0] = fmaf(su, fmaf(-z_up, kx, c[q][0] - c[q][2]), acc[0]);
        acc[2] = fmaf(sl, fmaf(-z_lo16, kx, c[q][2]), acc[2]);
        if (!ONE) {
            const float ky = Ky[q];
            acc[1] = fmaf(su, fmaf(-z_up, ky, c[q][1] - c[q][3]), acc[1]);
            acc[3] = fmaf(sl, fmaf(-z_lo16, ky, c[q][3]), acc[3]);
        }
    }
}

// TPW = k-tiles per math warp and stage (stage = 16 * TPW k-tiles).  M <= 8 tokens (one token tile).
// ONE: M == 1, the sums of the second token column of each accumulator fragment are not formed.
// XREG: K == 64 * 16 * TPW, i.e. a band is exactly one stage and a math warp meets the same
// k-tiles in every stage: its B fragments of x and its per-group sums of x are loaded once, from
// global memory, and stay in registers; no x travels through the stages.
// XS: 0, or (XREG only) the number of stages of the ring, known at compile time together with
// 4-token reduction rows: the loop over the bands is then unrolled over one turn of the ring and
// every stage, barrier and reduction address is a constant.
// XSM (not with XREG; M <= 4): x stays resident in shared memory for the whole launch instead of
// travelling through the stages slice by slice: each math warp fetches, once, exactly the
// columns it multiplies (the same k-tiles of every stage of every band) and forms their group
// sums, so no x copy, no per-stage x bytes on the barriers and no block-wide barrier is needed.
// sdiv: nullptr, or the inverse channel scales 1 / s (fp32 [K]): x is then multiplied by them while it
// is fetched (XREG and XSM only), fp16_rne(fp32(x) * inv_s), which folds the caller's diag(s)^-1 into
// this kernel.
// TB: 512 (4-bit codes) or 384 (the 3-bit storage, see load_piece).
template <int G, int TPW, bool ONE, bool XREG, int XS, bool XSM = false, int TB = 512>
__global__ void __launch_bounds__(kBandThreads, 1)
gemv_band_kernel(const BandProblems probs, const __half* __restrict__ x, int M, int K,
                 const BandLayout lay, unsigned int* status_word, const float* __restrict__ sdiv) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ unsigned int s_abort;
    using St = BandStage<G, TPW, TB>;
    constexpr int UT = St::kUT;
    constexpr int TPG = G / 64;                         // k-tiles per group
    constexpr int GPW = (TPW + TPG - 1) / TPG;          // groups touched by one warp in a stage
    static_assert(TPW % TPG == 0, "a warp's tiles must cover whole groups");
    static_assert(!(XREG && XSM), "x lives either in registers or in shared memory");
    const int S = lay.stages;
    const uint32_t sbase = smem_u32(smem);
    // barriers: full[s] at 8s, empty[s] at 64 + 8s, flush_req[s] at 128 + 8s
    const uint32_t bars = sbase + (uint32_t)lay.bar_off;

    const int ktiles = K / 64, ng = K / G;
    const int upb = XREG ? 1 : (ktiles + UT - 1) / UT;                // units (stages) per band
    const int nbands = probs.first_band[probs.count];
    // the blocks with one band more are the first ones: blocks start in index order, the last ones
    // on the SMs that the launch in front of this one frees last
    const int bq = nbands / (int)gridDim.x, br = nbands - bq * (int)gridDim.x;
    const int b0 = bq * (int)blockIdx.x + min((int)blockIdx.x, br);
    const int b1 = b0 + bq + ((int)blockIdx.x < br ? 1 : 0);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x < (unsigned)S) {
        mbar_init(bars + 8u * threadIdx.x, 1);                      // full: the copy warp's byte count
        // empty: math warps and the flush warp; with one-stage bands the flush warp alone (it has
        // seen every math warp's flush_req arrival on the same stage)
        mbar_init(bars + 64u + 8u * threadIdx.x, XREG ? 1 : kMathWarps + 1);
        mbar_init(bars + 128u + 8u * threadIdx.x, kMathWarps);      // flush_req: a band's sums are in red[stage]
        mbar_fence_init();
    } else if (threadIdx.x == 32) {
        s_abort = 0u;
    }
    __syncthreads();
    const WaitCtl ctl{status_word, &s_abort};
    // Programmatic dependent launch: the next kernel of the stream may be scheduled onto an SM as
    // soon as this block has left it, and this kernel may itself have started before the one in
    // front of it finished.  Weights, scales and zero points are constants of the layer, so the
    // weight-copy warp starts filling the ring at once; everything that touches x or y first
    // waits for the preceding kernel to complete (griddepcontrol.wait).
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // x may still be unwritten, but its lines can already be pulled into L2 (a hint; L2 stays
    // coherent), so that the loads after the wait below do not go to HBM
    if (warp == kMathWarps + 1) {
        const int lines = (M * K * 2 + 127) / 128;
        for (int i = lane; i < lines; i += 32) prefetch_l2(reinterpret_cast<const unsigned char*>(x) + (size_t)i * 128);
    }

    if (warp == kMathWarps + 2) {
        // ---------------------------------------------------------------- x-copy warp
        // lane m < M copies token m's slice of x for each stage (counted on the stage's barrier)
        if (XREG || XSM) return;
        asm volatile("griddepcontrol.wait;" ::: "memory");
        uint32_t stage = 0, phase = 0;
        for (int task = b0; task < b1; ++task) {
            for (int j = 0; j < upb; ++j) {
                const int kt = j * UT;
                const int nt = min(UT, ktiles - kt);
                if (lane == 0) mbar_wait_relaxed(bars + 64u + 8u * stage, phase ^ 1u, ctl);
                __syncwarp();
                if (lane < M)
                    bulk_load(sbase + stage * (uint32_t)lay.stage_bytes + St::kXOff + lane * St::kXRow,
                              x + (size_t)lane * K + (size_t)kt * 64, (uint32_t)(nt * 128), bars + 8u * stage);
                if (++stage == (uint32_t)S) { stage = 0; phase ^= 1u; }
            }
        }
        return;
    }
    if (warp == kMathWarps) {
        // ------------------------------------------------------------- weight-copy warp
        // lane 0 posts the stage's byte count (x included); lanes 0, 1, 2 each issue one bulk copy
        uint32_t stage = 0, phase = 0;
        const uint64_t once = l2_policy_evict_first();     // every packed byte is read exactly once
        for (int task = b0; task < b1; ++task) {
            const BandRef br = band_ref(probs, task);
            const int band = br.band;
            for (int j = 0; j < upb; ++j) {
                const int kt = j * UT;
                const int nt = min(UT, ktiles - kt);
                const int ngr = nt * 64 / G;
                const uint32_t dst = sbase + stage * (uint32_t)lay.stage_bytes;
                const uint32_t bar = bars + 8u * stage;
                if (lane == 0) {
                    mbar_wait_relaxed(bars + 64u + 8u * stage, phase ^ 1u, ctl);
                    mbar_arrive_expect_tx(bar, (uint32_t)(nt * TB + ngr * 48 + ((XREG || XSM) ? 0 : M * nt * 128)));
                }
                __syncwarp();
                const int gi0 = kt * 64 / G;
                if (lane == 0)
                    bulk_load_hint(dst, br.qweight + ((size_t)band * ktiles + kt) * TB, (uint32_t)(nt * TB), bar, once);
                else if (lane == 1)
                    bulk_load_hint(dst + St::kScOff, br.scales + ((size_t)band * ng + gi0) * 16, (uint32_t)(ngr * 32), bar, once);
                else if (lane == 2)
                    bulk_load(dst + St::kZOff, br.zeros + ((size_t)(band >> 1) * ng + gi0) * 16, (uint32_t)(ngr * 16), bar);
                if (++stage == (uint32_t)S) { stage = 0; phase ^= 1u; }
            }
        }
        if (lane != 0) return;
        // every copy issued above must have landed before the block may exit
        const int issued = (b1 - b0) * upb;
        const int pending = issued < S ? issued : S;
        for (int i = 0; i < pending; ++i) {
            if (stage == 0) { stage = S - 1; phase ^= 1u; } else { --stage; }
            const unsigned long long t0 = global_ns();
            while (!mbar_try_wait(bars + 8u * stage, phase) && global_ns() - t0 < drain_limit_ns(ctl)) {}
        }
        return;
    }

    // the channel scales are constants of the layer like the weights: with x in registers a lane
    // fetches the eight it needs before the dependency wait
    // (x resident in shared memory: the scales of the first batch of stage positions)
    constexpr int JB = ONE ? 4 : 2;                              // stage positions fetched per batch
    float4 sd0 = make_float4(1.0f, 1.0f, 1.0f, 1.0f), sd1 = sd0;
    float4 sa[XSM ? JB : 1], sb[XSM ? JB : 1];
    if (XREG && sdiv != nullptr && warp < kMathWarps) {
        sd0 = ld_const_f4(sdiv + warp * (TPW * 64) + lane * 8);
        sd1 = ld_const_f4(sdiv + warp * (TPW * 64) + lane * 8 + 4);
    }
    if (XSM && warp < kMathWarps) {
#pragma unroll
        for (int jj = 0; jj < JB; ++jj) {
            const int col = (jj * UT + warp * TPW) * 64 + lane * 8;
            sa[jj] = make_float4(1.0f, 1.0f, 1.0f, 1.0f);
            sb[jj] = sa[jj];
            if (sdiv != nullptr && jj < upb && lane * 8 < TPW * 64 && col < K) {
                sa[jj] = ld_const_f4(sdiv + col);
                sb[jj] = ld_const_f4(sdiv + col + 4);
            }
        }
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    float* xsum = reinterpret_cast<float*>(smem + lay.xsum_off);

    float* red = reinterpret_cast<float*>(smem + lay.red_off);
    if (warp == kMathWarps + 1) {
        // ------------------------------------------------------------------ flush warp
        // Walks the stages like a math warp.  The sums of a band wait in the reduction buffer of
        // the band's last stage; the flush warp is one of the arrivals on that stage's "empty"
        // barrier, so the buffer cannot be overwritten before it has been read and the math
        // warps never wait for the flush warp.
        uint32_t stage = 0, phase = 0, req_phase = 0;               // req_phase: one parity bit per stage
        for (int task = b0; task < b1; ++task) {
            const BandRef br = band_ref(probs, task);
            for (int j = 0; j < upb; ++j) {
                if (!XREG && !mbar_wait_relaxed(bars + 8u * stage, phase, ctl)) return;
                if (j == upb - 1) {
                    if (!mbar_wait_relaxed(bars + 128u + 8u * stage, (req_phase >> stage) & 1u, ctl)) return;
                    req_phase ^= 1u << stage;
                    const int rstride = lay.red_tokens * 16;            // floats per warp
                    const float* rb = red + stage * (kMathWarps * rstride);
                    for (int idx = lane; idx < M * 16; idx += 32) {  // idx = token * 16 + row
                        float s0 = 0.0f, s1 = 0.0f, s2 = 0.0f, s3 = 0.0f;
#pragma unroll
                        for (int w = 0; w < kMathWarps; w += 4) {
                            s0 += rb[w * rstride + idx]; s1 += rb[(w + 1) * rstride + idx];
                            s2 += rb[(w + 2) * rstride + idx]; s3 += rb[(w + 3) * rstride + idx];
                        }
                        br.y[(size_t)(idx >> 4) * br.n + br.band * 16 + (idx & 15)] = __float2half_rn((s0 + s1) + (s2 + s3));
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(bars + 64u + 8u * stage);
                if (++stage == (uint32_t)S) { stage = 0; phase ^= 1u; }
            }
        }
        return;
    }

    // -------------------------------------------------------------------- math warps
    // warp w owns k-tiles w*TPW .. w*TPW+TPW-1 of every stage, i.e. GPW whole groups
    const int g = lane >> 2, t = lane & 3;
    const bool tok_ok = g < M;
    // this lane's fixed byte offsets inside a stage
    const int o_w = warp * (TPW * TB) + lane * (TB / 32);
    const int o_sc = St::kScOff + warp * (GPW * 32) + g * 2;
    const int o_x = St::kXOff + g * St::kXRow + warp * (TPW * 128) + t * 8;
    const float* xs_lane = xsum + warp * (TPW * 8) + 2 * t;

    // B fragments: lanes without a token keep zeros for the whole kernel and never touch
    // shared memory (even a broadcast read costs wavefronts on the shared-memory pipe)
    uint2 xr[TPW][4];
#pragma unroll
    for (int v = 0; v < TPW; ++v)
#pragma unroll
        for (int jw = 0; jw < 4; ++jw) xr[v][jw] = make_uint2(0u, 0u);

    if constexpr (XREG) {
        // Each token's slice of x for this warp (TPW k-tiles = 32 lanes x 16 bytes) is fetched with
        // one coalesced 16-byte load per lane - every block asks L2 for the same few lines of x
        // at the same moment, so the number of requests matters - and brought into fragment
        // order through the warp's private 512-byte block of shared memory (the region that holds
        // the sums of x when x travels through the stages; not the reduction buffers: a warp that
        // runs ahead may already be writing its sums there).
        static_assert(TPW == 4, "the staging block holds 32 lanes x 16 bytes per token");
        unsigned char* xst = reinterpret_cast<unsigned char*>(xsum) + warp * 512;
        const uint4* xrow = reinterpret_cast<const uint4*>(x + (size_t)warp * (TPW * 64)) + lane;
#pragma unroll
        for (int m0 = 0; m0 < 8; m0 += 4) {
            if (m0 < M) {
                uint4 row[4];
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    if (m0 + i < M) row[i] = __ldg(xrow + (size_t)(m0 + i) * (K / 8));
                if (sdiv != nullptr) {
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        if (m0 + i < M) row[i] = scale8(row[i], sd0, sd1);
                }
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    if (m0 + i < M) {
                        *reinterpret_cast<uint4*>(xst + lane * 16) = row[i];
                        __syncwarp();
                        if (g == m0 + i) {
#pragma unroll
                            for (int v = 0; v < TPW; ++v)
#pragma unroll
                                for (int jw = 0; jw < 4; ++jw)
                                    xr[v][jw] = *reinterpret_cast<const uint2*>(xst + v * 128 + jw * 32 + t * 8);
                        }
                        __syncwarp();
                    }
                }
            }
        }
    }
    float XxR[GPW] = {}, XyR[GPW] = {};                  // XREG: 2^-24 times this warp's group sums of x
    if (XREG) {
        // the sums of x over this warp's groups (for the zero-point term) come straight from the
        // fragments: 16 values per lane and k-tile, the four lanes of a token, then each lane
        // fetches the two tokens of its accumulator columns
#pragma unroll
        for (int q = 0; q < GPW; ++q) {
            float part = 0.0f;
#pragma unroll
            for (int v = 0; v < TPG; ++v)
#pragma unroll
                for (int jw = 0; jw < 4; ++jw) {
                    const float2 f0 = __half22float2(*reinterpret_cast<const __half2*>(&xr[q * TPG + v][jw].x));
                    const float2 f1 = __half22float2(*reinterpret_cast<const __half2*>(&xr[q * TPG + v][jw].y));
                    part += (f0.x + f0.y) + (f1.x + f1.y);
                }
            part += __shfl_xor_sync(0xFFFFFFFFu, part, 1);
            part += __shfl_xor_sync(0xFFFFFFFFu, part, 2);
            part *= 1.0f / 16777216.0f;                  // the products carry 2^-24 (codes as subnormals)
            XxR[q] = __shfl_sync(0xFFFFFFFFu, part, 8 * t);
            XyR[q] = __shfl_sync(0xFFFFFFFFu, part, 8 * t + 4);
        }
    } else if (XSM) {
        // This warp's columns of x - TPW k-tiles at the same place of every stage of a band - from
        // global memory into the resident rows, scaled by 1 / s on the way if asked, and the sums
        // over each group (G / 8 lanes) into the table (times 2^-24: the products carry that
        // factor).  Nobody else reads these columns, so a warp-level barrier is enough.
        constexpr int LPG = G / 8;                              // lanes per group
        constexpr int MT = ONE ? 1 : 2;                         // the resident form is taken for M <= 2 only
        unsigned char* xb = smem + lay.xsum_off;
        float* xg = reinterpret_cast<float*>(smem + lay.xg_off);
        for (int j0 = 0; j0 < upb; j0 += JB) {
            uint4 v[JB][MT];
#pragma unroll
            for (int jj = 0; jj < JB; ++jj) {
                const int col = ((j0 + jj) * UT + warp * TPW) * 64 + lane * 8;
                const bool valid = j0 + jj < upb && lane * 8 < TPW * 64 && col < K;
                if (j0 > 0 && valid && sdiv != nullptr) {        // (the first batch's scales are there already)
                    sa[jj] = ld_const_f4(sdiv + col);
                    sb[jj] = ld_const_f4(sdiv + col + 4);
                }
#pragma unroll
                for (int m = 0; m < MT; ++m) {
                    v[jj][m] = make_uint4(0u, 0u, 0u, 0u);
                    if (valid && m < M) v[jj][m] = __ldg(reinterpret_cast<const uint4*>(x + (size_t)m * K + col));
                }
            }
#pragma unroll
            for (int jj = 0; jj < JB; ++jj) {
                const int col = ((j0 + jj) * UT + warp * TPW) * 64 + lane * 8;
                const bool valid = j0 + jj < upb && lane * 8 < TPW * 64 && col < K;   // the same for all lanes of a group
                float sum[MT];
#pragma unroll
                for (int m = 0; m < MT; ++m) {
                    if (valid && m < M) {
                        if (sdiv != nullptr) v[jj][m] = scale8(v[jj][m], sa[jj], sb[jj]);
                        *reinterpret_cast<uint4*>(xb + m * lay.x_row + col * 2) = v[jj][m];
                    }
                    const uint32_t u[4] = {v[jj][m].x, v[jj][m].y, v[jj][m].z, v[jj][m].w};
                    sum[m] = 0.0f;
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&u[e]));
                        sum[m] += f.x + f.y;
                    }
#pragma unroll
                    for (int off = LPG / 2; off >= 1; off >>= 1) sum[m] += __shfl_xor_sync(0xFFFFFFFFu, sum[m], off);
                }
                if (valid && (lane & (LPG - 1)) == 0) {
                    float4 o = make_float4(sum[0] * (1.0f / 16777216.0f), 0.0f, 0.0f, 0.0f);
                    if constexpr (!ONE) o.y = sum[1] * (1.0f / 16777216.0f);
                    *reinterpret_cast<float4*>(xg + (col / G) * 4) = o;
                }
            }
        }
        __syncwarp();
    } else {
        // x sums per k-tile (the 16 math warps), while the first stages are in flight.  (Deferring
        // them behind the first stage's products, and polling barriers ahead of use, were both
        // measured slower.)
        tile_sums_of_x(x, xsum, M, K, 8, warp, kMathWarps, lane);
        named_barrier_sync(3, kMathThreads);
    }

    if constexpr (XREG && XS > 0) {
        // ---- a band is one stage and the ring has XS stages: one turn of the ring per outer
        // iteration, all addresses constants of the slot
        constexpr uint32_t SB = ((St::kXOff + 127) / 128) * 128;          // stage bytes (no x part)
        constexpr int RS = 4 * 16;                                         // floats per warp in red[]
        float* const rb0 = red + warp * RS + 2 * t * 16 + g;               // red[stage][warp][token][row]
        const bool store_ok = t < 2;                                       // tokens 0 .. 3
        int o_z = St::kZOff + warp * (GPW * 16) + (b0 & 1) * 8 + g;
        uint32_t phase = 0;
        for (int task = b0;;) {
#pragma unroll
            for (int sl = 0; sl < XS; ++sl) {
                if (task >= b1) return;
                float acc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
                mbar_wait(bars + 8u * sl, phase, ctl);
                band_full_stage<G, TPW, ONE, TB>(smem + sl * SB, o_w, o_sc, o_z, xr, XxR, XyR, acc);
                if (store_ok) {
                    float* rb = rb0 + sl * (kMathWarps * RS);
                    rb[0] = acc[0];
                    rb[8] = acc[2];
                    if (!ONE) { rb[16] = acc[1]; rb[24] = acc[3]; }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(bars + 128u + 8u * sl);         // the flush warp frees the stage
                o_z ^= 8;
                ++task;
            }
            phase ^= 1u;
        }
    }

    if constexpr (XREG) {
        // ---- a band is one stage: one lean loop, every address advanced by increments
        const uint32_t sb = (uint32_t)lay.stage_bytes;
        const int rstride = lay.red_tokens * 16;
        const bool store_ok = 2 * t < lay.red_tokens;
        const unsigned char* st = smem;
        const unsigned char* const st_end = smem + (uint32_t)S * sb;
        float* rb = red + warp * rstride + 2 * t * 16 + g;             // red[stage][warp][token][row]
        uint32_t bar = bars, phase = 0;                                 // full[stage]; flush_req[stage] at + 128
        // odd bands of a matrix use the upper 8 bytes of the pair's zero-point block (every matrix
        // has an even number of bands, so a band's parity inside its matrix is the task's parity)
        int o_z = St::kZOff + warp * (GPW * 16) + (b0 & 1) * 8 + g;
        for (int task = b0; task < b1; ++task) {
            float acc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
            mbar_wait(bar, phase, ctl);
            band_full_stage<G, TPW, ONE, TB>(st, o_w, o_sc, o_z, xr, XxR, XyR, acc);
            if (store_ok) {
                rb[0] = acc[0];
                rb[8] = acc[2];
                if (!ONE) { rb[16] = acc[1]; rb[24] = acc[3]; }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar + 128u);                     // the flush warp frees the stage
            o_z ^= 8;
            st += sb; rb += kMathWarps * rstride; bar += 8u;
            if (st == st_end) { st = smem; rb -= S * (kMathWarps * rstride); bar = bars; phase ^= 1u; }
        }
        return;
    }

    uint32_t stage = 0, phase = 0;
    for (int task = b0; task < b1; ++task) {
        float acc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
        const int o_z = St::kZOff + warp * (GPW * 16) + (task & 1) * 8 + g;
        for (int j = 0; j < upb; ++j) {
            const int nt = min(UT, ktiles - j * UT) - warp * TPW;     // this warp's tiles: <= 0 .. TPW
            mbar_wait(bars + 8u * stage, phase, ctl);
            const unsigned char* st = smem + stage * (uint32_t)lay.stage_bytes;
            const float* xs = xs_lane + j * (UT * 8);
            // x resident: this lane's fragments and its two tokens' group sums at stage position j
            const unsigned char* xres = smem + lay.xsum_off + g * lay.x_row + ((j * UT + warp * TPW) * 64 + t * 4) * 2;
            const float* xgs = reinterpret_cast<const float*>(smem + lay.xg_off) +
                               ((j * UT + warp * TPW) * 64 / G) * 4 + 2 * (t & 1);
            const unsigned char* xfrag = XSM ? xres : st + o_x;
            if (nt >= TPW) {
                if (tok_ok) {
#pragma unroll
                    for (int v = 0; v < TPW; ++v)
#pragma unroll
                        for (int jw = 0; jw < 4; ++jw)
                            xr[v][jw] = *reinterpret_cast<const uint2*>(xfrag + v * 128 + jw * 32);
                }
                float Kx[GPW], Ky[GPW];
#pragma unroll
                for (int q = 0; q < GPW; ++q) {
                    if (XSM) {
                        const float2 X = *reinterpret_cast<const float2*>(xgs + q * 4);
                        Kx[q] = X.x;
                        Ky[q] = X.y;
                        continue;
                    }
                    float Xx = 0.0f, Xy = 0.0f;
#pragma unroll
                    for (int v = 0; v < TPG; ++v) {
                        const float2 X = *reinterpret_cast<const float2*>(xs + (q * TPG + v) * 8);
                        Xx += X.x;
                        Xy += X.y;
                    }
                    Kx[q] = Xx * (1.0f / 16777216.0f);
                    Ky[q] = Xy * (1.0f / 16777216.0f);
                }
                band_full_stage<G, TPW, ONE, TB>(st, o_w, o_sc, o_z, xr, Kx, Ky, acc);
            } else if (nt > 0) {
                // ---- ragged last stage of a band: whole groups only (K % G == 0), one at a time
#pragma unroll
                for (int q = 0; q < GPW; ++q) {
                    if (q * TPG < nt) {
                        float c[1][2][4];
                        float Xx = 0.0f, Xy = 0.0f;
#pragma unroll
                        for (int v = 0; v < TPG; ++v) {
                            const int tile = q * TPG + v;
                            const uint4 pk = load_piece<TB>(st + o_w + tile * TB);
                            uint2 xq[1][4] = {{make_uint2(0u, 0u), make_uint2(0u, 0u), make_uint2(0u, 0u), make_uint2(0u, 0u)}};
                            if (tok_ok) {
#pragma unroll
                                for (int jw = 0; jw < 4; ++jw)
                                    xq[0][jw] = *reinterpret_cast<const uint2*>(xfrag + tile * 128 + jw * 32);
                            }
                            if (XSM) {
                                if (v == 0) {                      // the table holds 2^-24 times the group's sums
                                    const float2 X = *reinterpret_cast<const float2*>(xgs + q * 4);
                                    Xx = X.x * 16777216.0f;
                                    Xy = X.y * 16777216.0f;
                                }
                            } else {
                                const float2 X = *reinterpret_cast<const float2*>(xs + tile * 8);
                                Xx += X.x;
                                Xy += X.y;
                            }
                            if (v == 0) block_mma<1, 2, true>(pk, xq, c);
                            else block_mma<1, 2, false>(pk, xq, c);
                        }
                        const float d_up = __half2float(*reinterpret_cast<const __half*>(st + o_sc + q * 32));
                        const float d_lo = __half2float(*reinterpret_cast<const __half*>(st + o_sc + q * 32 + 16));
                        const uint32_t zb = st[o_z + q * 16];
                        const float su = d_up * 16777216.0f, sl = d_lo * 1048576.0f;
                        const float zu = d_up * (float)(zb & 0xFu), zl = d_lo * (float)(zb >> 4);
                        const float lo_x = c[0][0][2] + c[0][1][2], lo_y = c[0][0][3] + c[0][1][3];
                        acc[0] = fmaf(su, (c[0][0][0] + c[0][1][0]) - lo_x, fmaf(-zu, Xx, acc[0]));
                        acc[1] = fmaf(su, (c[0][0][1] + c[0][1][1]) - lo_y, fmaf(-zu, Xy, acc[1]));
                        acc[2] = fmaf(sl, lo_x, fmaf(-zl, Xx, acc[2]));
                        acc[3] = fmaf(sl, lo_y, fmaf(-zl, Xy, acc[3]));
                    }
                }
            }
            if (j == upb - 1) {
                // the band's sums go to the reduction buffer of its last stage: red[stage][warp][token][row]
                // (only the tokens the buffer has room for: 4 when M <= 4, else all 8 of the fragment)
                const int rstride = lay.red_tokens * 16;
                float* rb = red + stage * (kMathWarps * rstride) + warp * rstride;
                if (2 * t < lay.red_tokens) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        if (ONE && (i & 1)) continue;
                        rb[(2 * t + (i & 1)) * 16 + g + (i >> 1) * 8] = acc[i];
                    }
                }
            }
            __syncwarp();
            if (lane == 0) {
                if (j == upb - 1) mbar_arrive(bars + 128u + 8u * stage);
                mbar_arrive(bars + 64u + 8u * stage);
            }
            if (++stage == (uint32_t)S) { stage = 0; phase ^= 1u; }
        }
    }
}

// ======================================================================== split-K kernel
constexpr int kFlushThreads = 64;
constexpr int kSplitkThreads = kMathThreads + 32 + kFlushThreads;   // + copy warp, two flush warps
constexpr int kUT = 8;                                 // k-tiles per work unit (512 input channels)
constexpr int kWT = kUT / 2;                           // k-tiles per math warp and stage
constexpr int kWBytes = kUT * kTileBytes;              // 32 KB of packed weights per stage: [band][k-tile][512]
constexpr int kScaleBytes = 8 * kUT * 32;              // [band][group][16] fp16
constexpr int kZeroBytes = 4 * kUT * 16;               // [band pair][group][16]
constexpr int kXRowBytes = kUT * 128 + 16;             // one token's slice, padded against bank conflicts
constexpr int kXOff = kWBytes + kScaleBytes + kZeroBytes;

// Shared-memory layout, computed once on the host and passed to the kernel.
struct SplitkLayout {
    int stage_bytes, stages, zero_off, xsum_off, red_off, bar_off, total;
};
inline SplitkLayout splitk_layout(int M, int K) {
    SplitkLayout l;
    const int mtok = M <= 8 ? 8 : 16;
    l.stage_bytes = kXOff + ((M * kXRowBytes + 127) / 128) * 128;
    const int red = 2 * (2 * mtok * 128 * 4);            // two buffers of [k-half][token][row] fp32
    const int xsum = (K / 64) * mtok * 4;                // [k-tile][token] fp32 sums of x
    int s = (kSmemBudget - red - xsum - kZeroRowBytes - 256) / l.stage_bytes;
    l.stages = s > 6 ? 6 : s;
    l.zero_off = l.stages * l.stage_bytes;
    l.xsum_off = l.zero_off + kZeroRowBytes;
    l.red_off = l.xsum_off + xsum;
    l.bar_off = l.red_off + red;
    l.total = l.bar_off + 256;
    return l;
}

// Work decomposition shared by the copy, math and flush warps.
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

// MT = number of 8-token column tiles (1: M <= 8, 2: M <= 16).
template <int G, int MT>
__global__ void __launch_bounds__(kSplitkThreads, 1)
gemv_splitk_kernel(const unsigned char* __restrict__ qweight, const __half* __restrict__ scales,
                   const unsigned char* __restrict__ zeros, const __half* __restrict__ x,
                   __half* __restrict__ y, float* __restrict__ partial, unsigned int* __restrict__ counters,
                   int M, int N, int K, const SplitkLayout lay, unsigned int* status_word, int tx_surplus) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ unsigned int s_abort;
    __shared__ unsigned int s_last;

    const int S = lay.stages;
    const uint32_t sbase = smem_u32(smem);
    // barriers: full[s] at 8s (copies landed), empty[s] at 64 + 8s (math warps done),
    // flush_req[b] at 192 + 8b (math warps handed over buffer b), red_free[b] at 208 + 8b
    const uint32_t bars = sbase + (uint32_t)lay.bar_off;

    const int ktiles = K / 64, ng = K / G;
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
    const WaitCtl ctl{status_word, &s_abort};
    constexpr int MTOK = MT * 8;

    if (warp == kMathWarps) {
        // ------------------------------------------------------------------ copy warp
        // lane 0 posts the byte count; then lanes 0-7 copy the 8 bands' weights, 8-15 their
        // scales, 16-19 the 4 band pairs' zero points, 20-31 the x rows
        uint32_t stage = 0, phase = 0;
        for (int p = 0; p < nu; ++p) {
            const int u = (p < nl) ? ul + p : u0 + (p - nl);
            const int slab = u / rg.ups, j = u - slab * rg.ups;
            const int kt = j * kUT;
            const int nt = min(kUT, ktiles - kt);
            const int ngr = nt * 64 / G;
            const uint32_t dst = sbase + stage * (uint32_t)lay.stage_bytes;
            const uint32_t bar = bars + 8u * stage;
            if (lane == 0) {
                mbar_wait_relaxed(bars + 64u + 8u * stage, phase ^ 1u, ctl);
                // tx_surplus is 0 except in the time-out test, which announces more bytes than the
                // copies below bring so that the stage never completes
                mbar_arrive_expect_tx(bar, (uint32_t)(nt * kTileBytes + ngr * (256 + 64) + M * nt * 128 + tx_surplus));
            }
            __syncwarp();
            const int gi0 = kt * 64 / G;
            if (lane < 8) {
                bulk_load(dst + lane * (kUT * 512), qweight + ((size_t)(slab * 8 + lane) * ktiles + kt) * 512,
                          (uint32_t)(nt * 512), bar);
            } else if (lane < 16) {
                const int b = lane - 8;
                bulk_load(dst + kWBytes + b * (kUT * 32), scales + ((size_t)(slab * 8 + b) * ng + gi0) * 16,
                          (uint32_t)(ngr * 32), bar);
            } else if (lane < 20) {
                const int pr = lane - 16;
                bulk_load(dst + kWBytes + kScaleBytes + pr * (kUT * 16),
                          zeros + ((size_t)(slab * 4 + pr) * ng + gi0) * 16, (uint32_t)(ngr * 16), bar);
            } else {
                for (int m = lane - 20; m < M; m += 12)
                    bulk_load(dst + kXOff + m * kXRowBytes, x + (size_t)m * K + (size_t)kt * 64,
                              (uint32_t)(nt * 128), bar);
            }
            if (++stage == (uint32_t)S) { stage = 0; phase ^= 1u; }
        }
        if (lane != 0) return;
        // every copy issued above must have landed before the block may exit
        const int pending = nu < S ? nu : S;
        for (int i = 0; i < pending; ++i) {
            if (stage == 0) { stage = S - 1; phase ^= 1u; } else { --stage; }
            const unsigned long long t0 = global_ns();
            while (!mbar_try_wait(bars + 8u * stage, phase) && global_ns() - t0 < drain_limit_ns(ctl)) {}
        }
        return;
    }

    // x sums per k-tile (all but the copy warp), while the first stages are in flight
    float* xsum = reinterpret_cast<float*>(smem + lay.xsum_off);
    tile_sums_of_x(x, xsum, M, K, MTOK, warp < kMathWarps ? warp : warp - 1, kMathWarps + 2, lane);
    named_barrier_sync(3, kSplitkThreads - 32);

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
                mbar_wait_relaxed(bars + 192u + 8u * b, use, ctl);
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
                        for (int i0 = ft; i0 < M * 128; i0 += 4 * kFlushThreads) {
                            float sum[4] = {0.0f, 0.0f, 0.0f, 0.0f};
                            for (int c = c_first; c <= c_last; ++c) {
                                const int cslot = (rg.start(c) / rg.ups == slab) ? 0 : 1;
                                const float* src = partial + (size_t)(c * 2 + cslot) * M * 128;
#pragma unroll
                                for (int q = 0; q < 4; ++q) {
                                    const int idx = i0 + q * kFlushThreads;
                                    if (idx < M * 128) sum[q] += __ldcg(src + idx);
                                }
                            }
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                const int idx = i0 + q * kFlushThreads;
                                if (idx < M * 128)
                                    y[(size_t)(idx >> 7) * N + slab * 128 + (idx & 127)] = __float2half_rn(sum[q]);
                            }
                        }
                        if (ft == 0) counters[slab] = 0u;           // ready for the next call
                    }
                    named_barrier_sync(2, kFlushThreads);           // s_last may be rewritten
                }
                ++nflush;
            }
        }
        return;
    }

    // -------------------------------------------------------------------- math warps
    // warp = (half, band): k-tiles kWT*half .. +kWT-1 of each stage, rows 16*band .. +15
    const int half = warp >> 3, band = warp & 7;
    constexpr int TPG = G / 64;
    float* red = reinterpret_cast<float*>(smem + lay.red_off);

    // stage-relative byte offsets of this lane's pieces
    const int w_off = band * (kUT * 512) + (kWT * half) * 512 + lane * 16;
    const int sc_off = kWBytes + band * (kUT * 32) + g * 2;
    const int z_off = kWBytes + kScaleBytes + (band >> 1) * (kUT * 16) + (band & 1) * 8 + g;
    int x_off[MT];
    bool tok_ok[MT];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
        tok_ok[mt] = (mt * 8 + g) < M;
        x_off[mt] = kXOff + (mt * 8 + g) * kXRowBytes + (kWT * half) * 128 + t * 8;
    }

    float acc[MT][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[mt][i] = 0.0f;

    uint32_t stage = 0, phase = 0;
    int nflush = 0;
    for (int p = 0; p < nu; ++p) {
        const int u = (p < nl) ? ul + p : u0 + (p - nl);
        const int slab = u / rg.ups, j = u - slab * rg.ups;
        const int ntw = min(kUT, ktiles - j * kUT) - kWT * half;      // tiles of this warp: <= 0, 2 or 4
        mbar_wait(bars + 8u * stage, phase, ctl);
        const unsigned char* st = smem + (size_t)stage * lay.stage_bytes;
        if (ntw > 0) {
            const unsigned char* xp[MT];
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) xp[mt] = st + x_off[mt];
            // one accumulation per group (TPG k-tiles; K % 128 == 0 makes the warp's tile count a
            // whole number of groups), then scale and zero point once per group
            constexpr int NCH = (MT == 1) ? 2 : 1;
#pragma unroll
            for (int q2 = 0; q2 < kWT / TPG; ++q2) {
                if (q2 * TPG < ntw) {
                    float c[MT][NCH][4];
                    float Xx[MT], Xy[MT];
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt) { Xx[mt] = 0.0f; Xy[mt] = 0.0f; }
#pragma unroll
                    for (int v2 = 0; v2 < TPG; ++v2) {
                        const int v = q2 * TPG + v2;
                        const int tile = kWT * half + v;               // k-tile inside the stage
                        const uint4 pk = *reinterpret_cast<const uint4*>(st + w_off + v * 512);
                        uint2 xq[MT][4];
#pragma unroll
                        for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
                            for (int jw = 0; jw < 4; ++jw) {
                                // lanes without a token must not touch shared memory (see the band kernel)
                                xq[mt][jw] = make_uint2(0u, 0u);
                                if (tok_ok[mt]) xq[mt][jw] = *reinterpret_cast<const uint2*>(xp[mt] + v * 128 + jw * 32);
                            }
                            const float2 X = *reinterpret_cast<const float2*>(
                                xsum + (j * kUT + tile) * MTOK + mt * 8 + 2 * t);
                            Xx[mt] += X.x;
                            Xy[mt] += X.y;
                        }
                        if (v2 == 0) block_mma<MT, NCH, true>(pk, xq, c);
                        else block_mma<MT, NCH, false>(pk, xq, c);
                    }
                    const int q = (kWT * half) / TPG + q2;             // group inside the stage
                    const float d_up = __half2float(*reinterpret_cast<const __half*>(st + sc_off + q * 32));
                    const float d_lo = __half2float(*reinterpret_cast<const __half*>(st + sc_off + q * 32 + 16));
                    const uint32_t zb = st[z_off + q * 16];
                    // integers below 2^23 become floats without a conversion instruction
                    const float z_up = __uint_as_float(0x4B000000u | (zb & 0xFu)) - 8388608.0f;
                    const float z_lo16 = __uint_as_float(0x4B000000u | (zb & 0xF0u)) - 8388608.0f;   // 16 * z
                    const float su = d_up * 16777216.0f, sl = d_lo * 1048576.0f;
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt) {
                        float d[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) d[i] = (NCH == 2) ? c[mt][0][i] + c[mt][NCH - 1][i] : c[mt][0][i];
                        d[0] -= d[2];                         // rows g carried the rows g+8 codes as well
                        d[1] -= d[3];
                        const float kx = Xx[mt] * (1.0f / 16777216.0f), ky = Xy[mt] * (1.0f / 16777216.0f);
                        acc[mt][0] = fmaf(su, fmaf(-z_up, kx, d[0]), acc[mt][0]);
                        acc[mt][1] = fmaf(su, fmaf(-z_up, ky, d[1]), acc[mt][1]);
                        acc[mt][2] = fmaf(sl, fmaf(-z_lo16, kx, d[2]), acc[mt][2]);
                        acc[mt][3] = fmaf(sl, fmaf(-z_lo16, ky, d[3]), acc[mt][3]);
                    }
                }
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(bars + 64u + 8u * stage);
        if (++stage == (uint32_t)S) { stage = 0; phase ^= 1u; }

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
        (void)slab;
    }
}

template <typename Kernel>
cudaError_t allow_big_smem(Kernel kernel, bool (&done)[64]) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (!done[dev & 63]) {
        e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget);
        if (e != cudaSuccess) return e;
        done[dev & 63] = true;
    }
    return cudaSuccess;
}

}  // namespace

bool gemv_uses_band_kernel(int M, int N, int sms) {
    // one 16-row band per task: needs enough bands to occupy the SMs, and few tokens (every
    // band re-reads its slice of x from L2)
    return M <= 8 && (N / 16) * 4 >= sms * 3;
}

size_t gemv_workspace_bytes(int M) {
    return kCounterBytes + (size_t)kGemvMaxBlocks * 2 * M * 128 * sizeof(float);
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

// Whether the band kernel can take x unscaled and fold the multiplication by 1 / s into
// its fetch of x (x in registers, or x resident in shared memory).
bool gemv_band_folds_scale(int M, int K, int group) {
    if (K == 64 * 16 * 4) return true;                          // x in registers, any M <= 8
    // x resident in shared memory: measured faster than x through the stages for one and two
    // tokens (7.7 against 7.9 us on 11008 -> 4096, 23.9 against 24.8 us on 8192 -> 28672 at M = 1),
    // slower for three and four (two k-tiles per warp and stage), so it is built for M <= 2
    if (M > 2) return false;
    const BandLayout l = group == 128 ? band_layout<128, 4>(M, K, false, true) : band_layout<64, 4>(M, K, false, true);
    return l.stages >= 4;
}

cudaError_t launch_gemv_band(const void* x, const GemvMatrix* mats, int count, int M, int K, int group,
                             unsigned int* status_word, int sms, bool serialize, cudaStream_t st,
                             const float* sdiv, int bits) {
    BandProblems pr;
    pr.count = count;
    int bands = 0;
    for (int i = 0; i < kMaxMulti; ++i) {
        const GemvMatrix& m = mats[i < count ? i : 0];
        pr.qweight[i] = reinterpret_cast<const unsigned char*>(m.qweight);
        pr.scales[i] = reinterpret_cast<const __half*>(m.scales);
        pr.zeros[i] = reinterpret_cast<const unsigned char*>(m.zeros);
        pr.y[i] = reinterpret_cast<__half*>(m.y);
        pr.n[i] = m.n;
        pr.first_band[i] = bands;
        if (i < count) bands += m.n / 16;
    }
    pr.first_band[kMaxMulti] = bands;
    for (int i = count; i <= kMaxMulti; ++i) pr.first_band[i] = bands;
    const int blocks = bands < sms ? bands : sms;
    // 64 k-tiles per stage while the stage's x slices stay small (M <= 2) or x lives in registers
    // (K = 4096: a band is one such stage); else 32
    const int tpw = (M <= 2 || K == 64 * 16 * 4) ? 4 : 2;
    cudaError_t e = cudaSuccess;
    // programmatic stream serialization: this launch may begin while the kernel in front of it in
    // the stream is still finishing (see the kernel: it waits before it touches x or y)
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.gridDim = dim3((unsigned)blocks);
    cfg.blockDim = dim3(kBandThreads);
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = serialize ? 0 : 1;
    const __half* xh = reinterpret_cast<const __half*>(x);
#define AWQ_BAND_GO(KERNEL, LAY)                                                                     \
    do {                                                                                             \
        static bool done[64] = {};                                                                   \
        cfg.dynamicSmemBytes = (LAY).total;                                                          \
        e = allow_big_smem(KERNEL, done);                                                            \
        if (e != cudaSuccess) return e;                                                              \
        e = cudaLaunchKernelEx(&cfg, KERNEL, pr, xh, M, K, LAY, status_word, sdiv);                  \
        if (e != cudaSuccess) return e;                                                              \
    } while (0)
#define AWQ_BAND_LAUNCH(GG, TT, ONE1, XR, TBB)                                                       \
    do {                                                                                             \
        const BandLayout lay = band_layout<GG, TT, TBB>(M, K, XR);                                   \
        const BandLayout layr = band_layout<GG, TT, TBB>(M, K, false, true);                         \
        if (XR && lay.stages == (TBB == 512 ? 5 : 6) && lay.red_tokens == 4) {                       \
            AWQ_BAND_GO((gemv_band_kernel<GG, TT, ONE1, XR, (XR ? (TBB == 512 ? 5 : 6) : 0), false, TBB>), lay); \
        } else if (XR) {                                                                             \
            if (lay.stages < 2) return cudaErrorInvalidValue;                                        \
            AWQ_BAND_GO((gemv_band_kernel<GG, TT, ONE1, XR, 0, false, TBB>), lay);                   \
        } else if (M <= 2 && layr.stages >= 4) {                                                     \
            AWQ_BAND_GO((gemv_band_kernel<GG, TT, ONE1, false, 0, !XR, TBB>), layr);                 \
        } else {                                                                                     \
            if (lay.stages < 2) return cudaErrorInvalidValue;  /* K too large for the x-sum table */ \
            if (sdiv != nullptr) return cudaErrorInvalidValue; /* callers ask gemv_band_folds_scale */ \
            AWQ_BAND_GO((gemv_band_kernel<GG, TT, ONE1, false, 0, false, TBB>), lay);                \
        }                                                                                            \
    } while (0)
    const bool xreg = tpw == 4 && K == 64 * 16 * 4;            // a band is exactly one stage
#define AWQ_BAND_PICK(GG, TBB)                                                                       \
    do {                                                                                             \
        if (tpw != 4) AWQ_BAND_LAUNCH(GG, 2, false, false, TBB);                                     \
        else if (M == 1 && xreg) AWQ_BAND_LAUNCH(GG, 4, true, true, TBB);                            \
        else if (M == 1) AWQ_BAND_LAUNCH(GG, 4, true, false, TBB);                                   \
        else if (xreg) AWQ_BAND_LAUNCH(GG, 4, false, true, TBB);                                     \
        else AWQ_BAND_LAUNCH(GG, 4, false, false, TBB);                                              \
    } while (0)
    if (bits == 3) { if (group == 128) AWQ_BAND_PICK(128, 384); else AWQ_BAND_PICK(64, 384); }
    else           { if (group == 128) AWQ_BAND_PICK(128, 512); else AWQ_BAND_PICK(64, 512); }
#undef AWQ_BAND_PICK
#undef AWQ_BAND_LAUNCH
#undef AWQ_BAND_GO
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_gemv_splitk(const void* x, const void* qweight, const void* scales, const void* zeros,
                               void* y, int M, int N, int K, int group, void* workspace,
                               unsigned int* status_word, int sms, cudaStream_t st, int tx_surplus) {
    const int ktiles = K / 64;
    const int ups = (ktiles + kUT - 1) / kUT;
    const int units = (N / 128) * ups;
    int blocks = sms < kGemvMaxBlocks ? sms : kGemvMaxBlocks;
    if (units < blocks) blocks = units;
    // Prefer a slightly smaller grid whose equal shares line up with slab boundaries (every
    // block then ends exactly one segment, and fewer partial sums are exchanged).
    for (int b = blocks; b * 20 >= blocks * 17; --b) {
        if (units % b != 0) continue;
        const int share = units / b;
        if (share % ups == 0 || ups % share == 0) { blocks = b; break; }
    }
    unsigned int* counters = reinterpret_cast<unsigned int*>(workspace);
    float* partial = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(workspace) + kCounterBytes);
    const SplitkLayout lay = splitk_layout(M, K);
    if (lay.stages < 2) return cudaErrorInvalidValue;          // K too large for the x-sum table
    cudaError_t e = cudaSuccess;
#define AWQ_SPLITK_LAUNCH(GG, MTT)                                                                   \
    do {                                                                                             \
        static bool done[64] = {};                                                                   \
        e = allow_big_smem(gemv_splitk_kernel<GG, MTT>, done);                                       \
        if (e != cudaSuccess) return e;                                                              \
        gemv_splitk_kernel<GG, MTT><<<blocks, kSplitkThreads, lay.total, st>>>(                      \
            reinterpret_cast<const unsigned char*>(qweight), reinterpret_cast<const __half*>(scales), \
            reinterpret_cast<const unsigned char*>(zeros), reinterpret_cast<const __half*>(x),       \
            reinterpret_cast<__half*>(y), partial, counters, M, N, K, lay, status_word, tx_surplus); \
    } while (0)
    if (group == 128) { if (M <= 8) AWQ_SPLITK_LAUNCH(128, 1); else AWQ_SPLITK_LAUNCH(128, 2); }
    else              { if (M <= 8) AWQ_SPLITK_LAUNCH(64, 1);  else AWQ_SPLITK_LAUNCH(64, 2); }
#undef AWQ_SPLITK_LAUNCH
    count_launch();
    return cudaGetLastError();
}

}  // namespace awq
