// The layer for a medium number of tokens (9 .. 32), Sec. 4.2's fused dequantize + product where
// it is still a bandwidth problem (4 M FLOP per weight byte against a ridge of about 280).
//
// The tensor-memory kernels pay about 9 us per launch (allocation, first copies, split-K hand-over,
// store drain) and re-read x for every 128-channel tile; the band matrix-vector kernel keeps its
// operands in registers and streams a band as one contiguous run, but every band reads all of x and
// its sixteen warps must add their sums per band.  This kernel keeps the band kernel's arithmetic
// and changes the decomposition:
//   * a work unit is 16 bands (256 output channels) x one chunk of K (1024 input channels); a
//     block takes a contiguous range of units that stay in one chunk as long as possible, so its
//     slice of x (M x 1024) is fetched once per chunk into shared memory, together with the
//     per-group sums of x that the zero-point term needs;
//   * every math warp owns ONE band of the unit: no sums meet between warps, nothing is reduced in
//     shared memory, the accumulators stay in registers for the whole unit;
//   * a stage of the ring is 16 bands x 4 k-tiles = 32 KB of packed weights brought by ONE tensor-map
//     copy (the bands' runs are K * 8 bytes apart in the band-major layout: sixteen bulk copies of
//     2 KB would cost sixteen times the copy engine's per-copy overhead); a unit's scales and zero
//     points come by two more tensor-map copies per unit;
//   * a unit's sums over ONE chunk are partial: they go to an fp32 workspace [chunk][token][channel],
//     and a second, tiny kernel adds the chunks in ascending order and rounds to fp16 once -
//     deterministic, no counters, no fences, no waiting between blocks.
// Every wait is bounded as in the other kernels.
//
// Measured on 8192 -> 28672 at 8 tokens (block start / end times by the global timer, in a working
// copy): 140 blocks with 6 units take 22.4 us each (3.7 us per 128 KB unit, 4.9 TB/s over all SMs
// while they run), the 8 blocks with 7 units 25 us, and the 4 of those whose range crosses into the
// next chunk (a new slice of x) 28.1 us, which is the kernel's 28.4 us.  Two remedies were built,
// bit-exact, and measured no better:
//   * equal shares of STAGES per block instead of units (a cut unit's second part in a slot of its
//     own, a table telling the reduce kernel which units were cut): with all SMs busy to the end
//     every block slows to 25.3 us (the memory system gives this access pattern about 4.7 TB/s), the
//     four crossing blocks still end at 29 us, and the reduce kernel's dependent loads cost 2 us;
//   * the next chunk's slice of x fetched at the start into a second buffer: 31.0 -> 30.1 us here,
//     but 42.8 -> 47.3 us on 28672 -> 8192 at 16 tokens (a fifth of the blocks cross there and
//     start later), 0.2 - 0.6 us slower on the 7B shapes.
// Stages of 32 KB (4 k-tiles per band) instead of 16 KB: 31.7 -> 31.0 us.
#include "tcgen05.cuh"

namespace awq {

namespace {

constexpr int kMidMathWarps = 16;
constexpr int kMidThreads = (kMidMathWarps + 1) * 32;   // + producer warp
constexpr int kMidSmem = 220 * 1024;
constexpr int kMidChunkTiles = 16;                       // k-tiles (64 columns) per chunk: 16, or 8 where that fills the SMs better
constexpr int kMidStageTiles = 4;                        // k-tiles per stage and band
constexpr int kMidStageBytes = kMidMathWarps * kMidStageTiles * 512;
constexpr int kMidStages = 4;

// the same product starting a new accumulation (C = 0)
__device__ __forceinline__ void mid_mma_first(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                              uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
        : "=f"(c[0]), "=f"(c[1]), "=f"(c[2]), "=f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(0.0f));
}
__device__ __forceinline__ void mid_mma(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                        uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

struct MidLayout {
    int mtok;            // M rounded up to a multiple of 8 (whole B fragments)
    int x_off, x_row;    // x slice [mtok][x_row bytes]
    int xg_off;          // fp32 [groups of the chunk][mtok]: 2^-24 times the sums of x
    int par_off;         // two buffers of a unit's parameters: scales [16 bands][groups][16] fp16, then
    int par_bytes;       //   zero points [8 band pairs][groups][16] bytes
    int z_in_par;        // offset of the zero points inside a parameter buffer
    int bar_off, total;
};

inline MidLayout mid_layout(int M, int group, int chunk_tiles = kMidChunkTiles) {
    MidLayout l;
    l.mtok = ((M + 7) / 8) * 8;
    const int groups = chunk_tiles * 64 / group;
    l.x_off = kMidStages * kMidStageBytes;
    l.x_row = chunk_tiles * 128 + 32;
    l.xg_off = l.x_off + ((l.mtok * l.x_row + 127) / 128) * 128;
    l.par_off = l.xg_off + ((groups * l.mtok * 4 + 127) / 128) * 128;
    l.z_in_par = kMidMathWarps * groups * 32;
    l.par_bytes = l.z_in_par + (kMidMathWarps / 2) * groups * 16;
    l.bar_off = l.par_off + 2 * l.par_bytes;
    l.total = l.bar_off + 256;
    return l;
}

// MT = 8-token B fragments per product (tokens rounded up to 8 MT); CT = k-tiles per chunk.
template <int G, int MT, int CT>
__global__ void __launch_bounds__(kMidThreads, 1)
gemv_mid_kernel(const __grid_constant__ CUtensorMap w_map, const __grid_constant__ CUtensorMap sc_map,
                const __grid_constant__ CUtensorMap z_map, const __half* __restrict__ x,
                float* __restrict__ partial, int M, int N, int K, const MidLayout lay,
                const __grid_constant__ UnitStarts starts, unsigned int* status_word) {
    extern __shared__ __align__(1024) unsigned char smem[];
    __shared__ unsigned int s_abort;
    constexpr int TPG = G / 64;                          // k-tiles per group
    constexpr int GPC = CT / TPG;                        // groups per chunk
    constexpr int S = kMidStages;
    const uint32_t sbase = smem_u32(smem);
    // barriers: full[s] at 8s, empty[s] at 64 + 8s, par_full[b] at 128 + 8b, par_empty[b] at 160 + 8b
    const uint32_t bars = sbase + (uint32_t)lay.bar_off;
    const int ktiles = K / 64, nbands = N / 16;
    const int nbg = (nbands + kMidMathWarps - 1) / kMidMathWarps;
    const int nchunks = (ktiles + CT - 1) / CT;
    const int units = nchunks * nbg;
    const int u0 = starts.v[blockIdx.x], u1 = starts.v[blockIdx.x + 1];
    (void)units;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x < (unsigned)S) {
        mbar_init(bars + 8u * threadIdx.x, 1);                           // full: the producer's byte count
        mbar_init(bars + 64u + 8u * threadIdx.x, kMidMathWarps);         // empty: every math warp is done with it
        if (threadIdx.x < 2u) {
            mbar_init(bars + 128u + 8u * threadIdx.x, 1);                // a unit's scales and zero points landed
            mbar_init(bars + 160u + 8u * threadIdx.x, kMidMathWarps);    // ... and are no longer needed
        }
        mbar_fence_init();
    } else if (threadIdx.x == 32) {
        s_abort = 0u;
    }
    __syncthreads();
    const WaitCtl ctl{status_word, &s_abort};
    // programmatic dependent launch: the packed arrays are constants of the layer and are copied
    // before the work in front of this launch has completed; x and the workspace are touched after it
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    if (warp == kMidMathWarps) {
        // ------------------------------------------------------------------ producer
        if (lane != 0) return;
        uint32_t stage = 0, phase = 0;
        int issued = 0;
        bool ok = true;
        for (int u = u0; u < u1 && ok; ++u) {
            const int c = u / nbg, bg = u - c * nbg;
            const int kt0 = c * CT;
            const int nt = min(CT, ktiles - kt0);
            const uint32_t pb = (uint32_t)(u - u0) & 1u, puse = ((uint32_t)(u - u0) >> 1) & 1u;
            if (!mbar_wait_relaxed(bars + 160u + 8u * pb, puse ^ 1u, ctl)) break;
            const uint32_t pdst = sbase + (uint32_t)lay.par_off + pb * (uint32_t)lay.par_bytes;
            mbar_arrive_expect_tx(bars + 128u + 8u * pb, (uint32_t)lay.par_bytes);
            tma_load_2d(pdst, &sc_map, (kt0 / TPG) * 16, bg * kMidMathWarps, bars + 128u + 8u * pb);
            tma_load_2d(pdst + (uint32_t)lay.z_in_par, &z_map, (kt0 / TPG) * 16, bg * (kMidMathWarps / 2),
                        bars + 128u + 8u * pb);
            for (int j = 0; j < nt; j += kMidStageTiles) {
                if (!mbar_wait_relaxed(bars + 64u + 8u * stage, phase ^ 1u, ctl)) { ok = false; break; }
                mbar_arrive_expect_tx(bars + 8u * stage, kMidStageBytes);
                // 16 bands x 4 k-tiles at (64-bit element kt * 64 of the band's run, first band)
                tma_load_2d(sbase + stage * kMidStageBytes, &w_map, (kt0 + j) * 64, bg * kMidMathWarps, bars + 8u * stage);
                ++issued;
                if (++stage == S) { stage = 0; phase ^= 1u; }
            }
        }
        // every copy issued above must have landed before the block may exit
        const int pending = issued < S ? issued : S;
        for (int i = 0; i < pending; ++i) {
            if (stage == 0) { stage = S - 1; phase ^= 1u; } else { --stage; }
            const unsigned long long t0 = global_ns();
            while (!mbar_try_wait(bars + 8u * stage, phase) && global_ns() - t0 < drain_limit_ns(ctl)) {}
        }
        return;
    }

    // -------------------------------------------------------------------- math warps
    asm volatile("griddepcontrol.wait;" ::: "memory");
    unsigned char* xs = smem + lay.x_off;
    float* xg = reinterpret_cast<float*>(smem + lay.xg_off);
    const int g = lane >> 2, t = lane & 3;
    const unsigned char* x_lane[MT];                     // this lane's row of each 8-token fragment
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) x_lane[mt] = xs + (mt * 8 + g) * lay.x_row + t * 8;
    const float* xg_lane = xg + 2 * t;

    uint32_t stage = 0, phase = 0;
    int cur_chunk = -1;
    for (int u = u0; u < u1; ++u) {
        const int c = u / nbg, bg = u - c * nbg;
        const int kt0 = c * CT;
        const int nt = min(CT, ktiles - kt0);
        if (c != cur_chunk) {
            // a new chunk: its slice of x (rows of nt * 64 halfs, absent tokens as zeros) and the sums
            // of x over each group and token, times 2^-24 (the products carry that factor)
            cur_chunk = c;
            named_barrier_sync(1, kMidMathWarps * 32);              // everybody is done with the old slice
            // From three token fragments on, all of a thread's loads leave before its first store (one
            // after the other they are a chain of latencies: 8192 -> 28672 at 24 tokens 55.8 -> 52.3 us;
            // with one or two fragments a thread has two or four loads, and the registers of a batch
            // cost the main loop more than the chain: 40.0 -> 41.0 us at 16 tokens).
            constexpr int FB = MT >= 3 ? 8 : 1;
            const int pieces_per_row = nt * 8, total = lay.mtok * pieces_per_row;
            for (int i0 = threadIdx.x; i0 < total; i0 += FB * kMidMathWarps * 32) {
                uint4 v[FB];
#pragma unroll
                for (int q = 0; q < FB; ++q) {
                    const int i = i0 + q * kMidMathWarps * 32;
                    const int m = i / pieces_per_row, p = i - m * pieces_per_row;
                    v[q] = make_uint4(0u, 0u, 0u, 0u);
                    if (i < total && m < M) v[q] = __ldg(reinterpret_cast<const uint4*>(x + (size_t)m * K + (size_t)kt0 * 64) + p);
                }
#pragma unroll
                for (int q = 0; q < FB; ++q) {
                    const int i = i0 + q * kMidMathWarps * 32;
                    const int m = i / pieces_per_row, p = i - m * pieces_per_row;
                    if (i < total) *reinterpret_cast<uint4*>(xs + m * lay.x_row + p * 16) = v[q];
                }
            }
            named_barrier_sync(1, kMidMathWarps * 32);
            const int ngr = nt / TPG;
            for (int item = warp; item < ngr * lay.mtok; item += kMidMathWarps) {
                const int gi = item / lay.mtok, m = item - gi * lay.mtok;
                const unsigned char* row = xs + m * lay.x_row + gi * (G * 2);
                float v = 0.0f;
#pragma unroll
                for (int e = 0; e < TPG; ++e) {
                    const float2 f = __half22float2(*reinterpret_cast<const __half2*>(row + e * 128 + lane * 4));
                    v += f.x + f.y;
                }
#pragma unroll
                for (int off = 16; off >= 1; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
                if (lane == 0) xg[gi * lay.mtok + m] = v * (1.0f / 16777216.0f);
            }
            named_barrier_sync(1, kMidMathWarps * 32);
        }
        const int band = bg * kMidMathWarps + warp;              // this warp's band (may lie beyond N / 16)
        const uint32_t pb = (uint32_t)(u - u0) & 1u, puse = ((uint32_t)(u - u0) >> 1) & 1u;
        mbar_wait(bars + 128u + 8u * pb, puse, ctl);
        const unsigned char* par = smem + lay.par_off + pb * lay.par_bytes;
        const unsigned char* psc = par + warp * (GPC * 32) + g * 2;
        const unsigned char* pz = par + lay.z_in_par + (warp >> 1) * (GPC * 16) + (warp & 1) * 8 + g;

        float acc[MT][4];
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[mt][i] = 0.0f;

        for (int j = 0; j < nt; j += kMidStageTiles) {
            mbar_wait(bars + 8u * stage, phase, ctl);
            const unsigned char* pw = smem + stage * kMidStageBytes + warp * (kMidStageTiles * 512) + lane * 16;
            const unsigned char* xp[MT];
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) xp[mt] = x_lane[mt] + j * 128;
            // the stage's two k-tiles are one group (G = 128) or two (G = 64)
#pragma unroll
            for (int q = 0; q < kMidStageTiles / TPG; ++q) {
                if (j + q * TPG >= nt) break;                       // a ragged last stage of the chunk
                // one accumulation chain per k-tile of the group and token fragment, interleaved word by
                // word, so that no product waits for the one before it
                float ca[TPG][MT][4];
                uint4 pk[TPG];
#pragma unroll
                for (int v = 0; v < TPG; ++v) pk[v] = *reinterpret_cast<const uint4*>(pw + (q * TPG + v) * 512);
#pragma unroll
                for (int jw = 0; jw < 4; ++jw)
#pragma unroll
                    for (int v = 0; v < TPG; ++v) {
                        const int tile = q * TPG + v;
                        // a byte of a packed word is (row g code) + 16 (row g+8 code) of one column: as an
                        // fp16 subnormal it is the upper rows' operand; the high nibble alone the lower rows'
                        const uint32_t w = (jw == 0) ? pk[v].x : (jw == 1) ? pk[v].y : (jw == 2) ? pk[v].z : pk[v].w;
                        const uint32_t w8 = __byte_perm(w, 0u, 0x4341u);
                        const uint32_t a0 = w & 0x00FF00FFu, a1 = w & 0x00F000F0u, a2 = w8, a3 = w8 & 0x00F000F0u;
#pragma unroll
                        for (int mt = 0; mt < MT; ++mt) {
                            const uint2 bf = *reinterpret_cast<const uint2*>(xp[mt] + tile * 128 + jw * 32);
                            if (jw == 0) mid_mma_first(ca[v][mt], a0, a1, a2, a3, bf.x, bf.y);
                            else mid_mma(ca[v][mt], a0, a1, a2, a3, bf.x, bf.y);
                        }
                    }
                float cc[MT][4];
#pragma unroll
                for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                    for (int i = 0; i < 4; ++i) cc[mt][i] = TPG == 2 ? ca[0][mt][i] + ca[TPG - 1][mt][i] : ca[0][mt][i];
                // per group: Delta * (2^24 D - z X); the lower rows entered 16 times too large
                const int gq = j / TPG + q;                         // group inside the chunk
                const float d_up = __half2float(*reinterpret_cast<const __half*>(psc + gq * 32));
                const float d_lo = __half2float(*reinterpret_cast<const __half*>(psc + gq * 32 + 16));
                const uint32_t zb = pz[gq * 16];
                const float z_up = __uint_as_float(0x4B000000u | (zb & 0xFu)) - 8388608.0f;
                const float z_lo16 = __uint_as_float(0x4B000000u | (zb & 0xF0u)) - 8388608.0f;
                const float su = d_up * 16777216.0f, sl = d_lo * 1048576.0f;
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) {
                    const float2 X = *reinterpret_cast<const float2*>(xg_lane + gq * lay.mtok + mt * 8);
                    acc[mt][0] = fmaf(su, fmaf(-z_up, X.x, cc[mt][0] - cc[mt][2]), acc[mt][0]);
                    acc[mt][1] = fmaf(su, fmaf(-z_up, X.y, cc[mt][1] - cc[mt][3]), acc[mt][1]);
                    acc[mt][2] = fmaf(sl, fmaf(-z_lo16, X.x, cc[mt][2]), acc[mt][2]);
                    acc[mt][3] = fmaf(sl, fmaf(-z_lo16, X.y, cc[mt][3]), acc[mt][3]);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bars + 64u + 8u * stage);
            if (++stage == S) { stage = 0; phase ^= 1u; }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(bars + 160u + 8u * pb);          // the unit's parameters may be replaced
        // the chunk's partial sums of this band, straight from the registers
        if (band < nbands) {
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int tok = mt * 8 + 2 * t + (i & 1), row = g + (i >> 1) * 8;
                    if (tok < M) partial[((size_t)c * M + tok) * N + band * 16 + row] = acc[mt][i];
                }
        }
    }
}

// y[m][n] = fp16(sum over the chunks, ascending, of partial[c][m][n]): four outputs per thread.
__global__ void __launch_bounds__(256)
gemv_mid_reduce_kernel(const float* __restrict__ partial, __half* __restrict__ y, int chunks, size_t mn) {
    // launched with programmatic stream serialization behind the kernel above: it may be resident
    // before that kernel has finished, and lets the launch behind it start its own weight copies
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const size_t i = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
    if (i >= mn) return;
    float4 s = *reinterpret_cast<const float4*>(partial + i);
    for (int c = 1; c < chunks; ++c) {
        const float4 v = *reinterpret_cast<const float4*>(partial + (size_t)c * mn + i);
        s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
    }
    const __half2 lo = __floats2half2_rn(s.x, s.y), hi = __floats2half2_rn(s.z, s.w);
    uint2 o;
    o.x = *reinterpret_cast<const uint32_t*>(&lo);
    o.y = *reinterpret_cast<const uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(y + i) = o;
}

}  // namespace

// k-tiles per chunk for a problem: 16, or 8 where the units (chunks x groups of 16 bands) then fill
// the blocks' equal shares much better (the slowest block sets the time).  Halving the chunk doubles
// the partial sums (M / 32 of the weight bytes at 8 k-tiles, written and read back) and the per-unit
// work (x slice, scales, filling the ring), so the gain has to be large.  Measured at 16 tokens:
// 4096 -> 4096 10.4 -> 7.9 us and 11008 -> 4096 18.7 -> 16.9 us (shares 0.43 -> 0.86 and
// 0.59 -> 0.79 full), but 28672 -> 8192 43.7 -> 51.6 us (0.87 -> 0.93; 33.9 -> 39.5 us at 4 tokens).
static int mid_chunk_tiles(int N, int K, int sms) {
    const int nbg = (N / 16 + kMidMathWarps - 1) / kMidMathWarps;
    auto efficiency = [&](int ct) {
        const int units = ((K / 64 + ct - 1) / ct) * nbg;
        const int blocks = units < sms ? units : sms;
        const int worst = (units + blocks - 1) / blocks;
        return (double)units / ((double)worst * sms);
    };
    return efficiency(8) > efficiency(16) + 0.15 ? 8 : 16;
}
// The workspace holds one fp32 [M][N] array per chunk; sized for the smaller chunk.
size_t gemv_mid_workspace_bytes(int M, int N, int K) {
    return kCounterBytes + (size_t)((K / 64 + 7) / 8) * M * N * sizeof(float);
}
bool gemv_mid_applies(int M, int N, int K, int group, int sms) {
    (void)N; (void)sms;
    if (M < 1 || M > 32 || K > 65536) return false;
    return mid_layout(M, group).total <= kMidSmem && encode_fn() != nullptr;
}

cudaError_t launch_gemv_mid(const void* x, const void* qweight, const void* scales, const void* zeros, void* y,
                            int M, int N, int K, int group, void* workspace, unsigned int* status_word, int sms,
                            bool serialize, cudaStream_t st) {
    EncodeTiledFn enc = encode_fn();
    if (!enc) return cudaErrorNotSupported;
    const int ct = mid_chunk_tiles(N, K, sms);
    const MidLayout lay = mid_layout(M, group, ct);
    const int ng = K / group, gpc = ct * 64 / group;
    const cuuint32_t estr[2] = {1, 1};
    CUtensorMap wmap, scmap, zmap;
    {
        // packed weights: one row of K * 8 bytes per band, as 64-bit elements (a box side is at most
        // 256 elements); boxes of 16 bands x 4 k-tiles (256 elements = 2 KB)
        const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)(N / 16)};
        const cuuint64_t strides[1] = {(cuuint64_t)K * 8};
        const cuuint32_t box[2] = {(cuuint32_t)(kMidStageTiles * 64), (cuuint32_t)kMidMathWarps};
        if (enc(&wmap, CU_TENSOR_MAP_DATA_TYPE_UINT64, 2, const_cast<void*>(qweight), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    {
        // scales: fp16 [band][group][16]; boxes of 16 bands x a chunk's groups
        const cuuint64_t dims[2] = {(cuuint64_t)ng * 16, (cuuint64_t)(N / 16)};
        const cuuint64_t strides[1] = {(cuuint64_t)ng * 32};
        const cuuint32_t box[2] = {(cuuint32_t)(gpc * 16), (cuuint32_t)kMidMathWarps};
        if (enc(&scmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(scales), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    {
        // zero points: bytes [band pair][group][16]; boxes of 8 pairs x a chunk's groups
        const cuuint64_t dims[2] = {(cuuint64_t)ng * 16, (cuuint64_t)(N / 32)};
        const cuuint64_t strides[1] = {(cuuint64_t)ng * 16};
        const cuuint32_t box[2] = {(cuuint32_t)(gpc * 16), (cuuint32_t)(kMidMathWarps / 2)};
        if (enc(&zmap, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(zeros), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    float* partial = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(workspace) + kCounterBytes);
    const int chunks = (K / 64 + ct - 1) / ct;
    const int units = chunks * ((N / 16 + kMidMathWarps - 1) / kMidMathWarps);
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    int blocks = units < sms ? units : sms;
    if (blocks > kUnitMaxBlocks) blocks = kUnitMaxBlocks;
    const UnitStarts starts = unit_starts(units, (N / 16 + kMidMathWarps - 1) / kMidMathWarps, blocks);
    cfg.gridDim = dim3((unsigned)blocks);
    cfg.blockDim = dim3(kMidThreads);
    cfg.dynamicSmemBytes = lay.total;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = serialize ? 0 : 1;
    cudaError_t e;
#define AWQ_MID_LAUNCH2(GG, MTT)                                                                    \
    do {                                                                                            \
        if (ct == 16) AWQ_MID_LAUNCH(GG, MTT, 16); else AWQ_MID_LAUNCH(GG, MTT, 8);                 \
    } while (0)
#define AWQ_MID_LAUNCH(GG, MTT, CTT)                                                                \
    do {                                                                                            \
        static bool done[64] = {};                                                                  \
        int dev = 0;                                                                                \
        e = cudaGetDevice(&dev);                                                                    \
        if (e != cudaSuccess) return e;                                                             \
        if (!done[dev & 63]) {                                                                      \
            e = cudaFuncSetAttribute(gemv_mid_kernel<GG, MTT, CTT>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMidSmem); \
            if (e != cudaSuccess) return e;                                                         \
            done[dev & 63] = true;                                                                  \
        }                                                                                           \
        e = cudaLaunchKernelEx(&cfg, gemv_mid_kernel<GG, MTT, CTT>, wmap, scmap, zmap,                   \
                               reinterpret_cast<const __half*>(x), partial, M, N, K, lay, starts, status_word); \
        if (e != cudaSuccess) return e;                                                             \
    } while (0)
#define AWQ_MID_PICK(GG)                                                                            \
    do {                                                                                            \
        if (lay.mtok <= 8) AWQ_MID_LAUNCH2(GG, 1);                                                  \
        else if (lay.mtok <= 16) AWQ_MID_LAUNCH2(GG, 2);                                            \
        else if (lay.mtok <= 24) AWQ_MID_LAUNCH2(GG, 3);                                            \
        else AWQ_MID_LAUNCH2(GG, 4);                                                                \
    } while (0)
    if (group == 128) AWQ_MID_PICK(128); else AWQ_MID_PICK(64);
#undef AWQ_MID_PICK
#undef AWQ_MID_LAUNCH2
#undef AWQ_MID_LAUNCH
    count_launch();
    e = launch_chunk_reduce(partial, y, chunks, (size_t)M * N, st);
    if (e != cudaSuccess) return e;
    return cudaGetLastError();
}

cudaError_t launch_chunk_reduce(const float* partial, void* y, int chunks, size_t mn, cudaStream_t st) {
    cudaLaunchConfig_t rcfg = {};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    rcfg.gridDim = dim3((unsigned)((mn / 4 + 255) / 256));
    rcfg.blockDim = dim3(256);
    rcfg.stream = st;
    rcfg.attrs = attr;
    rcfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&rcfg, gemv_mid_reduce_kernel, partial, reinterpret_cast<__half*>(y), chunks, mn);
    if (e != cudaSuccess) return e;
    count_launch();
    return cudaSuccess;
}

}  // namespace awq
