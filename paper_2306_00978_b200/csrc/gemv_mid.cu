// The layer for a medium number of tokens (9 .. 32), Sec. 4.2's fused dequantize + product where
// it is still a bandwidth problem (4 M FLOP per weight byte against a ridge of about 280).
//
// The tensor-memory kernels pay about 9 us per launch (allocation, first copies, split-K hand-over,
// store drain) and re-read x for every 128-channel tile; the band matrix-vector kernel keeps its
// operands in registers and streams a band as one contiguous run, but every band reads all of x.
// This kernel keeps the band kernel's arithmetic and streaming and changes the decomposition so
// that x is read once per block:
//   * a block owns ONE chunk of K (2048 input channels, 1024 above 16 tokens) and a range of
//     16-row bands.  Its slice of x (M x chunk) is fetched once and stays in shared memory,
//     together with the per-group sums of x that the zero-point term needs;
//   * a stage of the ring is one band's run of that chunk - contiguous in the band-major layout:
//     16 KB of packed weights, its scales, its zero points, three bulk copies (few large copies:
//     the copy engine's cost is per copy, not per byte);
//   * the 16 math warps are (token group) x (k slice): a warp multiplies its two k-tiles of the stage
//     by 16 tokens (two 8-token B fragments per A fragment; they are the same for every band, so
//     they are read from the x slice once and stay in registers) with the
//     same whole-byte-operand tensor-core products as the band kernel; the slices of a band meet in
//     shared memory and the math warps themselves add them, each thread a few outputs in slice
//     order (a single warp doing all 16 x 16 M additions per band would set the pace);
//   * a band's sums over ONE chunk are partial: they go to an fp32 workspace [chunk][token][channel],
//     and a second, tiny kernel adds the chunks in ascending order and rounds to fp16 once -
//     deterministic, no counters, no fences, no waiting between blocks.
// Every wait is bounded as in the other kernels.
#include "async_copy.cuh"
#include "common.cuh"

namespace awq {

namespace {

constexpr int kMidMathWarps = 16;
constexpr int kMidThreads = (kMidMathWarps + 1) * 32;   // + weight-copy warp
constexpr int kMidSmem = 216 * 1024;

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
    int kc_tiles;        // k-tiles (64 columns) per chunk
    int bps;             // bands per stage (2 up to 16 tokens: more k-tiles per warp between two reductions)
    int tg, ks, tpw;     // token groups of 16, k slices (bps * tg * ks = 16 warps), k-tiles per warp and stage
    int mtok;            // M rounded up to whole token groups
    int slot_bytes;      // one band's run of the chunk: weights, scales, zero points
    int stage_bytes, stages;
    int sc_off, z_off;   // inside a stage: scales [group][16] fp16, zero points [group][16] bytes
    int x_off, x_row;    // x slice [mtok][x_row bytes]
    int xg_off;          // fp32 [groups of the chunk][mtok]: 2^-24 times the sums of x
    int red_off;         // two buffers of [warp][16 tokens][16 rows] fp32
    int bar_off, total;
};

inline MidLayout mid_layout(int M, int group) {
    MidLayout l;
    l.mtok = ((M + 15) / 16) * 16;            // 16 or 32
    l.tg = l.mtok / 16;
    l.bps = 1;
    l.ks = kMidMathWarps / (l.tg * l.bps);    // 16 or 8 k slices
    l.kc_tiles = 2 * l.ks;                    // 2048 input channels up to 16 tokens, 1024 above
    l.tpw = 2;
    const int groups = l.kc_tiles * 64 / group;
    l.sc_off = l.kc_tiles * 512;
    l.z_off = l.sc_off + groups * 32;
    l.slot_bytes = ((l.z_off + groups * 16 + 127) / 128) * 128;
    l.stage_bytes = l.bps * l.slot_bytes;
    l.x_row = l.kc_tiles * 128 + 32;
    const int x_bytes = l.mtok * l.x_row;
    const int xg_bytes = groups * l.mtok * 4;
    const int red_bytes = 2 * kMidMathWarps * 256 * 4;
    int s = (kMidSmem - x_bytes - xg_bytes - red_bytes - 512) / l.stage_bytes;
    l.stages = s > 6 ? 6 : s;
    l.x_off = l.stages * l.stage_bytes;
    l.xg_off = l.x_off + ((x_bytes + 127) / 128) * 128;
    l.red_off = l.xg_off + ((xg_bytes + 127) / 128) * 128;
    l.bar_off = l.red_off + red_bytes;
    l.total = l.bar_off + 256;
    return l;
}

// Which chunk a block works on and which bands: the blocks are dealt to the chunks in proportion
// to their k-tiles (a ragged last chunk gets fewer), a chunk's bands evenly to its blocks.
struct MidShare {
    int chunk, tiles, b0, b1;
};
__host__ __device__ inline MidShare mid_share(int block, int blocks, int ktiles, int kc_tiles, int nbands) {
    const int nchunks = (ktiles + kc_tiles - 1) / kc_tiles;
    MidShare r = {0, 0, 0, 0};
    for (int c = 0; c < nchunks; ++c) {
        const int t0 = c * kc_tiles, t1 = (c + 1) * kc_tiles < ktiles ? (c + 1) * kc_tiles : ktiles;
        // every chunk gets at least one block: blocks >= nchunks, and the shares are cut so
        const int p0 = (int)(((long long)blocks * t0) / ktiles), p1 = (int)(((long long)blocks * t1) / ktiles);
        const int first = p0 > c ? p0 : c;
        int last = p1 > c + 1 ? p1 : c + 1;                       // exclusive
        if (c == nchunks - 1) last = blocks;
        if (block >= first && block < last) {
            const int pc = last - first, i = block - first;
            r.chunk = c;
            r.tiles = t1 - t0;
            r.b0 = (int)(((long long)nbands * i) / pc);
            r.b1 = (int)(((long long)nbands * (i + 1)) / pc);
            return r;
        }
    }
    return r;
}

template <int G>
__global__ void __launch_bounds__(kMidThreads, 1)
gemv_mid_kernel(const unsigned char* __restrict__ qweight, const __half* __restrict__ scales,
                const unsigned char* __restrict__ zeros, const __half* __restrict__ x,
                float* __restrict__ partial, int M, int N, int K, const MidLayout lay,
                unsigned int* status_word) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ unsigned int s_abort;
    constexpr int TPG = G / 64;                          // k-tiles per group
    const int S = lay.stages;
    const uint32_t sbase = smem_u32(smem);
    // barriers: full[s] at 8s, empty[s] at 64 + 8s
    const uint32_t bars = sbase + (uint32_t)lay.bar_off;
    const int ktiles = K / 64, ng = K / G, nbands = N / 16;
    const MidShare sh = mid_share((int)blockIdx.x, (int)gridDim.x, ktiles, lay.kc_tiles, nbands);
    const int kt0 = sh.chunk * lay.kc_tiles;             // first k-tile of the chunk
    const int nt = sh.tiles;                             // its k-tiles (a multiple of two: whole groups)
    const int ngr = nt * 64 / G;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x < 8u) {
        if (threadIdx.x < (unsigned)S) {
            mbar_init(bars + 8u * threadIdx.x, 1);                       // full: the copy warp's byte count
            mbar_init(bars + 64u + 8u * threadIdx.x, kMidMathWarps);     // empty: every math warp is done with it
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
        // ------------------------------------------------------------- weight-copy warp
        uint32_t stage = 0, phase = 0;
        const uint64_t once = l2_policy_evict_first();
        for (int band0 = sh.b0; band0 < sh.b1; band0 += lay.bps) {
            const int nb = min(lay.bps, sh.b1 - band0);              // bands of this stage
            const uint32_t bar = bars + 8u * stage;
            if (lane == 0) {
                mbar_wait_relaxed(bars + 64u + 8u * stage, phase ^ 1u, ctl);
                mbar_arrive_expect_tx(bar, (uint32_t)(nb * (nt * 512 + ngr * 48)));
            }
            __syncwarp();
            const int gi0 = kt0 * 64 / G;
            const int slot = lane / 3, what = lane - 3 * slot;       // lanes 3 slot .. 3 slot + 2: one band's three copies
            if (slot < nb) {
                const int band = band0 + slot;
                const uint32_t dst = sbase + stage * (uint32_t)lay.stage_bytes + slot * (uint32_t)lay.slot_bytes;
                if (what == 0)
                    bulk_load_hint(dst, qweight + ((size_t)band * ktiles + kt0) * 512, (uint32_t)(nt * 512), bar, once);
                else if (what == 1)
                    bulk_load_hint(dst + lay.sc_off, scales + ((size_t)band * ng + gi0) * 16, (uint32_t)(ngr * 32), bar, once);
                else
                    bulk_load(dst + lay.z_off, zeros + ((size_t)(band >> 1) * ng + gi0) * 16, (uint32_t)(ngr * 16), bar);
            }
            if (++stage == (uint32_t)S) { stage = 0; phase ^= 1u; }
        }
        if (lane != 0) return;
        // every copy issued above must have landed before the block may exit
        const int issued = (sh.b1 - sh.b0 + lay.bps - 1) / lay.bps;
        const int pending = issued < S ? issued : S;
        for (int i = 0; i < pending; ++i) {
            if (stage == 0) { stage = S - 1; phase ^= 1u; } else { --stage; }
            const unsigned long long t0 = global_ns();
            while (!mbar_try_wait(bars + 8u * stage, phase) && global_ns() - t0 < drain_limit_ns(ctl)) {}
        }
        return;
    }

    asm volatile("griddepcontrol.wait;" ::: "memory");
    float* red = reinterpret_cast<float*>(smem + lay.red_off);
    const int KS = lay.ks;

    // -------------------------------------------------------------------- math warps
    unsigned char* xs = smem + lay.x_off;
    float* xg = reinterpret_cast<float*>(smem + lay.xg_off);
    {
        // the block's slice of x: rows of nt * 64 halfs (16-byte pieces), absent tokens as zeros
        const int pieces_per_row = nt * 8;
        const int total = lay.mtok * pieces_per_row;
        for (int i = threadIdx.x; i < total; i += kMidMathWarps * 32) {
            const int m = i / pieces_per_row, p = i - m * pieces_per_row;
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if (m < M) v = __ldg(reinterpret_cast<const uint4*>(x + (size_t)m * K + (size_t)kt0 * 64) + p);
            *reinterpret_cast<uint4*>(xs + m * lay.x_row + p * 16) = v;
        }
        named_barrier_sync(1, kMidMathWarps * 32);
        // sums of x over each group of the chunk and each token, times 2^-24 (the products carry it)
        for (int item = warp; item < ngr * lay.mtok; item += kMidMathWarps) {
            const int gi = item / lay.mtok, m = item - gi * lay.mtok;
            const unsigned char* row = xs + m * lay.x_row + gi * (G * 2);
            float v = 0.0f;
#pragma unroll
            for (int e = 0; e < G / 64; ++e) {
                const float2 f = __half22float2(*reinterpret_cast<const __half2*>(row + e * 128 + lane * 4));
                v += f.x + f.y;
            }
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
            if (lane == 0) xg[gi * lay.mtok + m] = v * (1.0f / 16777216.0f);
        }
        named_barrier_sync(1, kMidMathWarps * 32);
    }

    const int g = lane >> 2, t = lane & 3;
    const int slot = warp / (lay.tg * KS);               // which band of the stage
    const int tg = (warp / KS) % lay.tg, ks = warp % KS;
    constexpr int kTPW = 2;                              // k-tiles per warp and stage (every layout has lay.tpw = 2)
    const int tpw = kTPW;
    const int my_tiles = min(tpw, nt - ks * tpw);        // this warp's k-tiles of a stage: <= 0, 2 or 4
    // this lane's fixed offsets
    const int o_w = (ks * tpw) * 512 + lane * 16;
    const int o_sc = lay.sc_off + (ks * tpw / TPG) * 32 + g * 2;
    // B fragments: a warp multiplies the same two k-tiles of the chunk in every band, so its
    // fragments of x (16 tokens x 128 columns: 32 registers) are read once and stay in registers
    uint2 xr[2][kTPW][4];
    {
        const unsigned char* x_lane0 = xs + (tg * 16 + g) * lay.x_row + ((ks * tpw) * 64 + t * 4) * 2;
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int v = 0; v < kTPW; ++v)
#pragma unroll
                for (int jw = 0; jw < 4; ++jw)
                    xr[mt][v][jw] = *reinterpret_cast<const uint2*>(x_lane0 + mt * 8 * lay.x_row + v * 128 + jw * 32);
    }
    const float* xg_lane = xg + (ks * tpw / TPG) * lay.mtok + tg * 16 + 2 * t;
    float* red_lane = red + warp * 256 + (2 * t) * 16 + g;

    uint32_t stage = 0, phase = 0, b = 0;
    for (int band0 = sh.b0; band0 < sh.b1; band0 += lay.bps) {
        const int band = band0 + slot;
        const bool have = band < sh.b1;                  // (the last stage of a range may hold one band only)
        float acc[2][4];
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[mt][i] = 0.0f;
        mbar_wait(bars + 8u * stage, phase, ctl);
        const unsigned char* st = smem + stage * (uint32_t)lay.stage_bytes + slot * (uint32_t)lay.slot_bytes;
        const unsigned char* pw = st + o_w;                              // this lane's pieces
        const unsigned char* psc = st + o_sc;
        const unsigned char* pz = st + lay.z_off + (ks * kTPW / TPG) * 16 + (band & 1) * 8 + g;
        // straight-line code: every shared-memory address is a base plus an immediate
#pragma unroll
        for (int q = 0; q < kTPW / TPG; ++q) {
            if (have && q * TPG < my_tiles) {
                float c[2][4];
#pragma unroll
                for (int v = 0; v < TPG; ++v) {
                    const int tile = q * TPG + v;
                    const uint4 pk = *reinterpret_cast<const uint4*>(pw + tile * 512);
                    const uint32_t wds[4] = {pk.x, pk.y, pk.z, pk.w};
#pragma unroll
                    for (int jw = 0; jw < 4; ++jw) {
                        // a byte of a packed word is (row g code) + 16 (row g+8 code) of one column: as an
                        // fp16 subnormal it is the upper rows' operand; the high nibble alone the lower rows'
                        const uint32_t w = wds[jw], w8 = __byte_perm(w, 0u, 0x4341u);
                        const uint32_t a0 = w & 0x00FF00FFu, a1 = w & 0x00F000F0u, a2 = w8, a3 = w8 & 0x00F000F0u;
                        const uint2 bf0 = xr[0][tile][jw], bf1 = xr[1][tile][jw];
                        if (v == 0 && jw == 0) {
                            mid_mma_first(c[0], a0, a1, a2, a3, bf0.x, bf0.y);
                            mid_mma_first(c[1], a0, a1, a2, a3, bf1.x, bf1.y);
                        } else {
                            mid_mma(c[0], a0, a1, a2, a3, bf0.x, bf0.y);
                            mid_mma(c[1], a0, a1, a2, a3, bf1.x, bf1.y);
                        }
                    }
                }
                // per group: Delta * (2^24 D - z X); the lower rows entered 16 times too large
                const float d_up = __half2float(*reinterpret_cast<const __half*>(psc + q * 32));
                const float d_lo = __half2float(*reinterpret_cast<const __half*>(psc + q * 32 + 16));
                const uint32_t zb = pz[q * 16];
                const float z_up = __uint_as_float(0x4B000000u | (zb & 0xFu)) - 8388608.0f;
                const float z_lo16 = __uint_as_float(0x4B000000u | (zb & 0xF0u)) - 8388608.0f;
                const float su = d_up * 16777216.0f, sl = d_lo * 1048576.0f;
#pragma unroll
                for (int mt = 0; mt < 2; ++mt) {
                    const float2 X = *reinterpret_cast<const float2*>(xg_lane + q * lay.mtok + mt * 8);
                    acc[mt][0] = fmaf(su, fmaf(-z_up, X.x, c[mt][0] - c[mt][2]), acc[mt][0]);
                    acc[mt][1] = fmaf(su, fmaf(-z_up, X.y, c[mt][1] - c[mt][3]), acc[mt][1]);
                    acc[mt][2] = fmaf(sl, fmaf(-z_lo16, X.x, c[mt][2]), acc[mt][2]);
                    acc[mt][3] = fmaf(sl, fmaf(-z_lo16, X.y, c[mt][3]), acc[mt][3]);
                }
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(bars + 64u + 8u * stage);
        if (++stage == (uint32_t)S) { stage = 0; phase ^= 1u; }
        // this slice's sums: red[b][warp][token 0..15][row 0..15]; then every thread adds the
        // slices of a few outputs in slice order and writes the chunk's partial sums.  One block
        // barrier per band: buffer b is rewritten two bands on, after the barrier of the band between.
        float* rb = red_lane + b * (kMidMathWarps * 256);
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int i = 0; i < 4; ++i)
                rb[(mt * 8 + (i & 1)) * 16 + (i >> 1) * 8] = acc[mt][i];
        named_barrier_sync(1, kMidMathWarps * 32);
        const float* rbase = red + b * (kMidMathWarps * 256);
        for (int idx = threadIdx.x; idx < lay.bps * lay.mtok * 16; idx += kMidMathWarps * 32) {
            // idx = (band of the stage * tokens + token) * 16 + row
            const int row = idx & 15, bt = idx >> 4, sl = bt / lay.mtok, tok = bt - sl * lay.mtok;
            if (band0 + sl >= sh.b1) continue;
            const float* src = rbase + ((sl * lay.tg + (tok >> 4)) * KS) * 256 + (tok & 15) * 16 + row;
            // all loads first, then a fixed-order sum (a serial load-add loop would be a chain of
            // sixteen shared-memory latencies per band)
            float v[kMidMathWarps];
#pragma unroll
            for (int k = 0; k < kMidMathWarps; ++k) v[k] = k < KS ? src[k * 256] : 0.0f;
#pragma unroll
            for (int w = 1; w < kMidMathWarps; w <<= 1)
#pragma unroll
                for (int k = 0; k < kMidMathWarps; k += 2 * w) v[k] += v[k + w];
            const float sum = v[0];
            if (tok < M) partial[((size_t)sh.chunk * M + tok) * N + (band0 + sl) * 16 + row] = sum;
        }
        b ^= 1u;
    }
}

// y[m][n] = fp16(sum over the chunks, ascending, of partial[c][m][n]): four outputs per thread.
__global__ void __launch_bounds__(256)
gemv_mid_reduce_kernel(const float* __restrict__ partial, __half* __restrict__ y, int chunks, size_t mn) {
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

// Chunks of K for M tokens (the workspace holds one fp32 [M][N] array per chunk).
int gemv_mid_chunks(int M, int K) {
    const int kc_tiles = M <= 16 ? 32 : 16;
    return (K / 64 + kc_tiles - 1) / kc_tiles;
}
size_t gemv_mid_workspace_bytes(int M, int N, int K) {
    return kCounterBytes + (size_t)gemv_mid_chunks(M, K) * M * N * sizeof(float);
}
bool gemv_mid_applies(int M, int N, int K, int group, int sms) {
    if (M < 1 || M > 32 || K > 65536) return false;
    const MidLayout lay = mid_layout(M, group);
    return lay.stages >= 2 && gemv_mid_chunks(M, K) <= sms && (N % 4) == 0;
}

cudaError_t launch_gemv_mid(const void* x, const void* qweight, const void* scales, const void* zeros, void* y,
                            int M, int N, int K, int group, void* workspace, unsigned int* status_word, int sms,
                            bool serialize, cudaStream_t st) {
    const MidLayout lay = mid_layout(M, group);
    float* partial = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(workspace) + kCounterBytes);
    const int chunks = gemv_mid_chunks(M, K);
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.gridDim = dim3((unsigned)sms);
    cfg.blockDim = dim3(kMidThreads);
    cfg.dynamicSmemBytes = lay.total;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = serialize ? 0 : 1;
    cudaError_t e;
#define AWQ_MID_LAUNCH(GG)                                                                          \
    do {                                                                                            \
        static bool done[64] = {};                                                                  \
        int dev = 0;                                                                                \
        e = cudaGetDevice(&dev);                                                                    \
        if (e != cudaSuccess) return e;                                                             \
        if (!done[dev & 63]) {                                                                      \
            e = cudaFuncSetAttribute(gemv_mid_kernel<GG>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMidSmem); \
            if (e != cudaSuccess) return e;                                                         \
            done[dev & 63] = true;                                                                  \
        }                                                                                           \
        e = cudaLaunchKernelEx(&cfg, gemv_mid_kernel<GG>, reinterpret_cast<const unsigned char*>(qweight), \
                               reinterpret_cast<const __half*>(scales),                             \
                               reinterpret_cast<const unsigned char*>(zeros),                       \
                               reinterpret_cast<const __half*>(x), partial, M, N, K, lay, status_word); \
        if (e != cudaSuccess) return e;                                                             \
    } while (0)
    if (group == 128) AWQ_MID_LAUNCH(128); else AWQ_MID_LAUNCH(64);
#undef AWQ_MID_LAUNCH
    count_launch();
    const size_t mn = (size_t)M * N;
    gemv_mid_reduce_kernel<<<(unsigned)((mn / 4 + 255) / 256), 256, 0, st>>>(partial, reinterpret_cast<__half*>(y),
                                                                             chunks, mn);
    count_launch();
    return cudaGetLastError();
}

}  // namespace awq
