// Prefill path of the layer for large token counts (Sec. 4.2: fused dequantize + matrix-matrix
// product): the dataflow of gemm_tcgen05.cu, run by PAIRS of thread blocks (a cluster of two SMs)
// that issue one tcgen05.mma.cta_group::2 of M = 256 output channels x N = 256 tokens.
//
// Why pairs, and why 128-channel stages.  With one block per 128 x 256 tile every 64-wide k-block
// moves 72 KB through shared memory and costs the single MMA-issuing thread two barrier polls,
// four MMAs and a commit; measured, that thread (not the tensor pipe, which sustains one
// 128 x 256 x 16 MMA per 128 cycles) set the pace at ~770 cycles per k-block.  In a pair each
// block stages only its half of the tokens (the tensor cores of both SMs read both halves), and
// a stage covers K = 128, so the polls and commits are paid once per eight MMAs: ~1120 cycles per
// stage against the pipe's 1024.
//
// Block r of a pair (r = rank in the cluster) owns
//   - A: output channels 128 r .. 128 r + 127 of the 256-channel slab, dequantized by its own
//        warps 8-15 into its own tensor memory (64 columns per stage),
//   - B: tokens 128 r .. 128 r + 127 of the 256-token tile in its own shared memory (two 64-wide
//        128-byte-swizzled halves per stage),
//   - D: the fp32 accumulator rows of its 128 channels x all 256 tokens in its own tensor memory,
//        drained by its own epilogue warps (4-7: tokens 0..127, 16-19: tokens 128..255).
// Only the leader (rank 0) issues MMAs.  Barriers that the leader's MMA thread waits on live in the
// leader's shared memory: x_full (both blocks' x copies complete their bytes there), a_full (16
// dequantizer warps, 8 of them arriving remotely), acc_empty (16 epilogue warps).  The MMA
// thread's tcgen05.commit arrives on "empty" and "acc_full" of BOTH blocks.
//
// Tile balance: with a workspace, and when whole tiles would leave pairs idle for long, the tiles'
// K loops are cut into equal ranges over the pairs (stream-K, see PieceIter and the epilogue).
//
// Every wait is bounded (about two seconds): a wait that runs out writes a code to the status word
// and every role of that block leaves its loop; the other block of the pair then runs into its
// own limits.  Both blocks meet at a cluster barrier before they free tensor memory and exit, so
// that no remote arrival can land in the shared memory of a block that has already gone.
#include "tcgen05.cuh"

namespace awq {

namespace {

constexpr int kPairThreads = 640;                // warps: 0 copy, 1 MMA, 4-7 and 16-19 epilogue, 8-15 dequant
constexpr int kPairTokens = 256;                 // tokens per tile (N of the MMA)
constexpr int kHalfTokens = 128;                 // tokens staged by each block

constexpr int kStageK = 128;                     // input channels per pipeline stage (two k-tiles)

struct PairCfg {
    static constexpr int kXHalfBytes = kHalfTokens * kBK * 2;                // 16 KB: one 64-wide swizzled half
    static constexpr int kXTileBytes = 2 * kXHalfBytes;                      // 128 tokens x 128 channels
    static constexpr int kWBytes = 2 * kTileBytes;                           // 8 bands x 2 k-tiles x 512 bytes
    static constexpr int kStageBytes = kXTileBytes + kWBytes;                // 40 KB
    static constexpr int kOutBytes = 8 * 2 * 2048;                           // 8 epilogue warps x 2 staging blocks
    static constexpr int kStages = 4;
    static constexpr int kAColumn0 = kPairTokens;                            // tensor memory: accumulator, then A
    static constexpr int kAColsPerStage = 64;                                // 8 columns per K = 16
    static constexpr int kTmemCols = 512;                                    // 256 + 4 x 64
    static constexpr int kSmemBytes = kStages * kStageBytes + kOutBytes + 1024 /*align*/ + 512 /*barriers*/;
};

// ---------------------------------------------------------------- cluster-scope PTX wrappers
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r;
}
__device__ __forceinline__ uint32_t cluster_id_x() {
    uint32_t r; asm volatile("mov.u32 %0, %%clusterid.x;" : "=r"(r)); return r;
}
__device__ __forceinline__ uint32_t num_clusters_x() {
    uint32_t r; asm volatile("mov.u32 %0, %%nclusterid.x;" : "=r"(r)); return r;
}
// address of the same shared-memory location in block `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_rank(uint32_t addr, uint32_t rank) {
    uint32_t r; asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank)); return r;
}
// Arrival on a barrier of another block of the cluster.  What is handed over lives in tensor
// memory or was written by the copy engine, and tcgen05.fence::before_thread_sync orders it, so
// the default release at block scope is enough; a cluster-scope release costs about a thousand
// cycles per arrival here.
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// x tile copy whose bytes are counted on a barrier of the pair's leader
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int c0, int c1,
                                                 uint32_t leader_bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(leader_bar) : "memory");
}
// D (both blocks' tensor memory) += A (tensor memory, 128 lanes per block) * B (both blocks' smem)
__device__ __forceinline__ void umma_pair_f16_a_tmem(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc,
                                                     uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// arrives on ONE barrier (a shared::cluster address) when the pair's MMAs issued so far are done
__device__ __forceinline__ void umma_pair_commit(uint32_t cluster_bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                 ::"r"(cluster_bar) : "memory");
}
__host__ __device__ constexpr uint32_t instr_desc_pair() {     // D fp32, A/B fp16 K-major, M = 256, N = 256
    return (1u << 4) | ((uint32_t)(kPairTokens >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
}

// Work of one pair: a sequence of pieces (tile, stages k0 .. k1-1 of the tile's K / 128).
// Without a workspace every piece is a whole tile and tiles go round-robin over the pairs.
// With one ("stream-K"), the tiles' stages are laid end to end and cut into equal contiguous
// ranges, one per pair, so that all pairs finish together whatever the tile count; a tile that
// a cut splits is summed up by the pair that holds its first stages (see the epilogue).
struct PieceIter {
    long long s, s_end;              // stream-K: global stage range still to do
    int tile, tile_step, total_tiles, nks;
    bool streamk;
    __device__ bool next(int& t, int& k0, int& k1) {
        if (streamk) {
            if (s >= s_end) return false;
            t = (int)(s / nks);
            k0 = (int)(s - (long long)t * nks);
            const long long left = s_end - s;
            k1 = left < (long long)(nks - k0) ? k0 + (int)left : nks;
            s += k1 - k0;
            return true;
        }
        if (tile >= total_tiles) return false;
        t = tile; k0 = 0; k1 = nks;
        tile += tile_step;
        return true;
    }
};
// first global stage of pair c when `total` stages are cut into `C` ranges that differ by at most one
__device__ __forceinline__ long long range_start(long long total, int C, int c) {
    const long long q = total / C, r = total % C;
    return (long long)c * q + (c < r ? c : r);
}
__device__ __forceinline__ unsigned int ld_acquire_u32(const unsigned int* p) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

constexpr int kPartialFloats = 256 * kPairTokens;    // one pair's fp32 accumulator (256 KB)

// ------------------------------------------------------------------------- the kernel
template <int G>
__global__ void __launch_bounds__(kPairThreads, 1)
gemm_pair_kernel(const __grid_constant__ CUtensorMap x_map, const __grid_constant__ CUtensorMap w_map,
                 const __grid_constant__ CUtensorMap y_map,
                 const __half* __restrict__ scales, const unsigned char* __restrict__ zeros,
                 int M, int N, int K, unsigned int* status_word,
                 float* partials, unsigned int* flags) {
    using Cfg = PairCfg;
    constexpr int S = Cfg::kStages;
    constexpr int GPS = kStageK / G;                 // quantization groups per stage: 1 or 2
    extern __shared__ unsigned char smem_dyn[];
    __shared__ unsigned int s_abort;
    __shared__ uint32_t s_tmem_base;

    const uint32_t dyn = smem_u32(smem_dyn);
    const uint32_t base = (dyn + 1023u) & ~1023u;                    // 1024-byte aligned stage ring
    unsigned char* base_ptr = smem_dyn + (base - dyn);
    // stage layout: [x, k-half 0 (128 tokens x 64) | x, k-half 1 | packed weights (8 bands x 1 KB)]
    auto x_addr = [&](int s) { return base + (uint32_t)s * Cfg::kStageBytes; };
    auto w_ptr = [&](int s) { return base_ptr + (size_t)s * Cfg::kStageBytes + Cfg::kXTileBytes; };
    const uint32_t out_base = base + (uint32_t)S * Cfg::kStageBytes;
    const uint32_t bars = out_base + (uint32_t)Cfg::kOutBytes;
    auto w_full = [&](int s) { return bars + 8u * (uint32_t)s; };               // own weights landed
    auto x_full = [&](int s) { return bars + 8u * (uint32_t)(S + s); };         // leader: both blocks' x landed
    auto a_full = [&](int s) { return bars + 8u * (uint32_t)(2 * S + s); };     // leader: both blocks' A stored
    auto empty = [&](int s) { return bars + 8u * (uint32_t)(3 * S + s); };      // stage free again
    const uint32_t acc_full = bars + 8u * (uint32_t)(4 * S);                    // accumulator complete
    const uint32_t acc_empty = bars + 8u * (uint32_t)(4 * S + 1);               // leader: accumulator drained

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const int m_tiles = (M + kPairTokens - 1) / kPairTokens;
    const int total_tiles = (N / 256) * m_tiles;
    const int cluster = (int)cluster_id_x(), num_clusters = (int)num_clusters_x();
    const int nks = K / kStageK;                     // stages per tile
    const long long total_stages = (long long)total_tiles * nks;
    PieceIter pieces;
    pieces.streamk = partials != nullptr;
    pieces.s = range_start(total_stages, num_clusters, cluster);
    pieces.s_end = range_start(total_stages, num_clusters, cluster + 1);
    pieces.tile = cluster; pieces.tile_step = num_clusters; pieces.total_tiles = total_tiles; pieces.nks = nks;
    int tile, k0, k1;

    if (threadIdx.x == 0) {
        s_abort = 0u;
        for (int s = 0; s < S; ++s) {
            mbar_init(w_full(s), 1); mbar_init(x_full(s), 1); mbar_init(a_full(s), 16); mbar_init(empty(s), 1);
        }
        mbar_init(acc_full, 1);
        mbar_init(acc_empty, 16);
        mbar_fence_init();
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&s_tmem_base)), "r"((uint32_t)Cfg::kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                      // both blocks' barriers exist before anyone arrives remotely
    tc_fence_after();
    const uint32_t tmem_base = s_tmem_base;
    const WaitCtl ctl{status_word, &s_abort};

    if (warp == 0) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            const uint32_t leader_x_full0 = map_to_rank(x_full(0), 0);
            uint32_t stage = 0, phase = 0;
            unsigned int issued = 0;
            bool ok = true;
            while (ok && pieces.next(tile, k0, k1)) {
                const int slab = (tile / m_tiles) * 2 + (int)rank;          // 128-channel slab of this block
                const int tok0 = (tile % m_tiles) * kPairTokens + (int)rank * kHalfTokens;
                for (int ks = k0; ks < k1; ++ks) {
                    if (!mbar_wait(empty(stage), phase ^ 1u, ctl)) { ok = false; break; }
                    if (rank == 0) mbar_arrive_expect_tx(x_full(stage), 2u * Cfg::kXTileBytes);
                    const uint32_t xbar = leader_x_full0 + 8u * stage;
                    tma_load_2d_pair(x_addr(stage), &x_map, ks * kStageK, tok0, xbar);
                    tma_load_2d_pair(x_addr(stage) + Cfg::kXHalfBytes, &x_map, ks * kStageK + kBK, tok0, xbar);
                    const uint32_t bar = w_full(stage);
                    mbar_arrive_expect_tx(bar, (uint32_t)Cfg::kWBytes);
                    // weights: box of 8 bands x 1 KB (256 words: two k-tiles) at (stage, first band)
                    tma_load_2d(x_addr(stage) + Cfg::kXTileBytes, &w_map, ks * 256, slab * 8, bar);
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
                    while (!mbar_try_wait(w_full(st), ph) && global_ns() - t0 < 100000000ull) {}
                }
                const unsigned long long t1 = global_ns();          // and the x halves (counted on the leader)
                while (global_ns() - t1 < 1000000ull) __nanosleep(1000);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------- MMA issuer (leader block only)
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = instr_desc_pair();
            const uint32_t peer_acc_full = map_to_rank(acc_full, 1);
            const uint32_t peer_empty0 = map_to_rank(empty(0), 1);
            uint32_t stage = 0, phase = 0;
            int local = 0;
            bool ok = true;
            for (; ok && pieces.next(tile, k0, k1); ++local) {
                if (!mbar_wait(acc_empty, ((uint32_t)local & 1u) ^ 1u, ctl)) { ok = false; break; }
                tc_fence_after();
                for (int ks = k0; ks < k1; ++ks) {
                    // both barriers are normally complete already: poll them together
                    const bool xr = mbar_try_wait(x_full(stage), phase), ar = mbar_try_wait(a_full(stage), phase);
                    if (!(xr && ar) &&
                        (!mbar_wait(x_full(stage), phase, ctl) || !mbar_wait(a_full(stage), phase, ctl))) {
                        ok = false; break;
                    }
                    tc_fence_after();
                    const uint32_t a_tmem = tmem_base + (uint32_t)(Cfg::kAColumn0 + stage * Cfg::kAColsPerStage);
                    const uint64_t bdesc = smem_desc_sw128(x_addr(stage));
#pragma unroll
                    for (int k = 0; k < kStageK / 16; ++k) {
                        // A: 8 columns per K = 16; B: 32 bytes per K = 16 inside a 64-wide half, halves 16 KB apart
                        const uint64_t boff = (uint64_t)(((k >> 2) * Cfg::kXHalfBytes + (k & 3) * 32) >> 4);
                        umma_pair_f16_a_tmem(tmem_base, a_tmem + (uint32_t)(8 * k), bdesc + boff, idesc,
                                             (ks > k0 || k > 0) ? 1u : 0u);
                    }
                    umma_pair_commit(empty(stage));
                    umma_pair_commit(peer_empty0 + 8u * stage);
                    if (++stage == S) { stage = 0; phase ^= 1u; }
                }
                if (ok) { umma_pair_commit(acc_full); umma_pair_commit(peer_acc_full); }
            }
        }
    } else if (warp >= 8 && warp < 16) {
        // -------------------------------------------------------------- dequantizers
        // one warp per 16-row band of this block's 128 channels, two k-tiles per stage; see
        // gemm_tcgen05.cu for the piece <-> register layout
        const int wi = warp - 8, quad = wi & 3, hsel = wi >> 2;
        const int band = 2 * quad + hsel;
        const int g = lane >> 2;
        const int ng = K / G;
        const uint32_t taddr_band = tmem_base + ((uint32_t)(quad * 32 + hsel * 16) << 16) + (uint32_t)Cfg::kAColumn0;
        const uint32_t leader_a_full0 = map_to_rank(a_full(0), 0);
        uint32_t stage = 0, phase = 0;
        bool ok = true;
        while (ok && pieces.next(tile, k0, k1)) {
            const int slab = (tile / m_tiles) * 2 + (int)rank;
            // this lane's rows' parameters: scales [band][group][16], zero bytes [band pair][group][16]
            const unsigned short* sc_g = reinterpret_cast<const unsigned short*>(scales) +
                                         (size_t)(slab * 8 + band) * ng * 16 + g;
            const unsigned char* z_g = zeros + (size_t)(slab * 4 + (band >> 1)) * ng * 16 + (band & 1) * 8 + g;
            // parameters of the current stage's groups and of the next stage's (fetched one stage ahead)
            uint32_t du[GPS], dl[GPS], zb[GPS], du1[GPS], dl1[GPS], zb1[GPS];
#pragma unroll
            for (int q = 0; q < GPS; ++q) {
                const int g0 = k0 * GPS + q;
                du1[q] = __ldg(sc_g + g0 * 16); dl1[q] = __ldg(sc_g + g0 * 16 + 8); zb1[q] = __ldg(z_g + g0 * 16);
            }
            for (int ks = k0; ks < k1; ++ks) {
#pragma unroll
                for (int q = 0; q < GPS; ++q) {
                    du[q] = du1[q]; dl[q] = dl1[q]; zb[q] = zb1[q];
                    const int gn = min((ks + 1) * GPS + q, ng - 1);
                    du1[q] = __ldg(sc_g + gn * 16); dl1[q] = __ldg(sc_g + gn * 16 + 8); zb1[q] = __ldg(z_g + gn * 16);
                }
                ok = mbar_wait(w_full(stage), phase, ctl);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
#pragma unroll
                for (int h = 0; h < 2; ++h) {                     // the stage's two 64-wide k-tiles
                    const int q = GPS == 2 ? h : 0;
                    const uint4 pk = *reinterpret_cast<const uint4*>(w_ptr(stage) + band * 1024 + h * 512 + lane * 16);
                    const uint32_t d_up = du[q] | (du[q] << 16), d_lo = dl[q] | (dl[q] << 16);
                    const uint32_t zu = 0x6400u + (zb[q] & 0xFu), zl = 0xD400u + ((zb[q] >> 4) << 4);
                    const uint32_t zlo = zu | (zu << 16), zhi = zl | (zl << 16);
                    const uint32_t wds[4] = {pk.x, pk.y, pk.z, pk.w};
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
                    tmem_st_16x32cols(taddr_band + stage * (uint32_t)Cfg::kAColsPerStage + 32u * h, v);
                }
                tmem_st_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(leader_a_full0 + 8u * stage);
                if (++stage == S) { stage = 0; phase ^= 1u; }
            }
        }
    } else if (warp >= 4) {
        // ------------------------------------------------------------------ epilogue
        // warps 4-7 drain token columns 0..127 of the accumulator, warps 16-19 columns 128..255
        const int quad = warp & 3;                     // TMEM lanes 32*quad .. +31
        const int half = warp >= 16 ? 1 : 0;
        const uint32_t leader_acc_empty = map_to_rank(acc_empty, 0);
        // this warp's part of a pair's fp32 partial tile: [rank][warp][chunk][register][lane]
        const size_t part_off = (size_t)((((int)rank * 8 + half * 4 + quad) * 4) * 1024 + lane);
        int local = 0;
        int obuf = 0;
        bool ok = true;
        for (; ok && pieces.next(tile, k0, k1); ++local) {
            const int slab = (tile / m_tiles) * 2 + (int)rank, mt = tile % m_tiles;
            // A piece that does not start the tile is a contribution: its fp32 sums go to this pair's
            // slot of the workspace.  A piece that starts the tile but does not end it waits for the
            // contributions of the pairs after this one (they were produced at the start of those
            // pairs' ranges, long before) and adds them in pair order: the sum is reproducible.
            const bool contributes = k0 > 0;
            int n_contrib = 0;
            if (k0 == 0 && k1 < nks) {
                const long long tile_end = (long long)(tile + 1) * nks;
                while (cluster + 1 + n_contrib < num_clusters &&
                       range_start(total_stages, num_clusters, cluster + 1 + n_contrib) < tile_end)
                    ++n_contrib;
            }
            // while this piece's MMAs run: wait for the contributions (normally there long ago) and
            // fetch the first one's first chunk, so that the drain below does not wait for memory
            for (int j = 0; j < n_contrib && ok; ++j) {
                const unsigned int* f = flags + cluster + 1 + j;
                const unsigned long long t0 = global_ns();
                while (ld_acquire_u32(f) < 16u) {                   // 16 epilogue warps of that pair
                    if (*ctl.abort) { ok = false; break; }
                    if (global_ns() - t0 > wait_limit_ns(ctl)) {
                        *ctl.abort = 1u;
                        atomicExch(ctl.status, kTimeoutCode);
                        ok = false;
                        break;
                    }
                    __nanosleep(64);
                }
            }
            float p[32];
            const float* src0 = partials + (size_t)(cluster + 1) * kPartialFloats + part_off;
            if (n_contrib > 0 && ok) {
#pragma unroll
                for (int i = 0; i < 32; ++i) p[i] = __ldcg(src0 + i * 32);
            }
            ok = ok && mbar_wait(acc_full, (uint32_t)local & 1u, ctl);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            tc_fence_after();
            const int n0 = slab * 128 + quad * 32;
            const int m0 = mt * kPairTokens + half * kHalfTokens;
            const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(half * kHalfTokens);
#pragma unroll 1
            for (int c = 0; c < kHalfTokens; c += 32) {
                uint32_t r[32];
                tmem_ld_32cols(taddr + (uint32_t)c, r);
                tmem_ld_wait();
                if (c + 32 >= kHalfTokens) {
                    // the accumulator is in registers: the MMA thread may start the next piece
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster(leader_acc_empty);
                }
                if (contributes) {
                    float* dst = partials + (size_t)cluster * kPartialFloats + part_off + (size_t)c * 32;
#pragma unroll
                    for (int i = 0; i < 32; ++i) __stcg(dst + i * 32, __uint_as_float(r[i]));
                    continue;
                }
                if (n_contrib > 0) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) + p[i]);
                    for (int j = 1; j < n_contrib; ++j) {
                        const float* src = partials + (size_t)(cluster + 1 + j) * kPartialFloats + part_off + (size_t)c * 32;
#pragma unroll
                        for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) + __ldcg(src + i * 32));
                    }
                    if (c + 32 < kHalfTokens) {                     // the next chunk of the first contribution
#pragma unroll
                        for (int i = 0; i < 32; ++i) p[i] = __ldcg(src0 + (size_t)(c + 32) * 32 + i * 32);
                    }
                }
                // stage the 32 x 32 block as [token][channel] fp16 and hand it to the copy engine
                // (rows past M are clipped by the tensor map)
                if (lane == 0) bulk_wait_read_1();                  // the store that last used this buffer
                __syncwarp();
                const uint32_t tb = out_base + (uint32_t)(((half * 4 + quad) * 2 + obuf) * 2048);
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
            if (contributes) {
                __threadfence();                                    // the sums before the flag
                __syncwarp();
                if (lane == 0) atomicAdd(flags + cluster, 1u);
            }
            if (lane == 0) {
                // the 16 readers of a slot count themselves in after the 16 writers; the last one
                // clears the flag, so the workspace is ready for the next launch
                for (int j = 0; j < n_contrib; ++j)
                    if (atomicAdd(flags + cluster + 1 + j, 1u) == 31u) atomicExch(flags + cluster + 1 + j, 0u);
            }
        }
        if (lane == 0) bulk_wait_all();                             // all of y written before exit
    }

    __syncwarp();
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                      // nothing of the pair still refers to this block
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;"
                     ::"r"(tmem_base), "r"((uint32_t)Cfg::kTmemCols) : "memory");
    }
}

// ------------------------------------------------------------------------------ host
// pairs that can be resident at once on the current device (0 if the query fails); cached
template <int G>
int resident_pairs(int sms, cudaError_t* err) {
    static bool done[64] = {};
    static int pairs[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    *err = cudaSuccess;
    if (!done[dev & 63]) {
        *err = cudaFuncSetAttribute(gemm_pair_kernel<G>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    PairCfg::kSmemBytes);
        if (*err != cudaSuccess) return 0;
        cudaLaunchConfig_t cfg = {};
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cfg.gridDim = dim3((unsigned)(sms & ~1));
        cfg.blockDim = dim3(kPairThreads);
        cfg.dynamicSmemBytes = PairCfg::kSmemBytes;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, gemm_pair_kernel<G>, &cfg) != cudaSuccess) {
            (void)cudaGetLastError();
            n = 0;
        }
        pairs[dev & 63] = n;
        done[dev & 63] = true;
    }
    return pairs[dev & 63];
}

template <int G>
cudaError_t launch_pair(const CUtensorMap& xmap, const CUtensorMap& wmap, const CUtensorMap& ymap,
                        const void* scales, const void* zeros, int M, int N, int K,
                        void* workspace, size_t workspace_bytes,
                        unsigned int* status_word, int sms, cudaStream_t st, bool* launched) {
    using Cfg = PairCfg;
    cudaError_t e;
    const int resident = resident_pairs<G>(sms, &e);
    if (e != cudaSuccess) return e;
    // pairs that cannot all be resident at once would leave SMs idle (and a tile's owner waiting)
    if (resident * 2 < sms - 4) { *launched = false; return cudaSuccess; }
    const long long tiles = (long long)(N / 256) * ((M + kPairTokens - 1) / kPairTokens);
    const long long stages = tiles * (K / kStageK);
    // Stream-K needs one fp32 tile per pair behind the counters at the head of the workspace.  It
    // costs every pair two more accumulator drains and a pass over a partial tile (about 10 us),
    // so it is used only when whole tiles would leave the pairs idle for longer than that: the
    // idle time of the last round-robin wave, in stages (~0.8 us each) per pair.  Launches of
    // more than about 0.3 ms run into the power limit, where idle pairs let the busy ones clock
    // higher and an even split gains nothing (measured: 5 % slower): those keep whole tiles.
    const long long waves = (tiles + resident - 1) / resident;
    const long long idle_stages = (waves * resident - tiles) * (K / kStageK) / resident;
    const bool streamk = workspace != nullptr && idle_stages > 25 && stages / resident < 400 &&
                         workspace_bytes >= kCounterBytes + (size_t)resident * kPartialFloats * sizeof(float) &&
                         (size_t)resident * sizeof(unsigned int) <= kCounterBytes;
    long long want = tiles;
    if (streamk && stages / 4 > want) want = stages / 4;          // at least four stages per pair
    const int clusters = (int)(want < resident ? want : resident);
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.gridDim = dim3((unsigned)(2 * clusters));
    cfg.blockDim = dim3(kPairThreads);
    cfg.dynamicSmemBytes = Cfg::kSmemBytes;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    float* partials = streamk ? reinterpret_cast<float*>(static_cast<unsigned char*>(workspace) + kCounterBytes)
                              : nullptr;
    unsigned int* flags = static_cast<unsigned int*>(workspace);
    e = cudaLaunchKernelEx(&cfg, gemm_pair_kernel<G>, xmap, wmap, ymap, reinterpret_cast<const __half*>(scales),
                           reinterpret_cast<const unsigned char*>(zeros), M, N, K, status_word, partials, flags);
    if (e != cudaSuccess) return e;
    count_launch();
    *launched = true;
    return cudaGetLastError();
}

}  // namespace

// Above 128 tokens always; below, where the one-SM kernel's 128-channel tiles re-read x too often:
// measured at M = 96 .. 128, 27.6 against 42 us on 4096 -> 11008; at M = 32 .. 128, 77 .. 84 against
// 98 .. 117 us on 8192 -> 28672; but 26.5 against 13 .. 19 us on 4096 -> 4096 (few tiles: the
// one-SM kernel with split-K wins).
bool gemm_pair_applies(int M, int N) {
    if (N % 256 != 0) return false;
    return M > 128 || (M > 64 && N >= 8192) || (M >= 32 && N >= 16384);
}

// workspace with which the pair kernel balances its tiles over all SM pairs (stream-K)
size_t gemm_pair_workspace_bytes(int sms) {
    return kCounterBytes + (size_t)(sms / 2) * kPartialFloats * sizeof(float);
}

// Launches the pair kernel if this device can keep (nearly) all its SMs busy with pairs;
// otherwise *launched is false and the caller uses the single-block kernel.
cudaError_t launch_gemm_pair(const CUtensorMap& xmap128, const CUtensorMap& wmap, const CUtensorMap& ymap,
                             const void* scales, const void* zeros, int M, int N, int K, int group,
                             void* workspace, size_t workspace_bytes,
                             unsigned int* status_word, int sms, cudaStream_t st, bool* launched) {
    if (group == 128)
        return launch_pair<128>(xmap128, wmap, ymap, scales, zeros, M, N, K, workspace, workspace_bytes,
                                status_word, sms, st, launched);
    return launch_pair<64>(xmap128, wmap, ymap, scales, zeros, M, N, K, workspace, workspace_bytes,
                           status_word, sms, st, launched);
}

}  // namespace awq
