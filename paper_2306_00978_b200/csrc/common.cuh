// Shared declarations of the library's translation units (host side and launchers).
#pragma once
#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <stdint.h>
#include "../../include/awq_b200.h"

namespace awq {

constexpr int kTileRows = 128;           // output channels per packed tile
constexpr int kTileCols = 64;            // input channels per packed tile
constexpr int kTileBytes = kTileRows * kTileCols / 2;   // 8 bands x 512 bytes
constexpr size_t kCounterBytes = 4096;   // head of the workspace: split-K arrival counters
constexpr int kMaxSlabs = int(kCounterBytes / sizeof(unsigned int));

// alpha is classified on the host so that the device takes the exact branch.
enum AlphaMode : int { kAlphaZero = 0, kAlphaOne = 1, kAlphaHalf = 2, kAlphaGeneral = 3 };

inline AlphaMode alpha_mode(float alpha) {
    if (alpha == 0.0f) return kAlphaZero;
    if (alpha == 1.0f) return kAlphaOne;
    if (alpha == 0.5f) return kAlphaHalf;
    return kAlphaGeneral;
}

void count_launch();

// launchers (each returns the cudaError_t of the launch)
cudaError_t launch_channel_scale(const float* a, float alpha, float* s, int K, cudaStream_t st);
// bits: 4 or 3 (3-bit codes in the 4-bit fields); clip: optional per-group range ratios [N][K/group]
cudaError_t launch_quantize_pack(const __half* W, const float* a, float alpha, int group, int bits,
                                 bool symmetric, const float* clip, uint32_t* qweight, __half* scales, uint8_t* zeros,
                                 int N, int K, cudaStream_t st);
constexpr int kMaxClipRatios = 32;
// ratios: HOST array of n_ratios <= kMaxClipRatios values; clip: device out, fp32 [N][K/group]
cudaError_t launch_clip_search(const __half* W, const float* a, float alpha, int group, int bits,
                               const float* ratios, int n_ratios, float* clip, int N, int K,
                               cudaStream_t st);
cudaError_t launch_unpack(const uint32_t* qweight, const __half* scales, const uint8_t* zeros,
                          int N, int K, int group, uint8_t* codes, uint16_t* scales_nk,
                          uint8_t* zeros_nk, cudaStream_t st);

// 3-bit storage <-> the 4-bit layout holding 3-bit codes (N * K / 32 pieces of 16 / 12 bytes)
cudaError_t launch_pack_int3(const void* q4, void* q3, int N, int K, cudaStream_t st);
cudaError_t launch_unpack_int3(const void* q3, void* q4, int N, int K, cudaStream_t st);

constexpr int kGemvMaxBlocks = 256;      // upper bound on the split-K matrix-vector kernel's grid

// Matrix-vector kernels.  The band kernel needs no workspace; the split-K kernel needs
// gemv_workspace_bytes(M): arrival counters + two fp32 partial-sum slots per block.
constexpr int kMaxMulti = 4;             // matrices that one band-kernel launch can serve
struct GemvMatrix {                      // one packed weight matrix and its output
    const void* qweight;
    const void* scales;
    const void* zeros;
    void* y;
    int n;
};
bool gemv_uses_band_kernel(int M, int N, int sms);
size_t gemv_workspace_bytes(int M);
// `count` matrices (1..kMaxMulti) sharing x, K and the group size, in one launch.
// bits: 4, or 3 for qweight in the 3-bit storage (384 bytes per block).
// serialize: launch without programmatic stream serialization (the kernel then starts only after
// everything in front of it in the stream has completed, its weight prefetch included).
// sdiv: nullptr, or the inverse channel scales (fp32 [K], device): the kernel multiplies x by them
// while it fetches it; only where gemv_band_folds_scale(M, K, group) holds.
cudaError_t launch_gemv_band(const void* x, const GemvMatrix* mats, int count, int M, int K, int group,
                             unsigned int* status_word, int sms, bool serialize, cudaStream_t st,
                             const float* sdiv = nullptr, int bits = 4);
bool gemv_band_folds_scale(int M, int K, int group);
// tx_surplus: 0, or (time-out test only) bytes announced on every stage's barrier beyond what the copies bring
cudaError_t launch_gemv_splitk(const void* x, const void* qweight, const void* scales, const void* zeros,
                               void* y, int M, int N, int K, int group, void* workspace,
                               unsigned int* status_word, int sms, cudaStream_t st, int tx_surplus = 0);

// medium token counts (gemv_mid.cu): blocks own a chunk of K, partial sums per chunk in the
// workspace (behind its counter head), a second kernel adds the chunks
bool gemv_mid_applies(int M, int N, int K, int group, int sms);
size_t gemv_mid_workspace_bytes(int M, int N, int K);
cudaError_t launch_gemv_mid(const void* x, const void* qweight, const void* scales, const void* zeros, void* y,
                            int M, int N, int K, int group, void* workspace, unsigned int* status_word, int sms,
                            bool serialize, cudaStream_t st);

// The chunked kernels (gemv_mid.cu, gemm_skinny.cu): first unit of every block (and the end of the
// last one); units are in chunk-major order, `per_chunk` of them per chunk of K.  Blocks start in index order, the last
// ones on the SMs that the launch in front of this one frees last, so the blocks that hold one unit
// more than the others are the first ones - except where the longer range would cross into the next
// chunk, which costs a second slice of x (measured on 28672 -> 8192 at 8 tokens: 6 units 22.4 us, 7
// units 25 us, 7 units and a crossing 28 us; with the longer ranges simply in front 28672 -> 8192 went
// 32.3 -> 34.3 us while 8192 -> 28672 went 31.0 -> 28.7 us).
constexpr int kUnitMaxBlocks = 256;
struct UnitStarts {
    int v[kUnitMaxBlocks + 1];
};
inline UnitStarts unit_starts(int units, int per_chunk, int blocks) {
    UnitStarts s;
    int size[kUnitMaxBlocks];
    const int q = units / blocks;
    int extra = units - q * blocks, pos = 0;
    for (int b = 0; b < blocks; ++b) {
        const bool crosses = q > 0 && pos / per_chunk != (pos + q) / per_chunk;      // with q + 1 units
        size[b] = q + ((extra > 0 && !crosses) ? 1 : 0);
        extra -= size[b] - q;
        pos += size[b];
    }
    for (int b = blocks - 1; b >= 0 && extra > 0; --b)                  // what could not be placed so
        if (size[b] == q) { ++size[b]; --extra; }
    s.v[0] = 0;
    for (int b = 0; b < blocks; ++b) s.v[b + 1] = s.v[b] + size[b];
    for (int b = blocks + 1; b <= kUnitMaxBlocks; ++b) s.v[b] = s.v[blocks];
    return s;
}

// y[m][n] = fp16(sum over the chunks, ascending, of partial[c][m][n]), mn = M * N a multiple of 4;
// launched with programmatic stream serialization behind the kernel that wrote the partial sums
cudaError_t launch_chunk_reduce(const float* partial, void* y, int chunks, size_t mn, cudaStream_t st);

// 17 .. 64 tokens on the tensor cores (gemm_skinny.cu): units of one 128-channel slab x one chunk of
// K, the chunk's slice of x resident in shared memory, partial sums per chunk in the workspace
bool gemm_skinny_applies(int M, int N, int K, int group);
size_t gemm_skinny_workspace_bytes(int M, int N, int K, int group, int sms);
cudaError_t launch_gemm_skinny(const void* x, const void* qweight, const void* scales, const void* zeros, void* y,
                               int M, int N, int K, int group, void* workspace, unsigned int* status_word, int sms,
                               bool serialize, cudaStream_t st);

// scale search (search.cu)
constexpr int kMaxSearchAlphas = 64;
size_t search_scratch_bytes(int M, int N, int K, int group);
void search_carve(void* base, int M, int N, int K, int group, float** s, void** xs, void** qweight,
                  void** scales, void** zeros, void** yq, float** yref, double** partials, float** losses);
cudaError_t launch_reference_product(const void* W, const void* X, float* yref, int M, int N, int K,
                                     cudaStream_t st);
cudaError_t launch_divide_by_scale(const void* X, const float* s, void* xs, int M, int K, cudaStream_t st);
// xs = fp16_rne(fp32(X) * inv_s); inverse_scale: inv_s = fp32(1 / s), correctly rounded
cudaError_t launch_multiply_by_inverse(const void* X, const float* inv_s, void* xs, int M, int K, cudaStream_t st);
cudaError_t launch_inverse_scale(const float* s, float* inv_s, int K, cudaStream_t st);
cudaError_t launch_mean_squared_difference(const void* yq, const float* yref, size_t n, double* partials,
                                           float* out, cudaStream_t st);

// the matrix-vector kernel's built-in scratch (no allocation): address on the current device
cudaError_t gemv_static_scratch(void** out);
int gemv_static_max_m();

cudaError_t launch_gemm(const void* x, const void* qweight, const void* scales, const void* zeros,
                        void* y, int M, int N, int K, int group, bool path_pair_allowed,
                        void* workspace, size_t workspace_bytes,
                        unsigned int* status_word, cudaStream_t st);
// optional workspace of the tensor-core path (0 if the shape has no use for one)
size_t gemm_workspace_bytes(int M, int N, int sms);

}  // namespace awq
