/*
 * awq_b200.h - C ABI of the B200 (sm_100a) W4A16 group-wise linear layer.
 *
 * The layer is  y = x . dequant(Wq)^T  with  dequant(q) = (q - z) * Delta  per group of
 * `group` consecutive input channels of one output row, where Wq was obtained by
 * round-to-nearest quantization of W * diag(s),  s = s_X^alpha  (AWQ: Eq. 2 - Eq. 5 of the
 * paper; the fused dequantize + matrix-vector / matrix-matrix product is its Sec. 4.2).
 *
 * Conventions for every call
 *  - All data pointers are DEVICE pointers on the current CUDA device, 16-byte aligned,
 *    owned by the caller.  The library keeps no pointer after a call returns, except the
 *    workspace registered with awq_set_workspace.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *    Calls enqueue work and return; they never synchronize unless stated.
 *  - Return value: AWQ_OK (0) or a positive AwqStatus code.  Nothing is printed, thrown
 *    or aborted.  awq_status_string() names a code.
 *  - Shapes: N (output channels) a multiple of 128, K (input channels) a multiple of 128,
 *    group 64, 128, 256, 512 or 1024 (dividing K), M >= 1.  W is fp16 [N][K] row-major, x fp16
 *    [M][K] row-major, y fp16 [M][N] row-major.  The paper's setting is 128; the searches
 *    (awq_search_alpha, awq_search_clip) take 64 and 128 only.
 *
 * Packed layout (layout version 3, "band-major": all data of 16 consecutive output rows - a
 * band - is contiguous along K)
 *  qweight: N*K/2 bytes.  Block (band, kt) = rows 16*band..+15, columns 64*kt..+63 is 512
 *    bytes at ((n/16)*(K/64) + k/64) * 512.  A block is 32 pieces of 16 bytes, piece index
 *    4*g + t (g = 0..7, t = 0..3) holding rows g and g+8 of the band.  32-bit word j (j = 0..3,
 *    little-endian, at byte 4j of the piece) holds columns c = 16j+4t .. +3 of the block for
 *    both rows - so the four pieces of a row pair interleave along K in runs of four columns,
 *    and word j of all four pieces together covers columns 16j..16j+15 - as eight 4-bit slots
 *      (g,c) (g,c+1) (g+8,c) (g+8,c+1) (g,c+2) (g,c+3) (g+8,c+2) (g+8,c+3),
 *    slot e stored at bits 4p..4p+3 with p = {0,4,1,5,2,6,3,7}[e]  (read from the low
 *    nibble up, the slots appear in the order 0,2,4,6,1,3,5,7 - the GPU order of Sec. 4.2).
 *    As one formula: code (n,k) sits in the byte at
 *      ((n/16)*(K/64) + k/64)*512 + 16*(4*(n%8) + (k%16)/4) + 4*((k%64)/16) + {0,2,1,3}[k%4],
 *    in its low nibble if n%16 < 8, else in its high nibble: every byte holds the codes of rows
 *    g and g+8 of one column.
 *  Stored groups: scales and zero points are stored per group for group <= 128 and per 128
 *    columns above (each group's entry group / 128 times in a row): G below is min(group, 128).
 *  scales: fp16 [N/16][K/G][16] (band, stored group, row in band).
 *  zeros:  bytes [N/32][K/G][16]: per pair of bands and stored group, bytes 0-7 belong to the even
 *    band, 8-15 to the odd one; byte n%8 of a band holds the zero point of row n (n%16 < 8)
 *    in its low nibble and of row n+8 in its high nibble.
 */
#ifndef AWQ_B200_H_
#define AWQ_B200_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum AwqStatus {
    AWQ_OK = 0,
    AWQ_ERR_NULL_POINTER = 1,
    AWQ_ERR_BAD_SHAPE = 2,      /* N % 128, K % 128, K % group != 0, M < 1, or too large */
    AWQ_ERR_BAD_GROUP = 3,      /* group not 64, 128, 256, 512 or 1024 (the searches: not 64 or 128) */
    AWQ_ERR_BAD_ALPHA = 4,      /* alpha outside [0, 1] or NaN */
    AWQ_ERR_MISALIGNED = 5,     /* a pointer is not 16-byte aligned */
    AWQ_ERR_NO_WORKSPACE = 6,   /* the call needs more workspace than was registered */
    AWQ_ERR_WRONG_DEVICE = 7,   /* current device is not compute capability 10.x */
    AWQ_ERR_CUDA = 8,           /* a CUDA runtime / driver call failed */
    AWQ_ERR_TIMEOUT = 9,        /* a bounded device-side wait ran out (see awq_poll_status) */
    AWQ_ERR_BAD_ARGUMENT = 10,
    AWQ_ERR_STATIC_LIMIT = 11   /* awq_linear_gemv_static: problem larger than its built-in scratch */
} AwqStatus;

/* Which kernel awq_linear_path runs. */
typedef enum AwqPath {
    AWQ_PATH_AUTO = 0,          /* what awq_linear does: the matrix-vector kernels for M <= 8; the
                                   chunked matrix-vector kernel for 9 <= M <= 16 (up to 24 where
                                   N * K >= 2^25), and where K > 4096 already from 3 tokens
                                   (N * K >= 2^26; from 2 where K >= 12288) or 5 tokens (N * K >= 2^25), and the chunked
                                   tensor-core kernel for the other M <= 64 (N a multiple of 128), if
                                   a workspace of awq_workspace_bytes is registered; else the
                                   tensor-core prefill kernels */
    AWQ_PATH_GEMV = 1,          /* fused dequant matrix-vector kernel, M <= 16: band kernel when
                                   M <= 8 and N/16 is not much below the SM count, else split-K */
    AWQ_PATH_GEMM = 2,          /* tcgen05 tensor-core kernel, any M >= 1: pairs of SMs
                                   (cta_group::2, 256 channels x 256 tokens per tile) when N is a
                                   multiple of 256 and M > 128 (M > 64 from N = 8192, M >= 32 from
                                   N = 16384), else one SM per tile */
    AWQ_PATH_GEMV_SPLITK = 3,   /* the split-K matrix-vector kernel, M <= 16 */
    AWQ_PATH_GEMM_1SM = 4,      /* the tensor-core kernel with one SM per tile, any M >= 1 */
    AWQ_PATH_GEMV_MID = 5,      /* the chunked matrix-vector kernel, M <= 32: work units of 16 bands
                                   x 1024 input channels, the unit's slice of x in shared memory, one
                                   band per warp; needs a workspace of awq_workspace_bytes (fp32 partial
                                   sums per chunk of K) */
    AWQ_PATH_GEMM_SKINNY = 6    /* the chunked tensor-core kernel, M <= 64, N a multiple of 128: work
                                   units of 128 channels x a chunk of K, the chunk's slice of x resident
                                   in shared memory; needs a workspace of awq_workspace_bytes */
} AwqPath;

/* Sizes of the packed arrays, in bytes (0 if the shape is not accepted). */
size_t awq_qweight_bytes(int N, int K);
size_t awq_scales_bytes(int N, int K, int group);
size_t awq_zeros_bytes(int N, int K, int group);

/*
 * Offline step (Eq. 2 - Eq. 5): fold s = act_mean_abs^alpha into W, quantize each group of
 * `group` input channels of each row to 4-bit codes with an fp16 scale Delta and an integer
 * zero point in [0,15], and write the three packed arrays described above.
 *   s_k = 1 if alpha == 0 or act_mean_abs[k] is not finite or <= 0, else act_mean_abs[k]^alpha
 *         (alpha = 1: identity; alpha = 0.5: correctly rounded fp32 sqrt; else fp64 pow -> fp32)
 *   w'  = fp32(W) * s_k                               (one fp32 multiply, kept in fp32)
 *   Delta = fp16_rne((max w' - min w') / 15) over the group; 1.0 if that is 0 or not finite
 *   z   = clamp(rne(-min w' / Delta), 0, 15)          (fp32 division, round half to even)
 *   q   = clamp(rne(w' / Delta) + z, 0, 15)
 * W: in, fp16 [N][K].  act_mean_abs: in, fp32 [K], may be NULL iff alpha == 0.
 * qweight / scales / zeros: out, awq_*_bytes() bytes each, fully overwritten.
 * The result is a pure function of the inputs (bit-reproducible).
 */
int awq_quantize_pack(const void* W, const float* act_mean_abs, float alpha, int group,
                      void* qweight, void* scales, void* zeros, int N, int K, void* stream);

/*
 * The same offline step with the two variants the method also uses (Sec. 3.2 weight clipping;
 * the INT3-g128 setting of the accuracy tables):
 *   bits: 4 or 3.  bits = 3 quantizes to 8 levels (Delta = fp16_rne(range / 7), z and q in
 *         [0,7]); the 3-bit codes occupy the same 4-bit fields, so the packed arrays, their
 *         sizes and awq_linear are unchanged (the paper does not describe a 3-bit storage).
 *   symmetric: 0, or 1 for the grid of Eq. 2 as printed: Delta = fp16_rne(max|w'| / 2^(bits-1)),
 *         q = clamp(rne(w' / Delta) + 2^(bits-1), 0, 2^bits - 1) and the stored zero point is
 *         2^(bits-1) for every group (Round(w'/Delta) spans 2^bits + 1 values; the largest,
 *         reached only by a group's biggest positive element, saturates at the top code).
 *   clip_ratio: NULL, or in, device, fp32 [N][K/group] (row-major): the group's range becomes
 *         [r * min w', r * max w'] (one fp32 multiply each) before Delta and z are formed; values
 *         outside saturate at codes 0 and 2^bits - 1.  awq_search_clip produces such an array.
 * awq_quantize_pack(...) is awq_quantize_pack_ex(..., bits = 4, symmetric = 0, clip_ratio = NULL, ...).
 * awq_search_clip scores the asymmetric grid only; with symmetric = 1 a clip_ratio shrinks max|w'|.
 * Errors: as awq_quantize_pack; AWQ_ERR_BAD_ARGUMENT for other `bits` or `symmetric`.
 */
int awq_quantize_pack_ex(const void* W, const float* act_mean_abs, float alpha, int group, int bits,
                         int symmetric, const float* clip_ratio, void* qweight, void* scales, void* zeros,
                         int N, int K, void* stream);

/*
 * Weight clipping (Sec. 3.2 names it in one sentence - clipping chosen to minimise the squared
 * quantization error - and gives no algorithm; this is the reading used).  For every group of w' = fp32(W) * s and
 * every ratio r_i of `ratios`, the group is quantized as awq_quantize_pack_ex would with
 * clip_ratio = r_i, and
 *   err_i = sum over k ascending of ((q_k - z) * Delta - w'_k)^2
 * is formed in fp32, one IEEE operation per step (multiply, subtract, square, add), a NaN counting
 * as +inf; clip_ratio[n][g] = the first r_i of least err_i.  The result is bit-reproducible.
 * ratios: in, HOST, n_ratios values in (0, 1], 1 <= n_ratios <= 32, read during the call.
 * clip_ratio: out, device, fp32 [N][K/group].  W, act_mean_abs, alpha, group, bits as above.
 * Errors: AWQ_ERR_BAD_ARGUMENT for a bad list or `bits`; shape / pointer errors as listed in AwqStatus.
 */
int awq_search_clip(const void* W, const float* act_mean_abs, float alpha, int group, int bits,
                    const float* ratios, int n_ratios, float* clip_ratio, int N, int K, void* stream);

/* Eq. 5 alone: s[k] as used by awq_quantize_pack.  s: out, fp32 [K]. */
int awq_channel_scale(const float* act_mean_abs, float alpha, float* s, int K, void* stream);

/*
 * The layer itself (Sec. 4.2, on-the-fly dequantization fused into the product):
 *   y[m][n] = sum_g Delta[g][n] * sum_{k in g} (q[n][k] - z[g][n]) * x[m][k],  stored as fp16.
 * x must already be divided by s (the paper folds diag(s)^-1 into the previous operator).
 * x: in, fp16 [M][K].  y: out, fp16 [M][N], fully overwritten; must not alias an input.
 * Which kernel runs is listed under AWQ_PATH_AUTO.  The matrix-vector kernels (M <= 8, and the
 * chunked one up to 24 tokens) are HBM-bound: the 4-bit codes enter warp-level tensor-core products
 * exactly, accumulation, zero point and Delta are fp32, one rounding to fp16 at the end.  The
 * tcgen05 kernels (the chunked one up to 64 tokens, the prefill kernels above) round
 * (q - z) * Delta once to fp16 and accumulate in fp32 in tensor memory.  Results are
 * bit-reproducible.
 * Workspace.  The split-K matrix-vector kernel (small N, M <= 16) needs the registered workspace;
 * the chunked kernels (partial sums per chunk of K, added in ascending order by a second small
 * kernel) and the prefill kernels' split-K / stream-K use it when it holds awq_workspace_bytes,
 * else awq_linear falls back to a kernel that needs none.  Calls that use the workspace must not
 * overlap on the GPU (issue them on one stream).
 * Stream order.  x and y follow plain stream order.  The packed arrays are treated as constants
 * of the layer: the band and chunked kernels are launched with programmatic stream serialization
 * and start copying qweight, scales and zeros into shared memory BEFORE the work in front of them
 * in the stream has completed; only their reads of x and their writes of y and of the workspace
 * wait for that work.  The library covers its own writers: the first
 * layer call after an awq_quantize_pack / awq_quantize_pack_ex on the same device is launched
 * fully serialized.  A caller who produces packed arrays by other means (its own kernel, a
 * copy) must make sure they are complete before the operation that directly precedes
 * awq_linear in the stream begins - a stream or event synchronization, or any other kernel in
 * between that does not itself signal programmatic launch completion early, is enough.
 * Errors: AWQ_ERR_NO_WORKSPACE if the split-K matrix-vector kernel is chosen (M <= 8, small N) and
 * awq_workspace_bytes(M,N,K,group) exceeds the registered size; shape / pointer errors as listed
 * in AwqStatus.
 */
int awq_linear(const void* x, const void* qweight, const void* scales, const void* zeros,
               void* y, int M, int N, int K, int group, void* stream);

/*
 * Several layers that read the same x in one call (Sec. 4.2, kernel fusion: the paper fuses the
 * Q, K and V projections into a single kernel because at batch 1 a kernel's run time is
 * comparable to its launch overhead).  y_i = x . dequant(Wq_i)^T for i < count, count <= 4; all
 * matrices share K and `group`, each has its own N.  `problems` is a HOST array read during the
 * call.  For M <= 8 with enough output rows in total the matrices are served by ONE launch of
 * the matrix-vector band kernel; otherwise this is the same as `count` awq_linear calls.  Each
 * output is what awq_linear would give with the band kernel (bit-identical when awq_linear picks
 * that kernel for the matrix on its own, within the usual tolerance otherwise).
 */
typedef struct AwqLinearProblem {
    const void* qweight;   /* packed weights of matrix i (device) */
    const void* scales;
    const void* zeros;
    void* y;               /* out, fp16 [M][N] (device) */
    int N;
} AwqLinearProblem;
int awq_linear_multi(const void* x, const AwqLinearProblem* problems, int count,
                     int M, int K, int group, void* stream);

/*
 * The layer with diag(s)^-1 folded in (Sec. 3.2: the inverse scale goes into a neighbouring operator,
 * so that no separate pass over the activations and no extra kernel launch is needed; Sec. 4.2: at
 * batch 1 a launch costs as much as the kernel).
 *   y = awq_linear(x', ...),   x'[m][k] = fp16_rne(fp32(x[m][k]) * inv_s[k])   (one fp32 multiply, one rounding)
 * - bit for bit what the caller would get by forming x' itself and calling awq_linear /
 * awq_linear_multi.  x: in, fp16 [M][K], NOT scaled.  inv_s: in, device, fp32 [K], 16-byte aligned:
 * 1 / s for the alpha the weights were quantized with (awq_inverse_channel_scale gives the correctly
 * rounded reciprocal of what awq_channel_scale gives); like the packed arrays it is a constant of
 * the layer and may be read before the stream dependency resolves.  (A multiplication, not the
 * division x / s: eight IEEE divisions per thread in the start-up of a launch that lasts a few
 * microseconds cost 0.3 - 1.5 us per launch; x * (1 / s) and x / s differ in the last bit of the fp16
 * result for a few elements in a thousand, which the method does not care about as long as the
 * quantizer's s and this inv_s belong together.)
 * Where the band matrix-vector kernel serves the call (M <= 8, enough output rows) and can keep x
 * on chip (K = 4096, or M <= 2 and M * K small enough for shared memory) the scaling happens while
 * the kernel fetches x: no extra launch, no extra memory.  Otherwise x' is first written to
 * x_scratch (device, fp16 [M][K], caller-owned) by a small kernel and the plain call follows;
 * x_scratch may be NULL if awq_linear_scaled_needs_scratch(M, N, K, group) returns 0 (for the
 * multi call: N = the sum of the matrices' N), else AWQ_ERR_NULL_POINTER.
 */
int awq_linear_scaled(const void* x, const float* inv_s, void* x_scratch, const void* qweight, const void* scales,
                      const void* zeros, void* y, int M, int N, int K, int group, void* stream);
int awq_linear_multi_scaled(const void* x, const float* inv_s, void* x_scratch, const AwqLinearProblem* problems,
                            int count, int M, int K, int group, void* stream);
/* inv_s[k] = fp32(1 / s[k]) (correctly rounded), s as awq_channel_scale gives it.  inv_s: out, fp32 [K]. */
int awq_inverse_channel_scale(const float* act_mean_abs, float alpha, float* inv_s, int K, void* stream);
int awq_linear_scaled_needs_scratch(int M, int N, int K, int group);

/*
 * 3-bit storage (the INT3-g128 setting of the paper's accuracy tables; the paper does not describe
 * how its kernels would store 3-bit codes, this is the layout used).  awq_quantize_pack_ex with
 * bits = 3 writes 3-bit codes into the 4-bit layout; awq_pack_int3 turns that array into the
 * dense one of 3/8 byte per weight, awq_unpack_int3 back:
 *  qweight3: N*K*3/8 bytes.  Bands, blocks and pieces are those of the 4-bit layout, but a block
 *    (band, kt) is 384 bytes at ((n/16)*(K/64) + k/64) * 384 and piece 4*g + t is 12 bytes = three
 *    little-endian words at byte 12*(4*g + t) of the block.  Let (j, p) be the word and the nibble
 *    that the 4-bit layout gives code (n,k) inside its piece (j = (k%64)/16, p from the slot table
 *    above).  For j < 3 the code keeps its place: bits 4p .. 4p+2 of word j.  For j = 3 (columns
 *    48..63 of the block) bit b of the code (b = 0, 1, 2) sits in the spare top bit of nibble p of
 *    word b: bit 4p+3 of word b.  In words: u_b = w_b | (((w_3 >> b) & 0x11111111) << 3).
 *  scales and zeros are unchanged.
 * awq_linear_int3: the layer on that storage.  Where the band matrix-vector kernel serves the call
 * (M <= 8 and N / 16 not far below the SM count) it streams the 3-bit array itself, 25 % fewer
 * weight bytes than the 4-bit layout; other shapes (split-K and tensor-core kernels read the
 * 4-bit layout) are first expanded into qweight_scratch (device, awq_qweight_bytes(N, K) bytes,
 * caller-owned; may be NULL when the band kernel applies, else AWQ_ERR_NULL_POINTER) and run as
 * awq_linear.  Results equal awq_linear on the expanded array bit for bit where the same kernel runs.
 */
size_t awq_qweight_bytes_int3(int N, int K);
int awq_pack_int3(const void* qweight, void* qweight3, int N, int K, void* stream);
int awq_unpack_int3(const void* qweight3, void* qweight, int N, int K, void* stream);
int awq_linear_int3(const void* x, const void* qweight3, const void* scales, const void* zeros, void* y,
                    void* qweight_scratch, int M, int N, int K, int group, void* stream);

/* Same as awq_linear with the kernel forced (for the small-batch crossover measurement).
 * A matrix-vector path with M > 16 or K > 65536 returns AWQ_ERR_BAD_SHAPE. */
int awq_linear_path(const void* x, const void* qweight, const void* scales, const void* zeros,
                    void* y, int M, int N, int K, int group, int path, void* stream);

/*
 * The matrix-vector kernel of awq_linear for callers that cannot allocate device memory.
 * (The paper has no counterpart: this is a deployment variant of the same computation.)
 *
 * Some hosts of this library may not call cudaMalloc at all - for example an inference
 * server whose memory pool owns the whole device and forbids allocations after start-up, or
 * code running where an allocation would synchronize the device or fail.  Such callers
 * cannot provide the workspace awq_set_workspace expects.  This entry point needs none: the
 * kernel's scratch (arrival counters and fp32 partial sums) lives in an array that is part
 * of the library's device image, about 2 MB, held by every GPU that loads the library until
 * the process exits.  The call itself allocates nothing: no cudaMalloc, no cudaFree, no
 * allocating library routine.
 *
 * Arguments, layouts and result are those of awq_linear with the split-K matrix-vector
 * kernel; the output is bit-identical to awq_linear_path(..., AWQ_PATH_GEMV_SPLITK, ...).
 * Limits: M <= 8 and K <= 65536; anything larger returns AWQ_ERR_STATIC_LIMIT and does nothing.
 * The first call on a device looks up the scratch array's device address (this can load the
 * library's device code), so make that first call before any stream capture begins.
 * All calls on a device share the one array, and each call re-zeroes its counters on `stream`
 * before the kernel: two calls that overlap on the GPU (different streams, or one stream with
 * work that is allowed to overlap) race and give undefined output.  Issue them on one stream.
 */
int awq_linear_gemv_static(const void* x, const void* qweight, const void* scales, const void* zeros,
                            void* y, int M, int N, int K, int group, void* stream);
/* Test aid for the entry point above (the paper has no counterpart): overwrites the arrival
 * counters at the head of the built-in scratch with the byte `value` on `stream`, as a call that
 * was cut short might leave them; awq_linear_gemv_static must still give the right result.
 * Allocates nothing. */
int awq_static_scratch_fill(int value, void* stream);

/*
 * Scale search (Sec. 3.2).  For each alpha_i of `alphas`: s = s_X^alpha_i (Eq. 5, s_X = act_mean_abs),
 * Wq = awq_quantize_pack(W, s), and
 *   loss_i = mean over (m, n) of ( awq_linear(fp16(X / s), Wq)[m][n] - sum_k X[m][k] W[n][k] )^2   (Eq. 4;
 * the paper does not name its norm: the mean squared difference has the same minimizer as any other
 * monotone function of the Frobenius norm).  The quantizer and the layer are the library's own
 * kernels, so the search scores exactly what deployment runs; the fp16 reference product W X is a
 * dense GEMM kernel of this library with fp32 accumulation and output.  Nothing is allocated: all
 * intermediate arrays live in `scratch`.  The paper uses 20 grid points over [0, 1]; the grid is the
 * caller's.
 * W: in, fp16 [N][K] (device).  act_mean_abs: in, fp32 [K] (device).  X: in, fp16 [M][K] calibration
 * activations (device), M >= 1.  alphas: in, HOST array of n_alphas <= 64 values in [0, 1].
 * losses: out, HOST array of n_alphas floats.  best_index: out, HOST, index of the first least loss
 * (a loss that is not finite is never chosen unless all are).  scratch: device memory of at least
 * awq_search_scratch_bytes(M, N, K, group) bytes, 256-byte aligned, owned by the caller.
 * The call enqueues on `stream` and then SYNCHRONIZES it (the result is returned on the host); it
 * must not run inside a stream capture.  A registered workspace is used as awq_linear uses it.
 * Errors: those of awq_quantize_pack and awq_linear; AWQ_ERR_BAD_ARGUMENT for a bad list or a
 * scratch that is too small.
 */
size_t awq_search_scratch_bytes(int M, int N, int K, int group);
int awq_search_alpha(const void* W, const float* act_mean_abs, const void* X, int M, int N, int K, int group,
                     const float* alphas, int n_alphas, float* losses, int* best_index,
                     void* scratch, size_t scratch_bytes, void* stream);

/* Workspace (scratch for partial sums and arrival counters).
 * awq_workspace_bytes: bytes awq_linear can use for this problem (0 if none).  For M <= 16 the
 * split-K matrix-vector kernel (small N) REQUIRES them.  For everything else they are OPTIONAL and
 * decide which kernel awq_linear takes:
 *  - the chunked kernels (AWQ_PATH_GEMV_MID up to 24 tokens, AWQ_PATH_GEMM_SKINNY up to 64) keep one
 *    fp32 [M][N] array of partial sums per chunk of K there; a second small kernel adds the chunks
 *    in ascending order.  Without a workspace of this size awq_linear takes the band
 *    matrix-vector kernel (M <= 8) or the prefill kernels instead (same result within the
 *    tolerance, slower);
 *  - the one-SM prefill kernel (M <= 128) splits each tile's K loop over several SMs (up to 16
 *    splits, fp32 partial sums added in split order by whichever SM finishes a tile last), which
 *    keeps all SMs busy when N / 128 is below the SM count;
 *  - the SM-pair prefill kernel (see AWQ_PATH_GEMM) cuts the tiles' K loops into equal ranges over
 *    all SM pairs (stream-K) and sums split tiles in a fixed order; without a workspace whole tiles
 *    go round-robin (same result up to fp32 summation order, slower when the tile count is not a
 *    multiple of the pair count).
 * awq_set_workspace: registers caller-owned device memory for the current device; the first
 * 4096 bytes are cleared with a synchronous cudaMemset.  Pass (NULL, 0) to unregister.
 * The memory must stay valid until it is unregistered or replaced. */
size_t awq_workspace_bytes(int M, int N, int K, int group);
int awq_set_workspace(void* dev_ptr, size_t bytes);

/* Test / debug: expand the packed arrays into canonical ones.
 * codes: out u8 [N][K]; scales_nk: out fp16 bits [N][K/group]; zeros_nk: out u8 [N][K/group]. */
int awq_unpack_canonical(const void* qweight, const void* scales, const void* zeros,
                         int N, int K, int group,
                         uint8_t* codes, uint16_t* scales_nk, uint8_t* zeros_nk, void* stream);

/* Reads and clears the device status word of the current device (synchronizes the device).
 * Returns AWQ_OK, or AWQ_ERR_TIMEOUT if a kernel gave up a bounded wait since the last poll
 * (its output is then undefined; the arrival counters at the head of the registered workspace
 * are cleared again so that later calls start clean), or AWQ_ERR_CUDA. */
int awq_poll_status(void);

/* How long a device-side wait (on a copy, on another block's partial sums) may last before the
 * kernel gives it up, records AWQ_ERR_TIMEOUT for awq_poll_status and runs to its end: default
 * about two seconds; 0 restores the default.  Applies to the current device; synchronizes it. */
int awq_set_wait_limit_us(unsigned int microseconds);
/* Test aid for the time-out path (no fault, trap or endless loop is involved): the next split-K
 * matrix-vector launch on the current device (awq_linear_path with AWQ_PATH_GEMV_SPLITK, or
 * awq_linear where it picks that kernel) announces 16 bytes more on each stage's copy barrier than
 * its copies deliver, so its first wait runs into the limit set with awq_set_wait_limit_us; the
 * kernel then returns by itself with undefined output.  One launch only; later calls are normal. */
int awq_test_stall_next_gemv(void);

const char* awq_status_string(int status);
/* Text of the last CUDA error seen by the calling thread's library calls ("" if none). */
const char* awq_last_cuda_error(void);
int awq_layout_version(void);
/* Number of kernels this library has launched in this process (all threads). */
unsigned long long awq_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* AWQ_B200_H_ */
