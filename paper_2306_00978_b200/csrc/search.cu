// Scale search of the method (Sec. 3.2): for each alpha of a caller-given list, s = s_X^alpha
// (Eq. 5), quantize W diag(s) with the library's own quantizer, run the library's own layer on
// diag(s)^-1 X, and measure the output error against the fp16 layer W X (Eq. 4).  Everything
// that the search evaluates is therefore exactly what deployment will run.  The reference product
// W X is a plain dense fp16 GEMM with fp32 accumulation and output; it runs once per search, on
// a small warp-level tensor-core kernel of this file (no library call, no allocation).
#include "async_copy.cuh"
#include "common.cuh"

namespace awq {

namespace {

constexpr int kLossBlocks = 1024;

// xs[m][k] = fp16_rne(fp32(X[m][k]) / s[k]): the caller's side of Eq. 4, one IEEE division and
// one rounding per element; eight elements per thread (K is a multiple of 128).
__global__ void divide_by_scale_kernel(const __half* __restrict__ X, const float* __restrict__ s,
                                       __half* __restrict__ xs, size_t chunks, int K) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= chunks) return;
    const int k0 = (int)((i * 8) % (size_t)K);
    const uint4 h = reinterpret_cast<const uint4*>(X)[i];
    const uint32_t w[4] = {h.x, h.y, h.z, h.w};
    uint32_t o[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const float lo = __half2float(__ushort_as_half((unsigned short)(w[e] & 0xFFFFu)));
        const float hi = __half2float(__ushort_as_half((unsigned short)(w[e] >> 16)));
        const unsigned short a = __half_as_ushort(__float2half_rn(__fdiv_rn(lo, s[k0 + 2 * e])));
        const unsigned short b = __half_as_ushort(__float2half_rn(__fdiv_rn(hi, s[k0 + 2 * e + 1])));
        o[e] = (uint32_t)a | ((uint32_t)b << 16);
    }
    reinterpret_cast<uint4*>(xs)[i] = make_uint4(o[0], o[1], o[2], o[3]);
}

// xs[m][k] = fp16_rne(fp32(X[m][k]) * inv_s[k]): what awq_linear_scaled computes inside the layer,
// as a kernel of its own for the shapes whose kernel cannot fold it.
__global__ void multiply_by_inverse_kernel(const __half* __restrict__ X, const float* __restrict__ inv_s,
                                           __half* __restrict__ xs, size_t chunks, int K) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= chunks) return;
    const int k0 = (int)((i * 8) % (size_t)K);
    const uint4 h = reinterpret_cast<const uint4*>(X)[i];
    const uint32_t w[4] = {h.x, h.y, h.z, h.w};
    uint32_t o[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w[e]));
        const __half2 r = __floats2half2_rn(__fmul_rn(f.x, inv_s[k0 + 2 * e]), __fmul_rn(f.y, inv_s[k0 + 2 * e + 1]));
        o[e] = *reinterpret_cast<const uint32_t*>(&r);
    }
    reinterpret_cast<uint4*>(xs)[i] = make_uint4(o[0], o[1], o[2], o[3]);
}
__global__ void inverse_scale_kernel(const float* __restrict__ s, float* __restrict__ inv_s, int K) {
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k < K) inv_s[k] = __frcp_rn(s[k]);
}

// Sum of (y_q - y_ref)^2: every block adds a fixed, interleaved share of the elements in fp64
// and the last kernel adds the blocks' sums in block order, so the loss is reproducible.
__global__ void __launch_bounds__(256)
sqdiff_partial_kernel(const __half* __restrict__ yq, const float* __restrict__ yref, size_t n,
                      double* __restrict__ partials) {
    __shared__ double s_sum[256];
    double acc = 0.0;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const float d = __half2float(yq[i]) - yref[i];
        acc += (double)d * (double)d;
    }
    s_sum[threadIdx.x] = acc;
    __syncthreads();
    for (int off = 128; off >= 1; off >>= 1) {
        if ((int)threadIdx.x < off) s_sum[threadIdx.x] += s_sum[threadIdx.x + off];
        __syncthreads();
    }
    if (threadIdx.x == 0) partials[blockIdx.x] = s_sum[0];
}
__global__ void sqdiff_final_kernel(const double* __restrict__ partials, int blocks, double inv_count,
                                    float* __restrict__ out) {
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    double t = 0.0;
    for (int i = 0; i < blocks; ++i) t += partials[i];
    *out = (float)(t * inv_count);
}

size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

struct SearchScratch {
    float* s;
    __half* xs;
    unsigned char* qweight;
    unsigned char* scales;
    unsigned char* zeros;
    __half* yq;
    float* yref;
    double* partials;
    float* losses;
    size_t total;
};
SearchScratch carve(void* base, int M, int N, int K, int group) {
    SearchScratch r;
    size_t off = 0;
    auto take = [&](size_t bytes) { const size_t o = off; off += align256(bytes); return static_cast<unsigned char*>(base) + o; };
    r.s = reinterpret_cast<float*>(take((size_t)K * 4));
    r.xs = reinterpret_cast<__half*>(take((size_t)M * K * 2));
    r.qweight = take((size_t)N * K / 2);
    r.scales = take((size_t)(K / group) * N * 2);
    r.zeros = take((size_t)(K / group) * N / 2);
    r.yq = reinterpret_cast<__half*>(take((size_t)M * N * 2));
    r.yref = reinterpret_cast<float*>(take((size_t)M * N * 4));
    r.partials = reinterpret_cast<double*>(take((size_t)kLossBlocks * 8));
    r.losses = reinterpret_cast<float*>(take((size_t)kMaxSearchAlphas * 4));
    r.total = off;
    return r;
}

// ---------------------------------------------------------------- dense reference product
// C[m][n] = sum_k X[m][k] * W[n][k]: both operands have K contiguous, which is the row / column
// operand form of the warp-level m16n8k16 product.  128 tokens x 128 channels per block, 32
// input channels per step, two shared-memory buffers filled by 16-byte asynchronous copies, eight
// warps of 64 x 32 outputs each.  Rows of 80 bytes keep the 8 x 16-byte row reads of a matrix
// load on distinct banks.
constexpr int kRefBM = 128, kRefBN = 128, kRefBK = 32, kRefRow = 80;   // bytes per staged row
constexpr int kRefTile = 128 * kRefRow;                                // one operand tile of one buffer

__device__ __forceinline__ void cp_async_16(uint32_t dst, const void* src, bool valid) {
    const int n = valid ? 16 : 0;                                     // 0: the 16 bytes are zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(n) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}

__global__ void __launch_bounds__(256)
reference_product_kernel(const __half* __restrict__ W, const __half* __restrict__ X, float* __restrict__ C,
                         int M, int N, int K) {
    __shared__ __align__(16) unsigned char sm[2 * 2 * kRefTile];      // [buffer][X tile | W tile]
    const uint32_t sbase = smem_u32(sm);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int m0 = blockIdx.y * kRefBM, n0 = blockIdx.x * kRefBN;
    const int wm = (warp >> 2) * 64, wn = (warp & 3) * 32;            // this warp's corner inside the tile

    auto fill = [&](int buf, int k0) {
        // 128 rows x 4 pieces of 16 bytes per operand: two pieces of each operand per thread
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int piece = tid + i * 256, row = piece >> 2, c = piece & 3;
            const uint32_t dst = sbase + buf * (2 * kRefTile) + row * kRefRow + c * 16;
            const bool ok = m0 + row < M;
            cp_async_16(dst, X + (size_t)(ok ? m0 + row : 0) * K + k0 + c * 8, ok);
            cp_async_16(dst + kRefTile, W + (size_t)(n0 + row) * K + k0 + c * 8, true);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };

    float acc[4][4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[i][j][e] = 0.0f;

    const int steps = K / kRefBK;
    fill(0, 0);
    for (int s = 0; s < steps; ++s) {
        if (s + 1 < steps) {
            fill((s + 1) & 1, (s + 1) * kRefBK);
            asm volatile("cp.async.wait_group 1;" ::: "memory");
        } else {
            asm volatile("cp.async.wait_group 0;" ::: "memory");
        }
        __syncthreads();
        const uint32_t xa = sbase + (s & 1) * (2 * kRefTile), wa = xa + kRefTile;
#pragma unroll
        for (int kk = 0; kk < kRefBK; kk += 16) {
            uint32_t a[4][4], b[2][4];
#pragma unroll
            for (int i = 0; i < 4; ++i)   // rows wm + 16 i + (lane % 16), columns kk + 8 (lane / 16)
                ldmatrix_x4(a[i], xa + (wm + 16 * i + (lane & 15)) * kRefRow + (kk + 8 * (lane >> 4)) * 2);
#pragma unroll
            for (int j = 0; j < 2; ++j)   // channels wn + 16 j + (lane % 8) + 8 (lane / 16), columns kk + 8 ((lane / 8) % 2)
                ldmatrix_x4(b[j], wa + (wn + 16 * j + (lane & 7) + 8 * (lane >> 4)) * kRefRow + (kk + 8 * ((lane >> 3) & 1)) * 2);
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint32_t b0 = b[j >> 1][2 * (j & 1)], b1 = b[j >> 1][2 * (j & 1) + 1];
                    asm volatile(
                        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                        : "+f"(acc[i][j][0]), "+f"(acc[i][j][1]), "+f"(acc[i][j][2]), "+f"(acc[i][j][3])
                        : "r"(a[i][0]), "r"(a[i][1]), "r"(a[i][2]), "r"(a[i][3]), "r"(b0), "r"(b1));
                }
        }
        __syncthreads();                                              // the buffer is refilled two steps on
    }
    const int g = lane >> 2, t = lane & 3;
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int col = n0 + wn + 8 * j + 2 * t;
            const int r0 = m0 + wm + 16 * i + g, r1 = r0 + 8;
            if (r0 < M) *reinterpret_cast<float2*>(C + (size_t)r0 * N + col) = make_float2(acc[i][j][0], acc[i][j][1]);
            if (r1 < M) *reinterpret_cast<float2*>(C + (size_t)r1 * N + col) = make_float2(acc[i][j][2], acc[i][j][3]);
        }
}

}  // namespace

size_t search_scratch_bytes(int M, int N, int K, int group) {
    return carve(nullptr, M, N, K, group).total;
}

// y_ref[m][n] = sum_k X[m][k] W[n][k], fp32 [M][N] row-major.
cudaError_t launch_reference_product(const void* W, const void* X, float* yref, int M, int N, int K,
                                     cudaStream_t st) {
    const dim3 grid((unsigned)(N / kRefBN), (unsigned)((M + kRefBM - 1) / kRefBM));
    reference_product_kernel<<<grid, 256, 0, st>>>(reinterpret_cast<const __half*>(W),
                                                   reinterpret_cast<const __half*>(X), yref, M, N, K);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_divide_by_scale(const void* X, const float* s, void* xs, int M, int K, cudaStream_t st) {
    const size_t chunks = (size_t)M * K / 8;
    divide_by_scale_kernel<<<(unsigned)((chunks + 255) / 256), 256, 0, st>>>(
        reinterpret_cast<const __half*>(X), s, reinterpret_cast<__half*>(xs), chunks, K);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_multiply_by_inverse(const void* X, const float* inv_s, void* xs, int M, int K, cudaStream_t st) {
    const size_t chunks = (size_t)M * K / 8;
    multiply_by_inverse_kernel<<<(unsigned)((chunks + 255) / 256), 256, 0, st>>>(
        reinterpret_cast<const __half*>(X), inv_s, reinterpret_cast<__half*>(xs), chunks, K);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_inverse_scale(const float* s, float* inv_s, int K, cudaStream_t st) {
    inverse_scale_kernel<<<(K + 255) / 256, 256, 0, st>>>(s, inv_s, K);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_mean_squared_difference(const void* yq, const float* yref, size_t n, double* partials,
                                           float* out, cudaStream_t st) {
    sqdiff_partial_kernel<<<kLossBlocks, 256, 0, st>>>(reinterpret_cast<const __half*>(yq), yref, n, partials);
    sqdiff_final_kernel<<<1, 32, 0, st>>>(partials, kLossBlocks, 1.0 / (double)n, out);
    count_launch();
    count_launch();
    return cudaGetLastError();
}

void search_carve(void* base, int M, int N, int K, int group, float** s, void** xs, void** qweight,
                  void** scales, void** zeros, void** yq, float** yref, double** partials, float** losses) {
    const SearchScratch r = carve(base, M, N, K, group);
    *s = r.s; *xs = r.xs; *qweight = r.qweight; *scales = r.scales; *zeros = r.zeros;
    *yq = r.yq; *yref = r.yref; *partials = r.partials; *losses = r.losses;
}

}  // namespace awq
