// Scale search of the method (Sec. 3.2): for each alpha of a caller-given list, s = s_X^alpha
// (Eq. 5), quantize W diag(s) with the library's own quantizer, run the library's own layer on
// diag(s)^-1 X, and measure the output error against the fp16 layer W X (Eq. 4).  Everything
// that the search evaluates is therefore exactly what deployment will run.  The reference product
// W X is a plain dense GEMM and comes from cuBLAS (fp16 inputs, fp32 accumulate and output).
#include <cublas_v2.h>

#include <mutex>

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

cublasHandle_t cublas_for_current_device(cublasStatus_t* status) {
    static std::mutex mu;
    static cublasHandle_t handles[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    std::lock_guard<std::mutex> lock(mu);
    *status = CUBLAS_STATUS_SUCCESS;
    if (!handles[dev & 63]) *status = cublasCreate(&handles[dev & 63]);
    return handles[dev & 63];
}

}  // namespace

size_t search_scratch_bytes(int M, int N, int K, int group) {
    return carve(nullptr, M, N, K, group).total;
}

// y_ref[m][n] = sum_k X[m][k] W[n][k], fp32 [M][N] row-major.
cudaError_t launch_reference_product(const void* W, const void* X, float* yref, int M, int N, int K,
                                     cudaStream_t st) {
    cublasStatus_t cs;
    cublasHandle_t h = cublas_for_current_device(&cs);
    if (cs != CUBLAS_STATUS_SUCCESS) return cudaErrorInitializationError;
    if (cublasSetStream(h, st) != CUBLAS_STATUS_SUCCESS) return cudaErrorUnknown;
    const float one = 1.0f, zero = 0.0f;
    // column-major view: C^T (N x M) = W^T-view (N x K) * X-view (K x M)
    cs = cublasGemmEx(h, CUBLAS_OP_T, CUBLAS_OP_N, N, M, K, &one, W, CUDA_R_16F, K, X, CUDA_R_16F, K, &zero,
                      yref, CUDA_R_32F, N, CUBLAS_COMPUTE_32F, CUBLAS_GEMM_DEFAULT);
    return cs == CUBLAS_STATUS_SUCCESS ? cudaSuccess : cudaErrorUnknown;
}

cudaError_t launch_divide_by_scale(const void* X, const float* s, void* xs, int M, int K, cudaStream_t st) {
    const size_t chunks = (size_t)M * K / 8;
    divide_by_scale_kernel<<<(unsigned)((chunks + 255) / 256), 256, 0, st>>>(
        reinterpret_cast<const __half*>(X), s, reinterpret_cast<__half*>(xs), chunks, K);
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
