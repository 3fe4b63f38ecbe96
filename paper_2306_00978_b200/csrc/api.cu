// C ABI of the library: argument checks, dispatch, workspace and status bookkeeping.
#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>

#include "common.cuh"

namespace awq {

namespace {

constexpr int kMaxDevices = 64;
std::atomic<unsigned long long> g_launches{0};
thread_local char t_cuda_error[256] = "";

struct DeviceState {
    void* workspace = nullptr;
    size_t workspace_bytes = 0;
    unsigned int* status_word = nullptr;   // device address of g_status on this device
    int cc_major = -1;
    int sms = 0;
    int tx_surplus_once = 0;               // time-out test: see awq_test_stall_next_gemv
    // Set when one of this library's kernels that writes packed arrays (the quantizer) has been
    // enqueued since the last matrix-vector launch: the band kernel prefetches weights before its
    // stream dependency resolves, so the first launch after such a writer is fully serialized.
    bool packed_written = false;
};
DeviceState g_dev[kMaxDevices];
std::mutex g_mutex;

// [0]: 0, or a code written by a kernel that gave up a wait; [1]: limit of a device-side wait in
// microseconds (0 = the built-in default)
__device__ unsigned int g_status[2];

int note_cuda(cudaError_t e) {
    if (e == cudaSuccess) return AWQ_OK;
    std::snprintf(t_cuda_error, sizeof(t_cuda_error), "%s: %s", cudaGetErrorName(e), cudaGetErrorString(e));
    return AWQ_ERR_CUDA;
}

// Per-device set-up on first use: compute capability and the status word's device address.
int device_state(DeviceState** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return note_cuda(e);
    if (dev < 0 || dev >= kMaxDevices) return AWQ_ERR_WRONG_DEVICE;
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceState& d = g_dev[dev];
    if (d.cc_major < 0) {
        int major = 0;
        e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
        if (e != cudaSuccess) return note_cuda(e);
        if (major == 10) {
            void* p = nullptr;
            e = cudaGetSymbolAddress(&p, g_status);
            if (e != cudaSuccess) return note_cuda(e);
            e = cudaMemset(p, 0, 2 * sizeof(unsigned int));
            if (e != cudaSuccess) return note_cuda(e);
            d.status_word = reinterpret_cast<unsigned int*>(p);
        }
        e = cudaDeviceGetAttribute(&d.sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return note_cuda(e);
        d.cc_major = major;
    }
    if (d.cc_major != 10) return AWQ_ERR_WRONG_DEVICE;
    *out = &d;
    return AWQ_OK;
}

// True once after a packed-array writer of this library was enqueued on the device.
bool take_packed_written(DeviceState* d) {
    std::lock_guard<std::mutex> lock(g_mutex);
    const bool w = d->packed_written;
    d->packed_written = false;
    return w;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Scales and zero points are stored per group up to 128 columns and per 128 columns above (each
// group's entry group / 128 times), so the layer kernels see groups of 64 or 128 only.
int stored_group(int group) { return group > 128 ? 128 : group; }

int check_shape(int N, int K, int group) {
    if (group != 64 && group != 128 && group != 256 && group != 512 && group != 1024) return AWQ_ERR_BAD_GROUP;
    if (N < 128 || K < 128 || N % 128 != 0 || K % 128 != 0 || K % group != 0) return AWQ_ERR_BAD_SHAPE;
    if (N / 128 > kMaxSlabs) return AWQ_ERR_BAD_SHAPE;
    if ((long long)N * K > (1LL << 33)) return AWQ_ERR_BAD_SHAPE;
    return AWQ_OK;
}

}  // namespace

void count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }

}  // namespace awq

using namespace awq;

extern "C" {

size_t awq_qweight_bytes(int N, int K) {
    return check_shape(N, K, 128) == AWQ_OK ? (size_t)N * K / 2 : 0;
}
size_t awq_scales_bytes(int N, int K, int group) {
    return check_shape(N, K, group) == AWQ_OK ? (size_t)(K / stored_group(group)) * N * 2 : 0;
}
size_t awq_zeros_bytes(int N, int K, int group) {
    return check_shape(N, K, group) == AWQ_OK ? (size_t)(K / stored_group(group)) * N / 2 : 0;
}

int awq_channel_scale(const float* act_mean_abs, float alpha, float* s, int K, void* stream) {
    if (!(alpha >= 0.0f && alpha <= 1.0f)) return AWQ_ERR_BAD_ALPHA;
    if (!s || (!act_mean_abs && alpha != 0.0f)) return AWQ_ERR_NULL_POINTER;
    if (K < 1) return AWQ_ERR_BAD_SHAPE;
    DeviceState* d;
    if (int rc = device_state(&d)) return rc;
    return note_cuda(launch_channel_scale(act_mean_abs, alpha, s, K, (cudaStream_t)stream));
}

int awq_quantize_pack_ex(const void* W, const float* act_mean_abs, float alpha, int group, int bits,
                         int symmetric, const float* clip_ratio, void* qweight, void* scales, void* zeros,
                         int N, int K, void* stream) {
    if (!(alpha >= 0.0f && alpha <= 1.0f)) return AWQ_ERR_BAD_ALPHA;
    if (int rc = check_shape(N, K, group)) return rc;
    if ((bits != 3 && bits != 4) || (symmetric != 0 && symmetric != 1)) return AWQ_ERR_BAD_ARGUMENT;
    if (!W || !qweight || !scales || !zeros || (!act_mean_abs && alpha != 0.0f)) return AWQ_ERR_NULL_POINTER;
    if (!aligned16(W) || !aligned16(qweight) || !aligned16(scales) || !aligned16(zeros) ||
        (reinterpret_cast<uintptr_t>(act_mean_abs) & 3u) || (reinterpret_cast<uintptr_t>(clip_ratio) & 3u))
        return AWQ_ERR_MISALIGNED;
    DeviceState* d;
    if (int rc = device_state(&d)) return rc;
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        d->packed_written = true;
    }
    return note_cuda(launch_quantize_pack(reinterpret_cast<const __half*>(W), act_mean_abs, alpha, group, bits,
                                          symmetric != 0, clip_ratio, reinterpret_cast<uint32_t*>(qweight),
                                          reinterpret_cast<__half*>(scales),
                                          reinterpret_cast<uint8_t*>(zeros), N, K, (cudaStream_t)stream));
}

int awq_quantize_pack(const void* W, const float* act_mean_abs, float alpha, int group,
                      void* qweight, void* scales, void* zeros, int N, int K, void* stream) {
    return awq_quantize_pack_ex(W, act_mean_abs, alpha, group, 4, 0, nullptr, qweight, scales, zeros, N, K, stream);
}

int awq_search_clip(const void* W, const float* act_mean_abs, float alpha, int group, int bits,
                    const float* ratios, int n_ratios, float* clip_ratio, int N, int K, void* stream) {
    if (!(alpha >= 0.0f && alpha <= 1.0f)) return AWQ_ERR_BAD_ALPHA;
    if (int rc = check_shape(N, K, group)) return rc;
    if (group > 128) return AWQ_ERR_BAD_GROUP;
    if ((bits != 3 && bits != 4) || n_ratios < 1 || n_ratios > kMaxClipRatios) return AWQ_ERR_BAD_ARGUMENT;
    if (!W || !ratios || !clip_ratio || (!act_mean_abs && alpha != 0.0f)) return AWQ_ERR_NULL_POINTER;
    if ((reinterpret_cast<uintptr_t>(W) & 1u) || (reinterpret_cast<uintptr_t>(act_mean_abs) & 3u) ||
        (reinterpret_cast<uintptr_t>(clip_ratio) & 3u))
        return AWQ_ERR_MISALIGNED;
    for (int i = 0; i < n_ratios; ++i)
        if (!(ratios[i] > 0.0f && ratios[i] <= 1.0f)) return AWQ_ERR_BAD_ARGUMENT;
    DeviceState* d;
    if (int rc = device_state(&d)) return rc;
    return note_cuda(launch_clip_search(reinterpret_cast<const __half*>(W), act_mean_abs, alpha, group, bits,
                                        ratios, n_ratios, clip_ratio, N, K, (cudaStream_t)stream));
}

// Where the chunked matrix-vector kernel beats the tensor-core kernels (measured, us, chunked against
// tensor-core: at 16 tokens 10.9 / 13.5 on 4096 -> 4096, 17.4 / 25.9 on 4096 -> 11008, 20.9 / 26.2 on
// 11008 -> 4096, 45 / 98 on 8192 -> 28672; at 24 tokens 14.0 / 13.9, 23.2 / 26.1, 27.4 / 26.2, 60.7 / 98;
// at 32 tokens 17.6 / 13.8, 28.4 / 25.8, 33.4 / 26.4, 79 / 81).
// With one token fragment its time does not depend on M (32 us on the 70B shapes for 1 .. 8 tokens),
// while the band kernel's grows with the tokens that travel through its stages.  Chunked / band, us:
//   8192 -> 28672   3 tokens 31.3 / 34.5   5: 31.9 / 38.9   8: 32.5 / 49.1
//   8192 -> 16384   3: 19.1 / 20.4   4: 19.2 / 20.7   8: 19.5 / 29.2
//   8192 -> 8192    3: 13.0 / 13.0   4: 12.8 / 13.4   8: 13.2 / 18.7
//   13824 -> 5120   3: 14.7 / 16.3   4: 14.8 / 17.5   8: 15.0 / 24.1
//   5120 -> 13824   3: 13.6 / 13.4   4: 13.6 / 13.8   5: 13.7 / 15.1
//   11008 -> 4096   4: 12.9 / 11.3   5: 13.1 / 12.9   6: 13.3 / 14.8   8: 13.1 / 16.1
// With 4096 input channels the band kernel keeps x in registers and wins up to 8 tokens
// (4096 -> 11008 at 8 tokens: 11.7 / 9.8; 4096 -> 4096: 6.5 / 6.9).
static bool mid_kernel_preferred(int M, int N, int K) {
    const long long nk = (long long)N * K;
    if (M < 2) return false;
    if (M == 2) return K >= 12288 && nk >= (1LL << 26);   // 13824 -> 5120: 13.6 / 14.2 us, 28672 -> 8192: 32.3 / 33.5 us
    if (M <= 8) return K > 4096 && nk >= (M <= 4 ? (1LL << 26) : (1LL << 25));
    if (M <= 16) return true;
    return M <= 24 && nk >= (1LL << 25);
}

static int resolve_path(int M, int K, int path) {
    if (path == AWQ_PATH_AUTO) return (M <= 8 && K <= 65536) ? AWQ_PATH_GEMV : AWQ_PATH_GEMM;
    return path;
}

size_t awq_workspace_bytes(int M, int N, int K, int group) {
    if (check_shape(N, K, group) != AWQ_OK || M < 1) return 0;
    group = stored_group(group);
    // optional for the tensor-core kernels: with it they spread their work evenly over the SMs
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
        (void)cudaGetLastError();
        sms = 160;                           // no device to ask: an upper bound for this GPU family
    }
    size_t gemm = gemm_workspace_bytes(M, N, sms);
    const size_t mid = (M <= 32 && gemv_mid_applies(M, N, K, group, sms)) ? gemv_mid_workspace_bytes(M, N, K) : 0;
    if (M > 8 && mid > gemm) gemm = mid;
    if (M > 8 && gemm_skinny_applies(M, N, K, group)) {
        const size_t skinny = gemm_skinny_workspace_bytes(M, N, K, group, sms);
        if (skinny > gemm) gemm = skinny;
    }
    if (M > 16) return gemm;
    const size_t gemv = gemv_workspace_bytes(M);   // required by the split-K matrix-vector kernel
    if (M <= 8) return gemv > mid ? gemv : mid;    // awq_linear never takes the tensor-core kernel here
    return gemv > gemm ? gemv : gemm;
}

int awq_set_workspace(void* dev_ptr, size_t bytes) {
    DeviceState* d;
    if (int rc = device_state(&d)) return rc;
    if ((dev_ptr == nullptr) != (bytes == 0)) return AWQ_ERR_BAD_ARGUMENT;
    if (dev_ptr) {
        if (!aligned16(dev_ptr)) return AWQ_ERR_MISALIGNED;
        if (bytes < kCounterBytes) return AWQ_ERR_BAD_ARGUMENT;
        if (int rc = note_cuda(cudaMemset(dev_ptr, 0, kCounterBytes))) return rc;
    }
    std::lock_guard<std::mutex> lock(g_mutex);
    d->workspace = dev_ptr;
    d->workspace_bytes = bytes;
    return AWQ_OK;
}

int awq_linear_path(const void* x, const void* qweight, const void* scales, const void* zeros,
                    void* y, int M, int N, int K, int group, int path, void* stream) {
    if (int rc = check_shape(N, K, group)) return rc;
    group = stored_group(group);
    if (M < 1 || (long long)M * K > (1LL << 40) || (long long)M * N > (1LL << 40)) return AWQ_ERR_BAD_SHAPE;
    if (!x || !qweight || !scales || !zeros || !y) return AWQ_ERR_NULL_POINTER;
    if (!aligned16(x) || !aligned16(qweight) || !aligned16(scales) || !aligned16(zeros) || !aligned16(y))
        return AWQ_ERR_MISALIGNED;
    if (path != AWQ_PATH_AUTO && path != AWQ_PATH_GEMV && path != AWQ_PATH_GEMM && path != AWQ_PATH_GEMV_SPLITK &&
        path != AWQ_PATH_GEMM_1SM && path != AWQ_PATH_GEMV_MID && path != AWQ_PATH_GEMM_SKINNY)
        return AWQ_ERR_BAD_ARGUMENT;
    const bool automatic = path == AWQ_PATH_AUTO;
    path = resolve_path(M, K, path);
    if (path == AWQ_PATH_GEMV_MID) {
        if (M > 32 || K > 65536) return AWQ_ERR_BAD_SHAPE;
    } else if (path == AWQ_PATH_GEMM_SKINNY) {
        if (!gemm_skinny_applies(M, N, K, group)) return AWQ_ERR_BAD_SHAPE;
    } else if (path != AWQ_PATH_GEMM && path != AWQ_PATH_GEMM_1SM && (M > 16 || K > 65536)) {
        return AWQ_ERR_BAD_SHAPE;
    }
    DeviceState* d;
    if (int rc = device_state(&d)) return rc;
    if (automatic && mid_kernel_preferred(M, N, K) && gemv_mid_applies(M, N, K, group, d->sms)) {
        std::lock_guard<std::mutex> lock(g_mutex);
        if (d->workspace_bytes >= gemv_mid_workspace_bytes(M, N, K)) path = AWQ_PATH_GEMV_MID;
    }
    if (automatic && path == AWQ_PATH_GEMM && M > 16 && M <= 64 && gemm_skinny_applies(M, N, K, group)) {
        // 17 .. 64 tokens: the chunked tensor-core kernel (measured against the prefill kernels at 32
        // and 64 tokens: 10.1 / 13.7 and 11.1 / 16.1 us on 4096 -> 4096, 20.7 / 26.2 and 20.8 / 31.4 us
        // on 4096 -> 11008, 66.5 / 80.9 and 73.5 / 81.2 us on 8192 -> 28672)
        std::lock_guard<std::mutex> lock(g_mutex);
        if (d->workspace_bytes >= gemm_skinny_workspace_bytes(M, N, K, group, d->sms)) path = AWQ_PATH_GEMM_SKINNY;
    }
    if (path == AWQ_PATH_GEMV_MID) {
        if (!gemv_mid_applies(M, N, K, group, d->sms)) return AWQ_ERR_BAD_SHAPE;
        void* ws = nullptr;
        {
            std::lock_guard<std::mutex> lock(g_mutex);
            if (d->workspace_bytes < gemv_mid_workspace_bytes(M, N, K)) return AWQ_ERR_NO_WORKSPACE;
            ws = d->workspace;
        }
        return note_cuda(launch_gemv_mid(x, qweight, scales, zeros, y, M, N, K, group, ws, d->status_word, d->sms,
                                         take_packed_written(d), (cudaStream_t)stream));
    }
    if (path == AWQ_PATH_GEMM_SKINNY) {
        void* ws = nullptr;
        {
            std::lock_guard<std::mutex> lock(g_mutex);
            if (d->workspace_bytes < gemm_skinny_workspace_bytes(M, N, K, group, d->sms)) return AWQ_ERR_NO_WORKSPACE;
            ws = d->workspace;
        }
        return note_cuda(launch_gemm_skinny(x, qweight, scales, zeros, y, M, N, K, group, ws, d->status_word,
                                            d->sms, take_packed_written(d), (cudaStream_t)stream));
    }
    const bool tensor_path = path == AWQ_PATH_GEMM || path == AWQ_PATH_GEMM_1SM;
    const cudaStream_t st = (cudaStream_t)stream;
    if (path == AWQ_PATH_GEMV && gemv_uses_band_kernel(M, N, d->sms)) {
        const GemvMatrix one = {qweight, scales, zeros, y, N};
        return note_cuda(launch_gemv_band(x, &one, 1, M, K, group, d->status_word, d->sms,
                                          take_packed_written(d), st));
    }
    (void)take_packed_written(d);               // every other kernel is plainly stream-ordered
    if (path == AWQ_PATH_GEMV || path == AWQ_PATH_GEMV_SPLITK) {
        void* ws = nullptr;
        {
            std::lock_guard<std::mutex> lock(g_mutex);
            if (d->workspace_bytes < gemv_workspace_bytes(M)) return AWQ_ERR_NO_WORKSPACE;
            ws = d->workspace;
        }
        int surplus = 0;
        {
            std::lock_guard<std::mutex> lock(g_mutex);
            surplus = d->tx_surplus_once;
            d->tx_surplus_once = 0;
        }
        return note_cuda(launch_gemv_splitk(x, qweight, scales, zeros, y, M, N, K, group, ws, d->status_word,
                                            d->sms, st, surplus));
    }
    void* ws = nullptr;
    size_t ws_bytes = 0;
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        ws = d->workspace;
        ws_bytes = d->workspace_bytes;
    }
    return note_cuda(launch_gemm(x, qweight, scales, zeros, y, M, N, K, group, path != AWQ_PATH_GEMM_1SM,
                                 ws, ws_bytes, d->status_word, st));
}

int awq_linear_gemv_static(const void* x, const void* qweight, const void* scales, const void* zeros,
                            void* y, int M, int N, int K, int group, void* stream) {
    if (int rc = check_shape(N, K, group)) return rc;
    group = stored_group(group);
    if (M < 1) return AWQ_ERR_BAD_SHAPE;
    if (M > gemv_static_max_m() || K > 65536) return AWQ_ERR_STATIC_LIMIT;
    if (!x || !qweight || !scales || !zeros || !y) return AWQ_ERR_NULL_POINTER;
    if (!aligned16(x) || !aligned16(qweight) || !aligned16(scales) || !aligned16(zeros) || !aligned16(y))
        return AWQ_ERR_MISALIGNED;
    DeviceState* d;
    if (int rc = device_state(&d)) return rc;
    void* scratch = nullptr;
    if (int rc = note_cuda(gemv_static_scratch(&scratch))) return rc;
    const cudaStream_t st = (cudaStream_t)stream;
    // the arrival counters must start at zero whatever an earlier call left behind
    if (int rc = note_cuda(cudaMemsetAsync(scratch, 0, kCounterBytes, st))) return rc;
    return note_cuda(launch_gemv_splitk(x, qweight, scales, zeros, y, M, N, K, group, scratch,
                                        d->status_word, d->sms, st));
}

int awq_set_wait_limit_us(unsigned int microseconds) {
    DeviceState* d;
    if (int rc = device_state(&d)) return rc;
    if (int rc = note_cuda(cudaDeviceSynchronize())) return rc;
    return note_cuda(cudaMemcpy(d->status_word + 1, &microseconds, sizeof(microseconds), cudaMemcpyHostToDevice));
}

int awq_test_stall_next_gemv(void) {
    DeviceState* d;
    if (int rc = device_state(&d)) return rc;
    std::lock_guard<std::mutex> lock(g_mutex);
    d->tx_surplus_once = 16;
    return AWQ_OK;
}

int awq_static_scratch_fill(int value, void* stream) {
    DeviceState* d;
    if (int rc = device_state(&d)) return rc;
    void* scratch = nullptr;
    if (int rc = note_cuda(gemv_static_scratch(&scratch))) return rc;
    return note_cuda(cudaMemsetAsync(scratch, value & 0xFF, kCounterBytes, (cudaStream_t)stream));
}

int awq_linear_multi(const void* x, const AwqLinearProblem* problems, int count,
                     int M, int K, int group, void* stream) {
    if (!problems || !x) return AWQ_ERR_NULL_POINTER;
    if (count < 1 || count > kMaxMulti) return AWQ_ERR_BAD_ARGUMENT;
    int total_n = 0;
    for (int i = 0; i < count; ++i) {
        const AwqLinearProblem& p = problems[i];
        if (int rc = check_shape(p.N, K, group)) return rc;
        if (!p.qweight || !p.scales || !p.zeros || !p.y) return AWQ_ERR_NULL_POINTER;
        if (!aligned16(p.qweight) || !aligned16(p.scales) || !aligned16(p.zeros) || !aligned16(p.y))
            return AWQ_ERR_MISALIGNED;
        total_n += p.N;
    }
    group = stored_group(group);
    if (M < 1) return AWQ_ERR_BAD_SHAPE;
    if (!aligned16(x)) return AWQ_ERR_MISALIGNED;
    DeviceState* d;
    if (int rc = device_state(&d)) return rc;
    if (M <= 8 && K <= 65536 && gemv_uses_band_kernel(M, total_n, d->sms)) {
        GemvMatrix mats[kMaxMulti];
        for (int i = 0; i < count; ++i)
            mats[i] = GemvMatrix{problems[i].qweight, problems[i].scales, problems[i].zeros, problems[i].y,
                                 problems[i].N};
        return note_cuda(launch_gemv_band(x, mats, count, M, K, group, d->status_word, d->sms,
                                          take_packed_written(d), (cudaStream_t)stream));
    }
    // otherwise one call per matrix, as awq_linear would run it
    for (int i = 0; i < count; ++i) {
        const AwqLinearProblem& p = problems[i];
        if (int rc = awq_linear(x, p.qweight, p.scales, p.zeros, p.y, M, p.N, K, group, stream)) return rc;
    }
    return AWQ_OK;
}

int awq_linear(const void* x, const void* qweight, const void* scales, const void* zeros,
               void* y, int M, int N, int K, int group, void* stream) {
    return awq_linear_path(x, qweight, scales, zeros, y, M, N, K, group, AWQ_PATH_AUTO, stream);
}

// ---- the layer with diag(s)^-1 folded in (Sec. 3.2: the inverse scale goes into the operator in front)
static bool scaled_call_folds(int M, int total_n, int K, int group, int sms) {
    return M <= 8 && K <= 65536 && gemv_uses_band_kernel(M, total_n, sms) && gemv_band_folds_scale(M, K, group);
}

int awq_linear_scaled_needs_scratch(int M, int N, int K, int group) {
    if (check_shape(N, K, group) != AWQ_OK || M < 1) return 1;
    group = stored_group(group);
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
        (void)cudaGetLastError();
        return 1;
    }
    return scaled_call_folds(M, N, K, group, sms) ? 0 : 1;
}

int awq_linear_multi_scaled(const void* x, const float* inv_s, void* x_scratch, const AwqLinearProblem* problems,
                            int count, int M, int K, int group, void* stream) {
    if (!problems || !x || !inv_s) return AWQ_ERR_NULL_POINTER;
    if (count < 1 || count > kMaxMulti) return AWQ_ERR_BAD_ARGUMENT;
    int total_n = 0;
    for (int i = 0; i < count; ++i) {
        const AwqLinearProblem& p = problems[i];
        if (int rc = check_shape(p.N, K, group)) return rc;
        if (!p.qweight || !p.scales || !p.zeros || !p.y) return AWQ_ERR_NULL_POINTER;
        if (!aligned16(p.qweight) || !aligned16(p.scales) || !aligned16(p.zeros) || !aligned16(p.y))
            return AWQ_ERR_MISALIGNED;
        total_n += p.N;
    }
    group = stored_group(group);
    if (M < 1 || (long long)M * K > (1LL << 40)) return AWQ_ERR_BAD_SHAPE;
    if (!aligned16(x) || !aligned16(inv_s) || !aligned16(x_scratch)) return AWQ_ERR_MISALIGNED;
    DeviceState* d;
    if (int rc = device_state(&d)) return rc;
    if (scaled_call_folds(M, total_n, K, group, d->sms)) {
        GemvMatrix mats[kMaxMulti];
        for (int i = 0; i < count; ++i)
            mats[i] = GemvMatrix{problems[i].qweight, problems[i].scales, problems[i].zeros, problems[i].y,
                                 problems[i].N};
        return note_cuda(launch_gemv_band(x, mats, count, M, K, group, d->status_word, d->sms,
                                          take_packed_written(d), (cudaStream_t)stream, inv_s));
    }
    // no kernel to fold it into: scale first (one more launch), then the plain calls
    if (!x_scratch) return AWQ_ERR_NULL_POINTER;
    if (int rc = note_cuda(launch_multiply_by_inverse(x, inv_s, x_scratch, M, K, (cudaStream_t)stream))) return rc;
    return awq_linear_multi(x_scratch, problems, count, M, K, group, stream);
}

int awq_linear_scaled(const void* x, const float* inv_s, void* x_scratch, const void* qweight, const void* scales,
                      const void* zeros, void* y, int M, int N, int K, int group, void* stream) {
    const AwqLinearProblem one = {qweight, scales, zeros, y, N};
    return awq_linear_multi_scaled(x, inv_s, x_scratch, &one, 1, M, K, group, stream);
}

// ---- 3-bit storage
size_t awq_qweight_bytes_int3(int N, int K) {
    return check_shape(N, K, 128) == AWQ_OK ? (size_t)N * K / 8 * 3 : 0;
}

int awq_pack_int3(const void* qweight, void* qweight3, int N, int K, void* stream) {
    if (int rc = check_shape(N, K, 128)) return rc;
    if (!qweight || !qweight3) return AWQ_ERR_NULL_POINTER;
    if (!aligned16(qweight) || !aligned16(qweight3)) return AWQ_ERR_MISALIGNED;
    DeviceState* d;
    if (int rc = device_state(&d)) return rc;
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        d->packed_written = true;
    }
    return note_cuda(launch_pack_int3(qweight, qweight3, N, K, (cudaStream_t)stream));
}

int awq_unpack_int3(const void* qweight3, void* qweight, int N, int K, void* stream) {
    if (int rc = check_shape(N, K, 128)) return rc;
    if (!qweight || !qweight3) return AWQ_ERR_NULL_POINTER;
    if (!aligned16(qweight) || !aligned16(qweight3)) return AWQ_ERR_MISALIGNED;
    DeviceState* d;
    if (int rc = device_state(&d)) return rc;
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        d->packed_written = true;
    }
    return note_cuda(launch_unpack_int3(qweight3, qweight, N, K, (cudaStream_t)stream));
}

int awq_linear_int3(const void* x, const void* qweight3, const void* scales, const void* zeros, void* y,
                    void* qweight_scratch, int M, int N, int K, int group, void* stream) {
    if (int rc = check_shape(N, K, group)) return rc;
    group = stored_group(group);
    if (M < 1 || (long long)M * K > (1LL << 40) || (long long)M * N > (1LL << 40)) return AWQ_ERR_BAD_SHAPE;
    if (!x || !qweight3 || !scales || !zeros || !y) return AWQ_ERR_NULL_POINTER;
    if (!aligned16(x) || !aligned16(qweight3) || !aligned16(scales) || !aligned16(zeros) || !aligned16(y) ||
        !aligned16(qweight_scratch))
        return AWQ_ERR_MISALIGNED;
    DeviceState* d;
    if (int rc = device_state(&d)) return rc;
    if (M <= 8 && K <= 65536 && gemv_uses_band_kernel(M, N, d->sms)) {
        const GemvMatrix one = {qweight3, scales, zeros, y, N};
        return note_cuda(launch_gemv_band(x, &one, 1, M, K, group, d->status_word, d->sms,
                                          take_packed_written(d), (cudaStream_t)stream, nullptr, 3));
    }
    // every other kernel reads the 4-bit layout: expand first (one more launch), then the plain call
    if (!qweight_scratch) return AWQ_ERR_NULL_POINTER;
    if (int rc = awq_unpack_int3(qweight3, qweight_scratch, N, K, stream)) return rc;
    return awq_linear(x, qweight_scratch, scales, zeros, y, M, N, K, group, stream);
}

int awq_inverse_channel_scale(const float* act_mean_abs, float alpha, float* inv_s, int K, void* stream) {
    if (int rc = awq_channel_scale(act_mean_abs, alpha, inv_s, K, stream)) return rc;
    return note_cuda(launch_inverse_scale(inv_s, inv_s, K, (cudaStream_t)stream));
}

size_t awq_search_scratch_bytes(int M, int N, int K, int group) {
    if (check_shape(N, K, group) != AWQ_OK || M < 1 || group > 128) return 0;
    return search_scratch_bytes(M, N, K, group);
}

int awq_search_alpha(const void* W, const float* act_mean_abs, const void* X, int M, int N, int K, int group,
                     const float* alphas, int n_alphas, float* losses, int* best_index,
                     void* scratch, size_t scratch_bytes, void* stream) {
    if (int rc = check_shape(N, K, group)) return rc;
    if (group > 128) return AWQ_ERR_BAD_GROUP;
    if (M < 1) return AWQ_ERR_BAD_SHAPE;
    if (!W || !act_mean_abs || !X || !alphas || !losses || !best_index || !scratch) return AWQ_ERR_NULL_POINTER;
    if (n_alphas < 1 || n_alphas > kMaxSearchAlphas) return AWQ_ERR_BAD_ARGUMENT;
    for (int i = 0; i < n_alphas; ++i)
        if (!(alphas[i] >= 0.0f && alphas[i] <= 1.0f)) return AWQ_ERR_BAD_ARGUMENT;
    if (scratch_bytes < search_scratch_bytes(M, N, K, group)) return AWQ_ERR_BAD_ARGUMENT;
    if (!aligned16(W) || !aligned16(X) || (reinterpret_cast<uintptr_t>(scratch) & 255u) != 0) return AWQ_ERR_MISALIGNED;
    const cudaStream_t st = (cudaStream_t)stream;
    float *s, *yref, *dev_losses;
    double* partials;
    void *xs, *qw, *sc, *zp, *yq;
    search_carve(scratch, M, N, K, group, &s, &xs, &qw, &sc, &zp, &yq, &yref, &partials, &dev_losses);
    if (int rc = note_cuda(launch_reference_product(W, X, yref, M, N, K, st))) return rc;
    for (int i = 0; i < n_alphas; ++i) {
        if (int rc = awq_channel_scale(act_mean_abs, alphas[i], s, K, stream)) return rc;
        if (int rc = awq_quantize_pack(W, act_mean_abs, alphas[i], group, qw, sc, zp, N, K, stream)) return rc;
        if (int rc = note_cuda(launch_divide_by_scale(X, s, xs, M, K, st))) return rc;
        if (int rc = awq_linear(xs, qw, sc, zp, yq, M, N, K, group, stream)) return rc;
        if (int rc = note_cuda(launch_mean_squared_difference(yq, yref, (size_t)M * N, partials, dev_losses + i, st)))
            return rc;
    }
    if (int rc = note_cuda(cudaMemcpyAsync(losses, dev_losses, (size_t)n_alphas * sizeof(float),
                                           cudaMemcpyDeviceToHost, st)))
        return rc;
    if (int rc = note_cuda(cudaStreamSynchronize(st))) return rc;
    int best = 0;
    bool have = false;
    for (int i = 0; i < n_alphas; ++i) {
        if (!std::isfinite(losses[i])) continue;
        if (!have || losses[i] < losses[best]) { best = i; have = true; }
    }
    *best_index = best;
    return AWQ_OK;
}

int awq_unpack_canonical(const void* qweight, const void* scales, const void* zeros,
                         int N, int K, int group,
                         uint8_t* codes, uint16_t* scales_nk, uint8_t* zeros_nk, void* stream) {
    if (int rc = check_shape(N, K, group)) return rc;
    if (!qweight || !scales || !zeros || !codes || !scales_nk || !zeros_nk) return AWQ_ERR_NULL_POINTER;
    DeviceState* d;
    if (int rc = device_state(&d)) return rc;
    return note_cuda(launch_unpack(reinterpret_cast<const uint32_t*>(qweight),
                                   reinterpret_cast<const __half*>(scales),
                                   reinterpret_cast<const uint8_t*>(zeros), N, K, group,
                                   codes, scales_nk, zeros_nk, (cudaStream_t)stream));
}

int awq_poll_status(void) {
    DeviceState* d;
    if (int rc = device_state(&d)) return rc;
    if (int rc = note_cuda(cudaDeviceSynchronize())) return rc;
    unsigned int v = 0;
    if (int rc = note_cuda(cudaMemcpy(&v, d->status_word, sizeof(v), cudaMemcpyDeviceToHost))) return rc;
    if (v != 0) {
        if (int rc = note_cuda(cudaMemset(d->status_word, 0, sizeof(v)))) return rc;
        // a kernel that gave up may have left arrival counters half-way: start them afresh
        void* ws = nullptr;
        size_t ws_bytes = 0;
        {
            std::lock_guard<std::mutex> lock(g_mutex);
            ws = d->workspace;
            ws_bytes = d->workspace_bytes;
        }
        if (ws && ws_bytes >= kCounterBytes)
            if (int rc = note_cuda(cudaMemset(ws, 0, kCounterBytes))) return rc;
        return AWQ_ERR_TIMEOUT;
    }
    return AWQ_OK;
}

const char* awq_status_string(int status) {
    switch (status) {
        case AWQ_OK: return "ok";
        case AWQ_ERR_NULL_POINTER: return "null pointer";
        case AWQ_ERR_BAD_SHAPE: return "bad shape (N, K multiples of 128; K % group == 0; M >= 1)";
        case AWQ_ERR_BAD_GROUP: return "group must be 64 or 128";
        case AWQ_ERR_BAD_ALPHA: return "alpha must lie in [0, 1]";
        case AWQ_ERR_MISALIGNED: return "pointer not 16-byte aligned";
        case AWQ_ERR_NO_WORKSPACE: return "registered workspace too small (see awq_workspace_bytes)";
        case AWQ_ERR_WRONG_DEVICE: return "current device is not compute capability 10.x";
        case AWQ_ERR_CUDA: return "CUDA call failed (see awq_last_cuda_error)";
        case AWQ_ERR_TIMEOUT: return "a device-side wait ran out";
        case AWQ_ERR_BAD_ARGUMENT: return "bad argument";
        case AWQ_ERR_STATIC_LIMIT: return "problem exceeds the built-in scratch of awq_linear_gemv_static (M <= 8, K <= 65536)";
        default: return "unknown status";
    }
}

const char* awq_last_cuda_error(void) { return t_cuda_error; }
int awq_layout_version(void) { return 3; }
unsigned long long awq_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
