// A caller of the library that knows nothing of Python or PyTorch: cudaMalloc'd buffers, the C
// entry points of include/awq_b200.h, and a check of the layer's output against a plain
// double-precision product formed from the library's own canonical dump of the packed arrays
// (awq_unpack_canonical); it also packs arrays on the host from the header's layout text and
// has the library unpack them.  Built and run by tests/test_c_abi_program.py; prints one line and
// returns 0 when every output is within the library's stated tolerance.
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdint>
#include <cstdio>
#include <cstdlib>
#include <vector>

#include "awq_b200.h"

#define CHECK_CUDA(call)                                                                   \
    do {                                                                                   \
        cudaError_t e_ = (call);                                                           \
        if (e_ != cudaSuccess) { std::printf("cuda error %s at %d\n", cudaGetErrorString(e_), __LINE__); return 2; } \
    } while (0)
#define CHECK_AWQ(call)                                                                    \
    do {                                                                                   \
        int rc_ = (call);                                                                  \
        if (rc_ != AWQ_OK) { std::printf("%s -> %d (%s)\n", #call, rc_, awq_status_string(rc_)); return 3; } \
    } while (0)

static uint32_t lcg(uint32_t& s) { s = s * 1664525u + 1013904223u; return s >> 8; }
static float uniform(uint32_t& s) { return (float)lcg(s) / 16777216.0f - 0.5f; }      // [-0.5, 0.5)

static int run(int M, int N, int K, int group) {
    uint32_t seed = 12345u + (uint32_t)(M * 7 + N + K + group);
    std::vector<__half> W((size_t)N * K), x((size_t)M * K);
    std::vector<float> a(K);
    for (auto& w : W) w = __float2half(0.08f * uniform(seed));
    for (auto& v : x) v = __float2half(2.0f * uniform(seed));
    for (auto& v : a) v = 0.5f + uniform(seed) * 0.5f + ((lcg(seed) % 100u) == 0u ? 10.0f : 0.0f);

    void *dW, *dx, *dy, *dq, *ds, *dz, *dws;
    float* da;
    const size_t qb = awq_qweight_bytes(N, K), sb = awq_scales_bytes(N, K, group), zb = awq_zeros_bytes(N, K, group);
    if (!qb || !sb || !zb) { std::printf("shape refused\n"); return 4; }
    CHECK_CUDA(cudaMalloc(&dW, W.size() * 2));
    CHECK_CUDA(cudaMalloc(&dx, x.size() * 2));
    CHECK_CUDA(cudaMalloc(&dy, (size_t)M * N * 2));
    CHECK_CUDA(cudaMalloc(&da, (size_t)K * 4));
    CHECK_CUDA(cudaMalloc(&dq, qb));
    CHECK_CUDA(cudaMalloc(&ds, sb));
    CHECK_CUDA(cudaMalloc(&dz, zb));
    const size_t wsb = awq_workspace_bytes(M, N, K, group);
    CHECK_CUDA(cudaMalloc(&dws, wsb ? wsb : 16));
    if (wsb) CHECK_AWQ(awq_set_workspace(dws, wsb));
    CHECK_CUDA(cudaMemcpy(dW, W.data(), W.size() * 2, cudaMemcpyHostToDevice));
    CHECK_CUDA(cudaMemcpy(dx, x.data(), x.size() * 2, cudaMemcpyHostToDevice));
    CHECK_CUDA(cudaMemcpy(da, a.data(), (size_t)K * 4, cudaMemcpyHostToDevice));

    CHECK_AWQ(awq_quantize_pack(dW, da, 0.5f, group, dq, ds, dz, N, K, nullptr));
    CHECK_AWQ(awq_linear(dx, dq, ds, dz, dy, M, N, K, group, nullptr));
    CHECK_AWQ(awq_poll_status());

    // canonical dump of what was packed, then y_ref = x . ((q - z) * Delta)^T in double
    uint8_t *dcodes, *dzn;
    uint16_t* dsn;
    const int ng = K / group;
    CHECK_CUDA(cudaMalloc(&dcodes, (size_t)N * K));
    CHECK_CUDA(cudaMalloc(&dsn, (size_t)N * ng * 2));
    CHECK_CUDA(cudaMalloc(&dzn, (size_t)N * ng));
    CHECK_AWQ(awq_unpack_canonical(dq, ds, dz, N, K, group, dcodes, dsn, dzn, nullptr));
    std::vector<uint8_t> codes((size_t)N * K), zn((size_t)N * ng);
    std::vector<__half> sn((size_t)N * ng), y((size_t)M * N);
    CHECK_CUDA(cudaMemcpy(codes.data(), dcodes, codes.size(), cudaMemcpyDeviceToHost));
    CHECK_CUDA(cudaMemcpy(zn.data(), dzn, zn.size(), cudaMemcpyDeviceToHost));
    CHECK_CUDA(cudaMemcpy(sn.data(), dsn, sn.size() * 2, cudaMemcpyDeviceToHost));
    CHECK_CUDA(cudaMemcpy(y.data(), dy, y.size() * 2, cudaMemcpyDeviceToHost));

    double num = 0.0, den = 0.0, max_abs = 0.0, max_ref = 0.0;
    for (int m = 0; m < M; ++m)
        for (int n = 0; n < N; ++n) {
            double ref = 0.0;
            for (int k = 0; k < K; ++k) {
                const int g = k / group;
                const double wq = ((double)codes[(size_t)n * K + k] - (double)zn[(size_t)n * ng + g]) *
                                  (double)__half2float(sn[(size_t)n * ng + g]);
                ref += wq * (double)__half2float(x[(size_t)m * K + k]);
            }
            const double d = (double)__half2float(y[(size_t)m * N + n]) - ref;
            num += d * d;
            den += ref * ref;
            max_abs = std::fmax(max_abs, std::fabs(d));
            max_ref = std::fmax(max_ref, std::fabs(ref));
        }
    const double rel = std::sqrt(num / den), mx = max_abs / max_ref;
    std::printf("M=%d N=%d K=%d g=%d rel_l2=%.3e max_abs_over_max_ref=%.3e\n", M, N, K, group, rel, mx);
    CHECK_AWQ(awq_set_workspace(nullptr, 0));
    cudaFree(dW); cudaFree(dx); cudaFree(dy); cudaFree(da); cudaFree(dq); cudaFree(ds); cudaFree(dz); cudaFree(dws);
    cudaFree(dcodes); cudaFree(dsn); cudaFree(dzn);
    return (rel <= 1e-3 && mx <= 5e-3) ? 0 : 1;
}

// The packed layout as an external packer would produce it, written from the layout text of
// awq_b200.h alone: random codes, zero points and scales are placed by the header's formulas,
// and the library's own canonical dump of those arrays must give them back.
static int check_header_layout(int N, int K, int group) {
    uint32_t seed = 777u + (uint32_t)(N + K + group);
    const int ng = K / group;
    std::vector<uint8_t> codes((size_t)N * K), zn((size_t)N * ng);
    std::vector<uint16_t> sn((size_t)N * ng);
    for (auto& c : codes) c = (uint8_t)(lcg(seed) & 15u);
    for (auto& z : zn) z = (uint8_t)(lcg(seed) & 15u);
    for (auto& v : sn) v = (uint16_t)(0x1400u + (lcg(seed) & 0x0FFFu));       // positive normal fp16 bit patterns
    std::vector<uint8_t> q((size_t)N * K / 2, 0), zp((size_t)N * ng / 2, 0);
    std::vector<uint16_t> sp((size_t)N * ng);
    static const int byte_of_column[4] = {0, 2, 1, 3};
    for (int n = 0; n < N; ++n) {
        for (int k = 0; k < K; ++k) {
            const size_t byte = ((size_t)(n / 16) * (K / 64) + k / 64) * 512 + 16 * (4 * (n % 8) + (k % 16) / 4) +
                                4 * ((k % 64) / 16) + byte_of_column[k % 4];
            q[byte] |= (uint8_t)(codes[(size_t)n * K + k] << ((n % 16 < 8) ? 0 : 4));
        }
        for (int g = 0; g < ng; ++g) {
            // zeros: bytes [N/32][K/group][16]; bytes 0-7 even band, 8-15 odd band; byte n%8, low / high nibble
            const size_t zb = ((size_t)(n / 32) * ng + g) * 16 + ((n / 16) % 2) * 8 + n % 8;
            zp[zb] |= (uint8_t)(zn[(size_t)n * ng + g] << ((n % 16 < 8) ? 0 : 4));
            // scales: fp16 [N/16][K/group][16]
            sp[((size_t)(n / 16) * ng + g) * 16 + n % 16] = sn[(size_t)n * ng + g];
        }
    }
    void *dq, *ds, *dz;
    uint8_t *dcodes, *dzn;
    uint16_t* dsn;
    CHECK_CUDA(cudaMalloc(&dq, q.size()));
    CHECK_CUDA(cudaMalloc(&ds, sp.size() * 2));
    CHECK_CUDA(cudaMalloc(&dz, zp.size()));
    CHECK_CUDA(cudaMalloc(&dcodes, codes.size()));
    CHECK_CUDA(cudaMalloc(&dsn, sn.size() * 2));
    CHECK_CUDA(cudaMalloc(&dzn, zn.size()));
    CHECK_CUDA(cudaMemcpy(dq, q.data(), q.size(), cudaMemcpyHostToDevice));
    CHECK_CUDA(cudaMemcpy(ds, sp.data(), sp.size() * 2, cudaMemcpyHostToDevice));
    CHECK_CUDA(cudaMemcpy(dz, zp.data(), zp.size(), cudaMemcpyHostToDevice));
    CHECK_AWQ(awq_unpack_canonical(dq, ds, dz, N, K, group, dcodes, dsn, dzn, nullptr));
    std::vector<uint8_t> codes2(codes.size()), zn2(zn.size());
    std::vector<uint16_t> sn2(sn.size());
    CHECK_CUDA(cudaMemcpy(codes2.data(), dcodes, codes2.size(), cudaMemcpyDeviceToHost));
    CHECK_CUDA(cudaMemcpy(zn2.data(), dzn, zn2.size(), cudaMemcpyDeviceToHost));
    CHECK_CUDA(cudaMemcpy(sn2.data(), dsn, sn2.size() * 2, cudaMemcpyDeviceToHost));
    cudaFree(dq); cudaFree(ds); cudaFree(dz); cudaFree(dcodes); cudaFree(dsn); cudaFree(dzn);
    const bool ok = codes2 == codes && zn2 == zn && sn2 == sn;
    std::printf("header layout N=%d K=%d g=%d: %s\n", N, K, group, ok ? "round trip ok" : "MISMATCH");
    return ok ? 0 : 1;
}

int main() {
    if (awq_layout_version() != 3) { std::printf("unexpected layout version\n"); return 5; }
    int bad = 0;
    bad |= check_header_layout(256, 384, 64);
    bad |= check_header_layout(128, 256, 128);
    bad |= run(1, 2432, 1152, 128);      // band matrix-vector kernel
    bad |= run(3, 256, 640, 64);         // split-K matrix-vector kernel
    bad |= run(40, 384, 1024, 128);      // one-SM tensor-core kernel (split-K with the workspace)
    bad |= run(300, 512, 512, 64);       // SM-pair tensor-core kernel
    std::printf(bad ? "FAILED\n" : "OK\n");
    return bad;
}
