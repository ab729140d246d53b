// Ceiling of the row gathers the DS-FACTO kernels are made of, measured on the device at hand.
//
// Both hot kernels read, per stored entry, one factor row (a_i in the stratum SGD, v_j in the
// recompute pass) of 4K bytes from a table that mostly sits in L2.  This program times nothing but
// that access: a lane group of (row bytes / 16) lanes loads uniformly random rows of a table as
// float4s, U rows requested before the first is used, and adds them up.  The rate it reaches is
// what a kernel with this access pattern can at best approach; it is printed as gathered GB/s and
// as rows per second for tables of the sizes the workloads have (one row block of A, all of V, a
// table far larger than L2).  Stand-alone: it shares nothing with the library.
#include <cuda_runtime.h>

#include <cstdint>
#include <cstdio>
#include <cstdlib>
#include <vector>

#define CK(call)                                                                                  \
    do {                                                                                          \
        cudaError_t e_ = (call);                                                                  \
        if (e_ != cudaSuccess) {                                                                  \
            std::fprintf(stderr, "%s: %s (line %d)\n", #call, cudaGetErrorString(e_), __LINE__);  \
            return 1;                                                                             \
        }                                                                                         \
    } while (0)

template <int LG, int U>
__global__ void __launch_bounds__(256) gather_kernel(const float4 *table, const uint32_t *row_ids, int64_t count,
                                                     float *sink) {
    constexpr int G = 256 / LG;
    const int g = threadIdx.x / LG, l = threadIdx.x % LG;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    const int64_t stride = (int64_t)gridDim.x * G * U;
    for (int64_t t = ((int64_t)blockIdx.x * G + g) * U; t + U <= count; t += stride) {
        uint32_t r[U];
        float4 v[U];
#pragma unroll
        for (int u = 0; u < U; ++u) r[u] = __ldg(row_ids + t + u);
#pragma unroll
        for (int u = 0; u < U; ++u) v[u] = __ldcg(table + (size_t)r[u] * LG + l);
#pragma unroll
        for (int u = 0; u < U; ++u) { acc.x += v[u].x; acc.y += v[u].y; acc.z += v[u].z; acc.w += v[u].w; }
    }
    if (acc.x + acc.y + acc.z + acc.w == 12345.678f) sink[0] = acc.x;   // never true for a zero table; keeps the loads
}

template <int LG, int U>
int measure(const char *what, int64_t rows, int64_t count, int sms) {
    float4 *table = nullptr;
    uint32_t *ids = nullptr;
    float *sink = nullptr;
    CK(cudaMalloc(&table, (size_t)rows * LG * sizeof(float4)));
    CK(cudaMemset(table, 0, (size_t)rows * LG * sizeof(float4)));
    CK(cudaMalloc(&ids, (size_t)count * sizeof(uint32_t)));
    CK(cudaMalloc(&sink, sizeof(float)));
    std::vector<uint32_t> h((size_t)count);
    uint64_t s = 88172645463325252ull;   // xorshift64: uniformly random rows
    for (int64_t i = 0; i < count; ++i) {
        s ^= s << 13; s ^= s >> 7; s ^= s << 17;
        h[(size_t)i] = (uint32_t)(s % (uint64_t)rows);
    }
    CK(cudaMemcpy(ids, h.data(), (size_t)count * sizeof(uint32_t), cudaMemcpyHostToDevice));
    cudaEvent_t e0, e1;
    CK(cudaEventCreate(&e0));
    CK(cudaEventCreate(&e1));
    const int grid = sms * 8;
    for (int w = 0; w < 3; ++w) gather_kernel<LG, U><<<grid, 256>>>(table, ids, count, sink);
    const int reps = 5;
    CK(cudaEventRecord(e0));
    for (int w = 0; w < reps; ++w) gather_kernel<LG, U><<<grid, 256>>>(table, ids, count, sink);
    CK(cudaEventRecord(e1));
    CK(cudaEventSynchronize(e1));
    CK(cudaGetLastError());
    float ms = 0.f;
    CK(cudaEventElapsedTime(&ms, e0, e1));
    ms /= reps;
    std::printf("%-28s row %4d B  table %8.1f MB  %d rows in flight per lane group: %7.3f ms  %8.1f GB/s  %7.2f G rows/s\n",
                what, LG * 16, (double)rows * LG * 16 / 1e6, U, ms, (double)count * LG * 16 / ms / 1e6, (double)count / ms / 1e6);
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    cudaFree(table);
    cudaFree(ids);
    cudaFree(sink);
    return 0;
}

int main() {
    int sms = 0;
    CK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, 0));
    const int64_t n64 = 100ll << 20;    // gathers of 64-byte rows (K = 16)
    const int64_t n512 = n64 / 8;       // gathers of 512-byte rows (K = 128)
    int rc = 0;
    rc |= measure<4, 4>("K=16, row block of A", 87891, n64, sms);
    rc |= measure<4, 8>("K=16, row block of A", 87891, n64, sms);
    rc |= measure<4, 8>("K=16, all of V", 1 << 20, n64, sms);
    rc |= measure<4, 8>("K=16, beyond L2", 11250000, n64, sms);
    rc |= measure<32, 2>("K=128, row block of A", 15625, n512, sms);
    rc |= measure<32, 4>("K=128, row block of A", 15625, n512, sms);
    rc |= measure<32, 4>("K=128, 100 k rows of V", 100000, n512, sms);
    rc |= measure<32, 4>("K=128, all of V", 1 << 20, n512, sms);
    return rc;
}
