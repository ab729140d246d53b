// Shared device helpers of the DS-FACTO kernels (sm_100a).
//
// Factor-row layout used by every kernel: a row (v_j or a_i) occupies Kp = 4*LG*NV floats, 16-byte
// aligned, K <= Kp, padding kept at zero.  A "lane group" of LG consecutive lanes (LG a power of
// two <= 32) owns one row: lane l holds float4 number l, l+LG, ... (NV of them), so the group's
// loads of one row are coalesced.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace dsf {

constexpr int kThreads = 256;
constexpr uint32_t kNoCol = 0xFFFFFFFFu;

template <int LG>
__device__ __forceinline__ uint32_t group_mask() {
    if (LG == 32) return 0xFFFFFFFFu;
    const uint32_t lane = threadIdx.x & 31u;
    return ((1u << LG) - 1u) << (lane & ~uint32_t(LG - 1));
}

// acc += c * r on four floats with two packed fp32x2 multiply-adds (each half rounds exactly as a scalar fmaf).
// Used by the stratum SGD sweep (512-byte rows: 21.3 -> 19.4 ms per sweep of 400 M entries; 64-byte rows: no
// change); the recompute pass got slower with it (14.4 -> 15.3 ms) and keeps scalar multiply-adds.
__device__ __forceinline__ void fma4(float4 &acc, const float c, const float4 r) {
    const float2 cc = make_float2(c, c);
    const float2 lo = __ffma2_rn(make_float2(r.x, r.y), cc, make_float2(acc.x, acc.y));
    const float2 hi = __ffma2_rn(make_float2(r.z, r.w), cc, make_float2(acc.z, acc.w));
    acc = make_float4(lo.x, lo.y, hi.x, hi.y);
}

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

// deterministic CTA-wide sum of two doubles; result valid in thread 0
__device__ __forceinline__ void block_sum2(double &a, double &b) {
    __shared__ double sh[2][kThreads / 32];
    a = warp_sum(a);
    b = warp_sum(b);
    const int wid = threadIdx.x >> 5, ln = threadIdx.x & 31;
    if (ln == 0) { sh[0][wid] = a; sh[1][wid] = b; }
    __syncthreads();
    if (threadIdx.x == 0) {
        double x = 0.0, y = 0.0;
        for (int i = 0; i < kThreads / 32; ++i) { x += sh[0][i]; y += sh[1][i]; }
        a = x; b = y;
    }
}

}  // namespace dsf
