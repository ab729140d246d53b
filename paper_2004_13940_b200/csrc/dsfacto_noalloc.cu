// dsfacto_score_loss_noalloc: scores, loss sum and multiplier sum of a batch of rows, for callers that
// must not allocate.
//
// Who needs this: code that runs where device allocation is forbidden or unsafe - inside a region
// that another framework has closed to cudaMalloc (a memory pool that owns the whole device, a
// serving loop with a fixed memory budget), or from a thread that must never block on the
// driver's allocation lock.  Such a caller already owns device buffers with the rows, the
// parameters and room for the results; the only thing the ordinary path would still allocate is the
// per-CTA partial sums of the loss reduction.  Here those live in a fixed array that is part of
// the library image.
#include "dsfacto.h"
#include "dsfacto_common.cuh"

#include <cmath>
#include <cstdint>

namespace {

using namespace dsf;

constexpr int kRowsPerCta = 1024;    // rows one CTA scores
constexpr int kMaxCtas = 65536;      // CTAs whose partial sums fit the scratch array
constexpr int kMaxDevices = 64;

// Scratch of the reduction: {sum of losses, sum of multipliers} per CTA, 1 MiB.  Every GPU that
// loads the library holds one copy until the process exits.  Each call overwrites the slots it
// uses before it reads them, so nothing has to start at zero; the contents of the last call stay.
static __device__ __align__(256) double g_noalloc_partials[2 * kMaxCtas];

// device address of g_noalloc_partials per device (the symbol itself is only a host-side stand-in)
double *g_partials_addr[kMaxDevices] = {nullptr};

// Same arithmetic as the recompute pass of the epoch (eq. (fm_model2), the multiplier G, the loss),
// one lane group per row, without storing the auxiliaries.
template <int LG, int NV>
__global__ void __launch_bounds__(kThreads) score_loss_kernel(int64_t m, const int64_t *indptr, const int32_t *idx,
                                                              const float *val, const float *y, const float *w,
                                                              const float *V, float w0, int loss, float *scores,
                                                              double *partials) {
    constexpr int G = kThreads / LG;
    constexpr int KP4 = LG * NV;
    const int g = threadIdx.x / LG;
    const int l = threadIdx.x % LG;
    const uint32_t gm = group_mask<LG>();
    const float4 *V4 = reinterpret_cast<const float4 *>(V);
    double loss_sum = 0.0, g_sum = 0.0;
    const int64_t first = (int64_t)blockIdx.x * kRowsPerCta;
    const int64_t stop = first + kRowsPerCta < m ? first + kRowsPerCta : m;

    for (int64_t row = first + g; row < stop; row += G) {
        const int64_t beg = indptr[row], end = indptr[row + 1];
        float4 acc[NV];
#pragma unroll
        for (int v = 0; v < NV; ++v) acc[v] = make_float4(0.f, 0.f, 0.f, 0.f);
        float q = 0.f, lin = 0.f;
        for (int64_t t0 = beg; t0 < end; t0 += LG) {
            const int64_t mine = t0 + l;
            int32_t jm = 0;
            float xm = 0.f;
            if (mine < end) { jm = __ldg(idx + mine); xm = __ldg(val + mine); lin = fmaf(__ldg(w + jm), xm, lin); }
            const int cnt = (int)((end - t0) < (int64_t)LG ? (end - t0) : (int64_t)LG);
            for (int u = 0; u < cnt; ++u) {
                const int32_t j = __shfl_sync(gm, jm, u, LG);
                const float x = __shfl_sync(gm, xm, u, LG);
#pragma unroll
                for (int v = 0; v < NV; ++v) {
                    const float4 vv = __ldg(V4 + (size_t)j * KP4 + v * LG + l);
                    const float px = vv.x * x, py = vv.y * x, pz = vv.z * x, pw = vv.w * x;
                    acc[v].x += px; acc[v].y += py; acc[v].z += pz; acc[v].w += pw;
                    q = fmaf(px, px, q); q = fmaf(py, py, q); q = fmaf(pz, pz, q); q = fmaf(pw, pw, q);
                }
            }
        }
        float sq = 0.f;
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            sq = fmaf(acc[v].x, acc[v].x, sq); sq = fmaf(acc[v].y, acc[v].y, sq);
            sq = fmaf(acc[v].z, acc[v].z, sq); sq = fmaf(acc[v].w, acc[v].w, sq);
        }
        float pair = sq - q;
#pragma unroll
        for (int o = LG / 2; o > 0; o >>= 1) {
            pair += __shfl_xor_sync(gm, pair, o, LG);
            lin += __shfl_xor_sync(gm, lin, o, LG);
        }
        if (l == 0) {
            const float f = w0 + lin + 0.5f * pair;
            const float yy = y[row];
            float li, gi;
            if (loss == DSFACTO_SQUARED) {
                gi = f - yy;
                li = 0.5f * gi * gi;
            } else {
                const float mg = yy * f;
                li = fmaxf(-mg, 0.f) + log1pf(expf(-fabsf(mg)));
                gi = -yy / (1.f + expf(mg));
            }
            scores[row] = f;
            loss_sum += (double)li;
            g_sum += (double)gi;
        }
    }
    block_sum2(loss_sum, g_sum);
    if (threadIdx.x == 0) {
        partials[2 * blockIdx.x] = loss_sum;
        partials[2 * blockIdx.x + 1] = g_sum;
    }
}

// sums[c] = sum over CTAs (fixed order) of partials[2*b + c]
__global__ void __launch_bounds__(kThreads) sum_partials_kernel(const double *partials, int nblocks, double *sums) {
    double s0 = 0.0, s1 = 0.0;
    for (int b = threadIdx.x; b < nblocks; b += kThreads) {
        s0 += partials[2 * b];
        s1 += partials[2 * b + 1];
    }
    block_sum2(s0, s1);
    if (threadIdx.x == 0) { sums[0] = s0; sums[1] = s1; }
}

template <int LG, int NV>
void launch_score_loss(int grid, cudaStream_t st, int64_t m, const int64_t *indptr, const int32_t *idx,
                       const float *val, const float *y, const float *w, const float *V, float w0, int loss,
                       float *scores, double *partials) {
    score_loss_kernel<LG, NV><<<grid, kThreads, 0, st>>>(m, indptr, idx, val, y, w, V, w0, loss, scores, partials);
}

}  // namespace

extern "C" int dsfacto_score_loss_noalloc(int64_t m, int32_t d, int32_t K, int32_t loss, const int64_t *indptr_dev,
                                          const int32_t *indices_dev, const float *values_dev, const float *y_dev,
                                          float w0, const float *w_dev, const float *V_dev, float *scores_dev,
                                          double *sums_dev, void *cuda_stream) {
    if (m < 1 || d < 1 || !indptr_dev || !indices_dev || !values_dev || !y_dev || !w_dev || !V_dev || !scores_dev || !sums_dev)
        return DSFACTO_ERR_INVALID_ARG;
    // rows of V are read 16 bytes at a time: a pointer that is not 16-byte aligned would fault on the device,
    // so it is refused here instead
    if ((reinterpret_cast<uintptr_t>(V_dev) & 15u) != 0) return DSFACTO_ERR_INVALID_ARG;
    if (loss != DSFACTO_SQUARED && loss != DSFACTO_LOGISTIC) return DSFACTO_ERR_INVALID_ARG;
    if (!std::isfinite(w0)) return DSFACTO_ERR_INVALID_ARG;
    // rows of V are read as float4 lane groups: K must be 4, 8, 16, 32, 64, 128 or 256
    if (K < 4 || K > 256 || (K & (K - 1)) != 0) return DSFACTO_ERR_INVALID_ARG;
    const int64_t ctas = (m + kRowsPerCta - 1) / kRowsPerCta;
    if (ctas > kMaxCtas) return DSFACTO_ERR_INVALID_ARG;  // more than 67,108,864 rows: scratch too small

    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return DSFACTO_ERR_CUDA;
    if (!g_partials_addr[dev]) {  // first call on this device: resolve the array's device address
        double *p = nullptr;
        if (cudaGetSymbolAddress((void **)&p, g_noalloc_partials) != cudaSuccess || !p) return DSFACTO_ERR_CUDA;
        g_partials_addr[dev] = p;
    }
    double *partials = g_partials_addr[dev];
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const int q4 = K / 4;
    const int LG = q4 < 32 ? q4 : 32, NV = q4 <= 32 ? 1 : 2;
    switch (LG * 10 + NV) {
    case 11: launch_score_loss<1, 1>((int)ctas, st, m, indptr_dev, indices_dev, values_dev, y_dev, w_dev, V_dev, w0, loss, scores_dev, partials); break;
    case 21: launch_score_loss<2, 1>((int)ctas, st, m, indptr_dev, indices_dev, values_dev, y_dev, w_dev, V_dev, w0, loss, scores_dev, partials); break;
    case 41: launch_score_loss<4, 1>((int)ctas, st, m, indptr_dev, indices_dev, values_dev, y_dev, w_dev, V_dev, w0, loss, scores_dev, partials); break;
    case 81: launch_score_loss<8, 1>((int)ctas, st, m, indptr_dev, indices_dev, values_dev, y_dev, w_dev, V_dev, w0, loss, scores_dev, partials); break;
    case 161: launch_score_loss<16, 1>((int)ctas, st, m, indptr_dev, indices_dev, values_dev, y_dev, w_dev, V_dev, w0, loss, scores_dev, partials); break;
    case 321: launch_score_loss<32, 1>((int)ctas, st, m, indptr_dev, indices_dev, values_dev, y_dev, w_dev, V_dev, w0, loss, scores_dev, partials); break;
    case 322: launch_score_loss<32, 2>((int)ctas, st, m, indptr_dev, indices_dev, values_dev, y_dev, w_dev, V_dev, w0, loss, scores_dev, partials); break;
    default: return DSFACTO_ERR_INVALID_ARG;
    }
    sum_partials_kernel<<<1, kThreads, 0, st>>>(partials, (int)ctas, sums_dev);
    if (cudaGetLastError() != cudaSuccess) return DSFACTO_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return DSFACTO_ERR_CUDA;
    return DSFACTO_OK;
}
