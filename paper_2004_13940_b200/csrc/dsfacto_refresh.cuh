// Recompute-pass kernels of the DS-FACTO epoch for sm_100a: auxiliaries, scores, multipliers, and the
// fp64 sums behind the objective.
#pragma once
#include "dsfacto_common.cuh"

namespace dsf {

// ------------------------------------------------------------------------------------------
// Recompute pass (eq. (compute_a_jk), eq. (fm_model2), multiplier G): one lane group per row.
//   a_ik = sum_j v_jk x_ij ; lin_i = sum_j w_j x_ij ; q_i = sum_j sum_k (v_jk x_ij)^2
//   f_i = w0 + lin_i + 1/2 (sum_k a_ik^2 - q_i)
// q_i is taken as sum_j x_ij^2 s_j with s_j = sum_k v_jk^2, which is the same sum regrouped: s_j is computed
// once per column after the parameters changed (model_view_kernel) and sits next to w_j, so the lane that
// owns an entry gets both with one 8-byte load and the K-wide part of an entry is K multiply-adds.
// MODE kScore: writes f only.  kTrain: writes A, G and per-CTA fp64 partial sums {sum l_i, sum G_i}.
// kEvaluate (held-out rows with labels; the quantities of the convergence figures of Section 5):
// writes nothing per row, per-CTA fp64 partial sums {sum l_i, sum t_i} with t_i = (f_i - y_i)^2 for
// the squared loss (RMSE) and t_i = [y_i f_i > 0] for the logistic loss (accuracy).
// kPartial (a handle that owns only a range of columns, Section 4.2's column blocks spread over
// workers): the sums run over the handle's own columns, so they are partial; writes a_ik, lin_i and
// q_i per row and stops there.  The partial sums of all shards are added outside and finish_kernel
// turns the totals into f_i, l_i and G_i.
// ------------------------------------------------------------------------------------------
enum { kScore = 0, kTrain = 1, kEvaluate = 2, kPartial = 3 };
struct RefreshArgs {
    int64_t n;
    const int64_t *indptr;
    const int32_t *idx;
    const float *val;
    const float *y;
    const float2 *pair;  // per column (w_j, s_j = sum_k v_jk^2)
    const float *V;
    float *A;
    float *G;
    float *f_out;
    float *lin_out, *q_out;  // kPartial: per-row partial sums
    double *partials;  // 2 per CTA
    float w0;
    int loss;
};

// Rows of 128 bytes and more keep 8 float4s per lane in flight and would take 88 to 100 registers:
// capped at 80 so that three CTAs stay resident (K = 128: 27.1 -> 22.3 ms per pass on 400 M entries;
// a cap of 64 registers spills too much: 24.5 ms).  Narrower rows fit 64 registers and four CTAs.
template <int LG, int NV, int MODE>
__global__ void __launch_bounds__(kThreads, (LG >= 8 ? 3 : 4)) refresh_kernel(const RefreshArgs a) {
    constexpr int G = kThreads / LG;
    constexpr int KP4 = LG * NV;
    const int g = threadIdx.x / LG;
    const int l = threadIdx.x % LG;
    const uint32_t gm = group_mask<LG>();
    const float4 *V4 = reinterpret_cast<const float4 *>(a.V);
    float4 *A4 = reinterpret_cast<float4 *>(a.A);
    constexpr bool TRAIN = MODE == kTrain;
    constexpr bool STORE_A = MODE == kTrain || MODE == kPartial;
    // the fp64 sums of a lane group live in shared memory: only its first lane touches them, once per row
    __shared__ double sums[2][G];
    if (l == 0) { sums[0][g] = 0.0; sums[1][g] = 0.0; }

    // The row pointers of the next row are requested while the current row is processed, and its
    // first batch of entries during the current row's last batch: a lane group never waits for the
    // pointer -> entry -> factor-row chain at a row start, except at its very first row.
    const int64_t row_first = (int64_t)blockIdx.x * G + g;
    const int row_step = (int)gridDim.x * G;
    int64_t nbeg = 0;      // the next row: its first entry and its length (a row holds at most d < 2^31 entries)
    int nlen = 0;
    int32_t jn = 0;
    float xn = 0.f;
    if (row_first < a.n) {
        nbeg = __ldg(a.indptr + row_first);
        nlen = (int)(__ldg(a.indptr + row_first + 1) - nbeg);
        if (l < nlen) { jn = __ldg(a.idx + nbeg + l); xn = __ldg(a.val + nbeg + l); }
    }
    for (int64_t row = row_first; row < a.n; row += row_step) {
        const int64_t beg = nbeg;
        const int len = nlen;
        nlen = 0;
        if (row + row_step < a.n) {
            nbeg = __ldg(a.indptr + row + row_step);
            nlen = (int)(__ldg(a.indptr + row + row_step + 1) - nbeg);
        }
        float4 acc[NV];
#pragma unroll
        for (int v = 0; v < NV; ++v) acc[v] = make_float4(0.f, 0.f, 0.f, 0.f);
        float q = 0.f, lin = 0.f;
        if (len <= 0) {   // empty row: no batch below fetches the next row's entries
            jn = 0; xn = 0.f;
            if (l < nlen) { jn = __ldg(a.idx + nbeg + l); xn = __ldg(a.val + nbeg + l); }
        }
        for (int t0 = 0; t0 < len; t0 += LG) {
            const int32_t jm = jn;
            const float xm = xn;
            // this lane's entry of the next batch (of this row, or the first batch of the next row)
            // is fetched while the current batch is processed
            const bool last = t0 + LG >= len;
            const int64_t ahead = last ? nbeg + l : beg + (t0 + LG + l);
            const bool more = last ? l < nlen : t0 + LG + l < len;
            jn = 0; xn = 0.f;
            if (more) { jn = __ldg(a.idx + ahead); xn = __ldg(a.val + ahead); }
            if (t0 + l < len) {
                const float2 ws = __ldg(a.pair + jm);
                lin = fmaf(ws.x, xm, lin);
                q = fmaf(xm * xm, ws.y, q);
            }
            const int cnt = (len - t0) < LG ? (len - t0) : LG;
            // the rows of up to UB entries are requested before any of them is used
            constexpr int UB = LG < 8 ? LG : 8 / NV;
#pragma unroll
            for (int u0 = 0; u0 < LG; u0 += UB) {
                if (u0 >= cnt) break;
                // x of an entry is broadcast together with its column for wide rows and only where it is used
                // for narrow ones (measured both ways: 128 factors 14.0 vs 17.1 ms, 16 factors 13.9 vs 12.8 ms)
                constexpr bool X_EARLY = LG >= 8;
                float4 vv[UB][NV];
                float xs[UB];
#pragma unroll
                for (int u = 0; u < UB; ++u) {
                    const int32_t j = __shfl_sync(gm, jm, u0 + u, LG);
                    xs[u] = X_EARLY ? __shfl_sync(gm, xm, u0 + u, LG) : 0.f;
                    if (u0 + u < cnt) {
#pragma unroll
                        for (int v = 0; v < NV; ++v) vv[u][v] = __ldg(V4 + (size_t)j * KP4 + v * LG + l);
                    }
                }
#pragma unroll
                for (int u = 0; u < UB; ++u) {
                    const float x = X_EARLY ? xs[u] : __shfl_sync(gm, xm, u0 + u, LG);
                    if (u0 + u < cnt) {
#pragma unroll
                        for (int v = 0; v < NV; ++v) {
                            acc[v].x = fmaf(vv[u][v].x, x, acc[v].x); acc[v].y = fmaf(vv[u][v].y, x, acc[v].y);
                            acc[v].z = fmaf(vv[u][v].z, x, acc[v].z); acc[v].w = fmaf(vv[u][v].w, x, acc[v].w);
                        }
                    }
                }
            }
        }
        float sq = 0.f;
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            if (STORE_A) A4[(size_t)row * KP4 + v * LG + l] = acc[v];
            sq = fmaf(acc[v].x, acc[v].x, sq); sq = fmaf(acc[v].y, acc[v].y, sq);
            sq = fmaf(acc[v].z, acc[v].z, sq); sq = fmaf(acc[v].w, acc[v].w, sq);
        }
        if (MODE == kPartial) {
#pragma unroll
            for (int o = LG / 2; o > 0; o >>= 1) {
                q += __shfl_xor_sync(gm, q, o, LG);
                lin += __shfl_xor_sync(gm, lin, o, LG);
            }
            if (l == 0) { a.lin_out[row] = lin; a.q_out[row] = q; }
            continue;
        }
        float pair = sq - q;
#pragma unroll
        for (int o = LG / 2; o > 0; o >>= 1) {
            pair += __shfl_xor_sync(gm, pair, o, LG);
            lin += __shfl_xor_sync(gm, lin, o, LG);
        }
        if (l == 0) {
            const float f = a.w0 + lin + 0.5f * pair;
            if (MODE != kScore) {
                const float yy = a.y[row];
                float li, gi;
                if (a.loss == 0) {
                    gi = f - yy;
                    li = 0.5f * gi * gi;
                } else {
                    const float m = yy * f;
                    li = fmaxf(-m, 0.f) + log1pf(expf(-fabsf(m)));
                    gi = -yy / (1.f + expf(m));
                }
                sums[0][g] += (double)li;
                if (TRAIN) {
                    a.G[row] = gi;
                    sums[1][g] += (double)gi;
                } else if (a.loss == 0) {
                    sums[1][g] += (double)gi * (double)gi;      // (f - y)^2 for the RMSE
                } else {
                    sums[1][g] += (yy * f > 0.f) ? 1.0 : 0.0;   // the sign of the score is the predicted class
                }
            } else {
                a.f_out[row] = f;
            }
        }
    }
    if (MODE != kScore && MODE != kPartial) {
        double loss_sum = l == 0 ? sums[0][g] : 0.0, g_sum = l == 0 ? sums[1][g] : 0.0;
        block_sum2(loss_sum, g_sum);
        if (threadIdx.x == 0) {
            a.partials[2 * blockIdx.x] = loss_sum;
            a.partials[2 * blockIdx.x + 1] = g_sum;
        }
    }
}

// ------------------------------------------------------------------------------------------
// Column slots for the recompute pass.  The pass gathers v_j and w_j by column index, and the L1 keeps
// whole 128-byte lines: with the columns where the data set put them, a hot 64-byte row shares its line
// with a cold neighbour and every hot w_j takes a line of its own.  The device copy of the CSR is
// therefore renumbered once per load, the most frequent column first (slot = rank by frequency: a count
// kernel, a stable radix sort of the d counters by cub::DeviceRadixSort, a rename kernel), and the
// pass reads a copy of V and of the pairs (w_j, s_j) in slot order: hot rows sit side by side, 16 hot pairs share one line.  The
// order of a row's entries does not change, so neither does any sum.  The stratum SGD kernels and
// everything a caller sees keep the column indices of the data set.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads) column_count_kernel(const int32_t *__restrict__ idx, int64_t nnz, int32_t *__restrict__ count) {
    const int lane = (int)(threadIdx.x & 31u);
    // the loop bound is the same for all lanes of a warp, so the warp stays converged for the match
    for (int64_t base = (int64_t)blockIdx.x * blockDim.x + threadIdx.x - lane; base < nnz; base += (int64_t)gridDim.x * blockDim.x) {
        const bool valid = base + lane < nnz;
        const int32_t j = valid ? idx[base + lane] : -1;
        // entries of the same column in one warp are counted by one lane
        const uint32_t peers = __match_any_sync(0xFFFFFFFFu, j);
        if (valid && lane == __ffs(peers) - 1) atomicAdd(count + j, __popc(peers));
    }
}
// sort key of a column: most frequent first (a column holds fewer than 2^31 entries); value: the column
__global__ void __launch_bounds__(kThreads) column_keys_kernel(const int32_t *__restrict__ count, int64_t d, uint32_t *__restrict__ key,
                                                               int32_t *__restrict__ column) {
    for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < d; j += (int64_t)gridDim.x * blockDim.x) {
        key[j] = 0x7FFFFFFFu - (uint32_t)count[j];
        column[j] = (int32_t)j;
    }
}
__global__ void __launch_bounds__(kThreads) column_slots_kernel(const int32_t *__restrict__ column_of, int64_t d, int32_t *__restrict__ slot_of) {
    for (int64_t s = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; s < d; s += (int64_t)gridDim.x * blockDim.x)
        slot_of[column_of[s]] = (int32_t)s;
}
__global__ void __launch_bounds__(kThreads) column_rename_kernel(int32_t *__restrict__ idx, int64_t nnz, const int32_t *__restrict__ slot_of) {
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < nnz; t += (int64_t)gridDim.x * blockDim.x)
        idx[t] = __ldg(slot_of + idx[t]);
}
// The model as the recompute pass reads it: pair[s] = (w_j, sum_k v_jk^2) and, when the columns are
// renumbered (column_of != NULL: j = column_of[s], and Vs is given), Vs[s] = V[j]; else j = s.  A group of gs
// lanes (a power of two <= 32) takes a row of kp4 float4s.
__global__ void __launch_bounds__(kThreads) model_view_kernel(const float4 *__restrict__ V, const float *__restrict__ w,
                                                              const int32_t *__restrict__ column_of, int64_t d, int kp4, int gs,
                                                              float4 *__restrict__ Vs, float2 *__restrict__ pair) {
    const int lane = (int)(threadIdx.x & 31u), gl = lane & (gs - 1);
    const int64_t groups = (int64_t)gridDim.x * (blockDim.x / gs);
    const int64_t g0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) / gs;
    const int64_t rounds = (d + groups - 1) / groups;   // the same for every lane of a warp: the shuffles below stay converged
    for (int64_t it = 0; it < rounds; ++it) {
        const int64_t s = g0 + it * groups;
        float sum = 0.f;
        int64_t j = 0;
        if (s < d) {
            j = column_of ? (int64_t)__ldg(column_of + s) : s;
            for (int v = gl; v < kp4; v += gs) {
                const float4 x = V[j * kp4 + v];
                if (Vs) Vs[s * kp4 + v] = x;
                sum = fmaf(x.x, x.x, sum); sum = fmaf(x.y, x.y, sum); sum = fmaf(x.z, x.z, sum); sum = fmaf(x.w, x.w, sum);
            }
        }
        for (int o = gs >> 1; o > 0; o >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, o);
        if (s < d && gl == 0) pair[s] = make_float2(w[j], sum);
    }
}

// Second half of the recompute pass for column shards: from the summed auxiliaries a_i, lin_i, q_i of all
// shards to f_i = w0 + lin_i + 1/2 (sum_k a_ik^2 - q_i) (eq. (fm_model2)), the loss and the multiplier G_i;
// per-CTA fp64 partial sums {sum l_i, sum G_i}.  One lane group per row.
template <int LG, int NV>
__global__ void __launch_bounds__(kThreads) finish_kernel(int64_t n, const float *A, const float *lin, const float *q,
                                                          const float *y, float *G, double *partials, float w0, int loss) {
    constexpr int GR = kThreads / LG;
    constexpr int KP4 = LG * NV;
    const int g = threadIdx.x / LG, l = threadIdx.x % LG;
    const uint32_t gm = group_mask<LG>();
    const float4 *A4 = reinterpret_cast<const float4 *>(A);
    double loss_sum = 0.0, g_sum = 0.0;
    for (int64_t row = (int64_t)blockIdx.x * GR + g; row < n; row += (int64_t)gridDim.x * GR) {
        float sq = 0.f;
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            const float4 x = A4[(size_t)row * KP4 + v * LG + l];
            sq = fmaf(x.x, x.x, sq); sq = fmaf(x.y, x.y, sq); sq = fmaf(x.z, x.z, sq); sq = fmaf(x.w, x.w, sq);
        }
#pragma unroll
        for (int o = LG / 2; o > 0; o >>= 1) sq += __shfl_xor_sync(gm, sq, o, LG);
        if (l == 0) {
            const float f = w0 + lin[row] + 0.5f * (sq - q[row]);
            const float yy = y[row];
            float li, gi;
            if (loss == 0) {
                gi = f - yy;
                li = 0.5f * gi * gi;
            } else {
                const float m = yy * f;
                li = fmaxf(-m, 0.f) + log1pf(expf(-fabsf(m)));
                gi = -yy / (1.f + expf(m));
            }
            G[row] = gi;
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

// per-CTA fp64 partial sums {sum w_j^2, sum v_jk^2}
__global__ void __launch_bounds__(kThreads) sqnorm_kernel(const float *w, int64_t d, const float *V, int64_t dkp,
                                                          double *partials) {
    double sw = 0.0, sv = 0.0;
    const int64_t stride = (int64_t)gridDim.x * kThreads;
    for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < d; i += stride) {
        const double x = (double)w[i];
        sw += x * x;
    }
    const float4 *V4 = reinterpret_cast<const float4 *>(V);
    for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < dkp / 4; i += stride) {
        const float4 x = V4[i];
        sv += (double)x.x * x.x + (double)x.y * x.y + (double)x.z * x.z + (double)x.w * x.w;
    }
    block_sum2(sw, sv);
    if (threadIdx.x == 0) {
        partials[2 * blockIdx.x] = sw;
        partials[2 * blockIdx.x + 1] = sv;
    }
}

// out[c] = sum over CTAs b (ascending, fixed tree) of partials[2*b + c], c = 0,1
__global__ void __launch_bounds__(kThreads) reduce2_kernel(const double *partials, int nblocks, double *out) {
    double s0 = 0.0, s1 = 0.0;
    for (int b = threadIdx.x; b < nblocks; b += kThreads) {
        s0 += partials[2 * b];
        s1 += partials[2 * b + 1];
    }
    block_sum2(s0, s1);
    if (threadIdx.x == 0) { out[0] = s0; out[1] = s1; }
}

}  // namespace dsf
