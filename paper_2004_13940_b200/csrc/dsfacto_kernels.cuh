// Device kernels of the DS-FACTO epoch for sm_100a.
//
// Layout shared by all kernels: a factor row (v_j or a_i) occupies Kp = 4*LG*NV floats, 16-byte
// aligned, K <= Kp, padding kept at zero.  A "lane group" of LG consecutive lanes (LG a power of
// two <= 32) owns one such row: lane l holds the float4s number l, l+LG, ... (NV of them), so a
// group's loads of one row are coalesced.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace dsf {

constexpr int kThreads = 256;
constexpr uint32_t kNoCol = 0xFFFFFFFFu;

__host__ __device__ constexpr int groups_per_cta(int LG) { return kThreads / LG; }
// entries one lane group walks sequentially per slab
__host__ __device__ constexpr int seq_len(int LG, int NV) {
    return groups_per_cta(LG) >= 64 ? 1024 / groups_per_cta(LG) : 16 / NV;
}

template <int LG>
__device__ __forceinline__ uint32_t group_mask() {
    if (LG == 32) return 0xFFFFFFFFu;
    const uint32_t lane = threadIdx.x & 31u;
    return ((1u << LG) - 1u) << (lane & ~uint32_t(LG - 1));
}

// ------------------------------------------------------------------------------------------
// Stratum SGD: one CTA per tile (r, (r+s) mod p) of inner round s.
//
// With G_i and a_i frozen, one stored entry (i,j,x) maps (w_j, v_j) affinely
// (eqs. (dsfacto_sgdupdatew), (dsfacto_sgdupdatev) regrouped):
//     v_j <- (1 - e) v_j + b a_i,   e = h (lambda_v - G_i x^2),  b = -h G_i x,  h = eta / n
//     w_j <- (1 - ew) w_j + b,      ew = h lambda_w
// A run of entries of one column is therefore a composition of affine maps.  The kernel keeps a
// composite as (D, B) with D = (product of (1-e)) - 1 and B the accumulated offset, starting from
// the identity (0, 0), so that the tiny per-entry shrink e (often below half an ulp of 1) is
// summed at full relative precision instead of being rounded away against v_j.  Composites of
// consecutive pieces combine as (D2,B2) o (D1,B1) = (D1 + D2 + D1 D2, B1 + D2 B1 + B2), and a
// finished run is applied once: v_j += D v_j + B.
//
// The tile's entries are sorted by (column, row).  They are consumed in slabs; inside a slab every
// lane group walks seq_len consecutive entries.  Runs that begin and end inside one group's piece
// are applied to global memory directly; pieces of runs that cross a group or slab boundary are
// written to shared-memory slots and stitched together in entry order by the first lane group,
// which also carries an open run from slab to slab.
// ------------------------------------------------------------------------------------------
struct SgdArgs {
    const int64_t *tile_ptr;   // p*p+1, tile t = s*p + r
    const uint2 *ent;          // packed: {(i_local << jbits) | j_local, bits of x}; wide: {i_local, j_local}
    const float *xw;           // wide layout only: x per entry
    const int64_t *row_start;  // p+1
    const int32_t *col_start;  // p+1
    const float *A;            // n * Kp
    const float *G;            // n
    float *w;                  // d
    float *V;                  // d * Kp
    int p, s, jbits;
    float h, lambda_w, lambda_v;
};

template <int LG, int NV, bool WIDE>
__global__ void __launch_bounds__(kThreads) sgd_round_kernel(const SgdArgs a) {
    constexpr int G = groups_per_cta(LG);
    constexpr int S = seq_len(LG, NV);
    constexpr int SLAB = G * S;
    constexpr int KP4 = LG * NV;  // float4s per factor row

    __shared__ float4 s_item[SLAB];          // {e, b, row (bits), j_local (bits)}
    __shared__ float4 s_slot_b[2 * G][KP4];  // offset part of a boundary piece
    __shared__ float4 s_slot_h[2 * G];       // {D, Dw, Bw, j_local (bits)}
    __shared__ int s_slot_flag[2 * G];       // 0 empty, 1 piece, 3 piece that ends its run
    __shared__ uint32_t s_prevj, s_nextj;

    const int tid = threadIdx.x;
    const int g = tid / LG;
    const int l = tid % LG;
    const int r = blockIdx.x;
    const int c = (r + a.s) % a.p;
    const int64_t t = (int64_t)a.s * a.p + r;
    const int64_t tb = a.tile_ptr[t], te = a.tile_ptr[t + 1];
    if (tb == te) return;
    const int64_t row0 = a.row_start[r];
    const int64_t col0 = a.col_start[c];
    const uint32_t jmask = a.jbits >= 32 ? 0xFFFFFFFFu : ((1u << a.jbits) - 1u);
    const float ew = a.h * a.lambda_w;
    const float4 *A4 = reinterpret_cast<const float4 *>(a.A);
    float4 *V4 = reinterpret_cast<float4 *>(a.V);

    // open run carried by lane group 0 from slab to slab
    bool has_carry = false;
    uint32_t cj = 0;
    float cD = 0.f, cDw = 0.f, cBw = 0.f;
    float4 cB[NV];

    auto apply = [&](uint32_t jl, float D, const float4 (&B)[NV], float Dw, float Bw) {
        const size_t col = (size_t)(col0 + jl);
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            float4 x = V4[col * KP4 + v * LG + l];
            x.x += fmaf(D, x.x, B[v].x);
            x.y += fmaf(D, x.y, B[v].y);
            x.z += fmaf(D, x.z, B[v].z);
            x.w += fmaf(D, x.w, B[v].w);
            V4[col * KP4 + v * LG + l] = x;
        }
        if (l == 0) {
            float wj = a.w[col];
            a.w[col] = wj + fmaf(Dw, wj, Bw);
        }
    };

    for (int64_t base = tb; base < te; base += SLAB) {
        const int count = (int)((te - base) < (int64_t)SLAB ? (te - base) : (int64_t)SLAB);
        // ---- stage the slab: one thread per entry gathers G_i and forms (e, b) ----
        for (int q = tid; q < count; q += kThreads) {
            const uint2 rec = a.ent[base + q];
            uint32_t il, jl;
            float x;
            if (WIDE) { il = rec.x; jl = rec.y; x = a.xw[base + q]; }
            else { il = rec.x >> a.jbits; jl = rec.x & jmask; x = __uint_as_float(rec.y); }
            const uint32_t row = (uint32_t)(row0 + il);
            const float gx = a.G[row] * x;
            const float e = a.h * (a.lambda_v - gx * x);
            const float b = -a.h * gx;
            s_item[q] = make_float4(e, b, __uint_as_float(row), __uint_as_float(jl));
        }
        if (tid == 0) {
            uint32_t pj = kNoCol, nj = kNoCol;
            if (base > tb) { const uint2 rec = a.ent[base - 1]; pj = WIDE ? rec.y : (rec.x & jmask); }
            if (base + count < te) { const uint2 rec = a.ent[base + count]; nj = WIDE ? rec.y : (rec.x & jmask); }
            s_prevj = pj;
            s_nextj = nj;
        }
        __syncthreads();

        // ---- every lane group walks its S consecutive entries ----
        {
            const int lo = g * S;
            const int hi = (lo + S < count) ? lo + S : count;
            int head_flag = 0, tail_flag = 0;
            if (lo < hi) {
                float4 av[S][NV];
#pragma unroll
                for (int u = 0; u < S; ++u) {
                    if (lo + u < hi) {
                        const size_t row = __float_as_uint(s_item[lo + u].z);
#pragma unroll
                        for (int v = 0; v < NV; ++v) av[u][v] = __ldg(A4 + row * KP4 + v * LG + l);
                    }
                }
                uint32_t cur = __float_as_uint(s_item[lo].w);
                const uint32_t before = (lo == 0) ? s_prevj : __float_as_uint(s_item[lo - 1].w);
                bool first_run = true;
                const bool left_open = (before == cur);
                float D = 0.f, Dw = 0.f, Bw = 0.f;
                float4 B[NV];
#pragma unroll
                for (int v = 0; v < NV; ++v) B[v] = make_float4(0.f, 0.f, 0.f, 0.f);

                auto flush = [&](bool lopen, bool ropen) {
                    if (!lopen && !ropen) {
                        apply(cur, D, B, Dw, Bw);
                    } else {
                        const int slot = lopen ? 2 * g : 2 * g + 1;
#pragma unroll
                        for (int v = 0; v < NV; ++v) s_slot_b[slot][v * LG + l] = B[v];
                        if (l == 0) s_slot_h[slot] = make_float4(D, Dw, Bw, __uint_as_float(cur));
                        const int f = ropen ? 1 : 3;
                        if (lopen) head_flag = f; else tail_flag = f;
                    }
                };
#pragma unroll
                for (int u = 0; u < S; ++u) {
                    if (lo + u < hi) {
                        const float4 it = s_item[lo + u];
                        const uint32_t jl = __float_as_uint(it.w);
                        if (jl != cur) {
                            flush(first_run && left_open, false);
                            first_run = false;
                            cur = jl;
                            D = 0.f; Dw = 0.f; Bw = 0.f;
#pragma unroll
                            for (int v = 0; v < NV; ++v) B[v] = make_float4(0.f, 0.f, 0.f, 0.f);
                        }
                        const float e = it.x, b = it.y;
                        // (D,B) <- step o (D,B):  D + (-e) + D(-e),  B + (-e)B + b a_i
                        D = fmaf(-e, D, D - e);
                        Dw = fmaf(-ew, Dw, Dw - ew);
                        Bw = fmaf(-ew, Bw, Bw + b);
#pragma unroll
                        for (int v = 0; v < NV; ++v) {
                            B[v].x = fmaf(b, av[u][v].x, fmaf(-e, B[v].x, B[v].x));
                            B[v].y = fmaf(b, av[u][v].y, fmaf(-e, B[v].y, B[v].y));
                            B[v].z = fmaf(b, av[u][v].z, fmaf(-e, B[v].z, B[v].z));
                            B[v].w = fmaf(b, av[u][v].w, fmaf(-e, B[v].w, B[v].w));
                        }
                    }
                }
                const uint32_t after = (hi == count) ? s_nextj : __float_as_uint(s_item[hi].w);
                flush(first_run && left_open, after == cur);
            }
            if (l == 0) {
                s_slot_flag[2 * g] = head_flag;
                s_slot_flag[2 * g + 1] = tail_flag;
            }
        }
        __syncthreads();

        // ---- lane group 0 stitches the boundary pieces together in entry order ----
        if (tid < LG) {
            for (int slot = 0; slot < 2 * G; ++slot) {
                const int f = s_slot_flag[slot];
                if (f == 0) continue;
                const float4 hd = s_slot_h[slot];
                if (has_carry) {
                    // piece (hd, slot_b) comes after the carried composite
#pragma unroll
                    for (int v = 0; v < NV; ++v) {
                        const float4 b2 = s_slot_b[slot][v * LG + l];
                        cB[v].x = fmaf(hd.x, cB[v].x, cB[v].x) + b2.x;
                        cB[v].y = fmaf(hd.x, cB[v].y, cB[v].y) + b2.y;
                        cB[v].z = fmaf(hd.x, cB[v].z, cB[v].z) + b2.z;
                        cB[v].w = fmaf(hd.x, cB[v].w, cB[v].w) + b2.w;
                    }
                    cBw = fmaf(hd.y, cBw, cBw) + hd.z;
                    cD = fmaf(cD, hd.x, cD + hd.x);
                    cDw = fmaf(cDw, hd.y, cDw + hd.y);
                } else {
#pragma unroll
                    for (int v = 0; v < NV; ++v) cB[v] = s_slot_b[slot][v * LG + l];
                    cD = hd.x; cDw = hd.y; cBw = hd.z;
                    cj = __float_as_uint(hd.w);
                    has_carry = true;
                }
                if (f & 2) {
                    apply(cj, cD, cB, cDw, cBw);
                    has_carry = false;
                }
            }
        }
        // no barrier needed here: the next slab's staging touches only s_item/s_prevj/s_nextj,
        // which the stitching above does not read; the slots are rewritten after the next barrier
    }
}

// ------------------------------------------------------------------------------------------
// Recompute pass (eq. (compute_a_jk), eq. (fm_model2), multiplier G): one lane group per row.
//   a_ik = sum_j v_jk x_ij ; lin_i = sum_j w_j x_ij ; q_i = sum_j sum_k (v_jk x_ij)^2
//   f_i = w0 + lin_i + 1/2 (sum_k a_ik^2 - q_i)
// TRAIN: writes A, G and per-CTA fp64 partial sums {sum l_i, sum G_i}; otherwise writes f only.
// ------------------------------------------------------------------------------------------
struct RefreshArgs {
    int64_t n;
    const int64_t *indptr;
    const int32_t *idx;
    const float *val;
    const float *y;
    const float *w;
    const float *V;
    float *A;
    float *G;
    float *f_out;
    double *partials;  // 2 per CTA
    float w0;
    int loss;
};

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

template <int LG, int NV, bool TRAIN>
__global__ void __launch_bounds__(kThreads) refresh_kernel(const RefreshArgs a) {
    constexpr int G = groups_per_cta(LG);
    constexpr int KP4 = LG * NV;
    const int g = threadIdx.x / LG;
    const int l = threadIdx.x % LG;
    const uint32_t gm = group_mask<LG>();
    const float4 *V4 = reinterpret_cast<const float4 *>(a.V);
    float4 *A4 = reinterpret_cast<float4 *>(a.A);
    double loss_sum = 0.0, g_sum = 0.0;

    for (int64_t row = (int64_t)blockIdx.x * G + g; row < a.n; row += (int64_t)gridDim.x * G) {
        const int64_t beg = a.indptr[row], end = a.indptr[row + 1];
        float4 acc[NV];
#pragma unroll
        for (int v = 0; v < NV; ++v) acc[v] = make_float4(0.f, 0.f, 0.f, 0.f);
        float q = 0.f, lin = 0.f;
        for (int64_t t0 = beg; t0 < end; t0 += LG) {
            const int64_t mine = t0 + l;
            int32_t jm = 0;
            float xm = 0.f;
            if (mine < end) { jm = __ldg(a.idx + mine); xm = __ldg(a.val + mine); lin = fmaf(__ldg(a.w + jm), xm, lin); }
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
            if (TRAIN) A4[(size_t)row * KP4 + v * LG + l] = acc[v];
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
            const float f = a.w0 + lin + 0.5f * pair;
            if (TRAIN) {
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
                a.G[row] = gi;
                loss_sum += (double)li;
                g_sum += (double)gi;
            } else {
                a.f_out[row] = f;
            }
        }
    }
    if (TRAIN) {
        block_sum2(loss_sum, g_sum);
        if (threadIdx.x == 0) {
            a.partials[2 * blockIdx.x] = loss_sum;
            a.partials[2 * blockIdx.x + 1] = g_sum;
        }
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
