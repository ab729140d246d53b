// Stratum SGD kernels of the DS-FACTO epoch for sm_100a.
//
// With G_i and a_i frozen, one stored entry (i,j,x) maps (w_j, v_j) affinely
// (eqs. (dsfacto_sgdupdatew), (dsfacto_sgdupdatev) regrouped):
//     v_j <- (1 - e) v_j + b a_i,   e = h (lambda_v - G_i x^2),  b = -h G_i x,  h = eta / n
//     w_j <- (1 - ew) w_j + b,      ew = h lambda_w
// so a run of entries of one column is a composition of affine maps.  A composite is kept as
// (D, B) with D = (product of (1-e)) - 1 and B the accumulated offset, starting from the identity
// (0, 0): the per-entry shrink e is often below half an ulp of 1, and summing it into D keeps it at
// full relative precision instead of losing it against v_j.  Consecutive pieces combine as
//     (D2,B2) o (D1,B1) = (D1 + D2 + D1 D2,  B1 + D2 B1 + B2)
// and a finished run is applied once: v_j += D v_j + B.
#pragma once
#include "dsfacto_common.cuh"

namespace dsf {

constexpr int kChunk = 1024;       // entries per CTA
constexpr int kWarpEntries = 128;  // entries per warp

// entries one lane group walks sequentially per pass
__host__ __device__ constexpr int chunk_seq_len(int LG, int NV) { return LG == 1 ? 4 : (LG == 2 ? 8 : 16 / NV); }
// floats per chunk record in global scratch: 3 header float4s + head offsets + tail offsets
__host__ __device__ constexpr int chunk_record_floats(int Kp) { return 12 + 2 * Kp; }

template <int NV>
struct Comp {
    float D, Dw, Bw;
    float4 B[NV];
};

template <int NV>
__device__ __forceinline__ void comp_identity(Comp<NV> &c) {
    c.D = 0.f; c.Dw = 0.f; c.Bw = 0.f;
#pragma unroll
    for (int v = 0; v < NV; ++v) c.B[v] = make_float4(0.f, 0.f, 0.f, 0.f);
}

// second o first (first acts first)
template <int NV>
__device__ __forceinline__ Comp<NV> compose(const Comp<NV> &first, const Comp<NV> &second) {
    Comp<NV> r;
#pragma unroll
    for (int v = 0; v < NV; ++v) {
        r.B[v].x = fmaf(second.D, first.B[v].x, first.B[v].x) + second.B[v].x;
        r.B[v].y = fmaf(second.D, first.B[v].y, first.B[v].y) + second.B[v].y;
        r.B[v].z = fmaf(second.D, first.B[v].z, first.B[v].z) + second.B[v].z;
        r.B[v].w = fmaf(second.D, first.B[v].w, first.B[v].w) + second.B[v].w;
    }
    r.Bw = fmaf(second.Dw, first.Bw, first.Bw) + second.Bw;
    r.D = fmaf(first.D, second.D, first.D + second.D);
    r.Dw = fmaf(first.Dw, second.Dw, first.Dw + second.Dw);
    return r;
}

template <int NV>
__device__ __forceinline__ Comp<NV> comp_shfl_up(const Comp<NV> &c, int delta) {
    Comp<NV> r;
    r.D = __shfl_up_sync(0xFFFFFFFFu, c.D, delta);
    r.Dw = __shfl_up_sync(0xFFFFFFFFu, c.Dw, delta);
    r.Bw = __shfl_up_sync(0xFFFFFFFFu, c.Bw, delta);
#pragma unroll
    for (int v = 0; v < NV; ++v) {
        r.B[v].x = __shfl_up_sync(0xFFFFFFFFu, c.B[v].x, delta);
        r.B[v].y = __shfl_up_sync(0xFFFFFFFFu, c.B[v].y, delta);
        r.B[v].z = __shfl_up_sync(0xFFFFFFFFu, c.B[v].z, delta);
        r.B[v].w = __shfl_up_sync(0xFFFFFFFFu, c.B[v].w, delta);
    }
    return r;
}

template <int NV>
__device__ __forceinline__ Comp<NV> comp_shfl(const Comp<NV> &c, int src) {
    Comp<NV> r;
    r.D = __shfl_sync(0xFFFFFFFFu, c.D, src);
    r.Dw = __shfl_sync(0xFFFFFFFFu, c.Dw, src);
    r.Bw = __shfl_sync(0xFFFFFFFFu, c.Bw, src);
#pragma unroll
    for (int v = 0; v < NV; ++v) {
        r.B[v].x = __shfl_sync(0xFFFFFFFFu, c.B[v].x, src);
        r.B[v].y = __shfl_sync(0xFFFFFFFFu, c.B[v].y, src);
        r.B[v].z = __shfl_sync(0xFFFFFFFFu, c.B[v].z, src);
        r.B[v].w = __shfl_sync(0xFFFFFFFFu, c.B[v].w, src);
    }
    return r;
}

// ------------------------------------------------------------------------------------------
// sgd_chunk_kernel: one CTA per chunk of kChunk consecutive entries of one tile.
//
// A launch covers tiles with pairwise disjoint column blocks: the p tiles of one inner round
// (sweep 0) or the p tiles of one row block (sweep 1).  A tile's entries are sorted by (column,
// row).  Every warp owns kWarpEntries consecutive entries and walks them in passes; inside a pass
// each lane group walks S consecutive entries sequentially.  A "boundary" sits before an entry
// whose column differs from the entry before it (the tile start counts).  A run that lies inside
// one lane group's piece is applied to the column state at once.  Runs that cross lane groups are
// joined by a segmented scan over the groups of the warp (shuffles); runs that cross warps by the
// first lane group of warp 0 (shared memory); runs that cross chunks by whichever chunk of the tile
// finishes last (records in global scratch plus one counter per tile - no CTA waits for another).
//
// Column state: in a direct tile it is (w_j, v_j).  In a tail tile (sweep 1, r > c) it is a
// per-column composite T_j, identity at the start of the epoch and applied to (w_j, v_j) by
// sgd_finalize_* after the sweep.  The sweep visits row blocks p-1, .., 0, so for column block c
// the tail tiles (r = p-1 .. c+1) and then the direct tiles (r = c .. 0) are each met in the
// stratified order of the rounds, and "T_j after v_j" restores the order c, .., 0, p-1, .., c+1.
// Meanwhile all entries of a row meet in one launch, so (a_i, G_i) come from L2 after first touch.
// ------------------------------------------------------------------------------------------
struct SgdChunkArgs {
    const int64_t *tile_ptr;   // p*p+1, tile t = s*p + r
    const uint2 *ent;          // packed: {(i_local << jbits) | j_local, bits of x}; wide: {i_local, j_local}
    const float *xw;           // wide layout only: x per entry
    const int64_t *row_start;  // p+1
    const int32_t *col_start;  // p+1
    const float *A;            // n * Kp
    const float *G;            // n
    float *w;                  // d
    float *V;                  // d * Kp
    float *Tb;                 // d * Kp  offset part of T_j            (sweep 1)
    float *Td;                 // d * 4   {D, Dw, Bw, -} of T_j         (sweep 1)
    const int2 *chunk_map;     // per CTA of this launch: {tile t, chunk index inside the tile}
    float *records;            // chunk_record_floats(Kp) floats per CTA of this launch
    int *tile_count;           // p*p, all zero between launches
    int p, jbits, sweep;
    float h, lambda_w, lambda_v;
};

template <int LG, int NV, bool WIDE>
__global__ void __launch_bounds__(kThreads) sgd_chunk_kernel(const SgdChunkArgs a) {
    constexpr int S = chunk_seq_len(LG, NV);
    constexpr int GW = 32 / LG;   // lane groups per warp
    constexpr int PASS = GW * S;  // entries per warp pass
    constexpr int PP = kWarpEntries / PASS;
    constexpr int KP4 = LG * NV;
    constexpr int NW = kThreads / 32;
    constexpr int BATCH = S < 8 ? S : 8;  // rows of A fetched ahead of use
    constexpr int REC4 = chunk_record_floats(4 * KP4) / 4;
    static_assert(PP >= 1 && PASS * PP == kWarpEntries, "a warp's entries must be whole passes");
    static_assert(NW * kWarpEntries == kChunk, "chunk = warps x entries per warp");
    typedef Comp<NV> C;

    __shared__ float4 s_item[NW][PASS];  // {e, b, row (bits), j_local (bits)}
    __shared__ float4 s_wB[NW][2][KP4];  // per warp: offsets of its head piece / open tail
    __shared__ float4 s_wH[NW][2];       // per warp: {D, Dw, Bw, column (bits)} of head / tail
    __shared__ int s_wflag[NW];          // warp saw a boundary
    __shared__ int s_last;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane / LG, l = lane % LG;
    const int2 cm = a.chunk_map[blockIdx.x];
    const int64_t t = cm.x;
    const int r = (int)(t % a.p), s = (int)(t / a.p);
    const int c = (r + s) % a.p;
    const bool tail_mode = a.sweep == 1 && r > c;
    const int64_t tb = a.tile_ptr[t], te = a.tile_ptr[t + 1];
    const int64_t cb = tb + (int64_t)cm.y * kChunk;
    const int64_t ce = (cb + kChunk < te) ? cb + kChunk : te;
    const int64_t wb = cb + (int64_t)warp * kWarpEntries;
    const int64_t we = (wb + kWarpEntries < ce) ? wb + kWarpEntries : ce;
    const int64_t row0 = a.row_start[r];
    const int64_t col0 = a.col_start[c];
    const uint32_t jmask = a.jbits >= 32 ? 0xFFFFFFFFu : ((1u << a.jbits) - 1u);
    const float ew = a.h * a.lambda_w;
    const float4 *A4 = reinterpret_cast<const float4 *>(a.A);
    float4 *V4 = reinterpret_cast<float4 *>(a.V);
    float4 *Tb4 = reinterpret_cast<float4 *>(a.Tb);
    float4 *Td4 = reinterpret_cast<float4 *>(a.Td);

    // applies a finished run to the state of local column jl (the LG lanes of one group)
    auto apply = [&](uint32_t jl, const C &x) {
        if (jl == kNoCol) return;
        const size_t col = (size_t)(col0 + jl);
        if (!tail_mode) {
#pragma unroll
            for (int v = 0; v < NV; ++v) {
                float4 y = V4[col * KP4 + v * LG + l];
                y.x += fmaf(x.D, y.x, x.B[v].x);
                y.y += fmaf(x.D, y.y, x.B[v].y);
                y.z += fmaf(x.D, y.z, x.B[v].z);
                y.w += fmaf(x.D, y.w, x.B[v].w);
                V4[col * KP4 + v * LG + l] = y;
            }
            if (l == 0) {
                const float wj = a.w[col];
                a.w[col] = wj + fmaf(x.Dw, wj, x.Bw);
            }
        } else {
#pragma unroll
            for (int v = 0; v < NV; ++v) {
                float4 y = Tb4[col * KP4 + v * LG + l];
                y.x = fmaf(x.D, y.x, y.x) + x.B[v].x;
                y.y = fmaf(x.D, y.y, y.y) + x.B[v].y;
                y.z = fmaf(x.D, y.z, y.z) + x.B[v].z;
                y.w = fmaf(x.D, y.w, y.w) + x.B[v].w;
                Tb4[col * KP4 + v * LG + l] = y;
            }
            if (l == 0) {
                float4 y = Td4[col];
                y.z = fmaf(x.Dw, y.z, y.z) + x.Bw;
                y.x = fmaf(y.x, x.D, y.x + x.D);
                y.y = fmaf(y.y, x.Dw, y.y + x.Dw);
                Td4[col] = y;
            }
        }
    };

    // ---------------- warp phase ----------------
    C wcarry;  // open run of this warp so far
    comp_identity(wcarry);
    bool wflag = false;  // a boundary has been seen in this warp
    uint32_t last_col = kNoCol;

    for (int pp = 0; pp < PP; ++pp) {
        const int64_t pb = wb + (int64_t)pp * PASS;
        if (pb >= we) break;
        const int cnt = (int)((we - pb) < (int64_t)PASS ? (we - pb) : (int64_t)PASS);
        // stage: one lane per entry gathers G_i and forms (e, b)
        for (int q = lane; q < cnt; q += 32) {
            const uint2 rec = a.ent[pb + q];
            uint32_t il, jl;
            float x;
            if (WIDE) { il = rec.x; jl = rec.y; x = a.xw[pb + q]; }
            else { il = rec.x >> a.jbits; jl = rec.x & jmask; x = __uint_as_float(rec.y); }
            const uint32_t row = (uint32_t)(row0 + il);
            const float gx = __ldg(a.G + row) * x;
            s_item[warp][q] = make_float4(a.h * (a.lambda_v - gx * x), -a.h * gx, __uint_as_float(row),
                                          __uint_as_float(jl));
        }
        uint32_t before = kNoCol;  // column of the entry just before this pass, if it is in the tile
        if (pp > 0) before = last_col;
        else if (pb > tb) {
            const uint2 rec = a.ent[pb - 1];
            before = WIDE ? rec.y : (rec.x & jmask);
        }
        __syncwarp();
        last_col = __float_as_uint(s_item[warp][cnt - 1].w);

        const int lo = g * S;
        const int hi = (lo + S < cnt) ? lo + S : cnt;
        bool hasb = false;
        uint32_t headcol = kNoCol;
        C cur, head;
        comp_identity(cur);
        comp_identity(head);
        if (lo < hi) {
            uint32_t prevj = (lo == 0) ? before : __float_as_uint(s_item[warp][lo - 1].w);
#pragma unroll
            for (int u0 = 0; u0 < S; u0 += BATCH) {
                float4 av[BATCH][NV];
#pragma unroll
                for (int u = 0; u < BATCH; ++u) {
                    if (lo + u0 + u < hi) {
                        const size_t row = __float_as_uint(s_item[warp][lo + u0 + u].z);
#pragma unroll
                        for (int v = 0; v < NV; ++v) av[u][v] = __ldg(A4 + row * KP4 + v * LG + l);
                    }
                }
#pragma unroll
                for (int u = 0; u < BATCH; ++u) {
                    if (lo + u0 + u < hi) {
                        const float4 it = s_item[warp][lo + u0 + u];
                        const uint32_t jl = __float_as_uint(it.w);
                        if (jl != prevj) {  // boundary before this entry
                            if (!hasb) { head = cur; headcol = prevj; hasb = true; }
                            else apply(prevj, cur);
                            comp_identity(cur);
                            prevj = jl;
                        }
                        const float e = it.x, b = it.y;
                        cur.D = fmaf(-e, cur.D, cur.D - e);
                        cur.Dw = fmaf(-ew, cur.Dw, cur.Dw - ew);
                        cur.Bw = fmaf(-ew, cur.Bw, cur.Bw + b);
#pragma unroll
                        for (int v = 0; v < NV; ++v) {
                            cur.B[v].x = fmaf(b, av[u][v].x, fmaf(-e, cur.B[v].x, cur.B[v].x));
                            cur.B[v].y = fmaf(b, av[u][v].y, fmaf(-e, cur.B[v].y, cur.B[v].y));
                            cur.B[v].z = fmaf(b, av[u][v].z, fmaf(-e, cur.B[v].z, cur.B[v].z));
                            cur.B[v].w = fmaf(b, av[u][v].w, fmaf(-e, cur.B[v].w, cur.B[v].w));
                        }
                    }
                }
            }
        }
        // ---- segmented inclusive scan over the lane groups of the warp ----
        // element of a group: (hasb, composite after its last boundary, or of its whole piece)
        C inc = cur;
        bool finc = hasb;
        if (GW > 1) {
#pragma unroll
            for (int delta = 1; delta < GW; delta <<= 1) {
                const C o = comp_shfl_up<NV>(inc, delta * LG);
                const bool of = __shfl_up_sync(0xFFFFFFFFu, (int)finc, delta * LG) != 0;
                if (g >= delta) {
                    if (!finc) inc = compose<NV>(o, inc);
                    finc = finc || of;
                }
            }
        }
        C ex;  // what is open on this group's left, from earlier groups of this pass
        bool fex = false;
        comp_identity(ex);
        if (GW > 1) {
            const C up = comp_shfl_up<NV>(inc, LG);
            const bool fup = __shfl_up_sync(0xFFFFFFFFu, (int)finc, LG) != 0;
            if (g > 0) { ex = up; fex = fup; }
        }
        if (hasb) {  // this group ends the run that was open on its left
            C closing = fex ? ex : compose<NV>(wcarry, ex);
            closing = compose<NV>(closing, head);
            if (fex || wflag) {
                apply(headcol, closing);
            } else {  // the run began before this warp: hand it to the CTA phase
#pragma unroll
                for (int v = 0; v < NV; ++v) s_wB[warp][0][v * LG + l] = closing.B[v];
                if (l == 0) s_wH[warp][0] = make_float4(closing.D, closing.Dw, closing.Bw, __uint_as_float(headcol));
            }
        }
        // open run at the end of the pass = inclusive result of the last group
        const C lastc = comp_shfl<NV>(inc, (GW - 1) * LG + l);
        const bool lastf = __shfl_sync(0xFFFFFFFFu, (int)finc, (GW - 1) * LG) != 0;
        wcarry = lastf ? lastc : compose<NV>(wcarry, lastc);
        wflag = wflag || lastf;
        __syncwarp();
    }
    if (lane < LG) {
#pragma unroll
        for (int v = 0; v < NV; ++v) s_wB[warp][1][v * LG + l] = wcarry.B[v];
        if (l == 0) {
            s_wH[warp][1] = make_float4(wcarry.D, wcarry.Dw, wcarry.Bw, __uint_as_float(last_col));
            s_wflag[warp] = wflag ? 1 : 0;
        }
    }
    __syncthreads();

    // ---------------- CTA phase: first lane group of warp 0 joins the warps ----------------
    const int nchunks = (int)((te - tb + kChunk - 1) / kChunk);
    if (tid < LG) {
        bool cta_flag = false;
        uint32_t cta_headcol = kNoCol, cta_tailcol = kNoCol;
        C cta_head, run;
        comp_identity(cta_head);
        comp_identity(run);
        for (int w = 0; w < NW; ++w) {
            C tl;
            const float4 th = s_wH[w][1];
            tl.D = th.x; tl.Dw = th.y; tl.Bw = th.z;
#pragma unroll
            for (int v = 0; v < NV; ++v) tl.B[v] = s_wB[w][1][v * LG + l];
            if (!s_wflag[w]) {
                run = compose<NV>(run, tl);
            } else {
                C hd;
                const float4 hh = s_wH[w][0];
                hd.D = hh.x; hd.Dw = hh.y; hd.Bw = hh.z;
#pragma unroll
                for (int v = 0; v < NV; ++v) hd.B[v] = s_wB[w][0][v * LG + l];
                const C closing = compose<NV>(run, hd);
                const uint32_t hc = __float_as_uint(hh.w);
                if (!cta_flag) { cta_head = closing; cta_headcol = hc; cta_flag = true; }
                else apply(hc, closing);
                run = tl;
            }
            if (__float_as_uint(th.w) != kNoCol) cta_tailcol = __float_as_uint(th.w);
        }
        if (nchunks == 1) {  // the tile starts and ends here: nothing stays open
            if (cta_flag) apply(cta_headcol, cta_head);
            apply(cta_tailcol, run);
        } else {
            float4 *rec4 = reinterpret_cast<float4 *>(a.records) + (size_t)blockIdx.x * REC4;
            if (l == 0) {
                rec4[0] = make_float4(cta_head.D, cta_head.Dw, cta_head.Bw, __uint_as_float(cta_headcol));
                rec4[1] = make_float4(run.D, run.Dw, run.Bw, __uint_as_float(cta_tailcol));
                rec4[2] = make_float4(__uint_as_float(cta_flag ? 1u : 0u), 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int v = 0; v < NV; ++v) {
                rec4[3 + v * LG + l] = cta_head.B[v];
                rec4[3 + KP4 + v * LG + l] = run.B[v];
            }
        }
    }
    if (nchunks == 1) return;

    // ---------------- tile phase: the chunk that finishes last joins the chunks ----------------
    __threadfence();
    __syncthreads();
    if (tid == 0) s_last = (atomicAdd(a.tile_count + t, 1) == nchunks - 1) ? 1 : 0;
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    if (tid < LG) {
        const float4 *base4 = reinterpret_cast<const float4 *>(a.records) + ((size_t)blockIdx.x - (size_t)cm.y) * REC4;
        C run;
        comp_identity(run);
        uint32_t tailcol = kNoCol;
        for (int k = 0; k < nchunks; ++k) {
            const float4 *rec4 = base4 + (size_t)k * REC4;
            const float4 hh = __ldcg(rec4 + 0);
            const float4 th = __ldcg(rec4 + 1);
            const float4 fl = __ldcg(rec4 + 2);
            C hd, tl;
            hd.D = hh.x; hd.Dw = hh.y; hd.Bw = hh.z;
            tl.D = th.x; tl.Dw = th.y; tl.Bw = th.z;
#pragma unroll
            for (int v = 0; v < NV; ++v) {
                hd.B[v] = __ldcg(rec4 + 3 + v * LG + l);
                tl.B[v] = __ldcg(rec4 + 3 + KP4 + v * LG + l);
            }
            if (__float_as_uint(fl.x) == 0u) {
                run = compose<NV>(run, tl);
            } else {
                apply(__float_as_uint(hh.w), compose<NV>(run, hd));
                run = tl;
            }
            tailcol = __float_as_uint(th.w);
        }
        apply(tailcol, run);  // the end of the tile closes the last run
        if (l == 0) a.tile_count[t] = 0;
    }
}

// After a row-block sweep: (w_j, v_j) <- T_j (w_j, v_j), then T_j <- identity.
__global__ void __launch_bounds__(kThreads) sgd_finalize_v_kernel(float *V, float *Tb, const float *Td, int64_t d,
                                                                  int kp4) {
    const int64_t total = d * kp4;
    float4 *V4 = reinterpret_cast<float4 *>(V);
    float4 *Tb4 = reinterpret_cast<float4 *>(Tb);
    const float4 *Td4 = reinterpret_cast<const float4 *>(Td);
    for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < total; i += (int64_t)gridDim.x * kThreads) {
        const float D = Td4[i / kp4].x;
        float4 y = V4[i];
        const float4 b = Tb4[i];
        y.x += fmaf(D, y.x, b.x);
        y.y += fmaf(D, y.y, b.y);
        y.z += fmaf(D, y.z, b.z);
        y.w += fmaf(D, y.w, b.w);
        V4[i] = y;
        Tb4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
}
__global__ void __launch_bounds__(kThreads) sgd_finalize_w_kernel(float *w, float *Td, int64_t d) {
    float4 *Td4 = reinterpret_cast<float4 *>(Td);
    for (int64_t j = (int64_t)blockIdx.x * kThreads + threadIdx.x; j < d; j += (int64_t)gridDim.x * kThreads) {
        const float4 tj = Td4[j];
        const float wj = w[j];
        w[j] = wj + fmaf(tj.y, wj, tj.z);
        Td4[j] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
}

}  // namespace dsf
