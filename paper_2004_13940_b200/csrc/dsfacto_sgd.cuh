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
// and a finished run is applied once: v_j <- (1 + D) v_j + B.
//
// During the SGD phase the column state is held in scaled form, v_j = (1 + sigma_j) u_j (and the
// same for w_j), with sigma_j = 0 at the start of the phase.  Applying a run then needs only the
// 8-byte scale pair of the column:  sigma' = sigma + D + sigma D,  u_j += B / (1 + sigma'),
// so the K-wide part is an add that nobody waits for (red.global.add; every column receives at
// most one per launch, so the result does not depend on timing).  sgd_finalize_* turns the state
// back into plain (w, V) at the end of the phase.  The scaled form breaks down only if some
// 1 + sigma reaches zero, i.e. a step so large that a run wipes its column; the parameters then
// become non-finite and the epoch reports divergence.
#pragma once
#include "dsfacto_common.cuh"

namespace dsf {

constexpr int kSgdThreads = 32;   // one warp per CTA: a finished warp frees its registers and shared memory at once
constexpr int kSgdWarps = kSgdThreads / 32;
constexpr int kWarpEntries = 512;                 // entries per warp
constexpr int kChunk = kSgdWarps * kWarpEntries;  // entries per CTA, at most (a launch may use shorter chunks)
constexpr int kSgdSpinLimit = 1 << 22;            // polls (about 100 ns each) before a dependency wait gives up
// Words of the launch's synchronisation array.  The ticket counter takes one atomic per CTA and the
// progress counters are polled by waiting CTAs, so every word sits in a 128-byte line of its own.
constexpr int kSyncStride = 32;                   // ints between two words
constexpr int kSyncTicket = 0;                    // next chunk to hand out
constexpr int kSyncError = kSyncStride;           // set when a dependency wait ran out
__host__ __device__ constexpr size_t sync_done(int c) { return (size_t)(2 + c) * kSyncStride; }  // finished tiles of column block c
__host__ __device__ constexpr size_t sync_words(int p) { return (size_t)(2 + p) * kSyncStride; }

// entries of one warp pass: sized so that the gathered rows of A fill about 4 KB of shared memory, but
// never fewer than 16 entries: with 8-entry passes (rows of 512 bytes and more) the fixed cost of a
// pass and its one exposed gather latency dominated (K = 128: 59.1 ms per sweep with 8, 46.7 with 16,
// 54.6 with 32 on the 400 M-entry workload)
__host__ __device__ constexpr int sgd_pass_len(int LG, int NV) {
    return 256 / (LG * NV) > 256 ? 256 : (256 / (LG * NV) < 16 ? 16 : 256 / (LG * NV));
}
// resident one-warp CTAs per SM the register budget is cut for: 24 for rows up to 256 bytes; wider
// rows hold 16 entries per lane group in flight and are limited by shared memory anyway
__host__ __device__ constexpr int sgd_min_ctas(int LG, int NV) { return LG * NV >= 32 ? 12 : 24; }
// floats per chunk record in global scratch: 3 header float4s + head offsets + tail offsets
__host__ __device__ constexpr int chunk_record_floats(int Kp) { return 12 + 2 * Kp; }

// shared-memory carve-up of one warp, in float4 units
template <int LG, int NV>
struct SgdSmem {
    static constexpr int GW = 32 / LG;
    static constexpr int KP4 = LG * NV;
    static constexpr int PASS = sgd_pass_len(LG, NV);
    static constexpr int S = PASS / GW;                  // entries a lane group walks per pass
    static constexpr int ITEM_STRIDE = S + 1;            // +1: lane groups land in different banks
    static constexpr int ROW_STRIDE = (S + (LG < 8 ? 1 : 0)) * KP4;
    static constexpr int ITEMS = 0;                      // GW * ITEM_STRIDE   {e, b, row, j_local}
    static constexpr int ROWS = ITEMS + GW * ITEM_STRIDE;  // GW * ROW_STRIDE  gathered rows a_i
    static constexpr int SCALES = ROWS + GW * ROW_STRIDE;  // GW * ITEM_STRIDE float4: scale pair of the
                                                         // column whose run starts at that entry
    static constexpr int WARP = SCALES + GW * ITEM_STRIDE;  // float4s per warp
    // per CTA, after the warps: per warp head/tail pieces, then the chunk head piece
    static constexpr int WPIECE = kSgdWarps * WARP;      // kSgdWarps * 2 * (KP4+1)
    static constexpr int CPIECE = WPIECE + kSgdWarps * 2 * (KP4 + 1);  // (KP4+1)
    static constexpr int TOTAL = CPIECE + (KP4 + 1);
    static constexpr int BYTES = TOTAL * 16 + 16 * kSgdWarps;  // + per-warp boundary flags
};

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
__device__ __forceinline__ Comp<NV> comp_shfl_down(const Comp<NV> &c, int delta) {
    Comp<NV> r;
    r.D = __shfl_down_sync(0xFFFFFFFFu, c.D, delta);
    r.Dw = __shfl_down_sync(0xFFFFFFFFu, c.Dw, delta);
    r.Bw = __shfl_down_sync(0xFFFFFFFFu, c.Bw, delta);
#pragma unroll
    for (int v = 0; v < NV; ++v) {
        r.B[v].x = __shfl_down_sync(0xFFFFFFFFu, c.B[v].x, delta);
        r.B[v].y = __shfl_down_sync(0xFFFFFFFFu, c.B[v].y, delta);
        r.B[v].z = __shfl_down_sync(0xFFFFFFFFu, c.B[v].z, delta);
        r.B[v].w = __shfl_down_sync(0xFFFFFFFFu, c.B[v].w, delta);
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

// a composite as stored in shared or global memory: KP4 offset float4s, then {D, Dw, Bw, column}
template <int LG, int NV>
__device__ __forceinline__ void comp_store(float4 *dst, const Comp<NV> &c, uint32_t col, int l) {
#pragma unroll
    for (int v = 0; v < NV; ++v) dst[v * LG + l] = c.B[v];
    if (l == 0) dst[LG * NV] = make_float4(c.D, c.Dw, c.Bw, __uint_as_float(col));
}
template <int LG, int NV>
__device__ __forceinline__ uint32_t comp_load(const float4 *src, Comp<NV> &c, int l) {
#pragma unroll
    for (int v = 0; v < NV; ++v) c.B[v] = src[v * LG + l];
    const float4 hd = src[LG * NV];
    c.D = hd.x; c.Dw = hd.y; c.Bw = hd.z;
    return __float_as_uint(hd.w);
}

__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gmem_src) {
    const unsigned s = (unsigned)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(s), "l"(gmem_src) : "memory");
}
// fire-and-forget adds into global memory
__device__ __forceinline__ void red_add4(float4 *p, float x, float y, float z, float w) {
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(x), "f"(y), "f"(z), "f"(w) : "memory");
}
__device__ __forceinline__ void red_add1(float *p, float x) {
    asm volatile("red.global.add.f32 [%0], %1;" ::"l"(p), "f"(x) : "memory");
}
// 1 / x by the special-function unit alone (within one unit in the last place): it scales an increment,
// so a correctly rounded reciprocal would buy nothing but instructions
__device__ __forceinline__ float rcp_fast(float x) {
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}
__device__ __forceinline__ void cp_async_wait_all() {
    asm volatile("cp.async.commit_group;\ncp.async.wait_group 0;\n" ::: "memory");
}

// One step of a segmented scan over the lane groups of a warp (all 32 lanes must call it).
// Each lane group contributes an element: `hasb` (it holds a run boundary), `head` (composite of
// what precedes its first boundary) and `cur` (composite after its last boundary, or of the whole
// element when it has none).  `carry`/`cflag` describe the run left open by earlier steps and are
// updated to the run left open after this step.  For a group with a boundary, `closing` becomes
// the composite of the run that ends at its first boundary and `outer` tells whether that run began
// before the first step (nothing to its left held a boundary).
template <int LG, int NV>
__device__ __forceinline__ void scan_step(bool hasb, const Comp<NV> &head, const Comp<NV> &cur, Comp<NV> &carry,
                                          bool &cflag, Comp<NV> &closing, bool &outer) {
    constexpr int GW = 32 / LG;
    const int lane = threadIdx.x & 31;
    const int g = lane / LG, l = lane % LG;
    Comp<NV> inc = cur;
    bool finc = hasb;
    if (GW > 1) {
#pragma unroll
        for (int delta = 1; delta < GW; delta <<= 1) {
            const Comp<NV> o = comp_shfl_up<NV>(inc, delta * LG);
            const bool of = __shfl_up_sync(0xFFFFFFFFu, (int)finc, delta * LG) != 0;
            if (g >= delta) {
                if (!finc) inc = compose<NV>(o, inc);
                finc = finc || of;
            }
        }
    }
    Comp<NV> ex;  // what is open on this group's left, from earlier groups of this step
    bool fex = false;
    comp_identity(ex);
    if (GW > 1) {
        const Comp<NV> up = comp_shfl_up<NV>(inc, LG);
        const bool fup = __shfl_up_sync(0xFFFFFFFFu, (int)finc, LG) != 0;
        if (g > 0) { ex = up; fex = fup; }
    }
    outer = false;
    if (hasb) {
        closing = compose<NV>(fex ? ex : compose<NV>(carry, ex), head);
        outer = !(fex || cflag);
    }
    const Comp<NV> lastc = comp_shfl<NV>(inc, (GW - 1) * LG + l);
    const bool lastf = __shfl_sync(0xFFFFFFFFu, (int)finc, (GW - 1) * LG) != 0;
    carry = lastf ? lastc : compose<NV>(carry, lastc);
    cflag = cflag || lastf;
}

// ------------------------------------------------------------------------------------------
// sgd_chunk_kernel: one CTA per chunk of kChunk consecutive entries of one tile (kSgdWarps warps; 1 today).
//
// A launch covers tiles with pairwise disjoint column blocks: the p tiles of one inner round
// (sweep 0) or the p tiles of one row block (sweep 1).  A tile's entries are sorted by (column,
// row).  Every warp owns kWarpEntries consecutive entries and walks them in passes.  Per pass:
//   1. one lane per entry turns the (prefetched) entry record and G_i into (e, b, row, column);
//      a "boundary" sits before an entry whose column differs from the entry before it (the tile
//      start counts), i.e. at every entry that starts a run;
//   2. the rows a_i of the whole pass, and the scale pair of every column whose run starts in the
//      pass, are gathered into shared memory with cp.async: one memory latency per pass;
//   3. each lane group walks S consecutive entries sequentially.  The piece before its first
//      boundary becomes its head; a run that starts and ends inside the group is applied on the
//      spot from the prefetched scale pair (stores and adds nobody waits for);
//   4. scan_step joins the pieces across the lane groups of the warp; the runs that end at the
//      groups' first boundaries are applied together.
// Runs that cross warps are joined by the same scan run by warp 0 over the warps' results (shared
// memory); runs that cross chunks by the same scan run by whichever chunk of the tile finishes
// last, over per-chunk records in global scratch (one counter per tile; no CTA waits for another).
//
// Column state: in a direct tile it is the scaled (w_j, v_j).  In a tail tile (sweep 1, r > c) it
// is a per-column composite T_j in the same scaled form, identity at the start of the epoch and
// applied to (w_j, v_j) by sgd_finalize_* after the sweep.  The sweep visits row blocks p-1, .., 0,
// so for column block c the tail tiles (r = p-1 .. c+1) and then the direct tiles (r = c .. 0) are
// each met in the stratified order of the rounds, and "T_j after v_j" restores the order
// c, .., 0, p-1, .., c+1.  Meanwhile all entries of a row meet in one launch, so (a_i, G_i) come
// from L2 after first touch.
// ------------------------------------------------------------------------------------------
struct SgdChunkArgs {
    const int64_t *tile_ptr;   // p*p+1, tiles in sweep order (slots)
    const uint2 *ent;          // packed: {(i_local << jbits) | j_local, bits of x}; wide: {i_local, j_local}
    const float *xw;           // wide layout only: x per entry
    const int64_t *row_start;  // p+1
    const int32_t *col_start;  // p+1
    const float *A;            // n * Kp
    const float *G;            // n
    float *w;                  // d        u-part of w_j
    float *V;                  // d * Kp   u-part of v_j
    float4 *S;                 // d        {sigma of v_j, sigma of w_j, -, -}
    float *Tw;                 // d        u-part of the w offset of T_j      (sweep 1)
    float *Tb;                 // d * Kp   u-part of the v offset of T_j      (sweep 1)
    float4 *TS;                // d        {D, Dw, -, -} of T_j               (sweep 1)
    const int4 *chunk_map;     // per chunk, in sweep order: {tile slot, chunk index inside the tile, number
                               // of earlier non-empty tiles of the same column block, -}
    float *records;            // chunk_record_floats(Kp) floats per chunk
    int *tile_count;           // p*p, all zero between launches
    int *sync;                 // sync_words(p) ints: ticket counter (zero at launch), error flag, finished
                               // tiles per column block (zero at the first launch of a sweep, kept between
                               // the launches of one sweep)
    int p, jbits, sweep;
    int chunk_base;            // first chunk of this launch in chunk_map (a launch may cover a range of rounds)
    int chunk_len;             // entries per chunk, <= kChunk: short chunks for small data sets, whose epoch is a
                               // chain of dependent tiles and is as long as p times the time one tile takes
    float h, lambda_w, lambda_v;
};

template <int LG, int NV, bool WIDE>
__global__ void __launch_bounds__(kSgdThreads, sgd_min_ctas(LG, NV)) sgd_chunk_kernel(const SgdChunkArgs a) {
    typedef SgdSmem<LG, NV> L;
    constexpr int GW = L::GW, KP4 = L::KP4, PASS = L::PASS, S = L::S;
    constexpr int PP = kWarpEntries / PASS;
    constexpr int EPL = (S + LG - 1) / LG;  // entries a lane holds per pass: lane l of group g holds the
                                            // entries g*S + l*EPL + q of the pass, q < EPL (those below S)
    constexpr int NW = kSgdWarps;
    constexpr int REC4 = chunk_record_floats(4 * KP4) / 4;
    static_assert(PASS * PP == kWarpEntries && S * GW == PASS, "a warp's entries must be whole passes");
    typedef Comp<NV> C;

    extern __shared__ float4 smem4[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane / LG, l = lane % LG;
    float4 *sw = smem4 + warp * L::WARP;
    float4 *s_item = sw + L::ITEMS + g * L::ITEM_STRIDE;
    float4 *s_rows = sw + L::ROWS + g * L::ROW_STRIDE;
    float4 *s_scale_all = sw + L::SCALES;
    float4 *s_scale = s_scale_all + g * L::ITEM_STRIDE;
    float4 *s_wpiece = smem4 + L::WPIECE;  // [warp][head/tail][KP4+1]
    float4 *s_cpiece = smem4 + L::CPIECE;
    int *s_wflag = reinterpret_cast<int *>(smem4 + L::TOTAL);

    // Chunks are handed out in sweep order by a ticket counter, so a CTA that holds a ticket knows that
    // every earlier chunk has been taken by a CTA that is running or done: waiting for earlier tiles of
    // the same column block can therefore not deadlock.  The wait is bounded all the same; on a
    // time-out the error flag makes every CTA leave and the host reports the failure.
    __shared__ int s_ticket, s_go;
    if (tid == 0) s_ticket = atomicAdd(a.sync + kSyncTicket, 1);
    __syncthreads();
    const int chunk = a.chunk_base + s_ticket;
    const int4 cm = a.chunk_map[chunk];
    const int64_t t = cm.x;  // tile slot: position of the tile in sweep order (the device order of tiles)
    int r, c;
    if (a.sweep == 1) { r = a.p - 1 - (int)(t / a.p); c = (int)(t % a.p); }
    else { r = (int)(t % a.p); c = (r + (int)(t / a.p)) % a.p; }
    const bool tail_mode = a.sweep == 1 && r > c;
    const int64_t tb = a.tile_ptr[t], te = a.tile_ptr[t + 1];
    const int64_t cb = tb + (int64_t)cm.y * a.chunk_len;
    const int64_t ce = (cb + a.chunk_len < te) ? cb + a.chunk_len : te;
    const int64_t wb = cb + (int64_t)warp * kWarpEntries;
    const int64_t we = (wb + kWarpEntries < ce) ? wb + kWarpEntries : ce;
    const int64_t row0 = a.row_start[r];
    const int64_t col0 = a.col_start[c];
    const uint32_t jmask = a.jbits >= 32 ? 0xFFFFFFFFu : ((1u << a.jbits) - 1u);
    const float ew = a.h * a.lambda_w;
    // everything a warp touches is addressed with 32-bit offsets from pointers set up once
    const float4 *A4 = reinterpret_cast<const float4 *>(a.A) + (size_t)row0 * KP4;  // rows of this row block
    const float *Gr = a.G + row0;
    const uint2 *entw = a.ent + wb;                      // this warp's entries
    const float *xww = WIDE ? a.xw + wb : nullptr;
    const int wlen = we > wb ? (int)(we - wb) : 0;
    // the column state this tile acts on (u-parts and scale pairs), shifted to the column block
    float4 *U4 = reinterpret_cast<float4 *>(tail_mode ? a.Tb : a.V) + (size_t)col0 * KP4;
    float *uw = (tail_mode ? a.Tw : a.w) + col0;
    float4 *Sc = (tail_mode ? a.TS : a.S) + col0;

    // column state <- run o column state, given the column's scale pair (lanes of one group)
    auto apply = [&](uint32_t jl, const C &x, float4 sc) {
        const float sg = fmaf(sc.x, x.D, sc.x + x.D);
        const float inv = rcp_fast(1.0f + sg);
#pragma unroll
        for (int v = 0; v < NV; ++v)
            red_add4(U4 + (size_t)jl * KP4 + v * LG + l, x.B[v].x * inv, x.B[v].y * inv, x.B[v].z * inv,
                     x.B[v].w * inv);
        if (l == 0) {
            const float sgw = fmaf(sc.y, x.Dw, sc.y + x.Dw);
            red_add1(uw + jl, x.Bw * rcp_fast(1.0f + sgw));
            Sc[jl] = make_float4(sg, sgw, 0.f, 0.f);
        }
    };
    // the same with the scale pair fetched from L2 (never through L1: another SM wrote it in this launch)
    auto apply_fetch = [&](uint32_t jl, const C &x) {
        if (jl == kNoCol) return;
        apply(jl, x, __ldcg(Sc + jl));
    };

    // ---------------- warp phase ----------------
    C wcarry;  // open run of this warp so far
    comp_identity(wcarry);
    bool wflag = false;  // a boundary has been seen in this warp
    uint32_t last_col = kNoCol;

    // entry records are fetched two passes ahead and G one pass ahead, into registers
    uint2 ent0[EPL], ent1[EPL];
    float xw0[EPL], xw1[EPL], g0[EPL];
    const int slot0 = l * EPL;          // this lane's first entry inside its group's S entries
    const int at0 = g * S + slot0;      // ... and inside the pass
    auto fetch_ent = [&](int pp, uint2 (&e)[EPL], float (&xv)[EPL]) {
#pragma unroll
        for (int q = 0; q < EPL; ++q) {
            const int at = pp * PASS + at0 + q;
            if (slot0 + q < S && at < wlen) {
                e[q] = entw[at];
                if (WIDE) xv[q] = xww[at];
            }
        }
    };
    auto fetch_g = [&](int pp, const uint2 (&e)[EPL], float (&gv)[EPL]) {
#pragma unroll
        for (int q = 0; q < EPL; ++q) {
            const int at = pp * PASS + at0 + q;
            if (slot0 + q < S && at < wlen) gv[q] = __ldg(Gr + (WIDE ? e[q].x : (e[q].x >> a.jbits)));
        }
    };
    fetch_ent(0, ent0, xw0);
    if (PP > 1) fetch_ent(1, ent1, xw1);
    fetch_g(0, ent0, g0);

    // the first fetches are under way; now make sure the earlier tiles of this column block are done
    if (tid == 0) {
        int go = 1;
        const volatile int *done = a.sync + sync_done(c);
        const volatile int *err = a.sync + kSyncError;
        for (int spin = 0; *done < cm.z; ++spin) {
            if (*err != 0 || spin > kSgdSpinLimit) { go = 0; break; }
            __nanosleep(100);
        }
        if (!go) atomicExch(a.sync + kSyncError, 1);
        __threadfence();
        s_go = go;
    }
    __syncthreads();
    if (!s_go) return;
    for (int pp = 0; pp < PP; ++pp) {
        if (pp * PASS >= wlen) break;
        const int cnt = (wlen - pp * PASS) < PASS ? (wlen - pp * PASS) : PASS;
        uint32_t before = kNoCol;  // column of the entry just before this pass, if it is in the tile
        if (pp > 0) before = last_col;
        else if (wb > tb) {
            const uint2 rec = entw[-1];
            before = WIDE ? rec.y : (rec.x & jmask);
        }
        // column of the entry just after this pass when it is known to this warp (its own next
        // pass); otherwise the last run of the pass is left open and closed by a later phase
        uint32_t after = kNoCol;
        const bool after_known = (pp + 1 < PP) && ((pp + 1) * PASS < wlen);
        // 1. items of this pass from the prefetched registers
        uint32_t jq[EPL], ilq[EPL];
        float eq[EPL], bq[EPL];
        bool cont = true;  // every entry this lane holds continues the run that is open at the pass start
#pragma unroll
        for (int q = 0; q < EPL; ++q) {
            jq[q] = kNoCol;
            ilq[q] = 0u;
            eq[q] = 0.f;
            bq[q] = 0.f;
            if (slot0 + q < S && at0 + q < cnt) {
                float x;
                if (WIDE) { ilq[q] = ent0[q].x; jq[q] = ent0[q].y; x = xw0[q]; }
                else { ilq[q] = ent0[q].x >> a.jbits; jq[q] = ent0[q].x & jmask; x = __uint_as_float(ent0[q].y); }
                const float gx = g0[q] * x;
                eq[q] = a.h * (a.lambda_v - gx * x);
                bq[q] = -a.h * gx;
                cont = cont && jq[q] == before;
            }
        }
        // A full pass inside one run (about two thirds of the passes on click-log data, where a few
        // columns hold most entries) has no boundary: nothing is applied and nothing needs the staging
        // in shared memory.  It takes the short way below.
        const bool one_run = cnt == PASS && before != kNoCol && __all_sync(0xFFFFFFFFu, cont);
        if (!one_run) {
#pragma unroll
            for (int q = 0; q < EPL; ++q)
                if (slot0 + q < S && at0 + q < cnt)
                    s_item[slot0 + q] = make_float4(eq[q], bq[q], __uint_as_float(ilq[q]), __uint_as_float(jq[q]));
        }
        // rotate the prefetch registers and start the next fetches
#pragma unroll
        for (int q = 0; q < EPL; ++q) { ent0[q] = ent1[q]; xw0[q] = xw1[q]; }
        if (after_known) after = __shfl_sync(0xFFFFFFFFu, WIDE ? ent0[0].y : (ent0[0].x & jmask), 0);
        if (pp + 1 < PP) fetch_g(pp + 1, ent0, g0);
        if (pp + 2 < PP) fetch_ent(pp + 2, ent1, xw1);
        if (one_run) {
            // Each lane group composes its S entries, rows a_i straight from global memory to registers
            // (entry u of the group sits in lane u / EPL of the group), then the groups' composites are
            // joined in order and appended to the open run.
            constexpr int UB = (S * NV <= 8) ? S : (8 / NV < 1 ? 1 : 8 / NV);  // rows requested before the first is used
            C cur;
            comp_identity(cur);
#pragma unroll
            for (int u0 = 0; u0 < S; u0 += UB) {
                float4 av[UB][NV];
                float eu[UB], bu[UB];
#pragma unroll
                for (int u = 0; u < UB; ++u) {
                    const int src = (u0 + u) / EPL, reg = (u0 + u) % EPL;
                    const uint32_t il = __shfl_sync(0xFFFFFFFFu, ilq[reg], src, LG);
                    eu[u] = __shfl_sync(0xFFFFFFFFu, eq[reg], src, LG);
                    bu[u] = __shfl_sync(0xFFFFFFFFu, bq[reg], src, LG);
#pragma unroll
                    for (int v = 0; v < NV; ++v) av[u][v] = __ldcg(A4 + (size_t)il * KP4 + v * LG + l);
                }
#pragma unroll
                for (int u = 0; u < UB; ++u) {
                    const float e = eu[u], b = bu[u];
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
            if (GW > 1) {
#pragma unroll
                for (int delta = 1; delta < GW; delta <<= 1) {
                    const C o = comp_shfl_down<NV>(cur, delta * LG);
                    if ((g & (2 * delta - 1)) == 0) cur = compose<NV>(cur, o);
                }
                cur = comp_shfl<NV>(cur, l);  // group 0 holds the whole pass
            }
            wcarry = compose<NV>(wcarry, cur);
            last_col = before;
            continue;
        }
        //    scale pairs of the columns whose runs end in this pass (an entry ends a run when the
        //    next entry has another column)
        {
            // the entry after this lane's last one is held by the next lane that holds entries
            const int next_lane = (slot0 + EPL < S) ? lane + 1 : (g + 1) * LG;
            const uint32_t first_of_next = __shfl_sync(0xFFFFFFFFu, jq[0], next_lane & 31);
#pragma unroll
            for (int q = 0; q < EPL; ++q) {
                const int at = at0 + q;
                const uint32_t nextcol = (q + 1 < EPL && slot0 + q + 1 < S) ? jq[q + 1 < EPL ? q + 1 : q] : first_of_next;
                bool ends;
                if (at + 1 < cnt) ends = nextcol != jq[q];
                else ends = after_known && after != jq[q];
                if (slot0 + q < S && at < cnt && ends) cp_async16(s_scale + slot0 + q, Sc + jq[q]);
            }
        }
        __syncwarp();
        // 2. gather the rows a_i of the pass
#pragma unroll
        for (int it = 0; it < PASS * KP4 / 32; ++it) {
            const int idx = lane + 32 * it;
            const int at = idx / KP4, part = idx % KP4;
            if (at < cnt) {
                const uint32_t il = __float_as_uint(sw[L::ITEMS + (at / S) * L::ITEM_STRIDE + (at % S)].z);
                cp_async16(sw + L::ROWS + (at / S) * L::ROW_STRIDE + (at % S) * KP4 + part, A4 + (size_t)il * KP4 + part);
            }
        }
        {
            const int at = cnt - 1;
            last_col = __float_as_uint(sw[L::ITEMS + (at / S) * L::ITEM_STRIDE + (at % S)].w);
        }
        cp_async_wait_all();
        __syncwarp();

        // 3. sequential walk of each lane group.  A run that ends before entry u is parked in the
        //    slots of entry u-1, which have been consumed: offsets over its row, {D, Dw, Bw} over
        //    its item.  The first such run of the group is its head piece; the others started inside
        //    the group and are marked in `emask` for step 5.
        const int lo = g * S;
        const int len = (lo >= cnt) ? 0 : ((cnt - lo < S) ? cnt - lo : S);
        bool hasb = false;
        int head_pos = -1;
        uint32_t headcol = kNoCol, emask = 0;
        C cur;
        comp_identity(cur);
        if (len > 0) {
            uint32_t prevj = (lo == 0) ? before
                                       : __float_as_uint(sw[L::ITEMS + (g - 1) * L::ITEM_STRIDE + (S - 1)].w);
#pragma unroll
            for (int u = 0; u < S; ++u) {
                if (u < len) {
                    const float4 it = s_item[u];
                    float4 av[NV];
#pragma unroll
                    for (int v = 0; v < NV; ++v) av[v] = s_rows[u * KP4 + v * LG + l];
                    const uint32_t jl = __float_as_uint(it.w);
                    if (jl != prevj) {  // boundary before this entry
                        if (u > 0) {
#pragma unroll
                            for (int v = 0; v < NV; ++v) s_rows[(u - 1) * KP4 + v * LG + l] = cur.B[v];
                            if (l == 0) s_item[u - 1] = make_float4(cur.D, cur.Dw, cur.Bw, __uint_as_float(prevj));
                        }
                        if (!hasb) { hasb = true; headcol = prevj; head_pos = u - 1; }
                        else emask |= 1u << (u - 1);
                        comp_identity(cur);
                        prevj = jl;
                    }
                    const float e = it.x, b = it.y;
                    cur.D = fmaf(-e, cur.D, cur.D - e);
                    cur.Dw = fmaf(-ew, cur.Dw, cur.Dw - ew);
                    cur.Bw = fmaf(-ew, cur.Bw, cur.Bw + b);
#pragma unroll
                    for (int v = 0; v < NV; ++v) {
                        cur.B[v].x = fmaf(b, av[v].x, fmaf(-e, cur.B[v].x, cur.B[v].x));
                        cur.B[v].y = fmaf(b, av[v].y, fmaf(-e, cur.B[v].y, cur.B[v].y));
                        cur.B[v].z = fmaf(b, av[v].z, fmaf(-e, cur.B[v].z, cur.B[v].z));
                        cur.B[v].w = fmaf(b, av[v].w, fmaf(-e, cur.B[v].w, cur.B[v].w));
                    }
                }
            }
        }
        // 4. join the pieces across the lane groups
        C head, closing;
        comp_identity(head);
        __syncwarp();
        if (hasb && head_pos >= 0) {
#pragma unroll
            for (int v = 0; v < NV; ++v) head.B[v] = s_rows[head_pos * KP4 + v * LG + l];
            const float4 hd = s_item[head_pos];
            head.D = hd.x; head.Dw = hd.y; head.Bw = hd.z;
        }
        bool outer;
        scan_step<LG, NV>(hasb, head, cur, wcarry, wflag, closing, outer);
        if (hasb) {
            if (outer) {
                comp_store<LG, NV>(s_wpiece + (warp * 2 + 0) * (KP4 + 1), closing, headcol, l);
            } else if (headcol != kNoCol) {
                // the run ended at entry lo + head_pos of this pass if that is >= 0 (its scale pair
                // was prefetched there), else in an earlier pass
                const int pos = lo + head_pos;
                if (pos >= 0) apply(headcol, closing, s_scale_all[(pos / S) * L::ITEM_STRIDE + (pos % S)]);
                else apply_fetch(headcol, closing);
            }
        }
        // 5. apply the runs parked in step 3, all lane groups side by side
        while (__any_sync(0xFFFFFFFFu, emask != 0)) {
            if (emask != 0) {
                const int pos = __ffs(emask) - 1;
                emask &= emask - 1;
                C x;
#pragma unroll
                for (int v = 0; v < NV; ++v) x.B[v] = s_rows[pos * KP4 + v * LG + l];
                const float4 hd = s_item[pos];
                x.D = hd.x; x.Dw = hd.y; x.Bw = hd.z;
                apply(__float_as_uint(hd.w), x, s_scale[pos]);
            }
        }
        __syncwarp();
    }
    if (lane < LG) {
        comp_store<LG, NV>(s_wpiece + (warp * 2 + 1) * (KP4 + 1), wcarry, last_col, l);
        if (l == 0) s_wflag[warp] = wflag ? 1 : 0;
    }
    // with several warps, each orders its own state updates before the tile's completion signal below
    // (warp 0 fences again before it signals)
    if (NW > 1) __threadfence();
    __syncthreads();
    if (warp != 0) return;

    // ---------------- chunk phase: warp 0 joins the warps ----------------
    const int nchunks = (int)((te - tb + a.chunk_len - 1) / a.chunk_len);
    C ccarry;
    comp_identity(ccarry);
    bool cflag = false;
    uint32_t ctailcol = kNoCol;
    for (int w0 = 0; w0 < NW; w0 += GW) {
        const int w = w0 + g;
        bool hasb = false;
        uint32_t headcol = kNoCol;
        C head, cur, closing;
        comp_identity(head);
        comp_identity(cur);
        if (w < NW) {
            comp_load<LG, NV>(s_wpiece + (w * 2 + 1) * (KP4 + 1), cur, l);
            if (s_wflag[w]) {
                hasb = true;
                headcol = comp_load<LG, NV>(s_wpiece + (w * 2 + 0) * (KP4 + 1), head, l);
            }
        }
        bool outer;
        scan_step<LG, NV>(hasb, head, cur, ccarry, cflag, closing, outer);
        if (hasb) {
            if (outer) comp_store<LG, NV>(s_cpiece, closing, headcol, l);
            else apply_fetch(headcol, closing);
        }
    }
    for (int w = 0; w < NW; ++w) {
        const uint32_t tc = __float_as_uint(s_wpiece[(w * 2 + 1) * (KP4 + 1) + KP4].w);
        if (tc != kNoCol) ctailcol = tc;
    }
    __syncwarp();
    if (nchunks == 1) {
        // the tile starts and ends in this chunk: its head piece belongs to no column, and the end
        // of the tile closes the run that is still open
        if (g == 0) apply_fetch(ctailcol, ccarry);
        __threadfence();
        __syncwarp();
        if (lane == 0) atomicAdd(a.sync + sync_done(c), 1);  // this tile of column block c is done
        return;
    }
    {
        float4 *rec4 = reinterpret_cast<float4 *>(a.records) + (size_t)chunk * REC4;
        if (lane < LG) {
            if (l == 0) {
                rec4[0] = cflag ? s_cpiece[KP4] : make_float4(0.f, 0.f, 0.f, __uint_as_float(kNoCol));
                rec4[1] = make_float4(ccarry.D, ccarry.Dw, ccarry.Bw, __uint_as_float(ctailcol));
                rec4[2] = make_float4(__uint_as_float(cflag ? 1u : 0u), 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int v = 0; v < NV; ++v) {
                rec4[3 + v * LG + l] = cflag ? s_cpiece[v * LG + l] : make_float4(0.f, 0.f, 0.f, 0.f);
                rec4[3 + KP4 + v * LG + l] = ccarry.B[v];
            }
        }
    }

    // ---------------- tile phase: the chunk that finishes last joins the chunks ----------------
    __threadfence();
    __syncwarp();
    int last = 0;
    if (lane == 0) last = (atomicAdd(a.tile_count + t, 1) == nchunks - 1) ? 1 : 0;
    last = __shfl_sync(0xFFFFFFFFu, last, 0);
    if (!last) return;
    __threadfence();
    const float4 *base4 = reinterpret_cast<const float4 *>(a.records) + ((size_t)chunk - (size_t)cm.y) * REC4;
    C tcarry;
    comp_identity(tcarry);
    bool tflag = false;
    // The next tile of this column block waits for this loop, so the records (and the scale pair of each
    // record's head column) of step k0 + GW are fetched before step k0 is scanned: one memory latency
    // for the whole loop instead of two per step.
    struct Rec {
        bool hasb;
        uint32_t headcol;
        C head, cur;
        float4 sc;
    };
    auto load_rec = [&](int k, Rec &x) {
        x.hasb = false;
        x.headcol = kNoCol;
        comp_identity(x.head);
        comp_identity(x.cur);
        x.sc = make_float4(0.f, 0.f, 0.f, 0.f);
        if (k < nchunks) {
            const float4 *rec4 = base4 + (size_t)k * REC4;
            const float4 hh = __ldcg(rec4 + 0);
            const float4 th = __ldcg(rec4 + 1);
            x.hasb = __float_as_uint(__ldcg(rec4 + 2).x) != 0u;
            x.head.D = hh.x; x.head.Dw = hh.y; x.head.Bw = hh.z;
            x.headcol = __float_as_uint(hh.w);
            x.cur.D = th.x; x.cur.Dw = th.y; x.cur.Bw = th.z;
#pragma unroll
            for (int v = 0; v < NV; ++v) {
                x.head.B[v] = __ldcg(rec4 + 3 + v * LG + l);
                x.cur.B[v] = __ldcg(rec4 + 3 + KP4 + v * LG + l);
            }
            // no chunk of this tile applies to a head column: its run is still open until this loop
            if (x.hasb && x.headcol != kNoCol) x.sc = __ldcg(Sc + x.headcol);
        }
    };
    Rec nxt;
    load_rec(g, nxt);
    for (int k0 = 0; k0 < nchunks; k0 += GW) {
        const Rec now = nxt;
        if (k0 + GW < nchunks) load_rec(k0 + GW + g, nxt);
        C closing;
        bool outer;
        scan_step<LG, NV>(now.hasb, now.head, now.cur, tcarry, tflag, closing, outer);
        // the first boundary of a tile is its start, whose head column is kNoCol: nothing to apply
        if (now.hasb && now.headcol != kNoCol) apply(now.headcol, closing, now.sc);
    }
    const uint32_t ttailcol = __float_as_uint(__ldcg(base4 + (size_t)(nchunks - 1) * REC4 + 1).w);
    if (g == 0) apply_fetch(ttailcol, tcarry);  // the end of the tile closes the last run
    __threadfence();
    __syncwarp();
    if (lane == 0) {
        a.tile_count[t] = 0;
        atomicAdd(a.sync + sync_done(c), 1);  // this tile of column block c is done
    }
}

// End of the SGD phase: back from the scaled state to plain parameters,
//     v_j <- (1 + D_T) ((1 + sigma_j) u_j + ub_j),   w_j likewise,
// where T_j = (D_T, ub_j) is the tail composite (identity unless the launch order was the row-block
// sweep), and reset of the scale pairs and of T_j.  Two kernels because the first reads the scale
// pairs that the second clears.
__global__ void __launch_bounds__(kThreads) sgd_finalize_v_kernel(float *V, float *Tb, const float4 *S,
                                                                  const float4 *TS, int64_t d, int kp4) {
    const int64_t total = d * kp4;
    float4 *V4 = reinterpret_cast<float4 *>(V);
    float4 *Tb4 = reinterpret_cast<float4 *>(Tb);
    for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < total; i += (int64_t)gridDim.x * kThreads) {
        const int64_t j = i / kp4;
        const float sg = S[j].x;
        float4 y = V4[i];
        y.x = fmaf(sg, y.x, y.x); y.y = fmaf(sg, y.y, y.y); y.z = fmaf(sg, y.z, y.z); y.w = fmaf(sg, y.w, y.w);
        if (Tb != nullptr) {
            const float dt = TS[j].x;
            const float4 b = Tb4[i];
            y.x += b.x; y.y += b.y; y.z += b.z; y.w += b.w;
            y.x = fmaf(dt, y.x, y.x); y.y = fmaf(dt, y.y, y.y); y.z = fmaf(dt, y.z, y.z); y.w = fmaf(dt, y.w, y.w);
            Tb4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        V4[i] = y;
    }
}
__global__ void __launch_bounds__(kThreads) sgd_finalize_w_kernel(float *w, float *Tw, float4 *S, float4 *TS, int64_t d) {
    for (int64_t j = (int64_t)blockIdx.x * kThreads + threadIdx.x; j < d; j += (int64_t)gridDim.x * kThreads) {
        float wj = w[j];
        wj = fmaf(S[j].y, wj, wj);
        S[j] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (Tw != nullptr) {
            wj += Tw[j];
            wj = fmaf(TS[j].y, wj, wj);
            Tw[j] = 0.f;
            TS[j] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        w[j] = wj;
    }
}

}  // namespace dsf
