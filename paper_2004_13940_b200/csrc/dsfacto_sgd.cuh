// Stratum SGD kernels of the DS-FACTO epoch for sm_100a.
//
// With G_i and a_i frozen, one stored entry (i,j,x) maps (w_j, v_j) affinely
// (eqs. (dsfacto_sgdupdatew), (dsfacto_sgdupdatev) regrouped):
//     v_j <- (1 - e) v_j + b a_i,   e = h (lambda_v - G_i x^2),  b = -h G_i x,  h = eta / n
//     w_j <- (1 - ew) w_j + b,      ew = h lambda_w
// The factor (1 - e) is the same for every k.  Writing P_t for the product of the factors of a
// column's entries 1..t (in the stratified order), the entries t = 1..T of a column give
//     v_T = P_T ( v_0 + sum_t (b_t / P_t) a_{i_t} ),
// so only the scalar P depends on the order; the K-wide part is a weighted sum of rows of A whose
// pieces join by addition.  P is kept as D = P - 1 (the per-entry shrink e is often below half an
// ulp of 1), pieces combine as D1 + D2 + D1 D2.  For w the factor is the constant (1 - ew), so its
// product over m entries is (1 - ew)^m and only the count m is carried.
//
// During the SGD phase the column state is held in scaled form, v_j = (1 + sigma_j) u_j and
// w_j = (1 - ew)^{m_j} uw_j with sigma_j = 0, m_j = 0 at the start of the phase.  A run of entries of
// column j starts its products from the column's own scale, P_0 = 1 + sigma_j and m_0 = m_j, so its sums
// U = sum_t (b_t / P_t) a_i and W = sum_t b_t (1 - ew)^{-m_t} need no scaling when they are applied:
//     u_j += U,  uw_j += W,  sigma_j <- P_T - 1,  m_j <- m_T.
// The K-wide part is an add that nobody waits for (red.global.add; every column receives at most one
// per tile and tiles of a column block are ordered, so the result does not depend on timing).  A slice of
// a run that is longer than a chunk cannot know the column's scale yet; it starts from P_0 = 1, m_0 = 0, and
// the slice that joins the run's slices scales the joined sums by 1 / (1 + sigma_j) and (1 - ew)^{-m_j}.
// sgd_finalize_* turns the state back into plain (w, V) at the end of the phase.  The scaled form
// breaks down only if some 1 + sigma reaches zero, i.e. a step so large that a run wipes its column;
// the parameters then become non-finite and the epoch reports divergence.
#pragma once
#include <type_traits>
#include "dsfacto_common.cuh"

namespace dsf {

constexpr int kSgdWarps = 1;                      // warps per CTA; every warp works on its own chunks
constexpr int kSgdThreads = 32 * kSgdWarps;
constexpr int kChunkMax = 4096;                   // most entries a chunk may hold
constexpr int kEntBlockMax = 256;                 // most entries of one block of the entry ring (a multiple of 32)
constexpr int kEntBlockDefault = 192;             // entries per block unless the chunks are shorter
constexpr int kEntBlockWide = 96;                 // ... for factor rows of 256 bytes and more
constexpr int kEntSlots = 3;                      // blocks the entry ring of a warp holds
constexpr int kSgdSpinLimit = 1 << 22;            // polls (200 ns of sleep plus a read from L2 each) before a dependency wait gives up
constexpr int kCopySpinLimit = 1 << 24;           // polls before the wait for a bulk copy into shared memory gives up
constexpr int kTicketStop = 0x40000000;           // ticket counter value that makes every warp leave
// Words of the launch's synchronisation array.  The ticket counter takes one atomic per chunk and the
// progress counters are polled by waiting warps, so every word sits in a 128-byte line of its own.
constexpr int kSyncStride = 32;                   // ints between two words
constexpr int kSyncTicket = 0;                    // next chunk to hand out
constexpr int kSyncError = kSyncStride;           // set when a wait ran out (1: earlier tile, 2: bulk copy, 3: debug check)
__host__ __device__ constexpr size_t sync_done(int c) { return (size_t)(2 + c) * kSyncStride; }  // finished chunks of column block c
__host__ __device__ constexpr size_t sync_words(int p) { return (size_t)(2 + p) * kSyncStride; }

// One unit of work of the sweep: a range of consecutive entries of one tile (entries of a tile are
// sorted by (column, row)).  Either whole runs (all entries of a column inside the tile), or a slice
// of one run that is longer than a chunk.  Built on the host when the tiles are bucketed.
struct ChunkDesc {
    int64_t ent_off;   // first entry in the entry array
    int32_t len;       // entries, 1 .. chunk length
    int32_t flags;     // kChunkSlice: slice of a long run; kChunkTail: the tile acts on the tail composite
    int32_t row0;      // first row of the tile's row block
    int32_t col0;      // first column of the tile's column block
    int32_t cblock;    // column block (index of its progress counter)
    int32_t need;      // chunks of the earlier tiles of that column block, in sweep order
    int32_t tile;      // tile slot
    int32_t nchunks;   // chunks of the tile
    int32_t run_id;    // slice: index of the long run (its join counter)
    int32_t slice;     // slice: number of this slice inside the run
    int32_t nslices;   // slice: slices of the run
    int32_t rec0;      // slice: record index of slice 0 of the run
    int32_t jl;        // slice: local column of the run
    int32_t pad;
};
static_assert(sizeof(ChunkDesc) == 64, "a chunk descriptor is 16 ints");
enum { kChunkSlice = 1, kChunkTail = 2 };

// lane layout and shared-memory staging of one warp
template <int LG, int NV>
struct SgdCfg {
    static constexpr int GW = 32 / LG;               // lane groups per warp = rows worked on side by side
    static constexpr int KP4 = LG * NV;              // float4s per factor row
    // rows of A gathered per stage: a whole pass for rows up to 128 bytes, half a pass for wider rows.  A
    // stage has a fixed cost (commit, wait, two warp barriers, the masks of its run starts), so short stages
    // are expensive: on the 400 M-entry workload with 512-byte rows a sweep takes 97 ms with 4-row stages,
    // 42 ms with 8, 26 ms with 16 and 34 ms with 32 (too few resident warps); 1024-byte rows 42 ms with 8,
    // 29 ms with 16; 256-byte rows 16 ms with 16, 20 ms with 32.
    static constexpr int RST = KP4 <= 8 ? 32 : 16;
    static constexpr int SP = 32 / RST;              // stages per 32-entry pass
    static constexpr int NBUF = 2;                   // stages in the ring (three were no faster on any workload)
    static constexpr int PD = NBUF - 1;              // stages requested ahead
    static constexpr int ROW4 = NBUF * RST * KP4;    // float4s of the row ring
    static constexpr int DG = SP == 1 ? PD : 1;      // passes ahead at which G_i and the scale records are requested
};
// entries one slot of the entry ring holds: a block of block_len entries, the four entries before it (a block
// that is not the first of its chunk brings the entry before its first one along) and the rounding of the
// copy's start and end to multiples of 4 entries
__host__ __device__ constexpr int sgd_ecap(int block_len) { return (block_len + 12 + 3) & ~3; }
template <int LG, int NV>
__host__ __device__ constexpr size_t sgd_warp_smem(bool wide, int block_len) {
    return (size_t)SgdCfg<LG, NV>::ROW4 * 16 + 32 * 8 + 32 * 4 + 40 * 4 + 32 +
           (size_t)kEntSlots * sgd_ecap(block_len) * (wide ? 12 : 8);
}
// floats of the record a slice of a long run leaves: {D, m, W, -} and the K-wide sum
__host__ __device__ constexpr int slice_record_floats(int Kp) { return 4 + Kp; }

__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gmem_src) {
    const unsigned s = (unsigned)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(s), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }
// fire-and-forget adds into global memory
__device__ __forceinline__ void red_add4(float4 *p, float x, float y, float z, float w) {
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(x), "f"(y), "f"(z), "f"(w) : "memory");
}
__device__ __forceinline__ void red_add1(float *p, float x) {
    asm volatile("red.global.add.f32 [%0], %1;" ::"l"(p), "f"(x) : "memory");
}
// 1 / x and 2^x by the special-function unit alone (within a unit or two in the last place): both scale
// an increment, so a correctly rounded result would buy nothing but instructions
__device__ __forceinline__ float rcp_fast(float x) {
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}
__device__ __forceinline__ float ex2_fast(float x) {
    float r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}
__device__ __forceinline__ int ld_acquire(const int *p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
// ---- mbarrier + bulk copy global -> shared (the entry records of a chunk arrive with one instruction) ----
__device__ __forceinline__ void mbar_init(uint64_t *bar, int count) {
    const unsigned s = (unsigned)__cvta_generic_to_shared(bar);
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(s), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, unsigned bytes) {
    const unsigned s = (unsigned)__cvta_generic_to_shared(bar);
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(s), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, unsigned parity) {
    const unsigned s = (unsigned)__cvta_generic_to_shared(bar);
    unsigned ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok)
        : "r"(s), "r"(parity)
        : "memory");
    return ok != 0;
}
// source and destination 16-byte aligned, bytes a multiple of 16
__device__ __forceinline__ void bulk_copy_g2s(void *smem_dst, const void *gmem_src, unsigned bytes, uint64_t *bar) {
    const unsigned d = (unsigned)__cvta_generic_to_shared(smem_dst);
    const unsigned b = (unsigned)__cvta_generic_to_shared(bar);
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(d),
                 "l"(gmem_src), "r"(bytes), "r"(b)
                 : "memory");
}

struct SgdArgs {
    const ChunkDesc *desc;     // chunks of this launch, in sweep order
    int nchunks;
    const uint2 *ent;          // packed: {(i_local << jbits) | j_local, bits of x}; wide: {i_local, j_local}
    const float *xw;           // wide layout only: x per entry
    const float *A;            // n * Kp
    const float *G;            // n
    float *w;                  // d        uw_j
    float *V;                  // d * Kp   u_j
    float4 *S;                 // d        {sigma_j, m_j (int bits), -, -} (16 bytes: fetched with one cp.async.cg)
    float *Tw;                 // d        the same three for the tail composite T_j (row-block sweep)
    float *Tb;                 // d * Kp
    float4 *TS;                // d
    float *records;            // slice_record_floats(Kp) floats per slice of a long run
    int *run_count;            // one per long run, all zero between launches
    int *sync;                 // sync_words(p) ints: ticket counter (zero at launch), error word, finished chunks
                               // per column block (zero at the first launch of a sweep, kept between the
                               // launches of one sweep)
    int64_t n, d;              // rows and columns of the data set (checks of the debug build)
    int jbits;
    int chunk_len;             // longest chunk of the plan
    int block_len;             // entries per block of the entry ring: a multiple of 32, at most kEntBlockMax
    int spin_limit;            // polls before the wait for an earlier tile gives up
    float h, lambda_v;
    float kappa_w;             // -log2(1 - ew): (1 - ew)^{-m} = 2^(m kappa_w)
};

#ifdef DSFACTO_DEBUG
// bounds-checked build: a failed check records its code and the offending value, and the access is skipped
#define DSF_CHECK(cond, code, value)                                    \
    do {                                                                \
        if (!(cond)) {                                                  \
            if (atomicCAS(a.sync + kSyncError, 0, 3) == 0) {            \
                a.sync[kSyncError + 1] = (code);                        \
                a.sync[kSyncError + 2] = (int)(value);                  \
            }                                                           \
        }                                                               \
    } while (0)
#define DSF_OK(cond) (cond)
#else
#define DSF_CHECK(cond, code, value) do { } while (0)
#define DSF_OK(cond) true
#endif

// ------------------------------------------------------------------------------------------
// sgd_sweep_kernel: persistent warps; each takes chunks in sweep order from a ticket counter.
//
// Pipeline of a warp: while chunk n is worked on, the ticket of chunk n+1 is drawn and its descriptor is
// loaded.  Entry records reach shared memory block by block through a ring of three slots (one bulk copy
// per block, completion on the slot's mbarrier): the blocks of the chunk at work two ahead of the passes,
// then the first blocks of chunk n+1, so a chunk may be much longer than a warp's shared memory and its
// fixed cost is spread over thousands of entries.  A chunk is walked in passes of 32 entries, one entry
// per lane for the scalar part:
//   scalar stage   G_i (requested one pass ahead) -> e, b; run boundaries by comparing neighbours;
//                  segmented scan of D = P - 1 over the lanes; coefficient c = b / P and the w
//                  coefficient; for every run that starts in the pass the scale record of its column
//                  (requested one pass ahead).  Results go to shared memory.
//   K-wide stage   the rows a_i of a stage (32 rows for K <= 32, fewer for wider rows; gathered with
//                  cp.async one stage ahead) are added with weight c.  The run that is open at
//                  the start of a stage and the run that is open at its end are spread over all lane
//                  groups (entry u goes to group u mod GW) and the groups keep their partial sums in
//                  registers until the run ends, then a shuffle tree joins them; runs that start and
//                  end inside a stage go to one lane group each.  A finished run is applied at once.
// A slice of a long run has no boundary at all: its sum, product and length go to a record, and the
// slice of the run that finishes last joins the records in order (scalar prefix products first, then a
// weighted sum of the K-wide parts) and applies the run.
//
// Order: a tile may touch column state only after the earlier tiles of its column block are done: one
// counter per column block counts finished chunks (after a fence), and a chunk waits until it has
// reached the number of chunks of the earlier tiles.  Slices do not wait, so they are counted only by
// the slice that joins their run, all at once, after the run has been applied.  Tickets are
// handed out in sweep order, so every chunk a warp may wait for is already held by a warp that is
// running: no deadlock, and no reliance on the order in which CTAs start.  The wait is bounded all
// the same; when it runs out the error word is set, the ticket counter jumps past the end, and every
// warp leaves at its next ticket.
//
// Column state: in a direct tile it is the scaled (w_j, v_j).  In a tail tile (row-block sweep, r > c)
// it is a per-column composite T_j in the same scaled form, identity at the start of the epoch and
// applied to (w_j, v_j) by sgd_finalize_* after the sweep.  The sweep visits row blocks p-1, .., 0,
// so for column block c the tail tiles (r = p-1 .. c+1) and then the direct tiles (r = c .. 0) are
// each met in the stratified order of the rounds, and "T_j after v_j" restores the order
// c, .., 0, p-1, .., c+1.  Meanwhile all entries of a row meet close together in time, so (a_i, G_i)
// come from L2 after first touch.
// ------------------------------------------------------------------------------------------
// (Rows up to 128 bytes: the two copies of the pass loop would take 116 registers; held to 96, a few bytes of
// spills, 21 instead of 17 resident warps: 22.1 -> 20.4 ms per sweep of 1.755 G entries.  Wider rows are
// slower with that cap: 19.3 -> 20.9 ms on 400 M entries with 512-byte rows; they are held to 128 registers, as
// more registers cost more than the few spilled bytes: 190 registers 22.5 ms.)
template <int LG, int NV, bool WIDE>
__global__ void __launch_bounds__(kSgdThreads, (LG * NV <= 8 ? 18 : 16)) sgd_sweep_kernel(const SgdArgs a) {
    typedef SgdCfg<LG, NV> C;
    constexpr int GW = C::GW, KP4 = C::KP4, RST = C::RST, SP = C::SP, NBUF = C::NBUF, PD = C::PD, DG = C::DG;
    constexpr unsigned FULL = 0xFFFFFFFFu;

    extern __shared__ __align__(128) unsigned char smem_raw[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane / LG, l = lane % LG;
    const int EB = a.block_len, PB = a.block_len >> 5;   // entries and passes per block of the entry ring
    const int ecap = sgd_ecap(EB);
    unsigned char *wbase = smem_raw + (size_t)warp * sgd_warp_smem<LG, NV>(WIDE, EB);
    float4 *rowb = reinterpret_cast<float4 *>(wbase);               // ring of row stages
    float2 *pc = reinterpret_cast<float2 *>(rowb + C::ROW4);        // per entry of the pass: {c, cw}
    uint32_t *pcol = reinterpret_cast<uint32_t *>(pc + 32);         // per entry of the pass: local column
    int *segpos = reinterpret_cast<int *>(pcol + 32);               // lane of the k-th run start of the pass (33 used)
    uint64_t *mbar = reinterpret_cast<uint64_t *>(segpos + 40);     // one per slot of the entry ring (4 words reserved)
    uint2 *ebuf = reinterpret_cast<uint2 *>(mbar + 4);              // kEntSlots x ecap entry records
    float *xbuf = reinterpret_cast<float *>(ebuf + kEntSlots * (size_t)ecap);  // wide layout: kEntSlots x ecap values

    if (lane == 0) {
#pragma unroll
        for (int q = 0; q < kEntSlots; ++q) mbar_init(mbar + q, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();

    const float4 *A4 = reinterpret_cast<const float4 *>(a.A);
    const int *dints = reinterpret_cast<const int *>(a.desc);
    const uint32_t jmask = a.jbits >= 32 ? 0xFFFFFFFFu : ((1u << a.jbits) - 1u);
    const unsigned nch = (unsigned)a.nchunks;
    int *err_word = a.sync + kSyncError;

    // ---- helpers of the chunk pipeline ----
    auto take_ticket = [&]() -> int {      // the value is valid in lane 0 only (nobody waits for it here)
        int t = 0;
        if (lane == 0) t = atomicAdd(a.sync + kSyncTicket, 1);
        return t;
    };
    auto load_desc = [&](int tk) -> int {  // lane f < 16 holds field f of the descriptor
        int v = 0;
        if ((unsigned)tk < nch && lane < 16) v = __ldg(dints + (size_t)tk * 16 + lane);
        return v;
    };
    // Entry ring.  The entries of a warp's chunks arrive as a stream of blocks of EB entries (the last block of a
    // chunk may be shorter), each with one bulk copy into the next of kEntSlots slots, so a chunk may be far
    // longer than the shared memory of a warp.  Block b > 0 of a chunk starts four entries early: the entry
    // before its first one (whose column tells whether a run starts there) sits in the same slot.  Stream
    // numbers count the blocks of this warp; q0 is the number of block 0 of the chunk at work.
    int q0 = 0, q_fetch = -1, q_issued = 0;   // block 0 of the chunk; the block the passes read; blocks requested
    int f_slot = 0, i_slot = 0;               // slot of the next block to read / to request
    unsigned parity_bits = 0;                 // bit s: parity the next wait on slot s expects
    int64_t off = 0, off1 = 0;                // first entry of the chunk at work / of the next chunk
    int len = 0, len1 = 0, nb = 0, nb1 = 0;   // their lengths and numbers of blocks
    bool have_next = false;                   // the next chunk's descriptor has arrived
    auto issue_block = [&](int64_t coff, int clen, int b, int slot) {
        const int64_t g0 = coff + (int64_t)b * EB;
        const int blen = clen - b * EB < EB ? clen - b * EB : EB;
        const int64_t a0 = (g0 & ~(int64_t)3) - (b > 0 ? 4 : 0);
        const int cnt4 = (int)(((g0 + blen + 3) & ~(int64_t)3) - a0);
        if (lane == 0) {
            mbar_expect_tx(mbar + slot, (unsigned)cnt4 * (WIDE ? 12u : 8u));
            bulk_copy_g2s(ebuf + (size_t)slot * ecap, a.ent + a0, (unsigned)cnt4 * 8u, mbar + slot);
            if (WIDE) bulk_copy_g2s(xbuf + (size_t)slot * ecap, a.xw + a0, (unsigned)cnt4 * 4u, mbar + slot);
        }
    };
    // requests every block that is known (the rest of the chunk at work, then the next chunk's) and has a free
    // slot: the slots of the blocks before q_fetch are free.  All lanes have read those blocks (callers
    // synchronise the warp first).
    auto pump = [&]() {
        while (q_issued < q_fetch + kEntSlots) {
            const int rel = q_issued - q0;
            if (rel < nb) issue_block(off, len, rel, i_slot);
            else if (have_next && rel - nb < nb1) issue_block(off1, len1, rel - nb, i_slot);
            else break;
            ++q_issued;
            i_slot = (i_slot + 1 == kEntSlots) ? 0 : i_slot + 1;
        }
    };
    auto wait_slot = [&](int slot) -> bool {
        const unsigned parity = (parity_bits >> slot) & 1u;
        parity_bits ^= 1u << slot;
        for (int spin = 0; spin < kCopySpinLimit; ++spin)
            if (mbar_try_wait(mbar + slot, parity)) return true;
        return false;
    };
    auto fail = [&](int code) {
        if (lane == 0) {
            atomicCAS(err_word, 0, code);
            atomicMax(a.sync + kSyncTicket, kTicketStop);
        }
    };
    // Wait until the `need` chunks of the earlier tiles of column block cblock are done.  `seen` is an earlier
    // reading of the counter (lane 0; it only grows), so that a tile that was ready long ago costs no round
    // trip to L2.
    auto wait_dep = [&](int cblock, int need, int seen) -> bool {
        int ok = 1;
        if (lane == 0 && seen < need) {
            const int *done = a.sync + sync_done(cblock);
            for (int spin = 0; ld_acquire(done) < need; ++spin) {
                if (spin >= a.spin_limit || ((spin & 7) == 7 && *(volatile int *)err_word != 0)) { ok = 0; break; }
                __nanosleep(200);
            }
        }
        ok = __shfl_sync(FULL, ok, 0);
        __syncwarp();   // lane 0's acquire comes before the other lanes' reads of the column state
        return ok != 0;
    };

    // ---- prologue of the pipeline ----
    int tk0 = __shfl_sync(FULL, take_ticket(), 0);
    if ((unsigned)tk0 >= nch) return;
    int dc = load_desc(tk0);
    int tk1 = kTicketStop, dn = 0, tk1_raw = 0, dep_seen_next = 0, cb1 = 0;
    int dep_seen = 0;           // lane 0: the progress counter of the chunk's column block, read ahead
    bool dead = false;          // a wait for entry records ran out

    for (;;) {
        // ---- fields of the current chunk ----
        off = ((int64_t)(uint32_t)__shfl_sync(FULL, dc, 0)) | ((int64_t)__shfl_sync(FULL, dc, 1) << 32);
        len = __shfl_sync(FULL, dc, 2);
        nb = (len + EB - 1) / EB;
        have_next = false;
        const int flags = __shfl_sync(FULL, dc, 3);
        const int row0 = __shfl_sync(FULL, dc, 4);
        const int col0 = __shfl_sync(FULL, dc, 5);
        const int cblock = __shfl_sync(FULL, dc, 6);
        const int need = __shfl_sync(FULL, dc, 7);
        const bool is_slice = (flags & kChunkSlice) != 0;
        const bool tail_mode = (flags & kChunkTail) != 0;

        // the ticket of the next chunk is asked for now; its descriptor and entries follow during the passes
        tk1_raw = take_ticket();

        const int shift = (int)(off & 3);
        const uint2 *eb = ebuf;      // entry `at` of the chunk is eb[at] while the passes read its block
        const float *xb = xbuf;
        int f_next_at = 0;           // pass whose entries are the first of the next block
        // the passes move on to the next block of the chunk: its slot is waited for, blocks further on are requested
        auto enter_block = [&]() {
            ++q_fetch;
            const int b = q_fetch - q0;
            __syncwarp();
            pump();
            if (!wait_slot(f_slot)) dead = true;
            const int at0 = shift + (b > 0 ? 4 : 0) - b * EB;
            eb = ebuf + (size_t)f_slot * ecap + at0;
            xb = xbuf + (size_t)f_slot * ecap + at0;
            f_slot = (f_slot + 1 == kEntSlots) ? 0 : f_slot + 1;
            f_next_at += PB;
        };
        const float4 *A4r = A4 + (size_t)row0 * KP4;
        const float *Gr = a.G + row0;
        float4 *U4 = reinterpret_cast<float4 *>(tail_mode ? a.Tb : a.V) + (size_t)col0 * KP4;
        float *uw = (tail_mode ? a.Tw : a.w) + col0;
        float4 *Sc = (tail_mode ? a.TS : a.S) + col0;
        DSF_CHECK(len >= 1 && len <= a.chunk_len, 10, len);

        // adds a finished run's sums to its column (the lanes of one group; sums already carry the column's scale)
        auto flush = [&](uint32_t col, const float4 (&sum)[NV], float sumw) {
            DSF_CHECK((int64_t)col0 + col < a.d, 12, col);
#pragma unroll
            for (int v = 0; v < NV; ++v)
                red_add4(U4 + (size_t)col * KP4 + v * LG + l, sum[v].x, sum[v].y, sum[v].z, sum[v].w);
            if (l == 0) red_add1(uw + col, sumw);
        };
        // sum over the lane groups, in a fixed order; every lane ends with the total
        auto reduce_groups = [&](float4 (&x)[NV], float &xw_) {
#pragma unroll
            for (int o = LG; o < 32; o <<= 1) {
#pragma unroll
                for (int v = 0; v < NV; ++v) {
                    x[v].x += __shfl_xor_sync(FULL, x[v].x, o);
                    x[v].y += __shfl_xor_sync(FULL, x[v].y, o);
                    x[v].z += __shfl_xor_sync(FULL, x[v].z, o);
                    x[v].w += __shfl_xor_sync(FULL, x[v].w, o);
                }
                xw_ += __shfl_xor_sync(FULL, xw_, o);
            }
        };

        bool alive = true;
        if (!is_slice) alive = wait_dep(cblock, need, dep_seen);   // a slice touches column state only when it joins its run
        if (!alive) { fail(1); break; }

        // ---- the chunk ----
        const int npass = (len + 31) >> 5;
        const int nstage = (len + RST - 1) / RST;
        const uint32_t col_init = is_slice ? (uint32_t)__shfl_sync(FULL, dc, 14) : kNoCol;
        float4 acc[NV];   // this lane group's share of the run that is open
        float accw = 0.f;
#pragma unroll
        for (int v = 0; v < NV; ++v) acc[v] = make_float4(0.f, 0.f, 0.f, 0.f);
        bool open_valid = is_slice;          // a run is open (for a slice: the run it belongs to)
        uint32_t open_col = col_init;
        float D_open = 0.f;                  // (scale of the column) x (product of the open run so far) - 1
        int m_open = 0;                      // entries of the column so far, the open run included

        // The passes of the chunk.  Compiled twice: SL = the chunk is a slice, i.e. lies inside one run, so no run
        // starts, no scale record is read or written before the end of the chunk and the K-wide part has no run to
        // close; the other copy handles chunks of whole runs.  Same arithmetic in both.
        auto run_passes = [&](auto slice_tag) {
            constexpr bool SL = decltype(slice_tag)::value;
            // What a pass needs from global memory is requested ahead of time.  Scalars (G_i of every entry, the scale
            // record of every column whose run starts in the pass) come DG passes ahead into a queue of registers;
            // the rows a_i come PD stages ahead with cp.async into the row ring, one commit group per stage.
            float gq[DG], xq[DG];
            uint32_t jq[DG];
            float4 scq[DG];
            uint32_t mq[DG];                     // run starts of the pass as a lane mask
            uint32_t il_c = 0, il_n = 0;         // local rows (one per lane) of the pass at work and of the next one
            auto fetch_pass = [&](int k, float &g_out, float4 &sc_out, uint32_t &mask_out, uint32_t &jl, float &x_out) -> uint32_t {
                const int at = 32 * k + lane;
                bool bnd = false;
                uint32_t il = 0;
                g_out = 0.f; x_out = 0.f; jl = kNoCol;
                if (k == f_next_at) enter_block();
                if (at < len && !dead) {
                    const uint2 rec = eb[at];
                    if (WIDE) { il = rec.x; jl = rec.y; x_out = xb[at]; }
                    else { il = rec.x >> a.jbits; jl = rec.x & jmask; x_out = __uint_as_float(rec.y); }
                    if (!SL) {
                        uint32_t prevj = col_init;
                        if (at > 0) prevj = WIDE ? eb[at - 1].y : (eb[at - 1].x & jmask);
                        bnd = jl != prevj;
                    }
                    DSF_CHECK((int64_t)row0 + il < a.n, 13, il);
                    DSF_CHECK(!SL || jl == col_init, 14, jl);
                    g_out = __ldg(Gr + il);
                    if (!SL && bnd) sc_out = __ldcg(Sc + jl);
                }
                mask_out = SL ? 0u : __ballot_sync(FULL, bnd);
                return il;
            };
            // rows of stage sp of a pass whose local rows are `il`: lane group q fetches the row of entry
            // sp*RST + it*GW + q, 16 bytes per lane (rows past the end of the chunk repeat row 0 of the block)
            int ring_issue = 0, ring_use = 0;     // row ring: slot of the next stage to request / to work on
            auto issue_rows = [&](uint32_t il, int sp) {
                float4 *dst = rowb + ring_issue * (RST * KP4) + g * KP4 + l;
#pragma unroll
                for (int it = 0; it < RST / GW; ++it) {
                    const uint32_t ir = __shfl_sync(FULL, il, sp * RST + it * GW + g);
#pragma unroll
                    for (int v = 0; v < NV; ++v)
                        cp_async16(dst + it * GW * KP4 + v * LG, A4r + (size_t)ir * KP4 + v * LG + l);
                }
                ring_issue = (ring_issue + 1 == NBUF) ? 0 : ring_issue + 1;
            };
#pragma unroll
            for (int q = 0; q < DG; ++q) {
                gq[q] = 0.f; xq[q] = 0.f; jq[q] = kNoCol; mq[q] = 0u; scq[q] = make_float4(0.f, 0.f, 0.f, 0.f);
                uint32_t il = 0;
                if (q < npass) il = fetch_pass(q, gq[q], scq[q], mq[q], jq[q], xq[q]);
                if (q == 0) il_n = il;
                if (SP == 1) {   // a stage is a pass: its rows are requested together with its scalars
                    if (q < nstage) issue_rows(il, 0);
                    cp_async_commit();
                }
            }
            if (SP > 1) {
#pragma unroll
                for (int s = 0; s < PD; ++s) {   // PD <= SP: the first PD stages belong to the first pass
                    if (s < nstage) issue_rows(il_n, s);
                    cp_async_commit();
                }
            }

            for (int k = 0; k < npass; ++k) {
                const int cnt = (len - 32 * k) < 32 ? (len - 32 * k) : 32;
                // this pass's scalars leave the queue; those of pass k + DG are requested
                const float g_c = gq[0], x_c = xq[0];
                const uint32_t jl_c = jq[0];
                const float4 sc_q0 = scq[0];
                const uint32_t mask = SL ? 0u : mq[0];
#pragma unroll
                for (int q = 0; q + 1 < DG; ++q) { gq[q] = gq[q + 1]; xq[q] = xq[q + 1]; jq[q] = jq[q + 1]; scq[q] = scq[q + 1]; mq[q] = mq[q + 1]; }
                il_c = il_n;
                uint32_t il_f = 0;
                if (k + DG < npass) il_f = fetch_pass(k + DG, gq[DG - 1], scq[DG - 1], mq[DG - 1], jq[DG - 1], xq[DG - 1]);
                if (dead) break;
                if (SP > 1) il_n = il_f;

                // ---- scalar stage ----
                float D;
                int m;
                {
                    const bool bnd_c = (mask >> lane) & 1u;
                    float e = 0.f, b = 0.f;
                    const float4 sc_c = sc_q0;
                    if (lane < cnt) {
                        const float gx = g_c * x_c;
                        e = a.h * (a.lambda_v - gx * x_c);
                        b = -a.h * gx;
                    }
                    const uint32_t below = mask & (0xFFFFFFFFu >> (31 - lane));   // run starts at or before this lane
                    const int start = 31 - __clz(below);                              // -1: the run was open before the pass
                    const int lim = below == 0 ? lane : lane - start;                 // earlier lanes of the same run
                    // a run starts from its column's scale, so that the sums need no scaling when they are applied
                    D = bnd_c ? fmaf(sc_c.x, -e, sc_c.x - e) : -e;
#pragma unroll
                    for (int delta = 1; delta < 32; delta <<= 1) {
                        const float up = __shfl_up_sync(FULL, D, delta);
                        if (delta <= lim) D = fmaf(up, D, up + D);
                    }
                    const int mj = SL ? 0 : __shfl_sync(FULL, bnd_c ? __float_as_int(sc_c.y) : 0, start < 0 ? 0 : start);
                    m = lim + 1 + mj;
                    if (below == 0) { D = fmaf(D_open, D, D_open + D); m = lane + 1 + m_open; }
                    const float c = b * rcp_fast(1.0f + D);
                    const float cw = b * ex2_fast((float)m * a.kappa_w);
                    pc[lane] = make_float2(c, cw);
                    if (mask != 0u) {   // only passes with a run start need the rest
                        pcol[lane] = jl_c;
                        if (bnd_c) segpos[__popc(mask & ((1u << lane) - 1u))] = lane;
                        if (lane == 0) segpos[__popc(mask)] = cnt;
                        // a run that ends inside the pass leaves its column's new scale record right here
                        if (lane + 1 < cnt && ((mask >> (lane + 1)) & 1u)) Sc[jl_c] = make_float4(D, __int_as_float(m), 0.f, 0.f);
                    }
                }
                __syncwarp();

                // ---- K-wide stages of this pass ----
#pragma unroll
                for (int sp = 0; sp < SP; ++sp) {
                    const int s = k * SP + sp;
                    if (s >= nstage) break;
                    if (s + PD < nstage) {
                        if (SP == 1) issue_rows(il_f, 0);
                        else if (sp + PD < SP) issue_rows(il_c, sp + PD);
                        else issue_rows(il_n, sp + PD - SP);
                    }
                    cp_async_commit();
                    cp_async_wait<PD>();
                    __syncwarp();
                    const float4 *rb = rowb + ring_use * (RST * KP4);
                    ring_use = (ring_use + 1 == NBUF) ? 0 : ring_use + 1;
                    const int e0 = sp * RST;
                    const int e1 = (e0 + RST < cnt) ? e0 + RST : cnt;
                    // entries [b0, b1) of the pass, entry u to lane group (u - b0) mod GW, into (acc, accw)
                    auto add_spread = [&](int b0, int b1) {
                        for (int u = b0 + g; u < b1; u += GW) {
                            const float2 cf = pc[u];
#pragma unroll
                            for (int v = 0; v < NV; ++v) {
                                const float4 r = rb[(u - e0) * KP4 + v * LG + l];
                                fma4(acc[v], cf.x, r);
                            }
                            accw += cf.y;
                        }
                    };
                    const uint32_t range = (e1 >= 32 ? 0xFFFFFFFFu : ((1u << e1) - 1u)) & ~((1u << e0) - 1u);
                    const uint32_t sub = mask & range;
                    if (sub == 0) {
                        if (e1 - e0 == RST) {
                            // a whole stage inside one run: the common case on click-log data
#pragma unroll
                            for (int q = 0; q < RST / GW; ++q) {
                                const float2 cf = pc[e0 + q * GW + g];
#pragma unroll
                                for (int v = 0; v < NV; ++v) {
                                    const float4 r = rb[(q * GW + g) * KP4 + v * LG + l];
                                    fma4(acc[v], cf.x, r);
                                }
                                accw += cf.y;
                            }
                        } else {
                            add_spread(e0, e1);
                        }
                    } else {
                        const int F = __ffs(sub) - 1, Lb = 31 - __clz(sub);
                        // 1. what is left of the open run, then the open run ends
                        add_spread(e0, F);
                        if (open_valid) {
                            reduce_groups(acc, accw);
                            if (g == 0) {
                                flush(open_col, acc, accw);
                                // (a run that ends inside the pass has left its scale record in the scalar stage)
                                if (F == 0 && l == 0) Sc[open_col] = make_float4(D_open, __int_as_float(m_open), 0.f, 0.f);
                            }
                        }
#pragma unroll
                        for (int v = 0; v < NV; ++v) acc[v] = make_float4(0.f, 0.f, 0.f, 0.f);
                        accw = 0.f;
                        // 2. runs that start and end inside the stage: one lane group each
                        const int i0 = __popc(mask & ((1u << F) - 1u));
                        const int nmid = __popc(sub) - 1;
                        for (int i = g; i < nmid; i += GW) {
                            const int s0 = segpos[i0 + i], s1 = segpos[i0 + i + 1];
                            DSF_CHECK(s0 >= e0 && s1 > s0 && s1 <= e1, 11, s0 * 64 + s1);
                            float4 tmp[NV];
                            float tmpw = 0.f;
#pragma unroll
                            for (int v = 0; v < NV; ++v) tmp[v] = make_float4(0.f, 0.f, 0.f, 0.f);
                            for (int u = s0; u < s1; ++u) {
                                const float2 cf = pc[u];
#pragma unroll
                                for (int v = 0; v < NV; ++v) {
                                    const float4 r = rb[(u - e0) * KP4 + v * LG + l];
                                    fma4(tmp[v], cf.x, r);
                                }
                                tmpw += cf.y;
                            }
                            flush(pcol[s0], tmp, tmpw);
                        }
                        __syncwarp();
                        // 3. the run that is open at the end of the stage
                        add_spread(Lb, e1);
                        open_valid = true;
                        open_col = pcol[Lb];
                    }
                    __syncwarp();
                }
                // the open run up to the end of this pass
                D_open = __shfl_sync(FULL, D, cnt - 1);
                m_open = __shfl_sync(FULL, m, cnt - 1);

                // the next chunk: its descriptor after the first pass, its entries a little later, so that neither
                // request is waited for
                if (k == 0) {
                    tk1 = __shfl_sync(FULL, tk1_raw, 0);
                    dn = load_desc(tk1);
                }
                if (k == (npass > 2 ? 2 : npass - 1) && (unsigned)tk1 < nch) {
                    off1 = ((int64_t)(uint32_t)__shfl_sync(FULL, dn, 0)) | ((int64_t)__shfl_sync(FULL, dn, 1) << 32);
                    len1 = __shfl_sync(FULL, dn, 2);
                    nb1 = (len1 + EB - 1) / EB;
                    cb1 = __shfl_sync(FULL, dn, 6);
                    have_next = true;
                    __syncwarp();
                    pump();   // the next chunk's first blocks, if slots are free; else they follow as the passes move on
                }
            }
        };
        if (is_slice) run_passes(std::integral_constant<bool, true>{});
        else run_passes(std::integral_constant<bool, false>{});
        cp_async_wait<0>();
        if (dead) { fail(2); break; }

        // ---- end of the chunk ----
        reduce_groups(acc, accw);
        int done_add = 1;   // what this chunk adds to the progress counter of its column block
        if (!is_slice) {
            if (open_valid && g == 0) {
                flush(open_col, acc, accw);
                if (l == 0) Sc[open_col] = make_float4(D_open, __int_as_float(m_open), 0.f, 0.f);
            }
        } else {
            const int run_id = __shfl_sync(FULL, dc, 10), slice = __shfl_sync(FULL, dc, 11);
            const int nslices = __shfl_sync(FULL, dc, 12), rec0 = __shfl_sync(FULL, dc, 13);
            float4 *rec4 = reinterpret_cast<float4 *>(a.records) + ((size_t)rec0 + slice) * (KP4 + 1);
            if (g == 0) {
                if (l == 0) rec4[0] = make_float4(D_open, __int_as_float(m_open), accw, 0.f);
#pragma unroll
                for (int v = 0; v < NV; ++v) rec4[1 + v * LG + l] = acc[v];
            }
            __threadfence();
            __syncwarp();
            // Slices do not wait for earlier tiles, so they must not count as progress before their run has been
            // applied: the slice that joins the run reports all of them.
            done_add = 0;
            int last = 0;
            if (lane == 0) last = (atomicAdd(a.run_count + run_id, 1) == nslices - 1) ? 1 : 0;
            last = __shfl_sync(FULL, last, 0);
            if (last) {
                // the slice that finishes last joins the run: scalar prefixes over the slices, then the weighted
                // sum of their K-wide parts, in a fixed order; the column's own scale comes last
                __threadfence();
                if (!wait_dep(cblock, need, dep_seen)) { fail(1); break; }
                const float4 *rbase = reinterpret_cast<const float4 *>(a.records) + (size_t)rec0 * (KP4 + 1);
                float Dp = 0.f, wt = 0.f;
                int mp = 0;
                float4 ut[NV];
#pragma unroll
                for (int v = 0; v < NV; ++v) ut[v] = make_float4(0.f, 0.f, 0.f, 0.f);
                for (int base = 0; base < nslices; base += 32) {
                    const int kx = base + lane;
                    float4 hd = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (kx < nslices) hd = __ldcg(rbase + (size_t)kx * (KP4 + 1));
                    float Di = hd.x;
                    int mi = __float_as_int(hd.y);
#pragma unroll
                    for (int delta = 1; delta < 32; delta <<= 1) {
                        const float upD = __shfl_up_sync(FULL, Di, delta);
                        const int upm = __shfl_up_sync(FULL, mi, delta);
                        if (lane >= delta) { Di = fmaf(upD, Di, upD + Di); mi += upm; }
                    }
                    float Dex = __shfl_up_sync(FULL, Di, 1);
                    int mex = __shfl_up_sync(FULL, mi, 1);
                    if (lane == 0) { Dex = 0.f; mex = 0; }
                    Dex = fmaf(Dp, Dex, Dp + Dex);
                    mex += mp;
                    const float sv = rcp_fast(1.0f + Dex);
                    wt = fmaf(hd.z, ex2_fast((float)mex * a.kappa_w), wt);
#pragma unroll
                    for (int q = 0; q < 32 / GW; ++q) {
                        const int kk = q * GW + g;
                        const float s_ = __shfl_sync(FULL, sv, kk);
                        if (base + kk < nslices) {
#pragma unroll
                            for (int v = 0; v < NV; ++v) {
                                const float4 r = __ldcg(rbase + (size_t)(base + kk) * (KP4 + 1) + 1 + v * LG + l);
                                fma4(ut[v], s_, r);
                            }
                        }
                    }
                    const float Dt = __shfl_sync(FULL, Di, 31);
                    mp += __shfl_sync(FULL, mi, 31);
                    Dp = fmaf(Dp, Dt, Dp + Dt);
                }
                float dummy = 0.f;
                reduce_groups(ut, dummy);
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) wt += __shfl_xor_sync(FULL, wt, o);
                const uint32_t col = (uint32_t)__shfl_sync(FULL, dc, 14);
                if (g == 0) {
                    const float4 sc = __ldcg(Sc + col);
                    const float inv = rcp_fast(1.0f + sc.x);
                    const int mj = __float_as_int(sc.y);
#pragma unroll
                    for (int v = 0; v < NV; ++v) {
                        ut[v].x *= inv; ut[v].y *= inv; ut[v].z *= inv; ut[v].w *= inv;
                    }
                    flush(col, ut, wt * ex2_fast((float)mj * a.kappa_w));
                    if (l == 0) Sc[col] = make_float4(fmaf(sc.x, Dp, sc.x + Dp), __int_as_float(mj + mp), 0.f, 0.f);
                }
                if (lane == 0) a.run_count[run_id] = 0;
                done_add = nslices;
            }
        }
        // This chunk is done: what it wrote becomes visible, then the progress counter of its column block goes
        // up by one (nobody waits for the add).  The first look at the counter of the next chunk's column block
        // is taken just before, so that its round trip overlaps the fence.
        if (lane == 0 && (unsigned)tk1 < nch) dep_seen_next = ld_acquire(a.sync + sync_done(cb1));
        if (done_add > 0) {
            __threadfence();
            __syncwarp();
            if (lane == 0) atomicAdd(a.sync + sync_done(cblock), done_add);
        }

        // ---- next chunk ----
        if ((unsigned)tk1 >= nch) break;
        dc = dn;
        tk0 = tk1;
        dep_seen = dep_seen_next;
        q0 += nb;
    }
    // leaving: nothing may still be on its way into this warp's shared memory (blocks that were requested
    // and never read: only when a wait ran out)
    cp_async_wait<0>();
    while (q_fetch + 1 < q_issued) {
        ++q_fetch;
        wait_slot(f_slot);
        f_slot = (f_slot + 1 == kEntSlots) ? 0 : f_slot + 1;
    }
}

// End of the SGD phase: back from the scaled state to plain parameters,
//     v_j <- (1 + D_T) ((1 + sigma_j) u_j + ub_j),
//     w_j <- (1 - ew)^{m_T} ((1 - ew)^{m_j} uw_j + ubw_j),
// where T_j = (D_T, m_T, ub_j, ubw_j) is the tail composite (identity unless the launch order was the
// row-block sweep), and reset of the scale records and of T_j.  Two kernels because the first reads
// the scale records that the second clears.  log1m_ew = log(1 - ew) in double.
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
__global__ void __launch_bounds__(kThreads) sgd_finalize_w_kernel(float *w, float *Tw, float4 *S, float4 *TS, int64_t d,
                                                                  double log1m_ew) {
    for (int64_t j = (int64_t)blockIdx.x * kThreads + threadIdx.x; j < d; j += (int64_t)gridDim.x * kThreads) {
        float wj = w[j];
        const int mj = __float_as_int(S[j].y);
        if (mj != 0) wj = fmaf((float)expm1((double)mj * log1m_ew), wj, wj);
        S[j] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (Tw != nullptr) {
            wj += Tw[j];
            const int mt = __float_as_int(TS[j].y);
            if (mt != 0) wj = fmaf((float)expm1((double)mt * log1m_ew), wj, wj);
            Tw[j] = 0.f;
            TS[j] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        w[j] = wj;
    }
}

}  // namespace dsf
