// Tile bucketing on the device for large loads (Section 4.2's partition of the data into p x p blocks, the
// order inside a block by (column, row)).  The host path of the library does the same with counting
// sorts per row block; for a data set of a billion entries the host's scatter is slower than the link
// (about 1.2 s against 0.3 s for the CSR arrays alone), so from 2^24 entries on the CSR copy that the
// recompute pass needs anyway is bucketed where it already is:
//   1. tile_keys_kernel: per stored entry (i, j, x) a 32-bit key (slot, phase, local column, row block inside
//      the slot) and a 64-bit payload (local row, bits of x), in CSR order;
//   2. a stable radix sort of the pairs by key (cub::DeviceRadixSort, a library primitive): inside a
//      (tile, column) the CSR order, rows ascending, survives;
//   3. pack_entries_kernel: the 8-byte entry records of the stratum SGD kernel; tile_bounds_kernel: the
//      tile pointers by binary search in the sorted keys;
//   4. plan_tiles_kernel: the chunks of every tile (whole runs packed greedily, long runs cut into
//      slices), the same cuts as plan_tile on the host makes from the column counts.
// With one row block per slot the result is bit for bit what the host path produces.
//
// Merged row blocks.  A column's entries in R consecutive row blocks follow one another in the stratified
// order (row block r is visited right before r - 1), so a slot may hold the tiles (r, c) of R consecutive row
// blocks: inside a column the row blocks descend, rows ascend inside a row block, and a column's run is R
// times as long.  Nothing changes for the stratum SGD kernel (a chunk names the first row of its slot, local
// rows count from there) or for the result's definition; runs are longer, so fewer passes hold a run start
// and fewer sums are applied.  Only the slot that holds the diagonal tile mixes tiles that act on the tail
// composite (r > c, phase 0) with tiles that act on the parameters (phase 1): the phase sorts before the
// column, so the slot lists its tail part first, and no chunk spans both.
#pragma once
#include "dsfacto_common.cuh"
#include "dsfacto_sgd.cuh"

namespace dsf {

struct TileKeyArgs {
    int64_t n;
    const int64_t *indptr;
    const int32_t *idx;
    const float *val;
    int32_t d, p;
    int sweep, jbits;
    int rbits;                // log2 of the row blocks per slot (0: one tile per slot)
    int32_t slot_rows;        // ceil(p / 2^rbits): slots per column block
    const int64_t *row_start;
    const int32_t *col_start;
    uint32_t *key;
    unsigned long long *payload;
};

// One warp per row (rows of a data set of this kind hold tens of entries).
__global__ void __launch_bounds__(kThreads) tile_keys_kernel(const TileKeyArgs a) {
    const int lane = (int)(threadIdx.x & 31u);
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const uint64_t p = (uint64_t)a.p;
    for (int64_t i = warp; i < a.n; i += nwarps) {
        const uint64_t r = ((uint64_t)i * p) / (uint64_t)a.n;                 // row block: floor(i p / n)
        const uint64_t sr = r >> a.rbits;                                     // its slot row, first row block sr << rbits
        const uint32_t il = (uint32_t)(i - a.row_start[sr << a.rbits]);
        const uint32_t rsub = (uint32_t)(((sr + 1) << a.rbits) - 1 - r);       // row blocks descend inside a slot
        const int64_t beg = a.indptr[i], end = a.indptr[i + 1];
        for (int64_t e = beg + lane; e < end; e += 32) {
            const uint32_t j = (uint32_t)a.idx[e];
            const uint64_t c = ((uint64_t)j * p) / (uint64_t)a.d;             // column block: floor(j p / d)
            uint64_t slot, phase = 1;
            if (a.sweep == 1) {
                slot = ((uint64_t)a.slot_rows - 1 - sr) * p + c;
                phase = r > c ? 0 : 1;                                        // tiles above the diagonal act on the tail composite
            } else {
                const uint64_t s = c >= r ? c - r : c + p - r;
                slot = s * p + r;
            }
            const uint32_t jl = j - (uint32_t)a.col_start[c];
            a.key[e] = (uint32_t)((((((slot << 1) | phase) << a.jbits) | jl) << a.rbits) | rsub);
            a.payload[e] = ((unsigned long long)il << 32) | (unsigned long long)__float_as_uint(a.val[e]);
        }
    }
}

__global__ void __launch_bounds__(kThreads) pack_entries_kernel(int64_t nnz, const uint32_t *__restrict__ key,
                                                                const unsigned long long *__restrict__ payload, int jbits,
                                                                int rbits, uint2 *__restrict__ ent) {
    const uint32_t jmask = jbits >= 32 ? 0xFFFFFFFFu : ((1u << jbits) - 1u);
    for (int64_t q = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; q < nnz; q += (int64_t)gridDim.x * blockDim.x) {
        const unsigned long long pl = payload[q];
        const uint32_t il = (uint32_t)(pl >> 32);
        ent[q] = make_uint2((jbits >= 32 ? 0u : (il << jbits)) | ((key[q] >> rbits) & jmask), (uint32_t)pl);
    }
}

// tile_ptr[s] = number of entries whose tile slot is below s, s = 0 .. ntiles
__global__ void __launch_bounds__(kThreads) tile_bounds_kernel(int64_t nnz, const uint32_t *__restrict__ key, int low_bits,
                                                               int64_t ntiles, int64_t *__restrict__ tile_ptr) {
    for (int64_t s = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; s <= ntiles; s += (int64_t)gridDim.x * blockDim.x) {
        const uint64_t bound = (uint64_t)s << low_bits;   // low_bits: key bits below the slot number
        int64_t lo = 0, hi = nnz;
        while (lo < hi) {
            const int64_t mid = lo + ((hi - lo) >> 1);
            if ((uint64_t)key[mid] < bound) lo = mid + 1; else hi = mid;
        }
        tile_ptr[s] = lo;
    }
}

struct TilePlanArgs {
    const uint32_t *key;       // sorted
    const int64_t *tile_ptr;   // ntiles + 1
    int64_t ntiles;
    int jbits, chunk_len;
    int rbits;                 // log2 of the row blocks per slot
    int32_t slot_rows;         // slots per column block
    // kPlanCount: per tile the number of chunks, of runs longer than a chunk and of their slices
    int64_t *count, *runs, *recs;
    // writing passes: where the tile's chunks go; kPlanFull also: chunks of the earlier tiles of the tile's
    // column block, number of the tile's first long run and of its first slice record, and the partition
    const int64_t *first, *need, *run0, *rec0;
    int p, sweep;
    const int64_t *row_start;
    const int32_t *col_start;
    ChunkDesc *out;
};
enum { kPlanCount = 0, kPlanPieces = 1, kPlanFull = 2 };

// One warp per tile; everything but the key reads is the same in all lanes.  kPlanCount counts, kPlanPieces
// writes what depends on the tile alone (entry offset, length, flags, local column and slice numbers; the
// host fills in the rest: plans cut into segments), kPlanFull writes complete descriptors for the plain plan,
// in which the tiles are visited in slot order.
template <int MODE>
__global__ void __launch_bounds__(kThreads) plan_tiles_kernel(const TilePlanArgs a) {
    const int lane = (int)(threadIdx.x & 31u);
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const uint32_t jmask = a.jbits >= 32 ? 0xFFFFFFFFu : ((1u << a.jbits) - 1u);
    const uint32_t idmask = a.jbits >= 31 ? 0xFFFFFFFFu : ((2u << a.jbits) - 1u);   // (phase, local column): what names a run
    const int64_t L = a.chunk_len;
    for (int64_t t = warp; t < a.ntiles; t += nwarps) {
        const int64_t beg = a.tile_ptr[t], nt = a.tile_ptr[t + 1] - beg;
        ChunkDesc *out = MODE != kPlanCount ? a.out + a.first[t] : nullptr;
        ChunkDesc proto{};   // what all chunks of the tile share
        int64_t next_run = 0, next_rec = 0, cur_run = 0, cur_rec0 = 0;
        if (MODE == kPlanFull) {
            int64_t r, c;   // r: the first row block of the slot
            if (a.sweep == 1) { r = ((int64_t)a.slot_rows - 1 - t / a.p) << a.rbits; c = t % a.p; }
            else { r = t % a.p; c = (r + t / a.p) % a.p; }
            proto.row0 = (int32_t)a.row_start[r];
            proto.col0 = a.col_start[c];
            proto.cblock = (int32_t)c;
            proto.need = (int32_t)a.need[t];
            proto.tile = (int32_t)t;
            proto.nchunks = (int32_t)(a.first[t + 1] - a.first[t]);
            next_run = a.run0[t];
            next_rec = a.rec0[t];
        }
        int64_t emitted = 0, nruns = 0, nrecs = 0;
        // (ph: phase of the chunk's runs; the host sets the tail flag of the pieces it orders itself)
        auto emit = [&](int64_t off, int64_t len, int flags, uint32_t jl, int64_t slice, int64_t nslices, uint32_t ph) {
            if (MODE != kPlanCount && lane == 0) {
                ChunkDesc d = proto;
                d.ent_off = beg + off;
                d.len = (int32_t)len;
                d.flags = flags | ((MODE == kPlanFull && a.sweep == 1 && ph == 0) ? kChunkTail : 0);
                d.jl = (int32_t)jl;
                d.slice = (int32_t)slice;
                d.nslices = (int32_t)nslices;
                if (MODE == kPlanFull && (flags & kChunkSlice)) { d.run_id = (int32_t)cur_run; d.rec0 = (int32_t)cur_rec0; }
                out[emitted] = d;
            }
            emitted += 1;
        };
        int64_t cur0 = 0, cur = 0;   // open chunk of whole runs: entries [cur0, cur0 + cur) of the tile
        uint32_t cur_ph = 1;         // ... and the phase of its runs
        auto take_run = [&](int64_t prev, int64_t len, uint32_t id) {
            const uint32_t jl = id & jmask, ph = a.jbits >= 31 ? 1u : (id >> a.jbits);
            if (cur > 0 && ph != cur_ph) {   // no chunk spans the tail part and the main part of a slot
                emit(cur0, cur, 0, 0u, 0, 0, cur_ph);
                cur = 0;
            }
            if (len > L) {
                if (cur > 0) emit(cur0, cur, 0, 0u, 0, 0, cur_ph);
                cur = 0;
                int64_t ns = (len + L - 1) / L;
                int64_t per = ((len + ns - 1) / ns + 31) & ~(int64_t)31;   // slices of whole passes, about equal
                if (per > L) per = L;
                ns = (len + per - 1) / per;
                nruns += 1;
                nrecs += ns;
                cur_run = next_run++;
                cur_rec0 = next_rec;
                next_rec += ns;
                for (int64_t k = 0; k < ns; ++k) {
                    const int64_t rest = len - k * per;
                    emit(prev + k * per, rest < per ? rest : per, kChunkSlice, jl, k, ns, ph);
                }
            } else if (cur + len > L) {
                emit(cur0, cur, 0, 0u, 0, 0, cur_ph);
                cur0 = prev;
                cur = len;
                cur_ph = ph;
            } else {
                if (cur == 0) { cur0 = prev; cur_ph = ph; }
                cur += len;
            }
        };
        int64_t run_start = 0;
        uint32_t run_jl = 0, carry = 0xFFFFFFFFu;   // (no local column has all bits set: d < 2^31)
        bool have = false;
        for (int64_t base = 0; base < nt; base += 32) {
            const int64_t pos = base + lane;
            const uint32_t jl = pos < nt ? ((a.key[beg + pos] >> a.rbits) & idmask) : 0xFFFFFFFFu;   // (phase, local column)
            uint32_t prevj = __shfl_up_sync(0xFFFFFFFFu, jl, 1);
            if (lane == 0) prevj = carry;
            uint32_t m = __ballot_sync(0xFFFFFFFFu, pos < nt && jl != prevj);
            carry = __shfl_sync(0xFFFFFFFFu, jl, 31);
            while (m) {
                const int b = __ffs(m) - 1;
                m &= m - 1;
                if (have) take_run(run_start, base + b - run_start, run_jl);
                run_start = base + b;
                run_jl = __shfl_sync(0xFFFFFFFFu, jl, b);
                have = true;
            }
        }
        if (have) take_run(run_start, nt - run_start, run_jl);
        if (cur > 0) emit(cur0, cur, 0, 0u, 0, 0, cur_ph);
        if (MODE == kPlanCount && lane == 0) { a.count[t] = emitted; a.runs[t] = nruns; a.recs[t] = nrecs; }
    }
}

// test knob: the first chunk of the sweep is made to wait for more finished chunks than there will ever be
__global__ void plan_extra_need_kernel(ChunkDesc *desc, int extra) { desc[0].need += extra; }

}  // namespace dsf
