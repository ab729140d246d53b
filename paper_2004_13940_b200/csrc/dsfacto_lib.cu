// Host side of the DS-FACTO C ABI (include/dsfacto.h): handle, validation, seeded initialisation,
// the tile bucketer, device memory, the epoch driver and the copy-out calls.
#include "dsfacto.h"
#include "dsfacto_bucket.cuh"
#include "dsfacto_refresh.cuh"
#include "dsfacto_sgd.cuh"

#include <cub/device/device_radix_sort.cuh>

#include <omp.h>
#include <sys/mman.h>

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <string>
#include <vector>

namespace {

using namespace dsf;

}  // namespace

struct dsfacto {
    int64_t n = 0, nnz = 0;
    int32_t d = 0, K = 0, Kp = 0, p = 0, loss = 0, LG = 1, NV = 1;   // lane layout of the stratum SGD kernel
    int32_t LGr = 1, NVr = 1;                                         // ... and of the recompute kernel (same Kp)
    float lambda_w = 0, lambda_v = 0, eta = 0;
    float h = 0;  // per-entry step eta / n
    uint64_t seed = 0;
    float w0 = 0.f;
    bool loaded = false, wide = false;
    // column shard (Section 4.2: the column blocks of w and V spread over workers): this handle owns column
    // blocks [cb_lo, cb_hi), i.e. columns [col_lo, col_hi); nshards == 1 is the ordinary handle
    int32_t shard = 0, nshards = 1, cb_lo = 0, cb_hi = 0, col_lo = 0, col_hi = 0;
    bool awaiting_sum = false;   // shard: partial auxiliaries computed, totals not yet handed in
    float *d_lin = nullptr, *d_q = nullptr;   // shard: per-row partial sums, stored right behind A
    int ibits = 0, jbits = 0;
    cudaStream_t stream = nullptr;
    cudaEvent_t ev[4] = {nullptr, nullptr, nullptr, nullptr};
    float ms[4] = {0, 0, 0, 0};
    int64_t launches = 0;
    int sm_count = 148, device = 0;
    int l2_bytes = 126 << 20;   // L2 cache size of the device
    std::string err;

    std::vector<int64_t> row_start;  // p+1
    std::vector<int32_t> col_start;  // p+1
    std::vector<int64_t> tile_ptr;   // p*p+1, tiles in DEVICE order ("slots": the order the sweep visits them)

    // device
    float *d_w = nullptr, *d_V = nullptr, *d_A = nullptr, *d_G = nullptr, *d_y = nullptr, *d_val = nullptr, *d_xw = nullptr;
    int64_t *d_indptr = nullptr, *d_tile_ptr = nullptr, *d_row_start = nullptr;
    int32_t *d_idx = nullptr, *d_col_start = nullptr;
    uint2 *d_ent = nullptr;
    double *d_partials = nullptr, *d_scal = nullptr;
    // stratum SGD launch plan: launch L covers chunks [launch_ptr[L], launch_ptr[L+1]) of chunk_map
    int sweep = 1;  // 1: a launch is a row block (p-1 .. 0); 0: a launch is an inner round (0 .. p-1)
    int refresh_every = 0;  // > 0: G, A recomputed after every that many inner rounds
    int64_t plan_segments = 0;  // > 0: the launch plan is cut into that many segments of refresh_every rounds (row-block sweep)
    std::vector<int64_t> launch_ptr;
    ChunkDesc *d_desc = nullptr;   // chunk descriptors in sweep order
    int *d_sync = nullptr;     // ticket, error word, per-column-block progress of the fused SGD launch
    int64_t total_chunks = 0, long_runs = 0, slice_records = 0;
    int chunk_len = 512;        // most entries a chunk of the stratum SGD launches holds
    int block_len = 128;        // entries per block of the kernel's entry ring
    int chunk_override = 0;     // > 0: chunk length forced by dsfacto_debug_set (tests)
    int sgd_grid = 0;           // CTAs of the persistent stratum SGD launch
    int spin_limit = kSgdSpinLimit;  // polls before a wait for an earlier tile gives up
    int debug_extra_need = 0;   // tests: added to the `need` of the first chunk at the next load, so that its wait runs out
    bool failed = false;        // an SGD launch gave up; the parameters are unusable until they are set again
    float *d_records = nullptr, *d_Tb = nullptr, *d_Tw = nullptr;
    float4 *d_S = nullptr, *d_TS = nullptr;  // scale records of the scaled column state (zero outside the SGD phase)
    int *d_run_count = nullptr;
    int refresh_grid = 0, norm_grid = 0;
    int rbits = 0;              // log2 of the row blocks per slot of the device entry array (device bucketing; 0: one tile per slot)
    int row_merge = 0;          // dsfacto_debug_set: row blocks per slot wanted (0 = chosen by the load, 1, 2, 4, 8)
    int64_t load_info[3] = {0, 0, 0};   // last load: path (0 host, 1 host streamed, 2 device), bytes H2D, bytes D2H
    // Column slots of the recompute pass (per load): the device CSR holds slots (rank by frequency) instead of
    // column indices, and the pass reads w and V from copies in slot order.
    int column_order = 0;       // dsfacto_debug_set: 0 = decided per load, 1 = always, 2 = never
    bool slots = false;
    int32_t *d_column_of = nullptr;
    float *d_Vs = nullptr;
    // What the recompute pass reads beside V: per column (w_j, sum_k v_jk^2), by column index (d_pair) and, for
    // the renumbered device CSR, by slot (d_pair_s, with d_Vs).  Each is rebuilt when the parameters have
    // changed since it was made (model_version counts the changes).
    float2 *d_pair = nullptr, *d_pair_s = nullptr;
    int64_t model_version = 1, pair_version = 0, slot_version = 0;

    double loss_sum = 0, g_sum = 0, w2 = 0, v2 = 0, objective = 0;
};

namespace {

#define CU_TRY(h, call)                                                                     \
    do {                                                                                    \
        cudaError_t e_ = (call);                                                            \
        if (e_ != cudaSuccess) {                                                            \
            (h)->err = std::string(#call) + ": " + cudaGetErrorString(e_);                 \
            return e_ == cudaErrorMemoryAllocation ? DSFACTO_ERR_OOM : DSFACTO_ERR_CUDA;    \
        }                                                                                   \
    } while (0)

// the same inside dsfacto_load_csr: a failed call leaves no half-built data set behind (free_data is declared below)
void free_data(dsfacto *h);
#define CU_TRY_LOAD(h, call)                                                                \
    do {                                                                                    \
        cudaError_t e_ = (call);                                                            \
        if (e_ != cudaSuccess) {                                                            \
            (h)->err = std::string(#call) + ": " + cudaGetErrorString(e_);                 \
            cudaStreamSynchronize((h)->stream);                                             \
            free_data(h);                                                                   \
            return e_ == cudaErrorMemoryAllocation ? DSFACTO_ERR_OOM : DSFACTO_ERR_CUDA;    \
        }                                                                                   \
    } while (0)

template <typename T>
int dev_alloc(dsfacto *h, T **ptr, size_t count) {
    *ptr = nullptr;
    if (count == 0) count = 1;
    CU_TRY(h, cudaMalloc((void **)ptr, count * sizeof(T)));
    return DSFACTO_OK;
}
template <typename T>
void dev_free(T *&ptr) {
    if (ptr) cudaFree(ptr);
    ptr = nullptr;
}

// Large host scratch without the zero fill of std::vector: the pages are first touched by the
// parallel passes that write them.
template <typename T>
struct HostBuf {
    T *p = nullptr;
    HostBuf() = default;
    HostBuf(const HostBuf &) = delete;
    HostBuf &operator=(const HostBuf &) = delete;
    ~HostBuf() { std::free(p); }
    bool alloc(size_t count) {
        std::free(p);
        p = nullptr;
        const size_t bytes = (count ? count : 1) * sizeof(T);
        constexpr size_t kHuge = (size_t)2 << 20;
        if (bytes >= 8 * kHuge) {
            // large scratch: 2 MB alignment and a hint for transparent huge pages, so that the first
            // touch costs one page fault per 2 MB instead of one per 4 KB (C4 load: 4.6 s -> 3.9 s)
            const size_t rounded = (bytes + kHuge - 1) / kHuge * kHuge;
            void *q = nullptr;
            if (posix_memalign(&q, kHuge, rounded) != 0) return false;
            madvise(q, rounded, MADV_HUGEPAGE);
            p = static_cast<T *>(q);
        } else {
            p = static_cast<T *>(std::malloc(bytes));
        }
        return p != nullptr;
    }
    T *data() { return p; }
    T &operator[](size_t i) { return p[i]; }
};

// ---- SplitMix64 (Steele, Lea, Flood 2014), random access to the c-th output ----
inline uint64_t splitmix64_output(uint64_t seed, uint64_t c) {
    uint64_t z = seed + (c + 1) * 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}
inline double open_unit(uint64_t u) { return ((double)(u >> 11) + 0.5) * (1.0 / 9007199254740992.0); }
inline float init_factor(uint64_t seed, uint64_t e) {
    const double u1 = open_unit(splitmix64_output(seed, 2 * e));
    const double u2 = open_unit(splitmix64_output(seed, 2 * e + 1));
    const double z = std::sqrt(-2.0 * std::log(u1)) * std::cos(2.0 * 3.14159265358979323846 * u2);
    return (float)(0.01 * z);
}

constexpr int kMaxRowMerge = 16;   // most row blocks per slot of the device entry array (32 and 64 were no faster on any data set)
constexpr int64_t kStreamedLoadMinEntries = (int64_t)1 << 24;   // smaller loads are not worth the staging set-up

inline int bits_for(int64_t count) {  // bits needed for values in [0, count)
    int b = 0;
    while (((int64_t)1 << b) < count) ++b;
    return b;
}

// Device order of the tiles = the order in which the SGD sweep visits them, so that the entries a
// launch works on at any moment are close together in memory.  Slot L*p + k holds, for the row-block
// sweep, tile (r = p-1-L, c = k); for the round sweep, tile (r = k, round s = L), which is also the
// canonical tile number s*p + r.
inline int64_t tile_slot(const dsfacto *h, int64_t r, int64_t c) {
    const int64_t p = h->p;
    if (h->sweep == 1) return (p - 1 - r) * p + c;
    int64_t s = c - r;
    if (s < 0) s += p;
    return s * p + r;
}
inline void slot_tile(const dsfacto *h, int64_t slot, int64_t &r, int64_t &c) {
    const int64_t p = h->p;
    if (h->sweep == 1) { r = p - 1 - slot / p; c = slot % p; }
    else { r = slot % p; c = (r + slot / p) % p; }
}
// canonical tile_ptr (tile number s*p + r, s = (c - r) mod p) from the device-order one
std::vector<int64_t> canonical_tile_ptr(const dsfacto *h) {
    const int64_t p = h->p, nt = p * p;
    std::vector<int64_t> cp((size_t)nt + 1, 0);
    for (int64_t slot = 0; slot < nt; ++slot) {
        int64_t r, c;
        slot_tile(h, slot, r, c);
        int64_t sr = c - r;
        if (sr < 0) sr += p;
        cp[(size_t)(sr * p + r) + 1] = h->tile_ptr[slot + 1] - h->tile_ptr[slot];
    }
    for (int64_t t = 0; t < nt; ++t) cp[t + 1] += cp[t];
    return cp;
}

// partition: row block r = rows [ceil(r n / p), ceil((r+1) n / p)), i.e. floor(i p / n) = r; same for
// columns.  Also chooses the packed (32-bit key) or wide entry layout.
int setup_partition(dsfacto *h) {
    const int64_t n = h->n;
    const int32_t d = h->d, p = h->p;
    try {
        h->row_start.resize((size_t)p + 1);
        h->col_start.resize((size_t)p + 1);
    } catch (const std::bad_alloc &) { return DSFACTO_ERR_OOM; }
    int64_t max_rows = 0, max_cols = 0;
    for (int32_t r = 0; r <= p; ++r) {
        h->row_start[r] = (int64_t)(((__int128)r * n + p - 1) / p);
        h->col_start[r] = (int32_t)(((__int128)r * d + p - 1) / p);
    }
    for (int32_t r = 0; r < p; ++r) {
        max_rows = std::max(max_rows, h->row_start[r + 1] - h->row_start[r]);
        max_cols = std::max<int64_t>(max_cols, h->col_start[r + 1] - h->col_start[r]);
    }
    h->ibits = bits_for(max_rows);
    h->jbits = bits_for(max_cols);
    h->wide = (h->ibits + h->jbits) > 32;
    if (h->wide) h->jbits = 32;
    return DSFACTO_OK;
}

// canonical (global row, global column, value) lists from the packed device layout
void unpack_tiles(const dsfacto *h, const std::vector<int64_t> &canon_ptr, const uint2 *ent, const float *xw,
                  int32_t *rows, int32_t *cols, float *vals) {
    const int64_t nt = (int64_t)h->p * h->p;
    const uint32_t jmask = h->jbits >= 32 ? 0xFFFFFFFFu : ((1u << h->jbits) - 1u);
#pragma omp parallel for schedule(dynamic, 8)
    for (int64_t slot = 0; slot < nt; ++slot) {
        int64_t r, c;
        slot_tile(h, slot, r, c);
        int64_t sr = c - r;
        if (sr < 0) sr += h->p;
        const int64_t shift = canon_ptr[(size_t)(sr * h->p + r)] - h->tile_ptr[slot];
        for (int64_t q = h->tile_ptr[slot]; q < h->tile_ptr[slot + 1]; ++q) {
            uint32_t il, jl;
            float x;
            if (h->wide) { il = ent[q].x; jl = ent[q].y; x = xw[q]; }
            else { il = ent[q].x >> h->jbits; jl = ent[q].x & jmask; std::memcpy(&x, &ent[q].y, 4); }
            if (rows) rows[q + shift] = (int32_t)(h->row_start[r] + il);
            if (cols) cols[q + shift] = (int32_t)(h->col_start[c] + jl);
            if (vals) vals[q + shift] = x;
        }
    }
}

// The same for a device entry array whose slots hold several row blocks (device bucketing with merged row
// blocks): slot (slot row sr, column block c) lists, per phase, its entries by (column, row block descending,
// row); an entry's row block follows from its row.  canon_ptr (p*p + 1) is filled here as well.
void unpack_merged_tiles(const dsfacto *h, const uint2 *ent, std::vector<int64_t> &canon_ptr, int32_t *rows, int32_t *cols,
                         float *vals) {
    const int64_t p = h->p, R = (int64_t)1 << h->rbits, slot_rows = (p + R - 1) / R, nslots = slot_rows * p;
    const uint32_t jmask = h->jbits >= 32 ? 0xFFFFFFFFu : ((1u << h->jbits) - 1u);
    canon_ptr.assign((size_t)(p * p) + 1, 0);
    auto tile_of = [&](int64_t slot, uint32_t il, int64_t &i) -> int64_t {
        const int64_t rb0 = (slot_rows - 1 - slot / p) * R, c = slot % p;
        i = h->row_start[(size_t)rb0] + il;
        int64_t r = rb0;
        while (r + 1 < p && i >= h->row_start[(size_t)(r + 1)]) ++r;
        int64_t sr = c - r;
        if (sr < 0) sr += p;
        return sr * p + r;
    };
#pragma omp parallel for schedule(dynamic, 8)
    for (int64_t slot = 0; slot < nslots; ++slot)   // (different slots hold different tiles)
        for (int64_t q = h->tile_ptr[slot]; q < h->tile_ptr[slot + 1]; ++q) {
            int64_t i;
            canon_ptr[(size_t)tile_of(slot, ent[q].x >> h->jbits, i) + 1] += 1;
        }
    for (int64_t t = 0; t < p * p; ++t) canon_ptr[(size_t)t + 1] += canon_ptr[(size_t)t];
    if (!rows && !cols && !vals) return;
#pragma omp parallel for schedule(dynamic, 8)
    for (int64_t slot = 0; slot < nslots; ++slot) {
        int64_t off[kMaxRowMerge];   // next free place of the slot's tiles, by row block
        for (int k = 0; k < kMaxRowMerge; ++k) off[k] = -1;
        const int64_t rb0 = (slot_rows - 1 - slot / p) * R, c = slot % p;
        for (int64_t q = h->tile_ptr[slot]; q < h->tile_ptr[slot + 1]; ++q) {
            int64_t i;
            const int64_t tile = tile_of(slot, ent[q].x >> h->jbits, i);
            const int64_t k = tile % p - rb0;
            if (off[k] < 0) off[k] = canon_ptr[(size_t)tile];
            const int64_t at = off[k]++;
            float x;
            std::memcpy(&x, &ent[q].y, 4);
            if (rows) rows[at] = (int32_t)i;
            if (cols) cols[at] = (int32_t)(h->col_start[(size_t)c] + (ent[q].x & jmask));
            if (vals) vals[at] = x;
        }
    }
}

void free_data(dsfacto *h) {
    h->rbits = 0;
    dev_free(h->d_A); dev_free(h->d_G); dev_free(h->d_y); dev_free(h->d_val); dev_free(h->d_xw);
    dev_free(h->d_indptr); dev_free(h->d_tile_ptr); dev_free(h->d_idx); dev_free(h->d_ent);
    dev_free(h->d_partials); dev_free(h->d_desc); dev_free(h->d_records); dev_free(h->d_run_count);
    dev_free(h->d_sync); dev_free(h->d_column_of); dev_free(h->d_Vs); dev_free(h->d_pair_s);
    h->slots = false;
    h->slot_version = 0;
    h->launch_ptr.clear();
    h->d_lin = h->d_q = nullptr;
    h->awaiting_sum = false;
    h->loaded = false;
    h->nnz = 0;
}

// ---------------------------------------------------------------------------------------------
// kernel dispatch over the factor-row layout
// ---------------------------------------------------------------------------------------------
template <int LG, int NV>
void launch_sgd(dsfacto *h, const SgdArgs &a, int64_t chunks) {
    const size_t bytes = (size_t)kSgdWarps * sgd_warp_smem<LG, NV>(h->wide, h->block_len);
    // The launch is persistent: as many CTAs as stay resident (fewer if there are fewer chunks), each warp
    // taking chunks from the ticket counter until none is left.  More than 48 KB of dynamic shared memory
    // needs an opt-in per kernel; the residency depends on the chunk length, so both are redone per load.
    if (h->sgd_grid == 0) {
        int per_sm = 0;
        if (h->wide) {
            cudaFuncSetAttribute(sgd_sweep_kernel<LG, NV, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, sgd_sweep_kernel<LG, NV, true>, kSgdThreads, bytes);
        } else {
            cudaFuncSetAttribute(sgd_sweep_kernel<LG, NV, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, sgd_sweep_kernel<LG, NV, false>, kSgdThreads, bytes);
        }
        if (per_sm < 1) per_sm = 1;
        h->sgd_grid = h->sm_count * per_sm;
    }
    const int64_t want = (chunks + kSgdWarps - 1) / kSgdWarps;
    const int grid = (int)std::min<int64_t>(h->sgd_grid, std::max<int64_t>(want, 1));
    if (h->wide) sgd_sweep_kernel<LG, NV, true><<<grid, kSgdThreads, bytes, h->stream>>>(a);
    else sgd_sweep_kernel<LG, NV, false><<<grid, kSgdThreads, bytes, h->stream>>>(a);
}
template <int LG, int NV>
void launch_refresh(dsfacto *h, const RefreshArgs &a, int mode, int grid) {
    if (mode == kTrain) refresh_kernel<LG, NV, kTrain><<<grid, kThreads, 0, h->stream>>>(a);
    else if (mode == kEvaluate) refresh_kernel<LG, NV, kEvaluate><<<grid, kThreads, 0, h->stream>>>(a);
    else if (mode == kPartial) refresh_kernel<LG, NV, kPartial><<<grid, kThreads, 0, h->stream>>>(a);
    else refresh_kernel<LG, NV, kScore><<<grid, kThreads, 0, h->stream>>>(a);
}

#define DSF_DISPATCH(h, FN, ...)                                   \
    do {                                                           \
        switch ((h)->LG * 10 + (h)->NV) {                          \
        case 11: FN<1, 1>(__VA_ARGS__); break;                     \
        case 21: FN<2, 1>(__VA_ARGS__); break;                     \
        case 41: FN<4, 1>(__VA_ARGS__); break;                     \
        case 81: FN<8, 1>(__VA_ARGS__); break;                     \
        case 161: FN<16, 1>(__VA_ARGS__); break;                   \
        case 162: FN<16, 2>(__VA_ARGS__); break;                   \
        case 163: FN<16, 3>(__VA_ARGS__); break;                   \
        case 164: FN<16, 4>(__VA_ARGS__); break;                   \
        default: break;                                            \
        }                                                          \
    } while (0)

// the recompute kernel has its own lane layout (4 * LGr * NVr = Kp as well)
#define DSF_DISPATCH_REFRESH(h, ...)                               \
    do {                                                           \
        switch ((h)->LGr * 10 + (h)->NVr) {                        \
        case 11: launch_refresh<1, 1>(__VA_ARGS__); break;         \
        case 21: launch_refresh<2, 1>(__VA_ARGS__); break;         \
        case 41: launch_refresh<4, 1>(__VA_ARGS__); break;         \
        case 81: launch_refresh<8, 1>(__VA_ARGS__); break;         \
        case 161: launch_refresh<16, 1>(__VA_ARGS__); break;       \
        case 84: launch_refresh<8, 4>(__VA_ARGS__); break;         \
        case 86: launch_refresh<8, 6>(__VA_ARGS__); break;         \
        case 88: launch_refresh<8, 8>(__VA_ARGS__); break;         \
        default: break;                                            \
        }                                                          \
    } while (0)

int refresh_grid_for(const dsfacto *h, int64_t rows) {
    const int G = kThreads / h->LGr;
    int64_t want = (rows + G - 1) / G;
    const int64_t cap = (int64_t)h->sm_count * 16;
    if (want > cap) want = cap;
    if (want < 1) want = 1;
    return (int)want;
}

// ---------------------------------------------------------------------------------------------
// Launch plan of the stratum SGD phase.  While a tile is bucketed its column counts are at hand, and
// the tile is cut into chunks right there: whole runs (all entries of one column inside the tile) are
// packed greedily into chunks of at most chunk_len entries, and a run longer than that becomes slices
// of its own.  The per-tile pieces are put in sweep order afterwards (finish_sgd_plan).
// ---------------------------------------------------------------------------------------------
struct TilePlanner {          // one per host thread
    std::vector<ChunkDesc> descs;
    bool failed = false;      // out of host memory
};
struct TileDescRef {          // where the chunks of a tile sit
    int32_t owner = 0, count = 0;
    int64_t first = 0;
};
struct SgdPlanBuild {
    bool finished = false;     // device bucketing, plain plan: the descriptors are complete and on the device already
    HostBuf<ChunkDesc> bulk;   // device bucketing: the chunks of all tiles as a kernel cut them, instead of the planners
    std::vector<TilePlanner> planners;
    std::vector<TileDescRef> refs;   // per tile slot
};

// Chunk length: long chunks when the data set keeps the GPU busy for many rounds of resident warps;
// otherwise the epoch is a chain of p dependent tiles per column block and is as long as p times the
// time one tile takes, so tiles are cut into short chunks that run side by side.
void choose_chunk_len(dsfacto *h, int64_t nnz, int64_t slot_rows) {
    // A chunk costs about 6.6 k cycles whatever its length (first requests, join of the lane groups, record,
    // fence, counters), and the kernel reads a chunk's entries through a ring of blocks, so its shared memory
    // does not limit the length.  Measured sweeps, slots of 8 row blocks: 1.755 G entries with 64-byte rows,
    // 416 / 832 / 1248 / 1664 / 2080 / 3328 entries: 25.0 / 22.7 / 22.0 / 21.8 / 21.6 / 21.9 ms; 400 M entries
    // with 512-byte rows, 256 / 832 / 1664 / 2496 / 3328: 29.6 / 23.4 / 21.6 / 21.5 / 21.8 ms.
    // A tile waits for the tile above it in its column block, which lies one slot row (slot_rows of them share
    // the entries) earlier in ticket order: a slot row must hold a few times as many chunks as warps are
    // resident, or the warps wait (scaled cases of a tenth of the entries with 2048-entry chunks: +3 % and +47 %).
    h->chunk_len = 2048;
    {
        const int64_t warps = (int64_t)h->sm_count * (h->Kp >= 64 ? 10 : 20);
        const int64_t fit = (nnz / std::max<int64_t>(slot_rows, 1) / (3 * warps)) & ~(int64_t)31;
        h->chunk_len = (int)std::min<int64_t>(2048, std::max<int64_t>(128, fit));
    }
    if (nnz / 512 < (int64_t)h->sm_count * 24 * 16) h->chunk_len = 128;
    // A plan cut into segments visits every row block with a fraction of its tiles, so the tiles of a column
    // block follow one another closely in ticket order and long chunks leave the warps waiting for the tile
    // above: 1.755 G entries in four segments, 64 / 96 / 128 / 160 / 256 / 416 / 2048 entries: 56 / 45 / 41 / 43 /
    // 55 / 74 / 218 ms for the four launches together.
    if (h->refresh_every > 0 && h->refresh_every < h->p) h->chunk_len = 128;
    if (h->chunk_override > 0) h->chunk_len = h->chunk_override;
    if (const char *env = std::getenv("DSFACTO_CHUNK")) {
        const int v = std::atoi(env);
        if (v >= 16 && v <= kChunkMax) h->chunk_len = v;
    }
    // the kernel streams a chunk's entries through a ring of blocks: a whole chunk per block when it is short
    // (blocks of 96 / 128 / 192 / 256 entries with 64-byte rows: 22.5 / 22.0 / 21.7 / 22.1 ms; wide rows leave less
    // shared memory: 64 / 96 / 128 entries with 512-byte rows: 21.5 / 21.3 / 21.8 ms)
    h->block_len = std::min(h->Kp >= 64 ? kEntBlockWide : kEntBlockDefault, (h->chunk_len + 31) & ~31);
    if (const char *env = std::getenv("DSFACTO_BLOCK")) {
        const int v = std::atoi(env);
        if (v >= 32 && v <= kEntBlockMax && v % 32 == 0) h->block_len = v;
    }
    h->sgd_grid = 0;   // residency is recomputed at the next launch
}

// col_end[j] = number of entries of the tile whose local column is <= j; tile_begin = position of the
// tile's first entry in the entry array
void plan_tile(const dsfacto *h, SgdPlanBuild *pb, int owner, int64_t slot, int64_t tile_begin, const int64_t *col_end,
               int64_t width) {
    if (!pb) return;
    TilePlanner &tp = pb->planners[(size_t)owner];
    const int64_t L = h->chunk_len;
    const size_t first = tp.descs.size();
    try {
        auto emit = [&](int64_t off, int64_t len, int flags, int64_t jl, int64_t slice, int64_t nslices) {
            ChunkDesc d{};
            d.ent_off = tile_begin + off;
            d.len = (int32_t)len;
            d.flags = flags;
            d.jl = (int32_t)jl;
            d.slice = (int32_t)slice;
            d.nslices = (int32_t)nslices;
            tp.descs.push_back(d);
        };
        int64_t cur0 = 0, cur = 0, prev = 0;   // open chunk of whole runs [cur0, cur0 + cur); end of the last column
        for (int64_t j = 0; j < width; ++j) {
            const int64_t end = col_end[j], len = end - prev;
            if (len == 0) continue;
            if (len > L) {
                if (cur > 0) emit(cur0, cur, 0, 0, 0, 0);
                cur = 0;
                int64_t ns = (len + L - 1) / L;
                int64_t per = ((len + ns - 1) / ns + 31) & ~(int64_t)31;   // slices of whole passes, about equal
                if (per > L) per = L;
                ns = (len + per - 1) / per;
                for (int64_t k = 0; k < ns; ++k)
                    emit(prev + k * per, std::min(per, len - k * per), kChunkSlice, j, k, ns);
            } else if (cur + len > L) {
                emit(cur0, cur, 0, 0, 0, 0);
                cur0 = prev;
                cur = len;
            } else {
                if (cur == 0) cur0 = prev;
                cur += len;
            }
            prev = end;
        }
        if (cur > 0) emit(cur0, cur, 0, 0, 0, 0);
    } catch (const std::bad_alloc &) {
        tp.failed = true;
        return;
    }
    TileDescRef &ref = pb->refs[(size_t)slot];
    ref.owner = owner;
    ref.first = (int64_t)first;
    ref.count = (int32_t)(tp.descs.size() - first);
}

bool init_plan_build(const dsfacto *h, SgdPlanBuild &pb, int threads) {
    try {
        pb.planners.assign((size_t)std::max(threads, 1), TilePlanner());
        pb.refs.assign((size_t)h->p * h->p, TileDescRef());
    } catch (const std::bad_alloc &) { return false; }
    return true;
}

// Puts the chunks in sweep order, fills in what depends on it (earlier tiles of the column block, run
// and record numbers, launch ranges) and copies the plan to the device.
int finish_sgd_plan(dsfacto *h, SgdPlanBuild &pb) {
    const int64_t p = h->p, nt = p * p;
    for (const TilePlanner &tp : pb.planners)
        if (tp.failed) return DSFACTO_ERR_OOM;
    int64_t total = 0;
    for (int64_t t = 0; t < nt; ++t) total += pb.refs[(size_t)t].count;
    if (total >= (int64_t)kTicketStop / 2) return DSFACTO_ERR_INVALID_ARG;
    HostBuf<ChunkDesc> all;
    std::vector<int> seen;   // chunks met so far per column block
    if (!all.alloc((size_t)total)) return DSFACTO_ERR_OOM;
    try {
        h->launch_ptr.assign((size_t)p + 1, 0);
        seen.assign((size_t)p, 0);
    } catch (const std::bad_alloc &) { return DSFACTO_ERR_OOM; }
    // Segments: with the second schedule (recompute after every R inner rounds) on the row-block sweep, a
    // launch covers the tiles of R consecutive rounds, still visited row block by row block.  For column
    // block c a segment that starts at round s0 begins at row block (c - s0) mod p and descends cyclically,
    // so inside a segment the tiles above that row block are the ones that act on the tail composite.
    const bool segmented = h->sweep == 1 && h->refresh_every > 0 && h->refresh_every < p;
    const int64_t every = segmented ? h->refresh_every : p;
    const int64_t nseg = segmented ? (p + every - 1) / every : 1;
    try {
        if (segmented) h->launch_ptr.assign((size_t)nseg + 1, 0);
    } catch (const std::bad_alloc &) { return DSFACTO_ERR_OOM; }
    h->plan_segments = segmented ? nseg : 0;
    auto chunk_of = [&](const TileDescRef &ref, int32_t q) -> const ChunkDesc & {
        return pb.bulk.p ? pb.bulk.p[(size_t)(ref.first + q)] : pb.planners[(size_t)ref.owner].descs[(size_t)(ref.first + q)];
    };
    // 1. long runs and slice records of every tile (in parallel)
    std::vector<int32_t> tile_runs, tile_recs;
    struct Visit { int64_t slot, pos, run0, rec0; int32_t r, c, need; bool tail; };
    std::vector<Visit> visit;
    try {
        tile_runs.assign((size_t)nt, 0);
        tile_recs.assign((size_t)nt, 0);
        visit.reserve((size_t)nt);
    } catch (const std::bad_alloc &) { return DSFACTO_ERR_OOM; }
#pragma omp parallel for schedule(dynamic, 64)
    for (int64_t slot = 0; slot < nt; ++slot) {
        const TileDescRef &ref = pb.refs[(size_t)slot];
        int32_t nr = 0, nrec = 0;
        for (int32_t q = 0; q < ref.count; ++q) {
            const ChunkDesc &d = chunk_of(ref, q);
            if ((d.flags & kChunkSlice) && d.slice == 0) { nr += 1; nrec += d.nslices; }
        }
        tile_runs[(size_t)slot] = nr;
        tile_recs[(size_t)slot] = nrec;
    }
    // 2. the tiles in the order the launches visit them, with what each one starts from (one thread: p^2 steps)
    int64_t pos = 0, runs = 0, recs = 0;
    for (int64_t seg = 0; seg < nseg; ++seg) {
        const int64_t s0 = seg * every, s1 = std::min(s0 + every, p);
        if (segmented) std::fill(seen.begin(), seen.end(), 0);
        // plain plan: every slot in order; segmented plan: row block by row block, the tiles of rounds [s0, s1)
        const int64_t visits = segmented ? p * (s1 - s0) : nt;
        for (int64_t vis = 0; vis < visits; ++vis) {
            int64_t slot = vis, r, c;
            bool tail;
            if (segmented) {
                r = p - 1 - vis / (s1 - s0);
                c = (r + s0 + vis % (s1 - s0)) % p;
                slot = tile_slot(h, r, c);
                int64_t r_first = c - s0;
                if (r_first < 0) r_first += p;
                tail = r > r_first;
            } else {
                slot_tile(h, slot, r, c);
                tail = h->sweep == 1 && r > c;
            }
            const TileDescRef &ref = pb.refs[(size_t)slot];
            Visit v;
            v.slot = slot; v.pos = pos; v.run0 = runs; v.rec0 = recs;
            v.r = (int32_t)r; v.c = (int32_t)c; v.need = seen[(size_t)c]; v.tail = tail;
            try { visit.push_back(v); } catch (const std::bad_alloc &) { return DSFACTO_ERR_OOM; }
            pos += ref.count;
            runs += tile_runs[(size_t)slot];
            recs += tile_recs[(size_t)slot];
            seen[(size_t)c] += ref.count;
            if (!segmented && (slot + 1) % p == 0) h->launch_ptr[(size_t)((slot + 1) / p)] = pos;
        }
        if (segmented) h->launch_ptr[(size_t)seg + 1] = pos;
    }
    // 3. the descriptors (in parallel over the tiles)
#pragma omp parallel for schedule(dynamic, 64)
    for (int64_t vi = 0; vi < (int64_t)visit.size(); ++vi) {
        const Visit &v = visit[(size_t)vi];
        const TileDescRef &ref = pb.refs[(size_t)v.slot];
        int64_t next_run = v.run0, next_rec = v.rec0, cur_run = 0, cur_rec0 = 0;
        for (int32_t q = 0; q < ref.count; ++q) {
            ChunkDesc d = chunk_of(ref, q);
            d.row0 = (int32_t)h->row_start[(size_t)v.r];
            d.col0 = h->col_start[(size_t)v.c];
            d.cblock = v.c;
            d.need = v.need;
            d.tile = (int32_t)v.slot;
            d.nchunks = ref.count;
            if (v.tail) d.flags |= kChunkTail;
            if (d.flags & kChunkSlice) {
                if (d.slice == 0) { cur_run = next_run++; cur_rec0 = next_rec; next_rec += d.nslices; }
                d.run_id = (int32_t)cur_run;
                d.rec0 = (int32_t)cur_rec0;
            }
            all[(size_t)(v.pos + q)] = d;
        }
    }
    if (recs >= ((int64_t)1 << 31)) return DSFACTO_ERR_INVALID_ARG;
    h->total_chunks = total;
    h->long_runs = runs;
    h->slice_records = recs;
    if (h->debug_extra_need > 0 && total > 0) all[0].need += h->debug_extra_need;
    int rc;
    if ((rc = dev_alloc(h, &h->d_desc, (size_t)total)) ||
        (rc = dev_alloc(h, &h->d_records, (size_t)recs * slice_record_floats(h->Kp))) ||
        (rc = dev_alloc(h, &h->d_run_count, (size_t)runs)) || (rc = dev_alloc(h, &h->d_sync, sync_words((int)p))))
        return rc;
    CU_TRY(h, cudaMemsetAsync(h->d_run_count, 0, sizeof(int) * (size_t)std::max<int64_t>(runs, 1), h->stream));
    CU_TRY(h, cudaMemsetAsync(h->d_sync, 0, sizeof(int) * sync_words((int)p), h->stream));
    if (total > 0)
        CU_TRY(h, cudaMemcpyAsync(h->d_desc, all.data(), sizeof(ChunkDesc) * (size_t)total, cudaMemcpyHostToDevice, h->stream));
    CU_TRY(h, cudaStreamSynchronize(h->stream));
    return DSFACTO_OK;
}

// The strata [L0, L1) of one epoch (inner rounds for the round sweep, row blocks for the row-block
// sweep; the whole sweep is [0, p)), then the return from the scaled state to plain parameters.
void run_sgd_phase(dsfacto *h, int64_t L0, int64_t L1) {
    h->model_version += 1;   // w and V change: the views of the recompute pass are out of date
    SgdArgs a{};
    a.ent = h->d_ent; a.xw = h->d_xw; a.A = h->d_A; a.G = h->d_G; a.w = h->d_w; a.V = h->d_V;
    a.S = h->d_S; a.Tb = h->d_Tb; a.Tw = h->d_Tw; a.TS = h->d_TS; a.records = h->d_records;
    a.run_count = h->d_run_count;
    a.n = h->n; a.d = h->d; a.jbits = h->jbits; a.chunk_len = h->chunk_len; a.block_len = h->block_len; a.spin_limit = h->spin_limit;
    a.h = h->h; a.lambda_v = h->lambda_v;
    const double ew = (double)h->h * (double)h->lambda_w;
    const double log1m_ew = std::log1p(-ew);           // log(1 - ew); -inf / NaN for absurd steps, which then diverge
    a.kappa_w = (float)(-log1m_ew / std::log(2.0));
    // One launch for the whole range: chunks are taken in sweep order (row block by row block, or round
    // by round) and a tile waits only for the earlier tiles of its own column block.  The counters of
    // finished tiles are cumulative over the sweep, so they are cleared at its first launch only; the
    // ticket counter restarts with every launch.
    // With a segmented plan (second schedule on the row-block sweep) a launch is one segment, whose chunks count
    // their earlier tiles from the segment's start: all words are cleared every time.
    int64_t first = L0, last = L1;
    if (h->plan_segments > 0) { first = L0 / h->refresh_every; last = first + 1; }
    if (L0 == 0 || h->plan_segments > 0) cudaMemsetAsync(h->d_sync, 0, sizeof(int) * sync_words(h->p), h->stream);
    else cudaMemsetAsync(h->d_sync + kSyncTicket, 0, sizeof(int), h->stream);
    a.sync = h->d_sync;
    const int64_t chunks = h->launch_ptr[(size_t)last] - h->launch_ptr[(size_t)first];
    a.desc = h->d_desc + h->launch_ptr[(size_t)first];
    a.nchunks = (int)chunks;
    if (chunks > 0) {
        DSF_DISPATCH(h, launch_sgd, h, a, chunks);
        h->launches += 1;
    }
    {   // back from the scaled state to plain (w, V); folds the tail composites in after a row-block sweep
        const int grid = h->sm_count * 8;
        sgd_finalize_v_kernel<<<grid, kThreads, 0, h->stream>>>(h->d_V, h->d_Tb, h->d_S, h->d_TS, h->d, h->Kp / 4);
        sgd_finalize_w_kernel<<<grid, kThreads, 0, h->stream>>>(h->d_w, h->d_Tw, h->d_S, h->d_TS, h->d, log1m_ew);
        h->launches += 2;
    }
}

template <int LG, int NV>
void launch_finish(dsfacto *h, int grid) {
    finish_kernel<LG, NV><<<grid, kThreads, 0, h->stream>>>(h->n, h->d_A, h->d_lin, h->d_q, h->d_y, h->d_G, h->d_partials,
                                                            h->w0, h->loss);
}

// V and the pairs (w_j, s_j) as the recompute pass reads them: by slot for the training rows when the load
// renumbered the columns of the device CSR, by column index otherwise (and always for rows a caller passes).
// Rebuilt only when the parameters changed since the last time: one pass over V (4 d Kp bytes read, twice
// that with the copy in slot order; tens of microseconds).
void model_view(dsfacto *h, RefreshArgs &a, bool training_rows) {
    const bool by_slot = training_rows && h->slots;
    int64_t &version = by_slot ? h->slot_version : h->pair_version;
    if (version != h->model_version) {
        const int kp4 = h->Kp / 4;
        int gs = 1;
        while (gs < kp4 && gs < 32) gs *= 2;
        const int64_t groups_per_cta = kThreads / gs;
        const int grid = (int)std::min<int64_t>(((int64_t)h->d + groups_per_cta - 1) / groups_per_cta, (int64_t)h->sm_count * 16);
        model_view_kernel<<<grid, kThreads, 0, h->stream>>>(reinterpret_cast<const float4 *>(h->d_V), h->d_w,
                                                             by_slot ? h->d_column_of : nullptr, (int64_t)h->d, kp4, gs,
                                                             by_slot ? reinterpret_cast<float4 *>(h->d_Vs) : nullptr,
                                                             by_slot ? h->d_pair_s : h->d_pair);
        h->launches += 1;
        version = h->model_version;
    }
    a.V = by_slot ? h->d_Vs : h->d_V;
    a.pair = by_slot ? h->d_pair_s : h->d_pair;
}

// Renumbers the columns of the device CSR by frequency (see the kernels).  Decided per load: it pays when
// the factors are larger than an L1 and the pass is long enough to hide the host's sort of d counters.
int order_columns(dsfacto *h) {
    h->slots = false;
    bool on = h->nnz >= ((int64_t)1 << 22) && (size_t)h->d * h->Kp * sizeof(float) >= ((size_t)1 << 20);
    if (const char *env = std::getenv("DSFACTO_COLUMN_ORDER")) on = std::strcmp(env, "0") != 0;
    if (h->column_order == 1) on = true;
    if (h->column_order == 2) on = false;
    if (!on || h->nnz == 0) return DSFACTO_OK;
    const size_t d = (size_t)h->d;
    // counters -> sort keys (most frequent first) with the column indices as values -> the sorted values are
    // the column of every slot; a stable sort, so equal counts keep the order of the column indices
    uint32_t *d_key = nullptr, *d_key_out = nullptr;
    int32_t *d_col = nullptr, *d_slot_of = nullptr;
    void *tmp = nullptr;
    auto cleanup = [&]() {
        dev_free(d_key); dev_free(d_key_out); dev_free(d_col); dev_free(d_slot_of);
        if (tmp) cudaFree(tmp);
        tmp = nullptr;
    };
    int rc;
    if ((rc = dev_alloc(h, &d_key, d)) || (rc = dev_alloc(h, &d_key_out, d)) || (rc = dev_alloc(h, &d_col, d)) ||
        (rc = dev_alloc(h, &d_slot_of, d)) || (rc = dev_alloc(h, &h->d_column_of, d)) ||
        (rc = dev_alloc(h, &h->d_Vs, d * h->Kp)) || (rc = dev_alloc(h, &h->d_pair_s, d))) {
        cleanup();
        return rc;
    }
    auto fail = [&](cudaError_t e) {
        h->err = std::string("column order: ") + cudaGetErrorString(e);
        cudaStreamSynchronize(h->stream);
        cleanup();
        return e == cudaErrorMemoryAllocation ? DSFACTO_ERR_OOM : DSFACTO_ERR_CUDA;
    };
    cudaError_t e;
    size_t tmp_bytes = 0;
    if ((e = cub::DeviceRadixSort::SortPairs(nullptr, tmp_bytes, d_key, d_key_out, d_col, h->d_column_of, (int64_t)d, 0, 32,
                                             h->stream)) != cudaSuccess)
        return fail(e);
    if ((e = cudaMalloc(&tmp, tmp_bytes ? tmp_bytes : 1)) != cudaSuccess) return fail(e);
    const int grid = (int)std::min<int64_t>((h->nnz + kThreads - 1) / kThreads, (int64_t)h->sm_count * 16);
    const int dgrid = (int)std::min<int64_t>(((int64_t)d + kThreads - 1) / kThreads, (int64_t)h->sm_count * 16);
    if ((e = cudaMemsetAsync(d_slot_of, 0, sizeof(int32_t) * d, h->stream)) != cudaSuccess) return fail(e);
    column_count_kernel<<<grid, kThreads, 0, h->stream>>>(h->d_idx, h->nnz, d_slot_of);
    column_keys_kernel<<<dgrid, kThreads, 0, h->stream>>>(d_slot_of, (int64_t)d, d_key, d_col);
    if ((e = cub::DeviceRadixSort::SortPairs(tmp, tmp_bytes, d_key, d_key_out, d_col, h->d_column_of, (int64_t)d, 0, 32,
                                             h->stream)) != cudaSuccess)
        return fail(e);
    column_slots_kernel<<<dgrid, kThreads, 0, h->stream>>>(h->d_column_of, (int64_t)d, d_slot_of);
    column_rename_kernel<<<grid, kThreads, 0, h->stream>>>(h->d_idx, h->nnz, d_slot_of);
    h->launches += 4;
    if ((e = cudaStreamSynchronize(h->stream)) != cudaSuccess || (e = cudaGetLastError()) != cudaSuccess) return fail(e);
    cleanup();
    h->slots = true;
    return DSFACTO_OK;
}

// Column shard, first half of the recompute pass: a_i, lin_i, q_i over the shard's own columns.
int run_partial_refresh(dsfacto *h) {
    RefreshArgs a{};
    a.n = h->n; a.indptr = h->d_indptr; a.idx = h->d_idx; a.val = h->d_val; a.y = h->d_y;
    model_view(h, a, true);
    a.A = h->d_A; a.G = h->d_G; a.f_out = nullptr;
    a.lin_out = h->d_lin; a.q_out = h->d_q;
    a.partials = h->d_partials; a.w0 = h->w0; a.loss = h->loss;
    DSF_DISPATCH_REFRESH(h, h, a, kPartial, h->refresh_grid);
    h->launches += 1;
    cudaEventRecord(h->ev[2], h->stream);   // (the epoch's phase timers expect both marks)
    cudaEventRecord(h->ev[3], h->stream);
    CU_TRY(h, cudaStreamSynchronize(h->stream));
    CU_TRY(h, cudaGetLastError());
    h->awaiting_sum = true;
    return DSFACTO_OK;
}

// Column shard, second half: the totals [A | lin | q] are in place; f, loss, G, the two sums, and the squared
// norms of the shard's own columns.
int run_finish(dsfacto *h) {
    DSF_DISPATCH(h, launch_finish, h, h->refresh_grid);
    reduce2_kernel<<<1, kThreads, 0, h->stream>>>(h->d_partials, h->refresh_grid, h->d_scal);
    double *np = h->d_partials + 2 * (size_t)h->refresh_grid;
    const int64_t cols = h->col_hi - h->col_lo;
    sqnorm_kernel<<<h->norm_grid, kThreads, 0, h->stream>>>(h->d_w + h->col_lo, cols, h->d_V + (size_t)h->col_lo * h->Kp,
                                                            cols * h->Kp, np);
    reduce2_kernel<<<1, kThreads, 0, h->stream>>>(np, h->norm_grid, h->d_scal + 2);
    h->launches += 4;
    double s[4];
    CU_TRY(h, cudaMemcpyAsync(s, h->d_scal, sizeof s, cudaMemcpyDeviceToHost, h->stream));
    CU_TRY(h, cudaStreamSynchronize(h->stream));
    CU_TRY(h, cudaGetLastError());
    h->loss_sum = s[0]; h->g_sum = s[1]; h->w2 = s[2]; h->v2 = s[3];
    // the regulariser share of the other shards is missing here: the caller adds the shares up
    h->objective = s[0] / (double)h->n + 0.5 * (double)h->lambda_w * s[2] + 0.5 * (double)h->lambda_v * s[3];
    h->awaiting_sum = false;
    return DSFACTO_OK;
}

// recompute pass + norms + objective; ends with a stream sync and the four sums on the host
int run_refresh(dsfacto *h, bool timed) {
    if (h->nshards > 1) return run_partial_refresh(h);
    RefreshArgs a{};
    a.n = h->n; a.indptr = h->d_indptr; a.idx = h->d_idx; a.val = h->d_val; a.y = h->d_y;
    model_view(h, a, true);
    a.A = h->d_A; a.G = h->d_G; a.f_out = nullptr;
    a.partials = h->d_partials; a.w0 = h->w0; a.loss = h->loss;
    DSF_DISPATCH_REFRESH(h, h, a, kTrain, h->refresh_grid);
    reduce2_kernel<<<1, kThreads, 0, h->stream>>>(h->d_partials, h->refresh_grid, h->d_scal);
    if (timed) cudaEventRecord(h->ev[2], h->stream);
    double *np = h->d_partials + 2 * (size_t)h->refresh_grid;
    sqnorm_kernel<<<h->norm_grid, kThreads, 0, h->stream>>>(h->d_w, h->d, h->d_V, (int64_t)h->d * h->Kp, np);
    reduce2_kernel<<<1, kThreads, 0, h->stream>>>(np, h->norm_grid, h->d_scal + 2);
    h->launches += 4;
    if (timed) cudaEventRecord(h->ev[3], h->stream);
    double s[4];
    CU_TRY(h, cudaMemcpyAsync(s, h->d_scal, sizeof s, cudaMemcpyDeviceToHost, h->stream));
    CU_TRY(h, cudaStreamSynchronize(h->stream));
    CU_TRY(h, cudaGetLastError());
    h->loss_sum = s[0]; h->g_sum = s[1]; h->w2 = s[2]; h->v2 = s[3];
    h->objective = s[0] / (double)h->n + 0.5 * (double)h->lambda_w * s[2] + 0.5 * (double)h->lambda_v * s[3];
    return DSFACTO_OK;
}

// V padded (d x Kp) <-> caller layout (d x K)
int upload_V(dsfacto *h, const float *V) {
    h->model_version += 1;
    if (h->Kp == h->K) {
        CU_TRY(h, cudaMemcpyAsync(h->d_V, V, sizeof(float) * (size_t)h->d * h->K, cudaMemcpyHostToDevice, h->stream));
    } else {
        CU_TRY(h, cudaMemsetAsync(h->d_V, 0, sizeof(float) * (size_t)h->d * h->Kp, h->stream));
        CU_TRY(h, cudaMemcpy2DAsync(h->d_V, sizeof(float) * h->Kp, V, sizeof(float) * h->K, sizeof(float) * h->K,
                                    (size_t)h->d, cudaMemcpyHostToDevice, h->stream));
    }
    CU_TRY(h, cudaStreamSynchronize(h->stream));
    return DSFACTO_OK;
}
int download_rows(dsfacto *h, float *dst, const float *src_dev, int64_t rows) {
    if (h->Kp == h->K) {
        CU_TRY(h, cudaMemcpyAsync(dst, src_dev, sizeof(float) * (size_t)rows * h->K, cudaMemcpyDeviceToHost, h->stream));
    } else {
        CU_TRY(h, cudaMemcpy2DAsync(dst, sizeof(float) * h->K, src_dev, sizeof(float) * h->Kp, sizeof(float) * h->K,
                                    (size_t)rows, cudaMemcpyDeviceToHost, h->stream));
    }
    CU_TRY(h, cudaStreamSynchronize(h->stream));
    return DSFACTO_OK;
}

// CSR checks shared by load_csr and predict.  Returns DSFACTO_OK or DSFACTO_ERR_INVALID_CSR.
int validate_csr(int64_t m, int32_t d, const int64_t *indptr, const int32_t *indices, const float *values) {
    if (indptr[0] != 0) return DSFACTO_ERR_INVALID_CSR;
    int bad = 0;
#pragma omp parallel for schedule(static) reduction(| : bad)
    for (int64_t i = 0; i < m; ++i) {
        const int64_t b = indptr[i], e = indptr[i + 1];
        if (e < b) { bad |= 1; continue; }
        int32_t prev = -1;
        for (int64_t t = b; t < e; ++t) {
            const int32_t j = indices[t];
            if (j <= prev || j >= d) bad |= 1;
            prev = j;
            if (!std::isfinite(values[t])) bad |= 1;
        }
    }
    return bad ? DSFACTO_ERR_INVALID_CSR : DSFACTO_OK;
}

// ---------------------------------------------------------------------------------------------
// Host tile bucketer.  Output order: tiles by (round s, row block r); inside a tile by (column,
// row).  Three passes over the stored entries: count per (thread, tile), scatter (keeps rows
// ascending inside a tile because threads own ascending row ranges), then a stable counting sort
// by local column inside every tile.
// ---------------------------------------------------------------------------------------------
void column_blocks(const dsfacto *h, std::vector<int32_t> &cb);

int bucket_tiles(dsfacto *h, const int64_t *indptr, const int32_t *indices, const float *values,
                 HostBuf<uint2> &ent, HostBuf<float> &xw, SgdPlanBuild *pb) {
    const int64_t n = h->n, nnz = indptr[n];
    const int32_t d = h->d, p = h->p;
    const int64_t nt = (int64_t)p * p;
    const bool wide = h->wide;
    const int jbits = h->jbits;
    int T = omp_get_max_threads();
    if (T > 64) T = 64;
    if ((int64_t)T > n) T = (int)std::max<int64_t>(1, n);

    std::vector<int32_t> cb;  // column block of every column
    std::vector<int64_t> rs;  // thread k owns rows [rs[k], rs[k+1]) chosen to balance stored entries
    try {
        column_blocks(h, cb);
        rs.resize((size_t)T + 1);
    } catch (const std::bad_alloc &) { return DSFACTO_ERR_OOM; }
    rs[0] = 0;
    for (int k = 1; k < T; ++k) {
        const int64_t target = (int64_t)((__int128)nnz * k / T);
        rs[k] = std::lower_bound(indptr, indptr + n + 1, target) - indptr;
        if (rs[k] > n) rs[k] = n;
        if (rs[k] < rs[k - 1]) rs[k] = rs[k - 1];
    }
    rs[T] = n;

    std::vector<uint32_t> counts;
    HostBuf<uint2> tmp_e;
    HostBuf<float> tmp_x;
    try {
        counts.assign((size_t)T * nt, 0u);
        if (!tmp_e.alloc((size_t)nnz) || (wide && !tmp_x.alloc((size_t)nnz)) || !ent.alloc((size_t)nnz) ||
            (wide && !xw.alloc((size_t)nnz)))
            return DSFACTO_ERR_OOM;
    } catch (const std::bad_alloc &) {
        return DSFACTO_ERR_OOM;
    }
    try { h->tile_ptr.assign((size_t)nt + 1, 0); } catch (const std::bad_alloc &) { return DSFACTO_ERR_OOM; }

#pragma omp parallel num_threads(T)
    {
        const int k = omp_get_thread_num();
        uint32_t *cnt = counts.data() + (size_t)k * nt;
        int64_t r = 0;
        for (int64_t i = rs[k]; i < rs[k + 1]; ++i) {
            while (i >= h->row_start[r + 1]) ++r;
            for (int64_t e = indptr[i]; e < indptr[i + 1]; ++e) {
                cnt[tile_slot(h, r, cb[indices[e]])] += 1;
            }
        }
    }
    // offsets: tile-major, thread-minor
    {
        int64_t run = 0;
        for (int64_t t = 0; t < nt; ++t) {
            h->tile_ptr[t] = run;
            for (int k = 0; k < T; ++k) run += counts[(size_t)k * nt + t];
        }
        h->tile_ptr[nt] = run;
    }
    std::vector<int64_t> offs;
    try { offs.resize((size_t)T * nt); } catch (const std::bad_alloc &) { return DSFACTO_ERR_OOM; }
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < nt; ++t) {
        int64_t run = h->tile_ptr[t];
        for (int k = 0; k < T; ++k) { offs[(size_t)k * nt + t] = run; run += counts[(size_t)k * nt + t]; }
    }
#pragma omp parallel num_threads(T)
    {
        const int k = omp_get_thread_num();
        int64_t *off = offs.data() + (size_t)k * nt;
        int64_t r = 0;
        for (int64_t i = rs[k]; i < rs[k + 1]; ++i) {
            while (i >= h->row_start[r + 1]) ++r;
            const uint32_t il = (uint32_t)(i - h->row_start[r]);
            for (int64_t e = indptr[i]; e < indptr[i + 1]; ++e) {
                const int32_t j = indices[e];
                const int32_t c = cb[j];
                const int64_t at = off[tile_slot(h, r, c)]++;
                const uint32_t jl = (uint32_t)(j - h->col_start[c]);
                if (wide) { tmp_e[at] = make_uint2(il, jl); tmp_x[at] = values[e]; }
                else {
                    uint32_t xb;
                    std::memcpy(&xb, &values[e], 4);
                    tmp_e[at] = make_uint2((il << jbits) | jl, xb);
                }
            }
        }
    }
    // stable counting sort by local column inside each tile
    const uint32_t jmask = jbits >= 32 ? 0xFFFFFFFFu : ((1u << jbits) - 1u);
    int64_t widest = 0;
    for (int32_t c = 0; c < p; ++c) widest = std::max<int64_t>(widest, h->col_start[c + 1] - h->col_start[c]);
    int sort_failed = 0;
#pragma omp parallel
    {
        std::vector<int64_t> hist;
        bool have = true;
        try { hist.resize((size_t)widest + 1); } catch (const std::bad_alloc &) { have = false; }
        if (!have) {
#pragma omp atomic write
            sort_failed = 1;
        }
#pragma omp barrier
        int stop;
#pragma omp atomic read
        stop = sort_failed;
#pragma omp for schedule(dynamic, 8)
        for (int64_t t = 0; t < nt; ++t) {
            const int64_t b = h->tile_ptr[t], e = h->tile_ptr[t + 1];
            if (b == e || stop) continue;
            int64_t r, c;
            slot_tile(h, t, r, c);
            (void)r;
            const int64_t width = h->col_start[c + 1] - h->col_start[c];
            std::fill(hist.begin(), hist.begin() + width + 1, (int64_t)0);
            for (int64_t q = b; q < e; ++q) {
                const uint32_t jl = wide ? tmp_e[q].y : (tmp_e[q].x & jmask);
                hist[jl + 1] += 1;
            }
            for (int64_t j = 0; j < width; ++j) hist[j + 1] += hist[j];
            for (int64_t q = b; q < e; ++q) {
                const uint32_t jl = wide ? tmp_e[q].y : (tmp_e[q].x & jmask);
                const int64_t at = b + hist[jl]++;
                ent[at] = tmp_e[q];
                if (wide) xw[at] = tmp_x[q];
            }
            plan_tile(h, pb, omp_get_thread_num(), t, b, hist.data(), width);   // hist[j] is now the end of column j
        }
    }
    return sort_failed ? DSFACTO_ERR_OOM : DSFACTO_OK;
}

// ---------------------------------------------------------------------------------------------
// Row-block bucketer (row-block sweep only, where the p tiles of a row block are stored one after
// another).  A row block is a unit of work: its entries are scattered by tile into a thread-local
// buffer that stays in cache (rows stay ascending), then every tile is counting-sorted by local
// column into the output.  Same result, bit for bit, as bucket_tiles; used when there are enough
// row blocks to keep the threads busy.
// ---------------------------------------------------------------------------------------------
struct RowBlockScratch {
    HostBuf<uint2> tmp_e;
    HostBuf<float> tmp_x;
    std::vector<int64_t> fill, hist;
    SgdPlanBuild *plan = nullptr;   // where the chunks of the bucketed tiles go (none: bucketing only)
    int owner = 0;                  // this thread's planner
};

bool use_row_block_bucketer(const dsfacto *h) {
    int T = omp_get_max_threads();
    if (T > 64) T = 64;
    return h->sweep == 1 && h->p >= 2 * T;
}

void column_blocks(const dsfacto *h, std::vector<int32_t> &cb) {
    cb.resize((size_t)h->d);
    for (int32_t c = 0; c < h->p; ++c)
        for (int32_t j = h->col_start[c]; j < h->col_start[c + 1]; ++j) cb[j] = c;
}

// counts per tile (slot order) -> h->tile_ptr; returns the largest number of entries of a row block
int64_t count_tiles_by_row_block(dsfacto *h, const std::vector<int32_t> &cb, const int64_t *indptr, const int32_t *indices) {
    const int64_t p = h->p, nt = p * p;
    try { h->tile_ptr.assign((size_t)nt + 1, 0); } catch (const std::bad_alloc &) { return -1; }
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t r = 0; r < p; ++r) {
        int64_t *cnt = h->tile_ptr.data() + 1 + (p - 1 - r) * p;   // slot (p-1-r)*p + c
        for (int64_t e = indptr[h->row_start[r]]; e < indptr[h->row_start[r + 1]]; ++e) cnt[cb[indices[e]]] += 1;
    }
    for (int64_t t = 0; t < nt; ++t) h->tile_ptr[t + 1] += h->tile_ptr[t];
    int64_t longest = 0;
    for (int64_t r = 0; r < p; ++r)
        longest = std::max(longest, indptr[h->row_start[r + 1]] - indptr[h->row_start[r]]);
    return longest;
}

// Entries of row block r, bucketed, to out_e (and out_x in the wide layout): tile (r, c) at offset
// tile_ptr[slot(r,c)] - tile_ptr[slot(r,0)].
void bucket_row_block(const dsfacto *h, int64_t r, const std::vector<int32_t> &cb, const int64_t *indptr,
                      const int32_t *indices, const float *values, RowBlockScratch &sc, uint2 *out_e, float *out_x) {
    const int64_t p = h->p;
    const bool wide = h->wide;
    const int jbits = h->jbits;
    const int64_t *tp = h->tile_ptr.data() + (p - 1 - r) * p;   // tile (r, c) = [tp[c], tp[c+1])
    const int64_t base = tp[0];
    for (int64_t c = 0; c < p; ++c) sc.fill[(size_t)c] = tp[c] - base;
    uint2 *tmp_e = sc.tmp_e.data();
    float *tmp_x = sc.tmp_x.data();
    for (int64_t i = h->row_start[r]; i < h->row_start[r + 1]; ++i) {
        const uint32_t il = (uint32_t)(i - h->row_start[r]);
        for (int64_t e = indptr[i]; e < indptr[i + 1]; ++e) {
            const int32_t j = indices[e];
            const int32_t c = cb[j];
            const int64_t at = sc.fill[(size_t)c]++;
            const uint32_t jl = (uint32_t)(j - h->col_start[c]);
            if (wide) { tmp_e[at] = make_uint2(il, jl); tmp_x[at] = values[e]; }
            else {
                uint32_t xb;
                std::memcpy(&xb, &values[e], 4);
                tmp_e[at] = make_uint2((il << jbits) | jl, xb);
            }
        }
    }
    const uint32_t jmask = jbits >= 32 ? 0xFFFFFFFFu : ((1u << jbits) - 1u);
    for (int64_t c = 0; c < p; ++c) {
        const int64_t b = tp[c] - base, e = tp[c + 1] - base;
        if (b == e) continue;
        const int64_t width = h->col_start[c + 1] - h->col_start[c];
        std::fill(sc.hist.begin(), sc.hist.begin() + width + 1, (int64_t)0);   // (sized for the widest column block)
        for (int64_t q = b; q < e; ++q) sc.hist[(wide ? tmp_e[q].y : (tmp_e[q].x & jmask)) + 1] += 1;
        for (int64_t j = 0; j < width; ++j) sc.hist[(size_t)j + 1] += sc.hist[(size_t)j];
        for (int64_t q = b; q < e; ++q) {
            const uint32_t jl = wide ? tmp_e[q].y : (tmp_e[q].x & jmask);
            const int64_t at = b + sc.hist[jl]++;
            out_e[at] = tmp_e[q];
            if (wide) out_x[at] = tmp_x[q];
        }
        plan_tile(h, sc.plan, sc.owner, (p - 1 - r) * p + c, tp[c], sc.hist.data(), width);   // hist[j]: end of column j
    }
}

bool alloc_row_block_scratch(const dsfacto *h, RowBlockScratch &sc, int64_t longest) {
    int64_t widest = 0;
    for (int32_t c = 0; c < h->p; ++c) widest = std::max<int64_t>(widest, h->col_start[(size_t)c + 1] - h->col_start[(size_t)c]);
    try {
        sc.fill.assign((size_t)h->p, 0);
        sc.hist.assign((size_t)widest + 1, 0);
    } catch (const std::bad_alloc &) { return false; }
    return sc.tmp_e.alloc((size_t)longest) && (!h->wide || sc.tmp_x.alloc((size_t)longest));
}

// host-only form: the whole entry array in host memory
int bucket_tiles_by_row_block(dsfacto *h, const int64_t *indptr, const int32_t *indices, const float *values,
                              HostBuf<uint2> &ent, HostBuf<float> &xw, SgdPlanBuild *pb) {
    const int64_t nnz = indptr[h->n];
    std::vector<int32_t> cb;
    try { column_blocks(h, cb); } catch (const std::bad_alloc &) { return DSFACTO_ERR_OOM; }
    const int64_t longest = count_tiles_by_row_block(h, cb, indptr, indices);
    if (longest < 0) return DSFACTO_ERR_OOM;
    if (!ent.alloc((size_t)nnz) || (h->wide && !xw.alloc((size_t)nnz))) return DSFACTO_ERR_OOM;
    int failed = 0;
#pragma omp parallel
    {
        RowBlockScratch sc;
        sc.plan = pb;
        sc.owner = omp_get_thread_num();
        if (!alloc_row_block_scratch(h, sc, longest)) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp barrier
        int stop;
#pragma omp atomic read
        stop = failed;
        if (!stop) {
#pragma omp for schedule(dynamic, 1)
            for (int64_t r = h->p - 1; r >= 0; --r) {
                const int64_t base = h->tile_ptr[(size_t)((h->p - 1 - r) * h->p)];
                bucket_row_block(h, r, cb, indptr, indices, values, sc, ent.data() + base, h->wide ? xw.data() + base : nullptr);
            }
        }
    }
    return failed ? DSFACTO_ERR_OOM : DSFACTO_OK;
}

// ---- page-locked staging memory, kept by the process between streamed loads ----
struct StagingArena {
    std::mutex mu;
    void *ptr = nullptr;
    size_t bytes = 0;
};
StagingArena g_staging;

// Streamed form: every thread buckets a row block into page-locked staging memory and sends it to its
// place in the device arrays while the other row blocks are being bucketed, so that neither a host
// copy of the whole entry array nor a copy from pageable memory is needed.  d_ent (and d_xw) must be
// allocated; tile_ptr is set.  Returns after all copies have completed.
// *no_staging is set when the page-locked staging memory could not be had; nothing has been copied
// then and the caller takes the non-streamed way.
int stream_tiles_by_row_block(dsfacto *h, const std::vector<int32_t> &cb, int64_t longest, const int64_t *indptr,
                              const int32_t *indices, const float *values, bool *no_staging, SgdPlanBuild *pb) {
    *no_staging = false;
    int T = omp_get_max_threads();
    if (T > 64) T = 64;
    const size_t per_entry = sizeof(uint2) + (h->wide ? sizeof(float) : 0);
    const size_t slot_bytes = ((size_t)std::max<int64_t>(longest, 1) * per_entry + 255) / 256 * 256;
    const size_t need = slot_bytes * 2 * (size_t)T;
    std::lock_guard<std::mutex> lock(g_staging.mu);   // one streamed load at a time per process
    if (g_staging.bytes < need) {
        if (g_staging.ptr) cudaFreeHost(g_staging.ptr);
        g_staging.ptr = nullptr;
        g_staging.bytes = 0;
        const char *env = std::getenv("DSFACTO_LOAD");   // "nostaging": behave as if the allocation had failed (tests)
        const bool refuse = env && std::strcmp(env, "nostaging") == 0;
        if (refuse || cudaHostAlloc(&g_staging.ptr, need, cudaHostAllocPortable) != cudaSuccess) {
            cudaGetLastError();   // not an error of the load: page-locked memory is a limited resource
            g_staging.ptr = nullptr;
            *no_staging = true;
            return DSFACTO_ERR_OOM;
        }
        g_staging.bytes = need;
    }
    char *arena = static_cast<char *>(g_staging.ptr);
    int failed = 0;   // 1: host memory, 2: CUDA
#pragma omp parallel num_threads(T)
    {
        const int k = omp_get_thread_num();
        RowBlockScratch sc;
        sc.plan = pb;
        sc.owner = k;
        cudaStream_t st = nullptr;
        cudaEvent_t ev[2] = {nullptr, nullptr};
        bool used[2] = {false, false};
        int mine = 0;
        if (!alloc_row_block_scratch(h, sc, longest)) mine = 1;
        if (!mine && (cudaSetDevice(h->device) != cudaSuccess ||
                      cudaStreamCreateWithFlags(&st, cudaStreamNonBlocking) != cudaSuccess ||
                      cudaEventCreateWithFlags(&ev[0], cudaEventDisableTiming) != cudaSuccess ||
                      cudaEventCreateWithFlags(&ev[1], cudaEventDisableTiming) != cudaSuccess))
            mine = 2;
        if (mine) {
#pragma omp atomic write
            failed = mine;
        }
#pragma omp barrier
        int stop;
#pragma omp atomic read
        stop = failed;
        if (!stop) {
            int turn = 0;
#pragma omp for schedule(dynamic, 1)
            for (int64_t r = h->p - 1; r >= 0; --r) {
                const int64_t s0 = (h->p - 1 - r) * h->p;
                const int64_t base = h->tile_ptr[(size_t)s0], len = h->tile_ptr[(size_t)(s0 + h->p)] - base;
                if (len == 0) continue;
                char *slot = arena + ((size_t)k * 2 + (size_t)turn) * slot_bytes;
                uint2 *se = reinterpret_cast<uint2 *>(slot);
                float *sx = h->wide ? reinterpret_cast<float *>(slot + (size_t)longest * sizeof(uint2)) : nullptr;
                cudaError_t ce = cudaSuccess;
                if (used[turn]) ce = cudaEventSynchronize(ev[turn]);   // the copy that last used this slot is done
                bucket_row_block(h, r, cb, indptr, indices, values, sc, se, sx);
                if (ce == cudaSuccess)
                    ce = cudaMemcpyAsync(h->d_ent + base, se, sizeof(uint2) * (size_t)len, cudaMemcpyHostToDevice, st);
                if (ce == cudaSuccess && h->wide)
                    ce = cudaMemcpyAsync(h->d_xw + base, sx, sizeof(float) * (size_t)len, cudaMemcpyHostToDevice, st);
                if (ce == cudaSuccess) ce = cudaEventRecord(ev[turn], st);
                used[turn] = true;
                turn ^= 1;
                if (ce != cudaSuccess) {
#pragma omp atomic write
                    failed = 2;
                }
            }
        }
        if (st) {
            if (cudaStreamSynchronize(st) != cudaSuccess) {
#pragma omp atomic write
                failed = 2;
            }
            cudaStreamDestroy(st);
        }
        for (auto &e : ev)
            if (e) cudaEventDestroy(e);
    }
    if (failed == 1) return DSFACTO_ERR_OOM;
    if (failed == 2) { h->err = "streamed load: a CUDA call failed"; return DSFACTO_ERR_CUDA; }
    return DSFACTO_OK;
}

}  // namespace

// =============================================================================================
// C ABI
// =============================================================================================
extern "C" {

const char *dsfacto_strerror(int status) {
    switch (status) {
    case DSFACTO_OK: return "ok";
    case DSFACTO_ERR_INVALID_ARG: return "invalid argument";
    case DSFACTO_ERR_INVALID_CSR: return "invalid CSR data or labels";
    case DSFACTO_ERR_NO_DATA: return "no data loaded";
    case DSFACTO_ERR_OOM: return "out of memory";
    case DSFACTO_ERR_CUDA: return "CUDA error";
    case DSFACTO_ERR_DIVERGED: return "objective is not finite";
    default: return "unknown status";
    }
}

const char *dsfacto_last_error(dsfacto_t *h) { return h ? h->err.c_str() : ""; }

static int create_handle(dsfacto_t **out, int64_t n, int32_t d, int32_t K, int32_t p, int32_t loss, float lambda_w,
                         float lambda_v, float eta, uint64_t seed, int32_t shard, int32_t nshards) {
    if (!out) return DSFACTO_ERR_INVALID_ARG;
    *out = nullptr;
    if (nshards < 1 || shard < 0 || shard >= nshards || nshards > p) return DSFACTO_ERR_INVALID_ARG;
    if (n < 1 || n >= ((int64_t)1 << 31) || d < 1 || K < 1 || K > 256 || p < 1 || p > 4096) return DSFACTO_ERR_INVALID_ARG;
    if (loss != DSFACTO_SQUARED && loss != DSFACTO_LOGISTIC) return DSFACTO_ERR_INVALID_ARG;
    if (!(lambda_w >= 0.f) || !(lambda_v >= 0.f) || !(eta > 0.f) || !std::isfinite(lambda_w) ||
        !std::isfinite(lambda_v) || !std::isfinite(eta))
        return DSFACTO_ERR_INVALID_ARG;
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1) return DSFACTO_ERR_CUDA;

    dsfacto *h = new (std::nothrow) dsfacto();
    if (!h) return DSFACTO_ERR_OOM;
    h->n = n; h->d = d; h->K = K; h->p = p; h->loss = loss;
    h->lambda_w = lambda_w; h->lambda_v = lambda_v; h->eta = eta; h->seed = seed;
    h->h = (float)((double)eta / (double)n);
    // factor-row layout: Kp = 4 * LG * NV >= K.  A lane group has at most 16 lanes, so that a warp always
    // works on two entries or more at a time: with K = 128 as one 32-lane group per row every entry paid
    // the scalar and control instructions of a whole warp (C5 epoch 69.1 ms; 57.9 ms with 16 x 2 float4)
    const int q4 = (K + 3) / 4;
    int LG = 1;
    while (LG < q4 && LG < 16) LG <<= 1;
    h->LG = LG;
    h->NV = (q4 + LG - 1) / LG;
    h->Kp = 4 * h->LG * h->NV;
    // The recompute kernel gives a row of 512 bytes and more to 8 lanes (four rows per warp instruction):
    // K = 128 per pass on 400 M entries, 22.3 ms as 32 x 1, 19.8 ms as 16 x 2, 17.5 ms as 8 x 4 float4.
    h->LGr = h->LG; h->NVr = h->NV;
    if (h->Kp >= 128) { h->LGr = 8; h->NVr = h->Kp / 32; }

    int dev = 0;
    cudaGetDevice(&dev);
    h->device = dev;
    cudaDeviceGetAttribute(&h->sm_count, cudaDevAttrMultiProcessorCount, dev);
    if (h->sm_count < 1) h->sm_count = 148;
    cudaDeviceGetAttribute(&h->l2_bytes, cudaDevAttrL2CacheSize, dev);
    if (h->l2_bytes < (1 << 20)) h->l2_bytes = 126 << 20;

    auto fail = [&](int rc) { dsfacto_destroy(h); return rc; };
    if (setup_partition(h)) return fail(DSFACTO_ERR_OOM);
    h->shard = shard; h->nshards = nshards;
    h->cb_lo = (int32_t)(((int64_t)shard * p) / nshards);
    h->cb_hi = (int32_t)(((int64_t)(shard + 1) * p) / nshards);
    h->col_lo = h->col_start[(size_t)h->cb_lo];
    h->col_hi = h->col_start[(size_t)h->cb_hi];

    for (auto &e : h->ev)
        if (cudaEventCreate(&e) != cudaSuccess) return fail(DSFACTO_ERR_CUDA);
    int rc;
    if ((rc = dev_alloc(h, &h->d_w, (size_t)d)) || (rc = dev_alloc(h, &h->d_V, (size_t)d * h->Kp)) ||
        (rc = dev_alloc(h, &h->d_row_start, (size_t)p + 1)) || (rc = dev_alloc(h, &h->d_col_start, (size_t)p + 1)) ||
        (rc = dev_alloc(h, &h->d_scal, 4)) || (rc = dev_alloc(h, &h->d_pair, (size_t)d)))
        return fail(rc);

    std::vector<float> V;
    try { V.resize((size_t)d * K); } catch (const std::bad_alloc &) { return fail(DSFACTO_ERR_OOM); }
#pragma omp parallel for schedule(static)
    for (int64_t e = 0; e < (int64_t)d * K; ++e) V[(size_t)e] = init_factor(seed, (uint64_t)e);
    h->w0 = 0.f;
    if (cudaMemset(h->d_w, 0, sizeof(float) * (size_t)d) != cudaSuccess) return fail(DSFACTO_ERR_CUDA);
    if ((rc = upload_V(h, V.data()))) return fail(rc);
    if (cudaMemcpy(h->d_row_start, h->row_start.data(), sizeof(int64_t) * ((size_t)p + 1), cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemcpy(h->d_col_start, h->col_start.data(), sizeof(int32_t) * ((size_t)p + 1), cudaMemcpyHostToDevice) != cudaSuccess)
        return fail(DSFACTO_ERR_CUDA);
    h->norm_grid = h->sm_count * 8;
    if (const char *env = std::getenv("DSFACTO_SWEEP")) h->sweep = (std::strcmp(env, "round") == 0) ? 0 : 1;
    if ((rc = dev_alloc(h, &h->d_S, (size_t)d))) return fail(rc);
    if (cudaMemset(h->d_S, 0, sizeof(float4) * (size_t)d) != cudaSuccess) return fail(DSFACTO_ERR_CUDA);
    if (h->sweep == 1) {
        if ((rc = dev_alloc(h, &h->d_Tb, (size_t)d * h->Kp)) || (rc = dev_alloc(h, &h->d_Tw, (size_t)d)) ||
            (rc = dev_alloc(h, &h->d_TS, (size_t)d)))
            return fail(rc);
        if (cudaMemset(h->d_Tb, 0, sizeof(float) * (size_t)d * h->Kp) != cudaSuccess ||
            cudaMemset(h->d_Tw, 0, sizeof(float) * (size_t)d) != cudaSuccess ||
            cudaMemset(h->d_TS, 0, sizeof(float4) * (size_t)d) != cudaSuccess)
            return fail(DSFACTO_ERR_CUDA);
    }
    *out = h;
    return DSFACTO_OK;
}

int dsfacto_create(dsfacto_t **out, int64_t n, int32_t d, int32_t K, int32_t p, int32_t loss, float lambda_w,
                   float lambda_v, float eta, uint64_t seed) {
    return create_handle(out, n, d, K, p, loss, lambda_w, lambda_v, eta, seed, 0, 1);
}

int dsfacto_create_shard(dsfacto_t **out, int64_t n, int32_t d, int32_t K, int32_t p, int32_t loss, float lambda_w,
                         float lambda_v, float eta, uint64_t seed, int32_t shard, int32_t nshards) {
    return create_handle(out, n, d, K, p, loss, lambda_w, lambda_v, eta, seed, shard, nshards);
}

int dsfacto_shard_columns(dsfacto_t *h, int32_t *col_lo, int32_t *col_hi) {
    if (!h) return DSFACTO_ERR_INVALID_ARG;
    if (col_lo) *col_lo = h->col_lo;
    if (col_hi) *col_hi = h->col_hi;
    return DSFACTO_OK;
}

void dsfacto_destroy(dsfacto_t *h) {
    if (!h) return;
    cudaStreamSynchronize(h->stream);
    free_data(h);
    dev_free(h->d_w); dev_free(h->d_V); dev_free(h->d_Tb); dev_free(h->d_Tw); dev_free(h->d_S); dev_free(h->d_TS); dev_free(h->d_row_start); dev_free(h->d_col_start); dev_free(h->d_scal); dev_free(h->d_pair);
    for (auto &e : h->ev)
        if (e) cudaEventDestroy(e);
    delete h;
}

int dsfacto_set_stream(dsfacto_t *h, void *cuda_stream) {
    if (!h) return DSFACTO_ERR_INVALID_ARG;
    CU_TRY(h, cudaStreamSynchronize(h->stream));
    h->stream = (cudaStream_t)cuda_stream;
    return DSFACTO_OK;
}

// entries of columns [lo, hi) only, as a CSR over the same rows
static int filter_columns(int64_t n, const int64_t *indptr, const int32_t *indices, const float *values, int32_t lo, int32_t hi,
                          HostBuf<int64_t> &f_indptr, HostBuf<int32_t> &f_indices, HostBuf<float> &f_values) {
    if (!f_indptr.alloc((size_t)n + 1)) return DSFACTO_ERR_OOM;
    int64_t *fp = f_indptr.data();
    fp[0] = 0;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        int64_t cnt = 0;
        for (int64_t t = indptr[i]; t < indptr[i + 1]; ++t) cnt += (indices[t] >= lo && indices[t] < hi) ? 1 : 0;
        fp[i + 1] = cnt;
    }
    for (int64_t i = 0; i < n; ++i) fp[i + 1] += fp[i];
    const int64_t kept = fp[n];
    if (!f_indices.alloc((size_t)std::max<int64_t>(kept, 1)) || !f_values.alloc((size_t)std::max<int64_t>(kept, 1))) return DSFACTO_ERR_OOM;
    int32_t *fi = f_indices.data();
    float *fv = f_values.data();
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        int64_t at = fp[i];
        for (int64_t t = indptr[i]; t < indptr[i + 1]; ++t)
            if (indices[t] >= lo && indices[t] < hi) { fi[at] = indices[t]; fv[at] = values[t]; ++at; }
    }
    return DSFACTO_OK;
}

// ---- tile bucketing on the device (see dsfacto_bucket.cuh) ----
// Whether this load goes that way: packed entry layout, keys of at most 32 bits, enough entries to be worth
// it (DSFACTO_LOAD=device: any non-empty load; any other value of DSFACTO_LOAD: never), and room on the
// device for the sort's buffers next to what the handle keeps.
static bool device_bucketing_wanted(const dsfacto *h, int64_t nnz, const char *load_env) {
    if (nnz <= 0 || h->wide) return false;
    if (bits_for((int64_t)h->p * h->p) + 1 + h->jbits > 32) return false;   // slot, phase, local column
    if (load_env) return std::strcmp(load_env, "device") == 0;
    // (small loads too: their epoch is a chain of dependent tiles per column block, which slots of several row
    // blocks shorten, and only this bucketer builds such slots; it is also the quicker load: create + load +
    // epoch on 20 k / 650 k / 3.7 M entries 1.4 / 8.4 / 15.9 ms against 19.8 / 15.7 / 17.7 ms on the host)
    size_t free_b = 0, total_b = 0;
    if (cudaMemGetInfo(&free_b, &total_b) != cudaSuccess) return false;
    // sort buffers 2 x (4 + 8) bytes and their scratch, then entry records, A, G and the launch plan
    const double need = (double)nnz * (24.0 + 1.0 + 8.0 + 2.0) + (double)h->n * 4.0 * (h->Kp + 2);
    return (double)free_b > need * 1.1;
}

// d_indptr, d_idx, d_val hold the CSR arrays (copies queued on the stream), d_ent is allocated.  Fills
// d_ent, h->tile_ptr and the per-tile pieces of the launch plan.
// Row blocks per slot (a power of two, as log2): merged row blocks make a column's runs longer (see
// dsfacto_bucket.cuh).  Only for the plain plan of the row-block sweep on an unsharded handle; up to 8, as
// many as keep the auxiliary rows of a slot row (re-read by every column block) within 55 % of L2, leave at
// least 16 slot rows, and fit the 32-bit keys and entry records.  Measured sweep times, 1 / 2 / 4 / 8 / 16 row
// blocks per slot: 1.755 G entries, 64-byte rows (45 MB of auxiliary rows per slot row at 8): 29.3 / 28.6 /
// 26.1 / 24.5 / 26.9 ms; 400 M entries, 512-byte rows (64 MB at 8): 26.6 / 24.7 / 23.1 / 22.1 / 24.0 ms.
static int choose_row_merge(const dsfacto *h, int64_t nnz) {
    const int64_t p = h->p;
    const bool segmented = h->refresh_every > 0 && h->refresh_every < p;
    if (h->sweep != 1 || segmented || h->nshards > 1) return 0;
    // Small data sets: their sweep is as long as the chain of dependent slots of a column block, so as many row
    // blocks per slot as there may be (3.7 M entries, p = 64, 1 / 2 / 4 / 8 / 16 per slot: 0.90 / 0.48 / 0.29 / 0.21 /
    // 0.15 ms per sweep; 650 k entries, p = 16: 0.068 -> 0.039 ms; 20 k entries, p = 4: 0.040 -> 0.024 ms).
    const bool small = nnz < kStreamedLoadMinEntries;
    int want = small ? kMaxRowMerge : 8;
    if (h->row_merge > 0) want = h->row_merge;
    if (const char *env = std::getenv("DSFACTO_ROW_MERGE")) {
        const int v = std::atoi(env);
        if (v >= 1 && v <= kMaxRowMerge) want = v;
    }
    int rbits = 0;
    while ((2 << rbits) <= want) {
        const int nb = rbits + 1;
        const int64_t R = (int64_t)1 << nb, slot_rows = (p + R - 1) / R;
        int64_t max_rows = 0;
        for (int64_t sr = 0; sr < slot_rows; ++sr)
            max_rows = std::max(max_rows, h->row_start[(size_t)std::min(p, (sr + 1) * R)] - h->row_start[(size_t)(sr * R)]);
        const bool forced = h->row_merge > 0 || std::getenv("DSFACTO_ROW_MERGE") != nullptr;
        if (bits_for(max_rows) + h->jbits > 32) break;
        if (bits_for(slot_rows * p) + 1 + h->jbits + nb > 32) break;
        if (!forced && ((!small && slot_rows < 16) || (double)max_rows * h->Kp * 4.0 > 0.55 * (double)h->l2_bytes)) break;
        if (slot_rows < 1) break;
        rbits = nb;
    }
    return rbits;
}

static int device_bucket_tiles(dsfacto *h, int64_t nnz, SgdPlanBuild &pb) {
    h->rbits = choose_row_merge(h, nnz);
    const int64_t slot_rows = ((int64_t)h->p + ((int64_t)1 << h->rbits) - 1) >> h->rbits;
    choose_chunk_len(h, nnz, slot_rows);   // merged row blocks: fewer and longer slot rows
    const int64_t nt = slot_rows * h->p;                       // slots of the device entry array
    const int low_bits = 1 + h->jbits + h->rbits;              // key bits below the slot number: phase, local column, row block
    const int kb = bits_for(nt) + low_bits;
    cudaStream_t st = h->stream;
    uint32_t *key[2] = {nullptr, nullptr};
    unsigned long long *pay[2] = {nullptr, nullptr};
    void *tmp = nullptr;
    int64_t *d_tp = nullptr, *d_plan = nullptr, *d_in = nullptr;   // tile pointers; per-tile counts; per-tile starting values
    ChunkDesc *d_out = nullptr;
    auto cleanup = [&]() {
        dev_free(key[0]); dev_free(key[1]); dev_free(pay[0]); dev_free(pay[1]);
        if (tmp) cudaFree(tmp);
        tmp = nullptr;
        dev_free(d_tp); dev_free(d_plan); dev_free(d_in); dev_free(d_out);
    };
    auto fail = [&](cudaError_t e) {
        h->err = std::string("device bucketing: ") + cudaGetErrorString(e);
        cudaStreamSynchronize(st);
        cleanup();
        return e == cudaErrorMemoryAllocation ? DSFACTO_ERR_OOM : DSFACTO_ERR_CUDA;
    };
    int rc;
    if ((rc = dev_alloc(h, &key[0], (size_t)nnz)) || (rc = dev_alloc(h, &key[1], (size_t)nnz)) ||
        (rc = dev_alloc(h, &pay[0], (size_t)nnz)) || (rc = dev_alloc(h, &pay[1], (size_t)nnz)) ||
        (rc = dev_alloc(h, &d_tp, (size_t)nt + 1)) || (rc = dev_alloc(h, &d_plan, 3 * (size_t)nt)) ||
        (rc = dev_alloc(h, &d_in, 4 * (size_t)nt + 1))) {
        cleanup();
        return rc;
    }
    cudaError_t e;
    size_t tmp_bytes = 0;
    if ((e = cub::DeviceRadixSort::SortPairs(nullptr, tmp_bytes, key[0], key[1], pay[0], pay[1], nnz, 0, kb, st)) != cudaSuccess)
        return fail(e);
    if ((e = cudaMalloc(&tmp, tmp_bytes ? tmp_bytes : 1)) != cudaSuccess) return fail(e);

    const int wide_grid = h->sm_count * 16;
    TileKeyArgs ka{};
    ka.n = h->n; ka.indptr = h->d_indptr; ka.idx = h->d_idx; ka.val = h->d_val; ka.d = h->d; ka.p = h->p;
    ka.sweep = h->sweep; ka.jbits = h->jbits; ka.row_start = h->d_row_start; ka.col_start = h->d_col_start;
    ka.rbits = h->rbits; ka.slot_rows = (int32_t)slot_rows;
    ka.key = key[0]; ka.payload = pay[0];
    tile_keys_kernel<<<wide_grid, kThreads, 0, st>>>(ka);
    if ((e = cub::DeviceRadixSort::SortPairs(tmp, tmp_bytes, key[0], key[1], pay[0], pay[1], nnz, 0, kb, st)) != cudaSuccess)
        return fail(e);
    pack_entries_kernel<<<wide_grid, kThreads, 0, st>>>(nnz, key[1], pay[1], h->jbits, h->rbits, h->d_ent);
    tile_bounds_kernel<<<(int)std::min<int64_t>((nt + kThreads) / kThreads, wide_grid), kThreads, 0, st>>>(nnz, key[1], low_bits, nt, d_tp);
    // the chunk plan: count per tile, then write.  The plain plan visits the tiles in slot order, so the kernel
    // can write complete descriptors straight into the handle's array; a plan cut into segments (second
    // schedule) gets the per-tile pieces and is put in order on the host as in the host path.
    const int64_t p = h->p;
    const bool segmented = h->sweep == 1 && h->refresh_every > 0 && h->refresh_every < p;
    TilePlanArgs pa{};
    pa.key = key[1]; pa.tile_ptr = d_tp; pa.ntiles = nt; pa.jbits = h->jbits; pa.chunk_len = h->chunk_len;
    pa.rbits = h->rbits; pa.slot_rows = (int32_t)slot_rows;
    pa.count = d_plan; pa.runs = d_plan + nt; pa.recs = d_plan + 2 * nt;
    pa.p = h->p; pa.sweep = h->sweep; pa.row_start = h->d_row_start; pa.col_start = h->d_col_start;
    plan_tiles_kernel<kPlanCount><<<wide_grid, kThreads, 0, st>>>(pa);
    h->launches += 4;
    std::vector<int64_t> cnt, in;   // cnt: counts, runs, recs per tile; in: first (nt + 1), need, run0, rec0
    try {
        h->tile_ptr.assign((size_t)nt + 1, 0);
        cnt.resize(3 * (size_t)nt);
        in.resize(4 * (size_t)nt + 1);
    } catch (const std::bad_alloc &) { cudaStreamSynchronize(st); cleanup(); return DSFACTO_ERR_OOM; }
    if ((e = cudaMemcpyAsync(h->tile_ptr.data(), d_tp, sizeof(int64_t) * ((size_t)nt + 1), cudaMemcpyDeviceToHost, st)) != cudaSuccess ||
        (e = cudaMemcpyAsync(cnt.data(), d_plan, sizeof(int64_t) * 3 * (size_t)nt, cudaMemcpyDeviceToHost, st)) != cudaSuccess ||
        (e = cudaStreamSynchronize(st)) != cudaSuccess || (e = cudaGetLastError()) != cudaSuccess)
        return fail(e);
    int64_t *first = in.data(), *need = first + nt + 1, *run0 = need + nt, *rec0 = run0 + nt;
    int64_t total = 0, runs = 0, recs = 0;
    std::vector<int64_t> seen;
    try {
        seen.assign((size_t)p, 0);
        if (!segmented) h->launch_ptr.assign((size_t)p + 1, 0);
    } catch (const std::bad_alloc &) { cleanup(); return DSFACTO_ERR_OOM; }
    for (int64_t t = 0; t < nt; ++t) {
        int64_t r, c;
        if (h->rbits > 0) c = t % p;   // (merged row blocks: row-block sweep, slot = slot row x column block)
        else slot_tile(h, t, r, c);
        TileDescRef &ref = pb.refs[(size_t)t];
        ref.owner = 0;
        ref.first = total;
        ref.count = (int32_t)cnt[(size_t)t];
        first[t] = total; need[t] = seen[(size_t)c]; run0[t] = runs; rec0[t] = recs;
        total += cnt[(size_t)t];
        runs += cnt[(size_t)(nt + t)];
        recs += cnt[(size_t)(2 * nt + t)];
        seen[(size_t)c] += cnt[(size_t)t];
        if (!segmented && h->rbits == 0 && (t + 1) % p == 0) h->launch_ptr[(size_t)((t + 1) / p)] = total;
    }
    first[nt] = total;
    // (with merged row blocks the plain plan is one launch over everything: only its two ends are looked up)
    if (!segmented && h->rbits > 0)
        for (int64_t k = 1; k <= p; ++k) h->launch_ptr[(size_t)k] = total;
    if (total >= (int64_t)kTicketStop / 2 || recs >= ((int64_t)1 << 31)) { cleanup(); return DSFACTO_ERR_INVALID_ARG; }
    if ((e = cudaMemcpyAsync(d_in, in.data(), sizeof(int64_t) * in.size(), cudaMemcpyHostToDevice, st)) != cudaSuccess) return fail(e);
    pa.first = d_in; pa.need = d_in + nt + 1; pa.run0 = pa.need + nt; pa.rec0 = pa.run0 + nt;
    if (segmented) {
        if (!pb.bulk.alloc((size_t)total)) { cudaStreamSynchronize(st); cleanup(); return DSFACTO_ERR_OOM; }
        if (total > 0) {
            if ((rc = dev_alloc(h, &d_out, (size_t)total))) { cudaStreamSynchronize(st); cleanup(); return rc; }
            pa.out = d_out;
            plan_tiles_kernel<kPlanPieces><<<wide_grid, kThreads, 0, st>>>(pa);
            h->launches += 1;
            if ((e = cudaMemcpyAsync(pb.bulk.data(), d_out, sizeof(ChunkDesc) * (size_t)total, cudaMemcpyDeviceToHost, st)) != cudaSuccess)
                return fail(e);
        }
    } else {
        // what finish_sgd_plan does for the host paths
        h->plan_segments = 0;
        h->total_chunks = total;
        h->long_runs = runs;
        h->slice_records = recs;
        if ((rc = dev_alloc(h, &h->d_desc, (size_t)total)) ||
            (rc = dev_alloc(h, &h->d_records, (size_t)recs * slice_record_floats(h->Kp))) ||
            (rc = dev_alloc(h, &h->d_run_count, (size_t)runs)) || (rc = dev_alloc(h, &h->d_sync, sync_words((int)p)))) {
            cudaStreamSynchronize(st);
            cleanup();
            return rc;
        }
        if ((e = cudaMemsetAsync(h->d_run_count, 0, sizeof(int) * (size_t)std::max<int64_t>(runs, 1), st)) != cudaSuccess ||
            (e = cudaMemsetAsync(h->d_sync, 0, sizeof(int) * sync_words((int)p), st)) != cudaSuccess)
            return fail(e);
        if (total > 0) {
            pa.out = h->d_desc;
            plan_tiles_kernel<kPlanFull><<<wide_grid, kThreads, 0, st>>>(pa);
            h->launches += 1;
            if (h->debug_extra_need > 0) plan_extra_need_kernel<<<1, 1, 0, st>>>(h->d_desc, h->debug_extra_need);
        }
        pb.finished = true;
    }
    if ((e = cudaStreamSynchronize(st)) != cudaSuccess || (e = cudaGetLastError()) != cudaSuccess) return fail(e);
    cleanup();
    return DSFACTO_OK;
}

// the device copy of the CSR arrays and labels, made before the handle's old data set is let go
struct PendingCsr {
    int64_t *indptr = nullptr;
    int32_t *idx = nullptr;
    float *val = nullptr, *y = nullptr;
    void release() { dev_free(indptr); dev_free(idx); dev_free(val); dev_free(y); }
};
static int load_validated(dsfacto_t *h, const int64_t *indptr, const int32_t *indices, const float *values, const float *y,
                          PendingCsr *pending);

int dsfacto_load_csr(dsfacto_t *h, const int64_t *indptr, const int32_t *indices, const float *values, const float *y) {
    if (!h || !indptr || !y) return DSFACTO_ERR_INVALID_ARG;
    const int64_t n = h->n;
    if (indptr[0] != 0 || indptr[n] < 0) return DSFACTO_ERR_INVALID_CSR;
    const int64_t nnz = indptr[n];
    if (nnz > 0 && (!indices || !values)) return DSFACTO_ERR_INVALID_ARG;
    int rc;
    int bad = 0;
    // A large load sends the CSR arrays to the device while the host checks them (0.1 s of checks against
    // 0.27 s on the link for 1.755 G entries).  The row pointers are checked first, so that the copies read
    // exactly the nnz entries they promise; the copies go into new device arrays, and the handle's old data
    // set is let go only after the checks: a rejected data set leaves the handle as it was.
    PendingCsr pending;
    const bool overlapped = h->nshards == 1 && nnz >= kStreamedLoadMinEntries;
    if (overlapped) {
#pragma omp parallel for schedule(static) reduction(| : bad)
        for (int64_t i = 0; i < n; ++i)
            if (indptr[i + 1] < indptr[i]) bad |= 1;
        if (bad) return DSFACTO_ERR_INVALID_CSR;
        if ((rc = dev_alloc(h, &pending.indptr, (size_t)n + 1)) || (rc = dev_alloc(h, &pending.idx, (size_t)nnz)) ||
            (rc = dev_alloc(h, &pending.val, (size_t)nnz)) || (rc = dev_alloc(h, &pending.y, (size_t)n))) {
            pending.release();
            return rc;
        }
        cudaError_t e;
        if ((e = cudaMemcpyAsync(pending.indptr, indptr, sizeof(int64_t) * ((size_t)n + 1), cudaMemcpyHostToDevice, h->stream)) != cudaSuccess ||
            (e = cudaMemcpyAsync(pending.idx, indices, sizeof(int32_t) * (size_t)nnz, cudaMemcpyHostToDevice, h->stream)) != cudaSuccess ||
            (e = cudaMemcpyAsync(pending.val, values, sizeof(float) * (size_t)nnz, cudaMemcpyHostToDevice, h->stream)) != cudaSuccess ||
            (e = cudaMemcpyAsync(pending.y, y, sizeof(float) * (size_t)n, cudaMemcpyHostToDevice, h->stream)) != cudaSuccess) {
            h->err = std::string("dsfacto_load_csr: ") + cudaGetErrorString(e);
            cudaStreamSynchronize(h->stream);
            pending.release();
            return DSFACTO_ERR_CUDA;
        }
    }
    rc = validate_csr(n, h->d, indptr, indices, values);
#pragma omp parallel for schedule(static) reduction(| : bad)
    for (int64_t i = 0; i < n; ++i)
        if (!std::isfinite(y[i])) bad |= 1;
    if (!rc && bad) rc = DSFACTO_ERR_INVALID_CSR;
    if (rc) {
        if (overlapped) { cudaStreamSynchronize(h->stream); pending.release(); }
        return rc;
    }

    // a column shard keeps only the stored entries of its own columns (all rows stay, some become empty)
    HostBuf<int64_t> f_indptr;
    HostBuf<int32_t> f_indices;
    HostBuf<float> f_values;
    if (h->nshards > 1) {
        rc = filter_columns(n, indptr, indices, values, h->col_lo, h->col_hi, f_indptr, f_indices, f_values);
        if (rc) return rc;
        indptr = f_indptr.data(); indices = f_indices.data(); values = f_values.data();
    }
    return load_validated(h, indptr, indices, values, y, overlapped ? &pending : nullptr);
}

static int load_validated(dsfacto_t *h, const int64_t *indptr, const int32_t *indices, const float *values, const float *y,
                          PendingCsr *pending) {
    const int64_t n = h->n, nnz = indptr[n];
    int rc = DSFACTO_OK;
    if (!pending) CU_TRY(h, cudaStreamSynchronize(h->stream));   // (the copies of a pending CSR are still under way)
    free_data(h);
    h->nnz = nnz;
    h->refresh_grid = refresh_grid_for(h, n);
    const size_t cnt = (size_t)std::max<int64_t>(nnz, 1);
    cudaStream_t st = h->stream;
    if (pending) {
        h->d_indptr = pending->indptr; h->d_idx = pending->idx; h->d_val = pending->val; h->d_y = pending->y;
        *pending = PendingCsr();
    } else {
        // the CSR copy for the recompute pass goes out first: from page-locked caller memory it overlaps
        // the host bucketing below
        if ((rc = dev_alloc(h, &h->d_indptr, (size_t)n + 1)) || (rc = dev_alloc(h, &h->d_idx, cnt)) ||
            (rc = dev_alloc(h, &h->d_val, cnt)) || (rc = dev_alloc(h, &h->d_y, (size_t)n))) {
            free_data(h);
            return rc;
        }
        CU_TRY_LOAD(h, cudaMemcpyAsync(h->d_indptr, indptr, sizeof(int64_t) * ((size_t)n + 1), cudaMemcpyHostToDevice, st));
        if (nnz > 0) {
            CU_TRY_LOAD(h, cudaMemcpyAsync(h->d_idx, indices, sizeof(int32_t) * (size_t)nnz, cudaMemcpyHostToDevice, st));
            CU_TRY_LOAD(h, cudaMemcpyAsync(h->d_val, values, sizeof(float) * (size_t)nnz, cudaMemcpyHostToDevice, st));
        }
        CU_TRY_LOAD(h, cudaMemcpyAsync(h->d_y, y, sizeof(float) * (size_t)n, cudaMemcpyHostToDevice, st));
    }

    // Tile lists.  With enough row blocks (row-block sweep) a row block is the unit of work; large
    // loads are then streamed: bucketed into page-locked staging memory and copied to the device
    // block by block, overlapping the bucketing of the other blocks.  DSFACTO_LOAD=stream takes that
    // way for small loads too, DSFACTO_LOAD=simple never.
    HostBuf<uint2> ent;
    HostBuf<float> xw;
    std::vector<int32_t> cb;
    int64_t longest = 0;
    choose_chunk_len(h, nnz, h->p);
    SgdPlanBuild pb;   // the chunks of the stratum SGD launches are cut while the tiles are bucketed
    if (!init_plan_build(h, pb, omp_get_max_threads())) { cudaStreamSynchronize(st); free_data(h); return DSFACTO_ERR_OOM; }
    const bool by_row_block = use_row_block_bucketer(h);
    const char *load_env = std::getenv("DSFACTO_LOAD");
    const bool on_device = device_bucketing_wanted(h, nnz, load_env);
    const bool streamed = !on_device && by_row_block && nnz > 0 &&
                          (nnz >= kStreamedLoadMinEntries ||
                           (load_env && (std::strcmp(load_env, "stream") == 0 || std::strcmp(load_env, "nostaging") == 0))) &&
                          !(load_env && std::strcmp(load_env, "simple") == 0);
    if (on_device) {
        // bucketed below, once the entry array is allocated; the tile pointers get their size here
        try { h->tile_ptr.assign((size_t)h->p * h->p + 1, 0); }
        catch (const std::bad_alloc &) { cudaStreamSynchronize(st); free_data(h); return DSFACTO_ERR_OOM; }
    } else if (streamed) {
        try { column_blocks(h, cb); } catch (const std::bad_alloc &) { cudaStreamSynchronize(st); free_data(h); return DSFACTO_ERR_OOM; }
        longest = count_tiles_by_row_block(h, cb, indptr, indices);
        if (longest < 0) { cudaStreamSynchronize(st); free_data(h); return DSFACTO_ERR_OOM; }
    } else {
        rc = by_row_block ? bucket_tiles_by_row_block(h, indptr, indices, values, ent, xw, &pb)
                          : bucket_tiles(h, indptr, indices, values, ent, xw, &pb);
        if (rc) { cudaStreamSynchronize(st); free_data(h); return rc; }
    }
    h->nnz = nnz;   // (free_data on an error path above resets it)
    if ((rc = dev_alloc(h, &h->d_A, (size_t)n * h->Kp + (h->nshards > 1 ? 2 * (size_t)n : 0))) || (rc = dev_alloc(h, &h->d_G, (size_t)n)) ||
        (rc = dev_alloc(h, &h->d_tile_ptr, h->tile_ptr.size())) || (rc = dev_alloc(h, &h->d_ent, cnt + 4)) ||
        (rc = dev_alloc(h, &h->d_partials, 2 * ((size_t)h->refresh_grid + (size_t)h->norm_grid))) ||
        (h->wide && (rc = dev_alloc(h, &h->d_xw, cnt + 4)))) {
        cudaStreamSynchronize(st);
        free_data(h);
        return rc;
    }
    bool copy_from_host = !streamed && !on_device;
    if (on_device) {
        if ((rc = device_bucket_tiles(h, nnz, pb))) { cudaStreamSynchronize(st); free_data(h); return rc; }
    }
    if (streamed) {
        bool no_staging = false;
        rc = stream_tiles_by_row_block(h, cb, longest, indptr, indices, values, &no_staging, &pb);
        if (rc && no_staging) {   // no page-locked memory to be had: bucket into pageable memory, one copy
            if (!init_plan_build(h, pb, omp_get_max_threads())) { cudaStreamSynchronize(st); free_data(h); return DSFACTO_ERR_OOM; }
            rc = bucket_tiles_by_row_block(h, indptr, indices, values, ent, xw, &pb);
            copy_from_host = true;
        }
        if (rc) { cudaStreamSynchronize(st); free_data(h); return rc; }
    }
    if (copy_from_host && nnz > 0) {
        CU_TRY_LOAD(h, cudaMemcpyAsync(h->d_ent, ent.data(), sizeof(uint2) * (size_t)nnz, cudaMemcpyHostToDevice, st));
        if (h->wide) CU_TRY_LOAD(h, cudaMemcpyAsync(h->d_xw, xw.data(), sizeof(float) * (size_t)nnz, cudaMemcpyHostToDevice, st));
    }
    CU_TRY_LOAD(h, cudaMemcpyAsync(h->d_tile_ptr, h->tile_ptr.data(), sizeof(int64_t) * h->tile_ptr.size(), cudaMemcpyHostToDevice, st));
    CU_TRY_LOAD(h, cudaStreamSynchronize(st));
    if (!pb.finished && (rc = finish_sgd_plan(h, pb))) { free_data(h); return rc; }
    if ((rc = order_columns(h))) { free_data(h); return rc; }
    {
        const int64_t nt1 = (int64_t)h->p * h->p + 1, plan_bytes = (int64_t)sizeof(ChunkDesc) * h->total_chunks;
        const int64_t csr_bytes = 8 * (n + 1) + 8 * nnz + 4 * n;   // indptr, idx, val, y
        const int64_t nt = nt1 - 1;
        h->load_info[0] = on_device ? 2 : (copy_from_host ? 0 : 1);
        // device bucketing: the per-tile counts come back, the per-tile starting values go out; only a plan
        // that is cut into segments sends its descriptors to the host and back
        h->load_info[1] = csr_bytes + 8 * nt1 + (on_device ? 8 * (4 * nt + 1) + (pb.finished ? 0 : plan_bytes) : plan_bytes + (h->wide ? 12 : 8) * nnz);
        h->load_info[2] = on_device ? 8 * nt1 + 24 * nt + (pb.finished ? 0 : plan_bytes) : 0;
    }
    h->failed = false;
    h->loaded = true;
    if (h->nshards > 1) {   // the partial sums sit right behind A, so that one buffer holds what the shards exchange
        h->d_lin = h->d_A + (size_t)n * h->Kp;
        h->d_q = h->d_lin + n;
    }
    rc = run_refresh(h, false);
    if (rc) return rc;
    if (h->nshards > 1) return DSFACTO_OK;   // no objective before the shards' partial sums have been added up
    return std::isfinite(h->objective) ? DSFACTO_OK : DSFACTO_ERR_DIVERGED;
}

// An SGD launch gave up (a bounded wait ran out, or a check of the debug build failed): the warps left
// in the middle of the sweep, so the parameters and the scaled state are a mixture.  The bookkeeping of
// the sweep is cleared and the handle refuses further epochs until the parameters are set again
// (dsfacto_set_params with w and V) or a data set is loaded after that.
static int sgd_gave_up(dsfacto *h, const int code[3]) {
    h->failed = true;
    char buf[160];
    if (code[0] == 1) std::snprintf(buf, sizeof buf, "stratum SGD: a wait for an earlier tile of the same column block timed out");
    else if (code[0] == 2) std::snprintf(buf, sizeof buf, "stratum SGD: a copy of entry records into shared memory did not arrive");
    else std::snprintf(buf, sizeof buf, "stratum SGD: debug check %d failed (value %d)", code[1], code[2]);
    h->err = buf;
    const size_t d = (size_t)h->d;
    cudaMemsetAsync(h->d_run_count, 0, sizeof(int) * (size_t)std::max<int64_t>(h->long_runs, 1), h->stream);
    cudaMemsetAsync(h->d_sync, 0, sizeof(int) * sync_words(h->p), h->stream);
    cudaMemsetAsync(h->d_S, 0, sizeof(float4) * d, h->stream);
    if (h->d_TS) {
        cudaMemsetAsync(h->d_TS, 0, sizeof(float4) * d, h->stream);
        cudaMemsetAsync(h->d_Tw, 0, sizeof(float) * d, h->stream);
        cudaMemsetAsync(h->d_Tb, 0, sizeof(float) * d * h->Kp, h->stream);
    }
    cudaStreamSynchronize(h->stream);
    return DSFACTO_ERR_CUDA;
}

static int epoch_impl(dsfacto_t *h);

int dsfacto_epoch(dsfacto_t *h) {
    if (!h) return DSFACTO_ERR_INVALID_ARG;
    if (!h->loaded) return DSFACTO_ERR_NO_DATA;
    if (h->failed) { h->err = "the last stratum SGD launch gave up: set the parameters again (dsfacto_set_params) first"; return DSFACTO_ERR_CUDA; }
    if (h->nshards > 1) return DSFACTO_ERR_INVALID_ARG;   // a column shard advances with dsfacto_shard_epoch_begin / _end
    return epoch_impl(h);
}

static int epoch_impl(dsfacto_t *h) {
    cudaStream_t st = h->stream;
    CU_TRY(h, cudaEventRecord(h->ev[0], st));
    const int64_t p = h->p;
    const int64_t every = (h->refresh_every > 0 && h->refresh_every < p) ? h->refresh_every : p;
    float t01 = 0, t12 = 0, t23 = 0;
    int rc = DSFACTO_OK;
    for (int64_t L0 = 0; L0 < p; L0 += every) {
        const int64_t L1 = std::min(L0 + every, p);
        if (L0 > 0) CU_TRY(h, cudaEventRecord(h->ev[0], st));
        // w0 step with the frozen multipliers: the share of the epoch's step that belongs to these rounds
        h->w0 = (float)((double)h->w0 - (double)h->h * ((double)(L1 - L0) / (double)p) * h->g_sum);
        run_sgd_phase(h, L0, L1);
        CU_TRY(h, cudaEventRecord(h->ev[1], st));
        rc = run_refresh(h, true);
        if (rc) return rc;
        float a01 = 0, a12 = 0, a23 = 0;
        cudaEventElapsedTime(&a01, h->ev[0], h->ev[1]);
        cudaEventElapsedTime(&a12, h->ev[1], h->ev[2]);
        cudaEventElapsedTime(&a23, h->ev[2], h->ev[3]);
        t01 += a01; t12 += a12; t23 += a23;
    }
    int sgd_error[3] = {0, 0, 0};  // set by the SGD kernel if one of its bounded waits ran out
    CU_TRY(h, cudaMemcpy(sgd_error, h->d_sync + kSyncError, sizeof sgd_error, cudaMemcpyDeviceToHost));
    if (sgd_error[0]) return sgd_gave_up(h, sgd_error);
    h->ms[0] = t01 + t12 + t23; h->ms[1] = t01; h->ms[2] = t12; h->ms[3] = t23;
    if (h->nshards > 1) return DSFACTO_OK;   // the objective exists only after the shards' sums have been added up
    return std::isfinite(h->objective) ? DSFACTO_OK : DSFACTO_ERR_DIVERGED;
}

// ---- column shards ----
int dsfacto_shard_partial_count(dsfacto_t *h, int64_t *count) {
    if (!h || !count) return DSFACTO_ERR_INVALID_ARG;
    *count = h->n * ((int64_t)h->Kp + 2);
    return DSFACTO_OK;
}

int dsfacto_shard_epoch_begin(dsfacto_t *h) {
    if (!h) return DSFACTO_ERR_INVALID_ARG;
    if (h->nshards < 2) return DSFACTO_ERR_INVALID_ARG;
    if (!h->loaded) return DSFACTO_ERR_NO_DATA;
    if (h->awaiting_sum) { h->err = "the summed auxiliaries of the last step have not been handed in (dsfacto_shard_epoch_end)"; return DSFACTO_ERR_INVALID_ARG; }
    return epoch_impl(h);   // w0 step, the strata over the shard's own tiles, then the partial recompute pass
}

int dsfacto_shard_partial(dsfacto_t *h, float *dst_dev, int64_t count) {
    if (!h || !dst_dev) return DSFACTO_ERR_INVALID_ARG;
    if (h->nshards < 2 || !h->loaded) return DSFACTO_ERR_INVALID_ARG;
    if (count != h->n * ((int64_t)h->Kp + 2)) return DSFACTO_ERR_INVALID_ARG;
    CU_TRY(h, cudaMemcpyAsync(dst_dev, h->d_A, sizeof(float) * (size_t)count, cudaMemcpyDeviceToDevice, h->stream));
    CU_TRY(h, cudaStreamSynchronize(h->stream));
    return DSFACTO_OK;
}

int dsfacto_shard_epoch_end(dsfacto_t *h, const float *summed_dev, int64_t count, double sums[4]) {
    if (!h || !summed_dev || !sums) return DSFACTO_ERR_INVALID_ARG;
    if (h->nshards < 2 || !h->loaded) return DSFACTO_ERR_INVALID_ARG;
    if (count != h->n * ((int64_t)h->Kp + 2)) return DSFACTO_ERR_INVALID_ARG;
    CU_TRY(h, cudaMemcpyAsync(h->d_A, summed_dev, sizeof(float) * (size_t)count, cudaMemcpyDeviceToDevice, h->stream));
    const int rc = run_finish(h);
    if (rc) return rc;
    sums[0] = h->loss_sum; sums[1] = h->g_sum; sums[2] = h->w2; sums[3] = h->v2;
    return DSFACTO_OK;
}

int dsfacto_bucket_host_shard(int64_t n, int32_t d, int32_t p, int32_t shard, int32_t nshards, const int64_t *indptr,
                              const int32_t *indices, const float *values, int64_t *kept, int64_t *tile_ptr, int32_t *rows,
                              int32_t *cols, float *vals) {
    if (n < 1 || n >= ((int64_t)1 << 31) || d < 1 || p < 1 || p > 4096 || !indptr || !tile_ptr || !kept) return DSFACTO_ERR_INVALID_ARG;
    if (nshards < 1 || shard < 0 || shard >= nshards || nshards > p) return DSFACTO_ERR_INVALID_ARG;
    if (indptr[0] != 0 || indptr[n] < 0) return DSFACTO_ERR_INVALID_CSR;
    if (indptr[n] > 0 && (!indices || !values)) return DSFACTO_ERR_INVALID_ARG;
    int rc = validate_csr(n, d, indptr, indices, values);
    if (rc) return rc;
    const int32_t lo = (int32_t)(((__int128)(((int64_t)shard * p) / nshards) * d + p - 1) / p);
    const int32_t hi = (int32_t)(((__int128)(((int64_t)(shard + 1) * p) / nshards) * d + p - 1) / p);
    HostBuf<int64_t> fp;
    HostBuf<int32_t> fi;
    HostBuf<float> fv;
    if ((rc = filter_columns(n, indptr, indices, values, lo, hi, fp, fi, fv))) return rc;
    *kept = fp[(size_t)n];
    return dsfacto_bucket_host(n, d, p, fp.data(), fi.data(), fv.data(), tile_ptr, rows, cols, vals);
}

int dsfacto_set_refresh_every(dsfacto_t *h, int32_t rounds) {
    if (!h || rounds < 0) return DSFACTO_ERR_INVALID_ARG;
    if (h->loaded) return DSFACTO_ERR_INVALID_ARG;   // the launch plan is fixed by dsfacto_load_csr
    if (rounds > 0 && h->nshards > 1) return DSFACTO_ERR_INVALID_ARG;   // column shards exchange once per epoch
    h->refresh_every = rounds;   // the launch plan built by dsfacto_load_csr is cut into segments of that many rounds
    return DSFACTO_OK;
}

int dsfacto_objective(dsfacto_t *h, double *out) {
    if (!h || !out) return DSFACTO_ERR_INVALID_ARG;
    if (!h->loaded) return DSFACTO_ERR_NO_DATA;
    *out = h->objective;
    return DSFACTO_OK;
}

int dsfacto_get_stats(dsfacto_t *h, double *mean_loss, double *sum_G) {
    if (!h) return DSFACTO_ERR_INVALID_ARG;
    if (!h->loaded) return DSFACTO_ERR_NO_DATA;
    if (mean_loss) *mean_loss = h->loss_sum / (double)h->n;
    if (sum_G) *sum_G = h->g_sum;
    return DSFACTO_OK;
}

int dsfacto_get_params(dsfacto_t *h, float *w0, float *w, float *V) {
    if (!h) return DSFACTO_ERR_INVALID_ARG;
    if (w0) *w0 = h->w0;
    if (w) {
        CU_TRY(h, cudaMemcpyAsync(w, h->d_w, sizeof(float) * (size_t)h->d, cudaMemcpyDeviceToHost, h->stream));
        CU_TRY(h, cudaStreamSynchronize(h->stream));
    }
    if (V) return download_rows(h, V, h->d_V, h->d);
    return DSFACTO_OK;
}

int dsfacto_set_params(dsfacto_t *h, const float *w0, const float *w, const float *V) {
    if (!h) return DSFACTO_ERR_INVALID_ARG;
    if (w0) { if (!std::isfinite(*w0)) return DSFACTO_ERR_INVALID_ARG; h->w0 = *w0; }
    if (w) {
        h->model_version += 1;
        CU_TRY(h, cudaMemcpyAsync(h->d_w, w, sizeof(float) * (size_t)h->d, cudaMemcpyHostToDevice, h->stream));
        CU_TRY(h, cudaStreamSynchronize(h->stream));
    }
    if (V) { int rc = upload_V(h, V); if (rc) return rc; }
    if (w && V) h->failed = false;   // a handle whose SGD launch gave up is usable again once w and V are replaced
    if (h->loaded) {
        int rc = run_refresh(h, false);
        if (rc) return rc;
        if (!std::isfinite(h->objective)) return DSFACTO_ERR_DIVERGED;
    }
    return DSFACTO_OK;
}

int dsfacto_get_aux(dsfacto_t *h, float *A, float *G) {
    if (!h) return DSFACTO_ERR_INVALID_ARG;
    if (!h->loaded) return DSFACTO_ERR_NO_DATA;
    if (G) {
        CU_TRY(h, cudaMemcpyAsync(G, h->d_G, sizeof(float) * (size_t)h->n, cudaMemcpyDeviceToHost, h->stream));
        CU_TRY(h, cudaStreamSynchronize(h->stream));
    }
    if (A) return download_rows(h, A, h->d_A, h->n);
    return DSFACTO_OK;
}

int dsfacto_get_tiles(dsfacto_t *h, int64_t *tile_ptr, int32_t *rows, int32_t *cols, float *vals) {
    if (!h) return DSFACTO_ERR_INVALID_ARG;
    if (!h->loaded) return DSFACTO_ERR_NO_DATA;
    const int64_t nt = (int64_t)h->p * h->p;
    std::vector<int64_t> canon;
    if (h->rbits == 0) {
        try { canon = canonical_tile_ptr(h); } catch (const std::bad_alloc &) { return DSFACTO_ERR_OOM; }
        if (tile_ptr) std::memcpy(tile_ptr, canon.data(), sizeof(int64_t) * ((size_t)nt + 1));
        if (!rows && !cols && !vals) return DSFACTO_OK;
    }
    HostBuf<uint2> ent;
    HostBuf<float> xw;
    if (!ent.alloc((size_t)h->nnz) || (h->wide && !xw.alloc((size_t)h->nnz))) return DSFACTO_ERR_OOM;
    if (h->nnz > 0) {
        CU_TRY(h, cudaMemcpyAsync(ent.data(), h->d_ent, sizeof(uint2) * (size_t)h->nnz, cudaMemcpyDeviceToHost, h->stream));
        if (h->wide) CU_TRY(h, cudaMemcpyAsync(xw.data(), h->d_xw, sizeof(float) * (size_t)h->nnz, cudaMemcpyDeviceToHost, h->stream));
        CU_TRY(h, cudaStreamSynchronize(h->stream));
    }
    if (h->rbits > 0) {   // (merged row blocks: the tile sizes come from the entries themselves)
        try { unpack_merged_tiles(h, ent.data(), canon, rows, cols, vals); } catch (const std::bad_alloc &) { return DSFACTO_ERR_OOM; }
        if (tile_ptr) std::memcpy(tile_ptr, canon.data(), sizeof(int64_t) * ((size_t)nt + 1));
        return DSFACTO_OK;
    }
    unpack_tiles(h, canon, ent.data(), xw.data(), rows, cols, vals);
    return DSFACTO_OK;
}

int dsfacto_bucket_host(int64_t n, int32_t d, int32_t p, const int64_t *indptr, const int32_t *indices,
                        const float *values, int64_t *tile_ptr, int32_t *rows, int32_t *cols, float *vals) {
    if (n < 1 || n >= ((int64_t)1 << 31) || d < 1 || p < 1 || p > 4096 || !indptr || !tile_ptr) return DSFACTO_ERR_INVALID_ARG;
    if (indptr[0] != 0 || indptr[n] < 0) return DSFACTO_ERR_INVALID_CSR;
    if (indptr[n] > 0 && (!indices || !values)) return DSFACTO_ERR_INVALID_ARG;
    int rc = validate_csr(n, d, indptr, indices, values);
    if (rc) return rc;
    dsfacto tmp;
    tmp.n = n; tmp.d = d; tmp.p = p;
    tmp.sweep = 1;   // row-block order inside, canonical order out, when there are enough row blocks
    if (!use_row_block_bucketer(&tmp)) tmp.sweep = 0;
    if ((rc = setup_partition(&tmp))) return rc;
    HostBuf<uint2> ent;
    HostBuf<float> xw;
    rc = tmp.sweep == 1 ? bucket_tiles_by_row_block(&tmp, indptr, indices, values, ent, xw, nullptr)
                        : bucket_tiles(&tmp, indptr, indices, values, ent, xw, nullptr);
    if (rc) return rc;
    std::vector<int64_t> canon;
    try { canon = canonical_tile_ptr(&tmp); } catch (const std::bad_alloc &) { return DSFACTO_ERR_OOM; }
    std::memcpy(tile_ptr, canon.data(), sizeof(int64_t) * canon.size());
    unpack_tiles(&tmp, canon, ent.data(), xw.data(), rows, cols, vals);
    return DSFACTO_OK;
}

// Scores m rows (training rows when indptr is NULL, otherwise a caller CSR copied to the device for
// the call).  mode kScore: scores_out fp32[m].  mode kEvaluate: labels y (host) and sums2 = {sum of
// losses, sum of squared errors or number of correct signs}.
static int score_rows(dsfacto_t *h, int mode, int64_t m, const int64_t *indptr, const int32_t *indices,
                      const float *values, const float *y, float *scores_out, double sums2[2]) {
    RefreshArgs a{};
    a.w0 = h->w0; a.loss = h->loss; a.n = m;
    int64_t *d_ip = nullptr;
    int32_t *d_ix = nullptr;
    float *d_vl = nullptr, *d_f = nullptr, *d_yy = nullptr;
    double *d_part = nullptr;
    int rc = DSFACTO_OK;
    auto cleanup = [&]() { dev_free(d_ip); dev_free(d_ix); dev_free(d_vl); dev_free(d_f); dev_free(d_yy); dev_free(d_part); };
    if (!indptr) {
        if (!h->loaded) return DSFACTO_ERR_NO_DATA;
        if (m != h->n) return DSFACTO_ERR_INVALID_ARG;
        a.indptr = h->d_indptr; a.idx = h->d_idx; a.val = h->d_val;
        model_view(h, a, true);
    } else {
        if (indptr[0] != 0 || indptr[m] < 0) return DSFACTO_ERR_INVALID_CSR;
        const int64_t nnz = indptr[m];
        if (nnz > 0 && (!indices || !values)) return DSFACTO_ERR_INVALID_ARG;
        if ((rc = validate_csr(m, h->d, indptr, indices, values))) return rc;
        const size_t cnt = (size_t)std::max<int64_t>(nnz, 1);
        if ((rc = dev_alloc(h, &d_ip, (size_t)m + 1)) || (rc = dev_alloc(h, &d_ix, cnt)) || (rc = dev_alloc(h, &d_vl, cnt))) {
            cleanup();
            return rc;
        }
        cudaMemcpyAsync(d_ip, indptr, sizeof(int64_t) * ((size_t)m + 1), cudaMemcpyHostToDevice, h->stream);
        if (nnz > 0) {
            cudaMemcpyAsync(d_ix, indices, sizeof(int32_t) * (size_t)nnz, cudaMemcpyHostToDevice, h->stream);
            cudaMemcpyAsync(d_vl, values, sizeof(float) * (size_t)nnz, cudaMemcpyHostToDevice, h->stream);
        }
        a.indptr = d_ip; a.idx = d_ix; a.val = d_vl;
        model_view(h, a, false);
    }
    const int grid = refresh_grid_for(h, m);
    cudaError_t e = cudaSuccess;
    if (mode == kScore) {
        if ((rc = dev_alloc(h, &d_f, (size_t)m))) { cleanup(); return rc; }
        a.f_out = d_f;
        DSF_DISPATCH_REFRESH(h, h, a, kScore, grid);
        h->launches += 1;
        e = cudaMemcpyAsync(scores_out, d_f, sizeof(float) * (size_t)m, cudaMemcpyDeviceToHost, h->stream);
    } else {
        if ((rc = dev_alloc(h, &d_yy, (size_t)m)) || (rc = dev_alloc(h, &d_part, 2 * (size_t)grid + 2))) { cleanup(); return rc; }
        cudaMemcpyAsync(d_yy, y, sizeof(float) * (size_t)m, cudaMemcpyHostToDevice, h->stream);
        a.y = d_yy; a.partials = d_part;
        DSF_DISPATCH_REFRESH(h, h, a, kEvaluate, grid);
        reduce2_kernel<<<1, kThreads, 0, h->stream>>>(d_part, grid, d_part + 2 * (size_t)grid);
        h->launches += 2;
        e = cudaMemcpyAsync(sums2, d_part + 2 * (size_t)grid, 2 * sizeof(double), cudaMemcpyDeviceToHost, h->stream);
    }
    if (e == cudaSuccess) e = cudaStreamSynchronize(h->stream);
    if (e == cudaSuccess) e = cudaGetLastError();
    cleanup();
    if (e != cudaSuccess) { h->err = cudaGetErrorString(e); return DSFACTO_ERR_CUDA; }
    return DSFACTO_OK;
}

int dsfacto_predict(dsfacto_t *h, int64_t m, const int64_t *indptr, const int32_t *indices, const float *values,
                    float *scores_out) {
    if (!h || !scores_out || m < 0) return DSFACTO_ERR_INVALID_ARG;
    if (m == 0) return DSFACTO_OK;
    return score_rows(h, kScore, m, indptr, indices, values, nullptr, scores_out, nullptr);
}

int dsfacto_evaluate(dsfacto_t *h, int64_t m, const int64_t *indptr, const int32_t *indices, const float *values,
                     const float *y, double *mean_loss, double *metric) {
    if (!h || !indptr || !y || m < 1) return DSFACTO_ERR_INVALID_ARG;
    int bad = 0;
#pragma omp parallel for schedule(static) reduction(| : bad)
    for (int64_t i = 0; i < m; ++i)
        if (!std::isfinite(y[i])) bad |= 1;
    if (bad) return DSFACTO_ERR_INVALID_CSR;
    double s[2] = {0.0, 0.0};
    const int rc = score_rows(h, kEvaluate, m, indptr, indices, values, y, nullptr, s);
    if (rc) return rc;
    if (mean_loss) *mean_loss = s[0] / (double)m;
    if (metric) *metric = h->loss == DSFACTO_SQUARED ? std::sqrt(s[1] / (double)m) : s[1] / (double)m;
    return DSFACTO_OK;
}

int dsfacto_set_eta(dsfacto_t *h, float eta) {
    if (!h || !(eta > 0.f) || !std::isfinite(eta)) return DSFACTO_ERR_INVALID_ARG;
    h->eta = eta;
    h->h = (float)((double)eta / (double)h->n);
    return DSFACTO_OK;
}

int dsfacto_last_epoch_ms(dsfacto_t *h, float ms[4]) {
    if (!h || !ms) return DSFACTO_ERR_INVALID_ARG;
    for (int i = 0; i < 4; ++i) ms[i] = h->ms[i];
    return DSFACTO_OK;
}

int dsfacto_debug_set(dsfacto_t *h, int32_t key, int64_t value) {
    if (!h) return DSFACTO_ERR_INVALID_ARG;
    switch (key) {
    case DSFACTO_DEBUG_SPIN_LIMIT:
        if (value < 1 || value > kSgdSpinLimit) return DSFACTO_ERR_INVALID_ARG;
        h->spin_limit = (int)value;
        return DSFACTO_OK;
    case DSFACTO_DEBUG_EXTRA_NEED:
        if (value < 0 || value > kTicketStop) return DSFACTO_ERR_INVALID_ARG;
        h->debug_extra_need = (int)value;
        return DSFACTO_OK;
    case DSFACTO_DEBUG_CHUNK_LEN:
        if (value != 0 && (value < 16 || value > kChunkMax)) return DSFACTO_ERR_INVALID_ARG;
        h->chunk_override = (int)value;
        return DSFACTO_OK;
    case DSFACTO_DEBUG_ROW_MERGE:
        if (value != 0 && value != 1 && value != 2 && value != 4 && value != 8 && value != kMaxRowMerge) return DSFACTO_ERR_INVALID_ARG;
        h->row_merge = (int)value;
        return DSFACTO_OK;
    case DSFACTO_DEBUG_COLUMN_ORDER:
        if (value < 0 || value > 2) return DSFACTO_ERR_INVALID_ARG;
        h->column_order = (int)value;
        return DSFACTO_OK;
    default:
        return DSFACTO_ERR_INVALID_ARG;
    }
}

int dsfacto_last_load(dsfacto_t *h, int64_t info[3]) {
    if (!h || !info) return DSFACTO_ERR_INVALID_ARG;
    if (!h->loaded) return DSFACTO_ERR_NO_DATA;
    for (int k = 0; k < 3; ++k) info[k] = h->load_info[k];
    return DSFACTO_OK;
}

int dsfacto_launch_count(dsfacto_t *h, int64_t *out) {
    if (!h || !out) return DSFACTO_ERR_INVALID_ARG;
    *out = h->launches;
    return DSFACTO_OK;
}

}  // extern "C"
