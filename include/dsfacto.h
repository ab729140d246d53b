/*
 * dsfacto.h - C ABI of the DS-FACTO training hot path (doubly-separable factorization machines,
 * arXiv 2004.13940) for one NVIDIA B200 (sm_100a).
 *
 * Model (Section 3.2, eq. (fm_model2)): f(x_i) = w0 + sum_j w_j x_ij
 *     + 1/2 sum_k [ (sum_j v_jk x_ij)^2 - sum_j v_jk^2 x_ij^2 ],  w in R^D, V in R^{D x K}.
 * Objective (eq. (fm_obj)): L = (1/N) sum_i l(f(x_i), y_i) + lambda_w/2 |w|^2 + lambda_v/2 |V|^2.
 * Auxiliaries (Table "Notations", eq. (compute_a_jk)): a_ik = sum_j v_jk x_ij and the multiplier
 *     G_i = dl/df (f - y for the squared loss, -y / (1 + exp(y f)) for the logistic loss).
 *
 * One epoch = one outer iteration of Algorithm 1 in its synchronous (DSGD-style) form:
 *   X is cut into a p x p grid of (row-block, column-block) tiles (figure "communication
 *   pattern"); in inner round s the tiles (r, (r+s) mod p), r = 0..p-1, are processed; every
 *   stored entry applies the stochastic updates (dsfacto_sgdupdatew)/(dsfacto_sgdupdatev) once,
 *   with G and A frozen; afterwards G and A are recomputed from the new parameters
 *   (Section 4.2, "Handling the staleness ...") and the objective is evaluated.
 *
 * Conventions
 *   - Every pointer argument is HOST memory, borrowed for the duration of the call; outputs are
 *     caller-allocated.  The library owns all device memory.
 *   - Return value: DSFACTO_OK (0) or a negative DSFACTO_ERR_* code; nothing is thrown.
 *   - Calls on one handle must not overlap in time.  Every call returns after its device work
 *     has completed.  There is no CPU fallback: without a usable CUDA device calls fail with
 *     DSFACTO_ERR_CUDA.
 *   - All device state is fp32 (X, y, w, V, A, G); sums that form the objective are fp64.
 */
#ifndef DSFACTO_H
#define DSFACTO_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct dsfacto dsfacto_t; /* opaque, owned by the library */

enum { DSFACTO_SQUARED = 0, DSFACTO_LOGISTIC = 1 }; /* l = 1/2 (f-y)^2 ; l = log(1+exp(-y f)), y = +-1 */

enum {
    DSFACTO_OK = 0,
    DSFACTO_ERR_INVALID_ARG = -1, /* null pointer, size or hyper-parameter out of range */
    DSFACTO_ERR_INVALID_CSR = -2, /* indptr not monotone, column ids not strictly increasing or out
                                     of [0,d), non-finite value or label */
    DSFACTO_ERR_NO_DATA = -3,     /* call needs dsfacto_load_csr first */
    DSFACTO_ERR_OOM = -4,         /* host or device allocation failed */
    DSFACTO_ERR_CUDA = -5,        /* CUDA runtime error (see dsfacto_last_error) */
    DSFACTO_ERR_DIVERGED = -6     /* objective is NaN or infinite */
};

/* Problem statement of Section 3.2 plus the partition of Section 4.2.
 *   n rows (1 <= n < 2^31), d columns (1 <= d), K latent factors (1 <= K <= 256), p tiles per side
 *   (1 <= p <= 4096; p may exceed d or n, the surplus blocks are empty), loss DSFACTO_SQUARED or
 *   DSFACTO_LOGISTIC, regularisers lambda_w, lambda_v >= 0, learning rate eta > 0.
 * The per-entry step is eta / n (the objective carries 1/N, the printed updates do not).
 * Initialisation (Algorithm 1, initialisation line): w0 = 0, w = 0, v_jk = 0.01 * z with z standard
 * normal: element e = j*K+k takes outputs 2e and 2e+1 of SplitMix64 seeded with `seed`, maps each
 * to (u>>11 + 0.5)/2^53 and applies Box-Muller (cosine branch); the product is rounded to fp32.
 * On success *out holds a new handle (release with dsfacto_destroy). */
int dsfacto_create(dsfacto_t **out, int64_t n, int32_t d, int32_t K, int32_t p, int32_t loss,
                   float lambda_w, float lambda_v, float eta, uint64_t seed);

/* Loads the training set X (CSR: indptr int64[n+1] with indptr[0] = 0, indices int32[nnz] strictly
 * increasing inside each row and in [0,d), values fp32[nnz] finite; stored zeros count as entries)
 * and labels y fp32[n] (finite).  Builds the p x p tile lists (figure "communication
 * pattern": row block of row i is floor(i*p/n), column block of column j is floor(j*p/d); tile
 * (r,c) belongs to round s = (c-r) mod p; tiles ordered by (s, r); inside a tile entries ordered
 * by (column, row)), copies CSR and tiles to the device and runs the recompute pass once, so that
 * A, G and the objective of the initial parameters exist.  Replaces any earlier data set.
 * Non-empty loads are bucketed on the device itself when the packed entry layout
 * applies (local row and column ids fit 32 bits together, tile number and local column id too) and the
 * device has room for the buffers of a sort (about 25 bytes per stored entry for the duration of the call):
 * the CSR copy that the recompute pass needs anyway is turned into (tile, local column) keys, sorted by a
 * stable radix sort, packed into entry records, and a kernel cuts the chunks of the stratum SGD launch; only
 * the CSR arrays cross the link, and from 2^24 stored entries on they are sent while the host still checks them
 * (a data set that fails the checks leaves the handle as it was, as on every path).  On this path the
 * row-block sweep stores several consecutive row blocks of a column block as one slot (up to 8, for loads of
 * fewer than 2^24 entries up to 16; see DSFACTO_DEBUG_ROW_MERGE).  DSFACTO_LOAD=device asks for this way
 * explicitly.  Otherwise, and with any other value of DSFACTO_LOAD, the tile lists are built on the host; there,
 * loads of 2^24 stored entries and more (with p at least twice the number of host threads) are
 * streamed: each host thread buckets one row block at a time into page-locked staging memory and
 * copies it to its place on the device while the other row blocks are being bucketed.  That staging
 * memory (two row blocks per host thread) is allocated on the first such load and kept by the process
 * for later loads; streamed loads of one process run one at a time.  The environment variable
 * DSFACTO_LOAD=stream streams smaller loads too, DSFACTO_LOAD=simple never streams; if the staging
 * memory cannot be had, the load falls back to one copy from pageable memory.  The resulting tile
 * lists are the same bit for bit on every path.  Page-locked caller arrays make the CSR copy overlap
 * the bucketing. */
int dsfacto_load_csr(dsfacto_t *h, const int64_t *indptr, const int32_t *indices,
                     const float *values, const float *y);

/* One epoch (Algorithm 1, body of the loop over t):
 *   w0 <- w0 - (eta/n) sum_i G_i                        (frozen G; df/dw0 = 1)
 *   for s = 0..p-1, for the tiles (r,(r+s) mod p), for each stored (i,j,x) in tile order:
 *       w_j  <- w_j  - (eta/n) (G_i x + lambda_w w_j)                          eq. (dsfacto_sgdupdatew)
 *       v_jk <- v_jk - (eta/n) (G_i (x a_ik - v_jk x^2) + lambda_v v_jk)       eq. (dsfacto_sgdupdatev)
 *   recompute a_ik (eq. (compute_a_jk)), f_i (eq. (fm_model2)), G_i and the objective (eq. (fm_obj)).
 * Returns DSFACTO_ERR_DIVERGED if the new objective is not finite (state is kept). */
int dsfacto_epoch(dsfacto_t *h);

/* Raw scores f(x_i), eq. (fm_model2), of m rows given as CSR (same rules as dsfacto_load_csr) with
 * the current parameters; scores_out fp32[m].  indptr == NULL scores the loaded training rows
 * (m must then equal n). */
int dsfacto_predict(dsfacto_t *h, int64_t m, const int64_t *indptr, const int32_t *indices,
                    const float *values, float *scores_out);

/* Held-out evaluation, the quantities the convergence figures of Section 5 plot beside the
 * objective: m >= 1 rows as CSR (same rules as dsfacto_load_csr; indptr must not be NULL) with labels
 * y fp32[m] (finite; +-1 for the logistic loss), scored with the current parameters.
 *   *mean_loss = (1/m) sum_i l(f(x_i), y_i) with the handle's loss;
 *   *metric    = sqrt((1/m) sum_i (f(x_i) - y_i)^2)   (RMSE)       for DSFACTO_SQUARED,
 *              = (1/m) #{ i : y_i f(x_i) > 0 }        (accuracy)   for DSFACTO_LOGISTIC; the predicted
 *                class is the sign of the fp32 score, and a score of exactly 0 predicts neither class.
 * Either output pointer may be NULL.  The training state (A, G, objective) is not touched. */
int dsfacto_evaluate(dsfacto_t *h, int64_t m, const int64_t *indptr, const int32_t *indices,
                     const float *values, const float *y, double *mean_loss, double *metric);

/* Sets the learning rate eta (> 0, finite) used by the following epochs; the per-entry step becomes
 * eta / n.  Step-size schedules (the experiments' file names mention a decay, the text does not define
 * it) are left to the caller: call this between epochs. */
int dsfacto_set_eta(dsfacto_t *h, float eta);

/* Second schedule, for shorter staleness (Section 4.2, "Handling the staleness ...": stale G and A
 * slow convergence, which is why they are recomputed after the update step).  rounds = 0 (default):
 * the recompute pass runs once per epoch, after all p inner rounds, as in Algorithm 1.  rounds = R >= 1:
 * dsfacto_epoch cuts the p inner rounds into segments of R consecutive rounds (the last may be
 * shorter) and runs the recompute pass after every segment; before a segment of m rounds w0 takes the
 * share m/p of its step, w0 <- w0 - (eta/n) (m/p) sum_i G_i, with the multipliers frozen for that
 * segment.  R >= p is the default schedule.  An epoch then costs ceil(p/R) recompute passes.
 * Must be called before dsfacto_load_csr (DSFACTO_ERR_INVALID_ARG afterwards): the load cuts its launch
 * plan into the segments. */
int dsfacto_set_refresh_every(dsfacto_t *h, int32_t rounds);

/* Objective eq. (fm_obj) as of the last recompute pass (after load_csr, epoch or set_params). */
int dsfacto_objective(dsfacto_t *h, double *out);

/* Copies out w0 (1), w (d) and V (d*K, row-major: V[j*K+k] = v_jk).  Any pointer may be NULL. */
int dsfacto_get_params(dsfacto_t *h, float *w0, float *w, float *V);

/* Overwrites the parameters (same layout as dsfacto_get_params; NULL keeps the current value) and,
 * if data is loaded, reruns the recompute pass.  Checkpoint/restore and test injection; the paper
 * has no counterpart. */
int dsfacto_set_params(dsfacto_t *h, const float *w0, const float *w, const float *V);

void dsfacto_destroy(dsfacto_t *h);

/* ---- inspection (tests, tooling) ---- */

/* Tile lists as built by dsfacto_load_csr, in the canonical order described there:
 * tile_ptr int64[p*p+1] (tile t = s*p + r), rows int32[nnz], cols int32[nnz] (global ids),
 * vals fp32[nnz]. */
int dsfacto_get_tiles(dsfacto_t *h, int64_t *tile_ptr, int32_t *rows, int32_t *cols, float *vals);

/* The host tile bucketer of dsfacto_load_csr on its own: same inputs (n rows, d columns, p tiles per
 * side, CSR arrays), same checks, same output layout as dsfacto_get_tiles.  Touches no GPU. */
int dsfacto_bucket_host(int64_t n, int32_t d, int32_t p, const int64_t *indptr, const int32_t *indices,
                        const float *values, int64_t *tile_ptr, int32_t *rows, int32_t *cols, float *vals);

/* Frozen auxiliaries of the last recompute pass: A fp32[n*K] row-major (a_ik), G fp32[n].
 * Either pointer may be NULL. */
int dsfacto_get_aux(dsfacto_t *h, float *A, float *G);

/* Mean loss (1/N) sum_i l_i and sum_i G_i of the last recompute pass.  Either pointer may be NULL. */
int dsfacto_get_stats(dsfacto_t *h, double *mean_loss, double *sum_G);

/* ---- plumbing ---- */

/* Runs all later device work of this handle on `cuda_stream` (a cudaStream_t passed as void*;
 * NULL = the legacy default stream).  The stream stays owned by the caller. */
int dsfacto_set_stream(dsfacto_t *h, void *cuda_stream);

/* Device time of the last dsfacto_epoch from CUDA events on the handle's stream, in milliseconds:
 * ms[0] whole epoch, ms[1] the p strata (update loop), ms[2] recompute pass (refresh + residual +
 * loss sums), ms[3] parameter norms + final reduction.  With dsfacto_set_refresh_every each figure is
 * the sum over the segments of the epoch. */
int dsfacto_last_epoch_ms(dsfacto_t *h, float ms[4]);

/* Test and debugging knobs of the stratum SGD launch.
 *   DSFACTO_DEBUG_SPIN_LIMIT  polls (a few hundred ns each, 1 .. 2^22, default 2^22) after which a wait for an
 *                             earlier tile of the same column block gives up; dsfacto_epoch then returns
 *                             DSFACTO_ERR_CUDA and the handle refuses further epochs until dsfacto_set_params
 *                             replaces w and V or dsfacto_load_csr loads a data set.
 *   DSFACTO_DEBUG_EXTRA_NEED  (takes effect at the next dsfacto_load_csr) the first chunk of the sweep is made to
 *                             wait for that many finished chunks more than its column block really has before
 *                             it; with a value larger than the number of chunks its wait runs out, so the
 *                             failure path above can be exercised without a fault or a hang.  0 = off.
 *   DSFACTO_DEBUG_CHUNK_LEN   (takes effect at the next dsfacto_load_csr) entries per chunk, 16 .. 4096, 0 = chosen
 *                             by the load; the environment variable DSFACTO_CHUNK does the same for every handle.
 *                             The sweep kernel reads a chunk's entries block by block; the environment variable
 *                             DSFACTO_BLOCK (a multiple of 32, 32 .. 256) sets the entries per block.
 *   DSFACTO_DEBUG_ROW_MERGE   (takes effect at the next dsfacto_load_csr that buckets on the device) row blocks per slot of
 *                             the device entry array, 1, 2, 4, 8 or 16 (as many of them as the 32-bit keys and records
 *                             allow), 0 = chosen by the load: a column's entries in consecutive row blocks follow one
 *                             another in the stratified order, so they can be stored and swept as one run.  Same
 *                             result up to rounding; the environment variable DSFACTO_ROW_MERGE does the same.
 *   DSFACTO_DEBUG_COLUMN_ORDER (takes effect at the next dsfacto_load_csr) the device copy of the CSR that the
 *                             recompute pass reads may number the columns by frequency, most frequent first, and
 *                             the pass then reads w and V from a copy in that order (hot factor rows side by
 *                             side in the caches; no sum changes).  0 = decided by the load (on from 2^22 stored
 *                             entries and 1 MB of factors), 1 = always, 2 = never; the environment variable
 *                             DSFACTO_COLUMN_ORDER=0/1 does the same for every handle.  Nothing a caller passes
 *                             or receives is renumbered.
 * The environment variable DSFACTO_SWEEP=round (read by dsfacto_create) stores and sweeps the tiles round by
 * round, exactly Algorithm 1's order, instead of row block by row block. */
enum { DSFACTO_DEBUG_SPIN_LIMIT = 0, DSFACTO_DEBUG_EXTRA_NEED = 1, DSFACTO_DEBUG_CHUNK_LEN = 2, DSFACTO_DEBUG_COLUMN_ORDER = 3,
       DSFACTO_DEBUG_ROW_MERGE = 4 };
int dsfacto_debug_set(dsfacto_t *h, int32_t key, int64_t value);

/* How the last dsfacto_load_csr built the tile lists: info[0] = 0 on the host with one copy, 1 on the host
 * streamed through page-locked staging memory, 2 on the device; info[1] = bytes it copied host -> device,
 * info[2] = bytes it copied device -> host.  DSFACTO_ERR_NO_DATA before the first load. */
int dsfacto_last_load(dsfacto_t *h, int64_t info[3]);

/* Number of kernels this handle has launched since creation. */
int dsfacto_launch_count(dsfacto_t *h, int64_t *out);

/* Text of the last CUDA/host error recorded on this handle ("" if none); valid until the next call. */
const char *dsfacto_last_error(dsfacto_t *h);

const char *dsfacto_strerror(int status);

/* ---- column shards: the partition of Section 4.2 across several GPUs ----
 *
 * Section 4.2 spreads the column blocks of w and V over the workers and lets every worker see the rows.
 * With G and A frozen the columns never interact during the update loop, so a shard that owns a contiguous
 * range of column blocks runs the strata of its own tiles without any exchange; only the recompute pass needs
 * the other shards: a_ik, lin_i = sum_j w_j x_ij and q_i = sum_j sum_k v_jk^2 x_ij^2 are sums over columns.
 * Each shard computes them over its own columns, the partial results are added up across the shards (one
 * all-reduce of n (Kp + 2) floats, outside this library: NCCL through torch.distributed in the Python
 * package), and every shard finishes the pass (f_i, l_i, G_i) from the totals.  The paper's own way of moving
 * column blocks between workers round by round is the distributed-memory form of the same partition.
 *
 * dsfacto_create_shard: like dsfacto_create for shard `shard` of `nshards` (1 <= nshards <= p); the handle
 *   owns column blocks [floor(shard p / nshards), floor((shard+1) p / nshards)).  w, V of other columns are
 *   held but never touched.  dsfacto_shard_columns returns the owned column range [col_lo, col_hi).
 * dsfacto_load_csr on a shard takes the WHOLE data set, keeps the stored entries of its own columns, builds
 *   their tile lists (the canonical lists restricted to those columns) and computes the partial auxiliaries of
 *   the initial parameters; the caller then adds the shards' partial buffers up and calls
 *   dsfacto_shard_epoch_end once before the first epoch.
 * One epoch of a shard:
 *   dsfacto_shard_epoch_begin   w0 step (identical on every shard), the p strata over the shard's tiles, the
 *                               partial recompute pass
 *   dsfacto_shard_partial       copies the partial buffer [A (n x Kp, Kp = K rounded up to the lane layout) |
 *                               lin (n) | q (n)], dsfacto_shard_partial_count floats, to DEVICE memory of the caller
 *   (the caller sums the buffers of all shards)
 *   dsfacto_shard_epoch_end     takes the summed buffer (DEVICE memory), finishes the recompute pass and returns
 *                               sums[4] = { sum_i l_i, sum_i G_i, sum of w_j^2 and sum of v_jk^2 over the shard's
 *                               OWN columns }; the objective eq. (fm_obj) is sums[0]/n + lambda_w/2 (sum of the
 *                               shards' sums[2]) + lambda_v/2 (sum of the shards' sums[3]).
 * dsfacto_epoch and dsfacto_set_refresh_every(> 0) are refused on a shard (DSFACTO_ERR_INVALID_ARG).
 * dsfacto_bucket_host_shard is dsfacto_bucket_host for one shard: the tile lists of the entries whose column
 * the shard owns (*kept = their number); it touches no GPU. */
int dsfacto_create_shard(dsfacto_t **out, int64_t n, int32_t d, int32_t K, int32_t p, int32_t loss,
                         float lambda_w, float lambda_v, float eta, uint64_t seed, int32_t shard, int32_t nshards);
int dsfacto_shard_columns(dsfacto_t *h, int32_t *col_lo, int32_t *col_hi);
int dsfacto_shard_partial_count(dsfacto_t *h, int64_t *count);
int dsfacto_shard_epoch_begin(dsfacto_t *h);
int dsfacto_shard_partial(dsfacto_t *h, float *dst_dev, int64_t count);
int dsfacto_shard_epoch_end(dsfacto_t *h, const float *summed_dev, int64_t count, double sums[4]);
int dsfacto_bucket_host_shard(int64_t n, int32_t d, int32_t p, int32_t shard, int32_t nshards, const int64_t *indptr,
                              const int32_t *indices, const float *values, int64_t *kept, int64_t *tile_ptr,
                              int32_t *rows, int32_t *cols, float *vals);

/* ---- for callers that cannot allocate ---- */

/* Scores, loss sum and multiplier sum of m rows, without any allocation.  (The paper has no
 * counterpart: this is a service entry point.)  It is meant for code that runs where cudaMalloc is
 * off limits - a process whose device memory is wholly owned by another pool, a serving loop with
 * a fixed memory budget, a thread that must not take the driver's allocation lock - and that
 * therefore keeps the rows, the parameters and the result buffers in device memory of its own.
 *
 * ALL pointers are DEVICE memory on the current device, owned by the caller, and no handle is
 * involved:
 *   indptr_dev int64[m+1], indices_dev int32[nnz], values_dev fp32[nnz]  rows as CSR (same rules
 *       as dsfacto_load_csr; they are NOT checked here, the caller vouches for them)
 *   y_dev fp32[m] labels; w0, w_dev fp32[d], V_dev fp32[d*K] row-major, 16-byte aligned parameters
 *   scores_dev fp32[m]  out: f(x_i), eq. (fm_model2)
 *   sums_dev fp64[2]    out: { sum_i l(f(x_i), y_i), sum_i G_i }
 *   cuda_stream         cudaStream_t as void* (NULL = legacy default stream)
 * Limits: K must be 4, 8, 16, 32, 64, 128 or 256 (rows of V are read as whole 16-byte lane groups);
 * 1 <= m <= 67,108,864 rows, because the per-CTA partial sums of the reduction live in a fixed
 * 1 MiB array inside the library image (every GPU that loads the library holds it until the
 * process exits).  Anything outside these limits returns DSFACTO_ERR_INVALID_ARG.
 * V_dev must be 16-byte aligned and none of the pointers may be NULL (DSFACTO_ERR_INVALID_ARG otherwise).
 * The first call on each device looks up that array's device address (a host-side query, once per
 * device), so make that first call before any stream capture begins.  All calls on a device share the array: it keeps the last call's
 * contents, every call overwrites the slots it uses before reading them (nothing needs clearing),
 * and two calls that overlap on the GPU (different streams or threads) race on it - serialise them.
 * The call performs no cudaMalloc/cudaFree and returns after its work on the stream has finished. */
int dsfacto_score_loss_noalloc(int64_t m, int32_t d, int32_t K, int32_t loss, const int64_t *indptr_dev,
                               const int32_t *indices_dev, const float *values_dev, const float *y_dev,
                               float w0, const float *w_dev, const float *V_dev, float *scores_dev,
                               double *sums_dev, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* DSFACTO_H */
