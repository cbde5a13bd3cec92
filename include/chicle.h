/*
 * chicle.h -- C ABI of libchicle: one CoCoA round for generalised linear models on one NVIDIA B200.
 *
 * A round (paper Sec. 2.2, Eq. 1, Eq. 2 and "CoCoA"; Sec. 5.1 "CoCoA"): K uni-task partitions of the
 * coordinates each run a sequential stochastic coordinate-descent solver against a private copy of the shared
 * vector v, the K updates are added into v, and the duality gap (the paper's convergence metric, Sec. 4.1 and
 * Sec. 5) can be evaluated. Every step runs in CUDA kernels of this library; there is no host fallback.
 *
 * Problem:   P(w) = (1/n) sum_i loss_i(x_i . w) + (lambda/2) |w|^2
 *   - hinge and logistic: solved in the dual. Coordinates are the n examples (rows of X, CSR or dense
 *     row-major), state alpha in R^n (signed: alpha_i = y_i a_i, a_i in [0,1]), shared vector
 *     v = X^T alpha in R^d, w = v / (lambda n).
 *   - ridge, loss_i(z) = (z - y_i)^2 / 2: solved in the primal over feature partitions. Coordinates are the d
 *     columns of X (CSC), state w in R^d, shared vector v = X w in R^n.
 *
 * Conventions
 *   - Every call returns a chicle_status_t. No C++ exception crosses this boundary. Out-parameters are left
 *     untouched on error. After any error other than CHICLE_ERR_CUDA the handle is usable, and unchanged with two
 *     exceptions: a partition call that runs out of memory (CHICLE_ERR_OOM) has released the old per-partition
 *     workspaces first (two of them do not fit at the largest problems) and leaves the handle without a partition,
 *     alpha and v kept: call chicle_partition again; and a round that ended with CHICLE_ERR_TIMEOUT or
 *     CHICLE_ERR_NUMERIC has left alpha and v part-way through the round (restore them with chicle_set_state).
 *   - All pointers named host_* are host memory; chicle_matrix_t says where its arrays live. The library copies
 *     what it needs at create time: the caller keeps ownership of everything it passes and may free it as soon
 *     as the call returns. Everything the library allocates is released by chicle_glm_destroy.
 *   - One handle is bound to one device and one stream, and is not thread-safe. Calls enqueue work on that
 *     stream; calls that return host scalars or copy to host memory synchronise the stream.
 *   - CHICLE_LOG=1 in the environment (read once per process): every failed call writes its message, and every
 *     round one line with its step count, solver variant, launches and phase times, to stderr; a round is then
 *     synchronised for its timings.
 *   - Kernels never trap. A device-side problem (a bounded wait that ran out, a non-finite step) is recorded in a
 *     status word that the next synchronising call returns as CHICLE_ERR_TIMEOUT / CHICLE_ERR_NUMERIC.
 *   - State machine (paper Sec. 3, ownership contract: data moves only between iterations):
 *       create -> partition -> { cocoa_round | duality_gap | partition | get_* | set_state }*
 *     chicle_cocoa_round before the first chicle_partition returns CHICLE_ERR_BAD_STATE. chicle_partition keeps
 *     alpha, v and the round counter (per-sample state travels with its sample, Sec. 4.4).
 */
#ifndef CHICLE_H
#define CHICLE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct chicle_glm chicle_glm_t; /* opaque, owned by the library */

typedef enum {
    CHICLE_OK = 0,
    CHICLE_ERR_INVALID_ARG = 1,
    CHICLE_ERR_BAD_STATE = 2,
    CHICLE_ERR_OOM = 3,
    CHICLE_ERR_CUDA = 4,
    CHICLE_ERR_UNSUPPORTED = 5,
    CHICLE_ERR_NUMERIC = 6,
    CHICLE_ERR_TIMEOUT = 7,
    CHICLE_ERR_INTERNAL = 8 /* only from a library built with -DCHICLE_DEBUG_BOUNDS: an index that a kernel loaded lay
                               outside its array; the access was skipped, the state is part-way through the call */
} chicle_status_t;

typedef enum { CHICLE_LOSS_HINGE_DUAL = 0, CHICLE_LOSS_LOGISTIC_DUAL = 1, CHICLE_LOSS_RIDGE_PRIMAL = 2 } chicle_loss_t;
typedef enum { CHICLE_FMT_DENSE_ROWMAJOR = 0, CHICLE_FMT_CSR = 1, CHICLE_FMT_CSC = 2 } chicle_format_t;
typedef enum { CHICLE_MEM_HOST = 0, CHICLE_MEM_DEVICE = 1 } chicle_memspace_t;

/* Caller-owned description of X (n_rows examples by n_cols features). All arrays live in `space`.
 *   dense:  values[i*ld + j], ld >= n_cols, indptr = indices = NULL, nnz ignored.
 *   CSR:    indptr[n_rows+1], indices[nnz] column ids, values[nnz]; ids unique inside a row.
 *   CSC:    indptr[n_cols+1], indices[nnz] row ids,    values[nnz]; ids unique inside a column.
 * Hinge and logistic accept dense or CSR; ridge accepts CSC. Any other pairing is CHICLE_ERR_UNSUPPORTED. */
typedef struct {
    chicle_format_t fmt;
    chicle_memspace_t space;
    int64_t n_rows, n_cols, nnz, ld;
    const int64_t *indptr;
    const int32_t *indices;
    const float *values;
} chicle_matrix_t;

/* Optional device allocator (for example one backed by a framework's caching allocator). Both callbacks or
 * neither; NULL struct or NULL callbacks select cudaMalloc / cudaFree on the handle's device. `alloc` returns
 * NULL on failure; returned pointers must be 256-byte aligned device memory. */
typedef struct {
    void *(*alloc)(void *ctx, size_t bytes);
    void (*free)(void *ctx, void *ptr);
    void *ctx;
} chicle_allocator_t;

/* Device timings of one round in milliseconds (CUDA events on the handle's stream). */
typedef struct {
    float ms_permutation; /* a2: visiting orders of this round                                  */
    float ms_local;       /* a3+a4: local SCD solvers                                           */
    float ms_reduce;      /* a5: v += sum_k dv_k                                                */
    float ms_total;       /* whole round                                                        */
    int64_t steps;        /* coordinate steps taken in this round, all partitions               */
    int32_t solver_variant; /* 0 dense ring, 1 sparse blocked, 2 sparse ring, 3 dense blocked (rows <= 128),
                               4 sparse look-ahead, 5 dense look-ahead (rows <= 128) */
    float ms_prepare;     /* part of ms_local before the look-ahead solver's first chain launch starts (variants 4, 5):
                             the prepare kernel of the whole round, or of its first slice when a long round is cut
                             into slices whose prepare kernels run beside the chain kernels; when H spans several
                             local epochs: the first epoch's; else 0 */
    int32_t solver_slices;   /* look-ahead solver: slices the round's walk was cut into (last local epoch); else 0   */
    int32_t cluster_ctas;    /* look-ahead solver: CTAs per partition (thread-block cluster size); else 1            */
    int32_t solver_launches; /* kernels the local solvers launched in this round (block tables, prepare, chain)      */
    int32_t order_launches;  /* kernels launched for this round's visiting orders                                    */
} chicle_round_stats_t;

/* Create a training problem (Sec. 2.2, Sec. 5.1: a GLM trained by CoCoA with a local SCD solver; Sec. 4.4:
 * samples and their per-sample state are held together). Copies X and the labels to `device`, computes the
 * squared norms of the coordinate vectors, zeroes alpha (or w) and v. `labels` has n_rows entries in X->space:
 * +1/-1 for hinge and logistic (anything else: CHICLE_ERR_INVALID_ARG), real targets for ridge. NaN or Inf in
 * values or labels: CHICLE_ERR_NUMERIC. `cuda_stream` is a cudaStream_t (NULL = the legacy default stream).
 * Synchronises the stream before returning. On success *out receives the handle. */
chicle_status_t chicle_glm_create(const chicle_matrix_t *X, const float *labels, float lambda, chicle_loss_t loss,
                                  int device, void *cuda_stream, const chicle_allocator_t *alloc,
                                  chicle_glm_t **out);

/* Random equal split of the coordinates into K disjoint covering partitions (Sec. 2.2: disjoint partitions D_k;
 * Sec. 3: the data parallelism can change between iterations; Appendix, baseline comparisons: data is assigned to tasks at random).
 * Integer rule: ids are ordered by mix64(mix64(seed) ^ id) (mix64 = one SplitMix64 output for that state) and
 * cut into K consecutive blocks, the first n mod K one longer. 1 <= K <= number of coordinates. Legal only
 * between rounds; keeps alpha, v and the round counter; (re)allocates the per-partition workspaces. */
chicle_status_t chicle_partition(chicle_glm_t *h, int32_t K, uint64_t seed);

/* The same, with partitions of given sizes (Sec. 3, load balancing: tasks may hold different numbers of samples, data
 * moves from slow to fast tasks between iterations; Sec. 4.5, rebalancing policy). The random order of the ids is the
 * one chicle_partition uses; it is cut into K consecutive blocks of host_sizes[0], ..., host_sizes[K-1] coordinates
 * (a host array, read during the call; every size >= 1, the sum equal to the number of coordinates, else
 * CHICLE_ERR_INVALID_ARG and the handle is unchanged). With equal sizes the result is chicle_partition's. A round with
 * H = 0 then takes as many steps in partition k as it has coordinates; the updates are added as before (every
 * coordinate has one owner, so no weighting by |D_k| / |D| is needed). */
chicle_status_t chicle_partition_sizes(chicle_glm_t *h, int32_t K, uint64_t seed, const int64_t *host_sizes);

/* ---- mobile data chunks (Sec. 3 core concepts: the samples live in many small fixed-size chunks that the scheduler
 * moves between immobile tasks; Sec. 4.4: a chunk holds samples and their per-sample state, their number varies with
 * their size). The five functions below are host-side integer logic: all pointers are HOST arrays, no GPU is touched,
 * no handle is needed. A placement is `chunk_off` (n_chunks + 1 ascending coordinate offsets, chunk c = coordinates
 * chunk_off[c] .. chunk_off[c+1]-1 in id order) and `chunk_task` (n_chunks task numbers). The paper fixes none of the
 * integer rules; the ones stated here are this library's. ---- */

/* Cuts the coordinates into chunks of at most chunk_bytes: coordinate i occupies 8 bytes per stored entry (sparse:
 * host_indptr[i+1] - host_indptr[i] entries; dense: host_indptr NULL and 4 * dense_dim bytes instead) plus 8 bytes of
 * state; a chunk is closed in front of the coordinate that would take it above chunk_bytes and holds at least one
 * coordinate. host_chunk_off needs room for n_coord + 1 entries. Returns the number of chunks, or -1 on bad arguments. */
int64_t chicle_chunks_cut(int64_t n_coord, const int64_t *host_indptr, int64_t dense_dim, int64_t chunk_bytes,
                          int64_t *host_chunk_off);

/* First placement (Appendix, baseline comparisons: data is assigned to tasks at random): the chunks, ordered by (mix64(mix64(seed) ^ chunk),
 * chunk), are dealt in K consecutive runs, the first n_chunks mod K tasks getting one more. 1 <= K <= n_chunks. */
chicle_status_t chicle_chunks_assign(int64_t n_chunks, int32_t K, uint64_t seed, int32_t *host_chunk_task);

/* Scale-in (Sec. 4.5 elastic scaling policy: the chunks of to-be-freed tasks are redistributed round-robin): tasks
 * K_new .. K_old-1 are freed; their chunks, in ascending chunk number, go to tasks 0, 1, .., K_new-1, 0, .. in turn.
 * No other chunk moves. In place. 1 <= K_new <= K_old. */
chicle_status_t chicle_chunks_scale_in(int64_t n_chunks, int32_t K_old, int32_t K_new, int32_t *host_chunk_task);

/* Scale-out (Sec. 4.5; Sec. 5.3: the chunks moved to new tasks are picked at random from every old task, which
 * reshuffles the samples): old task j, holding m_j chunks, gives away floor(m_j * (K_new - K_old) / K_new) of them,
 * the first ones in the order (mix64(mix64(seed ^ 0xA0761D6478BD642F) ^ chunk), chunk); the chunks given away are
 * dealt to tasks K_old .. K_new-1 in turn, old tasks in ascending order, the turn carrying over. No other chunk
 * moves. In place. 1 <= K_old <= K_new; a task number outside [0, K_old) on entry: CHICLE_ERR_INVALID_ARG. */
chicle_status_t chicle_chunks_scale_out(int64_t n_chunks, int32_t K_old, int32_t K_new, uint64_t seed,
                                        int32_t *host_chunk_task);

/* One step of the rebalancing policy (Sec. 4.5: chunks move gradually from slower to faster tasks until the
 * difference is below one chunk's processing time). host_time_per_sample[k] is task k's time per sample (the caller's
 * median over its window). A task's round time is its samples times that. The task with the longest round time (ties:
 * lowest number) gives its highest-numbered chunk to the task with the shortest (ties: lowest number), unless the two
 * times differ by no more than that chunk's processing time on the slow task, or the slow task holds one chunk only.
 * Returns 1 if a chunk moved, 0 if not, -1 on bad arguments. */
int chicle_chunks_rebalance_step(int64_t n_chunks, const int64_t *host_chunk_off, int32_t K,
                                 const double *host_time_per_sample, int32_t *host_chunk_task);

/* The partition a placement induces: coordinate i belongs to the task of its chunk; members in ascending id order
 * inside a partition (the owner map and the member lists are built on the device). Otherwise as chicle_partition:
 * legal between rounds, keeps alpha, v and the round counter (the state moves with the samples, Sec. 4.4); `seed` keys
 * the visiting orders of the rounds that follow. K <= n_chunks <= coordinates, offsets from 0 to the number of
 * coordinates and strictly increasing, tasks in [0, K), every task holding a chunk: else CHICLE_ERR_INVALID_ARG and
 * the handle is unchanged. The host arrays are read during the call. */
chicle_status_t chicle_partition_chunks(chicle_glm_t *h, int32_t K, uint64_t seed, int64_t n_chunks,
                                        const int64_t *host_chunk_off, const int32_t *host_chunk_task);

/* One CoCoA round (Sec. 2.2 Eq. 1, Eq. 2 and worker structure with L = 1; Sec. 5.1: SCD local solver, sigma =
 * number of tasks). Each partition draws this round's seeded visiting order (members ordered by
 * mix64(mix64(seed ^ 0xD1B54A32D192ED03) ^ mix64(round * 2^32 + epoch) ^ id)), walks it strictly in order for H
 * coordinate steps (H = 0: one local epoch, i.e. as many steps as the partition has coordinates) against
 * v_local = v + sigma' * (its own update so far), then v += sum_k dv_k in ascending k and the round counter
 * advances. sigma_prime > 0; sigma' >= K guarantees dual ascent. Asynchronous unless `stats` is non-NULL, in
 * which case the stream is synchronised and *stats filled. */
chicle_status_t chicle_cocoa_round(chicle_glm_t *h, int64_t H, float sigma_prime, chicle_round_stats_t *stats);

/* The same round with a step budget per partition (Sec. 3: the number of samples a task processes in an iteration is
 * set per task, so that slow and fast tasks finish together; Sec. 4.5). Partition k takes host_steps[k] coordinate
 * steps along the first host_steps[k] entries of the visiting order that chicle_cocoa_round would walk this round
 * (a host array of K entries, read during the call; 0 <= host_steps[k] <= size of partition k, else
 * CHICLE_ERR_INVALID_ARG and nothing is enqueued). A partition with budget 0 sits the round out; with every budget
 * equal to H (or to the partition's size) the result is chicle_cocoa_round's with that H (or H = 0), bit for bit.
 * The round counter advances even if every budget is 0. stats->steps is the sum of the budgets. */
chicle_status_t chicle_cocoa_round_steps(chicle_glm_t *h, const int64_t *host_steps, float sigma_prime,
                                         chicle_round_stats_t *stats);

/* ---- One job on several GPUs: the partitions spread over ranks, the shared vector replicated (Sec. 4.2 "Trainer and
 * solver": every iteration the trainer merges the solvers' updates and broadcasts the model; Sec. 4.3: that exchange is
 * one model-sized vector per task; Appendix "Example application"). Every rank creates a handle over the same data
 * and calls chicle_partition with the same K and seed, so all ranks hold the same partition map, visiting orders and
 * (in sparse formats) the same internal numbering of the entries. A rank then runs only the partitions it owns, the
 * ranks exchange their summed updates (an all-gather of `dim` floats per rank, done by the caller with any collective
 * library: the library itself never touches another GPU's memory), and every rank applies all of them in rank order.
 *
 * chicle_cocoa_round_delta: chicle_cocoa_round_steps (budget 0 for the partitions of other ranks), except that the sum
 * of the partitions' updates, in ascending k with an fp64 accumulator, is written to dev_delta (a device array of
 * `len` = length of the shared vector floats, in the library's internal order of the entries: only meaningful to
 * chicle_apply_deltas of a handle over the same data) and v is left as it was. The round counter advances.
 *
 * chicle_apply_deltas: v += dev_deltas[0] + ... + dev_deltas[count - 1] (count vectors of `len` floats one behind the
 * other on the device, added in that order with an fp64 accumulator; ridge: the residual is refreshed). Ranks that
 * apply the same vectors in the same order keep bit-identical copies of v. With one rank, a round_delta followed by
 * apply_deltas equals chicle_cocoa_round_steps up to one rounding per entry (the sum is rounded to fp32 before it
 * is added).
 *
 * chicle_export_state_of / chicle_import_state: the per-coordinate state (alpha, or w for ridge) is only current on
 * the rank that owns the coordinate's partition. export writes to dev_out (device, one float per coordinate) the
 * state of the coordinates whose partition k has host_keep[k] != 0 (K bytes on the host, read during the call) and 0
 * elsewhere; summing the ranks' exports (exact: one non-zero term per coordinate) gives the whole state, which import
 * copies into the handle. Needed before chicle_duality_gap, chicle_get_alpha and before a new partition changes the
 * ownership. All four calls are asynchronous on the handle's stream; bad arguments give CHICLE_ERR_INVALID_ARG with
 * nothing enqueued. */
chicle_status_t chicle_cocoa_round_delta(chicle_glm_t *h, const int64_t *host_steps, float sigma_prime, float *dev_delta,
                                         int64_t len, chicle_round_stats_t *stats);
chicle_status_t chicle_apply_deltas(chicle_glm_t *h, const float *dev_deltas, int32_t count, int64_t len);
chicle_status_t chicle_export_state_of(chicle_glm_t *h, const uint8_t *host_keep, float *dev_out, int64_t len);
chicle_status_t chicle_import_state(chicle_glm_t *h, const float *dev_state, int64_t len);

/* Duality gap P(w(alpha)) - D(alpha) of the current state (Sec. 4.1, Sec. 5: the metric solvers report), with
 * fp64 accumulation in a fixed order. host_gap / host_primal / host_dual may each be NULL. Synchronises. */
chicle_status_t chicle_duality_gap(chicle_glm_t *h, double *host_gap, double *host_primal, double *host_dual);

/* Copy out the state. `len` must equal the array's length: alpha has one entry per coordinate (n_rows for the
 * dual losses, n_cols = w for ridge); v has n_cols entries for the dual losses and n_rows for ridge. `space` says
 * where `out` lives. Synchronises. */
chicle_status_t chicle_get_alpha(chicle_glm_t *h, float *out, int64_t len, chicle_memspace_t space);
chicle_status_t chicle_get_v(chicle_glm_t *h, float *out, int64_t len, chicle_memspace_t space);

/* Partition map: host_owner[c] = partition of coordinate c; len = number of coordinates. Synchronises. */
chicle_status_t chicle_get_partition(chicle_glm_t *h, int32_t *host_owner, int64_t len);

/* Visiting order of partition k in local epoch 0 of round `round` under the current partition (any round >= 0, not
 * only the current one). len must equal the partition's size. Synchronises. */
chicle_status_t chicle_get_permutation(chicle_glm_t *h, int64_t round, int32_t k, int32_t *host_out, int64_t len);

/* Overwrite the state (checkpoint restore, or re-synchronising with an external trajectory). host_alpha has one
 * entry per coordinate; host_v may be NULL, in which case v is recomputed from alpha on the device
 * (v = X^T alpha, or X w) with floating-point atomics, whose order of additions is not fixed: unlike everything else
 * in the library, a v rebuilt this way (and what later rounds make of it) may differ in the last bits from run to run;
 * pass host_v for bit-reproducible runs. `round` >= 0 becomes the round counter. Synchronises. */
chicle_status_t chicle_set_state(chicle_glm_t *h, const float *host_alpha, const float *host_v, int64_t round);

/* Current round counter, partition count and coordinate / shared-vector lengths; any pointer may be NULL. */
chicle_status_t chicle_get_info(const chicle_glm_t *h, int64_t *round, int32_t *K, int64_t *n_coord, int64_t *dim);

/* Largest problem chicle_partition_noalloc accepts: its workspace is a fixed array inside the library image. */
#define CHICLE_NOALLOC_MAX_COORDS 131072

/* The partition map of chicle_partition, for callers that must not allocate device memory. (The paper has no
 * counterpart: this entry point exists for deployment reasons only.) Who needs it: code that asks for a partition
 * map from a place where the device allocator is off limits, e.g. a serving or real-time loop whose memory pool was
 * sized and frozen at start-up, a thread that holds a lock the allocator also wants, or a process whose device
 * memory is handed out by another component. chicle_partition allocates its sort workspace and the K x dim update
 * buffers; this call allocates nothing, on the host or on the device: no cudaMalloc, cudaFree, or framework
 * allocator. Its workspace (about 3.2 MB) is a static device array that every GPU loading this library holds until
 * the process ends.
 *   device, cuda_stream   where to run; the work is enqueued on the stream and the call does not synchronise.
 *   n_coord, K, seed      as in chicle_partition: 1 <= K <= n_coord <= CHICLE_NOALLOC_MAX_COORDS. A larger n_coord
 *                         is refused with CHICLE_ERR_UNSUPPORTED and a message; nothing is launched.
 *   dev_owner             out, device, n_coord int32: partition of every coordinate (what chicle_get_partition returns).
 *   dev_members           out, device, n_coord int32: coordinate ids grouped by partition, ascending inside a partition;
 *                         partition k occupies [off_k, off_{k+1}) with off_k = k*(n/K) + min(k, n mod K).
 *   host_errbuf           optional host buffer of errbuf_len bytes that receives the error text (no handle exists to
 *                         keep it). The caller owns both output arrays and the buffer.
 * The first call on a device looks up the device address of the workspace (cudaGetSymbolAddress) and remembers it;
 * make that first call outside any stream capture. That first call is also the one exception to "allocates
 * nothing": the CUDA runtime loads kernels and static device arrays lazily, so the lookup and the first launch of
 * each kernel may make the driver set device memory aside for the library's image. Callers with a frozen memory
 * budget make one call at start-up, before the region in which nothing may be allocated; every later call on that
 * device leaves the free device memory as it found it. The call makes `device` the current device of the calling
 * thread and leaves it so. All calls on a device share the one workspace, and it keeps
 * whatever the previous call left in it; nothing in it needs clearing because every pass overwrites what it then
 * reads. Two calls whose kernels overlap on the same GPU (different streams, or different host threads) race on it:
 * serialise them. Results are bit-identical to chicle_partition's. */
chicle_status_t chicle_partition_noalloc(int device, void *cuda_stream, int64_t n_coord, int32_t K, uint64_t seed,
                                         int32_t *dev_owner, int32_t *dev_members, char *host_errbuf,
                                         size_t errbuf_len);

/* Text of the last error on this handle (library-owned, valid until the next call on the handle). With h = NULL:
 * the text of the last failed chicle_glm_create on this thread. Never NULL. */
const char *chicle_last_error(const chicle_glm_t *h);

/* Release everything the handle owns. NULL is allowed. */
void chicle_glm_destroy(chicle_glm_t *h);

#ifdef __cplusplus
}
#endif
#endif /* CHICLE_H */
