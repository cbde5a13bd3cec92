// Internal declarations shared by the translation units of libchicle (not part of the public ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <string>

#include "chicle.h"

namespace chicle {

// ---- device status word (bit set by kernels, read by synchronising host calls) -------------------------
enum : uint32_t {
    ST_NONFINITE_INPUT = 1u << 0,  // NaN/Inf in values or labels
    ST_BAD_LABEL = 1u << 1,        // label not +-1 for a dual loss
    ST_BAD_INDEX = 1u << 2,        // index outside [0, dim) or indptr not monotone
    ST_WAIT_TIMEOUT = 1u << 3,     // a bounded wait inside a kernel ran out
    ST_NONFINITE_STEP = 1u << 4,   // a coordinate step produced NaN/Inf
    ST_BOUNDS = 1u << 5,           // a -DCHICLE_DEBUG_BOUNDS build: an index that a kernel loaded lay outside its array
};

// A -DCHICLE_DEBUG_BOUNDS build checks every index that the solvers and the gap kernels load from memory (visiting
// order entries, row extents, entry ids, record directory entries, record sizes) before it is used as an address.
// A failed check sets ST_BOUNDS in the status word and the access is skipped (the value is replaced by a harmless
// one): never a trap, never an out-of-range access. The normal build compiles the checks away.
#ifdef CHICLE_DEBUG_BOUNDS
#define CHICLE_IN_BOUNDS(status, cond) ((cond) ? true : (atomicOr((status), (uint32_t)ST_BOUNDS), false))
#else
#define CHICLE_IN_BOUNDS(status, cond) true
#endif


// One SplitMix64 output for state x (published generator; a bijection on 64-bit words).
__host__ __device__ __forceinline__ uint64_t mix64(uint64_t x)
{
    uint64_t z = x + 0x9E3779B97F4A7C15ULL;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
    return z ^ (z >> 31);
}
constexpr uint64_t kPermStream = 0xD1B54A32D192ED03ULL;

// ---- radix sort over (64-bit key, 32-bit value) pairs -------------------------------------------------------
constexpr int kSortThreads = 256;
constexpr int kSortItems = 16;
constexpr int kSortTile = kSortThreads * kSortItems;  // elements per block and pass

struct SortWorkspace {
    uint64_t *keys[2] = {nullptr, nullptr};
    int32_t *vals[2] = {nullptr, nullptr};
    uint32_t *hist = nullptr;      // 256 * nblk digit-major counters
    uint32_t *scan_sums = nullptr; // one per scan tile
    int64_t capacity = 0;          // elements
    int nblk = 0;
};

size_t sort_hist_entries(int64_t n);
size_t sort_scan_tiles(int64_t n);

// Stable LSD pass on 8 bits. digit = (keys_in[i] >> shift) & 255 when owner == nullptr, else
// (owner[vals_in[i]] >> shift) & 255. keys may be nullptr in owner mode (only values move).
cudaError_t radix_pass(const uint64_t *keys_in, const int32_t *vals_in, uint64_t *keys_out, int32_t *vals_out,
                       const int32_t *owner, int64_t n, int shift, uint32_t *hist, uint32_t *scan_sums,
                       cudaStream_t stream);

struct SolverParams;

// ---- handle -------------------------------------------------------------------------------------------------
struct Glm {
    int device = 0;
    cudaStream_t stream = nullptr;
    chicle_allocator_t alloc{nullptr, nullptr, nullptr};
    chicle_loss_t loss = CHICLE_LOSS_HINGE_DUAL;
    chicle_format_t fmt = CHICLE_FMT_DENSE_ROWMAJOR;
    int64_t n_rows = 0, n_cols = 0, nnz = 0;
    int64_t n_coord = 0; // coordinates: rows (dual losses) or columns (ridge)
    int64_t dim = 0;     // length of the shared vector
    int64_t n_examples = 0;
    float lambda = 0.f;

    // coordinate-major matrix on the device (dense: indptr/indices null, row c at values + c*dim)
    int64_t *indptr = nullptr;
    int32_t *indices = nullptr;
    float *values = nullptr;
    float *labels = nullptr; // per example
    float *sqnorm = nullptr; // per coordinate
    float *alpha = nullptr;  // per coordinate: signed dual variable, or w for ridge
    float *v = nullptr;      // shared vector, dim
    float *resid = nullptr;  // ridge only: v - y, refreshed by the reduction kernel
    // sparse problems: entry ids (positions in v) are frequency-ranked inside the library
    int32_t *new_of_old = nullptr; // dim; nullptr when ids are not remapped (dense)
    int32_t *old_of_new = nullptr; // dim
    float *perm_tmp = nullptr;     // dim, staging for translating v at the boundary
    int hot_variant = 0;           // 1 / 2: most non-zeros fall on the first ids, the solver keeps those in a direct
                                   // array (2: with room for coordinates of up to 128 entries); 0: flat ids

    // partition
    int32_t K = 0;
    uint64_t seed = 0;
    int32_t *owner = nullptr;   // n_coord
    int32_t *members = nullptr; // n_coord, grouped by partition, ascending id inside
    int64_t *part_off = nullptr; // K+1 (device)
    int64_t *h_part_off = nullptr; // K+1 (host)
    int64_t min_nk = 0;            // smallest partition
    int64_t *d_steps = nullptr;    // K (device, behind part_off): the step budgets of a round that gives each partition its own
    const int64_t *round_steps = nullptr; // the same on the host while such a round is being enqueued, else nullptr
    int32_t *perm = nullptr;    // epochs * n_coord
    int64_t perm_epochs = 0;
    float *U = nullptr;         // K * dim: per-partition accumulated update, zero between rounds
    int64_t U_rows = 0;

    // look-ahead solver: the per-block records that its prepare kernel writes every round (nullptr when they could
    // not be allocated: the blocked solver runs instead). The buffer is a ring of regions, one slice of a round each.
    void *la_rec = nullptr;
    void *la_dir = nullptr;          // per region: cluster-size entries per block
    unsigned long long *la_cursor = nullptr; // [r]: bytes of region r's pool handed out; [8..]: timing scratch
    size_t la_region_bytes = 0, la_pool_off = 0, la_dir_bytes = 0;
    int64_t la_region_blocks = 0;    // blocks a region has records for
    int la_regions = 0;
    int la_logC = 0;                 // log2 of the CTAs per partition (thread-block cluster)
    int la_depth = 2;                // blocks the dot products are taken ahead of the recurrence (2: with cross Gram matrices)
    bool la_overlap = true;          // prepare kernels beside the chain kernels (side stream) or alternating with them
    int32_t la_nzcap = 0, la_hotc = 0; // non-zeros per worker record; entry ids per CTA kept in shared memory
    size_t la_smem = 0;              // dynamic shared memory of the chain kernel
    int la_last_slices = 0;          // slices of the last round
    int solver_launches = 0;         // kernels the local solvers launched in the round being enqueued
    int64_t *la_blk_base = nullptr;  // per slice K+1: first block of each partition in the slice's numbering of the blocks
    int64_t *la_slice = nullptr;     // per slice 2K: every partition's step count and first step in that slice
    cudaStream_t la_stream = nullptr; // side stream (lowest priority) for the later slices' prepare kernels
    cudaEvent_t *la_ev_prep = nullptr; // per slice: its records are written
    cudaEvent_t *la_ev_done = nullptr; // per slice: its chain launch is done (its region is free)
    bool time_prepare = false; // record ev[4] between the prepare and the chain kernel (round statistics asked for)

    SortWorkspace sortws;
    double *gap_partials = nullptr; // gap kernel partial sums
    int gap_blocks = 0;
    double *gap_out = nullptr;      // 8 doubles on the device
    uint32_t *d_status = nullptr;
    uint32_t *h_status = nullptr;   // pinned
    double *h_gap = nullptr;        // pinned, 8 doubles

    int64_t round = 0;
    int sm_count = 148;
    int max_smem_optin = 0;
    cudaEvent_t ev[5] = {nullptr, nullptr, nullptr, nullptr, nullptr};
    std::string err;
};

// ---- kernels' host launchers (each returns the launch error, work is enqueued on g.stream) -----------------
cudaError_t launch_validate(Glm &g, bool values = true, bool rest = true); // the values array; labels and structure
cudaError_t launch_sqnorm(Glm &g);
cudaError_t launch_partition(Glm &g, int32_t K, uint64_t seed);           // fills owner, members
cudaError_t launch_partition_chunks(Glm &g, int32_t K, int64_t C, const int64_t *chunk_off, const int32_t *chunk_task); // device arrays
cudaError_t launch_permutation(Glm &g, int64_t round, int64_t epochs);    // fills perm[epochs * n_coord]
cudaError_t launch_local_solver(Glm &g, int64_t H, float sigma_prime, int *variant);
cudaError_t launch_reduce(Glm &g);                                        // v += sum_k U_k ; U = 0 ; resid
cudaError_t launch_sum_updates(Glm &g, float *delta);                     // delta = sum_k U_k ; U = 0 (v untouched)
cudaError_t launch_apply_deltas(Glm &g, const float *deltas, int count);  // v += sum_g deltas[g] ; resid
cudaError_t launch_mask_state(Glm &g, const unsigned char *keep, float *out); // out = state where keep[owner], else 0
cudaError_t launch_gap(Glm &g);                                           // fills gap_out[0..2]
cudaError_t launch_shared_vector(Glm &g);                                 // v = X^T alpha (or X w) from scratch
cudaError_t launch_refresh_resid(Glm &g);                                 // ridge: resid = v - y
cudaError_t launch_frequency_remap(Glm &g, uint32_t *counts, uint64_t *keys[2], int32_t *vals[2], uint32_t *hist,
                                   uint32_t *scan_sums, int64_t hot_ids, int32_t long_len, unsigned long long *mass);
cudaError_t launch_gather_f32(Glm &g, const float *src, const int32_t *map, int64_t n, float *dst); // dst[i] = src[map[i]]
cudaError_t launch_lookahead_solver(Glm &g, const struct SolverParams &P);
void lookahead_plan(Glm &g, int32_t K); // fills the la_* sizes for a partition into K
int lookahead_max_dense_dim();
int lookahead_max_slices();
int64_t lookahead_max_dim();
int blocked_solver_hot_ids();
int blocked_solver_short_cap();

} // namespace chicle
