// Host side of the C ABI declared in chicle.h: argument checks, the state machine, memory, and the order in
// which the kernels of a round are enqueued. No arithmetic of the method happens here.
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "chicle_internal.cuh"

namespace chicle {
bool solver_supports_dense(int64_t dim, int max_smem_optin);
}

using namespace chicle;

struct chicle_glm : public chicle::Glm {
    std::vector<void *> owned; // every device allocation, for destroy
};

namespace {

thread_local std::string g_create_error;

// CHICLE_LOG=1 in the environment: every failed call and every round writes a line to stderr (a round is then
// synchronised for its timings, like a round that was asked for statistics).
int log_level()
{
    static const int level = [] {
        const char *env = getenv("CHICLE_LOG");
        return env ? atoi(env) : 0;
    }();
    return level;
}

chicle_status_t fail(chicle_glm *h, chicle_status_t st, const std::string &msg)
{
    if (h) h->err = msg;
    else g_create_error = msg;
    if (log_level() >= 1) fprintf(stderr, "[chicle] error %d: %s\n", (int)st, msg.c_str());
    return st;
}

chicle_status_t fail_cuda(chicle_glm *h, cudaError_t e, const char *what)
{
    // A failed launch or copy: clear the sticky-less error so later calls report their own.
    (void)cudaGetLastError();
    const chicle_status_t st = e == cudaErrorMemoryAllocation ? CHICLE_ERR_OOM : CHICLE_ERR_CUDA;
    return fail(h, st, std::string(what) + ": " + cudaGetErrorString(e));
}

void *dev_alloc(chicle_glm *h, size_t bytes)
{
    if (bytes == 0) bytes = 256;
    void *p = nullptr;
    if (h->alloc.alloc) {
        p = h->alloc.alloc(h->alloc.ctx, bytes);
    } else if (cudaMalloc(&p, bytes) != cudaSuccess) {
        (void)cudaGetLastError();
        p = nullptr;
    }
    if (p) h->owned.push_back(p);
    return p;
}

void dev_free(chicle_glm *h, void *p)
{
    if (!p) return;
    for (size_t i = 0; i < h->owned.size(); ++i)
        if (h->owned[i] == p) {
            h->owned[i] = h->owned.back();
            h->owned.pop_back();
            break;
        }
    if (h->alloc.free) h->alloc.free(h->alloc.ctx, p);
    else (void)cudaFree(p);
}

template <typename T> bool alloc_into(chicle_glm *h, T *&dst, size_t count)
{
    dst = static_cast<T *>(dev_alloc(h, count * sizeof(T)));
    return dst != nullptr;
}

cudaError_t copy_in(void *dst, const void *src, size_t bytes, chicle_memspace_t space, cudaStream_t s)
{
    return cudaMemcpyAsync(dst, src, bytes, space == CHICLE_MEM_HOST ? cudaMemcpyHostToDevice : cudaMemcpyDeviceToDevice, s);
}

// Reads and clears the device status word. Stream must be idle or the caller accepts a sync here.
chicle_status_t check_status(chicle_glm *h)
{
    cudaError_t e = cudaMemcpyAsync(h->h_status, h->d_status, sizeof(uint32_t), cudaMemcpyDeviceToHost, h->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(h->stream);
    if (e != cudaSuccess) return fail_cuda(h, e, "status read");
    const uint32_t bits = *h->h_status;
    if (bits == 0) return CHICLE_OK;
    (void)cudaMemsetAsync(h->d_status, 0, sizeof(uint32_t), h->stream);
    if (bits & ST_BOUNDS) return fail(h, CHICLE_ERR_INTERNAL, "a bounds check of a CHICLE_DEBUG_BOUNDS build failed");
    if (bits & ST_WAIT_TIMEOUT) return fail(h, CHICLE_ERR_TIMEOUT, "a bounded wait inside a kernel ran out");
    if (bits & ST_BAD_INDEX) return fail(h, CHICLE_ERR_INVALID_ARG, "indptr not monotone or an index out of range");
    if (bits & ST_BAD_LABEL) return fail(h, CHICLE_ERR_INVALID_ARG, "labels must be +1 or -1 for hinge and logistic");
    if (bits & ST_NONFINITE_INPUT) return fail(h, CHICLE_ERR_NUMERIC, "NaN or Inf in values or labels");
    return fail(h, CHICLE_ERR_NUMERIC, "a coordinate step produced a non-finite value");
}

void destroy_impl(chicle_glm *h)
{
    if (!h) return;
    (void)cudaSetDevice(h->device);
    (void)cudaStreamSynchronize(h->stream);
    if (h->la_stream) {
        (void)cudaStreamSynchronize(h->la_stream);
        (void)cudaStreamDestroy(h->la_stream);
    }
    for (int i = 0; i < lookahead_max_slices(); ++i) {
        if (h->la_ev_prep && h->la_ev_prep[i]) (void)cudaEventDestroy(h->la_ev_prep[i]);
        if (h->la_ev_done && h->la_ev_done[i]) (void)cudaEventDestroy(h->la_ev_done[i]);
    }
    delete[] h->la_ev_prep;
    delete[] h->la_ev_done;
    while (!h->owned.empty()) dev_free(h, h->owned.back());
    if (h->h_status) (void)cudaFreeHost(h->h_status);
    if (h->h_gap) (void)cudaFreeHost(h->h_gap);
    delete[] h->h_part_off;
    for (auto &ev : h->ev)
        if (ev) (void)cudaEventDestroy(ev);
    (void)cudaGetLastError();
    delete h;
}

} // namespace

extern "C" {

chicle_status_t chicle_glm_create(const chicle_matrix_t *X, const float *labels, float lambda, chicle_loss_t loss,
                                  int device, void *cuda_stream, const chicle_allocator_t *alloc, chicle_glm_t **out)
{
    if (!X || !labels || !out) return fail(nullptr, CHICLE_ERR_INVALID_ARG, "X, labels and out must be non-NULL");
    if (!(lambda > 0.0f) || !(lambda < 3.0e38f)) return fail(nullptr, CHICLE_ERR_INVALID_ARG, "lambda must be positive and finite");
    if (X->n_rows <= 0 || X->n_cols <= 0) return fail(nullptr, CHICLE_ERR_INVALID_ARG, "empty matrix");
    if (X->n_rows > INT32_MAX || X->n_cols > INT32_MAX)
        return fail(nullptr, CHICLE_ERR_UNSUPPORTED, "more than 2^31-1 rows or columns");
    if ((int)loss < 0 || (int)loss > 2 || (int)X->fmt < 0 || (int)X->fmt > 2 || ((int)X->space != 0 && (int)X->space != 1))
        return fail(nullptr, CHICLE_ERR_INVALID_ARG, "unknown loss, format or memory space");
    const bool ridge = loss == CHICLE_LOSS_RIDGE_PRIMAL;
    if (ridge ? X->fmt != CHICLE_FMT_CSC : X->fmt == CHICLE_FMT_CSC)
        return fail(nullptr, CHICLE_ERR_UNSUPPORTED, "hinge/logistic take dense or CSR, ridge takes CSC");
    const bool dense = X->fmt == CHICLE_FMT_DENSE_ROWMAJOR;
    if (!X->values) return fail(nullptr, CHICLE_ERR_INVALID_ARG, "values is NULL");
    if (dense ? X->ld < X->n_cols : (!X->indptr || (X->nnz > 0 && !X->indices) || X->nnz < 0))
        return fail(nullptr, CHICLE_ERR_INVALID_ARG, dense ? "ld < n_cols" : "indptr/indices missing or nnz < 0");
    if (alloc && ((alloc->alloc == nullptr) != (alloc->free == nullptr)))
        return fail(nullptr, CHICLE_ERR_INVALID_ARG, "allocator needs both callbacks or neither");

    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev <= 0) {
        (void)cudaGetLastError();
        return fail(nullptr, CHICLE_ERR_CUDA, "no CUDA device available: this library has no host path");
    }
    if (device < 0 || device >= ndev) return fail(nullptr, CHICLE_ERR_INVALID_ARG, "device out of range");
    cudaError_t e = cudaSetDevice(device);
    if (e != cudaSuccess) return fail_cuda(nullptr, e, "cudaSetDevice");

    chicle_glm *h = new (std::nothrow) chicle_glm();
    if (!h) return fail(nullptr, CHICLE_ERR_OOM, "host allocation failed");
    h->device = device;
    h->stream = static_cast<cudaStream_t>(cuda_stream);
    if (alloc && alloc->alloc) h->alloc = *alloc;
    h->loss = loss;
    h->fmt = X->fmt;
    h->n_rows = X->n_rows;
    h->n_cols = X->n_cols;
    h->nnz = dense ? 0 : X->nnz;
    h->n_coord = ridge ? X->n_cols : X->n_rows;
    h->dim = ridge ? X->n_rows : X->n_cols;
    h->n_examples = X->n_rows;
    h->lambda = lambda;
    cudaDeviceProp prop;
    e = cudaGetDeviceProperties(&prop, device);
    if (e != cudaSuccess) { destroy_impl(h); return fail_cuda(nullptr, e, "cudaGetDeviceProperties"); }
    h->sm_count = prop.multiProcessorCount;
    h->max_smem_optin = (int)prop.sharedMemPerBlockOptin;
    if (prop.major < 10) {
        destroy_impl(h);
        return fail(nullptr, CHICLE_ERR_UNSUPPORTED, "built for sm_100a; this device is older");
    }
    if (dense && !solver_supports_dense(h->dim, h->max_smem_optin)) {
        destroy_impl(h);
        return fail(nullptr, CHICLE_ERR_UNSUPPORTED, "dense rows too long for the shared-memory solver; pass CSR");
    }

    auto bail = [&](chicle_status_t st, const std::string &msg) {
        destroy_impl(h);
        return fail(nullptr, st, msg);
    };
    auto bail_cuda = [&](cudaError_t err, const char *what) {
        destroy_impl(h);
        return fail_cuda(nullptr, err, what);
    };

    const size_t nvals = dense ? (size_t)h->n_coord * (size_t)h->dim : (size_t)h->nnz;
    // 4 spare elements behind values and indices: the solver's 16-byte bulk copies of a coordinate may read up to
    // 12 bytes past its last entry
    bool ok = alloc_into(h, h->values, nvals + 4) && alloc_into(h, h->labels, (size_t)h->n_examples) &&
              alloc_into(h, h->sqnorm, (size_t)h->n_coord) && alloc_into(h, h->alpha, (size_t)h->n_coord) &&
              alloc_into(h, h->v, (size_t)h->dim) && alloc_into(h, h->d_status, 64) &&
              alloc_into(h, h->gap_out, 8);
    if (ok && !dense) ok = alloc_into(h, h->indptr, (size_t)h->n_coord + 1) && alloc_into(h, h->indices, nvals + 4);
    if (ok && ridge) ok = alloc_into(h, h->resid, (size_t)h->dim);
    h->gap_blocks = h->sm_count * 8;
    if (ok) ok = alloc_into(h, h->gap_partials, (size_t)h->gap_blocks * 4);
    if (!ok) return bail(CHICLE_ERR_OOM, "device allocation failed");
    if (cudaMallocHost(&h->h_status, 64) != cudaSuccess || cudaMallocHost(&h->h_gap, 64) != cudaSuccess)
        return bail(CHICLE_ERR_OOM, "pinned host allocation failed");
    for (auto &ev : h->ev)
        if ((e = cudaEventCreate(&ev)) != cudaSuccess) return bail_cuda(e, "cudaEventCreate");
    {
        // the look-ahead solver's side stream: lowest priority, so that the chain kernels get their SMs first, and
        // non-blocking, so that it does not order itself against the legacy default stream
        int least = 0, greatest = 0;
        (void)cudaDeviceGetStreamPriorityRange(&least, &greatest);
        if ((e = cudaStreamCreateWithPriority(&h->la_stream, cudaStreamNonBlocking, least)) != cudaSuccess)
            return bail_cuda(e, "cudaStreamCreateWithPriority");
        const int ns = lookahead_max_slices();
        h->la_ev_prep = new (std::nothrow) cudaEvent_t[(size_t)ns]();
        h->la_ev_done = new (std::nothrow) cudaEvent_t[(size_t)ns]();
        if (!h->la_ev_prep || !h->la_ev_done) return bail(CHICLE_ERR_OOM, "host allocation failed");
        for (int i = 0; i < ns; ++i)
            if ((e = cudaEventCreateWithFlags(&h->la_ev_prep[i], cudaEventDisableTiming)) != cudaSuccess ||
                (e = cudaEventCreateWithFlags(&h->la_ev_done[i], cudaEventDisableTiming)) != cudaSuccess)
                return bail_cuda(e, "cudaEventCreate");
    }

    cudaStream_t s = h->stream;
    if (dense) {
        const cudaMemcpyKind kind = X->space == CHICLE_MEM_HOST ? cudaMemcpyHostToDevice : cudaMemcpyDeviceToDevice;
        e = cudaMemcpy2DAsync(h->values, (size_t)h->dim * 4, X->values, (size_t)X->ld * 4, (size_t)h->dim * 4,
                              (size_t)h->n_coord, kind, s);
    } else {
        // The structure first: its checks and the ranking of the ids need no values, so the values (half of the
        // bytes) travel on the side stream, behind the indices, while those kernels run.
        e = copy_in(h->indptr, X->indptr, ((size_t)h->n_coord + 1) * 8, X->space, s);
        if (e == cudaSuccess && nvals) e = copy_in(h->indices, X->indices, nvals * 4, X->space, s);
        if (e == cudaSuccess) e = cudaEventRecord(h->la_ev_prep[0], s);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(h->la_stream, h->la_ev_prep[0], 0);
        if (e == cudaSuccess) e = copy_in(h->values, X->values, nvals * 4, X->space, h->la_stream);
        if (e == cudaSuccess) e = cudaEventRecord(h->la_ev_done[0], h->la_stream);
    }
    if (e == cudaSuccess) e = copy_in(h->labels, labels, (size_t)h->n_examples * 4, X->space, s);
    if (e == cudaSuccess) e = cudaMemsetAsync(h->alpha, 0, (size_t)h->n_coord * 4, s);
    if (e == cudaSuccess) e = cudaMemsetAsync(h->v, 0, (size_t)h->dim * 4, s);
    if (e == cudaSuccess) e = cudaMemsetAsync(h->d_status, 0, 64 * sizeof(uint32_t), s);
    if (e != cudaSuccess) return bail_cuda(e, "copying the inputs");

    if (!dense) {
        // indptr must be sane before anything walks it: check its ends on the host side of the copy
        int64_t ends[2] = {0, 0};
        e = cudaMemcpyAsync(&ends[0], h->indptr, 8, cudaMemcpyDeviceToHost, s);
        if (e == cudaSuccess) e = cudaMemcpyAsync(&ends[1], h->indptr + h->n_coord, 8, cudaMemcpyDeviceToHost, s);
        if (e == cudaSuccess) e = cudaStreamSynchronize(s);
        if (e != cudaSuccess) return bail_cuda(e, "reading indptr");
        if (ends[0] != 0 || ends[1] != h->nnz) return bail(CHICLE_ERR_INVALID_ARG, "indptr[0] != 0 or indptr[last] != nnz");
    }
    e = launch_validate(*h, dense, true); // (sparse: the values are checked once they have arrived, below)
    if (e != cudaSuccess) return bail_cuda(e, "validation kernels");
    chicle_status_t st = check_status(h);
    if (st != CHICLE_OK) {
        const std::string msg = h->err;
        return bail(st, msg);
    }
    if (!dense) {
        // frequency-rank the entry ids (see remap.cu); temporaries are released before returning
        const int64_t dim = h->dim;
        uint32_t *counts = nullptr, *hist = nullptr, *sums = nullptr;
        uint64_t *keys[2] = {nullptr, nullptr};
        int32_t *vals[2] = {nullptr, nullptr};
        unsigned long long *mass = nullptr;
        float *labels_new = nullptr;
        bool ok2 = alloc_into(h, h->new_of_old, (size_t)dim) && alloc_into(h, h->old_of_new, (size_t)dim) &&
                   alloc_into(h, h->perm_tmp, (size_t)dim) && alloc_into(h, counts, (size_t)dim) &&
                   alloc_into(h, keys[0], (size_t)dim) && alloc_into(h, keys[1], (size_t)dim) &&
                   alloc_into(h, vals[0], (size_t)dim) && alloc_into(h, vals[1], (size_t)dim) &&
                   alloc_into(h, hist, sort_hist_entries(dim)) && alloc_into(h, sums, sort_scan_tiles(dim) + 1) &&
                   alloc_into(h, mass, 4);
        if (ok2 && ridge) ok2 = alloc_into(h, labels_new, (size_t)dim);
        if (!ok2) return bail(CHICLE_ERR_OOM, "device allocation failed (id ranking)");
        e = cudaMemsetAsync(counts, 0, (size_t)dim * 4, s);
        if (e == cudaSuccess) e = cudaMemsetAsync(mass, 0, 32, s);
        if (e == cudaSuccess) e = launch_frequency_remap(*h, counts, keys, vals, hist, sums, blocked_solver_hot_ids(), blocked_solver_short_cap(), mass);
        if (e == cudaSuccess && ridge) e = launch_gather_f32(*h, h->labels, h->old_of_new, dim, labels_new);
        unsigned long long host_mass2[2] = {0, 0};
        if (e == cudaSuccess) e = cudaMemcpyAsync(host_mass2, mass, 16, cudaMemcpyDeviceToHost, s);
        if (e == cudaSuccess) e = cudaStreamSynchronize(s);
        if (e != cudaSuccess) return bail_cuda(e, "id ranking kernels");
        if (ridge) {
            dev_free(h, h->labels);
            h->labels = labels_new;
        }
        dev_free(h, counts); dev_free(h, keys[0]); dev_free(h, keys[1]); dev_free(h, vals[0]); dev_free(h, vals[1]);
        dev_free(h, hist); dev_free(h, sums); dev_free(h, mass);
        h->hot_variant = h->nnz > 0 && (double)host_mass2[0] >= 0.5 * (double)h->nnz ? 1 : 0;
        // more than 1 % of the coordinates would not fit the short staging rows: take the variant with longer rows
        if (h->hot_variant && (double)host_mass2[1] > 0.01 * (double)h->n_coord) h->hot_variant = 2;
        const char *force = getenv("CHICLE_FORCE_VARIANT"); // debugging aid
        if (force && strcmp(force, "flat") == 0) h->hot_variant = 0;
        if (force && strcmp(force, "hot") == 0) h->hot_variant = 1;
        if (force && strcmp(force, "hot128") == 0) h->hot_variant = 2;
    }
    if (!dense) {
        e = cudaStreamWaitEvent(s, h->la_ev_done[0], 0);
        if (e == cudaSuccess) e = launch_validate(*h, true, false);
        if (e != cudaSuccess) return bail_cuda(e, "validation kernels");
        st = check_status(h);
        if (st != CHICLE_OK) {
            const std::string msg = h->err;
            return bail(st, msg);
        }
    }
    e = launch_sqnorm(*h);
    if (e == cudaSuccess) e = launch_refresh_resid(*h);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return bail_cuda(e, "preprocessing kernels");
    *out = h;
    return CHICLE_OK;
}

// A placement of data chunks on tasks (host arrays): chunk c holds coordinates off[c] .. off[c + 1] - 1.
struct ChunkPlacement {
    int64_t C;
    const int64_t *off;
    const int32_t *task;
};

static chicle_status_t partition_impl(chicle_glm_t *h, int32_t K, uint64_t seed, const int64_t *sizes, const ChunkPlacement *chunks = nullptr)
{
    if (!h) return CHICLE_ERR_INVALID_ARG;
    if (K < 1 || (int64_t)K > h->n_coord) return fail(h, CHICLE_ERR_INVALID_ARG, "need 1 <= K <= number of coordinates");
    std::vector<int64_t> chunk_sizes;
    if (chunks) {
        const int64_t C = chunks->C;
        if (C < K || C > h->n_coord || !chunks->off || !chunks->task || chunks->off[0] != 0 || chunks->off[C] != h->n_coord)
            return fail(h, CHICLE_ERR_INVALID_ARG, "chunk offsets must run from 0 to the number of coordinates, with K <= chunks <= coordinates");
        chunk_sizes.assign((size_t)K, 0);
        for (int64_t c = 0; c < C; ++c) {
            if (chunks->off[c + 1] <= chunks->off[c]) return fail(h, CHICLE_ERR_INVALID_ARG, "chunk offsets must increase strictly");
            if (chunks->task[c] < 0 || chunks->task[c] >= K) return fail(h, CHICLE_ERR_INVALID_ARG, "a chunk's task must lie in [0, K)");
            chunk_sizes[(size_t)chunks->task[c]] += chunks->off[c + 1] - chunks->off[c];
        }
        for (int32_t k = 0; k < K; ++k)
            if (chunk_sizes[(size_t)k] == 0) return fail(h, CHICLE_ERR_INVALID_ARG, "every task must hold at least one chunk");
        sizes = chunk_sizes.data();
    }
    if (sizes) {
        int64_t tot = 0;
        for (int32_t k = 0; k < K; ++k) {
            if (sizes[k] < 1 || sizes[k] > h->n_coord) return fail(h, CHICLE_ERR_INVALID_ARG, "every partition size must be at least 1");
            tot += sizes[k];
        }
        if (tot != h->n_coord) return fail(h, CHICLE_ERR_INVALID_ARG, "the partition sizes must add up to the number of coordinates");
    }
    cudaError_t e = cudaSetDevice(h->device);
    if (e != cudaSuccess) return fail_cuda(h, e, "cudaSetDevice");
    const int64_t n = h->n_coord;

    // Allocate everything new first so that a failure leaves the handle as it was.
    int32_t *owner = h->owner, *members = h->members, *perm = h->perm;
    bool fresh = false;
    if (!h->owner) {
        fresh = true;
        SortWorkspace w;
        bool ok = alloc_into(h, owner, (size_t)n) && alloc_into(h, members, (size_t)n) && alloc_into(h, perm, (size_t)n) &&
                  alloc_into(h, w.keys[0], (size_t)n) && alloc_into(h, w.keys[1], (size_t)n) &&
                  alloc_into(h, w.vals[0], (size_t)n) && alloc_into(h, w.vals[1], (size_t)n) &&
                  alloc_into(h, w.hist, sort_hist_entries(n)) && alloc_into(h, w.scan_sums, sort_scan_tiles(n) + 1);
        if (!ok) {
            dev_free(h, owner); dev_free(h, members); dev_free(h, perm);
            dev_free(h, w.keys[0]); dev_free(h, w.keys[1]); dev_free(h, w.vals[0]); dev_free(h, w.vals[1]);
            dev_free(h, w.hist); dev_free(h, w.scan_sums);
            return fail(h, CHICLE_ERR_OOM, "device allocation failed (partition workspaces)");
        }
        w.capacity = n;
        h->sortws = w;
    }
    float *U = h->U;
    int64_t *part_off = h->part_off;
    int64_t *h_off = h->h_part_off;
    const bool regrow = K != h->K || !h->U;
    if (regrow) {
        // synchronise before releasing buffers that queued kernels may still use (the side stream's kernels are
        // ordered before the end of the caller's stream in every round that completed; after a failed launch they
        // may not be)
        e = cudaStreamSynchronize(h->stream);
        if (e == cudaSuccess && h->la_stream) e = cudaStreamSynchronize(h->la_stream);
        if (e != cudaSuccess) return fail_cuda(h, e, "stream synchronise");
        float *newU = nullptr;
        int64_t *new_off = nullptr;
        int64_t *new_hoff = new (std::nothrow) int64_t[(size_t)K + 1];
        // release the old update workspace first: at the large configurations two of them do not fit
        dev_free(h, h->U);
        h->U = nullptr;
        bool ok = new_hoff && alloc_into(h, newU, (size_t)K * (size_t)h->dim) && alloc_into(h, new_off, 2 * (size_t)K + 2); // K+1 offsets, then K step budgets
        if (!ok) {
            delete[] new_hoff;
            dev_free(h, newU); dev_free(h, new_off);
            h->K = 0; // the old workspace is gone: a new partition call is required
            if (fresh) { h->owner = owner; h->members = members; h->perm = perm; h->perm_epochs = 1; }
            return fail(h, CHICLE_ERR_OOM, "device allocation failed (K x dim update workspace)");
        }
        dev_free(h, h->part_off);
        delete[] h->h_part_off;
        U = newU; part_off = new_off; h_off = new_hoff;
        // the look-ahead solver's per-round records (their number depends on K); without them the blocked solver runs
        dev_free(h, h->la_rec); dev_free(h, h->la_dir); dev_free(h, h->la_cursor); dev_free(h, h->la_blk_base); dev_free(h, h->la_slice);
        h->la_rec = nullptr; h->la_dir = nullptr; h->la_cursor = nullptr; h->la_blk_base = nullptr; h->la_slice = nullptr;
        const bool dense_fmt = h->fmt == CHICLE_FMT_DENSE_ROWMAJOR;
        if (dense_fmt ? h->dim <= lookahead_max_dense_dim() : h->dim <= lookahead_max_dim()) {
            lookahead_plan(*h, K);
            unsigned char *rec = nullptr, *dir = nullptr;
            if (alloc_into(h, rec, (size_t)h->la_regions * h->la_region_bytes) && alloc_into(h, dir, h->la_dir_bytes) &&
                alloc_into(h, h->la_cursor, 64) &&
                alloc_into(h, h->la_blk_base, (size_t)lookahead_max_slices() * ((size_t)K + 1)) &&
                alloc_into(h, h->la_slice, (size_t)lookahead_max_slices() * 2 * (size_t)K)) {
                h->la_rec = rec;
                h->la_dir = dir;
                (void)cudaMemsetAsync(h->la_cursor, 0, 64 * sizeof(unsigned long long), h->stream);
            } else {
                dev_free(h, rec); dev_free(h, dir); dev_free(h, h->la_cursor); dev_free(h, h->la_blk_base); dev_free(h, h->la_slice);
                h->la_cursor = nullptr; h->la_blk_base = nullptr; h->la_slice = nullptr;
            }
        }
    }
    if (fresh) { h->owner = owner; h->members = members; h->perm = perm; h->perm_epochs = 1; }
    h->U = U; h->part_off = part_off; h->h_part_off = h_off;
    h->d_steps = part_off + K + 1;
    h->U_rows = K;
    const int64_t base = n / K, extra = n % K;
    h_off[0] = 0;
    for (int32_t k = 1; k <= K; ++k) h_off[k] = sizes ? h_off[k - 1] + sizes[k - 1] : (int64_t)k * base + (k < extra ? k : extra);
    h->min_nk = n;
    for (int32_t k = 0; k < K; ++k) h->min_nk = h_off[k + 1] - h_off[k] < h->min_nk ? h_off[k + 1] - h_off[k] : h->min_nk;
    h->K = K;
    h->seed = seed;
    e = cudaMemcpyAsync(part_off, h_off, ((size_t)K + 1) * 8, cudaMemcpyHostToDevice, h->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(U, 0, (size_t)K * (size_t)h->dim * 4, h->stream);
    int64_t *d_coff = nullptr;
    int32_t *d_ctask = nullptr;
    if (chunks && e == cudaSuccess) {
        // the placement travels as two temporary device arrays, released once the kernels that read them are done
        if (!alloc_into(h, d_coff, (size_t)chunks->C + 1) || !alloc_into(h, d_ctask, (size_t)chunks->C)) {
            dev_free(h, d_coff);
            h->K = 0;
            return fail(h, CHICLE_ERR_OOM, "device allocation failed (chunk placement)");
        }
        e = cudaMemcpyAsync(d_coff, chunks->off, ((size_t)chunks->C + 1) * 8, cudaMemcpyHostToDevice, h->stream);
        if (e == cudaSuccess) e = cudaMemcpyAsync(d_ctask, chunks->task, (size_t)chunks->C * 4, cudaMemcpyHostToDevice, h->stream);
        if (e == cudaSuccess) e = launch_partition_chunks(*h, K, chunks->C, d_coff, d_ctask);
    } else if (e == cudaSuccess) {
        e = launch_partition(*h, K, seed);
    }
    // the host copy of part_off is reused by later calls, so finish the upload before returning
    if (e == cudaSuccess) e = cudaStreamSynchronize(h->stream);
    if (d_coff) dev_free(h, d_coff);
    if (d_ctask) dev_free(h, d_ctask);
    if (e != cudaSuccess) {
        h->K = 0; // the partition map is not valid: a new partition call is required
        return fail_cuda(h, e, "partition kernels");
    }
    return CHICLE_OK;
}

chicle_status_t chicle_partition(chicle_glm_t *h, int32_t K, uint64_t seed)
{
    try { return partition_impl(h, K, seed, nullptr); } catch (...) { return CHICLE_ERR_OOM; }
}

chicle_status_t chicle_partition_sizes(chicle_glm_t *h, int32_t K, uint64_t seed, const int64_t *host_sizes)
{
    if (h && !host_sizes) return fail(h, CHICLE_ERR_INVALID_ARG, "chicle_partition_sizes: sizes is NULL");
    try { return partition_impl(h, K, seed, host_sizes); } catch (...) { return CHICLE_ERR_OOM; }
}

chicle_status_t chicle_partition_chunks(chicle_glm_t *h, int32_t K, uint64_t seed, int64_t n_chunks, const int64_t *host_chunk_off,
                                        const int32_t *host_chunk_task)
{
    if (!h) return CHICLE_ERR_INVALID_ARG;
    const ChunkPlacement cp{n_chunks, host_chunk_off, host_chunk_task};
    try { return partition_impl(h, K, seed, nullptr, &cp); } catch (...) { return CHICLE_ERR_OOM; }
}

// One round. host_steps == nullptr: every partition takes H steps (0: one local epoch). Otherwise partition k takes
// host_steps[k] steps (H is 0 then).
// delta_out != nullptr: the summed update goes there (device, dim floats) and v stays as it is.
static chicle_status_t round_impl(chicle_glm_t *h, int64_t H, const int64_t *host_steps, float sigma_prime, chicle_round_stats_t *stats,
                                  float *delta_out = nullptr)
{
    chicle_round_stats_t log_stats;
    const bool logging = log_level() >= 1;
    if (logging && !stats) stats = &log_stats;
    if (h->K <= 0) return fail(h, CHICLE_ERR_BAD_STATE, "chicle_partition must be called before chicle_cocoa_round");
    if (H < 0) return fail(h, CHICLE_ERR_INVALID_ARG, "H must be >= 0");
    if (!(sigma_prime > 0.0f) || !(sigma_prime < 3.0e38f)) return fail(h, CHICLE_ERR_INVALID_ARG, "sigma_prime must be positive and finite");
    int64_t budget_total = 0;
    if (host_steps) {
        for (int32_t k = 0; k < h->K; ++k) {
            if (host_steps[k] < 0 || host_steps[k] > h->h_part_off[k + 1] - h->h_part_off[k])
                return fail(h, CHICLE_ERR_INVALID_ARG, "a partition's step budget must lie between 0 and its size");
            budget_total += host_steps[k];
        }
    }
    cudaError_t e = cudaSetDevice(h->device);
    if (e != cudaSuccess) return fail_cuda(h, e, "cudaSetDevice");
    const int64_t n = h->n_coord, min_nk = h->min_nk;
    const int64_t epochs = H == 0 ? 1 : (H + min_nk - 1) / min_nk;
    if (epochs > h->perm_epochs) {
        if (epochs > 1024 || (double)epochs * (double)n * 4.0 > 64e9)
            return fail(h, CHICLE_ERR_UNSUPPORTED, "H spans too many local epochs for one round");
        e = cudaStreamSynchronize(h->stream);
        if (e != cudaSuccess) return fail_cuda(h, e, "stream synchronise");
        int32_t *np = nullptr;
        if (!alloc_into(h, np, (size_t)epochs * (size_t)n)) return fail(h, CHICLE_ERR_OOM, "device allocation failed (visiting orders)");
        dev_free(h, h->perm);
        h->perm = np;
        h->perm_epochs = epochs;
    }
    cudaStream_t s = h->stream;
    if (stats) (void)cudaEventRecord(h->ev[0], s);
    e = launch_permutation(*h, h->round, epochs);
    if (e != cudaSuccess) return fail_cuda(h, e, "visiting-order kernels");
    if (stats) (void)cudaEventRecord(h->ev[1], s);
    int variant = 0;
    h->time_prepare = stats != nullptr;
    h->solver_launches = 0;
    if (host_steps) {
        // a pageable source: the runtime has taken its copy of the K words when the call returns
        e = cudaMemcpyAsync(h->d_steps, host_steps, (size_t)h->K * sizeof(int64_t), cudaMemcpyHostToDevice, s);
        if (e != cudaSuccess) return fail_cuda(h, e, "step budgets to the device");
        h->round_steps = host_steps;
    }
    if (!host_steps || budget_total > 0) e = launch_local_solver(*h, H, sigma_prime, &variant);
    else if (stats) (void)cudaEventRecord(h->ev[4], s); // nobody steps this round
    h->round_steps = nullptr;
    if (e != cudaSuccess) return fail_cuda(h, e, "local solver launch");
    if (stats) (void)cudaEventRecord(h->ev[2], s);
    e = delta_out ? launch_sum_updates(*h, delta_out) : launch_reduce(*h);
    if (e != cudaSuccess) return fail_cuda(h, e, "aggregation launch");
    if (stats) (void)cudaEventRecord(h->ev[3], s);
    h->round += 1;
    if (stats) {
        const chicle_status_t st = check_status(h); // synchronises
        if (st != CHICLE_OK) return st;
        chicle_round_stats_t r;
        std::memset(&r, 0, sizeof(r));
        (void)cudaEventElapsedTime(&r.ms_permutation, h->ev[0], h->ev[1]);
        (void)cudaEventElapsedTime(&r.ms_local, h->ev[1], h->ev[2]);
        (void)cudaEventElapsedTime(&r.ms_reduce, h->ev[2], h->ev[3]);
        (void)cudaEventElapsedTime(&r.ms_total, h->ev[0], h->ev[3]);
        int64_t steps = 0;
        for (int32_t k = 0; k < h->K; ++k) {
            const int64_t nk = h->h_part_off[k + 1] - h->h_part_off[k];
            steps += host_steps ? host_steps[k] : (nk <= 0 ? 0 : (H == 0 ? nk : H));
        }
        r.steps = steps;
        r.solver_variant = variant;
        if (variant >= 4) (void)cudaEventElapsedTime(&r.ms_prepare, h->ev[1], h->ev[4]);
        r.solver_slices = variant >= 4 ? h->la_last_slices : 0;
        r.cluster_ctas = variant == 4 ? (1 << h->la_logC) : 1;
        r.solver_launches = steps > 0 ? (h->solver_launches > 0 ? h->solver_launches : 1) : 0;
        r.order_launches = (int32_t)(epochs * (22 + 5 * (h->K <= 256 ? 1 : 2)));
        *stats = r;
        if (logging)
            fprintf(stderr, "[chicle] round %lld: K=%d steps=%lld solver=%d slices=%d ctas/partition=%d launches=%d; ms: orders %.3f, "
                    "local solvers %.3f (first prepare %.3f), aggregation %.3f\n", (long long)(h->round - 1), (int)h->K,
                    (long long)r.steps, (int)r.solver_variant, (int)r.solver_slices, (int)r.cluster_ctas,
                    (int)(r.solver_launches + r.order_launches + 1), r.ms_permutation, r.ms_local, r.ms_prepare, r.ms_reduce);
    }
    return CHICLE_OK;
}

chicle_status_t chicle_cocoa_round(chicle_glm_t *h, int64_t H, float sigma_prime, chicle_round_stats_t *stats)
{
    if (!h) return CHICLE_ERR_INVALID_ARG;
    try { return round_impl(h, H, nullptr, sigma_prime, stats); } catch (...) { return CHICLE_ERR_OOM; }
}

chicle_status_t chicle_cocoa_round_steps(chicle_glm_t *h, const int64_t *host_steps, float sigma_prime, chicle_round_stats_t *stats)
{
    if (!h) return CHICLE_ERR_INVALID_ARG;
    if (!host_steps) return fail(h, CHICLE_ERR_INVALID_ARG, "chicle_cocoa_round_steps: steps is NULL");
    try { return round_impl(h, 0, host_steps, sigma_prime, stats); } catch (...) { return CHICLE_ERR_OOM; }
}

chicle_status_t chicle_cocoa_round_delta(chicle_glm_t *h, const int64_t *host_steps, float sigma_prime, float *dev_delta, int64_t len,
                                         chicle_round_stats_t *stats)
{
    if (!h) return CHICLE_ERR_INVALID_ARG;
    if (!host_steps || !dev_delta || len != h->dim)
        return fail(h, CHICLE_ERR_INVALID_ARG, "chicle_cocoa_round_delta: steps or delta is NULL, or len is not the shared vector's length");
    try { return round_impl(h, 0, host_steps, sigma_prime, stats, dev_delta); } catch (...) { return CHICLE_ERR_OOM; }
}

chicle_status_t chicle_apply_deltas(chicle_glm_t *h, const float *dev_deltas, int32_t count, int64_t len)
{
    if (!h) return CHICLE_ERR_INVALID_ARG;
    if (!dev_deltas || count < 1 || len != h->dim)
        return fail(h, CHICLE_ERR_INVALID_ARG, "chicle_apply_deltas: deltas is NULL, count < 1, or len is not the shared vector's length");
    cudaError_t e = cudaSetDevice(h->device);
    if (e == cudaSuccess) e = launch_apply_deltas(*h, dev_deltas, count);
    if (e != cudaSuccess) return fail_cuda(h, e, "chicle_apply_deltas");
    return CHICLE_OK;
}

chicle_status_t chicle_export_state_of(chicle_glm_t *h, const uint8_t *host_keep, float *dev_out, int64_t len)
{
    if (!h) return CHICLE_ERR_INVALID_ARG;
    if (h->K <= 0) return fail(h, CHICLE_ERR_BAD_STATE, "chicle_export_state_of needs a partition");
    if (!host_keep || !dev_out || len != h->n_coord)
        return fail(h, CHICLE_ERR_INVALID_ARG, "chicle_export_state_of: keep or out is NULL, or len is not the number of coordinates");
    cudaError_t e = cudaSetDevice(h->device);
    // (the K words of the step budgets are free between rounds: the K bytes travel through them)
    unsigned char *d_keep = reinterpret_cast<unsigned char *>(h->d_steps);
    if (e == cudaSuccess) e = cudaMemcpyAsync(d_keep, host_keep, (size_t)h->K, cudaMemcpyHostToDevice, h->stream);
    if (e == cudaSuccess) e = launch_mask_state(*h, d_keep, dev_out);
    if (e != cudaSuccess) return fail_cuda(h, e, "chicle_export_state_of");
    return CHICLE_OK;
}

chicle_status_t chicle_import_state(chicle_glm_t *h, const float *dev_state, int64_t len)
{
    if (!h) return CHICLE_ERR_INVALID_ARG;
    if (!dev_state || len != h->n_coord)
        return fail(h, CHICLE_ERR_INVALID_ARG, "chicle_import_state: state is NULL or len is not the number of coordinates");
    cudaError_t e = cudaSetDevice(h->device);
    if (e == cudaSuccess) e = cudaMemcpyAsync(h->alpha, dev_state, (size_t)len * 4, cudaMemcpyDeviceToDevice, h->stream);
    if (e != cudaSuccess) return fail_cuda(h, e, "chicle_import_state");
    return CHICLE_OK;
}

chicle_status_t chicle_duality_gap(chicle_glm_t *h, double *host_gap, double *host_primal, double *host_dual)
{
    if (!h) return CHICLE_ERR_INVALID_ARG;
    cudaError_t e = cudaSetDevice(h->device);
    if (e == cudaSuccess) e = launch_gap(*h);
    if (e == cudaSuccess) e = cudaMemcpyAsync(h->h_gap, h->gap_out, 3 * sizeof(double), cudaMemcpyDeviceToHost, h->stream);
    if (e != cudaSuccess) return fail_cuda(h, e, "duality-gap kernels");
    const chicle_status_t st = check_status(h); // synchronises
    if (st != CHICLE_OK) return st;
    if (host_gap) *host_gap = h->h_gap[0];
    if (host_primal) *host_primal = h->h_gap[1];
    if (host_dual) *host_dual = h->h_gap[2];
    return CHICLE_OK;
}

static chicle_status_t copy_out(chicle_glm_t *h, const float *src, int64_t have, float *out, int64_t len,
                                chicle_memspace_t space, const char *what)
{
    if (!h) return CHICLE_ERR_INVALID_ARG;
    if (!out || len != have || ((int)space != 0 && (int)space != 1))
        return fail(h, CHICLE_ERR_INVALID_ARG, std::string(what) + ": out is NULL, len is wrong or space is unknown");
    cudaError_t e = cudaSetDevice(h->device);
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(out, src, (size_t)len * 4, space == CHICLE_MEM_HOST ? cudaMemcpyDeviceToHost : cudaMemcpyDeviceToDevice,
                            h->stream);
    if (e != cudaSuccess) return fail_cuda(h, e, what);
    return check_status(h);
}

chicle_status_t chicle_get_alpha(chicle_glm_t *h, float *out, int64_t len, chicle_memspace_t space)
{
    return copy_out(h, h ? h->alpha : nullptr, h ? h->n_coord : 0, out, len, space, "chicle_get_alpha");
}

chicle_status_t chicle_get_v(chicle_glm_t *h, float *out, int64_t len, chicle_memspace_t space)
{
    if (h && h->new_of_old) {
        // translate from the library's ranked ids to the caller's: tmp[old] = v[new_of_old[old]]
        if (cudaSetDevice(h->device) == cudaSuccess) {
            const cudaError_t e = launch_gather_f32(*h, h->v, h->new_of_old, h->dim, h->perm_tmp);
            if (e != cudaSuccess) return fail_cuda(h, e, "chicle_get_v");
        }
        return copy_out(h, h->perm_tmp, h->dim, out, len, space, "chicle_get_v");
    }
    return copy_out(h, h ? h->v : nullptr, h ? h->dim : 0, out, len, space, "chicle_get_v");
}

chicle_status_t chicle_get_partition(chicle_glm_t *h, int32_t *host_owner, int64_t len)
{
    if (!h) return CHICLE_ERR_INVALID_ARG;
    if (h->K <= 0) return fail(h, CHICLE_ERR_BAD_STATE, "no partition yet");
    if (!host_owner || len != h->n_coord) return fail(h, CHICLE_ERR_INVALID_ARG, "chicle_get_partition: bad out or len");
    cudaError_t e = cudaSetDevice(h->device);
    if (e == cudaSuccess) e = cudaMemcpyAsync(host_owner, h->owner, (size_t)len * 4, cudaMemcpyDeviceToHost, h->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(h->stream);
    if (e != cudaSuccess) return fail_cuda(h, e, "chicle_get_partition");
    return CHICLE_OK;
}

chicle_status_t chicle_get_permutation(chicle_glm_t *h, int64_t round, int32_t k, int32_t *host_out, int64_t len)
{
    if (!h) return CHICLE_ERR_INVALID_ARG;
    if (h->K <= 0) return fail(h, CHICLE_ERR_BAD_STATE, "no partition yet");
    if (round < 0 || k < 0 || k >= h->K) return fail(h, CHICLE_ERR_INVALID_ARG, "round or partition index out of range");
    const int64_t nk = h->h_part_off[k + 1] - h->h_part_off[k];
    if (!host_out || len != nk) return fail(h, CHICLE_ERR_INVALID_ARG, "chicle_get_permutation: bad out or len");
    cudaError_t e = cudaSetDevice(h->device);
    if (e == cudaSuccess) e = launch_permutation(*h, round, 1); // scratch use of the order buffer: rounds rebuild it
    if (e == cudaSuccess && nk > 0)
        e = cudaMemcpyAsync(host_out, h->perm + h->h_part_off[k], (size_t)nk * 4, cudaMemcpyDeviceToHost, h->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(h->stream);
    if (e != cudaSuccess) return fail_cuda(h, e, "chicle_get_permutation");
    return CHICLE_OK;
}

chicle_status_t chicle_set_state(chicle_glm_t *h, const float *host_alpha, const float *host_v, int64_t round)
{
    if (!h) return CHICLE_ERR_INVALID_ARG;
    if (!host_alpha || round < 0) return fail(h, CHICLE_ERR_INVALID_ARG, "chicle_set_state: alpha is NULL or round < 0");
    cudaError_t e = cudaSetDevice(h->device);
    if (e == cudaSuccess) e = cudaMemcpyAsync(h->alpha, host_alpha, (size_t)h->n_coord * 4, cudaMemcpyHostToDevice, h->stream);
    if (e == cudaSuccess) {
        if (host_v) {
            if (h->new_of_old) {
                // the caller's ids -> ranked ids: v[new] = host_v[old_of_new[new]]
                e = cudaMemcpyAsync(h->perm_tmp, host_v, (size_t)h->dim * 4, cudaMemcpyHostToDevice, h->stream);
                if (e == cudaSuccess) e = launch_gather_f32(*h, h->perm_tmp, h->old_of_new, h->dim, h->v);
            } else {
                e = cudaMemcpyAsync(h->v, host_v, (size_t)h->dim * 4, cudaMemcpyHostToDevice, h->stream);
            }
            if (e == cudaSuccess) e = launch_refresh_resid(*h);
        } else {
            e = launch_shared_vector(*h);
        }
    }
    if (e == cudaSuccess) e = cudaStreamSynchronize(h->stream);
    if (e != cudaSuccess) return fail_cuda(h, e, "chicle_set_state");
    h->round = round;
    return CHICLE_OK;
}

chicle_status_t chicle_get_info(const chicle_glm_t *h, int64_t *round, int32_t *K, int64_t *n_coord, int64_t *dim)
{
    if (!h) return CHICLE_ERR_INVALID_ARG;
    if (round) *round = h->round;
    if (K) *K = h->K;
    if (n_coord) *n_coord = h->n_coord;
    if (dim) *dim = h->dim;
    return CHICLE_OK;
}

const char *chicle_last_error(const chicle_glm_t *h) { return h ? h->err.c_str() : g_create_error.c_str(); }

void chicle_glm_destroy(chicle_glm_t *h) { destroy_impl(h); }

} // extern "C"
