// Streaming kernels: input validation, squared norms, aggregation of the K partition updates into the shared
// vector (Eq. 2 with the updates added), the duality gap (the paper's convergence metric), and the from-scratch
// shared vector used when a state is restored.
#include <math_constants.h>

#include <cstdlib>
#include <cstring>

#include "solver_common.cuh"

namespace chicle {

namespace {

constexpr int kThreads = 256;
constexpr int kWarpsPerBlock = kThreads / 32;

inline unsigned blocks_for(int64_t n, int t) { return (unsigned)((n + t - 1) / t); }

__device__ __forceinline__ double warp_sum_d(double x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

// ---------------------------------------------------------------------------------------- validation
__global__ void k_validate_values(const float *__restrict__ x, int64_t n, uint32_t *status)
{
    bool bad = false;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        bad |= !(fabsf(x[i]) <= CUDART_MAX_NORMAL_F);
    if (__any_sync(0xffffffffu, bad) && (threadIdx.x & 31) == 0) atomicOr(status, ST_NONFINITE_INPUT);
}

__global__ void k_validate_labels(const float *__restrict__ y, int64_t n, int need_pm1, uint32_t *status)
{
    uint32_t bits = 0;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        const float t = y[i];
        if (!(fabsf(t) <= CUDART_MAX_NORMAL_F)) bits |= ST_NONFINITE_INPUT;
        else if (need_pm1 && t != 1.0f && t != -1.0f) bits |= ST_BAD_LABEL;
    }
    if (bits) atomicOr(status, bits);
}

__global__ void k_validate_structure(const int64_t *__restrict__ indptr, const int32_t *__restrict__ indices,
                                     int64_t n_coord, int64_t nnz, int64_t dim, uint32_t *status)
{
    bool bad = false;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (int64_t c = tid; c < n_coord; c += stride) bad |= indptr[c + 1] < indptr[c];
    if (tid == 0) bad |= indptr[0] != 0 || indptr[n_coord] != nnz;
    for (int64_t e = tid; e < nnz; e += stride) bad |= indices[e] < 0 || indices[e] >= dim;
    if (bad) atomicOr(status, ST_BAD_INDEX);
}

// ---------------------------------------------------------------------------------------- squared norms
__global__ void __launch_bounds__(kThreads)
k_sqnorm(const int64_t *__restrict__ indptr, const float *__restrict__ values, int64_t n_coord, int64_t dim,
         float *__restrict__ out)
{
    const int lane = threadIdx.x & 31;
    const int64_t nw = (int64_t)gridDim.x * kWarpsPerBlock;
    for (int64_t c = (int64_t)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5); c < n_coord; c += nw) {
        const int64_t b = indptr ? indptr[c] : c * dim;
        const int64_t e = indptr ? indptr[c + 1] : b + dim;
        double s = 0.0;
        for (int64_t q = b + lane; q < e; q += 32) {
            const double x = (double)values[q];
            s = fma(x, x, s);
        }
        s = warp_sum_d(s);
        if (lane == 0) out[c] = (float)s;
    }
}

// ---------------------------------------------------------------------------------------- aggregation (a5)
// v[j] += sum_k U[k][j] with k ascending and an fp64 accumulator; U is cleared for the next round; for ridge
// the residual v - y that the next round's solvers gather from is refreshed in the same pass.
template <int VEC>
__global__ void __launch_bounds__(kThreads)
k_reduce_updates(float *__restrict__ v, float *__restrict__ U, int K, int64_t dim, const float *__restrict__ y,
                 float *__restrict__ resid)
{
    const int64_t nvec = dim / VEC;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < nvec; i += (int64_t)gridDim.x * blockDim.x) {
        double acc[VEC];
        if (VEC == 4) {
            const float4 t = reinterpret_cast<const float4 *>(v)[i];
            acc[0] = t.x; acc[1 % VEC] = t.y; acc[2 % VEC] = t.z; acc[3 % VEC] = t.w;
        } else {
            acc[0] = v[i];
        }
#pragma unroll 16
        for (int k = 0; k < K; ++k) {
            if (VEC == 4) {
                float4 *p = reinterpret_cast<float4 *>(U + (size_t)k * dim) + i;
                const float4 t = *p;
                acc[0] += t.x; acc[1 % VEC] += t.y; acc[2 % VEC] += t.z; acc[3 % VEC] += t.w;
                *p = make_float4(0.f, 0.f, 0.f, 0.f);
            } else {
                float *p = U + (size_t)k * dim + i;
                acc[0] += *p;
                *p = 0.f;
            }
        }
        if (VEC == 4) {
            const float4 o = make_float4((float)acc[0], (float)acc[1 % VEC], (float)acc[2 % VEC], (float)acc[3 % VEC]);
            reinterpret_cast<float4 *>(v)[i] = o;
            if (resid) {
                const float4 t = reinterpret_cast<const float4 *>(y)[i];
                reinterpret_cast<float4 *>(resid)[i] = make_float4(o.x - t.x, o.y - t.y, o.z - t.z, o.w - t.w);
            }
        } else {
            const float o = (float)acc[0];
            v[i] = o;
            if (resid) resid[i] = o - y[i];
        }
    }
}

// The same aggregation with the sum kept apart from v: delta[j] = sum_k U[k][j] (k ascending, fp64 accumulator), U
// cleared, v untouched. What a rank of a job spread over several GPUs hands to the others (Sec. 4.2: the trainer merges
// the solvers' updates and broadcasts the model).
__global__ void __launch_bounds__(kThreads)
k_sum_updates(float *__restrict__ U, int K, int64_t dim, float *__restrict__ delta)
{
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < dim; i += (int64_t)gridDim.x * blockDim.x) {
        double acc = 0.0;
#pragma unroll 16
        for (int k = 0; k < K; ++k) {
            float *p = U + (size_t)k * dim + i;
            acc += *p;
            *p = 0.f;
        }
        delta[i] = (float)acc;
    }
}

// v[j] += sum_g D[g][j] (g ascending, fp64 accumulator): the merged update of `count` ranks, each rank's vector `dim`
// long and the vectors one behind the other; every rank adds them in the same order, so the replicas of v stay equal
// bit for bit. Ridge: the residual is refreshed in the same pass.
__global__ void __launch_bounds__(kThreads)
k_apply_deltas(float *__restrict__ v, const float *__restrict__ D, int count, int64_t dim, const float *__restrict__ y,
               float *__restrict__ resid)
{
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < dim; i += (int64_t)gridDim.x * blockDim.x) {
        double acc = v[i];
        for (int g = 0; g < count; ++g) acc += D[(size_t)g * dim + i];
        const float o = (float)acc;
        v[i] = o;
        if (resid) resid[i] = o - y[i];
    }
}

// out[i] = keep[owner[i]] ? state[i] : 0: the part of the per-coordinate state that the partitions marked in `keep`
// own (K bytes on the device).
__global__ void __launch_bounds__(kThreads)
k_mask_state(const float *__restrict__ state, const int32_t *__restrict__ owner, const unsigned char *__restrict__ keep,
             int64_t n, float *__restrict__ out)
{
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        out[i] = keep[owner[i]] ? state[i] : 0.0f;
}

__global__ void k_resid(const float *__restrict__ v, const float *__restrict__ y, int64_t n, float *__restrict__ r)
{
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        r[i] = v[i] - y[i];
}

// ---------------------------------------------------------------------------------------- duality gap (a6)
// One streaming pass over the coordinate-major matrix. Sparse: a warp takes four consecutive coordinates at a time
// and issues all their index/value loads (then all gathers from the shared vector) before reducing anything, so
// that enough bytes are in flight to cover the memory latency; dot products and sums are fp64. Short dense rows: a
// thread per row with 128-bit loads. Lanes keep running fp64 sums over the coordinates they were assigned (a fixed
// assignment), the block adds its lanes and warps in a fixed order and writes 4 partial sums; a second kernel adds
// the blocks in a fixed order. Partials: dual losses {sum loss, sum gap term, |v|^2 slice, 0};
// ridge {sum (c_j . r)^2, sum w_j^2, sum r^2 slice, sum r*y slice} with r = v - y.
__device__ __forceinline__ double xlogx(double x) { return x > 0.0 ? x * log(x) : 0.0; }

// adds coordinate c's contribution, given its dot product with the shared vector (with v - y for ridge)
template <int LOSS>
__device__ __forceinline__ void gap_term(double dot, float label, float state, double inv_lam_n, double &s0, double &s1)
{
    if (LOSS == CHICLE_LOSS_RIDGE_PRIMAL) {
        const double w = (double)state;
        s0 += dot * dot;
        s1 += w * w;
    } else {
        const double y = (double)label;
        const double mu = y * dot * inv_lam_n; // (a multiplication: the fp64 division was a third of the streamed kernel's instructions)
        double a = y * (double)state;
        a = a < 0.0 ? 0.0 : (a > 1.0 ? 1.0 : a);
        double l, conj;
        if (LOSS == CHICLE_LOSS_HINGE_DUAL) {
            l = 1.0 - mu > 0.0 ? 1.0 - mu : 0.0;
            conj = -a;
        } else {
            l = mu < 0.0 ? -mu + log1p(exp(mu)) : log1p(exp(-mu));
            conj = xlogx(a) + xlogx(1.0 - a);
        }
        s0 += l;
        s1 += l + conj + a * mu;
    }
}

#ifndef CHICLE_GAP_ROWS
#define CHICLE_GAP_ROWS 4
#endif
constexpr int kGapRows = CHICLE_GAP_ROWS;   // coordinates a warp has in flight
constexpr int kGapChunks = 2; // 32-entry chunks per coordinate held in registers (longer ones loop)

template <int LOSS>
__global__ void __launch_bounds__(kThreads)
k_gap_partials(const int64_t *__restrict__ indptr, const int32_t *__restrict__ indices,
               const float *__restrict__ values, const float *__restrict__ labels, const float *__restrict__ state,
               const float *__restrict__ vec /* the shared vector */, const float *__restrict__ v,
               int64_t n_coord, int64_t dim, double lam_n, double *__restrict__ partials, uint32_t *status)
{
    __shared__ double sh[kThreads][2];
    __shared__ double sh2[kWarpsPerBlock][2];
    const double inv_lam_n = 1.0 / lam_n;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t nw = (int64_t)gridDim.x * kWarpsPerBlock;
    const int64_t gw = (int64_t)blockIdx.x * kWarpsPerBlock + warp;
    double s0 = 0.0, s1 = 0.0;
    if (indptr) {
        const int64_t ngroups = (n_coord + kGapRows - 1) / kGapRows;
        // the row pointers and per-coordinate scalars of a group are fetched one iteration ahead
        auto fetch_ip = [&](int64_t g) -> int64_t {
            if (g >= ngroups || lane > kGapRows) return 0;
            const int64_t c = g * kGapRows + lane;
            return indptr[c < n_coord ? c : n_coord];
        };
        auto fetch_scalars = [&](int64_t g, float &lab, float &sta) {
            lab = 0.0f;
            sta = 0.0f;
            const int64_t c = g * kGapRows + lane;
            if (g < ngroups && lane < kGapRows && c < n_coord) {
                sta = state[c];
                if (LOSS != CHICLE_LOSS_RIDGE_PRIMAL) lab = labels[c];
            }
        };
        int64_t ip_next = fetch_ip(gw);
        float lab_next, sta_next;
        fetch_scalars(gw, lab_next, sta_next);
        for (int64_t g = gw; g < ngroups; g += nw) {
            const int64_t c0 = g * kGapRows;
            const int64_t ip = ip_next;
            const float my_label = lab_next, my_state = sta_next;
            ip_next = fetch_ip(g + nw);
            fetch_scalars(g + nw, lab_next, sta_next);
            const bool owner = lane < kGapRows && c0 + lane < n_coord;
            int64_t rs[kGapRows], re[kGapRows];
#pragma unroll
            for (int r = 0; r < kGapRows; ++r) {
                rs[r] = __shfl_sync(0xffffffffu, ip, r);
                re[r] = __shfl_sync(0xffffffffu, ip, r + 1);
            }
            int32_t ix[kGapRows][kGapChunks];
            float xv[kGapRows][kGapChunks];
#pragma unroll
            for (int r = 0; r < kGapRows; ++r)
#pragma unroll
                for (int ch = 0; ch < kGapChunks; ++ch) {
                    const int64_t e = rs[r] + lane + 32 * ch;
                    ix[r][ch] = -1;
                    xv[r][ch] = 0.0f;
                    if (e < re[r]) {
                        ix[r][ch] = indices[e];
                        xv[r][ch] = values[e];
                        if (!CHICLE_IN_BOUNDS(status, ix[r][ch] >= 0 && (int64_t)ix[r][ch] < dim)) ix[r][ch] = -1;
                    }
                }
            double dot[kGapRows];
#pragma unroll
            for (int r = 0; r < kGapRows; ++r) {
                dot[r] = 0.0;
#pragma unroll
                for (int ch = 0; ch < kGapChunks; ++ch)
                    if (ix[r][ch] >= 0) {
                        double t = (double)vec[ix[r][ch]];
                        if (LOSS == CHICLE_LOSS_RIDGE_PRIMAL) t -= (double)labels[ix[r][ch]];
                        dot[r] = fma((double)xv[r][ch], t, dot[r]);
                    }
                for (int64_t e = rs[r] + 32 * kGapChunks + lane; e < re[r]; e += 32) { // the rest of a long coordinate
                    const int32_t i = indices[e];
                    if (!CHICLE_IN_BOUNDS(status, i >= 0 && (int64_t)i < dim)) continue;
                    double t = (double)vec[i];
                    if (LOSS == CHICLE_LOSS_RIDGE_PRIMAL) t -= (double)labels[i];
                    dot[r] = fma((double)values[e], t, dot[r]);
                }
            }
            double mine = 0.0;
#pragma unroll
            for (int r = 0; r < kGapRows; ++r) {
                const double d = warp_sum_d(dot[r]);
                if (lane == r) mine = d;
            }
            if (owner) gap_term<LOSS>(mine, my_label, my_state, inv_lam_n, s0, s1);
        }
    } else if (dim <= 64 && (dim & 3) == 0) {
        // short dense rows: a thread per row, 128-bit loads; a warp's 32 rows are contiguous in memory
        const int64_t stride = (int64_t)gridDim.x * kThreads;
        for (int64_t c = (int64_t)blockIdx.x * kThreads + threadIdx.x; c < n_coord; c += stride) {
            const float4 *row = reinterpret_cast<const float4 *>(values + c * dim);
            double dot = 0.0;
            for (int j4 = 0; j4 < (int)(dim >> 2); ++j4) {
                const float4 x = row[j4];
                dot = fma((double)x.x, (double)vec[4 * j4], dot);
                dot = fma((double)x.y, (double)vec[4 * j4 + 1], dot);
                dot = fma((double)x.z, (double)vec[4 * j4 + 2], dot);
                dot = fma((double)x.w, (double)vec[4 * j4 + 3], dot);
            }
            gap_term<LOSS>(dot, labels[c], state[c], inv_lam_n, s0, s1);
        }
    } else {
        for (int64_t c = gw; c < n_coord; c += nw) {
            const float *row = values + c * dim;
            double dot = 0.0;
            for (int64_t j = lane; j < dim; j += 32) dot = fma((double)row[j], (double)vec[j], dot);
            dot = warp_sum_d(dot);
            if (lane == 0) gap_term<LOSS>(dot, labels[c], state[c], inv_lam_n, s0, s1);
        }
    }
    // slice of the shared vector owned by this block
    double s2 = 0.0, s3 = 0.0;
    {
        const int64_t chunk = (dim + gridDim.x - 1) / gridDim.x;
        const int64_t b = (int64_t)blockIdx.x * chunk;
        const int64_t e = b + chunk < dim ? b + chunk : dim;
        for (int64_t j = b + threadIdx.x; j < e; j += kThreads) {
            if (LOSS == CHICLE_LOSS_RIDGE_PRIMAL) {
                const double y = (double)labels[j]; // targets
                const double r = (double)v[j] - y;
                s2 = fma(r, r, s2);
                s3 = fma(r, y, s3);
            } else {
                const double t = (double)v[j];
                s2 = fma(t, t, s2);
            }
        }
        s2 = warp_sum_d(s2);
        s3 = warp_sum_d(s3);
    }
    // fixed-order combination: threads in index order for the per-coordinate sums, warps in order for the slices
    sh[threadIdx.x][0] = s0;
    sh[threadIdx.x][1] = s1;
    if (lane == 0) {
        sh2[warp][0] = s2;
        sh2[warp][1] = s3;
    }
    __syncthreads();
    if (threadIdx.x < 2) {
        // pairwise tree over the 256 threads, fixed shape
        double t[kThreads / 32];
        for (int w = 0; w < kThreads / 32; ++w) {
            double a = 0.0;
            for (int l = 0; l < 32; ++l) a += sh[w * 32 + l][threadIdx.x];
            t[w] = a;
        }
        double tot = 0.0;
        for (int w = 0; w < kThreads / 32; ++w) tot += t[w];
        partials[(size_t)blockIdx.x * 4 + threadIdx.x] = tot;
    } else if (threadIdx.x < 4) {
        double tot = 0.0;
        for (int w = 0; w < kWarpsPerBlock; ++w) tot += sh2[w][threadIdx.x - 2];
        partials[(size_t)blockIdx.x * 4 + threadIdx.x] = tot;
    }
}

// Sparse formats, streamed: the coordinates of a block's tile lie one after the other in memory, so their indices and
// values are two contiguous ranges, which a producer warp brings into a shared-memory ring of two or three stages with bulk
// copies (16-byte aligned windows; the bytes in flight no longer depend on registers or on how many warps fit). The
// sixteen consumer warps take R coordinates per tile, 512 / R threads each (every thread a fixed subset of the
// coordinate's entries, all gathers from the shared vector issued before the first use), and add the partial dot
// products in a fixed order. A tile whose non-zeros do not fit a stage is read from global memory by the same threads.
// Gathers from the shared vector are what the warp-per-coordinate kernel is bound by on skewed data (a 32-byte sector
// of L2 traffic per 4-byte gather: 7 TB/s at config 2), so each block also keeps the first kGapHot entries of the
// vector in its shared memory (ids are frequency-ranked: they take most of the gathers); the kernel is used when the
// ids are skewed, one block per SM. Every wait is bounded; when one runs out the status word says so and all roles
// leave.
// Two shapes of the shared memory: 32 768 staged entries of the shared vector (128 KB) with stages of 3 584 non-zeros,
// or 22 528 entries (88 KB) with stages of 5 248: the larger stages hold tiles of 128 short coordinates, which halves
// the per-tile work (waits, extents, the fp64 gap terms) per non-zero.
constexpr int kGapHot = 32768, kGapCapNz = 3584;
constexpr int kGapHotWide = 22528, kGapCapNzWide = 5248;
// ... or 14 336 entries (56 KB) with stages of 6 912, for tiles of 128 coordinates of about 50 entries: 0.149 against
// 0.161 ms per call at 1 M coordinates, although fewer gathers find their entry staged. (A two-stage ring with a larger
// head was slower: 0.184 ms.)
constexpr int kGapHotWider = 14336, kGapCapNzWider = 6912;
constexpr int kGapConsumers = 512;

// Bounded wait without back-off (try_wait itself parks the thread for a while): every lane calls it, lane 0 polls.
__device__ __forceinline__ bool gap_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, uint32_t *status)
{
    int ok = 1;
    if ((threadIdx.x & 31) == 0) {
        ok = 0;
        for (uint32_t it = 0; it < kSpinLimit; ++it) {
            if (mbar_try_wait(bar, parity)) { ok = 1; break; }
            if ((it & 255u) == 255u && *abort_flag) break;
        }
        if (!ok && !*abort_flag) {
            *abort_flag = 1;
            atomicOr(status, ST_WAIT_TIMEOUT);
        }
    }
    return __shfl_sync(0xffffffffu, ok, 0) != 0;
}

__device__ __forceinline__ float gap_ldg_if(const float *p, bool on)
{
    float v;
    asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.u32 q, %2, 0;\n\tmov.f32 %0, 0f00000000;\n\t@q ld.global.nc.f32 %0, [%1];\n\t}"
                 : "=f"(v) : "l"(p), "r"((uint32_t)on));
    return v;
}

template <int HOT, int CAP, int STAGES> struct GapShared {
    static constexpr int kStageElems = CAP + 8; // + the window's alignment slack
    alignas(16) float vhot[HOT];           // the head of the shared vector (ridge: of v - y)
    alignas(16) int32_t idx[STAGES][kStageElems];
    alignas(16) float val[STAGES][kStageElems];
    alignas(8) uint64_t full[STAGES];  // the stage's copies have landed (or the tile was marked as not staged)
    alignas(8) uint64_t empty[STAGES]; // the consumer warps have finished with the stage
    long long base[STAGES];            // first element of the stage's window in the global arrays; -1: not staged
    double sh[kGapConsumers][2];
    double sh2[kGapConsumers / 32][2];
    int abort_flag;
};

template <int LOSS, int R, int PER, int HOT, int CAP, int STAGES>
__global__ void __launch_bounds__(kGapConsumers + 32, 1)
k_gap_stream(const int64_t *__restrict__ indptr, const int32_t *__restrict__ indices, const float *__restrict__ values,
             const float *__restrict__ labels, const float *__restrict__ state, const float *__restrict__ vec,
             const float *__restrict__ gvec /* what the dot products gather from: v, or for ridge the residual v - y */,
             int64_t n_coord, int64_t dim, double lam_n, double *__restrict__ partials, uint32_t *status)
{
    constexpr int TPR = kGapConsumers / R; // threads per coordinate
    constexpr int kMaxPer = PER;           // entries a thread keeps in flight (6 or 8: the fewer idle slots, the fewer instructions)
    extern __shared__ __align__(128) unsigned char gap_smem[];
    using Shared = GapShared<HOT, CAP, STAGES>;
    constexpr int kGapStages = STAGES;
    Shared &sm = *reinterpret_cast<Shared *>(gap_smem);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const double inv_lam_n = 1.0 / lam_n;
    volatile int *abort_flag = &sm.abort_flag;
    if (tid == 0) {
        sm.abort_flag = 0;
        for (int s2 = 0; s2 < kGapStages; ++s2) {
            mbar_init(smem_u32(&sm.full[s2]), 1);
            mbar_init(smem_u32(&sm.empty[s2]), kGapConsumers / 32);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    const int hot_n = (int)(dim < HOT ? dim : HOT);
    for (int i = tid; i < hot_n; i += kGapConsumers + 32)
        sm.vhot[i] = gvec[i];
    __syncthreads();
    const int64_t ntiles = (n_coord + R - 1) / R;
    const int64_t first = blockIdx.x, step = gridDim.x;
    double s0 = 0.0, s1 = 0.0;
    if (warp == kGapConsumers / 32) {
        // ------------------------------------------------ producer (the next tile's extent is fetched a tile ahead)
        int64_t k = 0;
        auto bounds = [&](int64_t t, int64_t &rs, int64_t &re) {
            rs = re = 0;
            if (t < ntiles && lane == 0) {
                const int64_t c0 = t * R, c1 = (c0 + R < n_coord) ? c0 + R : n_coord;
                rs = indptr[c0];
                re = indptr[c1];
            }
        };
        int64_t rs_n, re_n;
        bounds(first, rs_n, re_n);
        for (int64_t t = first; t < ntiles; t += step, ++k) {
            const int st = (int)(k % kGapStages);
            const int64_t rs = rs_n, re = re_n;
            bounds(t + step, rs_n, re_n);
            if (k >= kGapStages) {
                if (!gap_wait(smem_u32(&sm.empty[st]), (uint32_t)((k / kGapStages) - 1) & 1u, abort_flag, status)) break;
            }
            if (lane == 0) {
                const int64_t w0 = rs & ~(int64_t)3;
                const int64_t elems = ((re - w0) + 3) & ~(int64_t)3;
                const uint32_t bar = smem_u32(&sm.full[st]);
                // the stage was read by ordinary loads: order them before the copy engine's writes
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                if (elems > 0 && elems <= Shared::kStageElems) {
                    sm.base[st] = w0;
                    const uint32_t bytes = (uint32_t)elems * 4u;
                    mbar_arrive_expect_tx(bar, 2u * bytes);
                    bulk_g2s(smem_u32(&sm.idx[st][0]), indices + w0, bytes, bar);
                    bulk_g2s(smem_u32(&sm.val[st][0]), values + w0, bytes, bar);
                } else {
                    sm.base[st] = -1; // empty tile, or too many non-zeros for a stage: the consumers read global memory
                    __threadfence_block();
                    mbar_arrive(bar);
                }
            }
            __syncwarp();
        }
    } else {
        // ------------------------------------------------ consumers
        const int r = tid / TPR, sub = tid % TPR;
        int64_t k = 0;
        // the extent and the scalars of this thread's coordinate in the next tile are fetched a tile ahead
        auto fetch = [&](int64_t t, int64_t &rs, int64_t &re, float &lab, float &sta) {
            rs = re = 0;
            lab = sta = 0.0f;
            const int64_t c = t * R + r;
            if (t < ntiles && c < n_coord) {
                rs = indptr[c];
                re = indptr[c + 1];
                sta = state[c];
                if (LOSS != CHICLE_LOSS_RIDGE_PRIMAL) lab = labels[c];
            }
        };
        int64_t rs_n, re_n;
        float lab_n, sta_n;
        fetch(first, rs_n, re_n, lab_n, sta_n);
        for (int64_t t = first; t < ntiles; t += step, ++k) {
            const int st = (int)(k % kGapStages);
            const int64_t rs = rs_n, re = re_n;
            const float lab = lab_n, sta = sta_n;
            const bool owner = sub == 0 && t * R + r < n_coord;
            fetch(t + step, rs_n, re_n, lab_n, sta_n);
            if (!gap_wait(smem_u32(&sm.full[st]), (uint32_t)(k / kGapStages) & 1u, abort_flag, status)) break;
            const int64_t base = sm.base[st];
            // A coordinate's dot product is taken in fp32 (as the solvers take it), every thread its own entries in a
            // fixed order, and enters the fp64 sums over the coordinates once: a conversion and an fp64 multiply-add
            // per non-zero were what the kernel was bound by (instruction issue), not the memory traffic.
            float dot = 0.0f;
            if (base >= 0) {
                // staged: 32-bit offsets into the stage, every load unconditional (clamped) and the gathers beyond the
                // staged head of the vector predicated, so that nothing branches per non-zero
                const int hi = (int)(re - base);
                const uint32_t a_idx = smem_u32(&sm.idx[st][0]), a_val = smem_u32(&sm.val[st][0]);
                for (int e0 = (int)(rs - base) + sub; e0 < hi; e0 += TPR * kMaxPer) {
                    int32_t ii[kMaxPer];
                    float xx[kMaxPer], tt[kMaxPer], hh[kMaxPer];
#pragma unroll
                    for (int q = 0; q < kMaxPer; ++q) {
                        const int e = e0 + q * TPR;
                        const bool valid = e < hi;
                        const uint32_t o = 4u * (uint32_t)(valid ? e : 0);
                        ii[q] = lds_s32(a_idx + o); // (a slot beyond the coordinate's end reads the stage's first entry with x = 0)
                        const float x = lds_f32(a_val + o);
                        xx[q] = valid ? x : 0.0f;
                    }
#pragma unroll
                    for (int q = 0; q < kMaxPer; ++q) {
                        if (!CHICLE_IN_BOUNDS(status, ii[q] >= 0 && (int64_t)ii[q] < dim)) ii[q] = 0;
                        const bool far = ii[q] >= hot_n;
                        hh[q] = sm.vhot[far ? 0 : ii[q]];
                        tt[q] = gap_ldg_if(gvec + (far ? ii[q] : 0), far);
                    }
#pragma unroll
                    for (int q = 0; q < kMaxPer; ++q) {
                        // (x is 0 beyond the coordinate's end)
                        dot = fmaf(xx[q], ii[q] >= hot_n ? tt[q] : hh[q], dot);
                    }
                }
            } else {
                for (int64_t e = rs + sub; e < re; e += TPR) {
                    int32_t i = indices[e];
                    if (!CHICLE_IN_BOUNDS(status, i >= 0 && (int64_t)i < dim)) i = 0;
                    float t;
                    if (i < hot_n) t = sm.vhot[i];
                    else t = gvec[i];
                    dot = fmaf(values[e], t, dot);
                }
            }
            // the stage is free once every lane of the warp has read its entries
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sm.empty[st]));
#pragma unroll
            for (int o = 1; o < TPR; o <<= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
            if (owner) gap_term<LOSS>((double)dot, lab, sta, inv_lam_n, s0, s1);
        }
    }
    // slice of the shared vector owned by this block (consumer threads)
    double s2 = 0.0, s3 = 0.0;
    if (tid < kGapConsumers) {
        const int64_t chunk = (dim + gridDim.x - 1) / gridDim.x;
        const int64_t b = (int64_t)blockIdx.x * chunk;
        const int64_t e = b + chunk < dim ? b + chunk : dim;
        for (int64_t j = b + tid; j < e; j += kGapConsumers) {
            if (LOSS == CHICLE_LOSS_RIDGE_PRIMAL) {
                const double y = (double)labels[j]; // targets
                const double rr = (double)vec[j] - y;
                s2 = fma(rr, rr, s2);
                s3 = fma(rr, y, s3);
            } else {
                const double t = (double)vec[j];
                s2 = fma(t, t, s2);
            }
        }
        s2 = warp_sum_d(s2);
        s3 = warp_sum_d(s3);
        sm.sh[tid][0] = s0;
        sm.sh[tid][1] = s1;
        if (lane == 0) {
            sm.sh2[warp][0] = s2;
            sm.sh2[warp][1] = s3;
        }
    }
    __syncthreads();
    // fixed-order combination: threads in index order for the per-coordinate sums, warps in order for the slices
    if (tid < 2) {
        double tot = 0.0;
        for (int w = 0; w < kGapConsumers / 32; ++w) {
            double a = 0.0;
            for (int l = 0; l < 32; ++l) a += sm.sh[w * 32 + l][tid];
            tot += a;
        }
        partials[(size_t)blockIdx.x * 4 + tid] = tot;
    } else if (tid < 4) {
        double tot = 0.0;
        for (int w = 0; w < kGapConsumers / 32; ++w) tot += sm.sh2[w][tid - 2];
        partials[(size_t)blockIdx.x * 4 + tid] = tot;
    }
}

template <int LOSS>
__global__ void k_gap_final(const double *__restrict__ partials, int nblocks, double n, double lambda,
                            double *__restrict__ out)
{
    // 4 warps, one per partial sum: lane l adds blocks l, l+32, ... in order, then the 32 lanes are added in order
    __shared__ double lanes[4][32];
    __shared__ double tot[4];
    const int q = threadIdx.x >> 5, lane = threadIdx.x & 31;
    double t = 0.0;
    for (int b = lane; b < nblocks; b += 32) t += partials[(size_t)b * 4 + q];
    lanes[q][lane] = t;
    __syncthreads();
    if (threadIdx.x < 4) {
        double a = 0.0;
        for (int l = 0; l < 32; ++l) a += lanes[threadIdx.x][l];
        tot[threadIdx.x] = a;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        double primal, dual;
        if (LOSS == CHICLE_LOSS_RIDGE_PRIMAL) {
            const double cc = tot[0], ww = tot[1], rr = tot[2], ry = tot[3];
            primal = rr / (2.0 * n) + 0.5 * lambda * ww;
            dual = -(rr / (2.0 * n) + ry / n) - cc / (n * n * 2.0 * lambda);
        } else {
            const double lam_n = lambda * n;
            primal = tot[0] / n + 0.5 * lambda * tot[2] / (lam_n * lam_n);
            dual = primal - tot[1] / n;
        }
        out[0] = primal - dual;
        out[1] = primal;
        out[2] = dual;
    }
}

// ---------------------------------------------------------------------------------------- v from scratch
__global__ void __launch_bounds__(kThreads)
k_shared_vector(const int64_t *__restrict__ indptr, const int32_t *__restrict__ indices,
                const float *__restrict__ values, const float *__restrict__ state, int64_t n_coord, int64_t dim,
                float *__restrict__ v)
{
    const int lane = threadIdx.x & 31;
    const int64_t nw = (int64_t)gridDim.x * kWarpsPerBlock;
    for (int64_t c = (int64_t)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5); c < n_coord; c += nw) {
        const float s = state[c];
        if (s == 0.0f) continue;
        if (indptr) {
            const int64_t b = indptr[c], e = indptr[c + 1];
            for (int64_t q = b + lane; q < e; q += 32) atomicAdd(v + indices[q], s * values[q]);
        } else {
            const float *row = values + c * dim;
            for (int64_t j = lane; j < dim; j += 32) atomicAdd(v + j, s * row[j]);
        }
    }
}

} // namespace

cudaError_t launch_validate(Glm &g, bool values, bool rest)
{
    const int64_t nvals = g.indptr ? g.nnz : g.n_coord * g.dim;
    const unsigned grid = (unsigned)g.sm_count * 8;
    if (values) k_validate_values<<<grid, kThreads, 0, g.stream>>>(g.values, nvals, g.d_status);
    if (!rest) return cudaGetLastError();
    k_validate_labels<<<grid, kThreads, 0, g.stream>>>(g.labels, g.n_examples,
                                                       g.loss != CHICLE_LOSS_RIDGE_PRIMAL, g.d_status);
    if (g.indptr)
        k_validate_structure<<<grid, kThreads, 0, g.stream>>>(g.indptr, g.indices, g.n_coord, g.nnz, g.dim,
                                                              g.d_status);
    return cudaGetLastError();
}

cudaError_t launch_sqnorm(Glm &g)
{
    const unsigned grid = (unsigned)g.sm_count * 8;
    k_sqnorm<<<grid, kThreads, 0, g.stream>>>(g.indptr, g.values, g.n_coord, g.dim, g.sqnorm);
    return cudaGetLastError();
}

cudaError_t launch_reduce(Glm &g)
{
    const float *y = g.loss == CHICLE_LOSS_RIDGE_PRIMAL ? g.labels : nullptr;
    float *resid = g.loss == CHICLE_LOSS_RIDGE_PRIMAL ? g.resid : nullptr;
    if ((g.dim & 3) == 0) {
        const int64_t nvec = g.dim / 4;
        const int threads = nvec >= (int64_t)g.sm_count * 2 * kThreads ? kThreads : 64; // small vectors: more, smaller blocks
        unsigned grid = blocks_for(nvec, threads);
        if (grid > (unsigned)g.sm_count * 16) grid = (unsigned)g.sm_count * 16;
        k_reduce_updates<4><<<grid, threads, 0, g.stream>>>(g.v, g.U, g.K, g.dim, y, resid);
    } else {
        unsigned grid = blocks_for(g.dim, kThreads);
        if (grid > (unsigned)g.sm_count * 16) grid = (unsigned)g.sm_count * 16;
        k_reduce_updates<1><<<grid, kThreads, 0, g.stream>>>(g.v, g.U, g.K, g.dim, y, resid);
    }
    return cudaGetLastError();
}

cudaError_t launch_sum_updates(Glm &g, float *delta)
{
    unsigned grid = blocks_for(g.dim, kThreads);
    if (grid > (unsigned)g.sm_count * 16) grid = (unsigned)g.sm_count * 16;
    k_sum_updates<<<grid, kThreads, 0, g.stream>>>(g.U, g.K, g.dim, delta);
    return cudaGetLastError();
}

cudaError_t launch_apply_deltas(Glm &g, const float *deltas, int count)
{
    const float *y = g.loss == CHICLE_LOSS_RIDGE_PRIMAL ? g.labels : nullptr;
    float *resid = g.loss == CHICLE_LOSS_RIDGE_PRIMAL ? g.resid : nullptr;
    unsigned grid = blocks_for(g.dim, kThreads);
    if (grid > (unsigned)g.sm_count * 16) grid = (unsigned)g.sm_count * 16;
    k_apply_deltas<<<grid, kThreads, 0, g.stream>>>(g.v, deltas, count, g.dim, y, resid);
    return cudaGetLastError();
}

cudaError_t launch_mask_state(Glm &g, const unsigned char *keep, float *out)
{
    unsigned grid = blocks_for(g.n_coord, kThreads);
    if (grid > (unsigned)g.sm_count * 16) grid = (unsigned)g.sm_count * 16;
    k_mask_state<<<grid, kThreads, 0, g.stream>>>(g.alpha, g.owner, keep, g.n_coord, out);
    return cudaGetLastError();
}

cudaError_t launch_refresh_resid(Glm &g)
{
    if (g.loss != CHICLE_LOSS_RIDGE_PRIMAL) return cudaSuccess;
    k_resid<<<(unsigned)g.sm_count * 4, kThreads, 0, g.stream>>>(g.v, g.labels, g.dim, g.resid);
    return cudaGetLastError();
}

template <int LOSS, int R, int PER, int HOT = kGapHot, int CAP = kGapCapNz, int STAGES = 3>
cudaError_t launch_gap_stream_per(Glm &g, int nb, double lam_n)
{
    using Shared = GapShared<HOT, CAP, STAGES>;
    auto kern = k_gap_stream<LOSS, R, PER, HOT, CAP, STAGES>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(Shared));
    if (e != cudaSuccess) return e;
    kern<<<nb, kGapConsumers + 32, sizeof(Shared), g.stream>>>(g.indptr, g.indices, g.values, g.labels, g.alpha, g.v,
                                                                   LOSS == CHICLE_LOSS_RIDGE_PRIMAL ? g.resid : g.v, g.n_coord,
                                                                   g.dim, lam_n, g.gap_partials, g.d_status);
    return cudaGetLastError();
}

template <int LOSS, int R> cudaError_t launch_gap_stream(Glm &g, int nb, double lam_n)
{
    // entries a thread keeps in flight: 6 where that covers the average coordinate with some room, else 8
    const double avg = (double)g.nnz / (double)g.n_coord;
    if (avg * 1.15 <= 6.0 * (kGapConsumers / R)) return launch_gap_stream_per<LOSS, R, 6>(g, nb, lam_n);
    return launch_gap_stream_per<LOSS, R, 8>(g, nb, lam_n);
}

template <int LOSS> cudaError_t launch_gap_loss(Glm &g)
{
    const double n = (double)g.n_examples;
    const double lam_n = (double)g.lambda * n;
    int nb = g.gap_blocks;
    const char *force = getenv("CHICLE_FORCE_VARIANT"); // debugging aid: "gapwarp" selects the warp-per-coordinate kernel
    if (g.indptr && !(force && strcmp(force, "gapwarp") == 0)) {
        // sparse data: the streamed kernel, one block per SM; coordinates per tile: as many as keep a tile's non-zeros
        // comfortably inside a stage
        nb = g.sm_count < g.gap_blocks ? g.sm_count : g.gap_blocks;
        const double avg = (double)g.nnz / (double)g.n_coord;
        cudaError_t e;
        if (avg * 128 <= 3300) e = launch_gap_stream<LOSS, 128>(g, nb, lam_n);
        else if (avg <= 39.5 && avg * 128 * 1.05 <= kGapCapNzWide) // (four threads per coordinate, ten entries each)
            e = launch_gap_stream_per<LOSS, 128, 10, kGapHotWide, kGapCapNzWide>(g, nb, lam_n);
        else if (avg * 1.15 <= 60.0 && avg * 128 * 1.05 <= kGapCapNzWider) // (four threads per coordinate, fifteen entries each)
            e = launch_gap_stream_per<LOSS, 128, 15, kGapHotWider, kGapCapNzWider>(g, nb, lam_n);
        else if (avg * 64 <= 3300) e = launch_gap_stream<LOSS, 64>(g, nb, lam_n);
        else if (avg * 32 <= 3300) e = launch_gap_stream<LOSS, 32>(g, nb, lam_n);
        else e = launch_gap_stream<LOSS, 16>(g, nb, lam_n);
        if (e != cudaSuccess) return e;
    } else {
        k_gap_partials<LOSS><<<nb, kThreads, 0, g.stream>>>(g.indptr, g.indices, g.values, g.labels, g.alpha, g.v, g.v, g.n_coord,
                                                            g.dim, lam_n, g.gap_partials, g.d_status);
    }
    k_gap_final<LOSS><<<1, 128, 0, g.stream>>>(g.gap_partials, nb, n, (double)g.lambda, g.gap_out);
    return cudaGetLastError();
}

cudaError_t launch_gap(Glm &g)
{
    switch (g.loss) {
    case CHICLE_LOSS_HINGE_DUAL: return launch_gap_loss<CHICLE_LOSS_HINGE_DUAL>(g);
    case CHICLE_LOSS_LOGISTIC_DUAL: return launch_gap_loss<CHICLE_LOSS_LOGISTIC_DUAL>(g);
    default: return launch_gap_loss<CHICLE_LOSS_RIDGE_PRIMAL>(g);
    }
}

cudaError_t launch_shared_vector(Glm &g)
{
    cudaError_t e = cudaMemsetAsync(g.v, 0, (size_t)g.dim * sizeof(float), g.stream);
    if (e != cudaSuccess) return e;
    k_shared_vector<<<(unsigned)g.sm_count * 8, kThreads, 0, g.stream>>>(g.indptr, g.indices, g.values, g.alpha,
                                                                         g.n_coord, g.dim, g.v);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    return launch_refresh_resid(g);
}

} // namespace chicle
