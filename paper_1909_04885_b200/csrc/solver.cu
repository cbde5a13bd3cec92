// Local stochastic coordinate-descent solvers: one CTA per partition, walking the partition's visiting order
// strictly in order (paper Sec. 2.2 worker structure with L = 1 and "CoCoA"; Sec. 5.1: SCD local solver).
//
// Roles inside a CTA
//   warp 0        the chain: per step one dot product (lanes over the coordinate's entries, butterfly
//                 reduction), the scalar step in registers, the scatter into the local model.
//   warps 1..P    producers: run ahead of the chain and stage everything a step needs that does not depend on
//                 earlier steps into a ring of shared-memory slots -- the coordinate id from the visiting order,
//                 its entries, the read-only part of the shared vector at those entries (v is constant during a
//                 round), and per-coordinate constants with their divisions already done. Copies are cp.async;
//                 a slot is handed over through an mbarrier that the copies themselves arrive on.
//
// Local model: v_local = v + sigma' * U_k, where U_k is the partition's own accumulated update.
//   dense rows   v_local and U_k live in shared memory; U_k is written out once at the end.
//   sparse       U_k lives in global memory (one row of the K x dim workspace, zero at round start) and is only
//                ever touched by this CTA, so it stays in this SM's L1 / the L2; v is gathered by the producers.
//
// Every wait is bounded; when one runs out the kernel records it in the status word and all roles return.
#include <cstdlib>
#include <cstring>
#include <vector>

#include "solver_common.cuh"

namespace chicle {

namespace {

constexpr int kProdWarps = 4;
constexpr int kGroup = 4;              // packets a producer keeps in flight
constexpr int kSparseCap = 128;        // entries a sparse slot can hold; longer coordinates take the slow path
template <int LOSS, bool DENSE>
__global__ void __launch_bounds__(32 * (1 + kProdWarps), 1) k_local_scd(const SolverParams P)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const int k = blockIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nslot = P.nslot, cap = P.cap;

    // ---- carve shared memory
    uint64_t *bar_full = reinterpret_cast<uint64_t *>(smem_raw);
    uint64_t *bar_empty = bar_full + nslot;
    volatile long long *progress = reinterpret_cast<volatile long long *>(bar_empty + nslot);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(progress + 1);
    SlotHdr *hdrs = reinterpret_cast<SlotHdr *>(smem_raw + ((2 * nslot + 2) * 8 + 15) / 16 * 16);
    float *fbase = reinterpret_cast<float *>(reinterpret_cast<unsigned char *>(hdrs) +
                                             ((size_t)nslot * sizeof(SlotHdr) + 127) / 128 * 128);
    float *vloc = nullptr, *dv = nullptr, *s_val, *s_base = nullptr;
    int32_t *s_idx = nullptr;
    if (DENSE) {
        vloc = fbase;
        dv = fbase + cap;
        s_val = fbase + 2 * cap;
    } else {
        s_val = fbase;
        s_base = fbase + (size_t)nslot * cap;
        s_idx = reinterpret_cast<int32_t *>(fbase + 2 * (size_t)nslot * cap);
    }

    const int64_t off = P.part_off[k];
    const int64_t nk = P.part_off[k + 1] - off;
    const int64_t steps = partition_steps(P, k, nk);

    if (threadIdx.x == 0) {
        *progress = 0;
        *abort_flag = 0;
    }
    for (int s = threadIdx.x; s < nslot; s += blockDim.x) {
        mbar_init(smem_u32(&bar_full[s]), 33);  // 32 copy-completion arrivals + 1 plain arrival
        mbar_init(smem_u32(&bar_empty[s]), 32); // the chain warp's lanes
    }
    if (DENSE) {
        for (int j = threadIdx.x; j < cap; j += blockDim.x) {
            vloc[j] = j < P.dim ? P.vbase[j] : 0.0f;
            dv[j] = 0.0f;
        }
    }
    __syncthreads();
    if (steps == 0) {
        if (DENSE)
            for (int j = threadIdx.x; j < P.dim; j += blockDim.x) P.U[(size_t)k * P.dim + j] = 0.0f;
        return;
    }
    float *Uk = P.U + (size_t)k * (size_t)P.dim;

    if (warp == 0) {
        // =============================== the chain ===============================
        for (int64_t t = 0; t < steps; ++t) {
            const int s = (int)(t % nslot);
            const uint32_t use = (uint32_t)(t / nslot);
            if (!mbar_wait(smem_u32(&bar_full[s]), use & 1u, abort_flag, P.status)) return;
            const SlotHdr h = hdrs[s];
            float acc = 0.0f;
            float delta, new_state;
            if (DENSE) {
                const float *row = s_val + (size_t)s * cap;
                for (int j = lane; j < (int)P.dim; j += 32) acc = fmaf(row[j], vloc[j], acc);
                acc = warp_sum(acc);
                coordinate_step<LOSS>(acc, h, delta, new_state);
                if (!(fabsf(delta) <= CUDART_MAX_NORMAL_F)) {
                    if (lane == 0) atomicOr(P.status, ST_NONFINITE_STEP);
                    delta = 0.0f;
                    new_state = LOSS == CHICLE_LOSS_RIDGE_PRIMAL ? h.p1 : h.p3 * h.p1;
                }
                if (delta != 0.0f) {
                    const float sd = P.sigma * delta;
                    for (int j = lane; j < (int)P.dim; j += 32) {
                        const float x = row[j];
                        vloc[j] = fmaf(sd, x, vloc[j]);
                        dv[j] = fmaf(delta, x, dv[j]);
                    }
                }
            } else if (h.nnz <= cap) {
                const int32_t *ix = s_idx + (size_t)s * cap;
                const float *xv = s_val + (size_t)s * cap;
                const float *bv = s_base + (size_t)s * cap;
                // first two strided entries stay in registers (covers up to 64 entries without re-reading)
                int32_t j0 = 0, j1 = 0;
                float x0 = 0.0f, x1 = 0.0f, u0 = 0.0f, u1 = 0.0f;
                if (lane < h.nnz) {
                    j0 = ix[lane];
                    x0 = xv[lane];
                    u0 = Uk[j0];
                    acc = x0 * fmaf(P.sigma, u0, bv[lane]);
                }
                if (lane + 32 < h.nnz) {
                    j1 = ix[lane + 32];
                    x1 = xv[lane + 32];
                    u1 = Uk[j1];
                    acc = fmaf(x1, fmaf(P.sigma, u1, bv[lane + 32]), acc);
                }
                for (int e = lane + 64; e < h.nnz; e += 32)
                    acc = fmaf(xv[e], fmaf(P.sigma, Uk[ix[e]], bv[e]), acc);
                acc = warp_sum(acc);
                coordinate_step<LOSS>(acc, h, delta, new_state);
                if (!(fabsf(delta) <= CUDART_MAX_NORMAL_F)) {
                    if (lane == 0) atomicOr(P.status, ST_NONFINITE_STEP);
                    delta = 0.0f;
                    new_state = LOSS == CHICLE_LOSS_RIDGE_PRIMAL ? h.p1 : h.p3 * h.p1;
                }
                if (delta != 0.0f) {
                    if (lane < h.nnz) Uk[j0] = fmaf(delta, x0, u0);
                    if (lane + 32 < h.nnz) Uk[j1] = fmaf(delta, x1, u1);
                    for (int e = lane + 64; e < h.nnz; e += 32) {
                        const int32_t j = ix[e];
                        Uk[j] = fmaf(delta, xv[e], Uk[j]);
                    }
                }
            } else {
                // slow path: a coordinate with more entries than a slot holds is read straight from global memory
                const int32_t *ix = P.indices + h.row_start;
                const float *xv = P.values + h.row_start;
                for (int e = lane; e < h.nnz; e += 32) {
                    const int32_t j = ix[e];
                    acc = fmaf(xv[e], fmaf(P.sigma, Uk[j], P.vbase[j]), acc);
                }
                acc = warp_sum(acc);
                coordinate_step<LOSS>(acc, h, delta, new_state);
                if (!(fabsf(delta) <= CUDART_MAX_NORMAL_F)) {
                    if (lane == 0) atomicOr(P.status, ST_NONFINITE_STEP);
                    delta = 0.0f;
                    new_state = LOSS == CHICLE_LOSS_RIDGE_PRIMAL ? h.p1 : h.p3 * h.p1;
                }
                if (delta != 0.0f)
                    for (int e = lane; e < h.nnz; e += 32) {
                        const int32_t j = ix[e];
                        Uk[j] = fmaf(delta, xv[e], Uk[j]);
                    }
            }
            // The new alpha goes to global memory off the chain (a global store followed by the release that hands
            // the slot back would stall every step): it is parked in the slot and written out by the producer
            // that reuses the slot. Rounds that revisit coordinates need it in place at once.
            if (lane == 0) {
                if (P.multi_epoch) P.alpha[h.coord] = new_state;
                else hdrs[s].p1 = new_state;
            }
            __syncwarp();
            if (P.multi_epoch) {
                __threadfence_block();
                if (lane == 0) *progress = t + 1;
            }
            mbar_arrive(smem_u32(&bar_empty[s]));
        }
        if (!P.multi_epoch) {
            // results still parked in the ring: the last min(steps, nslot) steps
            const int live = steps < nslot ? (int)steps : nslot;
            for (int s = lane; s < live; s += 32) P.alpha[hdrs[s].coord] = hdrs[s].p1;
        }
        if (DENSE) {
            __syncwarp();
            for (int j = lane; j < (int)P.dim; j += 32) Uk[j] = dv[j];
        }
    } else {
        // =============================== producers ===============================
        // Producer warp w owns the slots [w*batch, (w+1)*batch): batch b of `batch` consecutive steps goes to warp
        // b mod P, so successive uses of a slot are always filled by the same warp and the parity waits on its
        // "empty" barrier can never be more than one phase behind.
        const int pw = warp - 1;
        const int batch = nslot / kProdWarps;
        const int64_t n_batches = (steps + batch - 1) / batch;
        for (int64_t b = pw; b < n_batches; b += kProdWarps) {
            const int64_t t0 = b * batch;
            const int cnt = (int)((steps - t0) < batch ? (steps - t0) : batch);
            const int64_t ep_first = t0 / nk, ep_last = (t0 + cnt - 1) / nk;
            int32_t c = 0, nnz = 0;
            int64_t rs = 0;
            float p0 = 0.f, p1 = 0.f, p2 = 0.f, p3 = 0.f;
            for (int64_t ep = ep_first; ep <= ep_last; ++ep) {
                // lanes [l_lo, l_hi) of this batch are steps of local epoch ep
                const int l_lo = (int)(ep * nk > t0 ? ep * nk - t0 : 0);
                const int l_hi = (int)((ep + 1) * nk - t0 < cnt ? (ep + 1) * nk - t0 : cnt);
                if (ep > 0) {
                    // alpha of a coordinate visited again in a later local epoch must be read after the chain
                    // wrote it: wait until the chain has finished the previous epoch
                    uint32_t it = 0;
                    while (*progress < ep * nk) {
                        if (*abort_flag) { cp_async_wait_all(); return; }
                        if (++it > kSpinLimit) {
                            *abort_flag = 1;
                            atomicOr(P.status, ST_WAIT_TIMEOUT);
                            cp_async_wait_all();
                            return;
                        }
                        __nanosleep(64);
                    }
                    __threadfence_block();
                }
                // ---- per-step headers: lane l prepares step t0 + l
                if (lane >= l_lo && lane < l_hi) {
                    const int64_t pos = t0 + lane - ep * nk;
                    c = P.perm[(size_t)ep * (size_t)P.n_coord + (size_t)(off + pos)];
                    if (DENSE) {
                        rs = (int64_t)c * P.dim;
                        nnz = (int32_t)P.dim;
                    } else {
                        rs = P.indptr[c];
                        nnz = (int32_t)(P.indptr[c + 1] - rs);
                    }
                    const float s = P.sqnorm[c];
                    const float st = __ldcg(P.alpha + c);
                    if (LOSS == CHICLE_LOSS_RIDGE_PRIMAL) {
                        p0 = P.inv_n;
                        p1 = st;
                        p2 = 1.0f / fmaf(P.sigma * s, P.inv_n, P.lambda);
                        p3 = P.lambda;
                    } else {
                        const float y = P.labels[c];
                        p0 = y / P.lam_n;
                        p1 = y * st;
                        p3 = y;
                        if (LOSS == CHICLE_LOSS_HINGE_DUAL) p2 = s > 0.0f ? P.lam_n / (P.sigma * s) : CUDART_INF_F;
                        else p2 = P.sigma * s / P.lam_n;
                    }
                }
                // ---- stage the packets, kGroup at a time
                for (int g0 = l_lo; g0 < l_hi; g0 += kGroup) {
                    int32_t idxr[kGroup][kSparseCap / 32];
                    int32_t g_nnz[kGroup];
                    int64_t g_rs[kGroup];
#pragma unroll
                    for (int g = 0; g < kGroup; ++g) {
                        const int l = g0 + g;
                        g_nnz[g] = __shfl_sync(0xffffffffu, nnz, l & 31);
                        g_rs[g] = __shfl_sync(0xffffffffu, rs, l & 31);
                        if (l >= l_hi) g_nnz[g] = -1;
                    }
                    // wait for the slots, then issue the index loads of the whole group
#pragma unroll
                    for (int g = 0; g < kGroup; ++g) {
                        if (g_nnz[g] < 0) continue;
                        const int64_t t = t0 + g0 + g;
                        const int s = (int)(t % nslot);
                        const uint32_t use = (uint32_t)(t / nslot);
                        if (use > 0 && !mbar_wait(smem_u32(&bar_empty[s]), (use - 1u) & 1u, abort_flag, P.status)) {
                            cp_async_wait_all();
                            return;
                        }
                        if (use > 0 && !P.multi_epoch && lane == 0) P.alpha[hdrs[s].coord] = hdrs[s].p1;
                        if (!DENSE && g_nnz[g] <= cap) {
#pragma unroll
                            for (int r = 0; r < kSparseCap / 32; ++r) {
                                const int e = r * 32 + lane;
                                idxr[g][r] = e < g_nnz[g] ? P.indices[g_rs[g] + e] : 0;
                            }
                        }
                    }
#pragma unroll
                    for (int g = 0; g < kGroup; ++g) {
                        if (g_nnz[g] < 0) continue;
                        const int l = g0 + g;
                        const int64_t t = t0 + l;
                        const int s = (int)(t % nslot);
                        const uint32_t bar = smem_u32(&bar_full[s]);
                        if (DENSE) {
                            const float *src = P.values + g_rs[g];
                            const uint32_t dst = smem_u32(s_val + (size_t)s * cap);
                            if ((P.dim & 3) == 0) {
                                for (int j4 = lane; j4 < (int)(P.dim >> 2); j4 += 32)
                                    cp_async16(dst + 16u * j4, src + 4 * j4);
                            } else {
                                for (int j = lane; j < (int)P.dim; j += 32) cp_async4(dst + 4u * j, src + j);
                            }
                        } else if (g_nnz[g] <= cap) {
                            const uint32_t dval = smem_u32(s_val + (size_t)s * cap);
                            const uint32_t dbase = smem_u32(s_base + (size_t)s * cap);
                            int32_t *dix = s_idx + (size_t)s * cap;
#pragma unroll
                            for (int r = 0; r < kSparseCap / 32; ++r) {
                                const int e = r * 32 + lane;
                                if (e < g_nnz[g]) {
                                    cp_async4(dval + 4u * e, P.values + g_rs[g] + e);
                                    cp_async4(dbase + 4u * e, P.vbase + idxr[g][r]);
                                    dix[e] = idxr[g][r];
                                }
                            }
                        }
                        cp_async_arrive_noinc(bar);
                        // header: every lane holds its own step's constants; lane l writes the header of step l
                        if (lane == l) {
                            SlotHdr hd;
                            hd.row_start = rs;
                            hd.coord = c;
                            hd.nnz = nnz;
                            hd.p0 = p0; hd.p1 = p1; hd.p2 = p2; hd.p3 = p3;
                            hd.pad[0] = hd.pad[1] = 0;
                            hdrs[s] = hd;
                        }
                        __syncwarp();
                        if (lane == l) mbar_arrive(bar);
                    }
                }
            }
        }
        cp_async_wait_all();
    }
}

template <int LOSS, bool DENSE>
cudaError_t launch_variant(Glm &g, const SolverParams &P, size_t smem)
{
    auto kern = k_local_scd<LOSS, DENSE>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kern<<<g.K, 32 * (1 + kProdWarps), smem, g.stream>>>(P);
    return cudaGetLastError();
}

size_t smem_bytes(bool dense, int cap, int nslot)
{
    size_t s = ((size_t)(2 * nslot + 2) * 8 + 15) / 16 * 16;
    s += ((size_t)nslot * sizeof(SlotHdr) + 127) / 128 * 128;
    if (dense) s += (size_t)(2 + nslot) * cap * 4;
    else s += (size_t)3 * nslot * cap * 4;
    return s + 128;
}

} // namespace

cudaError_t launch_blocked_solver(Glm &g, const SolverParams &P);
int blocked_solver_max_dense_dim();

bool solver_supports_dense(int64_t dim, int max_smem_optin)
{
    if (dim > (1 << 20)) return false;
    const int cap = (int)((dim + 31) / 32 * 32);
    return smem_bytes(true, cap, 4) <= (size_t)max_smem_optin;
}

cudaError_t launch_local_solver(Glm &g, int64_t H, float sigma_prime, int *variant)
{
    SolverParams P{};
    P.indptr = g.indptr;
    P.indices = g.indices;
    P.values = g.values;
    P.labels = g.labels;
    P.sqnorm = g.sqnorm;
    P.alpha = g.alpha;
    P.vbase = g.loss == CHICLE_LOSS_RIDGE_PRIMAL ? g.resid : g.v;
    P.U = g.U;
    P.part_off = g.part_off;
    P.perm = g.perm;
    P.status = g.d_status;
    P.n_coord = g.n_coord;
    P.dim = g.dim;
    P.H = H;
    P.steps_k = g.round_steps ? g.d_steps : nullptr;
    P.lam_n = g.lambda * (float)g.n_examples;
    P.inv_n = 1.0f / (float)g.n_examples;
    P.lambda = g.lambda;
    P.sigma = sigma_prime;
    const int64_t min_nk = g.min_nk;
    P.multi_epoch = (H != 0 && H > min_nk) ? 1 : 0;

    const bool dense = g.fmt == CHICLE_FMT_DENSE_ROWMAJOR;
    const size_t budget = (size_t)g.max_smem_optin;
    int cap, nslot = 64; // a multiple of the producer warp count; each producer owns nslot / P slots
    const char *force = getenv("CHICLE_FORCE_VARIANT"); // debugging aid: "ring" selects the unblocked solver
    const bool ring = force && strcmp(force, "ring") == 0;
    const bool blocked = force && strcmp(force, "blocked") == 0;
    if (g.la_rec && !ring && !blocked && (!dense || g.dim <= lookahead_max_dense_dim())) {
        *variant = dense ? 5 : 4;
        if (!P.multi_epoch) return launch_lookahead_solver(g, P);
        // H spans several local epochs: one prepare + chain pair per epoch. Partition k takes what is left of its H
        // steps, at most one pass over its coordinates, along that epoch's visiting order; the prepared headers of an
        // epoch see the state the epoch before left, and the accumulated updates carry over in U.
        const int64_t epochs = (H + min_nk - 1) / min_nk;
        std::vector<int64_t> steps((size_t)g.K);
        P.multi_epoch = 0;
        P.H = 0;
        P.steps_k = g.d_steps;
        const bool time_prepare = g.time_prepare;
        cudaError_t e = cudaSuccess;
        for (int64_t ep = 0; ep < epochs && e == cudaSuccess; ++ep) {
            int64_t total = 0;
            for (int32_t k = 0; k < g.K; ++k) {
                const int64_t nk = g.h_part_off[k + 1] - g.h_part_off[k];
                const int64_t left = H - ep * nk;
                steps[(size_t)k] = left <= 0 ? 0 : (left < nk ? left : nk);
                total += steps[(size_t)k];
            }
            if (total == 0) break;
            // a pageable source: the runtime has taken its copy when the call returns, and the copy is ordered behind
            // the kernels of the epoch before on the stream
            e = cudaMemcpyAsync(g.d_steps, steps.data(), (size_t)g.K * sizeof(int64_t), cudaMemcpyHostToDevice, g.stream);
            if (e != cudaSuccess) break;
            P.perm = g.perm + (size_t)ep * (size_t)g.n_coord;
            g.round_steps = steps.data();
            g.time_prepare = time_prepare && ep == 0; // the prepare time reported is the first epoch's
            e = launch_lookahead_solver(g, P);
        }
        g.round_steps = nullptr;
        g.time_prepare = time_prepare;
        return e;
    }
    if (dense && g.dim <= blocked_solver_max_dense_dim() && !ring) {
        *variant = 3;
        return launch_blocked_solver(g, P);
    }
    if (dense) {
        cap = (int)((g.dim + 31) / 32 * 32);
        while (nslot > 4 && smem_bytes(true, cap, nslot) > budget) nslot /= 2;
        if (smem_bytes(true, cap, nslot) > budget) return cudaErrorInvalidConfiguration;
        *variant = 0;
    } else {
        if (!ring) {
            *variant = 1;
            return launch_blocked_solver(g, P);
        }
        cap = kSparseCap;
        while (nslot > 4 && smem_bytes(false, cap, nslot) > budget / 2) nslot /= 2; // leave room for L1
        *variant = 2;
    }
    P.cap = cap;
    P.nslot = nslot;
    const size_t smem = smem_bytes(dense, cap, nslot);

    switch (g.loss) {
    case CHICLE_LOSS_HINGE_DUAL:
        return dense ? launch_variant<CHICLE_LOSS_HINGE_DUAL, true>(g, P, smem)
                     : launch_variant<CHICLE_LOSS_HINGE_DUAL, false>(g, P, smem);
    case CHICLE_LOSS_LOGISTIC_DUAL:
        return dense ? launch_variant<CHICLE_LOSS_LOGISTIC_DUAL, true>(g, P, smem)
                     : launch_variant<CHICLE_LOSS_LOGISTIC_DUAL, false>(g, P, smem);
    default:
        return launch_variant<CHICLE_LOSS_RIDGE_PRIMAL, false>(g, P, smem);
    }
}

} // namespace chicle
