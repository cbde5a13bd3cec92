// Local SCD solver for sparse coordinates (CSR rows / CSC columns): one CTA per partition, the visiting order
// walked strictly in order (paper Sec. 2.1 worker structure with L = 1; Sec. 5.1: SCD local solver), with the
// part of the local model that a block of steps can touch held in shared memory.
//
// The walk is cut into blocks of kB consecutive steps. For every block the helper warps build, ahead of the
// chain, a compact table of the distinct entries (features for the dual losses, rows for ridge) that the block's
// coordinates touch: an open-addressing hash table in shared memory whose slots carry the read-only shared
// vector v at that entry (Tv) and the partition's accumulated update U_k at that entry (Tu). Each staged
// coordinate stores, per non-zero, its value and the table slot. The chain warp then runs the block's steps
// entirely against shared memory: gather Tv + sigma' * Tu, butterfly reduction, scalar step, scatter into Tu.
//
// U_k's home is global memory (row k of the K x dim workspace, zero at round start). Entering a block, a slot's Tu
// comes either from the previous block's table (the slot is "carried": both blocks touch the entry, and the value
// is copied shared-to-shared once the chain has finished the previous block) or from global memory, gathered
// early while the chain is still busy (the entry is not in the previous block, so its global value is final: older
// blocks were written back before). After a block its table is written back to global memory off the critical
// path. The result is the same as walking the coordinates one by one against a full copy of the local model.
//
// Staging is pipelined three blocks deep: visiting-order entries are loaded three blocks ahead, the per-coordinate
// fields (indptr, label, norm, alpha) two blocks ahead, the non-zeros one block ahead (cp.async into a staging
// area). Blocks that do not fit (a coordinate longer than kCapB entries, or too many distinct entries) are walked
// by the chain directly against global memory. Every wait is bounded.
#include "solver_common.cuh"

namespace chicle {

namespace {

constexpr int kB = 32;                  // steps per block
constexpr int kCapB = 128;              // non-zeros staged per coordinate
constexpr int kHT = 4096;               // hash slots per block (a power of two)
constexpr int kMaxOcc = 3072;           // distinct entries a block may have before it is walked unstaged
#ifndef CHICLE_HELPER_WARPS
#define CHICLE_HELPER_WARPS 7
#endif
constexpr int kHelperWarps = CHICLE_HELPER_WARPS;
constexpr int kHelperThreads = 32 * kHelperWarps;
constexpr int kThreadsB = 32 + kHelperThreads;
constexpr uint16_t kNoCarry = 0xFFFFu;

struct BlockBuf {
    SlotHdr hdr[kB];
    float val[kB][kCapB];
    float Tv[kHT];
    float Tu[kHT];
    int32_t key[kHT];
    uint16_t pos[kB][kCapB];
    uint16_t occ[kHT];     // occupied slots, in insertion order
    uint16_t carry[kHT];   // slot of the same entry in the previous block's table, or kNoCarry
    int32_t n_occ, cnt, slow, pad;
};

struct Stage {
    int32_t idx[kB][kCapB];
    float val[kB][kCapB];
    SlotHdr hdr[kB];
    int32_t rowoff[kB + 1];
    int32_t cnt, slow;
};

struct SharedB {
    uint64_t full[2];
    uint64_t done[2];
    int32_t abort_flag;    // set by whoever ran out of patience; everyone watches it while waiting
    int32_t helper_abort;  // set by helpers only, before a helper barrier, so that they all leave together
    int32_t pad[2];
    Stage st;
    BlockBuf buf[2];
};
static_assert(sizeof(SharedB) <= 227 * 1024, "shared memory budget");

__device__ __forceinline__ void helper_bar() { asm volatile("bar.sync 1, %0;" ::"n"(kHelperThreads) : "memory"); }

__device__ __forceinline__ uint32_t hash_slot(int32_t idx) { return ((uint32_t)idx * 2654435761u) >> 20; }
static_assert(kHT == 4096, "hash_slot keeps 12 bits");

// When a round spans several local epochs a coordinate can come up again before its staged header was prepared
// from its new value (even inside one block), so the chain re-reads alpha itself: lane 0 wrote it, lane 0 reads it.
template <int LOSS>
__device__ __forceinline__ void refresh_state(SlotHdr &h, const float *alpha, int lane)
{
    float al = 0.0f;
    if (lane == 0) al = *reinterpret_cast<const volatile float *>(alpha + h.coord);
    al = __shfl_sync(0xffffffffu, al, 0);
    h.p1 = LOSS == CHICLE_LOSS_RIDGE_PRIMAL ? al : h.p3 * al;
}

template <int LOSS>
__global__ void __launch_bounds__(kThreadsB, 1) k_local_scd_blocked(const SolverParams P)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    SharedB &sh = *reinterpret_cast<SharedB *>(smem_raw);
    const int k = blockIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int *abort_flag = &sh.abort_flag;

    const int64_t off = P.part_off[k];
    const int64_t nk = P.part_off[k + 1] - off;
    const int64_t steps = nk <= 0 ? 0 : (P.H == 0 ? nk : P.H);
    if (threadIdx.x == 0) {
        sh.abort_flag = 0;
        sh.helper_abort = 0;
        for (int s = 0; s < 2; ++s) {
            mbar_init(smem_u32(&sh.full[s]), 1);
            mbar_init(smem_u32(&sh.done[s]), 1);
        }
    }
    __syncthreads();
    if (steps == 0) return;
    float *Uk = P.U + (size_t)k * (size_t)P.dim;
    const int64_t nblocks = (steps + kB - 1) / kB;

    if (warp == 0) {
        // =============================== the chain ===============================
        for (int64_t b = 0; b < nblocks; ++b) {
            BlockBuf &B = sh.buf[b & 1];
            if (!mbar_wait(smem_u32(&sh.full[b & 1]), (uint32_t)(b >> 1) & 1u, abort_flag, P.status)) return;
            const int cnt = B.cnt;
            if (!B.slow) {
                for (int j = 0; j < cnt; ++j) {
                    SlotHdr h = B.hdr[j];
                    if (P.multi_epoch) refresh_state<LOSS>(h, P.alpha, lane);
                    const uint16_t *ps = B.pos[j];
                    const float *xv = B.val[j];
                    float acc = 0.0f, x0 = 0.0f, x1 = 0.0f, u0 = 0.0f, u1 = 0.0f;
                    uint32_t s0 = 0, s1 = 0;
                    if (lane < h.nnz) {
                        s0 = ps[lane];
                        x0 = xv[lane];
                        u0 = B.Tu[s0];
                        acc = x0 * fmaf(P.sigma, u0, B.Tv[s0]);
                    }
                    if (lane + 32 < h.nnz) {
                        s1 = ps[lane + 32];
                        x1 = xv[lane + 32];
                        u1 = B.Tu[s1];
                        acc = fmaf(x1, fmaf(P.sigma, u1, B.Tv[s1]), acc);
                    }
                    for (int e = lane + 64; e < h.nnz; e += 32) {
                        const uint32_t s = ps[e];
                        acc = fmaf(xv[e], fmaf(P.sigma, B.Tu[s], B.Tv[s]), acc);
                    }
                    acc = warp_sum(acc);
                    float delta, new_state;
                    coordinate_step<LOSS>(acc, h, delta, new_state);
                    if (!(fabsf(delta) <= CUDART_MAX_NORMAL_F)) {
                        if (lane == 0) atomicOr(P.status, ST_NONFINITE_STEP);
                        delta = 0.0f;
                        new_state = LOSS == CHICLE_LOSS_RIDGE_PRIMAL ? h.p1 : h.p3 * h.p1;
                    }
                    if (delta != 0.0f) {
                        if (lane < h.nnz) B.Tu[s0] = fmaf(delta, x0, u0);
                        if (lane + 32 < h.nnz) B.Tu[s1] = fmaf(delta, x1, u1);
                        for (int e = lane + 64; e < h.nnz; e += 32) {
                            const uint32_t s = ps[e];
                            B.Tu[s] = fmaf(delta, xv[e], B.Tu[s]);
                        }
                    }
                    if (lane == 0) {
                        // parked in the header and written out by the helpers, off the chain, unless the round
                        // revisits coordinates and needs it in place at once
                        if (P.multi_epoch) P.alpha[h.coord] = new_state;
                        else B.hdr[j].p1 = new_state;
                    }
                    __syncwarp();
                }
            } else {
                // unstaged block: straight against global memory (U_k in global is current: the helpers wrote the
                // previous table back before handing this block over)
                for (int j = 0; j < cnt; ++j) {
                    SlotHdr h = B.hdr[j];
                    if (P.multi_epoch) refresh_state<LOSS>(h, P.alpha, lane);
                    const int32_t *ix = P.indices + h.row_start;
                    const float *xv = P.values + h.row_start;
                    float acc = 0.0f;
                    for (int e = lane; e < h.nnz; e += 32) {
                        const int32_t i = ix[e];
                        acc = fmaf(xv[e], fmaf(P.sigma, Uk[i], P.vbase[i]), acc);
                    }
                    acc = warp_sum(acc);
                    float delta, new_state;
                    coordinate_step<LOSS>(acc, h, delta, new_state);
                    if (!(fabsf(delta) <= CUDART_MAX_NORMAL_F)) {
                        if (lane == 0) atomicOr(P.status, ST_NONFINITE_STEP);
                        delta = 0.0f;
                        new_state = LOSS == CHICLE_LOSS_RIDGE_PRIMAL ? h.p1 : h.p3 * h.p1;
                    }
                    if (delta != 0.0f)
                        for (int e = lane; e < h.nnz; e += 32) {
                            const int32_t i = ix[e];
                            Uk[i] = fmaf(delta, xv[e], Uk[i]);
                        }
                    if (lane == 0) {
                        // parked in the header and written out by the helpers, off the chain, unless the round
                        // revisits coordinates and needs it in place at once
                        if (P.multi_epoch) P.alpha[h.coord] = new_state;
                        else B.hdr[j].p1 = new_state;
                    }
                    __syncwarp();
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh.done[b & 1]));
        }
        return;
    }

    // =============================== helpers ===============================
    const int ht = threadIdx.x - 32;      // 0 .. kHelperThreads-1; ht < 32 (helper warp 0) prepares the headers
    Stage &st = sh.st;

    // Header pipeline, in registers of the header threads: `c_far` is the coordinate of step ht of block b+3 (its
    // load is in flight), F_* are the fields of step ht of block b+2 (in flight), and block b+1's fields are
    // consumed into the staging area in iteration b.
    auto coord_of = [&](int64_t blk) -> int32_t {
        const int64_t t = blk * kB + ht;
        if (ht >= kB || blk >= nblocks || t >= steps) return -1;
        const int64_t ep = P.multi_epoch ? t / nk : 0;
        return P.perm[(size_t)ep * (size_t)P.n_coord + (size_t)(off + (t - ep * nk))];
    };
    struct Fields { int32_t c; int64_t rs, re; float y, s, al; };
    auto issue_fields = [&](int32_t c) -> Fields {
        Fields f{c, 0, 0, 0.f, 0.f, 0.f};
        if (c >= 0) {
            f.rs = P.indptr[c];
            f.re = P.indptr[c + 1];
            f.s = P.sqnorm[c];
            f.al = __ldcg(P.alpha + c);
            if (LOSS != CHICLE_LOSS_RIDGE_PRIMAL) f.y = P.labels[c];
        }
        return f;
    };
    // writes block `blk`'s header fields into the staging area (everything but the alpha-dependent p1 when
    // alpha has to be re-read later) and the prefix sums of the coordinate lengths
    auto stage_headers = [&](int64_t blk, const Fields &f) {
        if (ht < kB) {
            const int cnt = (int)((steps - blk * kB) < kB ? (steps - blk * kB) : kB);
            int32_t nnz = 0;
            if (f.c >= 0) {
                nnz = (int32_t)(f.re - f.rs);
                SlotHdr hd;
                hd.row_start = f.rs;
                hd.coord = f.c;
                hd.nnz = nnz;
                if (LOSS == CHICLE_LOSS_RIDGE_PRIMAL) {
                    hd.p0 = P.inv_n;
                    hd.p1 = f.al;
                    hd.p2 = 1.0f / fmaf(P.sigma * f.s, P.inv_n, P.lambda);
                    hd.p3 = P.lambda;
                } else {
                    hd.p0 = f.y / P.lam_n;
                    hd.p1 = f.y * f.al;
                    hd.p3 = f.y;
                    if (LOSS == CHICLE_LOSS_HINGE_DUAL) hd.p2 = f.s > 0.0f ? P.lam_n / (P.sigma * f.s) : CUDART_INF_F;
                    else hd.p2 = P.sigma * f.s / P.lam_n;
                }
                hd.pad[0] = hd.pad[1] = 0;
                st.hdr[ht] = hd;
            }
            // inclusive scan of nnz over the 32 header lanes -> rowoff
            int32_t inc = nnz;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int32_t y = __shfl_up_sync(0xffffffffu, inc, o);
                if (lane >= o) inc += y;
            }
            st.rowoff[ht + 1] = inc;
            const bool too_long = __any_sync(0xffffffffu, nnz > kCapB);
            if (ht == 0) {
                st.rowoff[0] = 0;
                st.cnt = cnt;
                st.slow = too_long ? 1 : 0;
            }
        }
    };
    // cp.async of block `blk`'s non-zeros into the staging area (headers of that block are in `st`)
    auto issue_entries = [&]() {
        if (st.slow) return;
        const int hw = ht >> 5;
        for (int j = hw; j < st.cnt; j += kHelperWarps) {
            const int nnz = st.hdr[j].nnz;
            const int64_t rs = st.hdr[j].row_start;
            for (int e = lane; e < nnz; e += 32) {
                cp_async4(smem_u32(&st.idx[j][e]), P.indices + rs + e);
                cp_async4(smem_u32(&st.val[j][e]), P.values + rs + e);
            }
        }
    };

    // ---- prologue: block 0 staged, block 1 fields and block 2 coordinates in flight
    Fields f_next;       // fields of block b+1 (arrived or in flight)
    Fields f_far;        // fields of block b+2 (in flight)
    int32_t c_far;       // coordinate of block b+3 (in flight)
    {
        Fields f0 = issue_fields(coord_of(0));
        f_next = issue_fields(coord_of(1));
        f_far = issue_fields(coord_of(2));
        c_far = coord_of(3);
        stage_headers(0, f0);
        helper_bar();
        issue_entries();
    }

    for (int64_t b = 0; b < nblocks; ++b) {
        BlockBuf &B = sh.buf[b & 1];
        BlockBuf &Prev = sh.buf[(b & 1) ^ 1];
        const bool have_prev = b > 0;
        // ---- S0: reset the table of this buffer (its previous block was written back in the last iteration)
        for (int p = ht; p < kHT; p += kHelperThreads) B.key[p] = -1;
        if (ht == 0) B.n_occ = 0;
        cp_async_wait_all();
        helper_bar(); // staging area holds block b's headers and non-zeros
        const int cnt = st.cnt;
        bool slow = st.slow != 0;
        const bool prev_slow = have_prev && Prev.slow != 0;
        // entries not in the previous table may be gathered from global memory now, unless the chain is writing
        // global memory itself (previous block unstaged)
        const bool early_ok = !prev_slow;
        // ---- S3: build the table
        if (ht < cnt) B.hdr[ht] = st.hdr[ht];
        if (!slow) {
            // insert: a helper warp takes whole coordinates; lanes over the non-zeros
            const int hw = ht >> 5;
            const uint32_t lt_mask = (1u << lane) - 1u;
            for (int j = hw; j < cnt; j += kHelperWarps) {
                const int nnz = st.hdr[j].nnz;
                for (int e0 = 0; e0 < nnz; e0 += 32) {
                    const int e = e0 + lane;
                    bool is_new = false;
                    uint32_t p = 0;
                    if (e < nnz) {
                        const int32_t idx = st.idx[j][e];
                        p = hash_slot(idx);
                        bool placed = false;
                        if (B.n_occ <= kMaxOcc) {
                            for (int probe = 0; probe < kHT; ++probe) {
                                // a plain read settles most probes (the key is already there, or the slot is
                                // taken by another key); only an empty slot needs the compare-and-swap
                                int32_t seen = *reinterpret_cast<volatile int32_t *>(&B.key[p]);
                                if (seen == -1) seen = atomicCAS(&B.key[p], -1, idx);
                                if (seen == -1) { is_new = true; placed = true; break; }
                                if (seen == idx) { placed = true; break; }
                                p = (p + 1) & (kHT - 1);
                            }
                        }
                        if (!placed) { B.slow = 2; p = 0; } // over-full: the block will be walked unstaged
                        B.pos[j][e] = (uint16_t)p;
                        B.val[j][e] = st.val[j][e];
                    }
                    // one counter update per warp for the new slots
                    const uint32_t newmask = __ballot_sync(0xffffffffu, is_new);
                    if (newmask) {
                        const int leader = __ffs(newmask) - 1;
                        int slot = 0;
                        if (lane == leader) slot = atomicAdd(&B.n_occ, __popc(newmask));
                        slot = __shfl_sync(0xffffffffu, slot, leader) + __popc(newmask & lt_mask);
                        if (is_new) B.occ[slot & (kHT - 1)] = (uint16_t)p;
                    }
                }
            }
        }
        helper_bar(); // all slots known
        if (!slow && (B.slow == 2 || B.n_occ > kMaxOcc)) slow = true;
        if (!slow) {
            // fill: per distinct entry, look it up in the previous table and fetch v and (if final) U_k
            const int n_occ = B.n_occ;
            for (int i = ht; i < n_occ; i += kHelperThreads) {
                const uint32_t p = B.occ[i];
                const int32_t idx = B.key[p];
                uint16_t cp = kNoCarry;
                if (have_prev && !prev_slow) {
                    uint32_t q = hash_slot(idx);
                    for (int probe = 0; probe < kHT; ++probe) {
                        const int32_t kq = Prev.key[q];
                        if (kq == idx) { cp = (uint16_t)q; break; }
                        if (kq == -1) break;
                        q = (q + 1) & (kHT - 1);
                    }
                }
                B.carry[p] = cp;
                cp_async4(smem_u32(&B.Tv[p]), P.vbase + idx);
                // U_k is only ever written by this SM, so a cached copy cannot be stale
                if (cp == kNoCarry && early_ok) cp_async4(smem_u32(&B.Tu[p]), Uk + idx);
            }
            cp_async_wait_all();
        }
        helper_bar(); // table built, staging area free
        // ---- S5: advance the staging pipeline: headers of block b+1 into the staging area, its non-zeros by
        //      cp.async, fields of block b+3 and coordinates of block b+4 into flight
        if (b + 1 < nblocks) stage_headers(b + 1, f_next);
        f_next = f_far;
        f_far = issue_fields(c_far);
        c_far = coord_of(b + 4);
        helper_bar();
        if (b + 1 < nblocks) issue_entries();
        // ---- S6: the chain must have finished block b-1 before its table is read
        if (have_prev) {
            if (!mbar_wait(smem_u32(&sh.done[(b - 1) & 1]), (uint32_t)((b - 1) >> 1) & 1u, abort_flag, P.status))
                sh.helper_abort = 1;
            helper_bar(); // a helper that gave up must not leave the others at a barrier
            if (sh.helper_abort) {
                cp_async_wait_all();
                return;
            }
        }
        if (have_prev && !P.multi_epoch && ht < Prev.cnt) P.alpha[Prev.hdr[ht].coord] = Prev.hdr[ht].p1;
        const bool write_back_first = have_prev && !prev_slow && slow; // an unstaged block reads global memory
        if (write_back_first) {
            for (int i = ht; i < Prev.n_occ; i += kHelperThreads) {
                const int p = Prev.occ[i];
                Uk[Prev.key[p]] = Prev.Tu[p];
            }
        }
        // ---- S7: complete the table: carried slots from the previous table, late gathers
        if (!slow) {
            const int n_occ = B.n_occ;
            for (int base = 0; base < n_occ; base += 4 * kHelperThreads) {
                uint32_t pp[4];
                uint16_t cc[4];
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    const int i = base + r * kHelperThreads + ht;
                    pp[r] = i < n_occ ? B.occ[i] : kHT;
                }
#pragma unroll
                for (int r = 0; r < 4; ++r) cc[r] = pp[r] < kHT ? B.carry[pp[r]] : kNoCarry;
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    if (cc[r] != kNoCarry) B.Tu[pp[r]] = Prev.Tu[cc[r]];
                    else if (!early_ok && pp[r] < kHT) B.Tu[pp[r]] = __ldcg(Uk + B.key[pp[r]]);
                }
            }
        }
        if (ht == 0) {
            B.cnt = cnt;
            B.slow = slow ? 1 : 0;
        }
        helper_bar();
        if (ht == 0) mbar_arrive(smem_u32(&sh.full[b & 1]));
        // ---- the previous table goes back to global memory, off the chain's critical path
        if (have_prev && !prev_slow && !write_back_first) {
            for (int i = ht; i < Prev.n_occ; i += kHelperThreads) {
                const int p = Prev.occ[i];
                Uk[Prev.key[p]] = Prev.Tu[p];
            }
        }
        helper_bar(); // the previous buffer may be rebuilt, and its global values are in place
    }
    // ---- epilogue: the last block's table
    {
        const int64_t b = nblocks - 1;
        BlockBuf &L = sh.buf[b & 1];
        if (!mbar_wait(smem_u32(&sh.done[b & 1]), (uint32_t)(b >> 1) & 1u, abort_flag, P.status)) sh.helper_abort = 1;
        helper_bar();
        if (sh.helper_abort) return;
        if (!P.multi_epoch && ht < L.cnt) P.alpha[L.hdr[ht].coord] = L.hdr[ht].p1;
        if (!L.slow)
            for (int i = ht; i < L.n_occ; i += kHelperThreads) {
                const int p = L.occ[i];
                Uk[L.key[p]] = L.Tu[p];
            }
    }
}

} // namespace

cudaError_t launch_blocked_solver(Glm &g, const SolverParams &P)
{
    const size_t smem = sizeof(SharedB);
    cudaError_t e;
    switch (g.loss) {
    case CHICLE_LOSS_HINGE_DUAL:
        e = cudaFuncSetAttribute(k_local_scd_blocked<CHICLE_LOSS_HINGE_DUAL>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        k_local_scd_blocked<CHICLE_LOSS_HINGE_DUAL><<<g.K, kThreadsB, smem, g.stream>>>(P);
        break;
    case CHICLE_LOSS_LOGISTIC_DUAL:
        e = cudaFuncSetAttribute(k_local_scd_blocked<CHICLE_LOSS_LOGISTIC_DUAL>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        k_local_scd_blocked<CHICLE_LOSS_LOGISTIC_DUAL><<<g.K, kThreadsB, smem, g.stream>>>(P);
        break;
    default:
        e = cudaFuncSetAttribute(k_local_scd_blocked<CHICLE_LOSS_RIDGE_PRIMAL>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        k_local_scd_blocked<CHICLE_LOSS_RIDGE_PRIMAL><<<g.K, kThreadsB, smem, g.stream>>>(P);
        break;
    }
    return cudaGetLastError();
}

} // namespace chicle
