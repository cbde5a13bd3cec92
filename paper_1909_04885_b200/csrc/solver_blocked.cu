// Local SCD solver for sparse coordinates (CSR rows / CSC columns): one CTA per partition, the visiting order
// walked strictly in order (paper Sec. 2.1 worker structure with L = 1; Sec. 5.1: SCD local solver), with the
// part of the local model that the next steps can touch held in shared memory.
//
// Local model: v_local = v + sigma' * U_k; U_k (the partition's accumulated update, zero at round start) has its
// home in row k of the K x dim workspace in global memory. Entry ids are frequency-ranked when the problem is
// created (id 0 is the most frequent feature), which gives two places for the live part of U_k:
//   hot   ids below HOT: a direct array in shared memory for the whole kernel (no look-up at all);
//   cold  the remaining ids: the walk is cut into blocks of kB consecutive steps and, per block, the helper warps
//         build a small open-addressing hash table in shared memory over the block's distinct cold ids.
// Every staged non-zero carries its value, the read-only v at its id (gathered by the helpers with cp.async; v is
// constant during a round) and a 16-bit slot (hot id, or HOT + table slot). The chain warp runs a block's steps
// entirely against shared memory: gather, butterfly reduction, scalar step in registers, scatter.
//
// A cold slot's U_k value comes from the previous block's table when that block touches the id too ("carried":
// copied shared-to-shared once the chain has finished the previous block) and from global memory otherwise,
// fetched early while the chain is still busy (the id is not in the previous block, so its global value is final:
// older blocks were written back before). A finished block's table goes back to global memory off the critical
// path, and so do the new alpha values, which the chain parks in the block's headers. The result equals walking
// the coordinates one by one against a full copy of the local model.
//
// Staging runs three blocks deep: visiting-order entries three blocks ahead, per-coordinate fields two blocks
// ahead (one helper warp does nothing else), non-zeros one block ahead (cp.async into a staging area). A block that
// does not fit (a coordinate longer than CAP, too many distinct cold ids) is walked by the chain against global
// memory for its cold ids. The roles hand blocks over through named hardware barriers (no polling); every role
// runs the same number of blocks and leaves only at the end, so each barrier always gets its full count.
#include "solver_common.cuh"

namespace chicle {

namespace {

constexpr int kB = 32;                  // steps per block
#ifndef CHICLE_HELPER_WARPS
#define CHICLE_HELPER_WARPS 7
#endif
constexpr int kHelperWarps = CHICLE_HELPER_WARPS; // warp 0 of them prepares headers, the others stage non-zeros
constexpr int kHelperThreads = 32 * kHelperWarps;
constexpr int kEntryWarps = kHelperWarps - 1;
constexpr int kEntryThreads = 32 * kEntryWarps;
constexpr int kThreadsB = 32 + kHelperThreads;
constexpr uint16_t kNoCarry = 0xFFFFu;

template <int HTC, int CAP> struct BlockBuf {
    SlotHdr hdr[kB];
    float val[kB][CAP];
    float vb[kB][CAP];      // v at the entry's id
    int32_t key[HTC];
    uint16_t pos[kB][CAP];  // index into the U array: hot id, or the block's table slot behind the hot ids
    uint16_t occ[HTC];      // occupied table slots, in insertion order
    uint16_t carry[HTC];    // slot of the same id in the previous block's table, or kNoCarry
    int32_t n_occ, cnt, slow, pad;
};

template <int CAP> struct Stage {
    int32_t idx[kB][CAP];
    float val[kB][CAP];
    uint16_t cold[kB * CAP]; // (coordinate << 8 | entry) of the staged block's cold non-zeros
    SlotHdr hdr[2][kB];      // headers of the block being built and of the next one
    int32_t cnt[2], slow[2];
    int32_t n_cold, pad;
};

template <int HOT, int HTC, int CAP> struct SharedB {
    // U_k in shared memory, one array so that the chain needs no case split: [0, HOT) the hot ids, then the cold
    // table of buffer 0, then the cold table of buffer 1
    alignas(16) float U[HOT + 2 * HTC];
    alignas(16) float red[32]; // the chain's reduction buffer
    Stage<CAP> st;
    BlockBuf<HTC, CAP> buf[2];
};

// Named hardware barriers. 1: among the helpers. 2 ("done"): the chain arrives when it has finished a block, the
// helpers wait. 3 ("full"): the helpers arrive when a block is ready, the chain waits. Blocking on a hardware
// barrier costs no issue slots and no shared-memory traffic, which matters because the chain's latency-bound loop
// shares the SM with the waiters (polling an mbarrier from 7 warps tripled the chain's step time).
__device__ __forceinline__ void helper_bar() { asm volatile("bar.sync 1, %0;" ::"n"(kHelperThreads) : "memory"); }
__device__ __forceinline__ void done_arrive() { __threadfence_block(); asm volatile("bar.arrive 2, %0;" ::"n"(kThreadsB) : "memory"); }
__device__ __forceinline__ void done_wait() { asm volatile("bar.sync 2, %0;" ::"n"(kThreadsB) : "memory"); }
__device__ __forceinline__ void full_arrive() { __threadfence_block(); asm volatile("bar.arrive 3, %0;" ::"n"(kThreadsB) : "memory"); }
__device__ __forceinline__ void full_wait() { asm volatile("bar.sync 3, %0;" ::"n"(kThreadsB) : "memory"); }

template <int HTC> __device__ __forceinline__ uint32_t hash_slot(int32_t idx)
{
    return (((uint32_t)idx * 2654435761u) >> 16) & (uint32_t)(HTC - 1);
}

// When a round spans several local epochs a coordinate can come up again before its staged header was prepared
// from its new value (even inside one block), so the chain re-reads alpha itself: lane 0 wrote it, lane 0 reads it.
template <int LOSS> __device__ __forceinline__ void refresh_state(SlotHdr &h, const float *alpha, int lane)
{
    float al = 0.0f;
    if (lane == 0) al = *reinterpret_cast<const volatile float *>(alpha + h.coord);
    al = __shfl_sync(0xffffffffu, al, 0);
    h.p1 = LOSS == CHICLE_LOSS_RIDGE_PRIMAL ? al : h.p3 * al;
}

template <int LOSS, int HOT, int HTC, int CAP>
__global__ void __launch_bounds__(kThreadsB, 1) k_local_scd_blocked(const SolverParams P)
{
    static_assert((HTC & (HTC - 1)) == 0 && HOT + 2 * HTC <= 65535 && CAP % 32 == 0 && CAP <= 256, "slot encoding");
    using Shared = SharedB<HOT, HTC, CAP>;
    using Buf = BlockBuf<HTC, CAP>;
    constexpr int kMaxOcc = HTC * 3 / 4; // distinct cold ids a block may have before it is walked unstaged
    constexpr int kChunks = CAP / 32;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    Shared &sh = *reinterpret_cast<Shared *>(smem_raw);
    const int k = blockIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    const int64_t off = P.part_off[k];
    const int64_t nk = P.part_off[k + 1] - off;
    const int64_t steps = nk <= 0 ? 0 : (P.H == 0 ? nk : P.H);
    float *Uk = P.U + (size_t)k * (size_t)P.dim;
    const int hot_n = HOT < P.dim ? HOT : (int)P.dim; // ids below hot_n live in Uhot
    for (int i = threadIdx.x; i < hot_n; i += kThreadsB) sh.U[i] = Uk[i];
    __syncthreads();
    if (steps == 0) return;
    const int64_t nblocks = (steps + kB - 1) / kB;

    if (warp == 0) {
        // =============================== the chain ===============================
        const uint32_t ubase = smem_u32(&sh.U[0]);
        const uint32_t redbuf = smem_u32(&sh.red[0]);
        for (int64_t b = 0; b < nblocks; ++b) {
            Buf &B = sh.buf[b & 1];
            full_wait();
            const int cnt = B.cnt;
            const bool staged = B.slow == 0;
            for (int j = 0; j < cnt; ++j) {
                const uint32_t hb = smem_u32(&B.hdr[j]);
                SlotHdr h;
                {
                    const int4 hi = lds_s32x4(hb);
                    const float4 hp = lds_f32x4(hb + 16);
                    h.row_start = ((int64_t)hi.y << 32) | (uint32_t)hi.x;
                    h.coord = hi.z;
                    h.nnz = hi.w;
                    h.p0 = hp.x; h.p1 = hp.y; h.p2 = hp.z; h.p3 = hp.w;
                }
                if (P.multi_epoch) refresh_state<LOSS>(h, P.alpha, lane);
                float acc = 0.0f, delta, new_state;
                if (staged) {
                    // all of the coordinate's entries in registers: the loads go out back to back
                    const uint32_t pb = smem_u32(&B.pos[j][0]) + 2u * lane;
                    const uint32_t xb = smem_u32(&B.val[j][0]) + 4u * lane;
                    const uint32_t vb = smem_u32(&B.vb[j][0]) + 4u * lane;
                    float x[kChunks], u[kChunks];
                    uint32_t ua[kChunks];
#pragma unroll
                    for (int c = 0; c < kChunks; ++c) {
                        x[c] = 0.0f;
                        u[c] = 0.0f;
                        ua[c] = 0xFFFFFFFFu;
                        if (lane + 32 * c < h.nnz) {
                            ua[c] = ubase + 4u * lds_u16(pb + 64u * c);
                            x[c] = lds_f32(xb + 128u * c);
                            const float vv = lds_f32(vb + 128u * c);
                            u[c] = lds_f32(ua[c]);
                            acc = fmaf(x[c], fmaf(P.sigma, u[c], vv), acc);
                        }
                    }
                    acc = warp_sum_smem(acc, redbuf, lane);
                    coordinate_step<LOSS>(acc, h, delta, new_state);
                    if (!(fabsf(delta) <= CUDART_MAX_NORMAL_F)) {
                        if (lane == 0) atomicOr(P.status, ST_NONFINITE_STEP);
                        delta = 0.0f;
                        new_state = LOSS == CHICLE_LOSS_RIDGE_PRIMAL ? h.p1 : h.p3 * h.p1;
                    }
                    if (delta != 0.0f) {
#pragma unroll
                        for (int c = 0; c < kChunks; ++c)
                            if (ua[c] != 0xFFFFFFFFu) sts_f32(ua[c], fmaf(delta, x[c], u[c]));
                    }
                } else {
                    // unstaged block: hot ids from shared memory, cold ids straight from global memory (current
                    // there: the helpers wrote the previous table back before handing this block over)
                    const int32_t *ix = P.indices + h.row_start;
                    const float *xv = P.values + h.row_start;
                    for (int e = lane; e < h.nnz; e += 32) {
                        const int32_t i = ix[e];
                        const float uu = i < hot_n ? sh.U[i] : Uk[i];
                        acc = fmaf(xv[e], fmaf(P.sigma, uu, P.vbase[i]), acc);
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
                            const int32_t i = ix[e];
                            if (i < hot_n) sh.U[i] = fmaf(delta, xv[e], sh.U[i]);
                            else Uk[i] = fmaf(delta, xv[e], Uk[i]);
                        }
                }
                if (lane == 0) {
                    // parked in the header and written out by the helpers, off the chain, unless the round revisits
                    // coordinates and needs it in place at once
                    if (P.multi_epoch) P.alpha[h.coord] = new_state;
                    else sts_f32(hb + 20, new_state); // the header's p1 field
                }
                __syncwarp();
            }
            __syncwarp();
            done_arrive();
        }
        // the hot part of U_k goes home
        __syncwarp();
        for (int i = lane; i < hot_n; i += 32) Uk[i] = sh.U[i];
        return;
    }

    // =============================== helpers ===============================
    const int ht = threadIdx.x - 32;     // 0 .. kHelperThreads-1
    const bool hdr_warp = ht < 32;       // helper warp 0 prepares headers, the others stage non-zeros
    const int et = ht - 32;              // index among the entry-staging threads (valid when !hdr_warp)
    const int ew = et >> 5;
    Stage<CAP> &st = sh.st;

    // Header pipeline, in registers of the header warp: the coordinate of step `lane` of block b+3 is in flight,
    // the fields of block b+2 are in flight, block b+1's fields are turned into headers during iteration b.
    auto coord_of = [&](int64_t blk) -> int32_t {
        const int64_t t = blk * kB + lane;
        if (blk >= nblocks || t >= steps) return -1;
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
    // header warp only: block `blk`'s headers and counters into staging slot blk & 1
    auto stage_headers = [&](int64_t blk, const Fields &f) {
        const int q = (int)(blk & 1);
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
            hd.pad[0] = hd.pad[1] = hd.pad[2] = hd.pad[3] = 0;
            st.hdr[q][lane] = hd;
        }
        const bool too_long = __any_sync(0xffffffffu, nnz > CAP);
        if (lane == 0) {
            st.cnt[q] = cnt;
            st.slow[q] = too_long ? 1 : 0;
        }
    };
    // entry warps only: cp.async of block `blk`'s non-zeros into the staging area
    auto issue_entries = [&](int64_t blk) {
        const int q = (int)(blk & 1);
        if (st.slow[q]) return;
        for (int j = ew; j < st.cnt[q]; j += kEntryWarps) {
            const int nnz = st.hdr[q][j].nnz;
            const int64_t rs = st.hdr[q][j].row_start;
            for (int e = lane; e < nnz; e += 32) {
                cp_async4(smem_u32(&st.idx[j][e]), P.indices + rs + e);
                cp_async4(smem_u32(&st.val[j][e]), P.values + rs + e);
            }
        }
    };

    // ---- prologue: block 0 staged, block 1 fields and block 2 coordinates in flight
    Fields f_next{-1, 0, 0, 0.f, 0.f, 0.f}, f_far{-1, 0, 0, 0.f, 0.f, 0.f};
    int32_t c_far = -1;
    if (hdr_warp) {
        const Fields f0 = issue_fields(coord_of(0));
        f_next = issue_fields(coord_of(1));
        f_far = issue_fields(coord_of(2));
        c_far = coord_of(3);
        stage_headers(0, f0);
    }
    helper_bar();
    if (!hdr_warp) issue_entries(0);

    const uint32_t lt_mask = (1u << lane) - 1u;
    for (int64_t b = 0; b < nblocks; ++b) {
        const int q = (int)(b & 1);
        Buf &B = sh.buf[q];
        Buf &Prev = sh.buf[q ^ 1];
        float *Tu = sh.U + HOT + q * HTC;          // this block's cold table values
        float *TuPrev = sh.U + HOT + (q ^ 1) * HTC; // the previous block's
        const bool have_prev = b > 0;
        // ---- S0: reset this buffer's table (its previous block was written back in the last iteration)
        for (int p = ht; p < HTC; p += kHelperThreads) B.key[p] = -1;
        if (ht == 0) {
            B.n_occ = 0;
            st.n_cold = 0;
        }
        cp_async_wait_all();
        helper_bar(); // the staging area holds block b's non-zeros; its headers are in st.hdr[q]
        const int cnt = st.cnt[q];
        bool slow = st.slow[q] != 0;
        const bool prev_slow = have_prev && Prev.slow != 0;
        // cold ids that are not in the previous table may be fetched from global memory now, unless the chain is
        // writing global memory itself (previous block unstaged)
        const bool early_ok = !prev_slow;
        if (hdr_warp) {
            // ---- the header warp advances the header pipeline while the others build the table
            if (lane < cnt) B.hdr[lane] = st.hdr[q][lane];
            if (b + 1 < nblocks) stage_headers(b + 1, f_next);
            f_next = f_far;
            f_far = issue_fields(c_far);
            c_far = coord_of(b + 4);
        } else if (!slow) {
            // ---- S3a: classify. An entry warp takes whole coordinates, lanes over the non-zeros: copy the value,
            //      start the gather of v, give hot ids their slot, collect cold ones in a list.
            for (int j = ew; j < cnt; j += kEntryWarps) {
                const int nnz = st.hdr[q][j].nnz;
                for (int e0 = 0; e0 < nnz; e0 += 32) {
                    const int e = e0 + lane;
                    bool cold = false;
                    if (e < nnz) {
                        const int32_t idx = st.idx[j][e];
                        B.val[j][e] = st.val[j][e];
                        cp_async4(smem_u32(&B.vb[j][e]), P.vbase + idx);
                        if (HOT > 0 && idx < HOT) B.pos[j][e] = (uint16_t)idx;
                        else cold = true;
                    }
                    const uint32_t m = __ballot_sync(0xffffffffu, cold);
                    if (m) {
                        const int leader = __ffs(m) - 1;
                        int base = 0;
                        if (lane == leader) base = atomicAdd(&st.n_cold, __popc(m));
                        base = __shfl_sync(0xffffffffu, base, leader);
                        if (cold) st.cold[base + __popc(m & lt_mask)] = (uint16_t)((j << 8) | e);
                    }
                }
            }
        }
        helper_bar(); // cold list complete; headers of block b+1 staged
        if (!hdr_warp && !slow) {
            // ---- S3b: hash the cold non-zeros, one per thread and pass
            const int n_cold = st.n_cold;
            for (int i0 = 0; i0 < n_cold; i0 += kEntryThreads) {
                const int i = i0 + et;
                bool is_new = false;
                uint32_t p = 0;
                if (i < n_cold) {
                    const uint32_t je = st.cold[i];
                    const int j = je >> 8, e = je & 255;
                    const int32_t idx = st.idx[j][e];
                    p = hash_slot<HTC>(idx);
                    bool placed = false;
                    if (B.n_occ <= kMaxOcc) {
                        for (int probe = 0; probe < HTC; ++probe) {
                            // a plain read settles most probes; only an empty slot needs the compare-and-swap
                            int32_t seen = *reinterpret_cast<volatile int32_t *>(&B.key[p]);
                            if (seen == -1) seen = atomicCAS(&B.key[p], -1, idx);
                            if (seen == -1) { is_new = true; placed = true; break; }
                            if (seen == idx) { placed = true; break; }
                            p = (p + 1) & (HTC - 1);
                        }
                    }
                    if (!placed) { B.slow = 2; p = 0; } // over-full: the block will be walked unstaged
                    B.pos[j][e] = (uint16_t)(HOT + q * HTC + p);
                }
                const uint32_t m = __ballot_sync(0xffffffffu, is_new);
                if (m) {
                    const int leader = __ffs(m) - 1;
                    int slot = 0;
                    if (lane == leader) slot = atomicAdd(&B.n_occ, __popc(m));
                    slot = __shfl_sync(0xffffffffu, slot, leader) + __popc(m & lt_mask);
                    if (is_new) B.occ[slot & (HTC - 1)] = (uint16_t)p;
                }
            }
        }
        helper_bar(); // all slots known
        if (!slow && (B.slow == 2 || B.n_occ > kMaxOcc)) slow = true;
        if (!slow) {
            // ---- S3c: per distinct cold id, look it up in the previous table and fetch U_k if it is final
            const int n_occ = B.n_occ;
            for (int i = ht; i < n_occ; i += kHelperThreads) {
                const uint32_t p = B.occ[i];
                const int32_t idx = B.key[p];
                uint16_t cp = kNoCarry;
                if (have_prev && !prev_slow) {
                    uint32_t r = hash_slot<HTC>(idx);
                    for (int probe = 0; probe < HTC; ++probe) {
                        const int32_t kr = Prev.key[r];
                        if (kr == idx) { cp = (uint16_t)r; break; }
                        if (kr == -1) break;
                        r = (r + 1) & (HTC - 1);
                    }
                }
                B.carry[p] = cp;
                // U_k is only ever written by this SM, so a cached copy cannot be stale
                if (cp == kNoCarry && early_ok) cp_async4(smem_u32(&Tu[p]), Uk + idx);
            }
        }
        cp_async_wait_all(); // v gathers and early U_k fetches have landed
        helper_bar();        // table built, staging area free
        // ---- S5: non-zeros of block b+1 into the staging area
        if (!hdr_warp && b + 1 < nblocks) issue_entries(b + 1);
        // ---- S6: the chain must have finished block b-1 before its table is read
        if (have_prev) done_wait();
        const bool write_back_first = have_prev && !prev_slow && slow; // an unstaged block reads global memory
        if (write_back_first) {
            for (int i = ht; i < Prev.n_occ; i += kHelperThreads) {
                const int p = Prev.occ[i];
                Uk[Prev.key[p]] = TuPrev[p];
            }
        }
        // ---- S7: complete the table: carried slots from the previous table, late fetches
        if (!slow) {
            const int n_occ = B.n_occ;
            for (int base = 0; base < n_occ; base += 4 * kHelperThreads) {
                uint32_t pp[4];
                uint16_t cc[4];
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    const int i = base + r * kHelperThreads + ht;
                    pp[r] = i < n_occ ? B.occ[i] : HTC;
                }
#pragma unroll
                for (int r = 0; r < 4; ++r) cc[r] = pp[r] < HTC ? B.carry[pp[r]] : kNoCarry;
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    if (cc[r] != kNoCarry) Tu[pp[r]] = TuPrev[cc[r]];
                    else if (!early_ok && pp[r] < HTC) Tu[pp[r]] = __ldcg(Uk + B.key[pp[r]]);
                }
            }
        }
        if (ht == 0) {
            B.cnt = cnt;
            B.slow = slow ? 1 : 0;
        }
        full_arrive(); // block b is ready (every helper's writes are ordered before its arrival)
        // ---- the previous block's results go back to global memory, off the chain's critical path
        if (have_prev && !P.multi_epoch && ht < Prev.cnt) P.alpha[Prev.hdr[ht].coord] = Prev.hdr[ht].p1;
        if (have_prev && !prev_slow && !write_back_first) {
            for (int i = ht; i < Prev.n_occ; i += kHelperThreads) {
                const int p = Prev.occ[i];
                Uk[Prev.key[p]] = TuPrev[p];
            }
        }
        helper_bar(); // the previous buffer may be rebuilt, and its global values are in place
    }
    // ---- epilogue: the last block's results
    {
        const int64_t b = nblocks - 1;
        Buf &L = sh.buf[b & 1];
        done_wait();
        if (!P.multi_epoch && ht < L.cnt) P.alpha[L.hdr[ht].coord] = L.hdr[ht].p1;
        if (!L.slow)
            for (int i = ht; i < L.n_occ; i += kHelperThreads) {
                const int p = L.occ[i];
                Uk[L.key[p]] = sh.U[HOT + (b & 1) * HTC + p];
            }
    }
}

template <int LOSS, int HOT, int HTC, int CAP> cudaError_t launch_one(Glm &g, const SolverParams &P)
{
    using Shared = SharedB<HOT, HTC, CAP>;
    static_assert(sizeof(Shared) <= 227 * 1024, "shared memory budget");
    auto kern = k_local_scd_blocked<LOSS, HOT, HTC, CAP>;
    const size_t smem = sizeof(Shared);
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kern<<<g.K, kThreadsB, smem, g.stream>>>(P);
    return cudaGetLastError();
}

// skewed ids (most non-zeros fall on a few thousand ids): a large direct array and a small table
constexpr int kHotA = 24576, kHtcA = 1024, kCapA = 96;
// flat ids: no direct array, everything through the table
constexpr int kHotB = 0, kHtcB = 4096, kCapB = 128;

template <int LOSS> cudaError_t launch_loss(Glm &g, const SolverParams &P)
{
    if (g.hot_variant) return launch_one<LOSS, kHotA, kHtcA, kCapA>(g, P);
    return launch_one<LOSS, kHotB, kHtcB, kCapB>(g, P);
}

} // namespace

int blocked_solver_hot_ids() { return kHotA; }

cudaError_t launch_blocked_solver(Glm &g, const SolverParams &P)
{
    switch (g.loss) {
    case CHICLE_LOSS_HINGE_DUAL: return launch_loss<CHICLE_LOSS_HINGE_DUAL>(g, P);
    case CHICLE_LOSS_LOGISTIC_DUAL: return launch_loss<CHICLE_LOSS_LOGISTIC_DUAL>(g, P);
    default: return launch_loss<CHICLE_LOSS_RIDGE_PRIMAL>(g, P);
    }
}

} // namespace chicle
