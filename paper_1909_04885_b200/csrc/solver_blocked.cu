// Local SCD solver for sparse coordinates (CSR rows / CSC columns) and for short dense rows: one CTA per partition, the visiting order
// walked strictly in order (paper Sec. 2.2 worker structure with L = 1; Sec. 5.1: SCD local solver), with the
// part of the local model that the next steps can touch held in shared memory.
//
// Local model: w_local = v + sigma' * U_k, where U_k (the partition's accumulated update, zero at round start) has
// its home in row k of the K x dim workspace in global memory. Shared memory holds w_local itself at the entries
// that matter, so a step is one gather, one reduction, the scalar step and one scatter (w_local += sigma' delta x);
// U_k is recovered as (w_local - v) / sigma' when an entry leaves shared memory. Entry ids are frequency-ranked when
// the problem is created (id 0 is the most frequent feature), which gives two places for the live part:
//   hot   ids below HOT: a direct array for the whole kernel (no look-up at all);
//   cold  the remaining ids: the walk is cut into blocks of kB consecutive steps and, per block, the helper warps
//         build a small open-addressing hash table over the block's distinct cold ids.
// Every staged non-zero carries its value and a 16-bit index into the shared array (hot id, or table slot).
//
// A cold slot's value comes from the previous block's table when that block touches the id too ("carried": copied
// shared-to-shared once the chain has finished the previous block) and from global memory otherwise, fetched early
// while the chain is still busy (the id is not in the previous block, so its global value is final: older blocks
// were written back before). A finished block's table goes back to global memory off the critical path, and so do
// the new alpha values, which the chain parks in the block's headers. The result equals walking the coordinates
// one by one against a full copy of the local model, up to rounding.
//
// The chain warp's loop is latency-bound and shares the SM with the helpers, and measurements showed that what
// slows it is load/store-unit traffic from the other warps (4-byte cp.async or plain global loads at a high rate
// made a step five times slower), not their arithmetic or their shared-memory atomics. Hence: the non-zeros of a
// coordinate arrive by bulk copies of the copy engine (16-byte aligned windows around the coordinate, one
// instruction per array), v is folded into the shared array instead of being gathered per non-zero, the roles hand
// blocks over through named hardware barriers (no polling), and the chain uses explicit 32-bit shared addresses.
//
// Staging runs three blocks deep: visiting-order entries three blocks ahead, per-coordinate fields two blocks
// ahead (one helper warp does nothing else), non-zeros one block ahead. A block that does not fit (a coordinate
// longer than CAP, too many distinct cold ids) is walked by the chain against global memory for its cold ids.
// Every role runs the same number of blocks and leaves only at the end, so each barrier always gets its full count;
// the one polled wait (for the bulk copies) is bounded.
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
    int32_t key[HTC];       // cold id in a table slot, -1 = empty
    float Tv[HTC];          // v at that id (to turn w_local back into U_k)
    uint16_t pos[kB][CAP];  // index into the W array: hot id, or this buffer's table slot behind the hot ids
    uint16_t occ[HTC];      // occupied table slots, in insertion order
    uint16_t carry[HTC];    // slot of the same id in the previous block's table, or kNoCarry
    int32_t n_occ, cnt, slow, pad;
};

template <int CAP> struct Stage {
    // Rows are 16-byte aligned windows of the global arrays: coordinate j's entry e sits at [j][shift[j] + e].
    alignas(16) int32_t idx[kB][CAP + 4];
    alignas(16) float val[kB][CAP + 4];
    alignas(8) uint64_t bar;  // counts the bytes of the bulk copies of the block being staged
    uint16_t cold[kB * CAP];  // (coordinate << 8 | entry) of the staged block's cold non-zeros
    SlotHdr hdr[2][kB];       // headers of the block being built and of the next one
    int32_t shift[2][kB];
    int32_t cnt[2], slow[2];
    int32_t n_cold, abort_flag;
};

template <int HOT, int HTC, int CAP> struct SharedB {
    // w_local in shared memory, one array so that the chain needs no case split: [0, HOT) the hot ids, then the
    // cold table of buffer 0, then the cold table of buffer 1
    alignas(16) float W[HOT + 2 * HTC + 32]; // + one dummy word per chain lane (always 0)
    alignas(16) float red[32]; // the chain's reduction buffer
    Stage<CAP> st;
    BlockBuf<HTC, CAP> buf[2];
};

// Named hardware barriers. 1: among the helpers. 2 ("done"): the chain arrives when it has finished a block, the
// helpers wait. 3 ("full"): the helpers arrive when a block is ready, the chain waits. Blocking on a hardware
// barrier costs no issue slots and no shared-memory traffic.
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

// What the chain keeps in registers for one step: header fields, and per 32-lane chunk of the coordinate this
// lane's value and the shared address of its w_local word (the lane's dummy word beyond the coordinate's length).
template <int CHUNKS> struct StepRegs {
    float4 p;
    int32_t coord, nnz;
    float x[CHUNKS];
    uint32_t wa[CHUNKS];
};

// The loads of a step's header, slots and values, as issued (nothing here waits for a result) ...
template <int CHUNKS> struct StepRaw {
    int4 hi;
    float4 p;
    uint32_t s[CHUNKS];
    float x[CHUNKS];
};
template <int CHUNKS, int CAP, bool DENSE>
__device__ __forceinline__ void issue_step(StepRaw<CHUNKS> &r, int j, uint32_t hdr0, uint32_t pos0, uint32_t val0, int lane)
{
    const uint32_t hb = hdr0 + 48u * j;
    r.hi = lds_s32x4(hb);
    r.p = lds_f32x4(hb + 16);
    const uint32_t pb = pos0 + (uint32_t)(2 * CAP) * j, xb = val0 + (uint32_t)(4 * CAP) * j;
#pragma unroll
    for (int c = 0; c < CHUNKS; ++c) {
        // dense rows: entry e of a row is simply id e; otherwise the staged slot (always a valid shared address to
        // read; the content counts only if the lane is active)
        r.s[c] = DENSE ? (uint32_t)(lane + 32 * c) : lds_u16(pb + 64u * c);
        r.x[c] = lds_f32(xb + 128u * c);
    }
}
// ... and their first use, placed where the results have long arrived.
template <int CHUNKS>
__device__ __forceinline__ void finish_step(StepRegs<CHUNKS> &r, const StepRaw<CHUNKS> &raw, uint32_t wbase, uint32_t dummy,
                                            int lane)
{
    r.p = raw.p;
    r.coord = raw.hi.z;
    r.nnz = raw.hi.w;
#pragma unroll
    for (int c = 0; c < CHUNKS; ++c) {
        const bool active = lane + 32 * c < r.nnz;
        r.wa[c] = wbase + 4u * (active ? raw.s[c] : dummy);
        r.x[c] = active ? raw.x[c] : 0.0f;
    }
}

template <int LOSS, bool DENSE, int HOT, int HTC, int CAP>
__global__ void __launch_bounds__(kThreadsB, 1) k_local_scd_blocked(const SolverParams P)
{
    static_assert((HTC & (HTC - 1)) == 0 && HOT + 2 * HTC + 32 <= 65535 && CAP % 32 == 0 && CAP <= 252, "slot encoding");
    using Shared = SharedB<HOT, HTC, CAP>;
    using Buf = BlockBuf<HTC, CAP>;
    constexpr int kMaxOcc = HTC * 3 / 4; // distinct cold ids a block may have before it is walked unstaged
    constexpr int kChunks = CAP / 32;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    Shared &sh = *reinterpret_cast<Shared *>(smem_raw);
    Stage<CAP> &st = sh.st;
    const int k = blockIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    const int64_t off = P.part_off[k];
    const int64_t nk = P.part_off[k + 1] - off;
    const int64_t steps = partition_steps(P, k, nk);
    float *Uk = P.U + (size_t)k * (size_t)P.dim;
    const int hot_n = HOT < P.dim ? HOT : (int)P.dim; // ids below hot_n live in the direct part of W
    const float inv_sigma = 1.0f / P.sigma;
    if (threadIdx.x == 0) {
        st.abort_flag = 0;
        mbar_init(smem_u32(&st.bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); // make the init visible to the copy engine
    }
    for (int i = threadIdx.x; i < hot_n; i += kThreadsB) sh.W[i] = fmaf(P.sigma, Uk[i], P.vbase[i]);
    if (threadIdx.x < 32) sh.W[HOT + 2 * HTC + threadIdx.x] = 0.0f;
    __syncthreads();
    if (steps == 0) return;
    const int64_t nblocks = (steps + kB - 1) / kB;

    if (warp == 0) {
        // =============================== the chain ===============================
        const uint32_t wbase = smem_u32(&sh.W[0]);
        const uint32_t redbuf = smem_u32(&sh.red[0]);
        const uint32_t dummy = HOT + 2 * HTC + lane; // this lane's dummy word in W
        const float sigma = P.sigma;
        for (int64_t b = 0; b < nblocks; ++b) {
            Buf &B = sh.buf[b & 1];
            full_wait();
            const int cnt = B.cnt;
            const bool staged = B.slow == 0;
            if (staged) {
                // Branch-free, software-pipelined walk: the next step's header, values and slots are loaded while
                // this step's reduction runs (they do not depend on it); lanes beyond the coordinate's length are
                // pointed at a private dummy word with value 0, so gather and scatter need no predicates.
                const uint32_t hdr0 = smem_u32(&B.hdr[0]);
                const uint32_t pos0 = smem_u32(&B.pos[0][0]) + 2u * lane;
                const uint32_t val0 = smem_u32(&B.val[0][0]) + 4u * lane;
                StepRegs<kChunks> cur;
                StepRaw<kChunks> raw;
                issue_step<kChunks, CAP, DENSE>(raw, 0, hdr0, pos0, val0, lane);
                finish_step<kChunks>(cur, raw, wbase, dummy, lane);
#pragma unroll 4 // measured: 12 % faster than the rolled loop (no register shuffling between steps)
                for (int j = 0; j < cnt; ++j) {
                    if (j + 1 < cnt) issue_step<kChunks, CAP, DENSE>(raw, j + 1, hdr0, pos0, val0, lane);
                    SlotHdr h;
                    h.row_start = 0;
                    h.coord = cur.coord;
                    h.nnz = cur.nnz;
                    h.p0 = cur.p.x; h.p1 = cur.p.y; h.p2 = cur.p.z; h.p3 = cur.p.w;
                    if (P.multi_epoch) refresh_state<LOSS>(h, P.alpha, lane);
                    float w[kChunks];
                    float acc = 0.0f, delta, new_state;
#pragma unroll
                    for (int c = 0; c < kChunks; ++c) {
                        w[c] = lds_f32(cur.wa[c]);
                        acc = fmaf(cur.x[c], w[c], acc);
                    }
                    acc = warp_sum_smem(acc, redbuf, lane);
                    coordinate_step<LOSS>(acc, h, delta, new_state);
                    // (a non-finite step is caught off the chain, when the helpers write alpha out)
                    if (delta != 0.0f) { // the same in every lane
                        const float sd = sigma * delta;
#pragma unroll
                        for (int c = 0; c < kChunks; ++c) sts_f32(cur.wa[c], fmaf(sd, cur.x[c], w[c]));
                    }
                    if (lane == 0) {
                        // parked in the header and written out by the helpers, off the chain, unless the round
                        // revisits coordinates and needs it in place at once
                        if (P.multi_epoch) P.alpha[h.coord] = new_state;
                        else sts_f32(hdr0 + 48u * j + 20u, new_state); // the header's p1 field
                    }
                    __syncwarp();
                    finish_step<kChunks>(cur, raw, wbase, dummy, lane);
                }
            } else {
                // unstaged block: hot ids from shared memory, cold ids straight from global memory (current there:
                // the helpers wrote the previous table back before handing this block over)
                for (int j = 0; j < cnt; ++j) {
                    SlotHdr h = B.hdr[j];
                    if (P.multi_epoch) refresh_state<LOSS>(h, P.alpha, lane);
                    float acc = 0.0f, delta, new_state;
                    const int32_t *ix = P.indices + h.row_start;
                    const float *xv = P.values + h.row_start;
                    for (int e = lane; e < h.nnz; e += 32) {
                        const int32_t i = DENSE ? e : ix[e];
                        const float ww = i < hot_n ? sh.W[i] : fmaf(sigma, Uk[i], P.vbase[i]);
                        acc = fmaf(xv[e], ww, acc);
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
                            const int32_t i = DENSE ? e : ix[e];
                            if (i < hot_n) sh.W[i] = fmaf(sigma * delta, xv[e], sh.W[i]);
                            else Uk[i] = fmaf(delta, xv[e], Uk[i]);
                        }
                    if (lane == 0) {
                        if (P.multi_epoch) P.alpha[h.coord] = new_state;
                        else B.hdr[j].p1 = new_state;
                    }
                    __syncwarp();
                }
            }
            __syncwarp();
            done_arrive();
        }
        return;
    }

    // =============================== helpers ===============================
    const int ht = threadIdx.x - 32;     // 0 .. kHelperThreads-1
    const bool hdr_warp = ht < 32;       // helper warp 0 prepares headers, the others stage non-zeros
    const int et = ht - 32;              // index among the entry-staging threads (valid when !hdr_warp)
    const int ew = et >> 5;
    volatile int *abort_flag = &st.abort_flag;

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
            if (DENSE) {
                f.rs = (int64_t)c * P.dim;
                f.re = f.rs + P.dim;
            } else {
                f.rs = P.indptr[c];
                f.re = P.indptr[c + 1];
            }
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
            st.shift[q][lane] = (int32_t)(f.rs & 3);
        }
        const bool too_long = __any_sync(0xffffffffu, nnz > CAP);
        if (lane == 0) {
            st.cnt[q] = cnt;
            st.slow[q] = too_long ? 1 : 0;
        }
        return too_long;
    };
    // header warp only: lane j starts the two bulk copies of coordinate j of the block whose fields are `f`
    // (16-byte aligned windows: up to 3 elements before the coordinate and up to 3 behind it come along)
    auto issue_entries = [&](const Fields &f, bool too_long) {
        if (too_long) return;
        uint32_t bytes = 0;
        int64_t first = 0;
        if (f.c >= 0 && f.re > f.rs) {
            first = f.rs & ~(int64_t)3;
            bytes = (uint32_t)(((f.re - first) + 3) & ~(int64_t)3) * 4u;
        }
        uint32_t total = DENSE ? bytes : 2u * bytes;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) total += __shfl_xor_sync(0xffffffffu, total, o);
        const uint32_t bar = smem_u32(&st.bar);
        if (lane == 0) mbar_arrive_expect_tx(bar, total);
        __syncwarp();
        if (bytes) {
            if (!DENSE) bulk_g2s(smem_u32(&st.idx[lane][0]), P.indices + first, bytes, bar);
            bulk_g2s(smem_u32(&st.val[lane][0]), P.values + first, bytes, bar);
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
        const bool too_long = stage_headers(0, f0);
        issue_entries(f0, too_long);
    }
    helper_bar();

    const uint32_t lt_mask = (1u << lane) - 1u;
    uint32_t n_staged = 0; // blocks whose non-zeros came through the bulk-copy barrier so far (its phase counter)
    for (int64_t b = 0; b < nblocks; ++b) {
        const int q = (int)(b & 1);
        Buf &B = sh.buf[q];
        Buf &Prev = sh.buf[q ^ 1];
        float *Tw = sh.W + HOT + q * HTC;          // this block's cold table: w_local at the slot's id
        float *TwPrev = sh.W + HOT + (q ^ 1) * HTC; // the previous block's
        const bool have_prev = b > 0;
        // ---- S0: reset this buffer's table (its previous block was written back in the last iteration)
        // (the helpers' loops use explicit shared addresses too: generic accesses cost them several times more)
        const uint32_t a_key = smem_u32(&B.key[0]), a_occ = smem_u32(&B.occ[0]), a_carry = smem_u32(&B.carry[0]);
        const uint32_t a_tv = smem_u32(&B.Tv[0]), a_tw = smem_u32(Tw), a_twp = smem_u32(TwPrev);
        const uint32_t a_keyp = smem_u32(&Prev.key[0]);
        const uint32_t a_bval = smem_u32(&B.val[0][0]), a_bpos = smem_u32(&B.pos[0][0]);
        const uint32_t a_sidx = smem_u32(&st.idx[0][0]), a_sval = smem_u32(&st.val[0][0]);
        const uint32_t a_cold = smem_u32(&st.cold[0]), a_ncold = smem_u32(&st.n_cold), a_nocc = smem_u32(&B.n_occ);
        const uint32_t a_hdrq = smem_u32(&st.hdr[q][0]), a_shiftq = smem_u32(&st.shift[q][0]);
        constexpr uint32_t kStageRow = (CAP + 4) * 4; // bytes per staged coordinate
        for (int p = ht; p < HTC; p += kHelperThreads) sts_s32(a_key + 4u * p, -1);
        if (ht == 0) {
            B.n_occ = 0;
            st.n_cold = 0;
        }
        const int cnt = st.cnt[q];
        bool slow = st.slow[q] != 0;
        if (!slow) {
            // the bulk copies of block b must have landed (bounded wait; lane 0 of each warp polls)
            if (!mbar_wait(smem_u32(&st.bar), n_staged & 1u, abort_flag, P.status)) slow = true;
            ++n_staged;
        }
        helper_bar(); // the staging area holds block b's non-zeros; its headers are in st.hdr[q]
        if (*abort_flag) slow = true; // copies that never landed: walk the block unstaged (the status word has it)
        const bool prev_slow = have_prev && Prev.slow != 0;
        // cold ids that are not in the previous table may be fetched from global memory now, unless the chain is
        // writing global memory itself (previous block unstaged)
        const bool early_ok = !prev_slow;
        bool next_too_long = false;
        Fields f_issue{-1, 0, 0, 0.f, 0.f, 0.f};
        if (hdr_warp) {
            // ---- the header warp advances the header pipeline while the others build the table
            if (lane < cnt) B.hdr[lane] = st.hdr[q][lane];
            f_issue = f_next;
            if (b + 1 < nblocks) next_too_long = stage_headers(b + 1, f_next);
            f_next = f_far;
            f_far = issue_fields(c_far);
            c_far = coord_of(b + 4);
        } else if (!slow) {
            // ---- S3a: classify. An entry warp takes whole coordinates, lanes over the non-zeros: copy the value,
            //      give hot ids their index, collect cold ones in a list.
            for (int j = ew; j < cnt; j += kEntryWarps) {
                const int nnz = lds_s32(a_hdrq + 48u * j + 12u);
                const int sft = lds_s32(a_shiftq + 4u * j);
                const uint32_t srow = kStageRow * j + 4u * sft;
                for (int e0 = 0; e0 < nnz; e0 += 32) {
                    const int e = e0 + lane;
                    bool cold = false;
                    if (e < nnz) {
                        sts_f32(a_bval + (uint32_t)(4 * CAP) * j + 4u * e, lds_f32(a_sval + srow + 4u * e));
                        if (!DENSE) {
                            const int32_t idx = lds_s32(a_sidx + srow + 4u * e);
                            if (HOT > 0 && idx < HOT) sts_u16(a_bpos + (uint32_t)(2 * CAP) * j + 2u * e, (uint32_t)idx);
                            else cold = true;
                        }
                    }
                    const uint32_t m = __ballot_sync(0xffffffffu, cold);
                    if (m) {
                        const int leader = __ffs(m) - 1;
                        int base = 0;
                        if (lane == leader) base = atoms_add(a_ncold, __popc(m));
                        base = __shfl_sync(0xffffffffu, base, leader);
                        if (cold) sts_u16(a_cold + 2u * (base + __popc(m & lt_mask)), (uint32_t)((j << 8) | e));
                    }
                }
            }
        }
        helper_bar(); // cold list complete; headers of block b+1 staged
        if (!hdr_warp && !slow) {
            // ---- S3b: hash the cold non-zeros, one per thread and pass
            const int n_cold = lds_s32(a_ncold);
            for (int i0 = 0; i0 < n_cold; i0 += kEntryThreads) {
                const int i = i0 + et;
                bool is_new = false;
                uint32_t p = 0;
                if (i < n_cold) {
                    const uint32_t je = lds_u16(a_cold + 2u * i);
                    const int j = je >> 8, e = je & 255;
                    const int32_t idx = lds_s32(a_sidx + kStageRow * j + 4u * (lds_s32(a_shiftq + 4u * j) + e));
                    p = hash_slot<HTC>(idx);
                    bool placed = false;
                    if (lds_s32(a_nocc) <= kMaxOcc) {
                        for (int probe = 0; probe < HTC; ++probe) {
                            // a plain read settles most probes; only an empty slot needs the compare-and-swap
                            int32_t seen = lds_s32(a_key + 4u * p);
                            if (seen == -1) seen = atoms_cas(a_key + 4u * p, -1, idx);
                            if (seen == -1) { is_new = true; placed = true; break; }
                            if (seen == idx) { placed = true; break; }
                            p = (p + 1) & (HTC - 1);
                        }
                    }
                    if (!placed) { B.slow = 2; p = 0; } // over-full: the block will be walked unstaged
                    sts_u16(a_bpos + (uint32_t)(2 * CAP) * j + 2u * e, (uint32_t)(HOT + q * HTC + p));
                }
                const uint32_t m = __ballot_sync(0xffffffffu, is_new);
                if (m) {
                    const int leader = __ffs(m) - 1;
                    int slot = 0;
                    if (lane == leader) slot = atoms_add(a_nocc, __popc(m));
                    slot = __shfl_sync(0xffffffffu, slot, leader) + __popc(m & lt_mask);
                    if (is_new) sts_u16(a_occ + 2u * (slot & (HTC - 1)), p);
                }
            }
        }
        helper_bar(); // all slots known; the staging area is free
        // ---- S5: the header warp starts the bulk copies of block b+1 (its fields are in f_issue)
        if (hdr_warp && b + 1 < nblocks) issue_entries(f_issue, next_too_long);
        if (!slow && (B.slow == 2 || B.n_occ > kMaxOcc)) slow = true;
        if (!slow) {
            // ---- S3c: per distinct cold id: v, a look-up in the previous table, and w_local if U_k is final
            const int n_occ = lds_s32(a_nocc);
            for (int base = 0; base < n_occ; base += 2 * kHelperThreads) {
                uint32_t pp[2];
                float vv[2], uu[2];
                bool fetch[2];
#pragma unroll
                for (int r = 0; r < 2; ++r) {
                    const int i = base + r * kHelperThreads + ht;
                    pp[r] = HTC;
                    fetch[r] = false;
                    vv[r] = uu[r] = 0.0f;
                    if (i >= n_occ) continue;
                    const uint32_t p = lds_u16(a_occ + 2u * i);
                    const int32_t idx = lds_s32(a_key + 4u * p);
                    uint32_t cp = kNoCarry;
                    if (have_prev && !prev_slow) {
                        uint32_t r2 = hash_slot<HTC>(idx);
                        for (int probe = 0; probe < HTC; ++probe) {
                            const int32_t kr = lds_s32(a_keyp + 4u * r2);
                            if (kr == idx) { cp = r2; break; }
                            if (kr == -1) break;
                            r2 = (r2 + 1) & (HTC - 1);
                        }
                    }
                    sts_u16(a_carry + 2u * p, cp);
                    pp[r] = p;
                    vv[r] = P.vbase[idx];
                    fetch[r] = cp == kNoCarry && early_ok;
                    if (fetch[r]) uu[r] = Uk[idx]; // only this SM writes U_k, so a cached copy cannot be stale
                }
#pragma unroll
                for (int r = 0; r < 2; ++r)
                    if (pp[r] < HTC) {
                        sts_f32(a_tv + 4u * pp[r], vv[r]);
                        if (fetch[r]) sts_f32(a_tw + 4u * pp[r], fmaf(P.sigma, uu[r], vv[r]));
                    }
            }
        }
        // ---- S6: the chain must have finished block b-1 before its table is read
        if (have_prev) done_wait();
        else helper_bar();
        const bool write_back_first = have_prev && !prev_slow && slow; // an unstaged block reads global memory
        if (write_back_first) {
            for (int i = ht; i < Prev.n_occ; i += kHelperThreads) {
                const int p = Prev.occ[i];
                Uk[Prev.key[p]] = (TwPrev[p] - Prev.Tv[p]) * inv_sigma;
            }
        }
        // ---- S7: complete the table: carried slots from the previous table, late fetches
        if (!slow) {
            const int n_occ = lds_s32(a_nocc);
            for (int base = 0; base < n_occ; base += 4 * kHelperThreads) {
                uint32_t pp[4], cc[4];
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    const int i = base + r * kHelperThreads + ht;
                    pp[r] = i < n_occ ? lds_u16(a_occ + 2u * i) : HTC;
                }
#pragma unroll
                for (int r = 0; r < 4; ++r) cc[r] = pp[r] < HTC ? lds_u16(a_carry + 2u * pp[r]) : kNoCarry;
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    if (cc[r] != kNoCarry) sts_f32(a_tw + 4u * pp[r], lds_f32(a_twp + 4u * cc[r]));
                    else if (!early_ok && pp[r] < HTC)
                        sts_f32(a_tw + 4u * pp[r], fmaf(P.sigma, __ldcg(Uk + lds_s32(a_key + 4u * pp[r])), lds_f32(a_tv + 4u * pp[r])));
                }
            }
        }
        if (ht == 0) {
            B.cnt = cnt;
            B.slow = slow ? 1 : 0;
        }
        full_arrive(); // block b is ready (every helper's writes are ordered before its arrival)
        // ---- the previous block's results go back to global memory, off the chain's critical path
        if (have_prev && !P.multi_epoch && ht < Prev.cnt) {
            const float a_new = Prev.hdr[ht].p1;
            if (!(fabsf(a_new) <= CUDART_MAX_NORMAL_F)) atomicOr(P.status, ST_NONFINITE_STEP);
            P.alpha[Prev.hdr[ht].coord] = a_new;
        }
        if (have_prev && !prev_slow && !write_back_first) {
            for (int i = ht; i < Prev.n_occ; i += kHelperThreads) {
                const int p = Prev.occ[i];
                Uk[Prev.key[p]] = (TwPrev[p] - Prev.Tv[p]) * inv_sigma;
            }
        }
        helper_bar(); // the previous buffer may be rebuilt, and its global values are in place
    }
    // ---- epilogue: the last block's results and the hot ids
    {
        const int64_t b = nblocks - 1;
        Buf &L = sh.buf[b & 1];
        const float *TwL = sh.W + HOT + (b & 1) * HTC;
        done_wait();
        if (!P.multi_epoch && ht < L.cnt) {
            const float a_new = L.hdr[ht].p1;
            if (!(fabsf(a_new) <= CUDART_MAX_NORMAL_F)) atomicOr(P.status, ST_NONFINITE_STEP);
            P.alpha[L.hdr[ht].coord] = a_new;
        }
        if (!L.slow)
            for (int i = ht; i < L.n_occ; i += kHelperThreads) {
                const int p = L.occ[i];
                Uk[L.key[p]] = (TwL[p] - L.Tv[p]) * inv_sigma;
            }
        for (int i = ht; i < hot_n; i += kHelperThreads) Uk[i] = (sh.W[i] - P.vbase[i]) * inv_sigma;
    }
}

template <int LOSS, bool DENSE, int HOT, int HTC, int CAP> cudaError_t launch_one(Glm &g, const SolverParams &P)
{
    using Shared = SharedB<HOT, HTC, CAP>;
    static_assert(sizeof(Shared) <= 227 * 1024, "shared memory budget");
    auto kern = k_local_scd_blocked<LOSS, DENSE, HOT, HTC, CAP>;
    const size_t smem = sizeof(Shared);
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kern<<<g.K, kThreadsB, smem, g.stream>>>(P);
    return cudaGetLastError();
}

// skewed ids (most non-zeros fall on a few thousand ids): a large direct array and a small table
constexpr int kHotA = 24576, kHtcA = 1024, kCapA = 96;
// the same for data whose coordinates are often longer than 96 entries: a smaller direct array buys room for them
constexpr int kHotA2 = 20480, kHtcA2 = 1024, kCapA2 = 128;
// flat ids: no direct array, everything through the table
constexpr int kHotB = 0, kHtcB = 4096, kCapB = 128;
// short dense rows: entry e of every row is id e, all of w_local is "hot", no table
constexpr int kHotD = 128, kHtcD = 32, kCapD = 128;

template <int LOSS> cudaError_t launch_loss(Glm &g, const SolverParams &P)
{
    if (g.fmt == CHICLE_FMT_DENSE_ROWMAJOR) return launch_one<LOSS, true, kHotD, kHtcD, kCapD>(g, P);
    if (g.hot_variant == 1) return launch_one<LOSS, false, kHotA, kHtcA, kCapA>(g, P);
    if (g.hot_variant == 2) return launch_one<LOSS, false, kHotA2, kHtcA2, kCapA2>(g, P);
    return launch_one<LOSS, false, kHotB, kHtcB, kCapB>(g, P);
}

} // namespace

int blocked_solver_hot_ids() { return kHotA; }
int blocked_solver_short_cap() { return kCapA; }
int blocked_solver_max_dense_dim() { return kCapD; }

cudaError_t launch_blocked_solver(Glm &g, const SolverParams &P)
{
    switch (g.loss) {
    case CHICLE_LOSS_HINGE_DUAL: return launch_loss<CHICLE_LOSS_HINGE_DUAL>(g, P);
    case CHICLE_LOSS_LOGISTIC_DUAL: return launch_loss<CHICLE_LOSS_LOGISTIC_DUAL>(g, P);
    default: return launch_loss<CHICLE_LOSS_RIDGE_PRIMAL>(g, P);
    }
}

} // namespace chicle
