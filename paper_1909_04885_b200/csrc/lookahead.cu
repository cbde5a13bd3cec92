// Local SCD solver with block look-ahead: the same result as walking a partition's visiting order coordinate by
// coordinate (paper Sec. 2.2 worker structure with L = 1; Sec. 5.1: SCD local solver), up to rounding order, with
// the work that does not depend on earlier steps taken off the sequential chain.
//
// The walk is cut into blocks of 32 consecutive steps. Inside a block, with w the local model at the block's start,
//     dot_j = x_j . w + sigma' * sum_{l < j} delta_l * (x_j . x_l),
// so once the 32 dot products against w and the strictly lower triangle of the block's Gram matrix G_jl = x_j . x_l
// are known, the 32 steps are a scalar recurrence run by one warp: a step costs the scalar map and a few fused
// multiply-adds, plus one shuffle per coordinate to hand the results round. The block then applies
// w += sigma' * sum_j delta_j x_j in parallel. Which coordinates meet in a block is fixed by the visiting order
// alone, not by the model, so everything structural is prepared for all blocks of all partitions at once by a
// throughput kernel that uses the whole GPU, and the latency-bound kernel (one CTA per partition) only consumes it.
//
//   k_lookahead_prepare   one CTA per block. Writes the block's record, one contiguous piece of memory: per-step
//                         headers (coordinate, constants of the scalar step), the scaled Gram triangle, the block's
//                         non-zeros packed row after row, and, for the entry ids that several coordinates of the
//                         block share, the transposed view ("which non-zeros touch id i": one list per shared id,
//                         in ascending coordinate order). An id that only one coordinate has is updated straight
//                         from that coordinate's row; a shared id by a few threads that add up its list in a fixed
//                         order: no atomics on the model, the same bits every run. Built with a shared-memory hash
//                         table whose slots carry a 32-bit membership mask; a non-zero's place in its list is the
//                         number of lower mask bits, so the lists need no sort and come out the same whatever order
//                         the threads ran in.
//   k_lookahead_chain     one CTA per partition, 16 warps. Per block: (G) all warps gather the dot products against
//                         the local model; (R) warp 0 runs the recurrence while warp 1 starts the bulk copy of the
//                         next block's record; (S) all threads apply the update. Entry ids below HOT (ids are
//                         frequency-ranked) live in shared memory for the whole kernel as w = v + sigma' U_k; the
//                         others are read from and added to row k of the update workspace in global memory.
//
// A record arrives by ONE bulk copy. Measured: fetching the 32 coordinates straight from the matrix with two small
// bulk copies each slowed whatever phase ran while those 64 copies landed by about 3 000 cycles per block (the
// slow phase moved with the point of issue), three times what the recurrence itself costs.
//
// A block with a coordinate longer than 128 entries does not fit the shared-memory buffers: the prepare kernel
// flags it and warp 0 walks it coordinate by coordinate. Rounds that span several local
// epochs revisit coordinates, whose state the headers would not know: those take the blocked solver instead.
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <vector>

#include "solver_common.cuh"

namespace chicle {

namespace {

constexpr int kLB = 32;          // steps per block
constexpr int kCapL = 128;       // longest coordinate a staged block can hold
constexpr int kMaxNz = kLB * kCapL;
constexpr int kHT = 4096;        // slots of the prepare kernel's hash table (>= kMaxNz)
constexpr int kPreThreads = 256;  // dense prepare kernel
constexpr int kPreThreadsS = 512; // sparse prepare kernel
constexpr int kChainThreads = 512;
constexpr int kChainWarps = kChainThreads / 32;
constexpr int kRowsPerWarp = kLB / kChainWarps;

struct alignas(16) LookHdr {
    int64_t row_start;
    int32_t coord;
    int32_t nnz;
    float p0, p1, p2, p3; // the constants of the scalar step (see coordinate_step)
    float q0;             // what the states of the block's earlier coordinates at round start contribute (see below)
    float pad[3];         // [0]: log of p2 for the logistic loss (the start of its Newton iteration needs it)
};
static_assert(sizeof(LookHdr) == 48, "header size");

// A block's record starts with this; behind it (sparse): val[total] f32, idx[total] i32 (the non-zeros row after row;
// the top bit of idx marks an id that more than one coordinate of the block has), ids[T] i32 (those shared ids),
// cpos[total] u16 (for a non-zero with a shared id: its place in the id's list; the lists lie one after the other,
// each in ascending coordinate order), off[T + 1] u16 (where each list starts). Dense: val[cnt * dim].
struct alignas(16) BlkHead {
    int32_t T;         // entry ids that more than one coordinate of the block has
    int32_t flags;     // bit 0: walk this block coordinate by coordinate (the record is the head alone)
    int32_t cnt;       // steps in the block (32 but for a partition's last block)
    int32_t total_nnz; // non-zeros of the block
    uint16_t roff[kLB + 8]; // where each coordinate's non-zeros start in val / idx ([32] = total)
    LookHdr hdr[kLB];
    float G[kLB * kLB]; // G[l * 32 + j]: the scaled Gram entry of coordinates l < j (see below), else 0
};
static_assert(sizeof(BlkHead) % 16 == 0, "bulk copy size");

__host__ __device__ constexpr uint32_t record_bytes(int total, int T, bool dense)
{
    return ((uint32_t)sizeof(BlkHead) + (dense ? 4u * total : 8u * total + 4u * T + 2u * total + 2u * (T + 1)) + 15u) & ~15u;
}

struct alignas(16) BlkDir { // where a block's record is
    unsigned long long offset; // bytes from the start of the record buffer (a multiple of 16)
    uint32_t bytes;            // a multiple of 16; 0: the record buffer was full
    uint32_t pad;
};

struct LookParams {
    SolverParams S;
    unsigned char *rec;         // the records
    BlkDir *dir;                // one per block
    unsigned long long *cursor; // [0]: bytes of `rec` handed out so far this round
    unsigned long long rec_cap; // bytes of `rec`
    const int64_t *blk_base;    // K + 1: the first block of each partition in this round's numbering of the blocks
    int32_t K;
    int64_t n_blocks;
};

#ifdef CHICLE_LA_TIMING
#define LA_T(acc) do { asm volatile("" ::: "memory"); t1 = clock64(); asm volatile("" ::: "memory"); acc += t1 - t0; t0 = t1; } while (0)
#else
#define LA_T(acc) do { } while (0)
#endif

__device__ __forceinline__ int64_t steps_of(const LookParams &P, int64_t k, int64_t nk) { return partition_steps(P.S, k, nk); }
__device__ __forceinline__ int64_t block_base(const LookParams &P, int64_t k) { return P.blk_base[k]; }
__device__ __forceinline__ void block_to_part(const LookParams &P, int64_t bid, int &k, int64_t &b)
{
    int32_t lo = 0, hi = P.K; // blk_base[lo] <= bid < blk_base[hi] (partitions may differ in size)
    while (hi - lo > 1) {
        const int32_t mid = (lo + hi) >> 1;
        if (P.blk_base[mid] <= bid) lo = mid;
        else hi = mid;
    }
    k = lo;
    b = bid - P.blk_base[lo];
}

// blk_base[k] = blocks of the partitions before k (one thread: K is small next to the work of a round)
__global__ void k_block_bases(SolverParams S, int32_t K, int64_t *__restrict__ blk_base)
{
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    int64_t run = 0;
    for (int32_t k = 0; k < K; ++k) {
        blk_base[k] = run;
        const int64_t steps = partition_steps(S, k, S.part_off[k + 1] - S.part_off[k]);
        run += (steps + kLB - 1) / kLB;
    }
    blk_base[K] = run;
}

// The constants of coordinate c's scalar step (see coordinate_step).
template <int LOSS> __device__ __forceinline__ LookHdr make_hdr(const SolverParams &P, int32_t c, int64_t rs, int32_t nnz)
{
    LookHdr hd;
    hd.q0 = 0.0f;
    hd.pad[0] = hd.pad[1] = hd.pad[2] = 0.0f;
    hd.row_start = rs;
    hd.coord = c;
    hd.nnz = nnz;
    const float s = P.sqnorm[c];
    const float al = P.alpha[c];
    if (LOSS == CHICLE_LOSS_RIDGE_PRIMAL) {
        hd.p0 = P.inv_n;
        hd.p1 = al;
        hd.p2 = 1.0f / fmaf(P.sigma * s, P.inv_n, P.lambda);
        hd.p3 = P.lambda;
    } else {
        const float y = P.labels[c];
        hd.p0 = y / P.lam_n;
        hd.p1 = y * al;
        hd.p3 = y;
        if (LOSS == CHICLE_LOSS_HINGE_DUAL) hd.p2 = s > 0.0f ? P.lam_n / (P.sigma * s) : CUDART_INF_F;
        else {
            hd.p2 = P.sigma * s / P.lam_n;
            hd.pad[0] = hd.p2 > 0.0f ? logf(hd.p2) : -CUDART_INF_F; // log q, for the start of the Newton iteration
        }
    }
    return hd;
}

// Loads that are issued only where `on` holds (0 elsewhere), with nothing waiting on them at the point of issue.
__device__ __forceinline__ float ldcg_if(const float *p, bool on)
{
    float v;
    asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.u32 q, %2, 0;\n\tmov.f32 %0, 0f00000000;\n\t@q ld.global.cg.f32 %0, [%1];\n\t}"
                 : "=f"(v) : "l"(p), "r"((uint32_t)on) : "memory");
    return v;
}
__device__ __forceinline__ void red_add_if(float *p, float v, bool on)
{
    asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.u32 q, %2, 0;\n\t@q red.global.add.f32 [%0], %1;\n\t}" ::"l"(p), "f"(v), "r"((uint32_t)on) : "memory");
}
__device__ __forceinline__ float ldca_if(const float *p, bool on)
{
    float v;
    asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.u32 q, %2, 0;\n\tmov.f32 %0, 0f00000000;\n\t@q ld.global.ca.f32 %0, [%1];\n\t}"
                 : "=f"(v) : "l"(p), "r"((uint32_t)on) : "memory");
    return v;
}

// The recurrence in the form the chain runs it. Every loss keeps one number s_j per coordinate that is linear in the
// dot product, a scalar map s -> out, and the update s_j += Ghat[l][j] * out_l for the later coordinates j > l:
//   hinge     s = a + (1 - y dot / (lambda n)) * lambda n / (sigma' |x|^2), out = a' = clip(s, 0, 1)
//   logistic  s = q a - y dot / (lambda n),                                  out = a' = sigmoid(root of z + q sigmoid(z) = s)
//   ridge     s = dot / n + lambda w,                                       out = delta = -s / (sigma' |c|^2 / n + lambda)
// With dot_j = m0_j + sigma' sum_{l<j} delta_l G_jl and delta_l = y_l (a'_l - a_l) this gives, for the dual losses,
// Ghat[l][j] = c_j y_l G_jl with c_j = -sigma' p2_j y_j / (lambda n) (hinge; 0 for a zero row) or -sigma' y_j / (lambda n)
// (logistic), and s_j starts at its value for m0_j minus q0_j = sum_{l<j} Ghat[l][j] a_l, so that the chain adds
// Ghat * a'_l and not Ghat * (a'_l - a_l). Ridge: Ghat[l][j] = sigma' G_jl / n, q0 = 0. The prepare kernel stores Ghat
// and q0; a step of the chain is then: the scalar map, one shuffle, one fused multiply-add.
template <int LOSS> __device__ __forceinline__ float gram_scale(const LookHdr &h, float sigma, float inv_n)
{
    if (LOSS == CHICLE_LOSS_RIDGE_PRIMAL) return sigma * inv_n;
    if (LOSS == CHICLE_LOSS_HINGE_DUAL) return h.p2 < CUDART_INF_F ? -sigma * h.p0 * h.p2 : 0.0f;
    return -sigma * h.p0;
}
template <int LOSS> __device__ __forceinline__ float recurrence_start(float m0, const LookHdr &h)
{
    if (LOSS == CHICLE_LOSS_RIDGE_PRIMAL) return fmaf(m0, h.p0, h.p3 * h.p1);
    if (LOSS == CHICLE_LOSS_HINGE_DUAL) return fmaf(1.0f - m0 * h.p0, h.p2, h.p1) - h.q0;
    return fmaf(h.p2, h.p1, -(m0 * h.p0)) - h.q0;
}
template <int LOSS> __device__ __forceinline__ float recurrence_map(float s, const LookHdr &h)
{
    if (LOSS == CHICLE_LOSS_RIDGE_PRIMAL) return -s * h.p2;
    if (LOSS == CHICLE_LOSS_HINGE_DUAL) return __saturatef(s);
    return logistic_root(s, h.p2, h.pad[0]);
}

__device__ __forceinline__ uint32_t hash_id(int32_t id) { return ((uint32_t)id * 2654435761u) >> 20; } // 12 bits

// Hands out `bytes` of the record buffer; false when it is full (cannot happen for a buffer sized by
// lookahead_workspace; checked all the same).
__device__ __forceinline__ bool take_record(const LookParams &P, uint32_t bytes, unsigned long long &offset)
{
    offset = atomicAdd(P.cursor, (unsigned long long)bytes);
    return offset + bytes <= P.rec_cap;
}

// ------------------------------------------------------------------------------------------------ prepare
template <int NZ, int HT, int THREADS> struct PreShared {
    int32_t idx[NZ];     // the block's non-zeros, row after row
    float val[NZ];
    uint16_t slot[NZ];   // table slot of each non-zero's id
    int32_t key[HT];        // id in a table slot, -1 = empty
    uint32_t mask[HT];      // bit j: coordinate j of the block has this id
    uint16_t soff[HT];      // start of the slot's list
    float lval[NZ];      // the values of the non-zeros with shared ids, list after list (for the Gram pass)
    float G[kLB][kLB + 1];
    int64_t rs[kLB];
    int32_t nnz[kLB];
    int32_t roff[kLB + 1];
    uint32_t warp_tot[THREADS / 32];
    float gsc[kLB], ys[kLB], as[kLB]; // per coordinate: its Gram scale, and what multiplies / enters from the earlier ones
    int32_t total, too_long;
    uint32_t bytes;
    unsigned long long offset;
};

// One block's record (all threads of the CTA; every return below is taken by all of them).
template <int LOSS, int NZ, int HT, int THREADS>
__device__ __forceinline__ void prepare_block(const LookParams &P, const int64_t bid, PreShared<NZ, HT, THREADS> &sh)
{
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    int k;
    int64_t b;
    block_to_part(P, bid, k, b);
    const int64_t nk = P.S.part_off[k + 1] - P.S.part_off[k];
    const int64_t off = P.S.part_off[k] + (P.S.first_k ? P.S.first_k[k] : 0); // of this launch's first step in the order
    const int64_t steps = steps_of(P, k, nk);
    const int cnt = (int)((steps - b * kLB) < kLB ? (steps - b * kLB) : kLB);
#ifdef CHICLE_LA_TIMING
    long long pt0 = clock64(), pt1 = 0;
#define PRE_T(i) do { asm volatile("" ::: "memory"); pt1 = clock64(); if (tid == 0) atomicAdd(P.cursor + 16 + (i), (unsigned long long)(pt1 - pt0)); pt0 = pt1; asm volatile("" ::: "memory"); } while (0)
#else
#define PRE_T(i) do { } while (0)
#endif

    // ---- headers (kept in registers of warp 0 until the record's place is known)
    LookHdr hd{0, 0, 0, 0.f, 0.f, 0.f, 0.f, 0.f, {0.f, 0.f, 0.f}};
    if (warp == 0) {
        if (lane < cnt) {
            const int32_t c = P.S.perm[off + b * kLB + lane];
            const int64_t rs = P.S.indptr[c], re = P.S.indptr[c + 1];
            hd = make_hdr<LOSS>(P.S, c, rs, (int32_t)(re - rs));
        }
        sh.rs[lane] = hd.row_start;
        sh.nnz[lane] = hd.nnz;
        sh.gsc[lane] = lane < cnt ? gram_scale<LOSS>(hd, P.S.sigma, P.S.inv_n) : 0.0f;
        sh.ys[lane] = LOSS == CHICLE_LOSS_RIDGE_PRIMAL ? 1.0f : hd.p3;
        sh.as[lane] = LOSS == CHICLE_LOSS_RIDGE_PRIMAL ? 0.0f : hd.p1;
        const bool too_long = __any_sync(0xffffffffu, hd.nnz > kCapL);
        int incl = too_long ? 0 : hd.nnz;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        // (a block with more non-zeros than this variant's arrays hold is walked in place as well)
        const bool over = too_long || __shfl_sync(0xffffffffu, incl, 31) > NZ;
        sh.roff[lane] = over ? 0 : incl - hd.nnz;
        if (lane == 31) {
            sh.roff[kLB] = over ? 0 : incl;
            sh.total = over ? 0 : incl;
            sh.too_long = over ? 1 : 0;
        }
    }
    for (int p = tid; p < HT; p += THREADS) {
        sh.key[p] = -1;
        sh.mask[p] = 0u;
    }
    __syncthreads();
    PRE_T(0);
    const int total = sh.total;
    bool slow = sh.too_long != 0;
    if (!slow) {
        // ---- the block's non-zeros into shared memory, every id into the table
        for (int j = warp; j < cnt; j += THREADS / 32) {
            const int n = sh.nnz[j], r0 = sh.roff[j];
            const int64_t rs = sh.rs[j];
            int32_t ids4[kCapL / 32];
            float vals4[kCapL / 32];
#pragma unroll
            for (int c = 0; c < kCapL / 32; ++c) { // all of the row's loads first
                const int e = lane + 32 * c;
                ids4[c] = e < n ? P.S.indices[rs + e] : -1;
                vals4[c] = e < n ? P.S.values[rs + e] : 0.0f;
            }
#pragma unroll
            for (int c = 0; c < kCapL / 32; ++c) {
                const int e = lane + 32 * c;
                if (e >= n) continue;
                const int32_t id = ids4[c];
                sh.idx[r0 + e] = id;
                sh.val[r0 + e] = vals4[c];
                uint32_t p = hash_id(id) & (HT - 1);
                for (int probe = 0; probe < HT; ++probe) {
                    int32_t seen = sh.key[p];
                    if (seen == -1) {
                        seen = atomicCAS(&sh.key[p], -1, id);
                        if (seen == -1) break;
                    }
                    if (seen == id) break;
                    p = (p + 1) & (HT - 1);
                }
                atomicOr(&sh.mask[p], 1u << j);
                sh.slot[r0 + e] = (uint16_t)p;
            }
        }
        __syncthreads();
    PRE_T(1);
    }
    // ---- number the shared ids (those with more than one bit in their mask) and lay out their lists: thread t owns
    //      slots t, t + 256, ...; its running counts (ids in the high half, list entries in the low half) follow those
    //      of the threads before it
    uint32_t mine = 0;
    if (!slow)
        for (int p = tid; p < HT; p += THREADS) {
            const uint32_t m = sh.mask[p];
            if (m & (m - 1u)) mine += (1u << 16) + (uint32_t)__popc(m);
        }
    uint32_t incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) sh.warp_tot[warp] = incl;
    __syncthreads();
    PRE_T(2);
    uint32_t run = incl - mine, all = 0;
    for (int w2 = 0; w2 < THREADS / 32; ++w2) {
        if (w2 < warp) run += sh.warp_tot[w2];
        all += sh.warp_tot[w2];
    }
    const int T = (int)(all >> 16), total_m = (int)(all & 0xffffu);
    // ---- the record's place (a block that is walked in place needs the head alone)
    if (tid == 0) {
        unsigned long long offset = 0;
        uint32_t bytes = slow ? (uint32_t)sizeof(BlkHead) : record_bytes(total, T, false);
        if (!take_record(P, bytes, offset)) { offset = 0; bytes = 0; } // the chain kernel reports it
        sh.offset = offset;
        sh.bytes = bytes;
        BlkDir d;
        d.offset = offset;
        d.bytes = bytes;
        d.pad = 0;
        P.dir[bid] = d;
    }
    __syncthreads();
    PRE_T(3);
    if (sh.bytes == 0) return;
    unsigned char *rec = P.rec + sh.offset;
    BlkHead &out = *reinterpret_cast<BlkHead *>(rec);
    if (warp == 0) {
        out.hdr[lane] = hd;
        out.roff[lane] = (uint16_t)sh.roff[lane];
        if (lane < 8) out.roff[kLB + lane] = (uint16_t)sh.roff[kLB];
        if (lane == 0) {
            out.T = T; out.flags = slow ? 1 : 0; out.cnt = cnt; out.total_nnz = total;
        }
    }
    if (slow) return; // the rest of the head is not read for such a block
    float *val_g = reinterpret_cast<float *>(rec + sizeof(BlkHead));
    int32_t *idx_g = reinterpret_cast<int32_t *>(val_g + total);
    int32_t *ids_g = idx_g + total;
    uint16_t *cpos_g = reinterpret_cast<uint16_t *>(ids_g + T);
    uint16_t *off_g = cpos_g + total;
    for (int p = tid; p < HT; p += THREADS) {
        const uint32_t m = sh.mask[p];
        if (m & (m - 1u)) {
            const uint32_t t = run >> 16, o = run & 0xffffu;
            ids_g[t] = sh.key[p];
            off_g[t] = (uint16_t)o;
            sh.soff[p] = (uint16_t)o;
            run += (1u << 16) + (uint32_t)__popc(m);
        }
    }
    if (tid == 0) off_g[T] = (uint16_t)total_m;
    __syncthreads();
    PRE_T(4);
    // ---- list entries: a non-zero's place in its id's list is the number of lower coordinates that have the id
    for (int j = warp; j < cnt; j += THREADS / 32) {
        const int n = sh.nnz[j], r0 = sh.roff[j];
        for (int e = lane; e < n; e += 32) {
            const int p = sh.slot[r0 + e];
            const uint32_t m = sh.mask[p];
            const bool shared_id = (m & (m - 1u)) != 0u;
            int pos = 0;
            if (shared_id) {
                pos = sh.soff[p] + __popc(m & ((1u << j) - 1u));
                sh.lval[pos] = sh.val[r0 + e];
            }
            val_g[r0 + e] = sh.val[r0 + e];
            idx_g[r0 + e] = sh.idx[r0 + e] | (shared_id ? (int32_t)0x80000000 : 0);
            cpos_g[r0 + e] = (uint16_t)pos;
            // for the Gram pass: the id itself is no longer needed, its mask and its list's start are
            sh.idx[r0 + e] = (int32_t)m;
            sh.slot[r0 + e] = sh.soff[p];
        }
    }
    __syncthreads();
    PRE_T(5);
    // ---- Gram triangle: a warp per coordinate j, lane l collects x_j . x_l over j's entries in ascending order. The
    //      lanes first look at 32 entries at once and keep those whose id an earlier coordinate has too; only these
    //      are then walked, their mask, list start and value handed round by shuffles.
    for (int j = warp; j < kLB; j += THREADS / 32) {
        float acc = 0.0f;
        if (j < cnt) {
            const int n = sh.nnz[j], r0 = sh.roff[j];
            const uint32_t below = (1u << j) - 1u, lt = (1u << lane) - 1u;
            const bool mine = lane < j;
            for (int e0 = 0; e0 < n; e0 += 32) {
                const int e = e0 + lane;
                uint32_t m_l = 0u;
                int so_l = 0;
                float x_l = 0.0f;
                if (e < n) {
                    m_l = (uint32_t)sh.idx[r0 + e];
                    so_l = sh.slot[r0 + e];
                    x_l = sh.val[r0 + e];
                }
                uint32_t todo = __ballot_sync(0xffffffffu, (m_l & below) != 0u);
                // two entries per turn, so that the second one's loads are under way while the first is added
                while (todo) {
                    const int src0 = __ffs(todo) - 1;
                    todo &= todo - 1u;
                    const bool two = todo != 0u;
                    const int src1 = two ? __ffs(todo) - 1 : src0;
                    todo &= todo - 1u;
                    const uint32_t m0 = __shfl_sync(0xffffffffu, m_l, src0), m1 = __shfl_sync(0xffffffffu, m_l, src1);
                    const int so0 = __shfl_sync(0xffffffffu, so_l, src0), so1 = __shfl_sync(0xffffffffu, so_l, src1);
                    const float x0 = __shfl_sync(0xffffffffu, x_l, src0), x1 = __shfl_sync(0xffffffffu, x_l, src1);
                    const bool on0 = (m0 >> lane) & 1u, on1 = two && ((m1 >> lane) & 1u);
                    const float v0 = sh.lval[on0 ? so0 + __popc(m0 & lt) : 0], v1 = sh.lval[on1 ? so1 + __popc(m1 & lt) : 0];
                    acc = fmaf(x0, on0 ? v0 : 0.0f, acc);
                    acc = fmaf(x1, on1 ? v1 : 0.0f, acc);
                }
            }
            if (!mine) acc = 0.0f;
        }
        acc *= sh.gsc[j] * sh.ys[lane];
        sh.G[lane][j] = acc; // row l, column j
        float q0 = acc * sh.as[lane];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) q0 += __shfl_xor_sync(0xffffffffu, q0, o);
        if (lane == 0 && j < cnt) out.hdr[j].q0 = q0;
    }
    __syncthreads();
    PRE_T(6);
    for (int i = tid; i < kLB * kLB; i += THREADS) out.G[i] = sh.G[i >> 5][i & 31];
    PRE_T(7);
}

// A CTA takes blocks blockIdx.x, blockIdx.x + gridDim.x, ...: one each when the grid has a CTA per block; a launch
// beside the chain kernels gets a grid that fits the SMs they leave, so that it never has CTAs waiting for an SM (which
// would take the SMs of a finished chain launch before the next chain launch's CTAs, which need a whole SM each).
template <int LOSS, int NZ, int HT, int THREADS>
__global__ void __launch_bounds__(THREADS, 1024 / THREADS) k_lookahead_prepare(const LookParams P)
{
    extern __shared__ __align__(16) unsigned char smem_pre[];
    using Shared = PreShared<NZ, HT, THREADS>;
    Shared &sh = *reinterpret_cast<Shared *>(smem_pre);
    for (int64_t bid = blockIdx.x; bid < P.n_blocks; bid += gridDim.x) {
        prepare_block<LOSS, NZ, HT, THREADS>(P, bid, sh);
        __syncthreads(); // the shared arrays are reused by the next block
    }
}

// Short dense rows: every row has every id, so the lists are implicit: headers, Gram triangle and the rows.
struct PreDenseShared {
    float row[kLB][kCapL + 1];
    float gsc[kLB], ys[kLB], as[kLB];
    unsigned long long offset;
    uint32_t bytes;
};

template <int LOSS> __device__ __forceinline__ void prepare_block_dense(const LookParams &P, const int64_t bid, PreDenseShared &sh)
{
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    int k;
    int64_t b;
    block_to_part(P, bid, k, b);
    const int64_t nk = P.S.part_off[k + 1] - P.S.part_off[k];
    const int64_t off = P.S.part_off[k] + (P.S.first_k ? P.S.first_k[k] : 0); // of this launch's first step in the order
    const int64_t steps = steps_of(P, k, nk);
    const int cnt = (int)((steps - b * kLB) < kLB ? (steps - b * kLB) : kLB);
    const int dim = (int)P.S.dim;
    if (tid == 0) {
        unsigned long long offset = 0;
        uint32_t bytes = record_bytes(cnt * dim, 0, true);
        if (!take_record(P, bytes, offset)) { offset = 0; bytes = 0; }
        sh.offset = offset;
        sh.bytes = bytes;
        BlkDir d;
        d.offset = offset;
        d.bytes = bytes;
        d.pad = 0;
        P.dir[bid] = d;
    }
    __syncthreads();
    if (sh.bytes == 0) return;
    unsigned char *rec = P.rec + sh.offset;
    BlkHead &out = *reinterpret_cast<BlkHead *>(rec);
    float *val_g = reinterpret_cast<float *>(rec + sizeof(BlkHead));
    for (int j = warp; j < kLB; j += kPreThreads / 32) {
        int32_t c = 0;
        if (j < cnt) c = P.S.perm[off + b * kLB + j];
        const int64_t rs = (int64_t)c * dim;
        for (int e = lane; e < dim; e += 32) {
            const float x = j < cnt ? P.S.values[rs + e] : 0.0f;
            sh.row[j][e] = x;
            if (j < cnt) val_g[j * dim + e] = x;
        }
        if (lane == 0) {
            LookHdr hd{0, 0, 0, 0.f, 0.f, 0.f, 0.f, 0.f, {0.f, 0.f, 0.f}};
            if (j < cnt) hd = make_hdr<LOSS>(P.S, c, rs, dim);
            out.hdr[j] = hd;
            out.roff[j] = (uint16_t)((j < cnt ? j : cnt) * dim);
            sh.gsc[j] = j < cnt ? gram_scale<LOSS>(hd, P.S.sigma, P.S.inv_n) : 0.0f;
            sh.ys[j] = LOSS == CHICLE_LOSS_RIDGE_PRIMAL ? 1.0f : hd.p3;
            sh.as[j] = LOSS == CHICLE_LOSS_RIDGE_PRIMAL ? 0.0f : hd.p1;
        }
    }
    if (tid < 8) out.roff[kLB + tid] = (uint16_t)(cnt * dim);
    if (tid == 0) {
        out.T = dim; out.flags = 0; out.cnt = cnt; out.total_nnz = cnt * dim;
    }
    __syncthreads();
    // a warp per coordinate j, lane l has x_j . x_l
    for (int j = warp; j < kLB; j += kPreThreads / 32) {
        float acc = 0.0f;
        if (lane < j)
            for (int e = 0; e < dim; ++e) acc = fmaf(sh.row[j][e], sh.row[lane][e], acc);
        acc *= sh.gsc[j] * sh.ys[lane];
        out.G[lane * kLB + j] = acc;
        float q0 = acc * sh.as[lane];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) q0 += __shfl_xor_sync(0xffffffffu, q0, o);
        if (lane == 0 && j < cnt) out.hdr[j].q0 = q0;
    }
}

// (blocks blockIdx.x, blockIdx.x + gridDim.x, ...: see k_lookahead_prepare)
template <int LOSS> __global__ void __launch_bounds__(kPreThreads) k_lookahead_prepare_dense(const LookParams P)
{
    __shared__ PreDenseShared sh;
    for (int64_t bid = blockIdx.x; bid < P.n_blocks; bid += gridDim.x) {
        prepare_block_dense<LOSS>(P, bid, sh);
        __syncthreads();
    }
}

// ------------------------------------------------------------------------------------------------ chain
template <bool DENSE, int HOT, int TMAX> struct ChainShared {
    static constexpr uint32_t kRecMax = record_bytes(kMaxNz, DENSE ? 0 : TMAX, DENSE);
    alignas(16) float W[HOT];                  // the local model v + sigma' U_k at the ids below HOT
    alignas(16) unsigned char rec[2][kRecMax]; // the records of two consecutive blocks
    alignas(8) uint64_t full[2];               // count the bytes of the bulk copies into rec[0] / rec[1]
    float m0[kLB];                             // the block's dot products against the model at its start
    float dj[kLB];                             // the block's deltas
    float prod[DENSE ? 4 : kMaxNz];            // delta_j * x of the non-zeros with shared ids, list after list
    float sink[32];                            // where a lane's stores go that have no target
    int abort_flag;
};

template <int LOSS, bool DENSE, int HOT, int TMAX, int NCH>
__global__ void __launch_bounds__(kChainThreads, 1) k_lookahead_chain(const LookParams P)
{
    using Shared = ChainShared<DENSE, HOT, TMAX>;
    extern __shared__ __align__(128) unsigned char smem_chain[];
    Shared &sh = *reinterpret_cast<Shared *>(smem_chain);
    const int k = blockIdx.x;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const SolverParams &S = P.S;

    const int64_t nk = S.part_off[k + 1] - S.part_off[k];
    const int64_t steps = steps_of(P, k, nk);
    const int64_t nblocks = (steps + kLB - 1) / kLB;
    const int64_t bid0 = block_base(P, k);
    float *Uk = S.U + (size_t)k * (size_t)S.dim;
    const int hot_n = HOT < S.dim ? HOT : (int)S.dim;
    const float sigma = S.sigma;
    const float inv_sigma = 1.0f / sigma;
    volatile int *abort_flag = &sh.abort_flag;

    if (tid == 0) {
        sh.abort_flag = 0;
        mbar_init(smem_u32(&sh.full[0]), 1);
        mbar_init(smem_u32(&sh.full[1]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int i = tid; i < hot_n; i += kChainThreads) sh.W[i] = fmaf(sigma, Uk[i], S.vbase[i]);
    __syncthreads();
    if (nblocks == 0) return;

    // ---- warp 1: where a block's record is, and the copy itself. The directory entry of block b + 2 is loaded while
    //      block b runs and first looked at a block later (an unconditional load from a clamped address, so that
    //      nothing has to wait for it at the point of issue).
    auto load_dir = [&](int64_t blk, uint32_t (&d)[4]) {
        const int64_t at = blk < nblocks ? blk : nblocks - 1;
        asm volatile("ld.global.v4.u32 {%0, %1, %2, %3}, [%4];"
                     : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
                     : "l"(P.dir + (bid0 + at))
                     : "memory");
    };
    auto issue = [&](int64_t blk, const uint32_t (&d)[4]) {
        if (blk >= nblocks || lane != 0) return;
        const uint32_t bar = smem_u32(&sh.full[blk & 1]);
        // the buffer was last written by ordinary stores: order them before the copy engine's writes
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        const unsigned long long offset = ((unsigned long long)d[1] << 32) | d[0];
        const uint32_t bytes = d[2] <= Shared::kRecMax ? d[2] : 0u;
        if (bytes == 0) {
            // no record (the prepare kernel ran out of room): nothing will arrive, say so now
            atomicOr(S.status, ST_WAIT_TIMEOUT);
            *abort_flag = 1;
            return;
        }
        mbar_arrive_expect_tx(bar, bytes);
        bulk_g2s(smem_u32(&sh.rec[blk & 1][0]), P.rec + offset, bytes, bar);
    };
    uint32_t next_dir[4] = {0u, 0u, 0u, 0u};
    if (warp == 1) {
        load_dir(0, next_dir);
        issue(0, next_dir);
        load_dir(1, next_dir);
    }

    bool aborted = false;
#ifdef CHICLE_LA_TIMING
    long long tw = 0, tg1 = 0, tg = 0, tr = 0, tp1 = 0, ts = 0, trw = 0, t0 = clock64(), t1 = 0;
#endif
    for (int64_t b = 0; b < nblocks; ++b) {
        unsigned char *rec = &sh.rec[b & 1][0];
        const BlkHead &H = *reinterpret_cast<const BlkHead *>(rec);
        // block b's record must have landed (bounded wait); one decision for the whole CTA, and at the same time the
        // barrier between block b-1's update of the model and block b's reads
        int ok = mbar_wait(smem_u32(&sh.full[b & 1]), (uint32_t)(b >> 1) & 1u, abort_flag, S.status) ? 1 : 0;
        ok = __syncthreads_and(ok);
        if (!ok) { aborted = true; break; }
        LA_T(tw);
        const int cnt = H.cnt;
        const bool slow = (H.flags & 1) != 0;
        if (slow) {
            if (warp == 1) {
                issue(b + 1, next_dir);
                load_dir(b + 2, next_dir);
            }
            if (warp == 0) {
                // coordinate by coordinate against the model: ids below HOT in shared memory, the rest in row k of
                // the update workspace
                for (int j = 0; j < cnt; ++j) {
                    const LookHdr h = H.hdr[j];
                    const int32_t *ix = S.indices + h.row_start;
                    const float *xv = S.values + h.row_start;
                    float acc = 0.0f, delta, new_state;
                    for (int e = lane; e < h.nnz; e += 32) {
                        const int32_t i = DENSE ? e : ix[e];
                        const float ww = i < hot_n ? sh.W[i] : fmaf(sigma, __ldcg(Uk + i), S.vbase[i]);
                        acc = fmaf(xv[e], ww, acc);
                    }
                    acc = warp_sum(acc);
                    coordinate_step<LOSS>(acc, h, delta, new_state);
                    if (!(fabsf(delta) <= CUDART_MAX_NORMAL_F)) {
                        if (lane == 0) atomicOr(S.status, ST_NONFINITE_STEP);
                        delta = 0.0f;
                        new_state = LOSS == CHICLE_LOSS_RIDGE_PRIMAL ? h.p1 : h.p3 * h.p1;
                    }
                    if (delta != 0.0f)
                        for (int e = lane; e < h.nnz; e += 32) {
                            const int32_t i = DENSE ? e : ix[e];
                            if (i < hot_n) sh.W[i] = fmaf(sigma * delta, xv[e], sh.W[i]);
                            else Uk[i] = fmaf(delta, xv[e], __ldcg(Uk + i));
                        }
                    if (lane == 0) S.alpha[h.coord] = new_state;
                    __syncwarp();
                }
            }
            continue;
        }
        const int total = H.total_nnz, T = H.T;
        const float *val = reinterpret_cast<const float *>(rec + sizeof(BlkHead));
        const int32_t *idx = reinterpret_cast<const int32_t *>(val + total);
        const int32_t *ids = idx + total;
        const uint16_t *cpos = reinterpret_cast<const uint16_t *>(ids + T);
        const uint16_t *offs = cpos + total;
        // ---------------- (G) dot products against the model at the block's start: warp w takes coordinates
        //                  w and w + 16; all loads of the two are issued before anything is reduced
        {
            float acc[kRowsPerWarp];
            int nn[kRowsPerWarp], r0[kRowsPerWarp];
#pragma unroll
            for (int r = 0; r < kRowsPerWarp; ++r) {
                const int j = warp + kChainWarps * r;
                r0[r] = H.roff[j] + lane;
                nn[r] = H.roff[j + 1] - H.roff[j];
                acc[r] = 0.0f;
            }
            int32_t id[kRowsPerWarp][NCH];
            float x[kRowsPerWarp][NCH];
#pragma unroll
            for (int r = 0; r < kRowsPerWarp; ++r)
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
                    const bool valid = lane + 32 * c < nn[r];
                    id[r][c] = -1;
                    x[r][c] = 0.0f;
                    if (valid) {
                        x[r][c] = val[r0[r] + 32 * c];
                        id[r][c] = DENSE ? lane + 32 * c : (idx[r0[r] + 32 * c] & 0x7fffffff);
                    }
                }
            // ids below HOT from shared memory; the others from row k of the update workspace (read at L2: the
            // updates are made there by reductions) and from v, every load issued before any is used
            float hv[kRowsPerWarp][NCH], uu[kRowsPerWarp][NCH], vb[kRowsPerWarp][NCH];
#pragma unroll
            for (int r = 0; r < kRowsPerWarp; ++r)
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
                    const int32_t i = id[r][c];
                    const bool cold = i >= hot_n;
                    hv[r][c] = sh.W[(i >= 0 && !cold) ? i : 0];
                    uu[r][c] = DENSE ? 0.0f : ldcg_if(Uk + (cold ? i : 0), cold);
                    vb[r][c] = DENSE ? 0.0f : ldca_if(S.vbase + (cold ? i : 0), cold);
                }
#pragma unroll
            for (int r = 0; r < kRowsPerWarp; ++r)
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
                    const float ww = id[r][c] >= hot_n ? fmaf(sigma, uu[r][c], vb[r][c]) : hv[r][c];
                    acc[r] = fmaf(x[r][c], ww, acc[r]); // x is 0 beyond the coordinate's length
                }
            if (NCH * 32 < kCapL) {
#pragma unroll
                for (int r = 0; r < kRowsPerWarp; ++r)
                    for (int e = lane + 32 * NCH; e < nn[r]; e += 32) {
                        const int a = r0[r] + e - lane;
                        const int32_t i = DENSE ? e : (idx[a] & 0x7fffffff);
                        const float ww = i < hot_n ? sh.W[i] : fmaf(sigma, __ldcg(Uk + i), S.vbase[i]);
                        acc[r] = fmaf(val[a], ww, acc[r]);
                    }
            }
            LA_T(tg1);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1)
#pragma unroll
                for (int r = 0; r < kRowsPerWarp; ++r) acc[r] += __shfl_xor_sync(0xffffffffu, acc[r], o);
            if (lane == 0) {
#pragma unroll
                for (int r = 0; r < kRowsPerWarp; ++r) sh.m0[warp + kChainWarps * r] = acc[r];
            }
        }
        __syncthreads();
        LA_T(tg);
        // ---------------- (R) the recurrence on warp 0; warp 1 starts the next block's copy meanwhile
        if (warp == 0) {
            // Four coordinates at a time. Lane q (and its copies q + 8, q + 16, q + 24, which compute the same) keeps
            // the states of coordinates 4q .. 4q + 3. Group g: its lane walks its four coordinates by itself (no
            // shuffle inside a group), the four results are handed round, and every lane adds what they mean for
            // its own four: the step per coordinate costs about half of one shuffle per coordinate.
            const int q = lane & 7;
            const float4 *G4 = reinterpret_cast<const float4 *>(H.G); // G4[l * 8 + q]: row l, columns 4q .. 4q + 3
            LookHdr hh[4];
            float s[4], mine[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                hh[i] = H.hdr[4 * q + i];
                s[i] = recurrence_start<LOSS>(sh.m0[4 * q + i], hh[i]);
                mine[i] = 0.0f;
            }
#pragma unroll
            for (int g = 0; g < kLB / 4; ++g) {
                float4 blk[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) blk[k] = G4[(4 * g + k) * 8 + q];
                // inside the group (the numbers matter on the lanes with q == g, where blk holds the group's own
                // triangle; the others run the same instructions on copies)
                float o[4];
                o[0] = recurrence_map<LOSS>(s[0], hh[0]);
                const float t1 = fmaf(o[0], blk[0].y, s[1]);
                o[1] = recurrence_map<LOSS>(t1, hh[1]);
                const float t2 = fmaf(o[1], blk[1].z, fmaf(o[0], blk[0].z, s[2]));
                o[2] = recurrence_map<LOSS>(t2, hh[2]);
                const float t3 = fmaf(o[2], blk[2].w, fmaf(o[1], blk[1].w, fmaf(o[0], blk[0].w, s[3])));
                o[3] = recurrence_map<LOSS>(t3, hh[3]);
#pragma unroll
                for (int i = 0; i < 4; ++i) mine[i] = q == g ? o[i] : mine[i];
                float og[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) og[k] = __shfl_sync(0xffffffffu, o[k], g);
                // (zero entries of the triangle make this a no-op for the groups at or before g, whose states are final)
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    s[0] = fmaf(og[k], blk[k].x, s[0]);
                    s[1] = fmaf(og[k], blk[k].y, s[1]);
                    s[2] = fmaf(og[k], blk[k].z, s[2]);
                    s[3] = fmaf(og[k], blk[k].w, s[3]);
                }
            }
            if (lane < 8) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int j = 4 * q + i;
                    const LookHdr &h = hh[i];
                    float my_delta = 0.0f;
                    if (j < cnt) {
                        float my_state;
                        if (LOSS == CHICLE_LOSS_RIDGE_PRIMAL) {
                            my_delta = mine[i];
                            my_state = h.p1 + mine[i];
                        } else {
                            my_delta = h.p3 * (mine[i] - h.p1);
                            my_state = h.p3 * mine[i];
                        }
                        if (!(fabsf(my_delta) <= CUDART_MAX_NORMAL_F)) {
                            atomicOr(S.status, ST_NONFINITE_STEP);
                            my_delta = 0.0f;
                            my_state = LOSS == CHICLE_LOSS_RIDGE_PRIMAL ? h.p1 : h.p3 * h.p1;
                        }
                        S.alpha[h.coord] = my_state;
                    }
                    sh.dj[j] = my_delta;
                }
            }
            LA_T(trw);
        } else if (warp == 1) {
            issue(b + 1, next_dir);
            load_dir(b + 2, next_dir);
        }
        __syncthreads();
        LA_T(tr);
        // ---------------- (S) the model update
        if (DENSE) {
            const int dim = (int)S.dim;
            if (tid < dim) {
                float sum = 0.0f;
#pragma unroll 8
                for (int j = 0; j < cnt; ++j) sum = fmaf(sh.dj[j], val[j * dim + tid], sum);
                sh.W[tid] = fmaf(sigma, sum, sh.W[tid]);
            }
        } else {
            // (A) row after row: a non-zero whose id no other coordinate of the block has is applied at once; the
            //     others leave their product delta_j * x at their place in the id's list. No two of a thread's
            //     non-zeros touch the same word, so all loads are issued before the first store.
            {
                int32_t i2[kRowsPerWarp][NCH];
                float p2[kRowsPerWarp][NCH], w2[kRowsPerWarp][NCH];
                int cp[kRowsPerWarp][NCH];
                int a0[kRowsPerWarp], n2[kRowsPerWarp];
                float d2[kRowsPerWarp];
#pragma unroll
                for (int r = 0; r < kRowsPerWarp; ++r) {
                    const int j = warp + kChainWarps * r;
                    a0[r] = H.roff[j] + lane;
                    n2[r] = H.roff[j + 1] - H.roff[j];
                    d2[r] = sh.dj[j];
                }
#pragma unroll
                for (int r = 0; r < kRowsPerWarp; ++r)
#pragma unroll
                    for (int c = 0; c < NCH; ++c) {
                        const bool valid = lane + 32 * c < n2[r];
                        const int a = valid ? a0[r] + 32 * c : 0;
                        i2[r][c] = valid ? idx[a] : 0x7fffffff; // (an id beyond every range: nothing to do)
                        p2[r][c] = d2[r] * val[a];
                        cp[r][c] = cpos[a];
                    }
#pragma unroll
                for (int r = 0; r < kRowsPerWarp; ++r)
#pragma unroll
                    for (int c = 0; c < NCH; ++c) w2[r][c] = sh.W[(i2[r][c] >= 0 && i2[r][c] < hot_n) ? i2[r][c] : 0];
                // one store per non-zero, its address chosen without a branch: the list place, the model word, or a
                // word of this lane's own that nobody reads; ids beyond HOT add to the workspace row instead
                const uint32_t a_prod = smem_u32(&sh.prod[0]), a_w = smem_u32(&sh.W[0]), a_sink = smem_u32(&sh.sink[lane]);
#pragma unroll
                for (int r = 0; r < kRowsPerWarp; ++r)
#pragma unroll
                    for (int c = 0; c < NCH; ++c) {
                        const int32_t i = i2[r][c];
                        const float p = p2[r][c];
                        const uint32_t addr = i < 0 ? a_prod + 4u * (uint32_t)cp[r][c] : (i < hot_n ? a_w + 4u * (uint32_t)i : a_sink);
                        sts_f32(addr, i < 0 ? p : fmaf(sigma, p, w2[r][c]));
                        // a reduction at L2, nothing to wait for; one coordinate per id and block, blocks in order: a
                        // fixed order of additions
                        red_add_if(Uk + ((i >= hot_n && i != 0x7fffffff) ? i : 0), p, i >= hot_n && i != 0x7fffffff && p != 0.0f);
                    }
                if (NCH * 32 < kCapL) {
#pragma unroll
                    for (int r = 0; r < kRowsPerWarp; ++r)
                        for (int e = lane + 32 * NCH; e < n2[r]; e += 32) {
                            const int a = a0[r] + e - lane;
                            const int32_t i = idx[a];
                            const float p = d2[r] * val[a];
                            if (i < 0) sh.prod[cpos[a]] = p;
                            else if (i < hot_n) sh.W[i] = fmaf(sigma, p, sh.W[i]);
                            else if (p != 0.0f) atomicAdd(Uk + i, p);
                        }
                }
            }
            LA_T(tp1);
            __syncthreads();
            // (B) four threads per shared id: each adds every fourth entry of the list (at most 8: a list has at most
            //     32), then the four partial sums are added in a fixed order; two ids per thread and pass, all loads
            //     first
            const int quarter = tid & 3;
            constexpr int kIdsPerPass = kChainThreads / 4;
            for (int tb = 0; tb < T; tb += 2 * kIdsPerPass) {
                float sum[2];
                int32_t i3[2];
                bool on[2];
                int o0[2], o1[2];
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int t = tb + u * kIdsPerPass + (tid >> 2);
                    on[u] = t < T;
                    o0[u] = on[u] ? offs[t] + quarter : 0;
                    o1[u] = on[u] ? offs[t + 1] : 0;
                    i3[u] = on[u] ? ids[t] : 0;
                }
                float v[2][8];
#pragma unroll
                for (int u = 0; u < 2; ++u)
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        const int o = o0[u] + 4 * q;
                        v[u][q] = o < o1[u] ? sh.prod[o] : 0.0f;
                    }
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    sum[u] = ((v[u][0] + v[u][1]) + (v[u][2] + v[u][3])) + ((v[u][4] + v[u][5]) + (v[u][6] + v[u][7]));
                    sum[u] += __shfl_xor_sync(0xffffffffu, sum[u], 1);
                    sum[u] += __shfl_xor_sync(0xffffffffu, sum[u], 2);
                }
#pragma unroll
                for (int u = 0; u < 2; ++u)
                    if (quarter == 0 && on[u] && sum[u] != 0.0f) {
                        if (i3[u] < hot_n) sh.W[i3[u]] = fmaf(sigma, sum[u], sh.W[i3[u]]);
                        else atomicAdd(Uk + i3[u], sum[u]);
                    }
            }
        }
        LA_T(ts);
    }
#ifdef CHICLE_LA_TIMING
#ifndef LA_TIMING_TID
#define LA_TIMING_TID 0
#endif
    if (blockIdx.x == 0 && tid == LA_TIMING_TID) {
        unsigned long long *d = P.cursor + 2;
        d[0] = tw; d[1] = tg1; d[2] = tg; d[3] = tr; d[4] = tp1; d[5] = ts; d[6] = nblocks; d[7] = trw;
    }
#endif
    if (aborted) {
        // the status word has the reason; give a copy that may still be in flight one more bounded wait, write nothing
        (void)mbar_wait(smem_u32(&sh.full[0]), 0u, abort_flag, S.status);
        return;
    }
    __syncthreads();
    for (int i = tid; i < hot_n; i += kChainThreads) Uk[i] = (sh.W[i] - S.vbase[i]) * inv_sigma;
}

constexpr int kHotSkew = 24064;
constexpr int kTmax = kMaxNz / 2; // an id is shared by at least two of a block's non-zeros

template <int LOSS, bool DENSE, int HOT, int TMAX, int NCH> cudaError_t launch_chain(Glm &g, const LookParams &P)
{
    using Shared = ChainShared<DENSE, HOT, TMAX>;
    static_assert(sizeof(Shared) <= 227 * 1024, "shared memory budget");
    auto kern = k_lookahead_chain<LOSS, DENSE, HOT, TMAX, NCH>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(Shared));
    if (e != cudaSuccess) return e;
    kern<<<g.K, kChainThreads, sizeof(Shared), g.stream>>>(P);
    e = cudaGetLastError();
#ifdef CHICLE_LA_TIMING
    unsigned long long t[12] = {0};
    (void)cudaStreamSynchronize(g.stream);
    (void)cudaMemcpy(t, P.cursor + 2, sizeof(t), cudaMemcpyDeviceToHost);
    const double nb = t[6] ? (double)t[6] : 1.0;
    fprintf(stderr, "lookahead chain, cycles per block (CTA 0): wait %.0f gather %.0f reduce+bar %.0f recurrence %.0f products %.0f "
            "lists %.0f (%llu blocks); warp 0's recurrence alone %.0f, then waiting for warp 1 %.0f\n", t[0] / nb, t[1] / nb, t[2] / nb,
            (t[3] + t[7]) / nb, t[4] / nb, t[5] / nb, t[6], t[7] / nb, t[3] / nb);
#endif
    return e;
}

template <int LOSS, int NZ, int HT, int THREADS> cudaError_t launch_prepare(Glm &g, const LookParams &P, unsigned nb, cudaStream_t stream)
{
    (void)g;
    using Shared = PreShared<NZ, HT, THREADS>;
    auto pre = k_lookahead_prepare<LOSS, NZ, HT, THREADS>;
    cudaError_t e = cudaFuncSetAttribute(pre, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(Shared));
    if (e != cudaSuccess) return e;
    pre<<<nb, THREADS, sizeof(Shared), stream>>>(P);
    return cudaGetLastError();
}

// The prepare kernel of one launch's blocks on `stream`.
template <int LOSS> cudaError_t launch_prepare_on(Glm &g, const LookParams &P, cudaStream_t stream)
{
    const unsigned nb = (unsigned)P.n_blocks;
    // beside the chain kernels: no more CTAs than fit the SMs the chains leave (see k_lookahead_prepare)
    const unsigned free_sms = (unsigned)(g.sm_count > g.K ? g.sm_count - g.K : 1);
    if (g.fmt == CHICLE_FMT_DENSE_ROWMAJOR) {
        const unsigned per_sm = 2048 / kPreThreads;
        const unsigned grid = stream == g.stream || nb < free_sms * per_sm ? nb : free_sms * per_sm;
        k_lookahead_prepare_dense<LOSS><<<grid, kPreThreads, 0, stream>>>(P);
        return cudaGetLastError();
    }
    // blocks of up to 2 048 non-zeros (32 coordinates of 50 on average, with room): the small variant, four CTAs per SM
    const double avg_block = 32.0 * (double)g.nnz / (double)g.n_coord;
    cudaError_t e;
    if (avg_block * 1.25 <= 2048.0) {
        const unsigned grid = stream == g.stream || nb < free_sms * 4 ? nb : free_sms * 4;
        e = launch_prepare<LOSS, 2048, 2048, 256>(g, P, grid, stream);
    } else {
        const unsigned grid = stream == g.stream || nb < free_sms * 2 ? nb : free_sms * 2;
        e = launch_prepare<LOSS, kMaxNz, kHT, kPreThreadsS>(g, P, grid, stream);
    }
#ifdef CHICLE_LA_TIMING
    if (e == cudaSuccess) {
        unsigned long long t[8] = {0};
        (void)cudaStreamSynchronize(stream);
        (void)cudaMemcpy(t, P.cursor + 16, sizeof(t), cudaMemcpyDeviceToHost);
        (void)cudaMemset(P.cursor + 16, 0, sizeof(t));
        fprintf(stderr, "lookahead prepare, cycles per CTA: headers %.0f insert %.0f count %.0f place %.0f number %.0f entries %.0f gram %.0f write %.0f\n",
                t[0] / (double)nb, t[1] / (double)nb, t[2] / (double)nb, t[3] / (double)nb, t[4] / (double)nb, t[5] / (double)nb,
                t[6] / (double)nb, t[7] / (double)nb);
    }
#endif
    return e;
}

// The chain kernel over the blocks that a prepare launch with the same parameters made (on the handle's stream).
template <int LOSS> cudaError_t launch_chain_on(Glm &g, const LookParams &P)
{
    if (g.fmt == CHICLE_FMT_DENSE_ROWMAJOR) return launch_chain<LOSS, true, kCapL, 4, 4>(g, P);
    if (g.hot_variant) return launch_chain<LOSS, false, kHotSkew, kTmax, 2>(g, P);
    return launch_chain<LOSS, false, 4, kTmax, 4>(g, P);
}

// A round's launches. One slice: prepare, then chain. Several slices (consecutive pieces of every partition's walk):
// the first slice's prepare on the handle's stream; the later slices' prepares on the side stream, behind the first
// one, so that they fill the SMs the chain kernels leave idle; every chain launch waits for its slice's prepare.
template <int LOSS> cudaError_t launch_slices(Glm &g, const LookParams *P, int n_slices)
{
    cudaError_t e = launch_prepare_on<LOSS>(g, P[0], g.stream);
    if (e != cudaSuccess) return e;
    if (g.time_prepare) (void)cudaEventRecord(g.ev[4], g.stream);
    if (n_slices > 1) {
        e = cudaEventRecord(g.la_ev[0], g.stream);
        if (e != cudaSuccess) return e;
    }
    e = launch_chain_on<LOSS>(g, P[0]); // enqueued before the side stream's work: it takes its SMs first
    if (e != cudaSuccess) return e;
    if (n_slices > 1) {
        e = cudaStreamWaitEvent(g.la_stream, g.la_ev[0], 0);
        for (int s = 1; s < n_slices && e == cudaSuccess; ++s) {
            e = launch_prepare_on<LOSS>(g, P[s], g.la_stream);
            if (e == cudaSuccess) e = cudaEventRecord(g.la_ev[s], g.la_stream);
        }
        for (int s = 1; s < n_slices && e == cudaSuccess; ++s) {
            e = cudaStreamWaitEvent(g.stream, g.la_ev[s], 0);
            if (e == cudaSuccess) e = launch_chain_on<LOSS>(g, P[s]);
        }
    }
    return e;
}

} // namespace

int lookahead_max_dense_dim() { return kCapL; }

// A round of many blocks is cut into this many slices at most (see launch_slices).
constexpr int kMaxSlices = 3;
int lookahead_max_slices() { return kMaxSlices; }

// Bytes of the record buffer and of the block directory that a problem of this shape needs (every block's record at
// its largest: a head, and 16 bytes per non-zero for the row-wise and the transposed copy; every slice may end in a
// ragged block per partition).
void lookahead_workspace(int64_t n_coord, int64_t nnz, int32_t K, bool dense, int64_t dim, size_t *rec_bytes, size_t *dir_bytes)
{
    const size_t max_blocks = (size_t)(n_coord / kLB + (int64_t)kMaxSlices * (K + 1));
    *dir_bytes = max_blocks * sizeof(BlkDir);
    *rec_bytes = max_blocks * (sizeof(BlkHead) + 32) + (dense ? (size_t)n_coord * (size_t)dim * 4 : (size_t)nnz * 16) + 256;
}

cudaError_t launch_lookahead_solver(Glm &g, const SolverParams &S)
{
    const int32_t K = g.K;
    std::vector<int64_t> steps((size_t)K), nb((size_t)K);
    int64_t total = 0, min_nb = (int64_t)1 << 62;
    for (int32_t k = 0; k < K; ++k) {
        const int64_t nk = g.h_part_off[k + 1] - g.h_part_off[k];
        steps[(size_t)k] = g.round_steps ? g.round_steps[k] : (S.H == 0 ? nk : S.H);
        nb[(size_t)k] = (steps[(size_t)k] + kLB - 1) / kLB;
        total += nb[(size_t)k];
        if (nb[(size_t)k] > 0 && nb[(size_t)k] < min_nb) min_nb = nb[(size_t)k];
    }
    if (total <= 0 || total > 0x7fffffff) return cudaErrorInvalidConfiguration;
    // Long walks are cut into slices so that all but the first slice's prepare work runs beside the chain kernels
    // (which occupy K SMs only; with more than half of the SMs taken by chains the prepare kernels would hold the
    // chains up instead: such rounds stay in one piece). CHICLE_LA_SLICES=1 keeps every round in one piece (to time the prepare kernel alone),
    // CHICLE_LA_SLICES=3 cuts short walks too (to test the slicing on small problems).
    const bool can_slice = g.la_stream && g.la_slice && min_nb >= 8; // every partition has blocks in every slice
    int n_slices = (can_slice && total >= 4096 && min_nb >= 64 && 2 * K <= g.sm_count) ? kMaxSlices : 1;
    const char *env = getenv("CHICLE_LA_SLICES");
    if (env && env[0] == '1' && env[1] == 0) n_slices = 1;
    if (env && env[0] == '3' && env[1] == 0 && can_slice) n_slices = kMaxSlices;

    LookParams P[kMaxSlices];
    for (int s = 0; s < kMaxSlices; ++s) {
        P[s] = LookParams{};
        P[s].S = S;
        P[s].rec = static_cast<unsigned char *>(g.la_rec);
        P[s].cursor = g.la_cursor;
        P[s].rec_cap = g.la_rec_bytes;
        P[s].K = K;
    }
    cudaError_t e = cudaMemsetAsync(g.la_cursor, 0, sizeof(unsigned long long), g.stream);
    if (e != cudaSuccess) return e;
    if (n_slices == 1) {
        P[0].dir = static_cast<BlkDir *>(g.la_dir);
        P[0].blk_base = g.la_blk_base;
        P[0].n_blocks = total;
        k_block_bases<<<1, 32, 0, g.stream>>>(P[0].S, K, g.la_blk_base);
    } else {
        // Slice s of partition k: blocks cut[s] .. cut[s + 1] of its walk. The prepare kernel of slice s + 1 should
        // be done when the chain launch of slice s is, so the slices grow by a factor a = 0.8 / rho, where rho is the
        // prepare time of a piece of the walk on the SMs the chains leave over its chain time: about
        // c K / (SMs - K) with c = SM-time of the prepare kernel per step over the chain's time per step, 1.2 to
        // 1.9 measured on the sparse configurations (2 assumed), 0.18 on short dense rows (0.25 assumed). The first
        // slice's prepare kernel is the part that stays exposed: 1 / (1 + a + a^2) of the walk.
        const double c_ratio = g.fmt == CHICLE_FMT_DENSE_ROWMAJOR ? 0.25 : 2.0;
        const double rho = c_ratio * (double)K / (double)(g.sm_count > K ? g.sm_count - K : 1);
        const double a = 0.8 / rho;
        double f1 = 1.0 / (1.0 + a + a * a);
        f1 = f1 < 1.0 / 64 ? 1.0 / 64 : (f1 > 0.5 ? 0.5 : f1);
        const double f2 = a * f1;
        std::vector<int64_t> h((size_t)kMaxSlices * 2 * (size_t)K);
        int64_t blocks[kMaxSlices] = {0, 0, 0};
        for (int32_t k = 0; k < K; ++k) {
            const int64_t nbk = nb[(size_t)k]; // 0, or at least 8
            int64_t c1 = (int64_t)((double)nbk * f1), c2 = (int64_t)((double)nbk * (f1 + f2));
            c1 = c1 < 1 ? 1 : c1;
            c2 = c2 < c1 + 1 ? c1 + 1 : c2;
            c2 = c2 > nbk - 1 ? nbk - 1 : c2;
            const int64_t cut[kMaxSlices + 1] = {0, nbk ? c1 : 0, nbk ? c2 : 0, nbk};
            for (int s = 0; s < kMaxSlices; ++s) {
                const int64_t first = cut[s] * kLB;
                const int64_t last = s + 1 == kMaxSlices ? steps[(size_t)k] : cut[s + 1] * kLB;
                h[((size_t)s * 2) * (size_t)K + (size_t)k] = last - first;
                h[((size_t)s * 2 + 1) * (size_t)K + (size_t)k] = first;
                blocks[s] += (last - first + kLB - 1) / kLB;
            }
        }
        // a pageable source: the runtime has taken its copy of these words when the call returns
        e = cudaMemcpyAsync(g.la_slice, h.data(), h.size() * sizeof(int64_t), cudaMemcpyHostToDevice, g.stream);
        if (e != cudaSuccess) return e;
        int64_t dir_off = 0;
        for (int s = 0; s < kMaxSlices; ++s) {
            P[s].S.H = 0;
            P[s].S.steps_k = g.la_slice + ((size_t)s * 2) * (size_t)K;
            P[s].S.first_k = g.la_slice + ((size_t)s * 2 + 1) * (size_t)K;
            P[s].dir = static_cast<BlkDir *>(g.la_dir) + dir_off;
            int64_t *bases = g.la_blk_base + (size_t)s * ((size_t)K + 1);
            P[s].blk_base = bases;
            P[s].n_blocks = blocks[s];
            dir_off += blocks[s];
            k_block_bases<<<1, 32, 0, g.stream>>>(P[s].S, K, bases);
        }
    }
    switch (g.loss) {
    case CHICLE_LOSS_HINGE_DUAL: return launch_slices<CHICLE_LOSS_HINGE_DUAL>(g, P, n_slices);
    case CHICLE_LOSS_LOGISTIC_DUAL: return launch_slices<CHICLE_LOSS_LOGISTIC_DUAL>(g, P, n_slices);
    default: return launch_slices<CHICLE_LOSS_RIDGE_PRIMAL>(g, P, n_slices);
    }
}

} // namespace chicle
