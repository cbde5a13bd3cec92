// Local SCD solver with block look-ahead: the same result as walking a partition's visiting order coordinate by
// coordinate (paper Sec. 2.2 worker structure with L = 1; Sec. 5.1: SCD local solver), up to rounding order, with
// everything that does not depend on the step before taken off the sequential chain.
//
// The walk is cut into blocks of 32 consecutive steps. With w the local model some steps back,
//     dot_j = x_j . w + sigma' * sum over the steps l since then of delta_l * (x_j . x_l),
// so once the dot products against an OLDER model and the Gram entries x_j . x_l are known, the steps are a scalar
// recurrence. A block's dot products are taken against the model as it was two blocks earlier (while the block
// before it is still being walked); what the block before contributes comes from the cross Gram matrix of the two
// blocks, what the block's own earlier steps contribute from its Gram triangle. Only the recurrence is sequential:
// one warp runs it block after block without waiting for a model update, while the other warps, and the other CTAs
// of the partition's thread-block cluster, apply block b's update to the model and take block b + 2's dot products.
//
//   k_lookahead_prepare   one CTA per block; nothing in it depends on the model. Writes the block's records: for
//                         the recurrence warp the per-step constants, the scaled Gram triangle and the scaled cross
//                         Gram matrix with the next block; for each CTA of the cluster the block's non-zeros whose
//                         entry id falls to that CTA (id mod cluster size), packed row after row, and for the ids
//                         that several coordinates of the block share the transposed view (one list per id, in
//                         ascending coordinate order), so that the model update needs no atomics and gives the same
//                         bits every run.
//   k_lookahead_chain     one cluster of C CTAs per partition. Entry ids below C * HOT (ids are frequency-ranked)
//                         live in shared memory for the whole kernel as w = v + sigma' U_k, id i in CTA i mod C;
//                         the others live in row k of the update workspace in global memory, which holds the model
//                         itself between the launches of a round (the first launch turns U_k into w in place, the
//                         last one turns it back): one gather or one reduction per non-zero.
//                         Warp 0 of CTA 0 runs the recurrence. The worker warps of every CTA loop over
//                         "wait for block b's deltas, apply them to my part of the model, take my part of block
//                         b + 2's dot products, send the 32 partial sums to CTA 0". Deltas and partial sums travel
//                         through distributed shared memory by asynchronous stores that complete on the receiver's
//                         mbarrier; no multicast, every wait bounded.
//
// Where many partitions leave the prepare kernels few SMs (one CTA per partition on sparse data), the dot products are
// taken one block ahead only, against the model after the block before: no cross Gram matrix (the prepare kernels are
// what bounds such rounds), and the recurrence warp waits for each block's dot products; and where the chains take more
// than half of the SMs, the prepare kernels alternate with the chain launches instead of running beside them.
//
// A block with more non-zeros than the shared-memory buffers hold is flagged by the prepare kernel: the pipeline
// drains, warp 0 of CTA 0 walks the block coordinate by coordinate against the whole model, and the pipeline starts
// again behind it. Rounds that span several local epochs run the pair of kernels once per epoch.
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <vector>

#include "solver_common.cuh"

namespace chicle {

namespace {

constexpr int kLB = 32;            // steps per block
constexpr int kMaxC = 8;           // CTAs per cluster at most (the portable limit)
constexpr int kCapL = 128;         // longest dense coordinate
constexpr int kIdBits = 26;        // entry ids of a staged non-zero (problems with more ids take the blocked solver)
constexpr uint32_t kIdMask = (1u << kIdBits) - 1u;
constexpr int kChainThreads = 512;
constexpr int kSubSlots = 4;       // worker records in shared memory: blocks b .. b + 3
constexpr int kHeadSlots = 3;      // recurrence records in shared memory
// Worker warps: all but the warps that share warp 0's scheduler (warp ids 0, 4, 8, 12), which stay out of its way.
constexpr int kWorkWarps = 12;
constexpr int kWorkThreads = kWorkWarps * 32;
constexpr int kBarWork = 1;        // named barrier of the worker warps

// Per-step constants for the recurrence warp (see coordinate_step for p0 .. p3).
struct alignas(16) CHdr {
    int32_t coord;
    float p0, p1, p2, p3;
    float A, B; // the recurrence's state starts at A + B * (dot product against the older model) (+ the cross terms)
    float lq;   // logistic: log of p2
};
static_assert(sizeof(CHdr) == 32, "header size");

// What the recurrence warp reads for one block.
struct alignas(16) ChainHead {
    int32_t cnt;    // steps in the block (32 but for a partition's last block)
    int32_t flags;  // bit 0: walk this block coordinate by coordinate
    int32_t pad[2];
    CHdr hdr[kLB];
    float q0n[kLB];      // what the states of this block's coordinates at round start contribute to the next block
    float G[kLB * kLB];  // G[l * 32 + j]: scaled Gram entry of this block's coordinates l < j, else 0
    float X[kLB * kLB];  // X[l * 32 + j]: scaled Gram entry of this block's l with the NEXT block's j (0: no carry)
};
static_assert(sizeof(ChainHead) % 16 == 0, "bulk copy size");

// What one CTA's workers read for one block. Behind it (sparse): val[n] f32, meta[n] u32 (entry id in the low bits,
// the coordinate's place in the block above them, the top bit marks an id that several coordinates of the block
// have), ids[T] u32 (those shared ids), cpos[n] u16 (for a non-zero with a shared id: its place in the id's list;
// the lists lie one after the other, each in ascending coordinate order), off[T + 1] u16 (where each list starts).
// Dense: val[cnt * dim].
struct alignas(16) SubHead {
    int32_t n;     // non-zeros of the block that fall to this CTA
    int32_t T;     // shared ids among them
    int32_t cnt;
    int32_t flags; // bit 0 as in ChainHead (the record is then this head alone)
    uint16_t roff[kLB + 8]; // where each coordinate's non-zeros start ([32] = n)
};
static_assert(sizeof(SubHead) == 96, "sub-record head");

__host__ __device__ constexpr uint32_t sub_bytes(int n, int T, bool dense)
{
    return ((uint32_t)sizeof(SubHead) + (dense ? 4u * n : 8u * n + 4u * T + 2u * n + 2u * (T + 1)) + 15u) & ~15u;
}

struct alignas(16) BlkDir { // where a record is
    unsigned long long offset; // bytes from the start of the launch's region of the record buffer (a multiple of 16)
    uint32_t bytes;            // a multiple of 16; 0: no record was written
    uint32_t flags;            // bit 0: the block is walked coordinate by coordinate
};

struct LookParams {
    SolverParams S;
    unsigned char *rec;          // this launch's region of the record buffer
    BlkDir *dirH;                // one per block: the recurrence warp's record
    BlkDir *dirS;                // C per block: the workers' records
    unsigned long long *cursor;  // bytes of the pool handed out so far in this launch
    unsigned long long *timing;  // scratch words of a -DCHICLE_LA_TIMING build
    unsigned long long pool_off; // the pool of worker records starts here (the heads lie before it, one per block)
    unsigned long long pool_cap; // bytes of the pool
    const int64_t *blk_base;     // K + 1: the first block of each partition in this launch's numbering of the blocks
    int32_t K, logC;
    int32_t depth;               // 2: a block's dot products are taken two blocks ahead and corrected with the cross
                                 // Gram matrix; 1: one block ahead, no cross Gram matrix (the recurrence waits for them)
    int32_t nzcap;               // non-zeros a worker record holds at most
    int32_t hotc;                // entry ids per CTA kept in shared memory
    int64_t n_blocks;
    int64_t drop_block;          // test aid: this block's records are left unpublished (-1: none)
    int64_t nnz;                 // entries of the matrix (what a coordinate's extent is checked against in a debug build)
    int32_t model_in;            // the round's first chain launch: row k of the update workspace holds U_k and is turned
                                 // into the local model w = v + sigma' U_k in place
    int32_t model_out;           // the round's last chain launch: the row is turned back into U_k. Between a round's
                                 // launches the row holds w itself: an id beyond the part in shared memory costs one
                                 // gather instead of two, and nothing is rounded from launch to launch
};

#ifdef CHICLE_LA_TIMING
#define LA_T(acc) do { asm volatile("" ::: "memory"); t1 = clock64(); asm volatile("" ::: "memory"); acc += t1 - t0; t0 = t1; } while (0)
#else
#define LA_T(acc) do { } while (0)
#endif

__device__ __forceinline__ int64_t steps_of(const LookParams &P, int64_t k, int64_t nk) { return partition_steps(P.S, k, nk); }
// (debug build) an entry id as loaded from the matrix: id 0 stands in for one outside [0, dim) (the call then ends with
// the bounds status, its arithmetic is of no interest; what matters is that nothing is addressed with the bad id)
__device__ __forceinline__ int32_t checked_id(const LookParams &P, int32_t id)
{
    return CHICLE_IN_BOUNDS(P.S.status, id >= 0 && (int64_t)id < P.S.dim) ? id : 0;
}
// (debug build) a visiting-order entry and the extent of its coordinate: an empty coordinate 0 if either is off
__device__ __forceinline__ void checked_extent(const LookParams &P, int32_t &c, int64_t &rs, int32_t &n)
{
    if (!CHICLE_IN_BOUNDS(P.S.status, c >= 0 && (int64_t)c < P.S.n_coord)) c = 0;
    rs = P.S.indptr[c];
    const int64_t len = P.S.indptr[c + 1] - rs;
    n = (int32_t)len;
    if (!CHICLE_IN_BOUNDS(P.S.status, rs >= 0 && len >= 0 && len <= 0x7fffffff && rs + len <= P.nnz)) { rs = 0; n = 0; }
}
// The same search over a copy of blk_base in shared memory (a launch with at most kBaseStaged - 1 partitions; block
// counts fit 32 bits): the dependent loads of the search cost 30 cycles each instead of an L2 round trip.
constexpr int kBaseStaged = 260;
__device__ __forceinline__ void block_to_part_staged(const int32_t *base, int32_t K, int64_t bid, int &k, int64_t &b)
{
    int32_t lo = 0, hi = K;
    while (hi - lo > 1) {
        const int32_t mid = (lo + hi) >> 1;
        if ((int64_t)base[mid] <= bid) lo = mid;
        else hi = mid;
    }
    k = lo;
    b = bid - (int64_t)base[lo];
}
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

// The constants of coordinate c's scalar step (see coordinate_step), and the line A + B * dot that the recurrence's
// state starts from (what the block's earlier coordinates contribute at their round-start states is taken off A
// once the Gram triangle is known).
template <int LOSS> __device__ __forceinline__ CHdr make_hdr(const SolverParams &P, int32_t c)
{
    CHdr hd;
    hd.coord = c;
    hd.lq = 0.0f;
    const float s = P.sqnorm[c];
    const float al = P.alpha[c];
    if (LOSS == CHICLE_LOSS_RIDGE_PRIMAL) {
        hd.p0 = P.inv_n;
        hd.p1 = al;
        hd.p2 = 1.0f / fmaf(P.sigma * s, P.inv_n, P.lambda);
        hd.p3 = P.lambda;
        hd.A = P.lambda * al;
        hd.B = P.inv_n;
    } else {
        const float y = P.labels[c];
        hd.p0 = y / P.lam_n;
        hd.p1 = y * al;
        hd.p3 = y;
        if (LOSS == CHICLE_LOSS_HINGE_DUAL) {
            const bool zero = !(s > 0.0f);
            hd.p2 = zero ? CUDART_INF_F : P.lam_n / (P.sigma * s);
            // a + (1 - y dot / (lambda n)) * p2; a zero row goes to a' = 1 whatever the model is
            hd.A = zero ? 2.0f : hd.p2 + hd.p1;
            hd.B = zero ? 0.0f : -hd.p0 * hd.p2;
        } else {
            hd.p2 = P.sigma * s / P.lam_n;
            hd.lq = hd.p2 > 0.0f ? logf(hd.p2) : -CUDART_INF_F; // log q, for the start of the Newton iteration
            hd.A = hd.p2 * hd.p1;
            hd.B = -hd.p0;
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

// The recurrence in the form the chain runs it. Every loss keeps one number s_j per coordinate that is linear in the
// dot product, a scalar map s -> out, and the update s_j += Ghat[l][j] * out_l for the later coordinates j:
//   hinge     s = a + (1 - y dot / (lambda n)) * lambda n / (sigma' |x|^2), out = a' = clip(s, 0, 1)
//   logistic  s = q a - y dot / (lambda n),                                  out = a' = sigmoid(root of z + q sigmoid(z) = s)
//   ridge     s = dot / n + lambda w,                                       out = delta = -s / (sigma' |c|^2 / n + lambda)
// With dot_j = (older dot)_j + sigma' sum_l delta_l G_jl and delta_l = y_l (a'_l - a_l) this gives, for the dual
// losses, Ghat[l][j] = c_j y_l G_jl with c_j = -sigma' p2_j y_j / (lambda n) (hinge; 0 for a zero row) or
// -sigma' y_j / (lambda n) (logistic), and s_j starts sum_l Ghat[l][j] a_l lower, so that the chain adds
// Ghat * a'_l and not Ghat * (a'_l - a_l). Ridge: Ghat[l][j] = sigma' G_jl / n, nothing to take off. The prepare kernel
// stores Ghat (inside a block and from a block to the next) and the sums; a step of the chain is then: the scalar
// map, one shuffle per four coordinates, one fused multiply-add.
template <int LOSS> __device__ __forceinline__ float gram_scale(const CHdr &h, float sigma, float inv_n)
{
    if (LOSS == CHICLE_LOSS_RIDGE_PRIMAL) return sigma * inv_n;
    if (LOSS == CHICLE_LOSS_HINGE_DUAL) return h.p2 < CUDART_INF_F ? -sigma * h.p0 * h.p2 : 0.0f;
    return -sigma * h.p0;
}
template <int LOSS> __device__ __forceinline__ float recurrence_map(float s, float p2, float lq)
{
    if (LOSS == CHICLE_LOSS_RIDGE_PRIMAL) return -s * p2;
    if (LOSS == CHICLE_LOSS_HINGE_DUAL) return __saturatef(s);
    return logistic_root(s, p2, lq);
}

// The most frequent ids (ids are frequency-ranked) are in most of a block's coordinates. Their part of the Gram
// matrices is taken from dense 32 x kHD tiles; only the other entries are walked through the table. Table slot: the id itself below kHD, a hashed slot above.
constexpr int kHD = 32;
constexpr int kHDS = kHD + 4; // row stride of the tiles: 16-byte loads of consecutive rows fall on different banks
template <int HT> __device__ __forceinline__ uint32_t home_slot(int32_t id)
{
    return id < kHD ? (uint32_t)id : kHD + (((uint32_t)id * 2654435761u) >> 16) % (uint32_t)(HT - kHD);
}
template <int HT> __device__ __forceinline__ uint32_t next_slot(uint32_t p) { return p + 1 < (uint32_t)HT ? p + 1 : kHD; }

// ------------------------------------------------------------------------------------------------ prepare
template <int NZ, int HT, int THREADS> struct PreShared {
    int32_t idx[NZ];     // the block's non-zeros, row after row (later: the membership mask of the non-zero's id)
    float val[NZ];
    uint16_t slot[NZ];   // table slot of each non-zero's id (later: where the id's list of values starts)
    int32_t key[HT];     // id in a table slot, -1 = empty
    uint32_t mask[HT];   // bit j: coordinate j of the block has this id
    uint16_t soff[HT];   // start of the slot's list in lval
    uint16_t coff[HT];   // a shared id: start of its list among the lists of its CTA's record
    float lval[NZ];      // the values of the block's non-zeros, one list per id, each in ascending coordinate order
    float G[kLB][kLB + 1];
    float X[kLB][kLB + 1];
    alignas(16) float Dc[kLB][kHDS]; // this block's entries with the kHD most frequent ids, dense
    alignas(16) float Dn[kLB][kHDS]; // the next block's
    CHdr hdr[kLB];
    float q0n[kLB];
    int64_t rs[kLB];
    int32_t nnz[kLB];
    int32_t roff[kLB + 1];
    uint16_t rc[kLB + 1][kMaxC]; // non-zeros of coordinate j that fall to CTA c; then where they start in c's record
    uint32_t cntTL[kMaxC], cntTL2[kMaxC], cntAll; // per CTA: shared ids (high half) and their list entries (low half); all list entries
    float gsc[kLB], ys[kLB], as[kLB]; // per coordinate: its Gram scale, and what multiplies / enters from the earlier ones
    float gscn[kLB];                  // the next block's coordinates: their Gram scales
    int64_t nrs[kLB];
    int32_t nnnz[kLB];
    unsigned long long sub_off[kMaxC];
    uint32_t sub_len[kMaxC];
    int32_t subT[kMaxC];
    int32_t ncls[kMaxC]; // the next block's non-zeros per CTA
    int32_t total, slow, carry, ncnt;
    int32_t base[kBaseStaged]; // blk_base of the first partitions, staged once per launch (see block_to_part_staged)
};

// One block's records (all threads of the CTA; every return below is taken by all of them).
template <int LOSS, int NZ, int HT, int THREADS>
__device__ __forceinline__ void prepare_block(const LookParams &P, const int64_t bid, PreShared<NZ, HT, THREADS> &sh)
{
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    constexpr int NW = THREADS / 32;
    const int C = 1 << P.logC;
    int k;
    int64_t b;
    if (P.K < kBaseStaged) block_to_part_staged(sh.base, P.K, bid, k, b);
    else block_to_part(P, bid, k, b);
    const int64_t nk = P.S.part_off[k + 1] - P.S.part_off[k];
    const int64_t off = P.S.part_off[k] + (P.S.first_k ? P.S.first_k[k] : 0); // of this launch's first step in the order
    const int64_t steps = steps_of(P, k, nk);
    const int cnt = (int)((steps - b * kLB) < kLB ? (steps - b * kLB) : kLB);
    const int64_t left = steps - (b + 1) * kLB; // steps behind this block
    const int ncnt = (left <= 0 || P.depth < 2) ? 0 : (left < kLB ? (int)left : kLB);
    ChainHead &out = *reinterpret_cast<ChainHead *>(P.rec + (size_t)bid * sizeof(ChainHead));
#ifdef CHICLE_LA_TIMING
    long long pt0 = clock64(), pt1 = 0;
#define PRE_T(i) do { asm volatile("" ::: "memory"); pt1 = clock64(); if (tid == 0) atomicAdd(P.timing + 16 + (i), (unsigned long long)(pt1 - pt0)); pt0 = pt1; asm volatile("" ::: "memory"); } while (0)
#else
#define PRE_T(i) do { } while (0)
#endif

    // ---- headers: warp 0 this block's coordinates, warp 1 the next block's
    if (warp == 0) {
        CHdr hd{0, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        int64_t rs = 0;
        int32_t n = 0;
        if (lane < cnt) {
            int32_t c = P.S.perm[off + b * kLB + lane];
            checked_extent(P, c, rs, n);
            hd = make_hdr<LOSS>(P.S, c);
        }
        sh.hdr[lane] = hd;
        sh.rs[lane] = rs;
        sh.nnz[lane] = n;
        sh.gsc[lane] = lane < cnt ? gram_scale<LOSS>(hd, P.S.sigma, P.S.inv_n) : 0.0f;
        sh.ys[lane] = LOSS == CHICLE_LOSS_RIDGE_PRIMAL ? 1.0f : hd.p3;
        sh.as[lane] = LOSS == CHICLE_LOSS_RIDGE_PRIMAL ? 0.0f : hd.p1;
        int incl = n;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        const int tot = __shfl_sync(0xffffffffu, incl, 31);
        const bool over = tot > NZ; // more non-zeros than this kernel's arrays hold: walked in place
        sh.roff[lane] = over ? 0 : incl - n;
        if (lane == 31) {
            sh.roff[kLB] = over ? 0 : incl;
            sh.total = over ? 0 : incl;
            sh.slow = over ? 1 : 0;
        }
    } else if (warp == 1) {
        CHdr hd{0, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        int64_t rs = 0;
        int32_t n = 0;
        if (lane < ncnt) {
            int32_t c = P.S.perm[off + (b + 1) * kLB + lane];
            checked_extent(P, c, rs, n);
            hd = make_hdr<LOSS>(P.S, c);
        }
        sh.nrs[lane] = rs;
        sh.nnnz[lane] = n;
        sh.gscn[lane] = lane < ncnt ? gram_scale<LOSS>(hd, P.S.sigma, P.S.inv_n) : 0.0f;
        int tot = n;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) tot += __shfl_xor_sync(0xffffffffu, tot, o);
        if (lane == 0) {
            sh.ncnt = ncnt;
            sh.carry = (ncnt > 0 && tot <= NZ) ? 1 : 0; // (and both blocks must be staged: see below)
        }
    }
    for (int p = tid; p < HT; p += THREADS) {
        sh.key[p] = -1;
        sh.mask[p] = 0u;
    }
    for (int p = tid; p < (kLB + 1) * kMaxC; p += THREADS) (&sh.rc[0][0])[p] = 0;
    for (int p = tid; p < kLB * kHDS; p += THREADS) {
        (&sh.Dc[0][0])[p] = 0.0f;
        (&sh.Dn[0][0])[p] = 0.0f;
    }
    if (tid < kMaxC) { sh.ncls[tid] = 0; sh.cntTL[tid] = 0u; sh.cntTL2[tid] = 0u; }
    if (tid == 0) sh.cntAll = 0u;
    __syncthreads();
    PRE_T(0);
    const int total = sh.total;
    const bool slow = sh.slow != 0;
    const bool carry = !slow && sh.carry != 0;
    if (!slow) {
        // ---- the block's non-zeros into shared memory, every id into the table; how many fall to each CTA. The
        //      first 128 entries of a coordinate are loaded before any is used.
        //      The loads of a warp's next coordinate are issued before this one's entries are inserted.
        int32_t ids_nx[4];
        float vals_nx[4];
        auto load4 = [&](int j, int32_t (&ids)[4], float (&vals)[4]) {
            const int n = j < cnt ? sh.nnz[j] : 0;
            const int64_t rs = j < cnt ? sh.rs[j] : 0;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int e = lane + 32 * c;
                ids[c] = e < n ? checked_id(P, P.S.indices[rs + e]) : -1;
                vals[c] = e < n ? P.S.values[rs + e] : 0.0f;
            }
        };
        load4(warp, ids_nx, vals_nx);
        for (int j = warp; j < cnt; j += NW) {
            const int n = sh.nnz[j], r0 = sh.roff[j];
            const int64_t rs = sh.rs[j];
            int per_class[kMaxC];
#pragma unroll
            for (int c = 0; c < kMaxC; ++c) per_class[c] = 0;
            int32_t ids4[4];
            float vals4[4];
#pragma unroll
            for (int c = 0; c < 4; ++c) { ids4[c] = ids_nx[c]; vals4[c] = vals_nx[c]; }
            load4(j + NW, ids_nx, vals_nx);
            auto take = [&](int e, int32_t id, float x) {
                const bool on = id >= 0;
                if (on) {
                    sh.idx[r0 + e] = id;
                    sh.val[r0 + e] = x;
                    uint32_t p = home_slot<HT>(id);
                    if (id < kHD) {
                        sh.key[p] = id;
                        sh.Dc[j][id] = x;
                    } else {
                        for (int probe = 0; probe < HT; ++probe) {
                            int32_t seen = sh.key[p];
                            if (seen == -1) {
                                seen = atomicCAS(&sh.key[p], -1, id);
                                if (seen == -1) break;
                            }
                            if (seen == id) break;
                            p = next_slot<HT>(p);
                        }
                    }
                    atomicOr(&sh.mask[p], 1u << j);
                    sh.slot[r0 + e] = (uint16_t)p;
                }
#pragma unroll
                for (int c = 0; c < kMaxC; ++c)
                    if (c < C) per_class[c] += __popc(__ballot_sync(0xffffffffu, on && (id & (C - 1)) == c));
            };
#pragma unroll
            for (int c = 0; c < 4; ++c)
                if (32 * c < n) take(lane + 32 * c, ids4[c], vals4[c]);
            for (int e0 = 128; e0 < n; e0 += 32) {
                const int e = e0 + lane;
                take(e, e < n ? checked_id(P, P.S.indices[rs + e]) : -1, e < n ? P.S.values[rs + e] : 0.0f);
            }
            if (lane == 0) {
#pragma unroll
                for (int c = 0; c < kMaxC; ++c) sh.rc[j][c] = (uint16_t)per_class[c];
            }
        }
    }
    __syncthreads();
    PRE_T(1);
    // ---- count the ids that more than one coordinate has, and their list entries, per CTA (shared-memory atomics:
    //      ids in the high half, list entries in the low half; only the totals are needed before the records' places
    //      are known)
    if (!slow)
        for (int p = tid; p < HT; p += THREADS) {
            const uint32_t m = sh.mask[p];
            if (m & (m - 1u)) atomicAdd(&sh.cntTL[sh.key[p] & (C - 1)], (1u << 16) + (uint32_t)__popc(m));
        }
    // where each coordinate's non-zeros start in each CTA's record (warp 0, lane = coordinate)
    if (warp == 0 && !slow) {
#pragma unroll
        for (int c = 0; c < kMaxC; ++c) {
            const int mine = sh.rc[lane][c];
            int incl = mine;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int t = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += t;
            }
            sh.rc[lane][c] = (uint16_t)(incl - mine);
            if (lane == 31) sh.rc[kLB][c] = (uint16_t)incl;
        }
    }
    __syncthreads();
    PRE_T(2);
    // ---- the records' places: the head has its own (one per block); the workers' records come from the pool. A
    //      block that the pool has no room for is walked in place like one that is too long.
    if (tid == 0) {
        unsigned long long need = 0;
        uint32_t len[kMaxC];
#pragma unroll
        for (int c = 0; c < kMaxC; ++c) {
            len[c] = c < C ? sub_bytes(sh.rc[kLB][c], (int)(sh.cntTL[c] >> 16), false) : 0u;
            need += len[c];
        }
        unsigned long long at = 0;
        int sl = sh.slow;
#pragma unroll
        for (int c = 0; c < kMaxC; ++c)
            if (c < C && sh.rc[kLB][c] > P.nzcap) sl = 1; // more of them fall to one CTA than its record holds
        if (!sl) {
            at = atomicAdd(P.cursor, need);
            if (at + need > P.pool_cap) sl = 2;
        }
        sh.slow = sl;
#pragma unroll
        for (int c = 0; c < kMaxC; ++c) {
            if (c >= C) continue;
            BlkDir d;
            if (sl) { // nothing to stage: the workers copy the first bytes of the head instead
                d.offset = (unsigned long long)bid * sizeof(ChainHead);
                d.bytes = 16u;
                d.flags = 1u;
            } else {
                d.offset = P.pool_off + at;
                d.bytes = len[c];
                d.flags = 0u;
                sh.sub_off[c] = d.offset;
                sh.sub_len[c] = len[c];
                sh.subT[c] = (int32_t)(sh.cntTL[c] >> 16);
                at += len[c];
            }
            if (bid == P.drop_block) d.bytes = 0u;
            P.dirS[bid * C + c] = d;
        }
    }
    __syncthreads();
    PRE_T(3);
    const bool walk = sh.slow != 0; // (slow, or no room in the pool)
    if (warp == 0 && lane == 0) {
        out.cnt = cnt;
        out.flags = walk ? 1 : 0;
        out.pad[0] = out.pad[1] = 0;
    }
    if (walk) {
        // the head carries the constants of the steps and nothing else; nothing is carried to the next block
        if (warp == 0) {
            out.hdr[lane] = sh.hdr[lane];
            out.q0n[lane] = 0.0f;
        }
        for (int i = tid; i < kLB * kLB; i += THREADS) out.X[i] = 0.0f;
        return;
    }
    // ---- the workers' record heads, shared-id tables and list starts
    if (tid < C) {
        SubHead &h = *reinterpret_cast<SubHead *>(P.rec + sh.sub_off[tid]);
        h.n = sh.rc[kLB][tid];
        h.T = sh.subT[tid];
        h.cnt = cnt;
        h.flags = 0;
    }
    for (int i = tid; i < C * (kLB + 8); i += THREADS) {
        const int c = i / (kLB + 8), j = i - c * (kLB + 8);
        reinterpret_cast<SubHead *>(P.rec + sh.sub_off[c])->roff[j] = sh.rc[j < kLB ? j : kLB][c];
    }
    for (int p = tid; p < HT; p += THREADS) {
        const uint32_t m = sh.mask[p];
        if (m == 0u) continue;
        // (numbered with atomics: the order varies from run to run, which moves records' contents about but changes no
        // result: every id's own sum is taken in coordinate order, in a shape that depends on the list's length alone)
        const uint32_t pc = (uint32_t)__popc(m);
        sh.soff[p] = (uint16_t)atomicAdd(&sh.cntAll, pc);
        if (m & (m - 1u)) {
            const int32_t id = sh.key[p];
            const int c = id & (C - 1);
            const uint32_t r = atomicAdd(&sh.cntTL2[c], (1u << 16) + pc);
            const uint32_t t = r >> 16, o = r & 0xffffu;
            unsigned char *rec = P.rec + sh.sub_off[c];
            const int n_c = sh.rc[kLB][c], T_c = sh.subT[c];
            uint32_t *ids_g = reinterpret_cast<uint32_t *>(rec + sizeof(SubHead) + 8u * n_c);
            uint16_t *off_g = reinterpret_cast<uint16_t *>(rec + sizeof(SubHead) + 8u * n_c + 4u * T_c + 2u * n_c);
            ids_g[t] = (uint32_t)id;
            off_g[t] = (uint16_t)o;
            sh.coff[p] = (uint16_t)o;
        }
    }
    if (tid < C) { // the end of the last list
        unsigned char *rec = P.rec + sh.sub_off[tid];
        const int n_c = sh.rc[kLB][tid], T_c = sh.subT[tid];
        reinterpret_cast<uint16_t *>(rec + sizeof(SubHead) + 8u * n_c + 4u * T_c + 2u * n_c)[T_c] = (uint16_t)(sh.cntTL[tid] & 0xffffu);
    }
    __syncthreads();
    PRE_T(4);
    // ---- the non-zeros into the workers' records, row after row: place = start of (coordinate, CTA) + rank among
    //      the coordinate's non-zeros of that CTA; a shared id's place in its list is the number of lower
    //      coordinates that have the id
    for (int j = warp; j < cnt; j += NW) {
        const int n = sh.nnz[j], r0 = sh.roff[j];
        int before[kMaxC];
#pragma unroll
        for (int c = 0; c < kMaxC; ++c) before[c] = sh.rc[j][c];
        for (int e0 = 0; e0 < n; e0 += 32) {
            const int e = e0 + lane;
            const bool on = e < n;
            const int32_t id = on ? sh.idx[r0 + e] : 0;
            const int cls = id & (C - 1);
            int place = 0;
#pragma unroll
            for (int c = 0; c < kMaxC; ++c) {
                if (c >= C) continue;
                const uint32_t bal = __ballot_sync(0xffffffffu, on && cls == c);
                if (cls == c) place = before[c] + __popc(bal & ((1u << lane) - 1u));
                before[c] += __popc(bal);
            }
            if (!on) continue;
            const int p = sh.slot[r0 + e];
            const uint32_t m = sh.mask[p];
            const bool shared_id = (m & (m - 1u)) != 0u;
            const int lower = __popc(m & ((1u << j) - 1u));
            const float x = sh.val[r0 + e];
            sh.lval[sh.soff[p] + lower] = x;
            unsigned char *rec = P.rec + sh.sub_off[cls];
            const int n_c = sh.rc[kLB][cls], T_c = sh.subT[cls];
            float *val_g = reinterpret_cast<float *>(rec + sizeof(SubHead));
            uint32_t *meta_g = reinterpret_cast<uint32_t *>(rec + sizeof(SubHead) + 4u * n_c);
            uint16_t *cpos_g = reinterpret_cast<uint16_t *>(rec + sizeof(SubHead) + 8u * n_c + 4u * T_c);
            val_g[place] = x;
            meta_g[place] = (uint32_t)id | ((uint32_t)j << kIdBits) | (shared_id ? 0x80000000u : 0u);
            cpos_g[place] = shared_id ? (uint16_t)(sh.coff[p] + lower) : (uint16_t)0;
            // for the Gram pass: the id itself is no longer needed, its mask and its list's start are (top bit: one of
            // the ids that the dense tiles cover)
            sh.idx[r0 + e] = (int32_t)m;
            sh.slot[r0 + e] = (uint16_t)(sh.soff[p] | (id < kHD ? 0x8000 : 0));
        }
    }
    __syncthreads();
    PRE_T(5);
    // ---- Gram triangle: a warp per coordinate j, lane l collects x_j . x_l over j's entries in ascending order. The
    //      lanes first look at 32 entries at once and keep those whose id an earlier coordinate has too; only these
    //      are then walked, their mask, list start and value handed round by shuffles.
    for (int j = warp; j < kLB; j += NW) {
        float acc = 0.0f;
        if (j < cnt) {
            const int n = sh.nnz[j], r0 = sh.roff[j];
            const uint32_t below = (1u << j) - 1u, lt = (1u << lane) - 1u;
            {
                const float4 *dj = reinterpret_cast<const float4 *>(&sh.Dc[j][0]);
                const float4 *dm = reinterpret_cast<const float4 *>(&sh.Dc[lane][0]);
#pragma unroll
                for (int h = 0; h < kHD / 4; ++h) {
                    const float4 a = dj[h], b4 = dm[h];
                    acc = fmaf(a.x, b4.x, acc); acc = fmaf(a.y, b4.y, acc); acc = fmaf(a.z, b4.z, acc); acc = fmaf(a.w, b4.w, acc);
                }
            }
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
                uint32_t todo = __ballot_sync(0xffffffffu, (m_l & below) != 0u && !(so_l & 0x8000)); // (not the dense ones)
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
            if (lane >= j) acc = 0.0f;
        }
        acc *= sh.gsc[j] * sh.ys[lane];
        sh.G[lane][j] = acc; // row l, column j
        float q0 = acc * sh.as[lane];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) q0 += __shfl_xor_sync(0xffffffffu, q0, o);
        if (lane == 0) sh.hdr[j].A -= q0;
    }
    PRE_T(6);
    // ---- cross Gram matrix with the next block: a warp per coordinate j of the next block, whose non-zeros come
    //      straight from the matrix and are looked up in this block's table; lane l collects x_j . x_l
    //      (the first 128 entries of a warp's next coordinate are loaded while it works on the current one)
    int32_t xids_nx[4];
    float xvals_nx[4];
    auto xload4 = [&](int j, int32_t (&ids)[4], float (&vals)[4]) {
        const bool have = carry && j < sh.ncnt;
        const int n = have ? sh.nnnz[j] : 0;
        const int64_t rs = have ? sh.nrs[j] : 0;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const int e = lane + 32 * c;
            ids[c] = e < n ? checked_id(P, P.S.indices[rs + e]) : -1;
            vals[c] = e < n ? P.S.values[rs + e] : 0.0f;
        }
    };
    xload4(warp, xids_nx, xvals_nx);
    for (int j = warp; j < kLB; j += NW) {
        float acc = 0.0f;
        int32_t ids4[4];
        float vals4[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) { ids4[c] = xids_nx[c]; vals4[c] = xvals_nx[c]; }
        xload4(j + NW, xids_nx, xvals_nx);
        if (carry && j < sh.ncnt) {
            const int n = sh.nnnz[j];
            const int64_t rs = sh.nrs[j];
            const uint32_t lt = (1u << lane) - 1u;
            int per_class[kMaxC];
#pragma unroll
            for (int c = 0; c < kMaxC; ++c) per_class[c] = 0;
            auto take = [&](int32_t id, float x_l) {
                uint32_t m_l = 0u;
                int so_l = 0;
#pragma unroll
                for (int c = 0; c < kMaxC; ++c)
                    if (c < C) per_class[c] += __popc(__ballot_sync(0xffffffffu, id >= 0 && (id & (C - 1)) == c));
                if (id >= 0 && id < kHD) sh.Dn[j][id] = x_l;
                else if (id >= 0) {
                    uint32_t p = home_slot<HT>(id);
                    for (int probe = 0; probe < HT; ++probe) {
                        const int32_t seen = sh.key[p];
                        if (seen == id) { m_l = sh.mask[p]; so_l = sh.soff[p]; break; }
                        if (seen == -1) break;
                        p = next_slot<HT>(p);
                    }
                }
                uint32_t todo = __ballot_sync(0xffffffffu, m_l != 0u);
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
            };
#pragma unroll
            for (int c = 0; c < 4; ++c)
                if (32 * c < n) take(ids4[c], vals4[c]);
            for (int e0 = 128; e0 < n; e0 += 32) {
                const int e = e0 + lane;
                take(e < n ? checked_id(P, P.S.indices[rs + e]) : -1, e < n ? P.S.values[rs + e] : 0.0f);
            }
            __syncwarp();
            {
                const float4 *dj = reinterpret_cast<const float4 *>(&sh.Dn[j][0]);
                const float4 *dm = reinterpret_cast<const float4 *>(&sh.Dc[lane][0]);
#pragma unroll
                for (int h = 0; h < kHD / 4; ++h) {
                    const float4 a = dj[h], b4 = dm[h];
                    acc = fmaf(a.x, b4.x, acc); acc = fmaf(a.y, b4.y, acc); acc = fmaf(a.z, b4.z, acc); acc = fmaf(a.w, b4.w, acc);
                }
            }
            if (lane >= cnt) acc = 0.0f;
            if (lane == 0) {
#pragma unroll
                for (int c = 0; c < kMaxC; ++c)
                    if (c < C && per_class[c]) atomicAdd(&sh.ncls[c], per_class[c]);
            }
        }
        acc *= sh.gscn[j] * sh.ys[lane];
        sh.X[lane][j] = acc; // row l (this block), column j (next block)
        float q0 = acc * sh.as[lane];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) q0 += __shfl_xor_sync(0xffffffffu, q0, o);
        if (lane == 0) sh.q0n[j] = q0;
    }
    __syncthreads();
    PRE_T(7);
    // (a next block that is walked in place because more of its non-zeros fall to one CTA than a record holds takes
    // nothing over either)
    bool keep = true;
#pragma unroll
    for (int c = 0; c < kMaxC; ++c)
        if (c < C && sh.ncls[c] > P.nzcap) keep = false;
    for (int i = tid; i < kLB * kLB; i += THREADS) {
        out.G[i] = sh.G[i >> 5][i & 31];
        out.X[i] = keep ? sh.X[i >> 5][i & 31] : 0.0f;
    }
    if (warp == 0) {
        out.hdr[lane] = sh.hdr[lane];
        out.q0n[lane] = keep ? sh.q0n[lane] : 0.0f;
    }
}

// A CTA takes blocks blockIdx.x, blockIdx.x + gridDim.x, ...: one each when the grid has a CTA per block; a launch
// beside the chain kernels gets a grid that fits the SMs they leave, so that it never has CTAs waiting for an SM (which
// would take the SMs of a finished chain launch before the next chain launch's CTAs, which need a whole SM each).
template <int LOSS, int NZ, int HT, int THREADS>
__global__ void __launch_bounds__(THREADS) k_lookahead_prepare(const LookParams P)
{
    extern __shared__ __align__(16) unsigned char smem_pre[];
    using Shared = PreShared<NZ, HT, THREADS>;
    Shared &sh = *reinterpret_cast<Shared *>(smem_pre);
    if (P.K < kBaseStaged) {
        for (int i = threadIdx.x; i <= P.K; i += THREADS) sh.base[i] = (int32_t)P.blk_base[i];
        __syncthreads();
    }
    for (int64_t bid = blockIdx.x; bid < P.n_blocks; bid += gridDim.x) {
        prepare_block<LOSS, NZ, HT, THREADS>(P, bid, sh);
        __syncthreads(); // the shared arrays are reused by the next block
    }
}

// Short dense rows: every row has every id, so the lists are implicit: constants, Gram triangle, cross Gram matrix
// and the rows themselves (one worker record: the model lives in one CTA).
constexpr int kPreThreads = 256;
struct PreDenseShared {
    float row[2 * kLB][kCapL + 1]; // this block's rows, then the next block's
    CHdr hdr[kLB];
    float gsc[kLB], ys[kLB], as[kLB], gscn[kLB];
    unsigned long long offset;
    uint32_t bytes;
    int32_t walk;
};

template <int LOSS> __device__ __forceinline__ void prepare_block_dense(const LookParams &P, const int64_t bid, PreDenseShared &sh)
{
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    constexpr int NW = kPreThreads / 32;
    int k;
    int64_t b;
    block_to_part(P, bid, k, b);
    const int64_t nk = P.S.part_off[k + 1] - P.S.part_off[k];
    const int64_t off = P.S.part_off[k] + (P.S.first_k ? P.S.first_k[k] : 0); // of this launch's first step in the order
    const int64_t steps = steps_of(P, k, nk);
    const int cnt = (int)((steps - b * kLB) < kLB ? (steps - b * kLB) : kLB);
    const int64_t left = steps - (b + 1) * kLB;
    const int ncnt = (left <= 0 || P.depth < 2) ? 0 : (left < kLB ? (int)left : kLB);
    const int dim = (int)P.S.dim;
    ChainHead &out = *reinterpret_cast<ChainHead *>(P.rec + (size_t)bid * sizeof(ChainHead));
    if (tid == 0) {
        const uint32_t bytes = sub_bytes(cnt * dim, 0, true);
        unsigned long long at = atomicAdd(P.cursor, (unsigned long long)bytes);
        BlkDir d;
        if (at + bytes > P.pool_cap) { // no room: walked in place
            d.offset = (unsigned long long)bid * sizeof(ChainHead);
            d.bytes = 16u;
            d.flags = 1u;
            sh.walk = 1;
        } else {
            d.offset = P.pool_off + at;
            d.bytes = bytes;
            d.flags = 0u;
            sh.walk = 0;
        }
        sh.offset = d.offset;
        if (bid == P.drop_block) d.bytes = 0u;
        P.dirS[bid] = d;
        out.cnt = cnt;
        out.flags = sh.walk;
        out.pad[0] = out.pad[1] = 0;
    }
    __syncthreads();
    const bool walk = sh.walk != 0;
    unsigned char *rec = P.rec + sh.offset;
    float *val_g = reinterpret_cast<float *>(rec + sizeof(SubHead));
    if (!walk && tid == 0) {
        SubHead &h = *reinterpret_cast<SubHead *>(rec);
        h.n = cnt * dim; h.T = 0; h.cnt = cnt; h.flags = 0;
    }
    if (!walk && tid < kLB + 8) reinterpret_cast<SubHead *>(rec)->roff[tid] = (uint16_t)((tid < cnt ? tid : cnt) * dim);
    for (int j = warp; j < 2 * kLB; j += NW) {
        const bool next = j >= kLB;
        const int jj = next ? j - kLB : j;
        const bool on = jj < (next ? ncnt : cnt);
        int32_t c = 0;
        if (on) c = P.S.perm[off + (b + (next ? 1 : 0)) * kLB + jj];
        if (!CHICLE_IN_BOUNDS(P.S.status, c >= 0 && (int64_t)c < P.S.n_coord)) c = 0;
        const int64_t rs = (int64_t)c * dim;
        for (int e = lane; e < dim; e += 32) {
            const float x = on ? P.S.values[rs + e] : 0.0f;
            sh.row[j][e] = x;
            if (on && !next && !walk) val_g[jj * dim + e] = x;
        }
        if (lane == 0) {
            CHdr hd{0, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
            if (on) hd = make_hdr<LOSS>(P.S, c);
            const float gs = on ? gram_scale<LOSS>(hd, P.S.sigma, P.S.inv_n) : 0.0f;
            if (next) sh.gscn[jj] = gs;
            else {
                sh.hdr[jj] = hd;
                sh.gsc[jj] = gs;
                sh.ys[jj] = LOSS == CHICLE_LOSS_RIDGE_PRIMAL ? 1.0f : hd.p3;
                sh.as[jj] = LOSS == CHICLE_LOSS_RIDGE_PRIMAL ? 0.0f : hd.p1;
            }
        }
    }
    __syncthreads();
    // a warp per column j; lane l has x_j . x_l: first inside the block (l < j), then from this block to the next
    for (int j = warp; j < 2 * kLB; j += NW) {
        const bool next = j >= kLB;
        const int jj = next ? j - kLB : j;
        float acc = 0.0f;
        if (!walk && (next ? lane < cnt : lane < jj))
            for (int e = 0; e < dim; ++e) acc = fmaf(sh.row[j][e], sh.row[lane][e], acc);
        acc *= (next ? sh.gscn[jj] : sh.gsc[jj]) * sh.ys[lane];
        (next ? out.X : out.G)[lane * kLB + jj] = acc;
        float q0 = acc * sh.as[lane];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) q0 += __shfl_xor_sync(0xffffffffu, q0, o);
        if (lane == 0) {
            if (next) out.q0n[jj] = q0;
            else sh.hdr[jj].A -= q0;
        }
    }
    __syncthreads();
    if (tid < kLB) out.hdr[tid] = sh.hdr[tid];
}

// (blocks blockIdx.x, blockIdx.x + gridDim.x, ...: see k_lookahead_prepare)
template <int LOSS> __global__ void __launch_bounds__(kPreThreads) k_lookahead_prepare_dense(const LookParams P)
{
    extern __shared__ __align__(16) unsigned char smem_pre[];
    PreDenseShared &sh = *reinterpret_cast<PreDenseShared *>(smem_pre);
    for (int64_t bid = blockIdx.x; bid < P.n_blocks; bid += gridDim.x) {
        prepare_block_dense<LOSS>(P, bid, sh);
        __syncthreads();
    }
}

// ------------------------------------------------------------------------------------------------ chain
// Cluster plumbing. Addresses in another CTA's shared memory come from mapa; data and the signal that it has landed
// travel together: an asynchronous store completes bytes on the receiver's mbarrier (no multicast anywhere).
__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t mapa_u32(uint32_t addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
// Data and the signal that it has landed travel together: an asynchronous store completes bytes on the receiver's
// mbarrier, straight from registers.
__device__ __forceinline__ void st_async_f32(uint32_t remote, float v, uint32_t remote_bar)
{
    asm volatile("st.async.shared::cluster.mbarrier::complete_tx::bytes.f32 [%0], %1, [%2];" ::"r"(remote), "f"(v), "r"(remote_bar)
                 : "memory");
}
__device__ __forceinline__ void st_async_f32x4_if(uint32_t remote, float a, float b, float c, float d, uint32_t remote_bar, bool on)
{
    asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.u32 q, %6, 0;\n\t"
                 "@q st.async.shared::cluster.mbarrier::complete_tx::bytes.v4.f32 [%0], {%1, %2, %3, %4}, [%5];\n\t}" ::"r"(remote),
                 "f"(a), "f"(b), "f"(c), "f"(d), "r"(remote_bar), "r"((uint32_t)on)
                 : "memory");
}
// Operations of a single lane as predicated instructions, not branches: a warp whose lanes part ways before a loop
// of shuffles may run the loop as separate groups of lanes that meet again at every shuffle (measured: 125 cycles per
// shuffle instead of 30 in the recurrence warp).
__device__ __forceinline__ void bulk_g2s_if(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar, bool on)
{
    asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.u32 q, %4, 0;\n\t"
                 "@q cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n\t}" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar), "r"((uint32_t)on)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx_if(uint32_t bar, uint32_t bytes, bool on)
{
    asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.u32 q, %2, 0;\n\t@q mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n\t}" ::"r"(bar),
                 "r"(bytes), "r"((uint32_t)on)
                 : "memory");
}
__device__ __forceinline__ float ld_cluster_f32(uint32_t remote)
{
    float v;
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(remote) : "memory");
    return v;
}
__device__ __forceinline__ void st_cluster_f32(uint32_t remote, float v)
{
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(remote), "f"(v) : "memory");
}
__device__ __forceinline__ void mbar_arrive_remote_release(uint32_t remote_bar)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(remote_bar) : "memory");
}
__device__ __forceinline__ void fence_cluster() { asm volatile("fence.acq_rel.cluster;" ::: "memory"); }
// One look at an mbarrier; the hardware may suspend the thread for up to `hint_ns` until the phase completes. The data
// that the pipeline's barriers guard is written into this CTA's shared memory by asynchronous stores and copies that
// complete on the barrier itself, so the default scope serves (as for a bulk copy); the two waits of the rare
// walked-in-place path, which order ordinary stores of another CTA, add a cluster-scope fence of their own.
__device__ __forceinline__ uint32_t mbar_try_wait_cluster(uint32_t a, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(a), "r"(parity), "r"(100000u)
        : "memory");
    return ok;
}
// Bounded wait of one warp on an mbarrier that another CTA of the cluster completes (every lane must call it). No
// pauses of its own (try_wait suspends the thread for a while by itself; the waits of the pipeline are short and on
// its critical path); gives up after about a second, or when the CTA is aborting. The result is the same on all
// lanes. One warp per CTA waits this way at a time.
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile int *abort_flag, uint32_t *status)
{
    // every lane looks at the barrier (one instruction for the warp either way) and the lanes agree by a vote, so
    // that the warp stays together
    if (__all_sync(0xffffffffu, mbar_try_wait_cluster(bar, parity) != 0u)) return true;
    const long long t_start = clock64();
    for (;;) {
        bool ok = false;
        for (int it = 0; it < 64 && !ok; ++it) ok = __all_sync(0xffffffffu, mbar_try_wait_cluster(bar, parity) != 0u);
        if (ok) return true;
        const bool stop = __any_sync(0xffffffffu, *abort_flag != 0);
        const bool late = __any_sync(0xffffffffu, clock64() - t_start > 2500000000ll); // more than a second at any clock
        if (stop || late) {
            if (!stop && (threadIdx.x & 31) == 0) {
                *abort_flag = 1;
                atomicOr(status, ST_WAIT_TIMEOUT);
            }
            __syncwarp();
            return false;
        }
    }
}
// The worker warps' barrier, with a vote: all of them take the same decision after a wait.
__device__ __forceinline__ bool work_bar_and(bool ok)
{
    uint32_t r;
    asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %1, 0;\n\tbar.red.and.pred p, %2, %3, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(r)
                 : "r"((uint32_t)ok), "n"(kBarWork), "n"(kWorkThreads)
                 : "memory");
    return r != 0;
}
__device__ __forceinline__ void work_bar()
{
    asm volatile("bar.sync %0, %1;" ::"n"(kBarWork), "n"(kWorkThreads) : "memory");
}

struct alignas(16) ChainCtl {
    uint64_t subfull[kSubSlots];   // count the bytes of the bulk copies into the workers' record slots
    uint64_t headfull[kHeadSlots]; // the same for the recurrence warp's records (CTA 0)
    uint64_t pbar[2];              // CTA 0: the partial dot products of a block have arrived from all CTAs
    uint64_t dbar[2];              // a block's deltas have arrived from CTA 0
    uint64_t ackbar;               // CTA 0: every CTA has applied all updates (before a block is walked in place)
    alignas(16) float pbuf[2][kMaxC][kLB];
    alignas(16) float dbuf[2][kLB];
    float sink[32]; // where a lane's stores go that have no target
    int abort_flag;
    int done; // the CTA's workers are through (the warps with no role sleep until then)
};

// Shared-memory layout of the chain kernel (sizes fixed at launch): control, recurrence records, worker records,
// products, the CTA's part of the model.
struct ChainLayout {
    uint32_t heads, subs, sub_stride, prod, w, total;
};
__host__ __device__ inline ChainLayout chain_layout(int nzcap, int hotc, bool dense, int dim)
{
    ChainLayout L;
    L.heads = (uint32_t)((sizeof(ChainCtl) + 127) & ~(size_t)127);
    L.subs = L.heads + kHeadSlots * (uint32_t)sizeof(ChainHead);
    L.sub_stride = dense ? sub_bytes(kLB * dim, 0, true) : sub_bytes(nzcap, nzcap / 2, false);
    L.prod = L.subs + kSubSlots * L.sub_stride;
    L.w = L.prod + 4u * (uint32_t)(dense ? kLB : nzcap);
    L.total = L.w + 4u * (uint32_t)(hotc > 0 ? hotc : 4);
    return L;
}

template <int LOSS, bool DENSE>
__global__ void __launch_bounds__(kChainThreads, 1) k_lookahead_chain(const LookParams P)
{
    extern __shared__ __align__(128) unsigned char smem_chain[];
    const SolverParams &S = P.S;
    const int logC = P.logC, C = 1 << logC;
    const uint32_t crank = cluster_ctarank();
    const int k = (int)(blockIdx.x >> logC);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const ChainLayout L = chain_layout(P.nzcap, P.hotc, DENSE, (int)S.dim);
    ChainCtl &ctl = *reinterpret_cast<ChainCtl *>(smem_chain);
    float *W = reinterpret_cast<float *>(smem_chain + L.w);
    float *prod = reinterpret_cast<float *>(smem_chain + L.prod);
    volatile int *abort_flag = &ctl.abort_flag;

    const int64_t nk = S.part_off[k + 1] - S.part_off[k];
    const int64_t steps = steps_of(P, k, nk);
    const int64_t nb = (steps + kLB - 1) / kLB;
    const int64_t bid0 = P.blk_base[k];
    float *Uk = S.U + (size_t)k * (size_t)S.dim;
    const float sigma = S.sigma;
    // entry ids below hot_total live in shared memory: id g in CTA g mod C at place g / C
    const int64_t hot_all = (int64_t)P.hotc << logC;
    const uint32_t hot_total = (uint32_t)(hot_all < S.dim ? hot_all : S.dim);
    const int hot_mine = hot_total > crank ? (int)((hot_total - crank + C - 1) >> logC) : 0;

    if (tid == 0) {
        ctl.abort_flag = 0;
        ctl.done = 0;
        for (int i = 0; i < kSubSlots; ++i) mbar_init(smem_u32(&ctl.subfull[i]), 1);
        for (int i = 0; i < kHeadSlots; ++i) mbar_init(smem_u32(&ctl.headfull[i]), 1);
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&ctl.pbar[i]), 1);
            mbar_init(smem_u32(&ctl.dbar[i]), 1);
        }
        mbar_init(smem_u32(&ctl.ackbar), (uint32_t)C);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        // armed for the first two blocks before anybody can send
        for (int i = 0; i < 2; ++i) {
            mbar_arrive_expect_tx(smem_u32(&ctl.pbar[i]), (uint32_t)(C * kLB * 4));
            mbar_arrive_expect_tx(smem_u32(&ctl.dbar[i]), (uint32_t)(kLB * 4));
        }
    }
    for (int l = tid; l < hot_mine; l += kChainThreads) {
        const size_t g = ((size_t)l << logC) + crank;
        W[l] = P.model_in ? fmaf(sigma, Uk[g], S.vbase[g]) : Uk[g];
    }
    // the ids beyond the part in shared memory that fall to this CTA (id mod C): the model in place
    const size_t cold0 = (size_t)hot_total + (((size_t)crank - (size_t)hot_total) & (size_t)(C - 1));
    if (P.model_in)
        for (size_t g = cold0 + ((size_t)tid << logC); g < (size_t)S.dim; g += (size_t)kChainThreads << logC)
            Uk[g] = fmaf(sigma, Uk[g], S.vbase[g]);
    __syncthreads();
    cluster_arrive();
    cluster_wait();

    const bool is_chain = crank == 0 && warp == 0;
    const bool is_worker = (warp & 3) != 0;
    bool aborted = false;

    if (is_chain && nb > 0) {
        // ============================== the recurrence warp =====================================================
        const int q = lane & 7, rep = lane >> 3;
        auto head_at = [&](int64_t blk) { return reinterpret_cast<const ChainHead *>(smem_chain + L.heads + (size_t)(blk % kHeadSlots) * sizeof(ChainHead)); };
        auto issue_head = [&](int64_t blk) {
            const bool on = blk < nb && lane == 0;
            const int64_t at = blk < nb ? blk : nb - 1;
            const uint32_t bar = smem_u32(&ctl.headfull[at % kHeadSlots]);
            mbar_arrive_expect_tx_if(bar, (uint32_t)sizeof(ChainHead), on);
            bulk_g2s_if(smem_u32(head_at(at)), P.rec + (size_t)(bid0 + at) * sizeof(ChainHead), (uint32_t)sizeof(ChainHead), bar, on);
        };
        for (int i = 0; i < kHeadSlots; ++i) issue_head(i);
        // where the deltas go: the copy `rep` of lane q sends the lane's four values to CTAs rep and rep + 4
        uint32_t d_dst[2], d_bar[2];
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const uint32_t c = (uint32_t)(rep + 4 * i) & (uint32_t)(C - 1);
            d_dst[i] = mapa_u32(smem_u32(&ctl.dbuf[0][4 * q]), c);
            d_bar[i] = mapa_u32(smem_u32(&ctl.dbar[0]), c);
        }
        float xs[4] = {0.f, 0.f, 0.f, 0.f}; // what the block before contributes to this block's states
        int64_t fp = 0, sc = 0;            // staged blocks and walked blocks so far
#ifdef CHICLE_LA_TIMING
        long long tw = 0, tr = 0, te = 0, t0 = clock64(), t1 = 0;
#endif
        for (int64_t b = 0; b < nb; ++b) {
            if (!mbar_wait_cluster(smem_u32(&ctl.headfull[b % kHeadSlots]), (uint32_t)(b / kHeadSlots) & 1u, abort_flag, S.status)) { aborted = true; break; }
            const ChainHead &H = *head_at(b);
            const int cnt = H.cnt;
            const uint32_t par = (uint32_t)(b & 1);
            if (H.flags & 1) {
                // ---- walked in place: wait until every CTA has applied all earlier updates, then coordinate by
                //      coordinate against the whole model (the other CTAs' parts through the cluster's shared memory)
                if (!mbar_wait_cluster(smem_u32(&ctl.ackbar), (uint32_t)sc & 1u, abort_flag, S.status)) { aborted = true; break; }
                fence_cluster(); // the other CTAs' updates of their parts of the model, made by ordinary stores
                ++sc;
                const uint32_t w_base = smem_u32(W);
                for (int j = 0; j < cnt; ++j) {
                    const CHdr h = H.hdr[j];
                    if (!CHICLE_IN_BOUNDS(S.status, h.coord >= 0 && (int64_t)h.coord < S.n_coord)) continue;
                    const int64_t rs = DENSE ? (int64_t)h.coord * S.dim : S.indptr[h.coord];
                    int n = DENSE ? (int)S.dim : (int)(S.indptr[h.coord + 1] - rs);
                    if (!CHICLE_IN_BOUNDS(S.status, DENSE || (rs >= 0 && n >= 0 && rs + n <= P.nnz))) n = 0;
                    const int32_t *ix = S.indices + rs;
                    const float *xv = S.values + rs;
                    float acc = 0.0f, delta, new_state;
                    for (int e = lane; e < n; e += 32) {
                        uint32_t g = DENSE ? (uint32_t)e : (uint32_t)ix[e];
                        if (!CHICLE_IN_BOUNDS(S.status, (int64_t)g < S.dim)) g = 0u;
                        const float ww = g < hot_total ? ld_cluster_f32(mapa_u32(w_base + 4u * (g >> logC), g & (uint32_t)(C - 1)))
                                                       : __ldcg(Uk + g);
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
                        for (int e = lane; e < n; e += 32) {
                            uint32_t g = DENSE ? (uint32_t)e : (uint32_t)ix[e];
                            if (!CHICLE_IN_BOUNDS(S.status, (int64_t)g < S.dim)) continue;
                            if (g < hot_total) {
                                const uint32_t a = mapa_u32(w_base + 4u * (g >> logC), g & (uint32_t)(C - 1));
                                st_cluster_f32(a, fmaf(sigma * delta, xv[e], ld_cluster_f32(a)));
                            } else Uk[g] = fmaf(sigma * delta, xv[e], __ldcg(Uk + g));
                        }
                    if (lane == 0) S.alpha[h.coord] = new_state;
                    __syncwarp();
                }
                // the walk's writes before the signal; the signal is a block of zero deltas
                __threadfence();
                fence_cluster();
                __syncwarp();
#pragma unroll
                for (int i = 0; i < 2; ++i)
                    st_async_f32x4_if(d_dst[i] + par * (uint32_t)(kLB * 4), 0.f, 0.f, 0.f, 0.f, d_bar[i] + par * 8u, rep + 4 * i < C);
                xs[0] = xs[1] = xs[2] = xs[3] = 0.0f;
            } else {
                // ---- four coordinates at a time. Lane q (and its copies q + 8, q + 16, q + 24, which compute the
                //      same) keeps the states of coordinates 4q .. 4q + 3. Group g: its lane walks its four coordinates
                //      by itself, the four results are handed round, and every lane adds what they mean for its own
                //      four, in this block and in the next.
                float hp1[4], hp2[4], hp3[4], hlq[4], s[4], mine[4];
                int32_t hcoord[4];
                float hA[4], hB[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const CHdr &h = H.hdr[4 * q + i];
                    hcoord[i] = h.coord; hp1[i] = h.p1; hp2[i] = h.p2; hp3[i] = h.p3; hlq[i] = h.lq; hA[i] = h.A; hB[i] = h.B;
                    mine[i] = 0.0f;
                }
                const float4 q0n = *reinterpret_cast<const float4 *>(&H.q0n[4 * q]);
                if (!mbar_wait_cluster(smem_u32(&ctl.pbar[fp & 1]), (uint32_t)(fp >> 1) & 1u, abort_flag, S.status)) { aborted = true; break; }
                LA_T(tw);
                float m0[4] = {0.f, 0.f, 0.f, 0.f};
                for (int c = 0; c < C; ++c) { // the CTAs' partial sums in a fixed order
                    const float4 pv = *reinterpret_cast<const float4 *>(&ctl.pbuf[fp & 1][c][4 * q]);
                    m0[0] += pv.x; m0[1] += pv.y; m0[2] += pv.z; m0[3] += pv.w;
                }
                __syncwarp();
#pragma unroll
                for (int i = 0; i < 4; ++i) s[i] = fmaf(hB[i], m0[i], hA[i]) + xs[i];
                xs[0] = -q0n.x; xs[1] = -q0n.y; xs[2] = -q0n.z; xs[3] = -q0n.w;
                const float4 *G4 = reinterpret_cast<const float4 *>(H.G); // G4[l * 8 + q]: row l, columns 4q .. 4q + 3
                const float4 *X4 = reinterpret_cast<const float4 *>(H.X);
#pragma unroll
                for (int g = 0; g < kLB / 4; ++g) {
                    float4 blk[4], nxt[4];
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) {
                        blk[kk] = G4[(4 * g + kk) * 8 + q];
                        nxt[kk] = X4[(4 * g + kk) * 8 + q];
                    }
                    // inside the group (the numbers matter on the lanes with q == g, where blk holds the group's own
                    // triangle; the others run the same instructions on copies)
                    float o[4];
                    o[0] = recurrence_map<LOSS>(s[0], hp2[0], hlq[0]);
                    const float t1 = fmaf(o[0], blk[0].y, s[1]);
                    o[1] = recurrence_map<LOSS>(t1, hp2[1], hlq[1]);
                    const float t2 = fmaf(o[1], blk[1].z, fmaf(o[0], blk[0].z, s[2]));
                    o[2] = recurrence_map<LOSS>(t2, hp2[2], hlq[2]);
                    const float t3 = fmaf(o[2], blk[2].w, fmaf(o[1], blk[1].w, fmaf(o[0], blk[0].w, s[3])));
                    o[3] = recurrence_map<LOSS>(t3, hp2[3], hlq[3]);
#pragma unroll
                    for (int i = 0; i < 4; ++i) mine[i] = q == g ? o[i] : mine[i];
                    float og[4];
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) og[kk] = __shfl_sync(0xffffffffu, o[kk], g);
                    // (zero entries of the triangle make this a no-op for the groups at or before g, whose states are final)
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) {
                        s[0] = fmaf(og[kk], blk[kk].x, s[0]);
                        s[1] = fmaf(og[kk], blk[kk].y, s[1]);
                        s[2] = fmaf(og[kk], blk[kk].z, s[2]);
                        s[3] = fmaf(og[kk], blk[kk].w, s[3]);
                        xs[0] = fmaf(og[kk], nxt[kk].x, xs[0]);
                        xs[1] = fmaf(og[kk], nxt[kk].y, xs[1]);
                        xs[2] = fmaf(og[kk], nxt[kk].z, xs[2]);
                        xs[3] = fmaf(og[kk], nxt[kk].w, xs[3]);
                    }
                }
                LA_T(tr);
                float dl[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int j = 4 * q + i;
                    float my_delta = 0.0f;
                    if (j < cnt) {
                        float my_state;
                        if (LOSS == CHICLE_LOSS_RIDGE_PRIMAL) {
                            my_delta = mine[i];
                            my_state = hp1[i] + mine[i];
                        } else {
                            my_delta = hp3[i] * (mine[i] - hp1[i]);
                            my_state = hp3[i] * mine[i];
                        }
                        if (!(fabsf(my_delta) <= CUDART_MAX_NORMAL_F)) {
                            atomicOr(S.status, ST_NONFINITE_STEP);
                            my_delta = 0.0f;
                            my_state = LOSS == CHICLE_LOSS_RIDGE_PRIMAL ? hp1[i] : hp3[i] * hp1[i];
                        }
                        if (CHICLE_IN_BOUNDS(S.status, hcoord[i] >= 0 && (int64_t)hcoord[i] < S.n_coord))
                            S.alpha[hcoord[i]] = my_state; // (the four copies of a lane store the same value)
                    }
                    dl[i] = my_delta;
                }
                // armed for block fp + 2 before the deltas go out (its dot products are sent only after they arrive)
                mbar_arrive_expect_tx_if(smem_u32(&ctl.pbar[fp & 1]), (uint32_t)(C * kLB * 4), lane == 0);
#pragma unroll
                for (int i = 0; i < 2; ++i)
                    st_async_f32x4_if(d_dst[i] + par * (uint32_t)(kLB * 4), dl[0], dl[1], dl[2], dl[3], d_bar[i] + par * 8u, rep + 4 * i < C);
                ++fp;
                LA_T(te);
            }
            __syncwarp();
            issue_head(b + kHeadSlots);
        }
#ifdef CHICLE_LA_TIMING
        if (blockIdx.x == 0 && lane == 0) {
            unsigned long long *d = P.timing;
            d[0] = tw; d[1] = tr; d[2] = te; d[3] = nb;
        }
#endif
    }
    if (is_worker && nb > 0) {
        // ============================== the worker warps ========================================================
        const int wt = (warp - 1 - (warp >> 2)) * 32 + lane; // 0 .. kWorkThreads - 1
        const uint32_t p_bar0 = mapa_u32(smem_u32(&ctl.pbar[0]), 0u);
        const uint32_t p_buf0 = mapa_u32(smem_u32(&ctl.pbuf[0][crank][0]), 0u);
        const uint32_t ack_bar = mapa_u32(smem_u32(&ctl.ackbar), 0u);
        const int dim = (int)S.dim;
        auto sub_at = [&](int64_t blk) { return smem_chain + L.subs + (size_t)(blk & (kSubSlots - 1)) * L.sub_stride; };
        // The directory entry of a block is loaded a block ahead of its use (an unconditional load from a clamped
        // address, so that nothing has to wait for it at the point of issue).
        auto load_dir = [&](int64_t blk, uint32_t (&d)[4]) {
            const int64_t at = blk < nb ? blk : nb - 1;
            asm volatile("ld.global.v4.u32 {%0, %1, %2, %3}, [%4];"
                         : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
                         : "l"(P.dirS + (((bid0 + at) << logC) + crank))
                         : "memory");
        };
        auto issue_sub = [&](int64_t blk, const uint32_t (&d)[4]) {
            const uint32_t bar = smem_u32(&ctl.subfull[blk & (kSubSlots - 1)]);
            // (the slot is only ever written by the copy engine and read by loads that are done by now)
            const unsigned long long offset = ((unsigned long long)d[1] << 32) | d[0];
            uint32_t bytes = d[2] <= L.sub_stride ? d[2] : 0u;
            if (!CHICLE_IN_BOUNDS(S.status, (offset & 15ull) == 0ull && offset + bytes <= P.pool_off + P.pool_cap))
                bytes = 0u; // (an entry that points outside the region: as if no record had been written)
            const bool mine = blk < nb && wt == 0;
            if (mine && bytes == 0) {
                // no record: nothing will arrive, say so now
                atomicOr(S.status, ST_WAIT_TIMEOUT);
                *abort_flag = 1;
            }
            mbar_arrive_expect_tx_if(bar, bytes, mine && bytes != 0);
            bulk_g2s_if(smem_u32(sub_at(blk)), P.rec + offset, bytes, bar, mine && bytes != 0);
        };
        // which of the blocks b .. b + 3 are walked in place
        bool sl0, sl1, sl2, sl3;
        {
            uint32_t d[4];
            load_dir(0, d); issue_sub(0, d); sl0 = (d[3] & 1u) != 0u;
            load_dir(1, d); issue_sub(1, d); sl1 = nb > 1 && (d[3] & 1u) != 0u;
            load_dir(2, d); issue_sub(2, d); sl2 = nb > 2 && (d[3] & 1u) != 0u;
            load_dir(3, d); issue_sub(3, d); sl3 = nb > 3 && (d[3] & 1u) != 0u;
        }
        int64_t fg = 0; // staged blocks whose dot products have been sent
        bool failed = false; // this warp gave up a wait (voted on at the next barrier)
#ifdef CHICLE_LA_TIMING
        long long wd = 0, ws = 0, wg = 0, ws1 = 0, wg0 = 0, wg1 = 0, t0 = clock64(), t1 = 0;
#endif

        // Block x's dot products against the model as it is now (this CTA's part), sent to CTA 0.
        auto take_dots = [&](int64_t x) -> bool {
            // Every warp waits for the record by itself (a barrier costs more than 200 cycles); a warp whose wait runs out
            // skips the work and says so at the next barrier's vote, so that all warps still meet there.
            bool ok = mbar_wait_cluster(smem_u32(&ctl.subfull[x & (kSubSlots - 1)]), (uint32_t)(x >> 2) & 1u, abort_flag, S.status);
            if (DENSE) ok = work_bar_and(ok); // (dense rows: the products of the call before have been read)
            if (!ok) {
                failed = true;
                ++fg;
                return !DENSE;
            }
            LA_T(wg0);
            const unsigned char *rec = sub_at(x);
            const SubHead &h = *reinterpret_cast<const SubHead *>(rec);
            // (debug build) a record whose sizes do not fit its slot is not read: as if its wait had run out
            if (!CHICLE_IN_BOUNDS(S.status, h.cnt >= 0 && h.cnt <= kLB &&
                                                (DENSE || (h.n >= 0 && h.n <= P.nzcap && h.T >= 0 && h.T <= P.nzcap / 2 && h.roff[kLB] == h.n)))) {
                failed = true;
                ++fg;
                return !DENSE;
            }
            const float *val = reinterpret_cast<const float *>(rec + sizeof(SubHead));
            const uint32_t slot = (uint32_t)(fg & 1);
            if (DENSE) {
                if (wt < kLB * 8) {
                    const int j = wt >> 3, qq = wt & 7;
                    float acc = 0.0f;
                    if (j < h.cnt)
                        for (int e = qq; e < dim; e += 8) acc = fmaf(val[j * dim + e], W[e], acc);
                    acc += __shfl_xor_sync(0xffffffffu, acc, 1);
                    acc += __shfl_xor_sync(0xffffffffu, acc, 2);
                    acc += __shfl_xor_sync(0xffffffffu, acc, 4);
                    if (qq == 0) prod[j] = acc;
                }
                work_bar();
                if (wt < kLB) {
                    st_async_f32(p_buf0 + (slot * (uint32_t)(kMaxC * kLB) + (uint32_t)wt) * 4u, prod[wt], p_bar0 + slot * 8u);
                }
            } else {
                const int n = h.n;
                const uint32_t *meta = reinterpret_cast<const uint32_t *>(val + n);
                // Eight threads per coordinate, each its every eighth non-zero: the first two with all loads issued
                // before anything is used. Ids below hot_total from shared memory; the others from row k of the
                // update workspace (read at L2: the updates are made there by reductions) and from v.
                if (wt < kLB * 8 && hot_total == 0u) {
                    // (no id in shared memory: every gather goes to L2, eight per thread in flight)
                    const int j = wt >> 3, qq = wt & 7;
                    const int lo = h.roff[j] + qq, hi = h.roff[j + 1];
                    float acc = 0.0f;
                    for (int e0 = lo; e0 < hi; e0 += 64) {
                        float x8[8], u8[8];
#pragma unroll
                        for (int u = 0; u < 8; ++u) {
                            const int e = e0 + 8 * u;
                            const bool on = e < hi;
                            x8[u] = on ? val[e] : 0.0f;
                            const uint32_t g = on ? (meta[e] & kIdMask) : 0u;
                            u8[u] = ldcg_if(Uk + g, on && CHICLE_IN_BOUNDS(S.status, (int64_t)g < S.dim));
                        }
#pragma unroll
                        for (int u = 0; u < 8; ++u) acc = fmaf(x8[u], u8[u], acc);
                    }
                    acc += __shfl_xor_sync(0xffffffffu, acc, 1);
                    acc += __shfl_xor_sync(0xffffffffu, acc, 2);
                    acc += __shfl_xor_sync(0xffffffffu, acc, 4);
                    if (qq == 0) st_async_f32(p_buf0 + (slot * (uint32_t)(kMaxC * kLB) + (uint32_t)j) * 4u, acc, p_bar0 + slot * 8u);
                } else if (wt < kLB * 8) {
                    const int j = wt >> 3, qq = wt & 7;
                    const int lo = h.roff[j] + qq, hi = h.roff[j + 1];
                    float x[2], hv[2], uu[2];
                    bool cold[2];
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                        const int e = lo + 8 * u;
                        const bool on = e < hi;
                        x[u] = on ? val[e] : 0.0f;
                        const uint32_t g = on ? (meta[e] & kIdMask) : 0u;
                        cold[u] = on && g >= hot_total && CHICLE_IN_BOUNDS(S.status, (int64_t)g < S.dim);
                        hv[u] = W[g < hot_total ? (g >> logC) : 0u];
                        uu[u] = ldcg_if(Uk + (cold[u] ? g : 0u), cold[u]);
                    }
                    float acc = x[0] * (cold[0] ? uu[0] : hv[0]);
                    acc = fmaf(x[1], cold[1] ? uu[1] : hv[1], acc);
                    // (longer coordinates: four at a time, again with all loads first: an id beyond the part of the
                    // model in shared memory costs a round trip to L2, which the four share)
                    for (int e0 = lo + 16; e0 < hi; e0 += 32) {
                        float x4[4], h4[4], u4[4];
                        bool c4[4];
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const int e = e0 + 8 * u;
                            const bool on = e < hi;
                            x4[u] = on ? val[e] : 0.0f;
                            const uint32_t g = on ? (meta[e] & kIdMask) : 0u;
                            c4[u] = on && g >= hot_total && CHICLE_IN_BOUNDS(S.status, (int64_t)g < S.dim);
                            h4[u] = W[g < hot_total ? (g >> logC) : 0u];
                            u4[u] = ldcg_if(Uk + (c4[u] ? g : 0u), c4[u]);
                        }
#pragma unroll
                        for (int u = 0; u < 4; ++u) acc = fmaf(x4[u], c4[u] ? u4[u] : h4[u], acc);
                    }
                    acc += __shfl_xor_sync(0xffffffffu, acc, 1);
                    acc += __shfl_xor_sync(0xffffffffu, acc, 2);
                    acc += __shfl_xor_sync(0xffffffffu, acc, 4);
                    if (qq == 0) st_async_f32(p_buf0 + (slot * (uint32_t)(kMaxC * kLB) + (uint32_t)j) * 4u, acc, p_bar0 + slot * 8u);
                }
                LA_T(wg1);
            }
            ++fg;
            return true;
        };

        // The loop starts `depth` blocks early: those turns only take the first blocks' dot products (one place in the
        // code for every phase keeps the loop small: the warps run at the pace instructions can be fetched).
        const int depth = P.depth;
        if (depth == 2) { sl2 = sl0; sl3 = sl1; sl0 = false; sl1 = false; } // flags of blocks b .. b + 3 for b = -2
        else { sl3 = sl2; sl2 = sl1; sl1 = sl0; sl0 = false; }              // ... for b = -1
#pragma unroll 1
        for (int64_t b = -depth; b < nb && !aborted; ++b) {
            uint32_t dn[4];
            load_dir(b + kSubSlots, dn);
            const uint32_t par = (uint32_t)(b & 1);
            if (b < 0) {
            } else if (sl0) {
                // walked in place by CTA 0: every update before it has been applied here (the barrier that ended
                // the block before); say so, and wait for the walk to end
                if (wt == 0) mbar_arrive_remote_release(ack_bar);
                bool ok = !failed && (wt >= 32 || mbar_wait_cluster(smem_u32(&ctl.dbar[par]), (uint32_t)(b >> 1) & 1u, abort_flag, S.status));
                if (wt < 32) fence_cluster(); // the walk's ordinary stores into this CTA's part of the model
                ok = work_bar_and(ok);
                if (!ok) { aborted = true; break; }
            } else {
                bool ok = !failed && (wt >= 32 || mbar_wait_cluster(smem_u32(&ctl.dbar[par]), (uint32_t)(b >> 1) & 1u, abort_flag, S.status));
                ok = work_bar_and(ok);
                if (!ok) { aborted = true; break; }
                LA_T(wd);
                // ---- block b's update of this CTA's part of the model
                const float *dl = ctl.dbuf[par];
                const unsigned char *rec = sub_at(b);
                const SubHead &h = *reinterpret_cast<const SubHead *>(rec);
                const float *val = reinterpret_cast<const float *>(rec + sizeof(SubHead));
                if (DENSE) {
                    if (wt < dim) {
                        float sum = 0.0f;
                        const int cnt = h.cnt;
#pragma unroll 8
                        for (int j = 0; j < cnt; ++j) sum = fmaf(dl[j], val[j * dim + wt], sum);
                        W[wt] = fmaf(sigma, sum, W[wt]);
                    }
                } else {
                    const int n = h.n, T = h.T;
                    const uint32_t *meta = reinterpret_cast<const uint32_t *>(val + n);
                    const uint32_t *ids = meta + n;
                    const uint16_t *cpos = reinterpret_cast<const uint16_t *>(ids + T);
                    const uint16_t *offs = cpos + n;
                    // (A) eight threads per coordinate. A non-zero whose id no other coordinate of the block has is
                    //     applied at once (no two of a block's non-zeros touch the same word then); the others leave
                    //     their product delta_j * x at their place in the id's list. One store per non-zero, its
                    //     address chosen without a branch: the list place, the model word, or a word that nobody reads;
                    //     ids beyond the part in shared memory add to the workspace row instead.
                    if (wt < kLB * 8 && hot_total == 0u) {
                        // (no id in shared memory: a list place or a reduction at L2, eight non-zeros per turn)
                        const int j = wt >> 3, qq = wt & 7;
                        const int lo = h.roff[j] + qq, hi = h.roff[j + 1];
                        const float d = dl[j];
                        const uint32_t a_prod = smem_u32(prod), a_sink = smem_u32(&ctl.sink[lane]);
                        for (int e0 = lo; e0 < hi; e0 += 64) {
                            uint32_t m8[8];
                            float p8[8];
                            int c8[8];
#pragma unroll
                            for (int u = 0; u < 8; ++u) {
                                const int e = e0 + 8 * u;
                                const bool on = e < hi;
                                m8[u] = on ? meta[e] : 0u;
                                p8[u] = on ? d * val[e] : 0.0f;
                                c8[u] = on ? cpos[e] : 0;
                            }
#pragma unroll
                            for (int u = 0; u < 8; ++u) {
                                const bool shared_id = (m8[u] >> 31) != 0u && CHICLE_IN_BOUNDS(S.status, c8[u] < P.nzcap);
                                sts_f32(shared_id ? a_prod + 4u * (uint32_t)c8[u] : a_sink, p8[u]);
                                const bool far = (m8[u] >> 31) == 0u && p8[u] != 0.0f && // (beyond the coordinate's end p8 is 0)
                                                 CHICLE_IN_BOUNDS(S.status, (int64_t)(m8[u] & kIdMask) < S.dim);
                                red_add_if(Uk + (far ? (m8[u] & kIdMask) : 0u), sigma * p8[u], far);
                            }
                        }
                    } else if (wt < kLB * 8) {
                        const int j = wt >> 3, qq = wt & 7;
                        const int lo = h.roff[j] + qq, hi = h.roff[j + 1];
                        const float d = dl[j];
                        const uint32_t a_prod = smem_u32(prod), a_w = smem_u32(W), a_sink = smem_u32(&ctl.sink[lane]);
                        uint32_t m[2];
                        float p[2], w2[2];
                        int cp[2];
                        bool on[2];
#pragma unroll
                        for (int u = 0; u < 2; ++u) {
                            const int e = lo + 8 * u;
                            on[u] = e < hi;
                            m[u] = on[u] ? meta[e] : 0u;
                            p[u] = on[u] ? d * val[e] : 0.0f;
                            cp[u] = on[u] ? cpos[e] : 0;
                        }
#pragma unroll
                        for (int u = 0; u < 2; ++u) {
                            const uint32_t g = m[u] & kIdMask;
                            w2[u] = W[(on[u] && g < hot_total) ? (g >> logC) : 0u];
                        }
#pragma unroll
                        for (int u = 0; u < 2; ++u) {
                            const uint32_t g = m[u] & kIdMask;
                            const bool shared_id = (m[u] >> 31) != 0u, hot = g < hot_total;
                            const bool list_ok = CHICLE_IN_BOUNDS(S.status, !shared_id || cp[u] < P.nzcap);
                            const uint32_t addr = (!on[u] || !list_ok) ? a_sink : (shared_id ? a_prod + 4u * (uint32_t)cp[u] : (hot ? a_w + 4u * (g >> logC) : a_sink));
                            sts_f32(addr, shared_id ? p[u] : fmaf(sigma, p[u], w2[u]));
                            const bool far = on[u] && !shared_id && !hot && p[u] != 0.0f && CHICLE_IN_BOUNDS(S.status, (int64_t)g < S.dim);
                            red_add_if(Uk + (far ? g : 0u), sigma * p[u], far); // a reduction at L2, nothing waits for it
                        }
                        for (int e = lo + 16; e < hi; e += 8) {
                            const uint32_t mm = meta[e];
                            const uint32_t g = mm & kIdMask;
                            const float pp = d * val[e];
                            if (mm & 0x80000000u) {
                                if (CHICLE_IN_BOUNDS(S.status, cpos[e] < P.nzcap)) prod[cpos[e]] = pp;
                            } else if (g < hot_total) W[g >> logC] = fmaf(sigma, pp, W[g >> logC]);
                            else if (pp != 0.0f && CHICLE_IN_BOUNDS(S.status, (int64_t)g < S.dim)) atomicAdd(Uk + g, sigma * pp);
                        }
                    }
                    work_bar();
                    LA_T(ws1);
                    // (B) four threads per shared id: each adds every fourth entry of the list (at most 8: a list has
                    //     at most 32), then the four partial sums are added in a fixed order; two ids per thread and
                    //     pass, all loads first
                    const int quarter = wt & 3;
                    constexpr int kIdsPerPass = kWorkThreads / 4;
                    for (int tb = 0; tb < T; tb += 2 * kIdsPerPass) {
                        float sum[2];
                        uint32_t g3[2];
                        bool on[2];
                        int o0[2], o1[2];
#pragma unroll
                        for (int u = 0; u < 2; ++u) {
                            const int t = tb + u * kIdsPerPass + (wt >> 2);
                            on[u] = t < T;
                            o0[u] = on[u] ? offs[t] + quarter : 0;
                            o1[u] = on[u] ? offs[t + 1] : 0;
                            g3[u] = on[u] ? ids[t] : 0u;
                            if (!CHICLE_IN_BOUNDS(S.status, o1[u] <= P.nzcap && (int64_t)g3[u] < S.dim)) { o1[u] = 0; on[u] = false; }
                        }
                        float vv[2][8];
#pragma unroll
                        for (int u = 0; u < 2; ++u)
#pragma unroll
                            for (int qq = 0; qq < 8; ++qq) {
                                const int o = o0[u] + 4 * qq;
                                vv[u][qq] = o < o1[u] ? prod[o] : 0.0f;
                            }
#pragma unroll
                        for (int u = 0; u < 2; ++u) {
                            sum[u] = ((vv[u][0] + vv[u][1]) + (vv[u][2] + vv[u][3])) + ((vv[u][4] + vv[u][5]) + (vv[u][6] + vv[u][7]));
                            sum[u] += __shfl_xor_sync(0xffffffffu, sum[u], 1);
                            sum[u] += __shfl_xor_sync(0xffffffffu, sum[u], 2);
                        }
#pragma unroll
                        for (int u = 0; u < 2; ++u)
                            if (quarter == 0 && on[u] && sum[u] != 0.0f) {
                                if (g3[u] < hot_total) W[g3[u] >> logC] = fmaf(sigma, sum[u], W[g3[u] >> logC]);
                                else atomicAdd(Uk + g3[u], sigma * sum[u]);
                            }
                    }
                }
                work_bar();
            }
            if (b >= 0) {
                mbar_arrive_expect_tx_if(smem_u32(&ctl.dbar[par]), (uint32_t)(kLB * 4), wt == 0); // for block b + 2
                issue_sub(b + kSubSlots, dn); // block b's slot is free
            }
            LA_T(ws);
            // dot products: of block b + 2 against the model as it is now; of block b + 1 first if block b was walked in
            // place (a block right behind a walked one starts from the model as the walk left it)
#pragma unroll 1
            for (int ahead = 1; ahead <= 2; ++ahead) {
                // (one block ahead: block b + 1 after block b's update, whatever block b was)
                const bool due = depth == 1 ? (ahead == 1 && b + 1 < nb && !sl1)
                                            : (ahead == 1 ? (sl0 && b + 1 < nb && !sl1) : (b + 2 < nb && !sl2 && !sl1));
                if (due && !take_dots(b + ahead)) { aborted = true; break; }
            }
            if (aborted) break;
            sl0 = sl1; sl1 = sl2; sl2 = sl3;
            sl3 = b + kSubSlots < nb && (dn[3] & 1u) != 0u;
            LA_T(wg);
        }
#ifdef CHICLE_LA_TIMING
        if (blockIdx.x == 0 && wt == 0) {
            unsigned long long *d = P.timing + 4;
            d[0] = wd; d[1] = ws; d[2] = wg; d[3] = ws1; d[4] = wg0; d[5] = wg1;
        }
#endif
    }
    if (is_worker && !aborted) {
        // the model goes back to row k: as it is, or after the round's last launch as the update U_k = (w - v) / sigma'
        const int wt = (warp - 1 - (warp >> 2)) * 32 + lane;
        work_bar();
        const float inv_sigma = 1.0f / sigma;
        for (int l = wt; l < hot_mine; l += kWorkThreads) {
            const size_t g = ((size_t)l << logC) + crank;
            Uk[g] = P.model_out ? (W[l] - S.vbase[g]) * inv_sigma : W[l];
        }
        if (P.model_out)
            for (size_t g = cold0 + ((size_t)wt << logC); g < (size_t)S.dim; g += (size_t)kWorkThreads << logC)
                Uk[g] = (__ldcg(Uk + g) - S.vbase[g]) * inv_sigma;
    }
    if (is_worker || nb == 0) {
        if ((tid & 31) == 0) *reinterpret_cast<volatile int *>(&ctl.done) = 1;
    } else if (!is_chain) {
        // a warp with no role sleeps until the workers are through: waiting at the cluster barrier from the start
        // would take issue slots from the recurrence warp, which shares its scheduler with these warps
        const volatile int *done = &ctl.done;
        for (uint32_t it = 0; it < (1u << 24) && !*done; ++it) __nanosleep(2000);
    }
    // nobody leaves while another CTA of the cluster may still write to, or read from, its shared memory
    __syncwarp();
    cluster_arrive();
    cluster_wait();
}

// blk_base of every slice in one launch: slice s of partition k takes slice[(2s) K + k] steps
__global__ void k_block_bases_slices(const int64_t *__restrict__ slice, int32_t K, int64_t *__restrict__ blk_base)
{
    if (threadIdx.x != 0) return;
    const int s = blockIdx.x;
    const int64_t *steps = slice + (size_t)s * 2 * (size_t)K;
    int64_t *out = blk_base + (size_t)s * ((size_t)K + 1);
    int64_t run = 0;
    for (int32_t k = 0; k < K; ++k) {
        out[k] = run;
        run += (steps[k] + kLB - 1) / kLB;
    }
    out[K] = run;
}

template <int LOSS, bool DENSE> cudaError_t launch_chain(Glm &g, const LookParams &P)
{
    auto kern = k_lookahead_chain<LOSS, DENSE>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)g.la_smem);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)g.K << g.la_logC, 1, 1);
    cfg.blockDim = dim3(kChainThreads, 1, 1);
    cfg.dynamicSmemBytes = g.la_smem;
    cfg.stream = g.stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 1u << g.la_logC;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, kern, P);
#ifdef CHICLE_LA_TIMING
    if (e == cudaSuccess) {
        unsigned long long t[12] = {0};
        (void)cudaStreamSynchronize(g.stream);
        (void)cudaMemcpy(t, P.timing, sizeof(t), cudaMemcpyDeviceToHost);
        const double nb = t[3] ? (double)t[3] : 1.0;
        fprintf(stderr, "lookahead chain, cycles per block (partition 0): waiting for dot products %.0f, recurrence %.0f, deltas %.0f; "
                "workers of CTA 0: waiting for deltas %.0f, update: row-wise %.0f, lists and copy issue %.0f, dot products: record wait %.0f, "
                "products %.0f, sums and sending %.0f (%llu blocks)\n",
                t[0] / nb, t[1] / nb, t[2] / nb, t[4] / nb, t[7] / nb, t[5] / nb, t[8] / nb, t[9] / nb, t[6] / nb, t[3]);
    }
#endif
    return e;
}

template <int LOSS, int NZ, int HT, int THREADS> cudaError_t launch_prepare(const LookParams &P, unsigned nb, cudaStream_t stream)
{
    using Shared = PreShared<NZ, HT, THREADS>;
    auto pre = k_lookahead_prepare<LOSS, NZ, HT, THREADS>;
    cudaError_t e = cudaFuncSetAttribute(pre, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(Shared));
    if (e != cudaSuccess) return e;
    pre<<<nb, THREADS, sizeof(Shared), stream>>>(P);
    return cudaGetLastError();
}

constexpr int kPreSmallNz = 2048;
constexpr int kPreMidNz = 3072;

// true: the prepare kernel with arrays for 2 048 non-zeros per block serves (32 coordinates of 50 on average, with room)
bool small_prepare(const Glm &g) { return 32.0 * (double)g.nnz / (double)g.n_coord * 1.25 <= (double)kPreSmallNz; }
// true: arrays for 3 072 non-zeros per block serve (two CTAs of 512 threads share an SM; with 4 096 it is one). Blocks
// with more are walked in place either way unless a cluster shares them out.
bool mid_prepare(const Glm &g) { return g.la_logC == 0 || 32.0 * (double)g.nnz / (double)g.n_coord * 1.1 <= (double)kPreMidNz; }

// The prepare kernel of one launch's blocks on `stream`.
template <int LOSS> cudaError_t launch_prepare_on(Glm &g, const LookParams &P, cudaStream_t stream)
{
    const unsigned nb = (unsigned)P.n_blocks;
    if (nb == 0) return cudaSuccess;
    // beside the chain kernels: no more CTAs than fit the SMs the chains leave (see k_lookahead_prepare)
    const int chain_sms = g.K << g.la_logC;
    const unsigned free_sms = (unsigned)(g.sm_count > chain_sms ? g.sm_count - chain_sms : 1);
    if (g.fmt == CHICLE_FMT_DENSE_ROWMAJOR) {
        const unsigned per_sm = 4;
        const unsigned grid = stream == g.stream || nb < free_sms * per_sm ? nb : free_sms * per_sm;
        auto pre = k_lookahead_prepare_dense<LOSS>;
        cudaError_t e = cudaFuncSetAttribute(pre, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(PreDenseShared));
        if (e != cudaSuccess) return e;
        pre<<<grid, kPreThreads, sizeof(PreDenseShared), stream>>>(P);
        return cudaGetLastError();
    }
    cudaError_t e;
    if (small_prepare(g)) {
        const unsigned grid = stream == g.stream || nb < free_sms * 3 ? nb : free_sms * 3;
        e = launch_prepare<LOSS, kPreSmallNz, 2048, 256>(P, grid, stream);
    } else if (mid_prepare(g)) {
        const unsigned grid = stream == g.stream || nb < free_sms * 2 ? nb : free_sms * 2;
        e = launch_prepare<LOSS, kPreMidNz, 4096, 512>(P, grid, stream);
    } else {
        const unsigned grid = stream == g.stream || nb < free_sms ? nb : free_sms;
        e = launch_prepare<LOSS, 4096, 4096, 512>(P, grid, stream);
    }
#ifdef CHICLE_LA_TIMING
    if (e == cudaSuccess) {
        unsigned long long t[8] = {0};
        (void)cudaStreamSynchronize(stream);
        (void)cudaMemcpy(t, P.timing + 16, sizeof(t), cudaMemcpyDeviceToHost);
        (void)cudaMemset(P.timing + 16, 0, sizeof(t));
        const double n = (double)nb;
        fprintf(stderr, "lookahead prepare, cycles per block: headers %.0f, load + insert %.0f, count %.0f, place %.0f, number %.0f, "
                "entries %.0f, gram %.0f, cross + write %.0f\n", t[0] / n, t[1] / n, t[2] / n, t[3] / n, t[4] / n, t[5] / n, t[6] / n, t[7] / n);
    }
#endif
    return e;
}

template <int LOSS> cudaError_t launch_chain_on(Glm &g, const LookParams &P)
{
    if (g.fmt == CHICLE_FMT_DENSE_ROWMAJOR) return launch_chain<LOSS, true>(g, P);
    return launch_chain<LOSS, false>(g, P);
}

// A round's launches, slice after slice (consecutive pieces of every partition's walk). The first slice's prepare
// kernel runs on the handle's stream; the later ones on the side stream, where they fill the SMs the chain kernels
// leave idle; every chain launch waits for its slice's prepare kernel. The records of slice s lie in region s mod R
// of the record buffer, so the prepare kernel of slice s also waits for the chain launch of slice s - R.
template <int LOSS> cudaError_t launch_slices(Glm &g, std::vector<LookParams> &P)
{
    const int S = (int)P.size(), R = g.la_regions;
    cudaError_t e = cudaMemsetAsync(g.la_cursor, 0, 4 * sizeof(unsigned long long), g.stream);
    if (e != cudaSuccess) return e;
    if (!g.la_overlap) {
        // the chains take most of the SMs: the prepare kernels get the whole GPU between the chain launches instead of
        // the few SMs beside them
        for (int s = 0; s < S && e == cudaSuccess; ++s) {
            if (s > 0) e = cudaMemsetAsync(g.la_cursor + (s % R), 0, sizeof(unsigned long long), g.stream);
            if (e == cudaSuccess) e = launch_prepare_on<LOSS>(g, P[s], g.stream);
            if (s == 0 && g.time_prepare) (void)cudaEventRecord(g.ev[4], g.stream);
            if (e == cudaSuccess) e = launch_chain_on<LOSS>(g, P[s]);
        }
        return e;
    }
    e = launch_prepare_on<LOSS>(g, P[0], g.stream);
    if (e != cudaSuccess) return e;
    if (g.time_prepare) (void)cudaEventRecord(g.ev[4], g.stream);
    if (S > 1) {
        e = cudaEventRecord(g.la_ev_prep[0], g.stream);
        if (e != cudaSuccess) return e;
    }
    e = launch_chain_on<LOSS>(g, P[0]); // enqueued before the side stream's work: it takes its SMs first
    if (e != cudaSuccess || S == 1) return e;
    e = cudaEventRecord(g.la_ev_done[0], g.stream);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(g.la_stream, g.la_ev_prep[0], 0);
    auto prepare_side = [&](int s) -> cudaError_t {
        cudaError_t e2 = cudaMemsetAsync(g.la_cursor + (s % R), 0, sizeof(unsigned long long), g.la_stream);
        if (e2 == cudaSuccess) e2 = launch_prepare_on<LOSS>(g, P[s], g.la_stream);
        if (e2 == cudaSuccess) e2 = cudaEventRecord(g.la_ev_prep[s], g.la_stream);
        return e2;
    };
    for (int s = 1; s < R && s < S && e == cudaSuccess; ++s) e = prepare_side(s);
    for (int s = 1; s < S && e == cudaSuccess; ++s) {
        if (s + R - 1 < S) { // its region is free once the chain launch of slice s - 1 is done
            e = cudaStreamWaitEvent(g.la_stream, g.la_ev_done[s - 1], 0);
            if (e == cudaSuccess) e = prepare_side(s + R - 1);
            if (e != cudaSuccess) break;
        }
        e = cudaStreamWaitEvent(g.stream, g.la_ev_prep[s], 0);
        if (e == cudaSuccess) e = launch_chain_on<LOSS>(g, P[s]);
        if (e == cudaSuccess && s + 1 < S) e = cudaEventRecord(g.la_ev_done[s], g.stream);
    }
    return e;
}

} // namespace

int lookahead_max_dense_dim() { return kCapL; }
int lookahead_max_slices() { return 64; }
int64_t lookahead_max_dim() { return (int64_t)1 << kIdBits; }

// Sizes the look-ahead solver for a partition into K: CTAs per cluster, what stays in shared memory, and the record
// buffer: `regions` regions that each hold one slice of a round (the recurrence records of its blocks, then a pool
// for the workers' records).
void lookahead_plan(Glm &g, int32_t K)
{
    const bool dense = g.fmt == CHICLE_FMT_DENSE_ROWMAJOR;
    int logC = 0;
    if (!dense && g.hot_variant) {
        // a cluster per partition, on at most half of the SMs: the prepare kernels need the rest
        while (logC < 3 && ((int64_t)K << (logC + 1)) * 2 <= g.sm_count) ++logC;
        const char *env = getenv("CHICLE_LA_CLUSTER");
        if (env && env[0] >= '1' && env[0] <= '8' && env[1] == 0) {
            const int want = env[0] - '0';
            logC = want >= 8 ? 3 : (want >= 4 ? 2 : (want >= 2 ? 1 : 0));
            while (logC > 0 && ((int64_t)K << logC) > g.sm_count) --logC;
        }
    }
    g.la_logC = logC;
    // Beside chains on at most half of the SMs the prepare kernels run on the side stream; otherwise they alternate with
    // the chain launches and have the whole GPU meanwhile (config 5, K = 128: 171 against 542 ms per round).
    g.la_overlap = ((int64_t)K << logC) * 2 <= g.sm_count;
    // Two blocks ahead pays where the chains bound the round: dense rows (the recurrence itself is the cost) and sparse
    // data with a cluster per partition. One CTA per partition on sparse data means many partitions: there the prepare
    // kernels bound the round and run 40 % faster without the cross Gram matrices (measured on the hashed workload: K = 64
    // 157 against 219 ms per round; K = 16 with four CTAs per partition 253 against 308 ms the other way round).
    g.la_depth = (dense || logC >= 1) && g.la_overlap ? 2 : 1;
    {
        const char *env = getenv("CHICLE_LA_DEPTH");
        if (env && (env[0] == '1' || env[0] == '2') && env[1] == 0) g.la_depth = env[0] - '0';
        env = getenv("CHICLE_LA_OVERLAP");
        if (env && (env[0] == '0' || env[0] == '1') && env[1] == 0) g.la_overlap = env[0] == '1';
    }
    const size_t budget = (size_t)(g.max_smem_optin > 0 ? g.max_smem_optin : 227 * 1024);
    if (dense) {
        g.la_nzcap = 0;
        g.la_hotc = (int32_t)g.dim;
    } else if (!g.hot_variant) {
        g.la_nzcap = 3072;
        g.la_hotc = 0;
    } else {
        g.la_nzcap = logC == 0 ? 2048 : (logC == 1 ? 1536 : 1024);
        const ChainLayout L0 = chain_layout(g.la_nzcap, 0, false, (int)g.dim);
        int64_t hotc = ((int64_t)budget - (int64_t)L0.total - 64) / 4;
        hotc = hotc < 0 ? 0 : (hotc / 32) * 32;
        const int64_t need = (g.dim + ((int64_t)1 << logC) - 1) >> logC; // per CTA for the whole model
        g.la_hotc = (int32_t)(hotc < need ? hotc : (need + 31) / 32 * 32);
    }
    g.la_smem = chain_layout(g.la_nzcap, g.la_hotc, dense, (int)g.dim).total;

    // slices: at most a sixteenth of the walk, but at least 256 blocks per partition; three regions
    const int64_t n = g.n_coord;
    const int64_t max_nk = (n + K - 1) / K + 1;
    const int64_t max_nb = (max_nk + kLB - 1) / kLB;
    int64_t per_part = (max_nb + 15) / 16;
    per_part = per_part < 256 ? 256 : per_part;
    per_part = per_part > max_nb ? max_nb : per_part;
    const bool whole = per_part >= max_nb; // a round is one slice
    // (partitions of unequal sizes: the largest may hold almost everything; a region then holds what a sixteenth of
    // the whole walk needs, and the launch cuts finer if a slice does not fit)
    int64_t region_blocks = whole ? n / kLB + K + 1 : per_part * K + K;
    if (region_blocks > n / kLB + K + 1) region_blocks = n / kLB + K + 1;
    g.la_region_blocks = region_blocks;
    g.la_regions = whole ? 1 : 3;
    {
        const char *env = getenv("CHICLE_LA_SLICES"); // forced slicing (tests): the ring as large problems have it
        if (env && atoi(env) > 1) g.la_regions = 3;
    }
    const double frac = whole ? 1.0 : (double)region_blocks / (double)(n / kLB + 1);
    const size_t C = (size_t)1 << logC;
    size_t pool;
    if (dense) pool = (size_t)region_blocks * sub_bytes(kLB * (int)g.dim, 0, true);
    else {
        const double all = 14.0 * (double)g.nnz;
        double part = whole ? all : 1.2 * frac * all + (double)(1 << 20);
        if (part > all) part = all;
        pool = (size_t)part + (size_t)region_blocks * C * 128 + 4096;
    }
    const size_t heads = ((size_t)region_blocks * sizeof(ChainHead) + 255) & ~(size_t)255;
    g.la_pool_off = heads;
    g.la_region_bytes = (heads + pool + 255) & ~(size_t)255;
    g.la_dir_bytes = (size_t)g.la_regions * (size_t)region_blocks * C * sizeof(BlkDir);
}

cudaError_t launch_lookahead_solver(Glm &g, const SolverParams &S)
{
    const int32_t K = g.K;
    std::vector<int64_t> steps((size_t)K), nb((size_t)K);
    int64_t total = 0, max_nb = 0;
    for (int32_t k = 0; k < K; ++k) {
        const int64_t nk = g.h_part_off[k + 1] - g.h_part_off[k];
        steps[(size_t)k] = g.round_steps ? g.round_steps[k] : (S.H == 0 ? nk : (nk > 0 ? S.H : 0));
        nb[(size_t)k] = (steps[(size_t)k] + kLB - 1) / kLB;
        total += nb[(size_t)k];
        if (nb[(size_t)k] > max_nb) max_nb = nb[(size_t)k];
    }
    if (total <= 0 || total > 0x7fffffff) return cudaErrorInvalidConfiguration;
    // Slices: fractions 0 = F_0 < F_1 < ... < F_S = 1 of every partition's walk. The first slice is small (its
    // prepare kernel is the one nothing hides), the next ones double, up to a sixteenth of the walk or 256 blocks of
    // the longest partition, whichever is more; a slice must fit a region of the record buffer.
    // CHICLE_LA_SLICES=1 keeps every round in one piece (to time the prepare kernel alone), CHICLE_LA_SLICES=n cuts
    // into n equal slices whatever the length (to test the slicing on small problems).
    const int max_slices = lookahead_max_slices();
    std::vector<double> F;
    const char *env = getenv("CHICLE_LA_SLICES");
    const int forced = env ? atoi(env) : 0;
    auto build = [&](double first, double cap) {
        F.assign(1, 0.0);
        double at = 0.0, len = first;
        while (at < 1.0 && (int)F.size() < max_slices) {
            at += len;
            F.push_back(at < 1.0 ? at : 1.0);
            len = len * 2.0 < cap ? len * 2.0 : cap;
        }
        F.back() = 1.0;
    };
    double cap = 1.0;
    if (forced >= 1 && (forced == 1 || g.la_stream)) {
        const int n = forced > max_slices ? max_slices : forced;
        F.assign(1, 0.0);
        for (int s = 1; s <= n; ++s) F.push_back((double)s / n);
    } else if ((g.la_overlap && !g.la_stream) || g.la_regions == 1 || max_nb < 512) {
        F = {0.0, 1.0};
    } else {
        cap = 1.0 / 16;
        if (cap * (double)max_nb < 256.0) cap = 256.0 / (double)max_nb;
        build(cap / 8, cap);
    }
    std::vector<int64_t> h;
    std::vector<int64_t> blocks;
    for (int attempt = 0; attempt < 24; ++attempt) {
        const int Sn = (int)F.size() - 1;
        h.assign((size_t)Sn * 2 * (size_t)K, 0);
        blocks.assign((size_t)Sn, 0);
        int64_t worst = 0;
        for (int32_t k = 0; k < K; ++k) {
            const int64_t nbk = nb[(size_t)k];
            int64_t prev = 0;
            for (int s = 0; s < Sn; ++s) {
                int64_t cut = s + 1 == Sn ? nbk : (int64_t)((double)nbk * F[(size_t)s + 1]);
                cut = cut < prev ? prev : (cut > nbk ? nbk : cut);
                const int64_t first = prev * kLB;
                const int64_t last = s + 1 == Sn ? steps[(size_t)k] : cut * kLB;
                h[((size_t)s * 2) * (size_t)K + (size_t)k] = last - first;
                h[((size_t)s * 2 + 1) * (size_t)K + (size_t)k] = first;
                blocks[(size_t)s] += (last - first + kLB - 1) / kLB;
                prev = cut;
            }
        }
        for (int s = 0; s < Sn; ++s) worst = blocks[(size_t)s] > worst ? blocks[(size_t)s] : worst;
        if (worst <= g.la_region_blocks) break;
        // finer: equal slices, twice as many as would just fit
        int n = (int)((total + g.la_region_blocks - 1) / g.la_region_blocks) * (attempt + 2);
        if (n > max_slices) n = max_slices;
        if (!g.la_stream || g.la_regions < 2 || attempt == 23) return cudaErrorInvalidConfiguration;
        F.assign(1, 0.0);
        for (int s = 1; s <= n; ++s) F.push_back((double)s / n);
    }
    const int Sn = (int)F.size() - 1;
    // a pageable source: the runtime has taken its copy of these words when the call returns
    cudaError_t e = cudaMemcpyAsync(g.la_slice, h.data(), h.size() * sizeof(int64_t), cudaMemcpyHostToDevice, g.stream);
    if (e != cudaSuccess) return e;
    k_block_bases_slices<<<Sn, 32, 0, g.stream>>>(g.la_slice, K, g.la_blk_base);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    const char *drop = getenv("CHICLE_TEST_DROP_RECORD"); // test aid: leave one block's records unpublished
    const size_t C = (size_t)1 << g.la_logC;
    std::vector<LookParams> P((size_t)Sn);
    for (int s = 0; s < Sn; ++s) {
        const int r = s % g.la_regions;
        LookParams &p = P[(size_t)s];
        p = LookParams{};
        p.S = S;
        p.S.H = 0;
        p.S.steps_k = g.la_slice + ((size_t)s * 2) * (size_t)K;
        p.S.first_k = g.la_slice + ((size_t)s * 2 + 1) * (size_t)K;
        p.rec = static_cast<unsigned char *>(g.la_rec) + (size_t)r * g.la_region_bytes;
        p.dirS = static_cast<BlkDir *>(g.la_dir) + (size_t)r * (size_t)g.la_region_blocks * C;
        p.cursor = g.la_cursor + r;
        p.timing = g.la_cursor + 8;
        p.pool_off = g.la_pool_off;
        p.pool_cap = g.la_region_bytes - g.la_pool_off;
        p.blk_base = g.la_blk_base + (size_t)s * ((size_t)K + 1);
        p.K = K;
        p.logC = g.la_logC;
        p.depth = g.la_depth;
        p.nzcap = g.la_nzcap;
        p.hotc = g.la_hotc;
        p.n_blocks = blocks[(size_t)s];
        p.drop_block = (drop && s == 0) ? atoll(drop) : -1;
        p.nnz = g.nnz;
        p.model_in = s == 0 ? 1 : 0;
        p.model_out = s == Sn - 1 ? 1 : 0;
    }
    g.la_last_slices = Sn;
    g.solver_launches += 1 + 2 * Sn; // block tables, then a prepare and a chain launch per slice
    switch (g.loss) {
    case CHICLE_LOSS_HINGE_DUAL: return launch_slices<CHICLE_LOSS_HINGE_DUAL>(g, P);
    case CHICLE_LOSS_LOGISTIC_DUAL: return launch_slices<CHICLE_LOSS_LOGISTIC_DUAL>(g, P);
    default: return launch_slices<CHICLE_LOSS_RIDGE_PRIMAL>(g, P);
    }
}

} // namespace chicle
