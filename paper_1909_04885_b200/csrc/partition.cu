// Partition of the coordinates into K random equal blocks, and the per-round visiting orders.
// Integer-only: the result is a pure function of (n, K, seed) and (seed, round, epoch).
#include "chicle_internal.cuh"

namespace chicle {

namespace {

__global__ void k_partition_keys(int64_t n, uint64_t s, uint64_t *__restrict__ keys, int32_t *__restrict__ ids)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) {
        keys[i] = mix64(s ^ (uint64_t)i);
        ids[i] = (int32_t)i;
    }
}

// position in key order -> partition: blocks of base+1 (the first `extra`) then base
__global__ void k_owner_from_rank(int64_t n, int64_t base, int64_t extra, const int32_t *__restrict__ sorted_ids,
                                  int32_t *__restrict__ owner)
{
    const int64_t pos = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (pos < n) {
        const int64_t thr = extra * (base + 1);
        const int64_t k = pos < thr ? pos / (base + 1) : extra + (pos - thr) / base;
        owner[sorted_ids[pos]] = (int32_t)k;
    }
}

__global__ void k_iota(int64_t n, int32_t *__restrict__ ids)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) ids[i] = (int32_t)i;
}

__global__ void k_perm_keys(int64_t n, uint64_t ab, const int32_t *__restrict__ members, uint64_t *__restrict__ keys,
                            int32_t *__restrict__ vals)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) {
        const int32_t id = members[i];
        keys[i] = mix64(ab ^ (uint64_t)(uint32_t)id);
        vals[i] = id;
    }
}

inline unsigned blocks_for(int64_t n, int t) { return (unsigned)((n + t - 1) / t); }

// Stable passes over the digits of owner[id]; the last pass writes into `final_out`.
cudaError_t owner_passes(Glm &g, int32_t K, const int32_t *in, int32_t *scratch, int32_t *final_out)
{
    int passes = 1;
    while (passes < 4 && (int64_t)K > (1LL << (8 * passes))) ++passes;
    const int32_t *src = in;
    cudaError_t e = cudaSuccess;
    for (int p = 0; p < passes; ++p) {
        int32_t *dst;
        if (p == passes - 1) dst = final_out;
        else dst = (src == scratch) ? g.sortws.vals[1] : scratch;
        // with at most 4 passes and distinct buffers for in / scratch / vals[1] / final_out no pass aliases
        e = radix_pass(nullptr, src, nullptr, dst, g.owner, g.n_coord, 8 * p, g.sortws.hist, g.sortws.scan_sums,
                       g.stream);
        if (e != cudaSuccess) return e;
        src = dst;
    }
    return e;
}

} // namespace

cudaError_t launch_partition(Glm &g, int32_t K, uint64_t seed)
{
    const int64_t n = g.n_coord;
    SortWorkspace &w = g.sortws;
    const int T = 256;
    k_partition_keys<<<blocks_for(n, T), T, 0, g.stream>>>(n, mix64(seed), w.keys[0], w.vals[0]);
    int cur = 0;
    for (int pass = 0; pass < 8; ++pass) {
        cudaError_t e = radix_pass(w.keys[cur], w.vals[cur], w.keys[cur ^ 1], w.vals[cur ^ 1], nullptr, n, 8 * pass,
                                   w.hist, w.scan_sums, g.stream);
        if (e != cudaSuccess) return e;
        cur ^= 1;
    }
    // 8 passes: the sorted ids are back in buffer 0
    k_owner_from_rank<<<blocks_for(n, T), T, 0, g.stream>>>(n, n / K, n % K, w.vals[cur], g.owner);
    // members: ids 0..n-1 (ascending) stably grouped by owner
    k_iota<<<blocks_for(n, T), T, 0, g.stream>>>(n, w.vals[0]);
    // in = vals[0]; scratch = reinterpret keys[0] storage as int32 (keys are dead now)
    cudaError_t e = owner_passes(g, K, w.vals[0], reinterpret_cast<int32_t *>(w.keys[0]), g.members);
    if (e != cudaSuccess) return e;
    return cudaGetLastError();
}

cudaError_t launch_permutation(Glm &g, int64_t round, int64_t epochs)
{
    const int64_t n = g.n_coord;
    SortWorkspace &w = g.sortws;
    const int T = 256;
    const uint64_t a = mix64(g.seed ^ kPermStream);
    for (int64_t e = 0; e < epochs; ++e) {
        const uint64_t b = mix64(((uint64_t)round << 32) + (uint64_t)e);
        k_perm_keys<<<blocks_for(n, T), T, 0, g.stream>>>(n, a ^ b, g.members, w.keys[0], w.vals[0]);
        int cur = 0;
        for (int pass = 0; pass < 8; ++pass) {
            cudaError_t err = radix_pass(w.keys[cur], w.vals[cur], w.keys[cur ^ 1], w.vals[cur ^ 1], nullptr, n,
                                         8 * pass, w.hist, w.scan_sums, g.stream);
            if (err != cudaSuccess) return err;
            cur ^= 1;
        }
        cudaError_t err = owner_passes(g, g.K, w.vals[cur], reinterpret_cast<int32_t *>(w.keys[0]),
                                       g.perm + (size_t)e * (size_t)n);
        if (err != cudaSuccess) return err;
    }
    return cudaGetLastError();
}

} // namespace chicle
