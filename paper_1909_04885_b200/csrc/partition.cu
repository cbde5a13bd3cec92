// Partition of the coordinates into K random equal blocks, and the per-round visiting orders.
// Integer-only: the result is a pure function of (n, K, seed) and (seed, round, epoch).
#include <cstdio>
#include <mutex>

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

// the same for blocks of given sizes: part_off[k] <= pos < part_off[k + 1]
__global__ void k_owner_from_offsets(int64_t n, int32_t K, const int64_t *__restrict__ part_off,
                                     const int32_t *__restrict__ sorted_ids, int32_t *__restrict__ owner)
{
    const int64_t pos = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (pos < n) {
        int32_t lo = 0, hi = K; // part_off[lo] <= pos < part_off[hi]
        while (hi - lo > 1) {
            const int32_t mid = (lo + hi) >> 1;
            if (part_off[mid] <= pos) lo = mid;
            else hi = mid;
        }
        owner[sorted_ids[pos]] = lo;
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

// After a stable sort on the upper 32 key bits only: elements whose upper halves agree stand next to each other in
// their old order; the thread at the head of such a run (they are rare and short: keys are 64-bit hashes) puts it
// into full-key order by insertion. Runs are disjoint, so the threads do not meet.
__global__ void k_order_runs(int64_t n, uint64_t *__restrict__ keys, int32_t *__restrict__ vals)
{
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i + 1 < n; i += (int64_t)gridDim.x * blockDim.x) {
        const uint32_t hi = (uint32_t)(keys[i] >> 32);
        if ((uint32_t)(keys[i + 1] >> 32) != hi) continue;
        if (i > 0 && (uint32_t)(keys[i - 1] >> 32) == hi) continue; // not the head of the run
        int64_t end = i + 2;
        while (end < n && (uint32_t)(keys[end] >> 32) == hi) ++end;
        for (int64_t a = i + 1; a < end; ++a) {
            const uint64_t ka = keys[a];
            const int32_t va = vals[a];
            int64_t b = a;
            while (b > i && keys[b - 1] > ka) {
                keys[b] = keys[b - 1];
                vals[b] = vals[b - 1];
                --b;
            }
            keys[b] = ka;
            vals[b] = va;
        }
    }
}

cudaError_t launch_partition(Glm &g, int32_t K, uint64_t seed)
{
    const int64_t n = g.n_coord;
    SortWorkspace &w = g.sortws;
    const int T = 256;
    k_partition_keys<<<blocks_for(n, T), T, 0, g.stream>>>(n, mix64(seed), w.keys[0], w.vals[0]);
    int cur = 0;
    for (int pass = 4; pass < 8; ++pass) { // the upper key halves; equal runs are ordered below
        cudaError_t e = radix_pass(w.keys[cur], w.vals[cur], w.keys[cur ^ 1], w.vals[cur ^ 1], nullptr, n, 8 * pass,
                                   w.hist, w.scan_sums, g.stream);
        if (e != cudaSuccess) return e;
        cur ^= 1;
    }
    {
        unsigned grid = blocks_for(n, T);
        if (grid > (unsigned)g.sm_count * 16) grid = (unsigned)g.sm_count * 16;
        k_order_runs<<<grid, T, 0, g.stream>>>(n, w.keys[cur], w.vals[cur]);
    }
    // an even number of passes: the sorted ids are back in buffer 0
    // (the offsets are on the device already: equal blocks, or the sizes the caller gave)
    k_owner_from_offsets<<<blocks_for(n, T), T, 0, g.stream>>>(n, K, g.part_off, w.vals[cur], g.owner);
    // members: ids 0..n-1 (ascending) stably grouped by owner
    k_iota<<<blocks_for(n, T), T, 0, g.stream>>>(n, w.vals[0]);
    // in = vals[0]; scratch = reinterpret keys[0] storage as int32 (keys are dead now)
    cudaError_t e = owner_passes(g, K, w.vals[0], reinterpret_cast<int32_t *>(w.keys[0]), g.members);
    if (e != cudaSuccess) return e;
    return cudaGetLastError();
}

// owner[i] = task of the chunk that holds coordinate i: chunk_off[c] <= i < chunk_off[c + 1]
__global__ void k_owner_from_chunks(int64_t n, int64_t C, const int64_t *__restrict__ chunk_off,
                                    const int32_t *__restrict__ chunk_task, int32_t *__restrict__ owner)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) {
        int64_t lo = 0, hi = C;
        while (hi - lo > 1) {
            const int64_t mid = (lo + hi) >> 1;
            if (chunk_off[mid] <= i) lo = mid;
            else hi = mid;
        }
        owner[i] = chunk_task[lo];
    }
}

cudaError_t launch_partition_chunks(Glm &g, int32_t K, int64_t C, const int64_t *chunk_off, const int32_t *chunk_task)
{
    const int64_t n = g.n_coord;
    SortWorkspace &w = g.sortws;
    const int T = 256;
    k_owner_from_chunks<<<blocks_for(n, T), T, 0, g.stream>>>(n, C, chunk_off, chunk_task, g.owner);
    // members: ids 0..n-1 (ascending) stably grouped by owner
    k_iota<<<blocks_for(n, T), T, 0, g.stream>>>(n, w.vals[0]);
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
        // four radix passes over the upper half of the 64-bit keys, then the rare runs with equal upper halves are
        // put into full-key order: the same order as eight passes give, at half the passes
        int cur = 0;
        for (int pass = 4; pass < 8; ++pass) {
            cudaError_t err = radix_pass(w.keys[cur], w.vals[cur], w.keys[cur ^ 1], w.vals[cur ^ 1], nullptr, n,
                                         8 * pass, w.hist, w.scan_sums, g.stream);
            if (err != cudaSuccess) return err;
            cur ^= 1;
        }
        {
            unsigned grid = blocks_for(n, T);
            if (grid > (unsigned)g.sm_count * 16) grid = (unsigned)g.sm_count * 16;
            k_order_runs<<<grid, T, 0, g.stream>>>(n, w.keys[cur], w.vals[cur]);
        }
        cudaError_t err = owner_passes(g, g.K, w.vals[cur], reinterpret_cast<int32_t *>(w.keys[0]),
                                       g.perm + (size_t)e * (size_t)n);
        if (err != cudaSuccess) return err;
    }
    return cudaGetLastError();
}

} // namespace chicle

namespace chicle {

// ---------------------------------------------------------------------------------------------------------------
// Partition without any allocation.
//
// Some callers are not allowed to allocate device memory when they need a partition map: code that runs inside a
// region where the allocator must not be touched (a memory pool that was sized and frozen at start-up, a real-time
// or serving loop with a fixed memory budget, a host thread that holds a lock the allocator also takes), or a
// process whose device memory is handed out entirely by someone else. chicle_partition() cannot serve them: it
// creates the sort workspace and the per-partition update buffers on its first call. The entry point below does
// the same integer work (same kernels, same order, same result) with its workspace in a fixed array that is part
// of the loaded library image, so no cudaMalloc, cudaFree or framework allocator is ever called.
//
// The array below is device memory owned by the CUDA module: every GPU that loads this library carries it until
// the process exits. In host code its name is only a handle for the symbol, not an address a kernel may
// dereference; the device address is fetched once per device with cudaGetSymbolAddress and that pointer is what
// the kernels get.
namespace {

constexpr int64_t kNoAllocMaxCoords = CHICLE_NOALLOC_MAX_COORDS;
constexpr size_t kNaKeysBytes = (size_t)kNoAllocMaxCoords * sizeof(uint64_t);                       // one key array
constexpr size_t kNaValsBytes = (size_t)kNoAllocMaxCoords * sizeof(int32_t);                        // one id array
constexpr size_t kNaHistBytes = (size_t)256 * ((kNoAllocMaxCoords + kSortTile - 1) / kSortTile) * sizeof(uint32_t);
constexpr size_t kNaSumsBytes = 4096;                                                               // scan tile sums
constexpr size_t kNaOffKeys0 = 0;
constexpr size_t kNaOffKeys1 = kNaOffKeys0 + kNaKeysBytes;
constexpr size_t kNaOffVals0 = kNaOffKeys1 + kNaKeysBytes;
constexpr size_t kNaOffVals1 = kNaOffVals0 + kNaValsBytes;
constexpr size_t kNaOffHist = kNaOffVals1 + kNaValsBytes;
constexpr size_t kNaOffSums = kNaOffHist + kNaHistBytes;
constexpr size_t kNaTotalBytes = kNaOffSums + kNaSumsBytes;
static_assert(kNaKeysBytes % 256 == 0 && kNaValsBytes % 256 == 0 && kNaHistBytes % 256 == 0, "256-byte carving");

static __device__ __align__(256) unsigned char g_noalloc_scratch[kNaTotalBytes];

constexpr int kNaMaxDevices = 64;
std::mutex g_na_mutex;
unsigned char *g_na_base[kNaMaxDevices] = {};

void na_message(char *buf, size_t len, const char *msg)
{
    if (buf && len) std::snprintf(buf, len, "%s", msg);
}

} // namespace

} // namespace chicle

extern "C" chicle_status_t chicle_partition_noalloc(int device, void *cuda_stream, int64_t n_coord, int32_t K,
                                                    uint64_t seed, int32_t *dev_owner, int32_t *dev_members,
                                                    char *host_errbuf, size_t errbuf_len)
{
    using namespace chicle;
    if (!dev_owner || !dev_members) {
        na_message(host_errbuf, errbuf_len, "dev_owner and dev_members must be non-NULL device pointers");
        return CHICLE_ERR_INVALID_ARG;
    }
    if (n_coord < 1 || n_coord > kNoAllocMaxCoords) {
        na_message(host_errbuf, errbuf_len,
                   "n_coord outside [1, CHICLE_NOALLOC_MAX_COORDS]: the built-in workspace holds at most 131072 "
                   "coordinates; use chicle_partition for larger problems");
        return CHICLE_ERR_UNSUPPORTED;
    }
    if (K < 1 || (int64_t)K > n_coord) {
        na_message(host_errbuf, errbuf_len, "need 1 <= K <= n_coord");
        return CHICLE_ERR_INVALID_ARG;
    }
    if (device < 0 || device >= kNaMaxDevices) {
        na_message(host_errbuf, errbuf_len, "device index out of range");
        return CHICLE_ERR_INVALID_ARG;
    }
    cudaError_t e = cudaSetDevice(device);
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        na_message(host_errbuf, errbuf_len, cudaGetErrorString(e));
        return CHICLE_ERR_CUDA;
    }
    unsigned char *base = nullptr;
    {
        // set-up, once per device, with that device current: turn the symbol into a device address
        std::lock_guard<std::mutex> lock(g_na_mutex);
        if (!g_na_base[device]) {
            void *p = nullptr;
            e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
            if (e != cudaSuccess || !p) {
                (void)cudaGetLastError();
                na_message(host_errbuf, errbuf_len, e != cudaSuccess ? cudaGetErrorString(e) : "cudaGetSymbolAddress returned NULL");
                return CHICLE_ERR_CUDA;
            }
            g_na_base[device] = static_cast<unsigned char *>(p);
        }
        base = g_na_base[device];
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    uint64_t *keys[2] = {reinterpret_cast<uint64_t *>(base + kNaOffKeys0), reinterpret_cast<uint64_t *>(base + kNaOffKeys1)};
    int32_t *vals[2] = {reinterpret_cast<int32_t *>(base + kNaOffVals0), reinterpret_cast<int32_t *>(base + kNaOffVals1)};
    uint32_t *hist = reinterpret_cast<uint32_t *>(base + kNaOffHist);
    uint32_t *sums = reinterpret_cast<uint32_t *>(base + kNaOffSums);
    // Nothing in the workspace has to start at zero: keys and ids are written before they are read, and every pass
    // writes all of its digit counters and tile sums before scanning them, so the previous call's leftovers are
    // never observed.
    const int64_t n = n_coord;
    const int T = 256;
    k_partition_keys<<<blocks_for(n, T), T, 0, stream>>>(n, mix64(seed), keys[0], vals[0]);
    int cur = 0;
    for (int pass = 0; pass < 8; ++pass) {
        e = radix_pass(keys[cur], vals[cur], keys[cur ^ 1], vals[cur ^ 1], nullptr, n, 8 * pass, hist, sums, stream);
        if (e != cudaSuccess) break;
        cur ^= 1;
    }
    if (e == cudaSuccess) {
        k_owner_from_rank<<<blocks_for(n, T), T, 0, stream>>>(n, n / K, n % K, vals[cur], dev_owner);
        k_iota<<<blocks_for(n, T), T, 0, stream>>>(n, vals[0]);
        int passes = 1;
        while (passes < 4 && (int64_t)K > (1LL << (8 * passes))) ++passes;
        const int32_t *src = vals[0];
        for (int p = 0; p < passes && e == cudaSuccess; ++p) {
            int32_t *dst = p == passes - 1 ? dev_members : (src == vals[0] ? vals[1] : vals[0]);
            e = radix_pass(nullptr, src, nullptr, dst, dev_owner, n, 8 * p, hist, sums, stream);
            src = dst;
        }
    }
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        na_message(host_errbuf, errbuf_len, cudaGetErrorString(e));
        return CHICLE_ERR_CUDA;
    }
    return CHICLE_OK;
}

