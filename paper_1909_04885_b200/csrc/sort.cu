// Stable least-significant-digit radix sort pass (8 bits) over (64-bit key, 32-bit value) pairs.
// Used by the partition step (order ids by their mixed key) and the per-round visiting orders.
//
// One pass = digit histogram per tile -> exclusive scan of the digit-major table -> stable scatter.
// The scatter ranks items inside a tile in index order: each warp owns a contiguous run of the tile and
// ranks its 32 items per step with match.any, so equal digits keep their input order (stability).
#include "chicle_internal.cuh"

namespace chicle {

namespace {

constexpr int kScanThreads = 256;
constexpr int kScanItems = 16;
constexpr int kScanTile = kScanThreads * kScanItems;

__device__ __forceinline__ uint32_t digit_of(const uint64_t *keys, const int32_t *vals, const int32_t *owner,
                                             int64_t i, int shift)
{
    if (owner) return (uint32_t)(owner[vals[i]] >> shift) & 255u;
    return (uint32_t)(keys[i] >> shift) & 255u;
}

__global__ void __launch_bounds__(kSortThreads)
k_radix_hist(const uint64_t *__restrict__ keys, const int32_t *__restrict__ vals, const int32_t *__restrict__ owner,
             int64_t n, int shift, uint32_t *__restrict__ hist, int nblk)
{
    __shared__ uint32_t h[256];
    h[threadIdx.x] = 0;
    __syncthreads();
    const int64_t base = (int64_t)blockIdx.x * kSortTile;
#pragma unroll 4
    for (int it = 0; it < kSortItems; ++it) {
        const int64_t i = base + (int64_t)it * kSortThreads + threadIdx.x;
        if (i < n) atomicAdd(&h[digit_of(keys, vals, owner, i, shift)], 1u);
    }
    __syncthreads();
    hist[(size_t)threadIdx.x * nblk + blockIdx.x] = h[threadIdx.x];
}

// exclusive scan of `m` counters, three kernels: tile sums, scan of the sums (one block), tile scans
__global__ void __launch_bounds__(kScanThreads) k_scan_tile_sums(const uint32_t *__restrict__ in, int64_t m,
                                                                 uint32_t *__restrict__ sums)
{
    __shared__ uint32_t red[kScanThreads / 32];
    const int64_t base = (int64_t)blockIdx.x * kScanTile + (int64_t)threadIdx.x * kScanItems;
    uint32_t s = 0;
#pragma unroll
    for (int j = 0; j < kScanItems; ++j)
        if (base + j < m) s += in[base + j];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t t = 0;
        for (int w = 0; w < kScanThreads / 32; ++w) t += red[w];
        sums[blockIdx.x] = t;
    }
}

__global__ void __launch_bounds__(1024) k_scan_sums(uint32_t *__restrict__ sums, int64_t nt)
{
    __shared__ uint32_t warp_tot[32];
    __shared__ uint32_t carry;
    if (threadIdx.x == 0) carry = 0;
    __syncthreads();
    for (int64_t base = 0; base < nt; base += 1024) {
        const int64_t i = base + threadIdx.x;
        const uint32_t x = i < nt ? sums[i] : 0u;
        uint32_t inc = x;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t y = __shfl_up_sync(0xffffffffu, inc, o);
            if ((threadIdx.x & 31) >= o) inc += y;
        }
        if ((threadIdx.x & 31) == 31) warp_tot[threadIdx.x >> 5] = inc;
        __syncthreads();
        if (threadIdx.x < 32) {
            uint32_t w = warp_tot[threadIdx.x], winc = w;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t y = __shfl_up_sync(0xffffffffu, winc, o);
                if (threadIdx.x >= o) winc += y;
            }
            warp_tot[threadIdx.x] = winc - w; // exclusive over warps
        }
        __syncthreads();
        const uint32_t c = carry;
        if (i < nt) sums[i] = c + warp_tot[threadIdx.x >> 5] + inc - x;
        __syncthreads();
        if (threadIdx.x == 1023) carry = c + warp_tot[31] + inc;
        __syncthreads();
    }
}

__global__ void __launch_bounds__(kScanThreads) k_scan_tiles(uint32_t *__restrict__ data, int64_t m,
                                                            const uint32_t *__restrict__ sums)
{
    __shared__ uint32_t warp_tot[kScanThreads / 32];
    const int64_t base = (int64_t)blockIdx.x * kScanTile + (int64_t)threadIdx.x * kScanItems;
    uint32_t x[kScanItems];
    uint32_t s = 0;
#pragma unroll
    for (int j = 0; j < kScanItems; ++j) {
        x[j] = base + j < m ? data[base + j] : 0u;
        s += x[j];
    }
    uint32_t inc = s;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t y = __shfl_up_sync(0xffffffffu, inc, o);
        if ((threadIdx.x & 31) >= o) inc += y;
    }
    if ((threadIdx.x & 31) == 31) warp_tot[threadIdx.x >> 5] = inc;
    __syncthreads();
    uint32_t off = sums[blockIdx.x];
    for (int w = 0; w < (int)(threadIdx.x >> 5); ++w) off += warp_tot[w];
    off += inc - s;
#pragma unroll
    for (int j = 0; j < kScanItems; ++j) {
        if (base + j < m) data[base + j] = off;
        off += x[j];
    }
}

__global__ void __launch_bounds__(kSortThreads)
k_radix_scatter(const uint64_t *__restrict__ keys_in, const int32_t *__restrict__ vals_in,
                uint64_t *__restrict__ keys_out, int32_t *__restrict__ vals_out, const int32_t *__restrict__ owner,
                int64_t n, int shift, const uint32_t *__restrict__ scanned, int nblk)
{
    constexpr int kWarps = kSortThreads / 32;
    __shared__ uint32_t cnt[kWarps][256];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int j = threadIdx.x; j < kWarps * 256; j += kSortThreads) (&cnt[0][0])[j] = 0;
    __syncthreads();

    const int64_t warp_base = (int64_t)blockIdx.x * kSortTile + (int64_t)warp * (kSortItems * 32);
    uint32_t dig[kSortItems];
    uint32_t rank[kSortItems];
    const uint32_t lt_mask = (1u << lane) - 1u;
#pragma unroll
    for (int it = 0; it < kSortItems; ++it) {
        const int64_t i = warp_base + it * 32 + lane;
        const bool valid = i < n;
        const uint32_t d = valid ? digit_of(keys_in, vals_in, owner, i, shift) : 256u;
        const uint32_t peers = __match_any_sync(0xffffffffu, d);
        const uint32_t before = valid ? cnt[warp][d] : 0u;
        __syncwarp();
        if (valid && (peers & lt_mask) == 0u) cnt[warp][d] = before + __popc(peers);
        __syncwarp();
        dig[it] = d;
        rank[it] = before + __popc(peers & lt_mask);
    }
    __syncthreads();
    {
        // thread t owns digit t: turn per-warp counts into start offsets in the output
        uint32_t run = scanned[(size_t)threadIdx.x * nblk + blockIdx.x];
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            const uint32_t c = cnt[w][threadIdx.x];
            cnt[w][threadIdx.x] = run;
            run += c;
        }
    }
    __syncthreads();
#pragma unroll
    for (int it = 0; it < kSortItems; ++it) {
        const int64_t i = warp_base + it * 32 + lane;
        if (i < n) {
            const uint32_t dst = cnt[warp][dig[it]] + rank[it];
            if (keys_out) keys_out[dst] = keys_in[i];
            vals_out[dst] = vals_in[i];
        }
    }
}

} // namespace

size_t sort_hist_entries(int64_t n) { return (size_t)256 * (size_t)((n + kSortTile - 1) / kSortTile); }
size_t sort_scan_tiles(int64_t n) { return (sort_hist_entries(n) + kScanTile - 1) / kScanTile; }

cudaError_t radix_pass(const uint64_t *keys_in, const int32_t *vals_in, uint64_t *keys_out, int32_t *vals_out,
                       const int32_t *owner, int64_t n, int shift, uint32_t *hist, uint32_t *scan_sums,
                       cudaStream_t stream)
{
    if (n <= 0) return cudaSuccess;
    const int nblk = (int)((n + kSortTile - 1) / kSortTile);
    const int64_t m = (int64_t)256 * nblk;
    const int nt = (int)((m + kScanTile - 1) / kScanTile);
    k_radix_hist<<<nblk, kSortThreads, 0, stream>>>(keys_in, vals_in, owner, n, shift, hist, nblk);
    k_scan_tile_sums<<<nt, kScanThreads, 0, stream>>>(hist, m, scan_sums);
    k_scan_sums<<<1, 1024, 0, stream>>>(scan_sums, nt);
    k_scan_tiles<<<nt, kScanThreads, 0, stream>>>(hist, m, scan_sums);
    k_radix_scatter<<<nblk, kSortThreads, 0, stream>>>(keys_in, vals_in, keys_out, vals_out, owner, n, shift, hist,
                                                       nblk);
    return cudaGetLastError();
}

} // namespace chicle
