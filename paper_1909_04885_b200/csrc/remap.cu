// Frequency ranking of the entry ids of a sparse problem (features for the dual losses, rows for ridge), done once
// when the problem is created: id 0 becomes the id that occurs in the most non-zeros, ties by ascending old id.
// The matrix indices are relabelled in place; the shared vector lives in the new id space inside the library and is
// translated at the boundary. The local solver keeps the most frequent ids of U_k in a direct shared-memory array.
#include "chicle_internal.cuh"

namespace chicle {

namespace {

constexpr int kT = 256;
inline unsigned blocks_for(int64_t n) { return (unsigned)((n + kT - 1) / kT); }

__global__ void k_count_ids(const int32_t *__restrict__ indices, int64_t nnz, uint32_t *__restrict__ counts)
{
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < nnz; e += (int64_t)gridDim.x * blockDim.x)
        atomicAdd(counts + indices[e], 1u);
}

__global__ void k_freq_keys(const uint32_t *__restrict__ counts, int64_t dim, uint64_t *__restrict__ keys,
                            int32_t *__restrict__ vals)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < dim) {
        keys[i] = ((uint64_t)(0xFFFFFFFFu - counts[i]) << 32) | (uint64_t)(uint32_t)i; // descending count, ascending id
        vals[i] = (int32_t)i;
    }
}

__global__ void k_invert(const int32_t *__restrict__ sorted_old, int64_t dim, int32_t *__restrict__ new_of_old,
                         int32_t *__restrict__ old_of_new)
{
    const int64_t pos = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (pos < dim) {
        const int32_t old = sorted_old[pos];
        new_of_old[old] = (int32_t)pos;
        old_of_new[pos] = old;
    }
}

__global__ void k_relabel(int32_t *__restrict__ indices, int64_t nnz, const int32_t *__restrict__ new_of_old)
{
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < nnz; e += (int64_t)gridDim.x * blockDim.x)
        indices[e] = new_of_old[indices[e]];
}

__global__ void k_mass_of_first(const uint32_t *__restrict__ counts, const int32_t *__restrict__ old_of_new, int64_t first,
                                unsigned long long *__restrict__ out)
{
    unsigned long long s = 0;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < first; i += (int64_t)gridDim.x * blockDim.x)
        s += counts[old_of_new[i]];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if ((threadIdx.x & 31) == 0 && s) atomicAdd(out, s);
}

// out[1] += number of coordinates with more than `long_len` entries
__global__ void k_count_long(const int64_t *__restrict__ indptr, int64_t n_coord, int32_t long_len,
                             unsigned long long *__restrict__ out)
{
    unsigned long long s = 0;
    for (int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; c < n_coord; c += (int64_t)gridDim.x * blockDim.x)
        s += (indptr[c + 1] - indptr[c]) > long_len ? 1u : 0u;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if ((threadIdx.x & 31) == 0 && s) atomicAdd(out + 1, s);
}

// dst[i] = src[map[i]]
__global__ void k_gather_f32(const float *__restrict__ src, const int32_t *__restrict__ map, int64_t n, float *__restrict__ dst)
{
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        dst[i] = src[map[i]];
}

} // namespace

// counts: dim zeroed uint32; keys/vals: two arrays of dim each; mass: two zeroed 64-bit words (non-zeros on the first
// hot_ids ids; coordinates longer than long_len).
cudaError_t launch_frequency_remap(Glm &g, uint32_t *counts, uint64_t *keys[2], int32_t *vals[2], uint32_t *hist,
                                   uint32_t *scan_sums, int64_t hot_ids, int32_t long_len, unsigned long long *mass)
{
    const int64_t dim = g.dim;
    const unsigned wide = (unsigned)g.sm_count * 8;
    k_count_ids<<<wide, kT, 0, g.stream>>>(g.indices, g.nnz, counts);
    k_freq_keys<<<blocks_for(dim), kT, 0, g.stream>>>(counts, dim, keys[0], vals[0]);
    int cur = 0;
    for (int pass = 0; pass < 8; ++pass) {
        cudaError_t e = radix_pass(keys[cur], vals[cur], keys[cur ^ 1], vals[cur ^ 1], nullptr, dim, 8 * pass, hist,
                                   scan_sums, g.stream);
        if (e != cudaSuccess) return e;
        cur ^= 1;
    }
    k_invert<<<blocks_for(dim), kT, 0, g.stream>>>(vals[cur], dim, g.new_of_old, g.old_of_new);
    k_relabel<<<wide, kT, 0, g.stream>>>(g.indices, g.nnz, g.new_of_old);
    const int64_t first = hot_ids < dim ? hot_ids : dim;
    k_mass_of_first<<<blocks_for(first), kT, 0, g.stream>>>(counts, g.old_of_new, first, mass);
    k_count_long<<<wide, kT, 0, g.stream>>>(g.indptr, g.n_coord, long_len, mass);
    return cudaGetLastError();
}

cudaError_t launch_gather_f32(Glm &g, const float *src, const int32_t *map, int64_t n, float *dst)
{
    k_gather_f32<<<(unsigned)g.sm_count * 4, kT, 0, g.stream>>>(src, map, n, dst);
    return cudaGetLastError();
}

} // namespace chicle
