// Mobile data chunks: where the chunk boundaries fall and which task holds which chunk. Host-side integer logic of the
// scheduler (the paper's Sec. 3 core concepts, Sec. 4.4 chunk format, Sec. 4.5 elastic scaling and rebalancing
// policies, Sec. 5.3 on how scaling out reshuffles); the placement these functions produce is turned into a partition
// on the device by chicle_partition_chunks. No GPU is touched here.
#include <algorithm>
#include <cstdint>
#include <utility>
#include <vector>

#include "chicle_internal.cuh"

namespace {

constexpr int64_t kStateBytes = 8;  // a sample's dual variable and label travel with it
constexpr int64_t kEntryBytes = 8;  // int32 index + fp32 value
constexpr uint64_t kScaleOutStream = 0xA0761D6478BD642FULL;

// chunks[first .. last) sorted by (mix64(salt ^ chunk), chunk)
void order_by_key(std::vector<int64_t> &chunks, uint64_t salt)
{
    std::vector<std::pair<uint64_t, int64_t>> keyed(chunks.size());
    for (size_t i = 0; i < chunks.size(); ++i) keyed[i] = {chicle::mix64(salt ^ (uint64_t)chunks[i]), chunks[i]};
    std::sort(keyed.begin(), keyed.end());
    for (size_t i = 0; i < chunks.size(); ++i) chunks[i] = keyed[i].second;
}

} // namespace

extern "C" {

int64_t chicle_chunks_cut(int64_t n_coord, const int64_t *host_indptr, int64_t dense_dim, int64_t chunk_bytes, int64_t *host_chunk_off)
{
    if (n_coord < 1 || chunk_bytes < 1 || !host_chunk_off || (!host_indptr && dense_dim < 1)) return -1;
    if (host_indptr)
        for (int64_t i = 0; i < n_coord; ++i)
            if (host_indptr[i + 1] < host_indptr[i]) return -1;
    int64_t C = 0, used = 0;
    host_chunk_off[0] = 0;
    for (int64_t i = 0; i < n_coord; ++i) {
        const int64_t bytes = (host_indptr ? kEntryBytes * (host_indptr[i + 1] - host_indptr[i]) : 4 * dense_dim) + kStateBytes;
        if (i > host_chunk_off[C] && used + bytes > chunk_bytes) {
            host_chunk_off[++C] = i;
            used = 0;
        }
        used += bytes;
    }
    host_chunk_off[++C] = n_coord;
    return C;
}

chicle_status_t chicle_chunks_assign(int64_t n_chunks, int32_t K, uint64_t seed, int32_t *host_chunk_task)
{
    try {
    if (K < 1 || (int64_t)K > n_chunks || !host_chunk_task) return CHICLE_ERR_INVALID_ARG;
    std::vector<int64_t> order((size_t)n_chunks);
    for (int64_t c = 0; c < n_chunks; ++c) order[(size_t)c] = c;
    order_by_key(order, chicle::mix64(seed));
    const int64_t base = n_chunks / K, extra = n_chunks % K;
    int64_t pos = 0;
    for (int32_t k = 0; k < K; ++k) {
        const int64_t m = base + (k < extra ? 1 : 0);
        for (int64_t i = 0; i < m; ++i) host_chunk_task[order[(size_t)(pos + i)]] = k;
        pos += m;
    }
    return CHICLE_OK;
    } catch (...) { return CHICLE_ERR_OOM; }
}

chicle_status_t chicle_chunks_scale_in(int64_t n_chunks, int32_t K_old, int32_t K_new, int32_t *host_chunk_task)
{
    try {
    if (K_new < 1 || K_new > K_old || n_chunks < 1 || !host_chunk_task) return CHICLE_ERR_INVALID_ARG;
    int32_t next = 0;
    for (int64_t c = 0; c < n_chunks; ++c) {
        if (host_chunk_task[c] >= K_new) {
            host_chunk_task[c] = next;
            next = next + 1 == K_new ? 0 : next + 1;
        }
    }
    return CHICLE_OK;
    } catch (...) { return CHICLE_ERR_OOM; }
}

chicle_status_t chicle_chunks_scale_out(int64_t n_chunks, int32_t K_old, int32_t K_new, uint64_t seed, int32_t *host_chunk_task)
{
    try {
    if (K_old < 1 || K_new < K_old || n_chunks < 1 || !host_chunk_task) return CHICLE_ERR_INVALID_ARG;
    const int32_t add = K_new - K_old;
    if (add == 0) return CHICLE_OK;
    std::vector<std::vector<int64_t>> held((size_t)K_old);
    for (int64_t c = 0; c < n_chunks; ++c) {
        const int32_t t = host_chunk_task[c];
        if (t < 0 || t >= K_old) return CHICLE_ERR_INVALID_ARG;
        held[(size_t)t].push_back(c);
    }
    const uint64_t salt = chicle::mix64(seed ^ kScaleOutStream);
    int32_t turn = 0;
    for (int32_t j = 0; j < K_old; ++j) {
        std::vector<int64_t> &mine = held[(size_t)j];
        order_by_key(mine, salt);
        const int64_t give = (int64_t)mine.size() * add / K_new;
        for (int64_t i = 0; i < give; ++i) {
            host_chunk_task[mine[(size_t)i]] = K_old + turn;
            turn = turn + 1 == add ? 0 : turn + 1;
        }
    }
    return CHICLE_OK;
    } catch (...) { return CHICLE_ERR_OOM; }
}

int chicle_chunks_rebalance_step(int64_t n_chunks, const int64_t *host_chunk_off, int32_t K, const double *host_time_per_sample,
                                 int32_t *host_chunk_task)
{
    try {
    if (K < 1 || n_chunks < 1 || !host_chunk_off || !host_time_per_sample || !host_chunk_task) return -1;
    std::vector<int64_t> samples((size_t)K, 0);
    for (int64_t c = 0; c < n_chunks; ++c) {
        if (host_chunk_task[c] < 0 || host_chunk_task[c] >= K) return -1;
        samples[(size_t)host_chunk_task[c]] += host_chunk_off[c + 1] - host_chunk_off[c];
    }
    int32_t slow = 0, fast = 0;
    double t_slow = 0.0, t_fast = 0.0;
    for (int32_t k = 0; k < K; ++k) {
        const double t = (double)samples[(size_t)k] * host_time_per_sample[k];
        if (k == 0 || t > t_slow) { slow = k; t_slow = t; } // ties: the lower task number
        if (k == 0 || t < t_fast) { fast = k; t_fast = t; }
    }
    if (slow == fast) return 0;
    int64_t last = -1, held = 0;
    for (int64_t c = 0; c < n_chunks; ++c)
        if (host_chunk_task[c] == slow) { last = c; ++held; }
    if (held <= 1) return 0;
    const double one_chunk = (double)(host_chunk_off[last + 1] - host_chunk_off[last]) * host_time_per_sample[slow];
    if (t_slow - t_fast <= one_chunk) return 0;
    host_chunk_task[last] = fast;
    return 1;
    } catch (...) { return -1; }
}

} // extern "C"
