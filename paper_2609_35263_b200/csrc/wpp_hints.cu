// Prefix hints (Section 4.3): chained hashes of full token blocks (GPU and host) and the counted, sharded index
// with the gallop-and-bisect probe (host).
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>
#include <new>
#include <unordered_map>

#include "../../include/wpp.h"
#include "wpp_host.h"

namespace {

__host__ __device__ inline uint64_t mix64(uint64_t x) {     // splitmix64 finaliser
    x ^= x >> 30;
    x *= 0xBF58476D1CE4E5B9ull;
    x ^= x >> 27;
    x *= 0x94D049BB133111EBull;
    x ^= x >> 31;
    return x;
}
__host__ __device__ inline uint64_t token_term(int32_t token, uint32_t k) {
    return mix64((((uint64_t)(uint32_t)token << 32) | k) ^ 0xD6E8FEB86659FD93ull);
}
__host__ __device__ inline uint64_t chain_step(uint64_t parent, uint64_t digest, uint64_t extra, uint64_t salt_term) {
    return mix64(parent ^ mix64(digest + extra) ^ salt_term);
}

// One warp per token block: lanes add the terms of their tokens, a shuffle tree adds the lanes.  What is left
// where the block's hash will go is mix64(digest + extraKeys): everything of the chain step that does not depend
// on the parent hash is done here, in parallel.
__global__ void __launch_bounds__(256) wpp_block_digest_kernel(const int32_t* __restrict__ tokens,
                                                                const int64_t* __restrict__ token_offsets,
                                                                const int64_t* __restrict__ block_offsets,
                                                                int num_requests, int block_size,
                                                                const uint64_t* __restrict__ extra,
                                                                uint64_t* __restrict__ out, int64_t total_blocks) {
    const int lane = threadIdx.x & 31;
    const int64_t warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    for (int64_t blk = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5; blk < total_blocks; blk += warps) {
        int lo = 0, hi = num_requests;              // largest i with block_offsets[i] <= blk
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (block_offsets[mid] <= blk) lo = mid; else hi = mid;
        }
        const int32_t* src = tokens + token_offsets[lo] + (blk - block_offsets[lo]) * block_size;
        uint64_t d = 0;
        for (int k = lane; k < block_size; k += 32) d += token_term(src[k], (uint32_t)k);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
        if (lane == 0) out[blk] = mix64(d + (extra ? extra[blk] : 0ull));
    }
}

// One thread per request walks its blocks in order: H_i = mix64(H_{i-1} xor m_i xor salt term).  The chain is
// sequential by definition; the loads are not, so eight of them are in flight ahead of it.
__global__ void wpp_hash_chain_kernel(const int64_t* __restrict__ block_offsets, int num_requests, uint64_t salt_term,
                                      uint64_t* __restrict__ hashes) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= num_requests) return;
    uint64_t h = 0;
    const int64_t end = block_offsets[i + 1];
    int64_t b = block_offsets[i];
    if (b + 8 <= end) {
        uint64_t cur[8], nxt[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) cur[k] = hashes[b + k];
        for (; b + 8 <= end; b += 8) {
            const bool more = b + 16 <= end;
            if (more) {                         // the next eight are requested before this eight is chained
#pragma unroll
                for (int k = 0; k < 8; ++k) nxt[k] = hashes[b + 8 + k];
            }
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                h = mix64(h ^ cur[k] ^ salt_term);
                cur[k] = h;
            }
#pragma unroll
            for (int k = 0; k < 8; ++k) hashes[b + k] = cur[k];
            if (more) {
#pragma unroll
                for (int k = 0; k < 8; ++k) cur[k] = nxt[k];
            }
        }
    }
    for (; b < end; ++b) {
        h = mix64(h ^ hashes[b] ^ salt_term);
        hashes[b] = h;
    }
}

constexpr int kShards = 16;
struct Key {
    int32_t window;
    uint64_t hash;
    bool operator==(const Key& o) const { return window == o.window && hash == o.hash; }
};
struct KeyHash {
    size_t operator()(const Key& k) const { return (size_t)mix64(k.hash ^ ((uint64_t)(uint32_t)k.window << 1)); }
};

}  // namespace

struct wpp_hint_index {
    std::unordered_map<Key, int64_t, KeyHash> map[kShards];
    mutable std::mutex lock[kShards];
    static int shard(uint64_t h) { return (int)((h >> 7) & (kShards - 1)); }
    bool has(int32_t window, uint64_t h) const {
        const int s = shard(h);
        std::lock_guard<std::mutex> g(lock[s]);
        return map[s].count(Key{window, h}) != 0;
    }
};

extern "C" int wpp_hash_blocks(const wpp_ctx* ctx, const int32_t* tokens, const int64_t* token_offsets,
                               const int64_t* block_offsets, int32_t num_requests, int32_t block_size, uint64_t salt,
                               const uint64_t* extra, uint64_t* hashes_out, int64_t total_blocks, void* cuda_stream) {
    if (!ctx || num_requests < 0 || block_size < 1 || total_blocks < 0) return WPP_ERR_INVALID_ARG;
    if (num_requests == 0 || total_blocks == 0) return WPP_OK;
    if (!tokens || !token_offsets || !block_offsets || !hashes_out) return WPP_ERR_INVALID_ARG;
    if (int rc = wpp_ctx_check_device(ctx)) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    int64_t blocks = (total_blocks * 32 + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    wpp_block_digest_kernel<<<(unsigned)blocks, 256, 0, st>>>(tokens, token_offsets, block_offsets, num_requests,
                                                              block_size, extra, hashes_out, total_blocks);
    wpp_hash_chain_kernel<<<(unsigned)((num_requests + 31) / 32), 32, 0, st>>>(
        block_offsets, num_requests, salt * 0x9E3779B97F4A7C15ull, hashes_out);
    return cudaGetLastError() == cudaSuccess ? WPP_OK : WPP_ERR_CUDA;
}

extern "C" int wpp_hash_blocks_host(const int32_t* tokens, int64_t n_tokens, int32_t block_size, uint64_t salt,
                                    const uint64_t* extra, uint64_t* hashes_out) {
    if (n_tokens < 0 || block_size < 1) return WPP_ERR_INVALID_ARG;
    const int64_t n = n_tokens / block_size;
    if (n == 0) return WPP_OK;
    if (!tokens || !hashes_out) return WPP_ERR_INVALID_ARG;
    uint64_t h = 0;
    for (int64_t b = 0; b < n; ++b) {
        uint64_t d = 0;
        for (int k = 0; k < block_size; ++k) d += token_term(tokens[b * block_size + k], (uint32_t)k);
        h = chain_step(h, d, extra ? extra[b] : 0ull, salt * 0x9E3779B97F4A7C15ull);
        hashes_out[b] = h;
    }
    return WPP_OK;
}

extern "C" int wpp_hint_index_create(wpp_hint_index** out) {
    if (!out) return WPP_ERR_INVALID_ARG;
    *out = new (std::nothrow) wpp_hint_index();
    return *out ? WPP_OK : WPP_ERR_INVALID_ARG;
}
extern "C" int wpp_hint_index_destroy(wpp_hint_index* idx) {
    delete idx;
    return WPP_OK;
}
extern "C" int wpp_hint_index_add(wpp_hint_index* idx, int32_t window, const uint64_t* hashes, int64_t n) {
    if (!idx || n < 0 || (n > 0 && !hashes)) return WPP_ERR_INVALID_ARG;
    for (int64_t i = 0; i < n; ++i) {
        const int s = wpp_hint_index::shard(hashes[i]);
        std::lock_guard<std::mutex> g(idx->lock[s]);
        idx->map[s][Key{window, hashes[i]}] += 1;
    }
    return WPP_OK;
}
extern "C" int wpp_hint_index_remove(wpp_hint_index* idx, int32_t window, const uint64_t* hashes, int64_t n) {
    if (!idx || n < 0 || (n > 0 && !hashes)) return WPP_ERR_INVALID_ARG;
    for (int64_t i = 0; i < n; ++i) {
        const int s = wpp_hint_index::shard(hashes[i]);
        std::lock_guard<std::mutex> g(idx->lock[s]);
        auto it = idx->map[s].find(Key{window, hashes[i]});
        if (it == idx->map[s].end()) continue;
        if (--it->second <= 0) idx->map[s].erase(it);
    }
    return WPP_OK;
}
extern "C" int64_t wpp_hint_index_size(const wpp_hint_index* idx) {
    if (!idx) return -1;
    int64_t n = 0;
    for (int s = 0; s < kShards; ++s) {
        std::lock_guard<std::mutex> g(idx->lock[s]);
        n += (int64_t)idx->map[s].size();
    }
    return n;
}

extern "C" int wpp_hint_probe(const wpp_hint_index* idx, int32_t window, const uint64_t* hashes, int64_t n_blocks,
                              int64_t* matched_blocks, int32_t* probes_or_null) {
    if (!idx || n_blocks < 0 || !matched_blocks || (n_blocks > 0 && !hashes)) return WPP_ERR_INVALID_ARG;
    int32_t probes = 0;
    int64_t lo = 0, hi = n_blocks + 1;          // depth lo matches (0: nothing known), depth hi misses (or is past the end)
    for (int64_t d = 1; d <= n_blocks; d *= 2) {
        ++probes;
        if (idx->has(window, hashes[d - 1])) {
            lo = d;
        } else {
            hi = d;
            break;
        }
    }
    while (hi - lo > 1) {
        const int64_t mid = (lo + hi) / 2;
        ++probes;
        if (idx->has(window, hashes[mid - 1])) lo = mid; else hi = mid;
    }
    *matched_blocks = lo;
    if (probes_or_null) *probes_or_null = probes;
    return WPP_OK;
}

extern "C" int wpp_hint_probe_recurrent(const wpp_hint_index* idx, int32_t window, const uint64_t* hashes,
                                        int64_t limit_blocks, int64_t* matched_blocks, int32_t* probes_or_null) {
    if (!idx || limit_blocks < 0 || !matched_blocks || (limit_blocks > 0 && !hashes)) return WPP_ERR_INVALID_ARG;
    int32_t probes = 0;
    int64_t d = limit_blocks;                   // snapshots are sparse: walk back from the attention-limited endpoint
    for (; d >= 1; --d) {
        ++probes;
        if (idx->has(window, hashes[d - 1])) break;
    }
    *matched_blocks = d;
    if (probes_or_null) *probes_or_null = probes;
    return WPP_OK;
}
