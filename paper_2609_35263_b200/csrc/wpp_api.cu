// C-ABI entry points that touch CUDA: context, tensor-map construction, argument checks and launches.
// There is no CPU fallback: without a usable device wpp_create fails and nothing else can be called.
#include <cuda.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#include <mutex>
#include <new>

#include "../../include/wpp.h"
#include "wpp_device.h"
#include "wpp_host.h"
#include "wpp_plan_format.h"

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// A tensor map depends only on (base pointer, extents, strides, box); serving loops call with the same pools and
// the same query buffers wave after wave, so the context keeps the maps it has encoded.
struct MapKey {
    const void* base;
    uint64_t dims[4], strides[3];
    uint32_t box[4];
    int rank;
};
struct MapEntry {
    MapKey key;
    CUtensorMap map;
    uint64_t used;      // 0 = empty; else the tick of the last use (least recently used entry is replaced)
};
constexpr int kMapCacheEntries = 32;
constexpr int kLateRescaleOnPct = 30, kLateRescaleOffPct = 15;   // share of key steps that rescale O (see choose_late_rescale)

struct wpp_ctx {
    int device;
    int sm_count;
    int smem_optin;
    int last_cuda_error;
    int64_t launches;
    EncodeTiledFn encode_tiled;
    void* static_scratch;           // device address of the built-in scratch array on this context's device
    // Where a moved row reference rescales O (see the attention kernel's kLate) is chosen per launch from what the
    // kernels of earlier launches counted: key steps and steps that rescaled, added up in mapped host memory.
    unsigned long long* stats_host; // [0] key steps, [1] rescaling steps (pinned, mapped; the kernels add to it)
    unsigned long long* stats_dev;  // the same two words as the device sees them
    unsigned long long seen_steps, seen_moves;   // the counters when the choice was last looked at
    int rescale_mode;               // 0: always before the exponentials (default), 1: always after, 2: chosen from the counters
    int late_rescale;               // the current choice
    std::mutex* map_lock;
    uint64_t map_tick;
    MapEntry maps[kMapCacheEntries];
};

// ---------------------------------------------------------------------------------------------------------------
// Built-in scratch for the entry point that allocates nothing (wpp_prefill_attention_varlen_static, below).
// Some callers of this library cannot call cudaMalloc when a wave is due: the serving process has handed all free
// device memory to the KV page pool, and an allocation on the execution path would fail or stall the stream.
#define WPP_STATIC_SCRATCH_BYTES (16u << 20)
static __device__ __align__(256) unsigned char wpp_static_scratch[WPP_STATIC_SCRATCH_BYTES];

extern "C" size_t wpp_static_scratch_bytes(void) { return (size_t)WPP_STATIC_SCRATCH_BYTES; }

// In host code the array's name is only a handle, not a device address.  The address is looked up once per
// device, with that device current (the symbol resolves to the current device's copy).  The look-up is also
// what makes the CUDA runtime load this module on the device, i.e. what reserves the 16 MiB there: it runs
// inside wpp_create, at start-up, so that no later call has to find memory for it.
static std::mutex g_scratch_lock;
static void* g_scratch_ptr[64];

static cudaError_t static_scratch_address(int device, void** out) {
    std::lock_guard<std::mutex> guard(g_scratch_lock);
    if (device < 0 || device >= 64) return cudaErrorInvalidDevice;
    if (!g_scratch_ptr[device]) {
        int cur = -1;
        cudaError_t e = cudaGetDevice(&cur);
        if (e != cudaSuccess) return e;
        if (cur != device && (e = cudaSetDevice(device)) != cudaSuccess) return e;
        void* ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, wpp_static_scratch);
        if (cur != device) cudaSetDevice(cur);
        if (e != cudaSuccess) return e;
        if (!ptr) return cudaErrorInvalidSymbol;
        g_scratch_ptr[device] = ptr;
    }
    *out = g_scratch_ptr[device];
    return cudaSuccess;
}

extern "C" int wpp_ctx_sm_count(const wpp_ctx* ctx) { return ctx ? ctx->sm_count : 148; }

static int cuda_fail(const wpp_ctx* ctx, int err) {
    if (ctx) const_cast<wpp_ctx*>(ctx)->last_cuda_error = err;
    return WPP_ERR_CUDA;
}

extern "C" int wpp_create(wpp_ctx** out, int cuda_device) {
    if (!out) return WPP_ERR_INVALID_ARG;
    *out = nullptr;
    int n = 0;
    cudaError_t e = cudaGetDeviceCount(&n);
    if (e != cudaSuccess || cuda_device < 0 || cuda_device >= n) return WPP_ERR_CUDA;
    cudaDeviceProp prop;
    if ((e = cudaGetDeviceProperties(&prop, cuda_device)) != cudaSuccess) return WPP_ERR_CUDA;
    if (prop.major != 10) return WPP_ERR_UNSUPPORTED;   // the kernels are built for sm_100a only
    wpp_ctx* c = static_cast<wpp_ctx*>(calloc(1, sizeof(wpp_ctx)));
    if (!c) return WPP_ERR_INVALID_ARG;
    c->device = cuda_device;
    c->sm_count = prop.multiProcessorCount;
    c->smem_optin = (int)prop.sharedMemPerBlockOptin;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn) {
        free(c);
        return WPP_ERR_CUDA;
    }
    c->encode_tiled = reinterpret_cast<EncodeTiledFn>(fn);
    if (static_scratch_address(cuda_device, &c->static_scratch) != cudaSuccess) {
        free(c);
        return WPP_ERR_CUDA;
    }
    c->map_lock = new (std::nothrow) std::mutex();
    if (!c->map_lock) {
        free(c);
        return WPP_ERR_INVALID_ARG;
    }
    // two counters the attention kernels add to and the next call reads without synchronising (a missing mapping
    // only means that the choice they feed stays at its default)
    void* hp = nullptr;
    if (cudaHostAlloc(&hp, 64, cudaHostAllocMapped | cudaHostAllocPortable) == cudaSuccess) {
        memset(hp, 0, 64);
        void* dp = nullptr;
        if (cudaHostGetDevicePointer(&dp, hp, 0) == cudaSuccess) {
            c->stats_host = static_cast<unsigned long long*>(hp);
            c->stats_dev = static_cast<unsigned long long*>(dp);
        } else {
            cudaFreeHost(hp);
        }
    }
    (void)cudaGetLastError();
    *out = c;
    return WPP_OK;
}

extern "C" int wpp_destroy(wpp_ctx* ctx) {
    if (ctx) {
        delete ctx->map_lock;
        if (ctx->stats_host) cudaFreeHost(ctx->stats_host);
    }
    free(ctx);
    return WPP_OK;
}

extern "C" int wpp_set_rescale_mode(wpp_ctx* ctx, int mode) {
    if (!ctx || mode < 0 || mode > 2) return WPP_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> guard(*ctx->map_lock);
    ctx->rescale_mode = mode;
    return WPP_OK;
}

extern "C" int wpp_rescale_stats(const wpp_ctx* ctx, uint64_t* key_steps, uint64_t* rescaling_steps, int* late) {
    if (!ctx) return WPP_ERR_INVALID_ARG;
    volatile unsigned long long* s = ctx->stats_host;
    if (key_steps) *key_steps = s ? s[0] : 0;
    if (rescaling_steps) *rescaling_steps = s ? s[1] : 0;
    if (late) *late = ctx->rescale_mode == 1 || (ctx->rescale_mode == 2 && ctx->late_rescale);
    return WPP_OK;
}

// The choice for the next launch: with the counters' increase since the last look, once there are enough steps to
// judge by; between the two thresholds the choice stays what it was.
static int choose_late_rescale(const wpp_ctx* cctx) {
    wpp_ctx* c = const_cast<wpp_ctx*>(cctx);
    std::lock_guard<std::mutex> guard(*c->map_lock);
    if (c->rescale_mode != 2) return c->rescale_mode == 1;
    if (!c->stats_host) return 0;
    volatile unsigned long long* s = c->stats_host;
    const unsigned long long steps = s[0], moves = s[1];
    const unsigned long long ds = steps - c->seen_steps, dm = moves - c->seen_moves;
    if (ds >= 4096) {
        if (dm * 100 >= ds * kLateRescaleOnPct) c->late_rescale = 1;
        else if (dm * 100 < ds * kLateRescaleOffPct) c->late_rescale = 0;
        c->seen_steps = steps;
        c->seen_moves = moves;
    }
    return c->late_rescale;
}

// Every launching entry point runs with the context's device current: a call made with another device current
// would launch there with this device's pointers and tensor maps.
extern "C" int wpp_ctx_check_device(const wpp_ctx* ctx) {
    int cur = -1;
    cudaError_t e = cudaGetDevice(&cur);
    if (e != cudaSuccess) return cuda_fail(ctx, (int)e);
    return cur == ctx->device ? WPP_OK : WPP_ERR_INVALID_ARG;
}

extern "C" int wpp_last_cuda_error(const wpp_ctx* ctx) { return ctx ? ctx->last_cuda_error : 0; }
extern "C" int64_t wpp_launch_count(const wpp_ctx* ctx) { return ctx ? ctx->launches : 0; }

extern "C" int wpp_selftest_bounded_wait(const wpp_ctx* ctx, int64_t limit_cycles, int32_t* status_dev,
                                         int64_t* waited_cycles_dev, void* cuda_stream) {
    if (!ctx || !status_dev || limit_cycles < 1 || limit_cycles > (1ll << 30)) return WPP_ERR_INVALID_ARG;
    if (int rc = wpp_ctx_check_device(ctx)) return rc;
    int e = wpp_launch_selftest_wait((long long)limit_cycles, status_dev,
                                     reinterpret_cast<long long*>(waited_cycles_dev), cuda_stream);
    if (e != 0) return cuda_fail(ctx, e);
    const_cast<wpp_ctx*>(ctx)->launches += 1;
    return WPP_OK;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

// bf16 tensor map with 128-byte swizzle; dims/strides innermost first, strides in bytes for dims 1..rank-1.
// Looked up in the context's cache first (six maps per attention call; encoding them costs more than a small
// wave's kernel).
static int make_map(const wpp_ctx* cctx, CUtensorMap* m, const void* base, int rank, const uint64_t* dims,
                    const uint64_t* strides_bytes, const uint32_t* box) {
    wpp_ctx* ctx = const_cast<wpp_ctx*>(cctx);
    MapKey key;
    memset(&key, 0, sizeof(key));
    key.base = base;
    key.rank = rank;
    for (int i = 0; i < rank; ++i) { key.dims[i] = dims[i]; key.box[i] = box[i]; }
    for (int i = 0; i < rank - 1; ++i) key.strides[i] = strides_bytes[i];
    std::lock_guard<std::mutex> guard(*ctx->map_lock);
    const uint64_t tick = ++ctx->map_tick;
    int victim = 0;
    for (int i = 0; i < kMapCacheEntries; ++i) {
        MapEntry& en = ctx->maps[i];
        if (en.used && memcmp(&en.key, &key, sizeof(key)) == 0) {
            en.used = tick;
            *m = en.map;
            return WPP_OK;
        }
        if (en.used < ctx->maps[victim].used) victim = i;
    }
    cuuint64_t gd[4];
    cuuint64_t gs[3];
    cuuint32_t bx[4], es[4];
    for (int i = 0; i < rank; ++i) { gd[i] = dims[i]; bx[i] = box[i]; es[i] = 1; }
    for (int i = 0; i < rank - 1; ++i) gs[i] = strides_bytes[i];
    CUresult r = ctx->encode_tiled(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), gd,
                                   gs, bx, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cuda_fail(ctx, (int)r);
    MapEntry& en = ctx->maps[victim];
    memcpy(&en.key, &key, sizeof(key));
    en.map = *m;
    en.used = tick;
    return WPP_OK;
}

extern "C" int wpp_kv_append(const wpp_ctx* ctx, const wpp_batch_desc* desc, const void* k_new, const void* v_new,
                             void* k_cache, void* v_cache, const int32_t* block_tables, const int32_t* prefix_lens,
                             const int32_t* chunk_lens, const void* plan_host, const void* plan_dev,
                             int32_t* status_dev, void* cuda_stream) {
    if (!ctx) return WPP_ERR_INVALID_ARG;
    wpp_batch_desc d;
    int rc = wpp_resolve_desc(desc, &d);
    if (rc != WPP_OK) return rc;
    const WppPlanHeader* hd = nullptr;
    if ((rc = wpp_check_plan(plan_host, &d, &hd)) != WPP_OK) return rc;
    if (hd->total_new_tokens == 0) return WPP_OK;
    if ((rc = wpp_ctx_check_device(ctx)) != WPP_OK) return rc;
    if (!k_new || !v_new || !k_cache || !v_cache || !block_tables || !prefix_lens || !chunk_lens || !plan_dev)
        return WPP_ERR_INVALID_ARG;
    if (!aligned16(k_new) || !aligned16(v_new) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(plan_dev))
        return WPP_ERR_INVALID_ARG;
    wpp::AppendParams p;
    memset(&p, 0, sizeof(p));
    p.plan = plan_dev;
    p.k_new = static_cast<const uint4*>(k_new);
    p.v_new = static_cast<const uint4*>(v_new);
    p.k_cache = static_cast<uint4*>(k_cache);
    p.v_cache = static_cast<uint4*>(v_cache);
    p.block_tables = block_tables;
    p.prefix_lens = prefix_lens;
    p.chunk_lens = chunk_lens;
    p.status = status_dev;
    p.kvnew_token_stride = d.kvnew_token_stride / 8;
    p.kvnew_head_stride = d.kvnew_head_stride / 8;
    p.kv_page_stride = d.kv_page_stride / 8;
    p.kv_head_stride = d.kv_head_stride / 8;
    p.kv_token_stride = d.kv_token_stride / 8;
    p.num_requests = d.num_requests;
    p.num_kv_heads = d.num_kv_heads;
    p.vec_per_row = d.head_dim / 8;
    p.page_size = d.page_size;
    p.max_blocks = d.max_blocks_per_req;
    p.num_pages = d.num_pages;
    p.total_new_tokens = hd->total_new_tokens;
    int e = wpp_launch_append(&p, ctx->sm_count, cuda_stream);
    if (e != 0) return cuda_fail(ctx, e);
    const_cast<wpp_ctx*>(ctx)->launches += 1;
    return WPP_OK;
}

extern "C" int wpp_prefill_attention_varlen(const wpp_ctx* ctx, const wpp_batch_desc* desc, const void* q, void* out,
                                            float* lse_or_null, const void* k_cache, const void* v_cache,
                                            const int32_t* block_tables, const int32_t* prefix_lens,
                                            const int32_t* chunk_lens, const void* plan_host, const void* plan_dev,
                                            void* workspace, size_t workspace_bytes, int32_t* status_dev,
                                            void* cuda_stream) {
    if (!ctx) return WPP_ERR_INVALID_ARG;
    wpp_batch_desc d;
    int rc = wpp_resolve_desc(desc, &d);
    if (rc != WPP_OK) return rc;
    const WppPlanHeader* hd = nullptr;
    if ((rc = wpp_check_plan(plan_host, &d, &hd)) != WPP_OK) return rc;
    if (hd->tile_m > WPP_MAX_TILE_M || hd->shape < 1 || hd->shape > 2) return WPP_ERR_PLAN_MISMATCH;
    if (hd->total_new_tokens == 0 || hd->num_units == 0) return WPP_OK;
    if ((rc = wpp_ctx_check_device(ctx)) != WPP_OK) return rc;
    if (!q || !out || !k_cache || !v_cache || !block_tables || !prefix_lens || !chunk_lens || !plan_dev)
        return WPP_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(out) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(plan_dev))
        return WPP_ERR_INVALID_ARG;
    // the workspace always holds the tile counter, and the split partials behind it when the plan has any
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) != 0) return WPP_ERR_INVALID_ARG;
    if (workspace_bytes < hd->workspace_bytes) return WPP_ERR_WORKSPACE_TOO_SMALL;
    if (d.num_pages == 0) return WPP_ERR_INVALID_ARG;

    CUtensorMap tq[4], tk, tv;
    for (int i = 0; i < 4; ++i) {       // boxes of 128, 64, 32, 16 query rows (packed heads take fewer rows per head)
        const uint64_t dims[3] = {(uint64_t)d.head_dim, (uint64_t)d.num_q_heads, (uint64_t)hd->total_new_tokens};
        const uint64_t strides[2] = {(uint64_t)d.q_head_stride * 2, (uint64_t)d.q_token_stride * 2};
        const uint32_t box[3] = {64, 1, (uint32_t)(128 >> i)};
        if ((rc = make_map(ctx, &tq[i], q, 3, dims, strides, box)) != WPP_OK) return rc;
    }
    {
        const uint64_t dims[4] = {(uint64_t)d.head_dim, (uint64_t)d.page_size, (uint64_t)d.num_kv_heads,
                                  (uint64_t)d.num_pages};
        const uint64_t strides[3] = {(uint64_t)d.kv_token_stride * 2, (uint64_t)d.kv_head_stride * 2,
                                     (uint64_t)d.kv_page_stride * 2};
        // the small shape works on 64-key steps: its boxes have at most 64 rows (half a 128-token page)
        const uint32_t box_rows = (hd->shape == 2 && d.page_size > 64) ? 64u : (uint32_t)d.page_size;
        const uint32_t box[4] = {64, box_rows, 1, 1};
        if ((rc = make_map(ctx, &tk, k_cache, 4, dims, strides, box)) != WPP_OK) return rc;
        if ((rc = make_map(ctx, &tv, v_cache, 4, dims, strides, box)) != WPP_OK) return rc;
    }

    wpp::AttnParams p;
    memset(&p, 0, sizeof(p));
    p.plan = plan_dev;
    p.block_tables = block_tables;
    p.prefix_lens = prefix_lens;
    p.chunk_lens = chunk_lens;
    p.out = static_cast<__nv_bfloat16*>(out);
    p.lse = lse_or_null;
    p.tile_counter = static_cast<uint32_t*>(workspace);
    p.ws_o = reinterpret_cast<float*>(static_cast<char*>(workspace) + WPP_WS_HEADER_BYTES);
    p.ws_lse = p.ws_o + (size_t)hd->num_split_slots * 2 * WPP_HALF_M * d.head_dim;
    p.status = status_dev;
    p.o_token_stride = d.o_token_stride;
    p.o_head_stride = d.o_head_stride;
    p.num_q_heads = d.num_q_heads;
    p.group = d.num_q_heads / d.num_kv_heads;
    p.page_size = d.page_size;
    p.max_blocks = d.max_blocks_per_req;
    p.num_pages = d.num_pages;
    const double scale = d.sm_scale > 0.f ? (double)d.sm_scale : 1.0 / sqrt((double)d.head_dim);
    p.scale_log2 = (float)(scale * 1.4426950408889634);

    // the counter the CTAs take their tiles from starts at zero (a memset node on the caller's stream)
    int e = (int)cudaMemsetAsync(workspace, 0, WPP_WS_HEADER_BYTES, (cudaStream_t)cuda_stream);
    if (e != 0) return cuda_fail(ctx, e);
    p.stats = ctx->stats_dev;
    e = hd->shape == 2 ? wpp_launch_attention_small(d.head_dim, tq, &tk, &tv, &p, hd->num_ctas, cuda_stream)
                       : wpp_launch_attention(d.head_dim, tq, &tk, &tv, &p, hd->num_ctas, choose_late_rescale(ctx),
                                              cuda_stream);
    if (e != 0) return cuda_fail(ctx, e);
    const_cast<wpp_ctx*>(ctx)->launches += 1;
    if (hd->num_combine > 0) {
        wpp::CombineParams c;
        memset(&c, 0, sizeof(c));
        c.plan = plan_dev;
        c.ws_o = p.ws_o;
        c.ws_lse = p.ws_lse;
        c.out = p.out;
        c.lse = lse_or_null;
        c.o_token_stride = d.o_token_stride;
        c.o_head_stride = d.o_head_stride;
        c.num_q_heads = d.num_q_heads;
        c.head_dim = d.head_dim;
        c.tile_m = hd->tile_m;
        e = wpp_launch_combine(&c, hd->num_combine, cuda_stream);
        if (e != 0) return cuda_fail(ctx, e);
        const_cast<wpp_ctx*>(ctx)->launches += 1;
    }
    return WPP_OK;
}

// ---------------------------------------------------------------------------------------------------------------
// Entry point that allocates nothing: the tile counter and the split-KV partials live in the built-in scratch array
// whose address wpp_create looked up.
extern "C" int wpp_prefill_attention_varlen_static(const wpp_ctx* ctx, const wpp_batch_desc* desc, const void* q,
                                                   void* out, float* lse_or_null, const void* k_cache,
                                                   const void* v_cache, const int32_t* block_tables,
                                                   const int32_t* prefix_lens, const int32_t* chunk_lens,
                                                   const void* plan_host, const void* plan_dev, int32_t* status_dev,
                                                   void* cuda_stream) {
    if (!ctx || !ctx->static_scratch) return WPP_ERR_INVALID_ARG;
    wpp_batch_desc d;
    int rc = wpp_resolve_desc(desc, &d);
    if (rc != WPP_OK) return rc;
    const WppPlanHeader* hd = nullptr;
    if ((rc = wpp_check_plan(plan_host, &d, &hd)) != WPP_OK) return rc;
    if (hd->workspace_bytes > (uint64_t)WPP_STATIC_SCRATCH_BYTES) return WPP_ERR_WORKSPACE_TOO_SMALL;
    return wpp_prefill_attention_varlen(ctx, desc, q, out, lse_or_null, k_cache, v_cache, block_tables, prefix_lens,
                                        chunk_lens, plan_host, plan_dev, ctx->static_scratch,
                                        (size_t)WPP_STATIC_SCRATCH_BYTES, status_dev, cuda_stream);
}

// ---------------------------------------------------------------------------------------------------------------
// Recurrent-state layer.  Workspace of the chunk-parallel form: block offsets, then per (block, head) the cut mask,
// the decay products at sub-block ends and the ten operand arrays the preparation kernel leaves for the chain kernel.
struct KdaWorkspace {
    int64_t max_blocks, n_bh;
    size_t off_blk, off_mask, off_e, off_u0, off_op[6], off_sq[2], bytes;
};
static size_t up1k(size_t x) { return (x + 1023) / 1024 * 1024; }
static KdaWorkspace kda_workspace(const wpp_kda_desc* d) {
    KdaWorkspace w;
    w.max_blocks = d->total_tokens / 64 + 2 * (int64_t)d->num_requests;      // a chunk of C tokens touches <= C/64 + 2 blocks
    w.n_bh = w.max_blocks * d->num_heads;
    size_t off = 0;
    w.off_blk = off;  off += up1k(sizeof(int32_t) * ((size_t)d->num_requests + 1));
    w.off_mask = off; off += up1k(sizeof(uint64_t) * (size_t)w.n_bh);
    w.off_e = off;    off += up1k(sizeof(float) * (size_t)w.n_bh * 64 * 128);
    w.off_u0 = off;   off += up1k(sizeof(float) * (size_t)w.n_bh * 64 * 128);
    for (int i = 0; i < 6; ++i) { w.off_op[i] = off; off += up1k(2 * (size_t)w.n_bh * 64 * 128); }
    for (int i = 0; i < 2; ++i) { w.off_sq[i] = off; off += up1k(2 * (size_t)w.n_bh * 64 * 64); }
    w.bytes = off;
    return w;
}
static bool kda_desc_ok(const wpp_kda_desc* desc) {
    return desc && desc->num_requests >= 0 && desc->num_heads >= 1 && desc->num_slots >= 0 && desc->snap_interval >= 0 &&
           desc->max_snaps >= 0 && desc->total_tokens >= 0 && desc->layout >= 0 && desc->layout <= 3;
}

extern "C" size_t wpp_kda_workspace_bytes(const wpp_kda_desc* desc) {
    if (!kda_desc_ok(desc)) return 0;
    return kda_workspace(desc).bytes;
}

extern "C" int wpp_kda_chunk(const wpp_ctx* ctx, const wpp_kda_desc* desc, const void* q, const void* k, const void* v,
                             const float* alpha, const float* beta, const int64_t* row_offsets,
                             const int32_t* prefix_lens, float* state_pool, const int32_t* state_in,
                             const int32_t* state_out, const int32_t* snap_slots, void* out, void* workspace,
                             size_t workspace_bytes, int32_t* status_dev, void* cuda_stream) {
    if (!ctx || !kda_desc_ok(desc)) return WPP_ERR_INVALID_ARG;
    if (desc->d_k != 128 || desc->d_v != 128) return WPP_ERR_UNSUPPORTED;
    if (desc->num_requests > 65535) return WPP_ERR_UNSUPPORTED;      // one grid row per request
    if (desc->num_requests == 0) return WPP_OK;
    if (int rc = wpp_ctx_check_device(ctx)) return rc;
    if (!row_offsets || !state_in || !state_out) return WPP_ERR_INVALID_ARG;
    if (desc->num_slots > 0 && !state_pool) return WPP_ERR_INVALID_ARG;
    if (desc->total_tokens > 0 && (!q || !k || !v || !alpha || !beta || !out)) return WPP_ERR_INVALID_ARG;
    if (desc->snap_interval > 0 && !prefix_lens) return WPP_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(alpha) || !aligned16(out) || !aligned16(state_pool))
        return WPP_ERR_INVALID_ARG;
    // Which form: the chunk-parallel tensor-core form needs a workspace and pays off from about a block of tokens
    // per request; the token-by-token forms need none.
    const KdaWorkspace w = kda_workspace(desc);
    bool tensor_form = desc->layout == 3;
    if (desc->layout == 0)
        tensor_form = workspace && workspace_bytes >= w.bytes && desc->total_tokens >= 64 * (int64_t)desc->num_requests;
    if (tensor_form) {
        if (!workspace || workspace_bytes < w.bytes) return WPP_ERR_WORKSPACE_TOO_SMALL;
        if ((reinterpret_cast<uintptr_t>(workspace) & 255) != 0) return WPP_ERR_INVALID_ARG;
        if (w.n_bh * 64 > 0x7fffffffll || desc->total_tokens > 0x7fffffffll) return WPP_ERR_UNSUPPORTED;
        char* ws = static_cast<char*>(workspace);
        wpp::KdaTcParams p;
        memset(&p, 0, sizeof(p));
        p.q = static_cast<const __nv_bfloat16*>(q);
        p.k = static_cast<const __nv_bfloat16*>(k);
        p.v = static_cast<const __nv_bfloat16*>(v);
        p.alpha = alpha;
        p.beta = beta;
        p.row_offsets = row_offsets;
        p.prefix_lens = prefix_lens;
        p.state_pool = state_pool;
        p.state_in = state_in;
        p.state_out = state_out;
        p.snap_slots = desc->max_snaps > 0 ? snap_slots : nullptr;
        p.out = static_cast<__nv_bfloat16*>(out);
        p.status = status_dev;
        p.num_requests = desc->num_requests;
        p.num_heads = desc->num_heads;
        p.num_slots = desc->num_slots;
        p.snap_interval = desc->snap_interval;
        p.max_snaps = desc->max_snaps;
        p.blk_off = reinterpret_cast<int32_t*>(ws + w.off_blk);
        p.ws_mask = reinterpret_cast<unsigned long long*>(ws + w.off_mask);
        p.ws_e = reinterpret_cast<float*>(ws + w.off_e);
        p.ws_u0 = reinterpret_cast<float*>(ws + w.off_u0);
        __nv_bfloat16** ops[6] = {&p.ws_w0_h, &p.ws_w0_l, &p.ws_qt_h, &p.ws_qt_l, &p.ws_kb_h, &p.ws_kb_l};
        __nv_bfloat16** sqs[2] = {&p.ws_m_h, &p.ws_m_l};
        CUtensorMap maps[13];
        int rc;
        for (int i = 0; i < 6; ++i) {
            *ops[i] = reinterpret_cast<__nv_bfloat16*>(ws + w.off_op[i]);
            const uint64_t dims[2] = {128, (uint64_t)w.n_bh * 64};
            const uint64_t strides[1] = {256};
            const uint32_t box[2] = {64, 64};
            if ((rc = make_map(ctx, &maps[i], *ops[i], 2, dims, strides, box)) != WPP_OK) return rc;
        }
        for (int i = 0; i < 2; ++i) {
            *sqs[i] = reinterpret_cast<__nv_bfloat16*>(ws + w.off_sq[i]);
            const uint64_t dims[2] = {64, (uint64_t)w.n_bh * 64};
            const uint64_t strides[1] = {128};
            const uint32_t box[2] = {64, 64};
            if ((rc = make_map(ctx, &maps[6 + i], *sqs[i], 2, dims, strides, box)) != WPP_OK) return rc;
        }
        // fp32 arrays (U0, alpha) as bf16 maps with twice the elements per row: the copies move bytes
        {
            const uint64_t dims[2] = {256, (uint64_t)w.n_bh * 64};
            const uint64_t strides[1] = {512};
            const uint32_t box[2] = {64, 64};
            if ((rc = make_map(ctx, &maps[8], p.ws_u0, 2, dims, strides, box)) != WPP_OK) return rc;
        }
        if (desc->total_tokens > 0) {
            const uint64_t H = (uint64_t)desc->num_heads, T = (uint64_t)desc->total_tokens;
            const void* in[3] = {q, k, v};
            const uint32_t box[3] = {64, 1, 64};
            for (int i = 0; i < 3; ++i) {
                const uint64_t dims[3] = {128, H, T};
                const uint64_t strides[2] = {256, 256 * H};
                if ((rc = make_map(ctx, &maps[9 + i], in[i], 3, dims, strides, box)) != WPP_OK) return rc;
            }
            const uint64_t dims[3] = {256, H, T};
            const uint64_t strides[2] = {512, 512 * H};
            if ((rc = make_map(ctx, &maps[12], alpha, 3, dims, strides, box)) != WPP_OK) return rc;
        }
        int e = wpp_launch_kda_tc(&p, maps, desc->total_tokens > 0 ? (int)w.max_blocks : 0, ctx->sm_count, cuda_stream);
        if (e != 0) return cuda_fail(ctx, e);
        const_cast<wpp_ctx*>(ctx)->launches += 3;
        return WPP_OK;
    }
    wpp::KdaParams p;
    memset(&p, 0, sizeof(p));
    p.q = static_cast<const __nv_bfloat16*>(q);
    p.k = static_cast<const __nv_bfloat16*>(k);
    p.v = static_cast<const __nv_bfloat16*>(v);
    p.alpha = alpha;
    p.beta = beta;
    p.row_offsets = row_offsets;
    p.prefix_lens = prefix_lens;
    p.state_pool = state_pool;
    p.state_in = state_in;
    p.state_out = state_out;
    p.snap_slots = desc->max_snaps > 0 ? snap_slots : nullptr;
    p.out = static_cast<__nv_bfloat16*>(out);
    p.status = status_dev;
    p.num_requests = desc->num_requests;
    p.num_heads = desc->num_heads;
    p.num_slots = desc->num_slots;
    p.snap_interval = desc->snap_interval;
    p.max_snaps = desc->max_snaps;
    int e = wpp_launch_kda(&p, ctx->sm_count, desc->layout, cuda_stream);
    if (e != 0) return cuda_fail(ctx, e);
    const_cast<wpp_ctx*>(ctx)->launches += 1;
    return WPP_OK;
}
