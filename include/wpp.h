/*
 * wpp.h — C ABI of the chunked-prefill attention path of one pipeline stage.
 *
 * One call processes one *wave*: a ragged batch of request chunks (paper,
 * Section 4 "Waves and lanes").  For request i the caller states
 *   prefix_lens[i] = P_i  tokens of the request already in the paged KV cache
 *                         (the reused cached prefix plus earlier chunks; this is the
 *                         "starting token" of the chunk span, Section 4.6),
 *   chunk_lens[i]  = C_i  new tokens in this wave (the span's "length"),
 *   block_tables[i][j]    physical page holding tokens [j*B, (j+1)*B) of request i
 *                         (Section 3.2: ceil(n/B) logical blocks, physically
 *                         non-contiguous, shareable between requests).
 * T = sum_i C_i; the chunks' rows are concatenated in request order in q, k_new,
 * v_new and out.  Query head h reads KV head h / (num_q_heads / num_kv_heads)
 * (grouped-query attention, Section 3.1).
 *
 * General rules
 *   - Every function returns a wpp_status (0 = WPP_OK).  Nothing throws, nothing
 *     synchronises the device, and nothing allocates device memory unless said so.
 *   - "host" / "device" on each pointer says where the memory lives.  The caller owns
 *     every buffer; device buffers are borrowed until the work queued on
 *     `cuda_stream` (a cudaStream_t passed as void*) has completed.
 *   - bf16 tensors are passed as void*; inner (head_dim) elements are contiguous and
 *     every row start and stride must be a multiple of 16 bytes.
 *   - Problems the host can see are reported before anything is launched.  Problems
 *     only the device can see (a page id outside [0, num_pages), a bounded wait that
 *     ran out, lengths on the device that differ from the plan's) set *status_dev (first error wins, never cleared by the library), the
 *     affected work is skipped, and nothing traps; read it after your own sync.
 *   - A request appears at most once per wave; successive chunks of a request go in
 *     successive calls on the same stream (Section 4.6: order is preserved on each
 *     stage's execution stream).  wpp_kv_append must precede
 *     wpp_prefill_attention_varlen for the same wave on that stream: attention reads
 *     the chunk's own K/V from the pages.
 */
#ifndef WPP_H_
#define WPP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    WPP_OK = 0,
    WPP_ERR_INVALID_ARG = 1,        /* null pointer, negative size, misaligned pointer or stride */
    WPP_ERR_UNSUPPORTED = 2,        /* dtype, head_dim, page_size or head ratio outside the supported set */
    WPP_ERR_BOUNDS = 3,             /* ceil((P_i + C_i) / B) > max_blocks_per_req, or page id out of range */
    WPP_ERR_POSITION_MISMATCH = 4,  /* span start != tokens actually cached (Section 4.6: execution fails) */
    WPP_ERR_WORKSPACE_TOO_SMALL = 5,
    WPP_ERR_PLAN_MISMATCH = 6,      /* plan buffer corrupt, too small, or built for another batch description; device
                                       side: a request's prefix_lens / chunk_lens are not those the plan was made for */
    WPP_ERR_CUDA = 7,               /* CUDA runtime/driver error; see wpp_last_cuda_error */
    WPP_ERR_TIMEOUT = 8,            /* device side: a bounded barrier wait expired; the tile was abandoned */
    WPP_ERR_ALIASED_APPEND = 9      /* wpp_validate_batch: two writers, or a writer and a reader, share a slot */
} wpp_status;

enum { WPP_BF16 = 1 };

/* Opaque per-device context: SM count, shared-memory limit, driver entry points.  Owns host memory only. */
typedef struct wpp_ctx wpp_ctx;

/* Create a context for CUDA device `cuda_device`.  It makes no cudaMalloc; it does look up the device address of
 * the library's built-in scratch array (see wpp_prefill_attention_varlen_static), which is what makes the CUDA
 * runtime place that array (wpp_static_scratch_bytes() bytes) on the device: create the context at start-up, before
 * the KV pool is sized from the free memory.  WPP_ERR_CUDA if the device or driver is unusable (there is no CPU
 * fallback).  *out is host memory owned by the library until wpp_destroy.  Every launching entry point must be
 * called with the context's device current (WPP_ERR_INVALID_ARG otherwise).  The context caches the tensor maps
 * it encodes, keyed by (pointer, extents, strides); it may be used from several host threads.  It also owns 64
 * bytes of pinned host memory mapped for the device, to which the attention kernels add two counters (see
 * wpp_set_rescale_mode): everything enqueued through the context must have completed before wpp_destroy. */
int wpp_create(wpp_ctx** out, int cuda_device);
int wpp_destroy(wpp_ctx* ctx);
const char* wpp_status_string(int status);
/* Last cudaError_t / CUresult seen by this context (0 if none). */
int wpp_last_cuda_error(const wpp_ctx* ctx);

/* Description of one wave.  Strides are in ELEMENTS (bf16), inner dim contiguous.
 * Pools: element (page, kv_head, slot, e) of K lives at
 *   k_cache + page*kv_page_stride + kv_head*kv_head_stride + slot*kv_token_stride + e,
 * V likewise in v_cache with the same strides.  A stride of 0 selects the dense default
 * of the layouts [num_pages][Hkv][B][d] (pools) and [T][H][d] (q, k_new/v_new, out). */
typedef struct {
    int32_t num_requests;        /* R >= 0 */
    int32_t num_q_heads;         /* Hq, a multiple of num_kv_heads */
    int32_t num_kv_heads;        /* Hkv */
    int32_t head_dim;            /* d in {64, 128} */
    int32_t page_size;           /* B in {16, 32, 64, 128} tokens per page */
    int32_t max_blocks_per_req;  /* row stride of block_tables, in elements */
    int32_t num_pages;           /* pool size, for bounds checks */
    int32_t dtype;               /* WPP_BF16 */
    float sm_scale;              /* 0 selects 1/sqrt(head_dim) */
    int32_t reserved0;
    int64_t kv_page_stride, kv_head_stride, kv_token_stride;
    int64_t q_token_stride, q_head_stride;
    int64_t kvnew_token_stride, kvnew_head_stride;
    int64_t o_token_stride, o_head_stride;
} wpp_batch_desc;

/* Planner knobs; a zero field selects the library default. */
typedef struct {
    int32_t tile_m;           /* query rows per work tile: 128 or 256 (default 256: two 128-row halves) */
    int32_t tile_n;           /* keys per inner step: 128 */
    int32_t force_kv_splits;  /* >= 2: split every tile's key range into this many parts (when it has that many
                                 key steps); 1: never split; 0: library decides (all tiles when there are fewer of
                                 them than CTAs; the tiles of a partly filled last round when the tiles are long and
                                 the rounds few; wpp_plan_info.workspace_bytes says what the partials need) */
    int32_t max_ctas;         /* persistent CTAs to launch (default: SM count of the context, 148 without one) */
    int32_t order;            /* order in which the persistent CTAs take the tiles at run time.  0: stream order -
                                 tiles that read the same (request, KV head) pages are neighbours and so run at the
                                 same time: the pages are fetched from DRAM once and shared through L2; 1: longest
                                 tile first */
    int32_t shape;            /* which attention kernel runs the plan.  1: one CTA per SM working on both 128-row halves
                                 of a tile against 128-key steps (long tiles: the two halves and the tensor pipe overlap
                                 inside the CTA); 2: two small CTAs per SM, each working on one half against 64-key
                                 steps (short tiles: one CTA's tile start and end hide under the other's steps);
                                 0: the library decides from the mean number of key steps per half */
} wpp_plan_opts;

typedef struct {
    int64_t num_tiles;          /* work tiles in the plan (split parts count separately) */
    int64_t num_split_tiles;    /* of which write partial results to the workspace */
    int64_t num_combine_tiles;  /* tiles the combine pass merges (0: no combine pass) */
    int64_t num_ctas;           /* persistent CTAs the attention kernel will be launched with */
    int64_t total_new_tokens;   /* T */
    int64_t key_steps;          /* sum over tiles of 128-row x 128-key steps (work incl. tile quantisation) */
    int64_t flops;              /* algorithmic: 4 * d * Hq * sum_i (C_i P_i + C_i (C_i + 1) / 2) */
    int64_t shape;              /* attention kernel the plan is for: 1 or 2, see wpp_plan_opts.shape */
    size_t workspace_bytes;     /* device scratch wpp_prefill_attention_varlen needs for this plan (never 0) */
    size_t plan_bytes;          /* bytes of plan_host actually used; copy that many to the device */
} wpp_plan_info;

/* Upper bound on the plan size for a wave of this description with `total_new_tokens` rows under these opts
 * (0 if the description or opts are invalid). */
size_t wpp_plan_bytes(const wpp_ctx* ctx_or_null, const wpp_batch_desc* desc, int64_t total_new_tokens,
                      const wpp_plan_opts* opts_or_null);

/* Host-side work split (integer arithmetic only; no CUDA call).  Cuts the wave into work tiles
 * (request, query-row range, query head, key-step range), decides which tiles are split along the keys,
 * orders them (opts->order) and sizes the workspace; the persistent CTAs of the attention kernel take tiles in that
 * order as they become free.  Equal-sized chunks cost different amounts because they attend to different prefix
 * lengths (Section 6), which is why tiles are not preassigned to CTAs.
 *   prefix_lens_host, chunk_lens_host : host int32 [R].
 *   cached_lens_host_or_null          : host int32 [R]; tokens each request really has in the cache after
 *                                       materialisation.  If given and != prefix_lens, returns
 *                                       WPP_ERR_POSITION_MISMATCH (Section 4.6).
 *   plan_host / plan_host_bytes       : caller-owned host buffer (pinned if it is to be copied asynchronously);
 *                                       the caller copies info->plan_bytes bytes of it to the device.
 * Deterministic: equal inputs give byte-identical plans.  ctx may be NULL (plans for 148 SMs). */
int wpp_plan_tiles(const wpp_ctx* ctx_or_null, const wpp_batch_desc* desc,
                   const int32_t* prefix_lens_host, const int32_t* chunk_lens_host,
                   const int32_t* cached_lens_host_or_null, const wpp_plan_opts* opts_or_null,
                   void* plan_host, size_t plan_host_bytes, wpp_plan_info* info);

/* Optional host-side check of a wave (host copies of everything): page ids in range, table long enough, no slot
 * written by two requests, no written slot inside another request's readable range.  block_tables_host is
 * int32 [R][max_blocks_per_req]. */
int wpp_validate_batch(const wpp_batch_desc* desc, const int32_t* block_tables_host,
                       const int32_t* prefix_lens_host, const int32_t* chunk_lens_host);

/* KV append (the chunk's K/V go into the blocks reserved for them, Section 4.1 steps 3-5): for every new token t of
 * request i,
 * pos = P_i + t, page = block_tables[i][pos / B], slot = pos % B; copies k_new[q_off_i + t][h][0..d) and
 * v_new[...] bit for bit to k_cache / v_cache [page][h][slot][0..d).  No other pool byte is written.
 *   k_new, v_new : device, bf16 [T][Hkv][d] (read).     k_cache, v_cache : device pools (written).
 *   block_tables : device int32 [R][max_blocks_per_req]; prefix_lens, chunk_lens : device int32 [R].
 *   plan_dev     : device copy of the plan made for this wave (provides row offsets and T).
 *   plan_host    : the host plan it was copied from (read during the call only, for launch sizing).
 *   status_dev   : device int32, sticky first-error word (may be NULL).
 * One kernel on cuda_stream, 16-byte vector copies.  A page id outside [0, num_pages) sets
 * *status_dev = WPP_ERR_BOUNDS and that token is skipped.  A request whose prefix_lens[i] or chunk_lens[i] on the
 * device differ from the lengths the plan was made for sets WPP_ERR_PLAN_MISMATCH and none of its tokens is written
 * (Section 4.6: a position mismatch fails execution rather than writing against the wrong cache state). */
int wpp_kv_append(const wpp_ctx* ctx, const wpp_batch_desc* desc, const void* k_new, const void* v_new,
                  void* k_cache, void* v_cache, const int32_t* block_tables, const int32_t* prefix_lens,
                  const int32_t* chunk_lens, const void* plan_host, const void* plan_dev, int32_t* status_dev,
                  void* cuda_stream);

/* Chunked-prefill attention (Section 4.1 step 5; Section 3.1: token n attends to all n previous positions):
 * for chunk row t of request i and query head h, with g = h / (Hq/Hkv) and n = P_i + t + 1,
 *   s_j = sm_scale * <q[q_off_i + t][h], K_j[g]>,  j < n,   K_j = k_cache[block_tables[i][j / B]][g][j % B],
 *   out[q_off_i + t][h] = sum_j softmax(s)_j V_j[g]   (bf16, round to nearest even),
 *   lse[q_off_i + t][h] = log sum_j exp(s_j)          (fp32, natural log; optional).
 * bf16 inputs, fp32 scores/accumulation on tensor cores, probabilities rounded to bf16 before the PV product.
 * Slots >= P_i + C_i and pages no table references never influence the result, whatever bits they hold.
 *   q, out        : device bf16 [T][Hq][d];  lse_or_null : device fp32 [T][Hq].
 *   k_cache, v_cache, block_tables, prefix_lens, chunk_lens : device, read only.
 *   plan_host / plan_dev : as for wpp_kv_append.
 *   workspace     : device scratch of >= info.workspace_bytes bytes, 256-byte aligned, required: holds the
 *                   counter the persistent CTAs take their tiles from (zeroed by this call on the stream) and
 *                   the split-KV partial results; contents are undefined afterwards.  Two calls that may run
 *                   at the same time need a workspace each.
 * A request whose prefix_lens[i] or chunk_lens[i] on the device differ from the plan's sets *status_dev =
 * WPP_ERR_PLAN_MISMATCH; its tiles are skipped (its output rows are not computed; rows of split tiles read as zero).
 * Enqueues a 256-byte memset and one persistent kernel (the shape the plan names), plus one combine kernel iff the
 * plan has split tiles.
 * Results are bit-reproducible for a given plan, whichever CTA takes which tile (no atomics on outputs; partials
 * are merged in a fixed order). */
int wpp_prefill_attention_varlen(const wpp_ctx* ctx, const wpp_batch_desc* desc, const void* q, void* out,
                                 float* lse_or_null, const void* k_cache, const void* v_cache,
                                 const int32_t* block_tables, const int32_t* prefix_lens,
                                 const int32_t* chunk_lens, const void* plan_host, const void* plan_dev,
                                 void* workspace, size_t workspace_bytes, int32_t* status_dev,
                                 void* cuda_stream);

/* Same computation as wpp_prefill_attention_varlen for callers that have no device memory to give and cannot
 * get any.  (The paper has no counterpart; this is a convenience of this library.)  A prefill stage usually runs
 * inside a serving process whose cache manager has already claimed every free byte of HBM for KV pages, and on an
 * execution stream that must not stall: there a cudaMalloc at call time either fails or synchronises the whole
 * device.  This entry point therefore allocates nothing, neither directly nor through any library: the tile
 * counter and the split-KV partial results live in a fixed scratch array that is part of the library image
 * (wpp_static_scratch_bytes() bytes, 16 MiB; every GPU that loads the library holds it until the process exits).
 *   - Arguments as for wpp_prefill_attention_varlen, without workspace / workspace_bytes.
 *   - A plan that needs more scratch than the array holds is rejected with WPP_ERR_WORKSPACE_TOO_SMALL before
 *     anything is launched (plan with fewer key splits, or use the caller-workspace entry point).
 *   - The array's device address is looked up by wpp_create (once per device, with that device current), so that
 *     the memory is placed at start-up and no call of this entry point has anything left to set up; create the
 *     context before any stream capture begins.
 *     (Like any CUDA kernel, the attention kernels are loaded onto the device by their first launch; this entry
 *     point adds nothing to that.)
 *   - All calls on a device share the one array and it keeps whatever the last call left in it.  The call zeroes
 *     the tile counter itself (a memset node on the stream) and every partial row is written before the combine
 *     pass reads it, but two calls whose kernels overlap on the GPU, e.g. on different streams, race on it:
 *     serialise them. */
int wpp_prefill_attention_varlen_static(const wpp_ctx* ctx, const wpp_batch_desc* desc, const void* q, void* out,
                                        float* lse_or_null, const void* k_cache, const void* v_cache,
                                        const int32_t* block_tables, const int32_t* prefix_lens,
                                        const int32_t* chunk_lens, const void* plan_host, const void* plan_dev,
                                        int32_t* status_dev, void* cuda_stream);
/* Size in bytes of the built-in scratch array used by wpp_prefill_attention_varlen_static. */
size_t wpp_static_scratch_bytes(void);

/* Self-test of the bounded waits the kernels rely on (no counterpart in the paper): launches one warp that waits,
 * for at most limit_cycles SM clocks (1 .. 2^30), on a barrier nothing ever arrives on.  The wait gives up, the
 * kernel ends normally, *status_dev becomes WPP_ERR_TIMEOUT (if it was 0) and *waited_cycles_dev (device int64,
 * may be NULL) receives how long the warp waited.  Nothing hangs or traps; the context stays usable. */
int wpp_selftest_bounded_wait(const wpp_ctx* ctx, int64_t limit_cycles, int32_t* status_dev,
                              int64_t* waited_cycles_dev, void* cuda_stream);

/* Number of kernels the library has launched through this context so far (for launch accounting). */
int64_t wpp_launch_count(const wpp_ctx* ctx);

/* The attention kernel keeps a reference per query row for its exponentials and rescales the row's accumulator when
 * the reference has to move.  It exists in two orders of work: rescale before the step's exponentials (best when
 * references move now and then: every workload whose scores do not keep growing along the sequence) or after them
 * (best when most steps move a reference).  Both are within the tolerance; they differ in rounding order.
 *   wpp_set_rescale_mode : 0 = always before (default: outputs are bit-reproducible from call to call),
 *                          1 = always after,
 *                          2 = chosen per call from what the kernels of earlier launches on this context counted -
 *                              their key steps and the steps that rescaled, added up in two words of pinned host
 *                              memory that wpp_create maps for the device and that the call reads without
 *                              synchronising: at least 30 % of the steps rescaling: after; under 15 %: before; in
 *                              between: as it was.  Outputs may then differ in the last bit from call to call.
 *   wpp_rescale_stats    : the counters so far (either pointer may be null) and the order the next call would use. */
int wpp_set_rescale_mode(wpp_ctx* ctx, int mode);
int wpp_rescale_stats(const wpp_ctx* ctx, uint64_t* key_steps, uint64_t* rescaling_steps, int* late);

/* ---------------------------------------------------------------------------------------------------------
 * Wave-budget planner (Section 4.5, "Pipeline Scheduling": Maximum Pipeline Utilization).  Host only, integer
 * arithmetic only, no CUDA call; it produces the chunk_lens the calls above consume: the step directly upstream of
 * the attention path.  With P pipeline stages the executor keeps a ring of R = 2P waves and the planner aims at
 * S = R + (F - 1) P waves of work; it picks the wave budget from the ladder b_0 = M, b_{j+1} = max(b_min,
 * alignDown_B(b_j / 2)) (Eq. design-budget) by the estimate n(b) = max(W / b, N_{>b/2}) of the waves a budget b
 * yields, where the pieces are the unscheduled suffixes of admitted requests and their most recent chunks still in
 * the ring, W their token sum and N_{>b/2} the number of pieces larger than half a wave.
 * Rules, in the paper's order: the largest budget with n(b) >= S, b_min if none; once a budget supplies R waves the
 * next smaller one is only taken if the pieces it would newly split (size in (b_{j+1}, b_j]) are at most 12.5 % of
 * W; a burst asking for a budget two or more ladder steps larger takes effect at once, a one-step increase after
 * R/2 consecutive decisions asked for it, a decrease (one step) after R consecutive decisions asked for it and
 * only while the budget in force misses the target by a whole wave (n(b_cur) <= S - 1: the paper names a
 * hysteresis check without defining it; this is the reading taken).  Packing is first come, first served: a
 * request that fits takes its whole suffix; one that does not gets the leftover space as a fragment unless the
 * fragment is smaller than max(b_min, b / 2), in which case packing stops (nobody overtakes it). */
typedef struct {
    int32_t num_stages;   /* P >= 1 */
    int32_t fill_factor;  /* F >= 1 (the paper's matched experiments use 2) */
    int32_t block_size;   /* B >= 1 */
    int32_t max_lanes;    /* requests a wave may carry (maximum batch size) >= 1 */
    int64_t max_budget;   /* M: multiple of B, <= 2^31 - 1 */
    int64_t min_budget;   /* b_min: multiple of B, B <= b_min <= M */
} wpp_wave_config;

/* Planner state carried from one decision to the next; start from all zeros (budget M in force). */
typedef struct {
    int32_t cur;          /* ladder index of the budget in force (0 = M) */
    int32_t direction;    /* pending change: -1 towards larger budgets, +1 towards smaller, 0 none */
    int32_t count;        /* consecutive decisions that asked for the pending change */
    int32_t reserved;
} wpp_wave_state;

typedef struct {
    int64_t budget;       /* budget in force for this wave */
    int64_t work;         /* W */
    int64_t wave_tokens;  /* sum of chunk_lens */
    int32_t target_index; /* ladder index the selection rule asked for, before hysteresis */
    int32_t budget_index; /* ladder index in force */
    int32_t lanes;        /* requests in the wave */
    int32_t defer;        /* 1: a lone request below half capacity; it may wait one iteration for company */
} wpp_wave_info;

#define WPP_WAVE_RING_BUSY 1         /* flags of wpp_plan_waves */
#define WPP_WAVE_ADMISSION_PENDING 2
#define WPP_WAVE_ALREADY_DEFERRED 4

/* The ladder of budgets for cfg: writes min(*count, capacity) entries to ladder_out (may be NULL with capacity 0)
 * and the ladder's length to *count.  WPP_ERR_INVALID_ARG for an invalid configuration. */
int wpp_wave_ladder(const wpp_wave_config* cfg, int64_t* ladder_out, int32_t capacity, int32_t* count);

/* One planning decision of rank 0.
 *   remaining_host : host int64 [num_requests], unscheduled suffix tokens per admitted request in arrival order
 *                    (0 = finished); inflight_host : host int64 [num_inflight], the most recently committed chunks
 *                    still in the ring (either may be NULL when its count is 0).
 *   state          : in/out, see wpp_wave_state.
 *   flags          : WPP_WAVE_* bits; `defer` is reported only when the ring is busy, admission has further
 *                    requests pending and this wave has not been deferred before.
 *   chunk_lens_host: out, host int32 [num_requests]: tokens of each request in this wave (0 = not in it); the
 *                    caller advances its positions by the spans it actually accepts.
 * Returns WPP_ERR_INVALID_ARG for null pointers, negative lengths or an invalid configuration or state. */
int wpp_plan_waves(const wpp_wave_config* cfg, wpp_wave_state* state, const int64_t* remaining_host,
                   int32_t num_requests, const int64_t* inflight_host, int32_t num_inflight, int32_t flags,
                   int32_t* chunk_lens_host, wpp_wave_info* info);

/* ---------------------------------------------------------------------------------------------------------
 * Prefix hints (Section 4.3): chained hashes of full token blocks and a counted index probed by galloping and
 * bisecting.  This is the step that produces prefix_lens: the number of leading blocks of a request whose keys
 * are in the index, times the block size, is the reuse candidate.
 *
 * Eq. design-hash: H_{-1} = 0, H_i = hash(B_i, extraKeys_i, salt, H_{i-1}) over the FULL blocks of a request.  The
 * paper does not name the hash; this library uses 64-bit arithmetic with mix64 = the splitmix64 finaliser:
 *   term_k = mix64(((token_k mod 2^32) << 32 | k) xor 0xD6E8FEB86659FD93)   (k = position inside the block)
 *   digest_i = sum_k term_k (mod 2^64)
 *   H_i = mix64(H_{i-1} xor mix64(digest_i + extraKeys_i) xor (salt * 0x9E3779B97F4A7C15)). */

/* Chained block hashes of a batch of requests, on the GPU (two small kernels on `cuda_stream`).
 *   tokens        : device int32 [token_offsets[R]], the requests' token ids back to back.
 *   token_offsets : device int64 [R+1], start of each request in `tokens`.
 *   block_offsets : device int64 [R+1], exclusive scan of floor(n_i / block_size): where each request's hashes go.
 *   extra_keys_or_null : device uint64 [total_blocks] or NULL (all zero).
 *   hashes_out    : device uint64 [total_blocks]; request i's H_0.. are at hashes_out[block_offsets[i]..].
 * Partial last blocks are not hashed.  Returns WPP_ERR_INVALID_ARG for null pointers or sizes < 0, WPP_ERR_CUDA for
 * a launch failure. */
int wpp_hash_blocks(const wpp_ctx* ctx, const int32_t* tokens, const int64_t* token_offsets,
                    const int64_t* block_offsets, int32_t num_requests, int32_t block_size, uint64_t salt,
                    const uint64_t* extra_keys_or_null, uint64_t* hashes_out, int64_t total_blocks,
                    void* cuda_stream);

/* The same chain for one request on the host (host pointers; hashes_out holds n_tokens / block_size entries). */
int wpp_hash_blocks_host(const int32_t* tokens, int64_t n_tokens, int32_t block_size, uint64_t salt,
                         const uint64_t* extra_keys_or_null, uint64_t* hashes_out);

/* Counted index keyed by (cache window, H_i): a key's counter goes up when a block joins the cache tree and down
 * when it is detached; the entry disappears at zero.  Sharded by hash, one mutex per shard; safe to call from
 * several host threads. */
typedef struct wpp_hint_index wpp_hint_index;
int wpp_hint_index_create(wpp_hint_index** out);
int wpp_hint_index_destroy(wpp_hint_index* idx);
int wpp_hint_index_add(wpp_hint_index* idx, int32_t window, const uint64_t* hashes_host, int64_t n);
int wpp_hint_index_remove(wpp_hint_index* idx, int32_t window, const uint64_t* hashes_host, int64_t n);
int64_t wpp_hint_index_size(const wpp_hint_index* idx);     /* number of keys; -1 for NULL */

/* Longest cached prefix of a request, in blocks: probes depths 1, 2, 4, ... until the first miss, then bisects
 * between the last match and that miss (about log2 N probes instead of N; exact when presence is monotone in
 * depth, which chained keys added prefix by prefix guarantee).  The index may change while the probe runs; the
 * result is a hint that the caller's authoritative walk confirms.
 *   hashes_host : host uint64 [n_blocks], H_0 .. of the request;  *matched_blocks and *probes_or_null are outputs. */
int wpp_hint_probe(const wpp_hint_index* idx, int32_t window, const uint64_t* hashes_host, int64_t n_blocks,
                   int64_t* matched_blocks, int32_t* probes_or_null);

/* Endpoint of a recurrent-state cache (Section 4.3): snapshots exist only at sparse boundaries, so presence is not
 * monotone in depth and the probe walks backward from the attention-limited endpoint `limit_blocks` until it meets a
 * depth whose key is in the index under `window` (the recurrent cache's window id); *matched_blocks is that depth,
 * 0 if there is none.  The reuse candidate of a request is the minimum of its caches' endpoints (and, across
 * ranks, the all-rank minimum); lowering it may call for another backward scan from the lower endpoint. */
int wpp_hint_probe_recurrent(const wpp_hint_index* idx, int32_t window, const uint64_t* hashes_host,
                             int64_t limit_blocks, int64_t* matched_blocks, int32_t* probes_or_null);

/* ---------------------------------------------------------------------------------------------------------
 * Recurrent-state layer of a chunk (Section 3.1, the simplified KDA update; Section 3.2, snapshots): the other
 * cache type of a hybrid model's stage.  Per request and head, token by token over the chunk,
 *     S_t = (I - beta_t k_t k_t^T) Diag(alpha_t) S_{t-1} + beta_t k_t v_t^T,      o_t = S_t^T q_t,
 * with S (d_k x d_v, fp32) resumed from the state after exactly the reused prefix - a recurrent layer cannot
 * resume from anything else - and written back at the chunk end and, optionally, at sparse periodic boundaries.
 * Heads are independent.  No normalisation or scaling of q or k is applied here (the update has none).
 * Two forms compute it.  The chunk-parallel form (layout 3) works on blocks of 64 sequence positions: per block the
 * products Kt Kh^T, Qt Kh^T (Kt, Kh, Qt: keys and queries scaled by the decay products inside the block), Kt S_0,
 * T (V - Kt S_0), Qt S_0, tril(Qt Kh^T) U and Kb^T U run on the tensor cores with the fp32 state in tensor memory;
 * every operand is split into two bf16 terms (16 significant bits, three MMAs per product), accumulation is fp32.
 * It needs a workspace (wpp_kda_workspace_bytes).  The token-by-token forms (layouts 1, 2) use fp32 fused
 * multiply-adds on CUDA cores in token order and need no workspace.  Outputs are rounded to bf16, states stay fp32. */
typedef struct {
    int32_t num_requests;   /* R >= 0 */
    int32_t num_heads;      /* H >= 1: state heads */
    int32_t d_k;            /* 128 */
    int32_t d_v;            /* 128 */
    int32_t num_slots;      /* slots of state_pool, each H * d_k * d_v floats */
    int32_t snap_interval;  /* > 0: snapshot whenever the tokens folded into S reach a multiple of it; 0: none */
    int32_t max_snaps;      /* row length of snap_slots (0 when snap_interval is 0) */
    int32_t layout;         /* 0: the library chooses (the chunk-parallel form when a large enough workspace is given
                             * and the wave has at least 64 tokens per request on average, else 1 or 2);
                             * 1: token by token, one CTA per (request, head); 2: token by token, four CTAs per
                             * (request, head) of 32 columns each; 3: chunk-parallel on the tensor cores */
    int64_t total_tokens;   /* T = row_offsets[R] */
} wpp_kda_desc;

/* One launch on `cuda_stream` for the whole ragged batch; request i owns rows [row_offsets[i], row_offsets[i+1]).
 *   q, k        : device bf16 [T, H, d_k], dense;  v : device bf16 [T, H, d_v];  all 16-byte aligned.
 *   alpha       : device fp32 [T, H, d_k] (the per-channel decay Diag(alpha_t));  beta : device fp32 [T, H].
 *   row_offsets : device int64 [R+1], exclusive scan of the chunk lengths.
 *   prefix_lens : device int32 [R], tokens already folded into the resumed state (needed for periodic snapshots:
 *                 boundaries are multiples of snap_interval in sequence positions); may be NULL if snap_interval = 0.
 *   state_pool  : device fp32 [num_slots, H, d_k, d_v], 16-byte aligned; the library reads and writes slots in
 *                 place and owns none of it.
 *   state_in    : device int32 [R]: slot holding S after the reused prefix, or -1 for the zero state.
 *   state_out   : device int32 [R]: slot that receives the state after the chunk, or -1.  May equal state_in[i];
 *                 no slot may be written for one request and read or written for another in the same call.
 *   snap_slots  : device int32 [R, max_snaps] or NULL: slot for the n-th boundary inside the chunk, -1 = skip;
 *                 boundaries past max_snaps are skipped.
 *   out         : device bf16 [T, H, d_v].
 *   workspace   : device scratch for the chunk-parallel form, 256-byte aligned, wpp_kda_workspace_bytes(desc)
 *                 bytes (about 160 KB per 64 tokens and head); may be NULL (0 bytes) for the other forms.  Contents
 *                 are undefined afterwards; calls that may overlap on the GPU need a workspace each.
 *   status_dev  : device int32 or NULL; a slot id outside [-1, num_slots) sets it to WPP_ERR_BOUNDS (if it was 0)
 *                 and that request's state is neither read (zero state used) nor written there.
 * A request with an empty chunk copies state_in to state_out.  Returns WPP_ERR_INVALID_ARG for null or misaligned
 * pointers or negative sizes, WPP_ERR_UNSUPPORTED for d_k, d_v other than 128, WPP_ERR_WORKSPACE_TOO_SMALL when
 * layout 3 is asked for without enough workspace, WPP_ERR_CUDA for a launch failure.  The chunk-parallel form
 * enqueues three kernels (block offsets, per-block preparation, the chain over the blocks), the others one. */
int wpp_kda_chunk(const wpp_ctx* ctx, const wpp_kda_desc* desc, const void* q, const void* k, const void* v,
                  const float* alpha, const float* beta, const int64_t* row_offsets, const int32_t* prefix_lens,
                  float* state_pool, const int32_t* state_in, const int32_t* state_out, const int32_t* snap_slots,
                  void* out, void* workspace, size_t workspace_bytes, int32_t* status_dev, void* cuda_stream);

/* Bytes of workspace the chunk-parallel form of wpp_kda_chunk needs for a wave of this description (depends on
 * num_requests, num_heads and total_tokens only); 0 for an invalid description. */
size_t wpp_kda_workspace_bytes(const wpp_kda_desc* desc);

#ifdef __cplusplus
}
#endif
#endif /* WPP_H_ */
