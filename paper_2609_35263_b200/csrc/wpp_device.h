// Kernel parameter blocks and launch entry points shared by the launch code and the kernel files.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "../../include/wpp.h"

namespace wpp {

struct AttnParams {
    const void* plan;                // device copy of the plan
    const int32_t* block_tables;     // [R][max_blocks]
    const int32_t* prefix_lens;      // [R]
    const int32_t* chunk_lens;       // [R]
    __nv_bfloat16* out;              // [T][Hq][d]
    float* lse;                      // [T][Hq] or null
    float* ws_o;                     // split partials: [slots][2][128][d]
    float* ws_lse;                   // [slots][2][128], log2 units
    int32_t* status;                 // sticky device status word or null
    uint32_t* tile_counter;          // zeroed before the launch: index of the next tile nobody has taken yet
    unsigned long long* stats;       // or null: [0] += key steps of the softmax warps, [1] += those that rescaled O
    int64_t o_token_stride, o_head_stride;
    int32_t num_q_heads, group, page_size, max_blocks, num_pages;
    float scale_log2;                // sm_scale * log2(e)
};

struct AppendParams {
    const void* plan;
    const uint4* k_new;
    const uint4* v_new;
    uint4* k_cache;
    uint4* v_cache;
    const int32_t* block_tables;
    const int32_t* prefix_lens;
    const int32_t* chunk_lens;
    int32_t* status;
    int64_t kvnew_token_stride, kvnew_head_stride;       // in 16-byte units
    int64_t kv_page_stride, kv_head_stride, kv_token_stride;
    int32_t num_requests, num_kv_heads, vec_per_row, page_size, max_blocks, num_pages;
    int64_t total_new_tokens;
};

struct CombineParams {
    const void* plan;
    const float* ws_o;
    const float* ws_lse;
    __nv_bfloat16* out;
    float* lse;
    int64_t o_token_stride, o_head_stride;
    int32_t num_q_heads, head_dim, tile_m;
};

struct KdaParams {
    const __nv_bfloat16* q;
    const __nv_bfloat16* k;
    const __nv_bfloat16* v;
    const float* alpha;
    const float* beta;
    const int64_t* row_offsets;
    const int32_t* prefix_lens;
    float* state_pool;
    const int32_t* state_in;
    const int32_t* state_out;
    const int32_t* snap_slots;
    __nv_bfloat16* out;
    int32_t* status;
    int32_t num_requests, num_heads, num_slots, snap_interval, max_snaps;
};

// Chunk-parallel (tensor-core) form of the recurrent layer: the inputs of KdaParams plus the workspace arrays the
// preparation kernel fills for the chain kernel.  bh = (global block index) * num_heads + head.
struct KdaTcParams {
    const __nv_bfloat16* q;
    const __nv_bfloat16* k;
    const __nv_bfloat16* v;
    const float* alpha;
    const float* beta;
    const int64_t* row_offsets;
    const int32_t* prefix_lens;
    float* state_pool;
    const int32_t* state_in;
    const int32_t* state_out;
    const int32_t* snap_slots;
    __nv_bfloat16* out;
    int32_t* status;
    int32_t num_requests, num_heads, num_slots, snap_interval, max_snaps;
    int32_t* blk_off;               // [R+1] exclusive scan of the requests' block counts
    unsigned long long* ws_mask;    // [bh] bit t: token t of the block starts a sub-block
    float* ws_e;                    // [bh][64][128] decay product at a sub-block's last token (other rows unused)
    __nv_bfloat16 *ws_w0_h, *ws_w0_l, *ws_qt_h, *ws_qt_l, *ws_kb_h, *ws_kb_l;   // [bh][64][128] hi / lo bf16 terms
    __nv_bfloat16 *ws_m_h, *ws_m_l;                                             // [bh][64][64]
    float* ws_u0;                                                               // [bh][64][128]
};

}  // namespace wpp

extern "C" {
// maps: 0..5 the operand arrays W0, Qt, Kb (hi, lo each), 6..7 M (hi, lo), 8 U0, 9..12 q, k, v, alpha
int wpp_launch_kda_tc(const wpp::KdaTcParams* p, const CUtensorMap* maps, int max_blocks, int num_sms, void* stream);
int wpp_launch_attention(int head_dim, const CUtensorMap* tq, const CUtensorMap* tk, const CUtensorMap* tv,
                         const wpp::AttnParams* p, int num_ctas, int late_rescale, void* stream);
int wpp_launch_attention_small(int head_dim, const CUtensorMap* tq, const CUtensorMap* tk, const CUtensorMap* tv,
                               const wpp::AttnParams* p, int num_ctas, void* stream);
int wpp_launch_append(const wpp::AppendParams* p, int num_sms, void* stream);
int wpp_launch_combine(const wpp::CombineParams* p, int num_combine, void* stream);
int wpp_launch_kda(const wpp::KdaParams* p, int num_sms, int layout, void* stream);
int wpp_launch_selftest_wait(long long limit_cycles, int32_t* status, long long* waited_cycles, void* stream);
}
