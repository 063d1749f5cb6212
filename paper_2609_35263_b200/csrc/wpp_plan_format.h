// Internal layout of the plan buffer that wpp_plan_tiles writes on the host and the kernels read on the
// device.  Plain structs, 4-byte fields, byte offsets from the start of the buffer; nothing here is ABI.
#pragma once
#include <stdint.h>

#define WPP_PLAN_MAGIC 0x31505057u /* "WPP1" */
#define WPP_PLAN_VERSION 2u
#define WPP_TILE_N 128             /* keys per step */
#define WPP_HALF_M 128             /* query rows per tensor-core tile (one TMEM lane per row) */

struct WppPlanHeader {
    uint32_t magic, version;
    uint64_t desc_hash;             // hash of the batch description + lengths the plan was made for
    int32_t num_requests, num_ctas, num_units, num_combine;
    int32_t num_split_slots;        // partial-result slots of tile_m rows each in the workspace
    int32_t tile_m, tile_n, head_dim;
    int64_t total_new_tokens, key_steps, flops;
    uint64_t workspace_bytes, plan_bytes;
    uint32_t off_q_offsets;         // int32 [R+1]   exclusive scan of chunk_lens
    uint32_t off_cta_begin;         // int32 [num_ctas+1] range of units owned by each persistent CTA
    uint32_t off_units;             // WppUnit [num_units]
    uint32_t off_combine;           // WppCombine [num_combine]
    uint32_t pad[8];
};

// One work tile: rows [q_row0, q_row0+num_rows) of request `request`'s chunk, one query head,
// key steps [kv_begin, kv_end) of 128 keys each (absolute key index = step*128 + column).
struct WppUnit {
    int32_t request, q_row0, num_rows, q_head;
    int32_t kv_begin, kv_end;
    int32_t split_slot;             // -1: writes the final output; else partial slot in the workspace
    int32_t cost;                   // 128x128 steps (both halves), what the CTA assignment balanced
};

struct WppCombine {
    int32_t request, q_row0, num_rows, q_head;
    int32_t slot0, num_splits;      // partial slots [slot0, slot0+num_splits), merged in increasing order
    int32_t pad0, pad1;
};

// Workspace layout: fp32 O_part[num_split_slots][tile_m][head_dim] followed by fp32 lse_part[num_split_slots][tile_m]
// (log2 units of the scaled scores; -inf marks a row with no visible key in that part).
