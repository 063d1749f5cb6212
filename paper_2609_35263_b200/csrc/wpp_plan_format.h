// Internal layout of the plan buffer that wpp_plan_tiles writes on the host and the kernels read on the
// device.  Plain structs, 4-byte fields, byte offsets from the start of the buffer; nothing here is ABI.
#pragma once
#include <stdint.h>

#define WPP_PLAN_MAGIC 0x31505057u /* "WPP1" */
#define WPP_PLAN_VERSION 7u
#define WPP_TILE_N 128             /* keys per step */
#define WPP_WS_HEADER_BYTES 256
#define WPP_HALF_M 128             /* query rows per tensor-core tile (one TMEM lane per row) */

struct WppPlanHeader {
    uint32_t magic, version;
    uint64_t desc_hash;             // hash of the batch description the plan was made for (the lengths are stored)
    int32_t num_requests, num_ctas, num_units, num_combine;
    int32_t num_split_slots;        // partial-result slots of 2 x 128 rows each in the workspace
    int32_t tile_m, tile_n, head_dim;
    int64_t total_new_tokens, key_steps, flops;
    uint64_t workspace_bytes, plan_bytes;
    uint32_t off_q_offsets;         // int32 [R+1]   exclusive scan of chunk_lens
    uint32_t off_prefix;            // int32 [R]     prefix_lens the plan was made for: the kernels compare them (and
                                    //               the row offsets) with the lengths they are launched with
    uint32_t off_units;             // WppUnit [num_units] in the order the persistent CTAs take them
    uint32_t off_combine;           // WppCombine [num_combine]
    int32_t shape;                  // 1: two-half CTAs, one per SM; 2: single-half CTAs, two per SM (work item = half a unit)
    int32_t nonempty_halves;
    uint32_t pad[6];
};

// One work tile = two 128-row "halves" that share one K/V stream (same request, same KV head).  Each half
// is rows [row0, row0+rows) of the request's chunk for `pack` consecutive query heads of that KV group
// (head, head+1, ...): head k of the half sits in tensor rows [k*128/pack, k*128/pack + rows).  pack is 1
// for row blocks longer than 64 rows; shorter blocks pack 2, 4 or 8 heads so that the 128-row MMA tile is not
// mostly padding.  rows == 0 marks an unused half.  Usually the halves are consecutive row blocks of one
// head; a short block gives the second half the next heads of the group instead.  The tile covers key steps
// [kv_begin, kv_end) of 128 keys (absolute key = step*128 + column); each half additionally stops at its own
// causal end.
struct WppUnit {
    int32_t request, kv_begin, kv_end;
    int32_t split_slot;             // -1: writes the final output; else partial slot in the workspace
    int32_t row0[2], rows[2], head[2];
    int32_t cost;                   // 128x128 steps over both halves
    int32_t pack;                   // query heads per half: 1, 2, 4 or 8
};

// One half tile whose key range was split: partial slots [slot0, slot0+num_splits) merged in increasing order.
struct WppCombine {
    int32_t request, row0, rows, head;
    int32_t slot0, num_splits;
    int32_t half;                   // which half of the slot the rows live in
    int32_t lane0;                  // first tensor row of this head inside the half (packed heads)
};

// Workspace layout: WPP_WS_HEADER_BYTES of header (byte 0: a uint32 counter, the next tile of the order nobody has
// taken yet; bytes 8 and 16: two uint64 counters of the SM-wide kernel, key steps and steps that rescaled an
// accumulator; byte 24: a uint32 count of CTAs that have finished - the attention call zeroes the header on the
// stream before the launch), then fp32
// O_part[num_split_slots][2][128][head_dim] followed by fp32 lse_part[num_split_slots][2][128] (log2 units of the
// scaled scores; -inf marks a row with no visible key in that part).
