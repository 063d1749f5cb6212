// Internal host-side declarations shared by the planner and the launch code.
#pragma once
#include <stdint.h>

#include "../../include/wpp.h"
#include "wpp_plan_format.h"

#define WPP_DEFAULT_TILE_M 256
#define WPP_MAX_TILE_M 256
/* a plan whose halves average at most this many 128-key steps runs on the small kernel shape */
#define WPP_SMALL_SHAPE_MAX_STEPS 1

#ifdef __cplusplus
extern "C" {
#endif
int wpp_resolve_desc(const wpp_batch_desc* in, wpp_batch_desc* out);
uint64_t wpp_desc_hash(const wpp_batch_desc* resolved);
int wpp_check_plan(const void* plan_host, const wpp_batch_desc* resolved, const struct WppPlanHeader** out);
int wpp_ctx_sm_count(const wpp_ctx* ctx);
int wpp_ctx_check_device(const wpp_ctx* ctx);   /* WPP_OK iff the context's device is the current one */
#ifdef __cplusplus
}
#endif
