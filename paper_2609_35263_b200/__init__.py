"""B200-native chunked-prefill attention over a paged, prefix-reused KV cache (C-ABI library + thin binding)."""
from .binding import (  # noqa: F401
    BatchDesc,
    Context,
    Plan,
    PlanInfo,
    PlanOpts,
    WppError,
    load_library,
    make_desc,
    wpp_kv_append,
    wpp_plan_tiles,
    wpp_prefill_attention_varlen,
    wpp_prefill_attention_varlen_static,
    wpp_selftest_bounded_wait,
    wpp_static_scratch_bytes,
    wpp_validate_batch,
)
