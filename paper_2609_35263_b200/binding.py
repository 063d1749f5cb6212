"""ctypes binding of libwpp.so: argument marshalling only — every step of the path runs in the library.

The functions carry the C names (wpp_plan_tiles, wpp_kv_append, wpp_prefill_attention_varlen).  Tensors are
torch tensors used as device memory; streams are torch streams.  There is no fallback: if the library cannot be
loaded, or no sm_100 device is present, the calls raise.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("WPP_LIB_PATH") or os.path.join(_HERE, "libwpp.so")   # override: a differently built library

WPP_OK = 0
WPP_BF16 = 1
STATUS_NAMES = {
    0: "WPP_OK", 1: "WPP_ERR_INVALID_ARG", 2: "WPP_ERR_UNSUPPORTED", 3: "WPP_ERR_BOUNDS",
    4: "WPP_ERR_POSITION_MISMATCH", 5: "WPP_ERR_WORKSPACE_TOO_SMALL", 6: "WPP_ERR_PLAN_MISMATCH",
    7: "WPP_ERR_CUDA", 8: "WPP_ERR_TIMEOUT", 9: "WPP_ERR_ALIASED_APPEND",
}


class WppError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)}")


class BatchDesc(ctypes.Structure):
    _fields_ = [
        ("num_requests", ctypes.c_int32), ("num_q_heads", ctypes.c_int32), ("num_kv_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32), ("page_size", ctypes.c_int32), ("max_blocks_per_req", ctypes.c_int32),
        ("num_pages", ctypes.c_int32), ("dtype", ctypes.c_int32), ("sm_scale", ctypes.c_float),
        ("reserved0", ctypes.c_int32),
        ("kv_page_stride", ctypes.c_int64), ("kv_head_stride", ctypes.c_int64), ("kv_token_stride", ctypes.c_int64),
        ("q_token_stride", ctypes.c_int64), ("q_head_stride", ctypes.c_int64),
        ("kvnew_token_stride", ctypes.c_int64), ("kvnew_head_stride", ctypes.c_int64),
        ("o_token_stride", ctypes.c_int64), ("o_head_stride", ctypes.c_int64),
    ]


class PlanOpts(ctypes.Structure):
    _fields_ = [("tile_m", ctypes.c_int32), ("tile_n", ctypes.c_int32), ("force_kv_splits", ctypes.c_int32),
                ("max_ctas", ctypes.c_int32), ("order", ctypes.c_int32), ("shape", ctypes.c_int32)]


class PlanInfo(ctypes.Structure):
    _fields_ = [("num_tiles", ctypes.c_int64), ("num_split_tiles", ctypes.c_int64),
                ("num_combine_tiles", ctypes.c_int64), ("num_ctas", ctypes.c_int64),
                ("total_new_tokens", ctypes.c_int64), ("key_steps", ctypes.c_int64), ("flops", ctypes.c_int64),
                ("shape", ctypes.c_int64), ("workspace_bytes", ctypes.c_size_t), ("plan_bytes", ctypes.c_size_t)]


class WaveConfig(ctypes.Structure):
    _fields_ = [("num_stages", ctypes.c_int32), ("fill_factor", ctypes.c_int32), ("block_size", ctypes.c_int32),
                ("max_lanes", ctypes.c_int32), ("max_budget", ctypes.c_int64), ("min_budget", ctypes.c_int64)]


class WaveState(ctypes.Structure):
    _fields_ = [("cur", ctypes.c_int32), ("direction", ctypes.c_int32), ("count", ctypes.c_int32),
                ("reserved", ctypes.c_int32)]

    def as_tuple(self):
        return (int(self.cur), int(self.direction), int(self.count))


class WaveInfo(ctypes.Structure):
    _fields_ = [("budget", ctypes.c_int64), ("work", ctypes.c_int64), ("wave_tokens", ctypes.c_int64),
                ("target_index", ctypes.c_int32), ("budget_index", ctypes.c_int32), ("lanes", ctypes.c_int32),
                ("defer", ctypes.c_int32)]


class KdaDesc(ctypes.Structure):
    _fields_ = [("num_requests", ctypes.c_int32), ("num_heads", ctypes.c_int32), ("d_k", ctypes.c_int32),
                ("d_v", ctypes.c_int32), ("num_slots", ctypes.c_int32), ("snap_interval", ctypes.c_int32),
                ("max_snaps", ctypes.c_int32), ("layout", ctypes.c_int32), ("total_tokens", ctypes.c_int64)]


WAVE_RING_BUSY, WAVE_ADMISSION_PENDING, WAVE_ALREADY_DEFERRED = 1, 2, 4

EXPORTS = ["wpp_create", "wpp_destroy", "wpp_status_string", "wpp_last_cuda_error", "wpp_plan_bytes",
           "wpp_plan_tiles", "wpp_validate_batch", "wpp_kv_append", "wpp_prefill_attention_varlen",
           "wpp_launch_count", "wpp_set_rescale_mode", "wpp_rescale_stats", "wpp_prefill_attention_varlen_static",
           "wpp_static_scratch_bytes",
           "wpp_selftest_bounded_wait", "wpp_wave_ladder", "wpp_plan_waves",
           "wpp_hash_blocks", "wpp_hash_blocks_host", "wpp_hint_index_create", "wpp_hint_index_destroy",
           "wpp_hint_index_add", "wpp_hint_index_remove", "wpp_hint_index_size", "wpp_hint_probe",
           "wpp_hint_probe_recurrent", "wpp_kda_chunk", "wpp_kda_workspace_bytes"]

_lib = None


def load_library() -> ctypes.CDLL:
    """Load libwpp.so (built in-tree by paper_2609_35263_b200.build); raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2609_35263_b200.build` "
                              "(there is no fallback path)")
        lib = ctypes.CDLL(LIB_PATH)
        vp, i32p = ctypes.c_void_p, ctypes.c_void_p
        lib.wpp_create.argtypes = [ctypes.POINTER(vp), ctypes.c_int]
        lib.wpp_destroy.argtypes = [vp]
        lib.wpp_status_string.restype = ctypes.c_char_p
        lib.wpp_status_string.argtypes = [ctypes.c_int]
        lib.wpp_last_cuda_error.argtypes = [vp]
        lib.wpp_launch_count.argtypes = [vp]
        lib.wpp_launch_count.restype = ctypes.c_int64
        lib.wpp_set_rescale_mode.argtypes = [vp, ctypes.c_int]
        lib.wpp_rescale_stats.argtypes = [vp, ctypes.POINTER(ctypes.c_uint64), ctypes.POINTER(ctypes.c_uint64),
                                          ctypes.POINTER(ctypes.c_int)]
        lib.wpp_plan_bytes.restype = ctypes.c_size_t
        lib.wpp_plan_bytes.argtypes = [vp, ctypes.POINTER(BatchDesc), ctypes.c_int64, ctypes.POINTER(PlanOpts)]
        lib.wpp_plan_tiles.argtypes = [vp, ctypes.POINTER(BatchDesc), i32p, i32p, i32p, ctypes.POINTER(PlanOpts),
                                       vp, ctypes.c_size_t, ctypes.POINTER(PlanInfo)]
        lib.wpp_validate_batch.argtypes = [ctypes.POINTER(BatchDesc), i32p, i32p, i32p]
        lib.wpp_kv_append.argtypes = [vp, ctypes.POINTER(BatchDesc), vp, vp, vp, vp, i32p, i32p, i32p, vp, vp,
                                      i32p, vp]
        lib.wpp_prefill_attention_varlen.argtypes = [vp, ctypes.POINTER(BatchDesc), vp, vp, vp, vp, vp, i32p, i32p,
                                                     i32p, vp, vp, vp, ctypes.c_size_t, i32p, vp]
        lib.wpp_prefill_attention_varlen_static.argtypes = [vp, ctypes.POINTER(BatchDesc), vp, vp, vp, vp, vp, i32p,
                                                            i32p, i32p, vp, vp, i32p, vp]
        lib.wpp_selftest_bounded_wait.argtypes = [vp, ctypes.c_int64, i32p, vp, vp]
        lib.wpp_static_scratch_bytes.restype = ctypes.c_size_t
        lib.wpp_static_scratch_bytes.argtypes = []
        lib.wpp_hash_blocks.argtypes = [vp, vp, vp, vp, ctypes.c_int32, ctypes.c_int32, ctypes.c_uint64, vp, vp,
                                        ctypes.c_int64, vp]
        lib.wpp_hash_blocks_host.argtypes = [vp, ctypes.c_int64, ctypes.c_int32, ctypes.c_uint64, vp, vp]
        lib.wpp_hint_index_create.argtypes = [ctypes.POINTER(vp)]
        lib.wpp_hint_index_destroy.argtypes = [vp]
        lib.wpp_hint_index_add.argtypes = [vp, ctypes.c_int32, vp, ctypes.c_int64]
        lib.wpp_hint_index_remove.argtypes = [vp, ctypes.c_int32, vp, ctypes.c_int64]
        lib.wpp_hint_index_size.argtypes = [vp]
        lib.wpp_hint_index_size.restype = ctypes.c_int64
        lib.wpp_hint_probe.argtypes = [vp, ctypes.c_int32, vp, ctypes.c_int64, ctypes.POINTER(ctypes.c_int64),
                                       ctypes.POINTER(ctypes.c_int32)]
        lib.wpp_hint_probe_recurrent.argtypes = [vp, ctypes.c_int32, vp, ctypes.c_int64, ctypes.POINTER(ctypes.c_int64),
                                                 ctypes.POINTER(ctypes.c_int32)]
        lib.wpp_wave_ladder.argtypes = [ctypes.POINTER(WaveConfig), vp, ctypes.c_int32, ctypes.POINTER(ctypes.c_int32)]
        lib.wpp_plan_waves.argtypes = [ctypes.POINTER(WaveConfig), ctypes.POINTER(WaveState), vp, ctypes.c_int32, vp,
                                       ctypes.c_int32, ctypes.c_int32, vp, ctypes.POINTER(WaveInfo)]
        lib.wpp_kda_chunk.argtypes = [vp, ctypes.POINTER(KdaDesc)] + [vp] * 13 + [ctypes.c_size_t, vp, vp]
        lib.wpp_kda_workspace_bytes.restype = ctypes.c_size_t
        lib.wpp_kda_workspace_bytes.argtypes = [ctypes.POINTER(KdaDesc)]
        _lib = lib
    return _lib


def _check(status: int, where: str):
    if status != WPP_OK:
        raise WppError(status, where)


class Context:
    """wpp_ctx for one CUDA device."""

    def __init__(self, device: int = 0):
        lib = load_library()
        self._h = ctypes.c_void_p()
        _check(lib.wpp_create(ctypes.byref(self._h), int(device)), "wpp_create")
        self.device = int(device)

    @property
    def handle(self):
        return self._h

    def launch_count(self) -> int:
        return int(load_library().wpp_launch_count(self._h))

    def set_rescale_mode(self, mode: int) -> None:
        """0: rescale before the exponentials (default); 1: after; 2: the library chooses from what its kernels counted."""
        _check(load_library().wpp_set_rescale_mode(self._h, int(mode)), "wpp_set_rescale_mode")

    def rescale_stats(self):
        """(key steps, steps that rescaled an accumulator, whether the next call rescales after the exponentials)."""
        s, m, late = ctypes.c_uint64(0), ctypes.c_uint64(0), ctypes.c_int(0)
        _check(load_library().wpp_rescale_stats(self._h, ctypes.byref(s), ctypes.byref(m), ctypes.byref(late)),
               "wpp_rescale_stats")
        return int(s.value), int(m.value), bool(late.value)

    def last_cuda_error(self) -> int:
        return int(load_library().wpp_last_cuda_error(self._h))

    def close(self):
        if self._h:
            load_library().wpp_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def make_desc(num_requests, num_q_heads, num_kv_heads, head_dim, page_size, max_blocks_per_req, num_pages,
              sm_scale: float = 0.0, **strides) -> BatchDesc:
    d = BatchDesc()
    d.num_requests, d.num_q_heads, d.num_kv_heads = int(num_requests), int(num_q_heads), int(num_kv_heads)
    d.head_dim, d.page_size = int(head_dim), int(page_size)
    d.max_blocks_per_req, d.num_pages = int(max_blocks_per_req), int(num_pages)
    d.dtype = WPP_BF16
    d.sm_scale = float(sm_scale)
    for k, v in strides.items():
        setattr(d, k, int(v))
    return d


def _np_i32(x) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(x, dtype=np.int32))


class Plan:
    """Host plan buffer (pinned when CUDA is present), its device copy and the planner's summary."""

    def __init__(self, host: torch.Tensor, info: PlanInfo):
        self.host = host
        self.info = info
        self.dev: Optional[torch.Tensor] = None

    @property
    def plan_bytes(self) -> int:
        return int(self.info.plan_bytes)

    def to_device(self, device="cuda", non_blocking=True, out: Optional[torch.Tensor] = None) -> "Plan":
        """Copy the used part of the host plan to the device (into `out` if given) on the current stream."""
        if out is not None:
            out[: self.plan_bytes].copy_(self.host[: self.plan_bytes], non_blocking=non_blocking)
            self.dev = out
        else:
            self.dev = self.host[: self.plan_bytes].to(device, non_blocking=non_blocking)
        return self

    def host_bytes(self) -> bytes:
        return bytes(self.host[: self.plan_bytes].numpy().tobytes())


def wpp_plan_tiles(ctx: Optional[Context], desc: BatchDesc, prefix_lens, chunk_lens, cached_lens=None,
                   opts: Optional[PlanOpts] = None, pin: Optional[bool] = None,
                   out: Optional[torch.Tensor] = None) -> Plan:
    """Host-side work split; returns a Plan whose .host buffer must be copied to the device (.to_device()).

    `out` may be a reusable host uint8 tensor (pinned for asynchronous copies) of at least wpp_plan_bytes bytes."""
    lib = load_library()
    P, C = _np_i32(prefix_lens), _np_i32(chunk_lens)
    T = int(C.astype(np.int64).sum())
    h = ctx.handle if ctx is not None else None
    optp = ctypes.byref(opts) if opts is not None else None
    nbytes = int(lib.wpp_plan_bytes(h, ctypes.byref(desc), T, optp))
    if nbytes == 0:
        # let wpp_plan_tiles report the precise error
        nbytes = 4096
    if out is not None and out.numel() >= nbytes and out.dtype == torch.uint8 and out.device.type == "cpu":
        host, nbytes = out, out.numel()
    else:
        pin = torch.cuda.is_available() if pin is None else pin
        host = torch.empty(nbytes, dtype=torch.uint8, pin_memory=bool(pin))
    info = PlanInfo()
    cached = _np_i32(cached_lens) if cached_lens is not None else None
    st = lib.wpp_plan_tiles(h, ctypes.byref(desc), P.ctypes.data, C.ctypes.data,
                            cached.ctypes.data if cached is not None else None, optp,
                            host.data_ptr(), nbytes, ctypes.byref(info))
    _check(st, "wpp_plan_tiles")
    return Plan(host, info)


def wpp_validate_batch(desc: BatchDesc, block_tables, prefix_lens, chunk_lens) -> int:
    bt, P, C = _np_i32(block_tables), _np_i32(prefix_lens), _np_i32(chunk_lens)
    return int(load_library().wpp_validate_batch(ctypes.byref(desc), bt.ctypes.data, P.ctypes.data, C.ctypes.data))


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def wpp_kv_append(ctx: Context, desc: BatchDesc, k_new, v_new, k_cache, v_cache, block_tables, prefix_lens,
                  chunk_lens, plan: Plan, status=None, stream=None) -> None:
    """Queue the KV append of one wave on `stream` (device tensors; int32 metadata on the device)."""
    st = load_library().wpp_kv_append(ctx.handle, ctypes.byref(desc), _ptr(k_new), _ptr(v_new), _ptr(k_cache),
                                      _ptr(v_cache), _ptr(block_tables), _ptr(prefix_lens), _ptr(chunk_lens),
                                      ctypes.c_void_p(plan.host.data_ptr()), _ptr(plan.dev), _ptr(status),
                                      _stream(stream))
    _check(st, "wpp_kv_append")


def wpp_prefill_attention_varlen(ctx: Context, desc: BatchDesc, q, out, lse, k_cache, v_cache, block_tables,
                                 prefix_lens, chunk_lens, plan: Plan, workspace=None, status=None,
                                 stream=None) -> None:
    """Queue chunked-prefill attention of one wave on `stream`; results land in `out` (and `lse` if given)."""
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    st = load_library().wpp_prefill_attention_varlen(
        ctx.handle, ctypes.byref(desc), _ptr(q), _ptr(out), _ptr(lse), _ptr(k_cache), _ptr(v_cache),
        _ptr(block_tables), _ptr(prefix_lens), _ptr(chunk_lens), ctypes.c_void_p(plan.host.data_ptr()),
        _ptr(plan.dev), _ptr(workspace), ws_bytes, _ptr(status), _stream(stream))
    _check(st, "wpp_prefill_attention_varlen")


def wpp_static_scratch_bytes() -> int:
    """Size of the scratch array built into the library (used by wpp_prefill_attention_varlen_static)."""
    return int(load_library().wpp_static_scratch_bytes())


def wpp_prefill_attention_varlen_static(ctx: Context, desc: BatchDesc, q, out, lse, k_cache, v_cache, block_tables,
                                        prefix_lens, chunk_lens, plan: Plan, status=None, stream=None) -> None:
    """wpp_prefill_attention_varlen without a caller workspace and without any allocation.

    For callers that cannot obtain device memory at call time (a serving process whose KV page pool already owns
    all free HBM, an execution stream that must not be stalled by cudaMalloc).  Split-KV partials go to a fixed
    16 MiB array inside the library; plans that need more raise WPP_ERR_WORKSPACE_TOO_SMALL.  All calls on a
    device share that array, so calls whose kernels could overlap on the GPU must be serialised.  The first call
    on a device does a one-time address look-up (the context's device must be current) and should come before any
    stream capture."""
    st = load_library().wpp_prefill_attention_varlen_static(
        ctx.handle, ctypes.byref(desc), _ptr(q), _ptr(out), _ptr(lse), _ptr(k_cache), _ptr(v_cache),
        _ptr(block_tables), _ptr(prefix_lens), _ptr(chunk_lens), ctypes.c_void_p(plan.host.data_ptr()),
        _ptr(plan.dev), _ptr(status), _stream(stream))
    _check(st, "wpp_prefill_attention_varlen_static")


def wpp_selftest_bounded_wait(ctx: Context, limit_cycles: int, status, waited_cycles=None, stream=None) -> None:
    """Launch the bounded-wait self-test: a warp waits at most `limit_cycles` on a barrier nothing arrives on."""
    st = load_library().wpp_selftest_bounded_wait(ctx.handle, int(limit_cycles), _ptr(status), _ptr(waited_cycles),
                                                  _stream(stream))
    _check(st, "wpp_selftest_bounded_wait")


def wpp_wave_ladder(cfg: WaveConfig):
    """The budgets the wave planner chooses from, largest first (Eq. design-budget)."""
    lib = load_library()
    n = ctypes.c_int32(0)
    _check(lib.wpp_wave_ladder(ctypes.byref(cfg), None, 0, ctypes.byref(n)), "wpp_wave_ladder")
    out = np.zeros(n.value, dtype=np.int64)
    _check(lib.wpp_wave_ladder(ctypes.byref(cfg), out.ctypes.data_as(ctypes.c_void_p), n.value, ctypes.byref(n)),
           "wpp_wave_ladder")
    return out.tolist()


def wpp_plan_waves(cfg: WaveConfig, state: WaveState, remaining, inflight=(), flags: int = 0):
    """One planning decision (Section 4.5): updates `state` in place, returns (chunk_lens int32 array, WaveInfo)."""
    rem = np.ascontiguousarray(np.asarray(remaining, dtype=np.int64))
    inf = np.ascontiguousarray(np.asarray(inflight, dtype=np.int64))
    chunks = np.zeros(rem.shape[0], dtype=np.int32)
    info = WaveInfo()
    st = load_library().wpp_plan_waves(
        ctypes.byref(cfg), ctypes.byref(state), rem.ctypes.data_as(ctypes.c_void_p) if rem.size else None,
        int(rem.size), inf.ctypes.data_as(ctypes.c_void_p) if inf.size else None, int(inf.size), int(flags),
        chunks.ctypes.data_as(ctypes.c_void_p) if rem.size else None, ctypes.byref(info))
    _check(st, "wpp_plan_waves")
    return chunks, info


def wpp_hash_blocks(ctx: Context, tokens, token_offsets, block_offsets, block_size: int, salt: int = 0, extra_keys=None,
                    stream=None, total_blocks: Optional[int] = None, out=None):
    """Chained hashes of the full token blocks of a batch of requests on the GPU (Eq. design-hash).

    tokens: cuda int32; token_offsets, block_offsets: cuda int64 [R+1]; returns a cuda int64 tensor holding the
    64-bit hashes' bit patterns, request i's at [block_offsets[i], block_offsets[i+1])."""
    R = int(token_offsets.numel()) - 1
    if total_blocks is None:                 # reads the last offset back from the device: pass it to avoid the sync
        total_blocks = int(block_offsets[-1].item()) if R >= 0 and block_offsets.numel() else 0
    total = int(total_blocks)
    if out is None:
        out = torch.empty(total, dtype=torch.int64, device=tokens.device)
    st = load_library().wpp_hash_blocks(ctx.handle, _ptr(tokens), _ptr(token_offsets), _ptr(block_offsets), max(R, 0),
                                        int(block_size), ctypes.c_uint64(int(salt) & (2 ** 64 - 1)), _ptr(extra_keys),
                                        _ptr(out), total, _stream(stream))
    _check(st, "wpp_hash_blocks")
    return out


def wpp_hash_blocks_host(tokens, block_size: int, salt: int = 0, extra_keys=None) -> np.ndarray:
    """The same chain for one request on the host; returns uint64 [len(tokens) // block_size]."""
    t = np.ascontiguousarray(np.asarray(tokens, dtype=np.int32))
    out = np.zeros(t.size // int(block_size), dtype=np.uint64)
    e = None if extra_keys is None else np.ascontiguousarray(np.asarray(extra_keys, dtype=np.uint64))
    st = load_library().wpp_hash_blocks_host(
        t.ctypes.data_as(ctypes.c_void_p) if t.size else None, int(t.size), int(block_size),
        ctypes.c_uint64(int(salt) & (2 ** 64 - 1)), e.ctypes.data_as(ctypes.c_void_p) if e is not None else None,
        out.ctypes.data_as(ctypes.c_void_p) if out.size else None)
    _check(st, "wpp_hash_blocks_host")
    return out


class HintIndex:
    """Counted index keyed by (cache window, chained block hash) with the gallop-and-bisect probe (Section 4.3)."""

    def __init__(self):
        self.handle = ctypes.c_void_p()
        _check(load_library().wpp_hint_index_create(ctypes.byref(self.handle)), "wpp_hint_index_create")

    def close(self):
        if self.handle:
            load_library().wpp_hint_index_destroy(self.handle)
            self.handle = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @staticmethod
    def _u64(hashes):
        return np.ascontiguousarray(np.asarray(hashes, dtype=np.uint64))

    def add(self, window: int, hashes) -> None:
        h = self._u64(hashes)
        _check(load_library().wpp_hint_index_add(self.handle, int(window),
                                                 h.ctypes.data_as(ctypes.c_void_p) if h.size else None, int(h.size)),
               "wpp_hint_index_add")

    def remove(self, window: int, hashes) -> None:
        h = self._u64(hashes)
        _check(load_library().wpp_hint_index_remove(self.handle, int(window),
                                                    h.ctypes.data_as(ctypes.c_void_p) if h.size else None, int(h.size)),
               "wpp_hint_index_remove")

    def __len__(self) -> int:
        return int(load_library().wpp_hint_index_size(self.handle))

    def probe(self, window: int, hashes):
        """(matched blocks, number of probes) for a request's chained hashes H_0 .."""
        h = self._u64(hashes)
        m, p = ctypes.c_int64(0), ctypes.c_int32(0)
        _check(load_library().wpp_hint_probe(self.handle, int(window),
                                             h.ctypes.data_as(ctypes.c_void_p) if h.size else None, int(h.size),
                                             ctypes.byref(m), ctypes.byref(p)), "wpp_hint_probe")
        return int(m.value), int(p.value)

    def probe_recurrent(self, window: int, hashes, limit_blocks: int):
        """(endpoint in blocks, number of probes) of a recurrent-state cache: the deepest snapshot boundary at or
        below `limit_blocks` whose key is in the index, found by scanning backward (Section 4.3)."""
        h = self._u64(hashes)
        limit = min(int(limit_blocks), int(h.size))
        m, p = ctypes.c_int64(0), ctypes.c_int32(0)
        _check(load_library().wpp_hint_probe_recurrent(self.handle, int(window),
                                                       h.ctypes.data_as(ctypes.c_void_p) if h.size else None, limit,
                                                       ctypes.byref(m), ctypes.byref(p)), "wpp_hint_probe_recurrent")
        return int(m.value), int(p.value)


def wpp_kda_workspace_bytes(num_requests: int, num_heads: int, total_tokens: int) -> int:
    """Bytes of workspace the chunk-parallel (tensor-core) form of wpp_kda_chunk needs for such a wave."""
    desc = KdaDesc(int(num_requests), int(num_heads), 128, 128, 0, 0, 0, 0, int(total_tokens))
    return int(load_library().wpp_kda_workspace_bytes(ctypes.byref(desc)))


def wpp_kda_chunk(ctx: Context, q, k, v, alpha, beta, row_offsets, state_pool, state_in, state_out, out=None,
                  prefix_lens=None, snap_interval: int = 0, snap_slots=None, status=None, stream=None, layout: int = 0,
                  workspace=None):
    """Queue the recurrent-state (KDA) layer of one wave on `stream` (Section 3.1 update, Section 3.2 snapshots).

    q, k: cuda bf16 [T, H, 128]; v: cuda bf16 [T, H, 128]; alpha: cuda fp32 [T, H, 128]; beta: cuda fp32 [T, H];
    row_offsets: cuda int64 [R+1]; state_pool: cuda fp32 [slots, H, 128, 128] (updated in place); state_in,
    state_out: cuda int32 [R] (-1: zero state / do not store); snap_slots: cuda int32 [R, max_snaps] with
    prefix_lens (cuda int32 [R]) and snap_interval > 0 for periodic snapshots.  layout 0 lets the library choose:
    the chunk-parallel tensor-core form when `workspace` (cuda uint8, wpp_kda_workspace_bytes bytes, 256-byte
    aligned) is given and the chunks average 64 tokens or more, else a token-by-token form; 1, 2: token by token
    with one / four CTAs per (request, head); 3: chunk-parallel.  Returns the cuda bf16 output."""
    T, H, dk = (int(x) for x in q.shape)
    dv = int(v.shape[2])
    R = int(row_offsets.numel()) - 1
    if out is None:
        out = torch.empty((T, H, dv), dtype=torch.bfloat16, device=q.device)
    max_snaps = 0 if snap_slots is None else int(snap_slots.shape[1])
    desc = KdaDesc(R, H, dk, dv, int(state_pool.shape[0]), int(snap_interval), max_snaps, int(layout), T)
    ws_bytes = 0 if workspace is None else int(workspace.numel() * workspace.element_size())
    st = load_library().wpp_kda_chunk(ctx.handle, ctypes.byref(desc), _ptr(q), _ptr(k), _ptr(v), _ptr(alpha), _ptr(beta),
                                      _ptr(row_offsets), _ptr(prefix_lens), _ptr(state_pool), _ptr(state_in),
                                      _ptr(state_out), _ptr(snap_slots), _ptr(out), _ptr(workspace), ws_bytes,
                                      _ptr(status), _stream(stream))
    _check(st, "wpp_kda_chunk")
    return out
