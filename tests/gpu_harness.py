"""Runs one wave through the C-ABI library on cuda:0 and returns everything a parity test needs."""
import numpy as np
import torch

import paper_2609_35263_b200 as wpp

_CTX = None


def ctx():
    global _CTX
    if _CTX is None:
        _CTX = wpp.Context(0)
    return _CTX


def desc_of(w, sm_scale=0.0):
    return wpp.make_desc(w.num_requests, w.num_q_heads, w.num_kv_heads, w.head_dim, w.page_size,
                         w.max_blocks_per_req, w.num_pages, sm_scale=sm_scale)


def device_inputs(w, inp=None, device="cuda"):
    """Inputs on the device: generated there (same bits as on the CPU) or copied from given CPU tensors."""
    if inp is None:
        return dict(q=w.q(device), k_new=w.k_new(device), v_new=w.v_new(device),
                    k_pool=w.k_pool(device), v_pool=w.v_pool(device))
    return {k: v.to(device) for k, v in inp.items()}


def run_wave(w, dev_inp, opts=None, sm_scale=0.0, want_lse=True, poison_out=True, do_append=True,
             do_attention=True, launch_prefix_lens=None, launch_chunk_lens=None, shape=None):
    """plan -> H2D plan -> wpp_kv_append -> wpp_prefill_attention_varlen on the current stream.
    launch_prefix_lens / launch_chunk_lens: device arrays the kernels get instead of the lengths the plan was made
    for (a host-made mismatch).  shape: 1 or 2 overrides the planner's choice of attention kernel."""
    if shape is not None:
        o = opts or wpp.PlanOpts()
        opts = wpp.PlanOpts(o.tile_m, o.tile_n, o.force_kv_splits, o.max_ctas, o.order, shape)
    c = ctx()
    d = desc_of(w, sm_scale)
    plan = wpp.wpp_plan_tiles(c, d, w.prefix_lens, w.chunk_lens, opts=opts).to_device()
    dev = torch.device("cuda")
    bt = torch.from_numpy(w.block_tables).to(dev)
    P = torch.from_numpy(np.asarray(w.prefix_lens if launch_prefix_lens is None else launch_prefix_lens,
                                    dtype=np.int32)).to(dev)
    C = torch.from_numpy(np.asarray(w.chunk_lens if launch_chunk_lens is None else launch_chunk_lens,
                                    dtype=np.int32)).to(dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    T = w.total_new_tokens
    out = torch.empty(T, w.num_q_heads, w.head_dim, dtype=torch.bfloat16, device=dev)
    lse = torch.empty(T, w.num_q_heads, dtype=torch.float32, device=dev) if want_lse else None
    if poison_out:
        out.view(torch.int16).fill_(0x7FC0)          # NaN: any row the kernel forgets shows up
        if lse is not None:
            lse.fill_(float("nan"))
    ws = None
    if plan.info.workspace_bytes:
        ws = torch.empty(int(plan.info.workspace_bytes), dtype=torch.uint8, device=dev)
        ws.fill_(0xFF)                                # NaN patterns in the scratch too
    if do_append:
        wpp.wpp_kv_append(c, d, dev_inp["k_new"], dev_inp["v_new"], dev_inp["k_pool"], dev_inp["v_pool"], bt, P, C,
                          plan, status=status)
    if do_attention:
        wpp.wpp_prefill_attention_varlen(c, d, dev_inp["q"], out, lse, dev_inp["k_pool"], dev_inp["v_pool"], bt, P,
                                         C, plan, workspace=ws, status=status)
    torch.cuda.synchronize()
    return dict(out=out, lse=lse, status=int(status.item()), plan=plan, k_pool=dev_inp["k_pool"],
                v_pool=dev_inp["v_pool"])


def compare(gpu_out_f64: np.ndarray, ref: np.ndarray):
    """Error figures against the fp64 oracle: the stated tolerances plus scale-relative ones."""
    diff = np.abs(gpu_out_f64 - ref)
    rms = float(np.sqrt(np.mean(ref ** 2))) if ref.size else 0.0
    return dict(max_abs=float(diff.max()) if diff.size else 0.0,
                mean_abs=float(diff.mean()) if diff.size else 0.0,
                rms_ref=rms, max_ref=float(np.abs(ref).max()) if ref.size else 0.0,
                nan=int(np.isnan(gpu_out_f64).sum()))


# The benchmark spec's tolerance for bf16 inputs with fp32 accumulation, and tighter scale-relative gates that a
# kernel dropping whole key tiles at long context could not pass.
MAX_ABS_TOL = 2e-2
MEAN_ABS_TOL = 2e-3
REL_MEAN_TOL = 5e-3     # mean|delta| <= this * rms(reference)
REL_MAX_TOL = 1e-2      # max|delta|  <= this * max|reference|  (plus one bf16 ulp of slack at the top value)


def assert_close(gpu_out_f64, ref, what=""):
    e = compare(gpu_out_f64, ref)
    assert e["nan"] == 0, f"{what}: {e['nan']} NaN outputs"
    assert e["max_abs"] <= MAX_ABS_TOL and e["mean_abs"] <= MEAN_ABS_TOL, f"{what}: {e}"
    assert e["mean_abs"] <= REL_MEAN_TOL * e["rms_ref"] + 1e-6, f"{what}: relative mean gate {e}"
    assert e["max_abs"] <= REL_MAX_TOL * e["max_ref"] + 2e-3, f"{what}: relative max gate {e}"
    return e


# ---------------------------------------------------------------------------------------------------------------
# Workloads whose pools are too large to copy to the host as a whole: the oracle gets one request at a time.
def request_slice(w, dev_inp, i):
    """Host copy of everything request `i` touches, as a one-request problem with a private pool.

    The request's pages are gathered through its block-table row from the device pools (call this BEFORE the wave
    runs: the append writes into those pages) and renumbered 0..n-1; q / k_new / v_new are the request's rows.
    Returns a dict the oracle's entry points accept (bf16 CPU tensors, int32 arrays)."""
    P, C = int(w.prefix_lens[i]), int(w.chunk_lens[i])
    nb = (P + C + w.page_size - 1) // w.page_size
    ids = torch.from_numpy(w.block_tables[i, :nb].astype(np.int64)).to(dev_inp["k_pool"].device)
    off = w.q_offsets
    r0, r1 = int(off[i]), int(off[i + 1])
    return dict(q=dev_inp["q"][r0:r1].cpu(), k_new=dev_inp["k_new"][r0:r1].cpu(), v_new=dev_inp["v_new"][r0:r1].cpu(),
                k_pool=dev_inp["k_pool"][ids].cpu(), v_pool=dev_inp["v_pool"][ids].cpu(),
                block_tables=np.arange(nb, dtype=np.int32).reshape(1, nb),
                prefix_lens=np.array([P], dtype=np.int32), chunk_lens=np.array([C], dtype=np.int32),
                page_ids=ids, rows=(r0, r1))


def appended_pages_of(dev_inp, sl):
    """The request's pages as they are on the device now (after the wave), in the slice's numbering."""
    return dev_inp["k_pool"][sl["page_ids"]], dev_inp["v_pool"][sl["page_ids"]]
