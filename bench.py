#!/usr/bin/env python
"""Benchmark of the chunked-prefill attention hot path (plan -> KV append -> paged attention).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config cfg3] [--impl reference]

One step = one wave through the whole path: wpp_plan_tiles on the host, the plan's H2D copy, wpp_kv_append
and wpp_prefill_attention_varlen, all through the C ABI.  Default workload: the concurrency-128 high-reuse
configuration (80 % of 128 requests share a 16384-token prefix).  Prints ONE JSON line on rank 0.

  value      new (query) tokens per second with every input resident in HBM
  e2e        the same through host buffers: per step H2D of q/k_new/v_new/metadata from pinned memory and D2H of out
  roofline   attention kernel: algorithmic FLOPs (4 d Hq sum(C P + C(C+1)/2)) / CUDA-event time vs measured bf16 peak
  cpu_baseline  the fp64 oracle on this machine's host cores on a bounded seeded sample, extrapolated by visible pairs

`--impl reference` times the oracle alone (the only reference there is: the paper ships no code).
Multi-GPU: the path does not shard (one stage, one GPU); N > 1 runs N independent replicas ("weak").
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "prefill-attention tokens/s at concurrency 128, high prefix reuse"
# DRAM traffic is not measured by this script (it would need a profiler): `roofline.traffic` scales a figure from an
# ncu capture by the work of the launch timed here, and `roofline.traffic_source` says so in the JSON line.
# Attention: dram__bytes_read.sum + dram__bytes_write.sum of one launch / its 128-row x 128-key steps, captured on the
# 16-request cut of the concurrency-128 workload (--config cfg3_r16, 1.4 GB resident).
DRAM_BYTES_PER_KEY_STEP = 607.6
DRAM_SOURCE = ("estimate: 607.6 DRAM bytes per 128x128 key step (dram__bytes_read.sum + dram__bytes_write.sum of one "
               "wpp_attn_kernel launch, ncu capture on the 16-request cut of this workload) x this launch's key steps; "
               "not measured in this run")
# Recurrent layer: dram read + write bytes of one wpp_kda_chunk launch on the default wave (8 x 2,048 tokens, 32 heads)
# / its 524,288 (token, head) pairs; other wave shapes scale with the pairs (the state traffic per request is small).
KDA_DRAM_BYTES_PER_TOKEN_HEAD = 1571.3
# Chunk-parallel form: (673.3 MB + 1156.4 MB) of the preparation kernel + (1233.3 MB + 137.7 MB) of the chain kernel on
# the same wave / 524,288 pairs.
KDA_TC_DRAM_BYTES_PER_TOKEN_HEAD = 6104.9
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
NOMINAL_BF16_TFLOPS = 2250.0        # dense bf16 of the data sheet (context only: no kernel reaches it under the power cap)


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            d = json.load(open(path))
            return d, "measured"
        except Exception:
            pass
    return dict(FALLBACK_PEAKS), "fallback"


def build_workload(name):
    import wpp_workloads as W
    if name in W.CONFIG_BUILDERS:
        return W.CONFIG_BUILDERS[name]()
    if name.startswith("cfg3_r"):         # cfg3_r16: the first 16 requests' worth of the same draw (for profiling)
        return W.cfg3(num_requests=int(name[6:]))
    if name.startswith("cfg5_"):          # cfg5_C1024_P4096
        parts = dict((p[0], int(p[1:])) for p in name.split("_")[1:])
        return W.cfg5_cell(parts["C"], parts["P"])
    raise SystemExit(f"unknown config {name}")


def describe_config(w, world=1):
    """The workload description both arms print (same keys, so the two lines can be matched)."""
    return {"workload": w.name, "requests": w.num_requests, "new_tokens": w.total_new_tokens,
            "served_tokens": int((w.prefix_lens.astype(np.int64) + w.chunk_lens).sum()),
            "q_heads": w.num_q_heads, "kv_heads": w.num_kv_heads, "head_dim": w.head_dim,
            "page_size": w.page_size, "parallelism": "replicas only" if world > 1 else "single GPU"}


def roofline_times(w, flops, peaks):
    """(tensor-bound ms, HBM-bound ms) of one attention launch: FLOPs at the bf16 peak, compulsory bytes (Q in, O
    out, each unique KV page once) at the copy bandwidth."""
    kv_bytes = w.unique_kv_pages() * w.num_kv_heads * w.page_size * w.head_dim * 2 * 2
    qo_bytes = 2 * w.total_new_tokens * w.num_q_heads * w.head_dim * 2
    t_flops = flops / (float(peaks.get("bf16_tflops", FALLBACK_PEAKS["bf16_tflops"])) * 1e12)
    t_bytes = (kv_bytes + qo_bytes) / (float(peaks.get("hbm_gbs", FALLBACK_PEAKS["hbm_gbs"])) * 1e9)
    return t_flops * 1e3, t_bytes * 1e3, kv_bytes, qo_bytes


def measure_other_config(name, ctx, dev, peaks, steps=3, warmup=3):
    """One more workload under the same clock: append + attention through the C ABI, CUDA events on the launching
    stream, L2 flushed between steps when the inputs fit it.  Returns the kernel time, TFLOP/s and the fraction of
    the roofline time (the slower of FLOPs at the tensor peak and compulsory bytes at HBM bandwidth)."""
    import torch
    import paper_2609_35263_b200 as wpp
    w = build_workload(name)
    desc = wpp.make_desc(w.num_requests, w.num_q_heads, w.num_kv_heads, w.head_dim, w.page_size,
                         w.max_blocks_per_req, w.num_pages)
    q, k_new, v_new, k_pool, v_pool = w.q(dev), w.k_new(dev), w.v_new(dev), w.k_pool(dev), w.v_pool(dev)
    bt, P, C = (torch.from_numpy(x).to(dev) for x in (w.block_tables, w.prefix_lens, w.chunk_lens))
    out = torch.empty(w.total_new_tokens, w.num_q_heads, w.head_dim, dtype=torch.bfloat16, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    plan = wpp.wpp_plan_tiles(ctx, desc, w.prefix_lens, w.chunk_lens).to_device()
    ws = torch.empty(max(256, int(plan.info.workspace_bytes)), dtype=torch.uint8, device=dev)
    flops = float(plan.info.flops)
    t_flops, t_bytes, kv_bytes, qo_bytes = roofline_times(w, flops, peaks)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if kv_bytes + qo_bytes < 2 * (126 << 20) else None
    stream = torch.cuda.current_stream()
    times = []
    for i in range(warmup + steps):
        if i == warmup:
            torch.cuda.synchronize()         # the timed steps start from an idle device (and the library has seen
                                             # what its kernels counted during the warm-up)
        if flush is not None:
            flush.fill_(i & 0xFF)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        wpp.wpp_kv_append(ctx, desc, k_new, v_new, k_pool, v_pool, bt, P, C, plan, status=status)
        a.record(stream)
        wpp.wpp_prefill_attention_varlen(ctx, desc, q, out, None, k_pool, v_pool, bt, P, C, plan, workspace=ws,
                                         status=status)
        b.record(stream)
        if i >= warmup:
            times.append((a, b))
    torch.cuda.synchronize()
    if int(status.item()) != 0:
        raise SystemExit(f"device status {int(status.item())} on {name}")
    ms = statistics.mean(a.elapsed_time(b) for a, b in times)
    return {"workload": w.name, "steps": steps, "new_tokens": w.total_new_tokens, "kernel_ms": ms,
            "tokens_per_s": w.total_new_tokens / (ms * 1e-3), "tflops": flops / (ms * 1e-3) / 1e12,
            "bound": "tensor" if t_flops >= t_bytes else "hbm", "roofline_ms": max(t_flops, t_bytes),
            "frac_of_roofline_time": max(t_flops, t_bytes) / ms,
            "l2": "flushed between steps" if flush is not None else "inputs larger than L2",
            "rescale_in_use": "after" if ctx.rescale_stats()[2] else "before"}


OTHER_CONFIGS = ("cfg2", "cfg4", "cfg4_alt", "cfg5_C256_P0", "cfg5_C1024_P4096", "cfg5_C4096_P32768")


def measure_yardsticks(dev):
    """The two library kernels the roofline denominators were measured with, timed again in this run on this GPU
    (boxes of the pool differ by a few percent): a bf16 8192^3 torch.matmul, best of 10, and a 2 GiB copy, best of 5.
    Measurement only: the denominators of `roofline` stay the recorded ones."""
    import torch
    a = torch.randn(8192, 8192, device=dev, dtype=torch.bfloat16)
    b = torch.randn(8192, 8192, device=dev, dtype=torch.bfloat16)
    c = torch.empty(8192, 8192, device=dev, dtype=torch.bfloat16)
    best = float("inf")
    for i in range(13):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        torch.matmul(a, b, out=c)
        e1.record()
        e1.synchronize()
        if i >= 3:
            best = min(best, e0.elapsed_time(e1))
    tflops = 2 * 8192 ** 3 / (best * 1e-3) / 1e12
    del a, b, c
    src = torch.empty(1 << 30, device=dev, dtype=torch.bfloat16)
    dst = torch.empty_like(src)
    best_c = float("inf")
    for i in range(7):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        dst.copy_(src)
        e1.record()
        e1.synchronize()
        if i >= 2:
            best_c = min(best_c, e0.elapsed_time(e1))
    gbs = 2 * src.numel() * 2 / (best_c * 1e-3) / 1e9
    del src, dst
    return {"bf16_matmul_8192_tflops_best": tflops, "copy_1gi_bf16_gbs_best": gbs,
            "how": "torch.matmul and Tensor.copy_ (library kernels, yardsticks only), CUDA events"}


class ClockSampler:
    """nvidia-smi clocks / throttle reasons sampled every 200 ms while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.proc = None
        self.gpu_index = gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu_index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "200"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1])); pw.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(pw) if pw else None, "samples": len(sm), "reasons": sorted(reasons)}


class OracleSampler:
    """Times the fp64 oracle on seeded samples of (request, row, head) units; extrapolates by visible pairs."""

    def __init__(self, w, dev_available):
        import torch
        import oracle
        self.oracle, self.w = oracle, w
        dev = "cuda" if dev_available else "cpu"
        # inputs straight from the generators (never from the CUDA path), moved to the host
        self.q = w.q(dev).cpu()
        k_new, v_new = w.k_new(dev).cpu(), w.v_new(dev).cpu()
        k_pool, v_pool = w.k_pool(dev).cpu(), w.v_pool(dev).cpu()
        if dev_available:
            torch.cuda.empty_cache()
        self.kp, self.vp = oracle.oracle_append(k_new, v_new, k_pool, v_pool, w.block_tables, w.prefix_lens,
                                                w.chunk_lens)
        self.rng = np.random.default_rng(12345)
        self.P = w.prefix_lens.astype(np.int64)
        self.C = w.chunk_lens.astype(np.int64)
        self.live = np.nonzero(self.C > 0)[0]
        self.total_pairs = w.visible_pairs * w.num_q_heads
        self.rate = None          # visible pairs per second, from a probe
        self.mean_pairs = None

    def draw(self, n):
        i = self.live[self.rng.integers(0, self.live.size, size=n)]
        t = (self.rng.random(n) * self.C[i]).astype(np.int64)
        h = self.rng.integers(0, self.w.num_q_heads, size=n)
        return np.stack([i, t, h], axis=1).astype(np.int32)

    def run(self, units):
        w = self.w
        t0 = time.perf_counter()
        self.oracle.oracle_attention_units(self.q, self.kp, self.vp, w.block_tables, w.prefix_lens, w.chunk_lens,
                                           units)
        dt = time.perf_counter() - t0
        return dt, int((self.P[units[:, 0]] + units[:, 1] + 1).sum())

    def sample(self, seconds_target):
        if self.rate is None:
            probe = self.draw(256)
            dt, pairs = self.run(probe)
            self.rate, self.mean_pairs = pairs / max(dt, 1e-6), pairs / probe.shape[0]
        n = int(max(256, min(2_000_000, seconds_target * self.rate / self.mean_pairs)))
        dt, pairs = self.run(self.draw(n))
        t_full = dt * self.total_pairs / pairs
        return {"value": self.w.total_new_tokens / t_full, "unit": "tokens/s",
                "cores": self.oracle.oracle_threads(), "kind": "oracle",
                "sample": f"{n} seeded (request,row,head) units = {pairs:.3e} of {self.total_pairs:.3e} visible "
                          f"pairs, {dt:.1f} s of fp64 CPU work, extrapolated by visible-pair count",
                "sample_seconds": dt}


def run_reference(args):
    """Reference arm: the oracle as it stands on the host cores; each step is a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import torch
    w = build_workload(args.config)
    smp = OracleSampler(w, torch.cuda.is_available())
    per_step = max(1.0, min(15.0, 90.0 / max(1, args.steps + args.warmup)))
    vals, last = [], None
    for s in range(args.warmup + args.steps):
        last = smp.sample(per_step)
        if s >= args.warmup:
            vals.append(last["value"])
    v = float(np.mean(vals))
    line = {"impl": "reference", "metric": METRIC, "value": v, "unit": "tokens/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * w.total_new_tokens / v,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": dict(describe_config(w), note="fp64 CPU oracle, one bounded seeded sample per step; "
                           "ms_per_step is the extrapolated time of a full wave"),
            "cpu_baseline": {"value": v, "unit": "tokens/s", "cores": last["cores"], "kind": "oracle",
                             "sample": last["sample"]},
            "e2e": {"value": v, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def run_waves(args):
    """Host-only leg for the wave-budget planner (Section 4.5): wpp_plan_waves through the C ABI and the oracle
    walk the same seeded serving loop (bursty arrivals, one wave per decision, the last R waves in flight); both
    are timed on the host cores and their decisions compared.  No GPU is touched."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import paper_2609_35263_b200 as wpp
    from oracle import waves as O
    P, F, B, lanes, M, b_min = 4, 2, 64, 64, 16384, 1024
    cfg = wpp.WaveConfig(P, F, B, lanes, M, b_min)
    R = 2 * P
    rng = np.random.default_rng(7)
    decisions = 20000
    arrivals = [[int(x) for x in rng.integers(1, 40000, rng.integers(1, 8))] if rng.random() < 0.12 else []
                for _ in range(decisions)]

    def loop(decide):
        queue, ring, trace = [], [], []
        t0 = time.perf_counter()
        for it in range(decisions):
            queue += arrivals[it]
            chunks, budget = decide(queue, [c for wv in ring for c in wv])
            trace.append((budget, sum(chunks)))
            ring = (ring + [[c for c in chunks if c]])[-R:]
            queue = [r - c for r, c in zip(queue, chunks) if r - c > 0]
        return time.perf_counter() - t0, trace

    st = wpp.WaveState()

    def decide_c(queue, inflight):
        ch, info = wpp.wpp_plan_waves(cfg, st, queue, inflight)
        return ch.tolist(), int(info.budget)

    ost = [O.BudgetState()]

    def decide_o(queue, inflight):
        ost[0], b, ch, _ = O.plan_wave(P, F, M, b_min, B, lanes, queue, inflight, ost[0])
        return ch, b

    for _ in range(max(0, args.warmup)):
        st = wpp.WaveState()
        loop(decide_c)
    st = wpp.WaveState()
    t_c, trace_c = loop(decide_c)
    t_o, trace_o = loop(decide_o)
    if trace_c != trace_o:
        raise SystemExit("wpp_plan_waves and the oracle took different decisions")
    budgets = sorted({b for b, _ in trace_c}, reverse=True)
    line = {"metric": "wave-planning decisions/s (host, through the binding)", "value": decisions / t_c,
            "unit": "decisions/s", "n_gpus": 0, "steps": decisions, "warmup": args.warmup,
            "ms_per_step": 1e3 * t_c / decisions, "higher_is_better": True, "vs_baseline": None, "dtype": "int64",
            "data": "synthetic", "gpu_launches": 0,
            "config": {"workload": "seeded serving loop", "P": P, "F": F, "M": M, "b_min": b_min, "B": B,
                       "max_lanes": lanes, "budgets_used": budgets,
                       "tokens_scheduled": int(sum(t for _, t in trace_c)), "decisions_identical_to_oracle": True},
            "cpu_baseline": {"value": decisions / t_o, "unit": "decisions/s", "cores": 1, "kind": "oracle",
                             "sample": f"the same {decisions} decisions"}}
    print(json.dumps(line))


def run_waves_sim(args):
    """Wave planner and attention path together (Section 4.5 with this library's kernels): a burst of admitted
    requests is cut into waves by wpp_plan_waves, once with the budget fixed at M and once with the paper's budget
    ladder; every wave's chunk_lens go through wpp_plan_tiles, wpp_kv_append and wpp_prefill_attention_varlen on
    the GPU and its time is measured; a P-stage pipeline whose stages each take that time is then simulated
    (stage s starts wave w when it has finished wave w-1 and stage s-1 has finished wave w).  One GPU stands in
    for every stage: the stages' attention work is the same, their other layers are not modelled."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import torch
    import paper_2609_35263_b200 as wpp
    import wpp_workloads as W
    from wpp_workloads.generate import make_workload
    dev = torch.device("cuda", 0)
    P_stages, F, B, M, lanes = 4, 2, 64, 16384, 64
    rng = np.random.default_rng(11)
    R = 40
    sharer = rng.random(R) < 0.8
    cached = np.where(sharer, 16384, rng.integers(0, 129, R) * 64).astype(np.int64)
    suffix = rng.integers(500, 24001, R).astype(np.int64)
    w = make_workload("waves_sim", 11, rng, cached, suffix, 64, 8, 128, B, shared_tokens=16384, sharers=sharer)
    ctx = wpp.Context(0)
    desc = wpp.make_desc(R, w.num_q_heads, w.num_kv_heads, w.head_dim, B, w.max_blocks_per_req, w.num_pages)
    k_pool, v_pool = w.k_pool(dev), w.v_pool(dev)
    bt = torch.from_numpy(w.block_tables).to(dev)
    g = torch.Generator(device=dev).manual_seed(5)
    q = torch.randn(M, w.num_q_heads, w.head_dim, device=dev, generator=g).to(torch.bfloat16)
    kn = torch.randn(M, w.num_kv_heads, w.head_dim, device=dev, generator=g).to(torch.bfloat16)
    vn = torch.randn(M, w.num_kv_heads, w.head_dim, device=dev, generator=g).to(torch.bfloat16)
    out = torch.empty_like(q)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    ws = torch.empty(64 << 20, dtype=torch.uint8, device=dev)
    ring = 2 * P_stages

    def run_policy(b_min, n_req):
        # the first n_req requests form the burst; the planner starts from an idle system (floor budget in force)
        cfg = wpp.WaveConfig(P_stages, F, B, lanes, M, b_min)
        st = wpp.WaveState(len(wpp.wpp_wave_ladder(cfg)) - 1, 0, 0, 0)
        done = np.zeros(R, dtype=np.int64)
        done[n_req:] = suffix[n_req:]
        inflight, times, sizes, budgets = [], [], [], []
        while True:
            chunks, info = wpp.wpp_plan_waves(cfg, st, (suffix - done).tolist(), [c for wv in inflight for c in wv])
            if int(info.wave_tokens) == 0:
                break
            Pw = (cached + done).astype(np.int32)
            Cw = chunks.astype(np.int32)
            plan = wpp.wpp_plan_tiles(ctx, desc, Pw, Cw, opts=wpp.PlanOpts(0, 0, 0, 0, args.plan_order))
            plan.to_device()
            if int(plan.info.workspace_bytes) > ws.numel():
                raise SystemExit("workspace too small for the simulation")
            Pd, Cd = torch.from_numpy(Pw).to(dev), torch.from_numpy(Cw).to(dev)
            T = int(Cw.sum())
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            wpp.wpp_kv_append(ctx, desc, kn[:T], vn[:T], k_pool, v_pool, bt, Pd, Cd, plan, status=status)
            wpp.wpp_prefill_attention_varlen(ctx, desc, q[:T], out[:T], None, k_pool, v_pool, bt, Pd, Cd, plan,
                                             workspace=ws, status=status)
            b.record()
            torch.cuda.synchronize()
            times.append(a.elapsed_time(b))
            sizes.append(T)
            budgets.append(int(info.budget))
            done += chunks
            inflight = (inflight + [[int(c) for c in chunks if c]])[-ring:]
        if int(status.item()) != 0:
            raise SystemExit(f"device status {int(status.item())}")
        finish = [0.0] * P_stages                       # finish time of the latest wave on each stage
        for t in times:
            prev = 0.0
            for s_ in range(P_stages):
                start = max(finish[s_], prev)
                finish[s_] = prev = start + t
        makespan = finish[-1]
        return {"waves": len(times), "budgets_used": sorted(set(budgets), reverse=True),
                "stage_busy_ms": float(sum(times)), "makespan_ms": float(makespan),
                "fill": float(sum(times) / makespan), "tokens_per_s": float(sum(sizes) / (makespan * 1e-3)),
                "mean_wave_ms": float(np.mean(times)), "max_wave_ms": float(np.max(times))}

    run_policy(M, R)                                    # warm-up pass (allocator, tensor maps, clocks)
    bursts = {}
    for n_req in (R, 12, 4):
        bursts[f"{n_req} requests, {int(suffix[:n_req].sum())} new tokens"] = {
            "budget_fixed_at_M": run_policy(M, n_req), "budget_ladder": run_policy(1024, n_req)}
    big = next(iter(bursts.values()))
    line = {"metric": "simulated 4-stage pipeline: new tokens/s for one burst of admitted requests",
            "value": big["budget_ladder"]["tokens_per_s"], "unit": "tokens/s", "n_gpus": 1, "higher_is_better": True,
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "bursts of 40, 12 and 4 requests, 80 % sharing a 16384-token cached prefix, "
                                   "suffixes 500-24000", "P": P_stages, "F": F, "M": M, "b_min": 1024, "B": B},
            "bursts": bursts}
    print(json.dumps(line))


def run_hints(args):
    """Prefix hints (Section 4.3) at the size of the paper's stress experiment: 64 requests of 200K tokens.  The
    chained block hashes are computed on the GPU (timed with CUDA events against the measured copy bandwidth: the
    kernels read 4 bytes per token and write 8 bytes per block), the index is filled with a cached part of every
    request and probed from the host (gallop and bisect), and the answers are checked against the linear scan of the
    oracle on a sample."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import torch
    import paper_2609_35263_b200 as wpp
    from oracle import hints as O
    peaks, peak_kind = load_peaks()
    dev = torch.device("cuda", 0)
    ctx = wpp.Context(0)
    R, n_tok, B = 64, 200000, 64
    rng = np.random.default_rng(13)
    shared = rng.integers(0, 150000, 100000).astype(np.int32)                  # half of every prompt is common
    reqs = [np.concatenate([shared, rng.integers(0, 150000, n_tok - shared.size).astype(np.int32)]) for _ in range(R)]
    tok_off = (np.arange(R + 1, dtype=np.int64) * n_tok)
    blk_off = (np.arange(R + 1, dtype=np.int64) * (n_tok // B))
    tokens = torch.from_numpy(np.concatenate(reqs)).to(dev)
    to_d, bo_d = torch.from_numpy(tok_off).to(dev), torch.from_numpy(blk_off).to(dev)
    total_blocks = int(blk_off[-1])
    out = torch.empty(total_blocks, dtype=torch.int64, device=dev)
    for _ in range(max(3, args.warmup)):
        wpp.wpp_hash_blocks(ctx, tokens, to_d, bo_d, B, salt=1, total_blocks=total_blocks, out=out)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    steps = max(5, args.steps)
    torch.cuda.synchronize()
    a.record()
    for _ in range(steps):
        wpp.wpp_hash_blocks(ctx, tokens, to_d, bo_d, B, salt=1, total_blocks=total_blocks, out=out)
    b.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / steps
    hashes = out.cpu().numpy().view(np.uint64).reshape(R, n_tok // B)
    nbytes = tokens.numel() * 4 + out.numel() * 8
    idx = wpp.HintIndex()
    cached = [int(rng.integers(0, n_tok // B + 1)) for _ in range(R)]
    for i in range(R):
        idx.add(0, hashes[i, :cached[i]])
    t0 = time.perf_counter()
    res = [idx.probe(0, hashes[i]) for i in range(R)]
    t_probe = (time.perf_counter() - t0) / R
    oidx = O.HintIndex()
    for i in range(R):
        oidx.add(0, hashes[i, :cached[i]].tolist())
    for i in range(0, R, 8):                                                   # a sample against the definition
        want = O.longest_prefix_linear(oidx, 0, hashes[i].tolist())
        if res[i][0] != want or hashes[i, :4].tolist() != O.chained_hashes(reqs[i][:4 * B].tolist(), B, 1):
            raise SystemExit("hint probe or hashes disagree with the oracle")
    hbm = float(peaks.get("hbm_gbs", FALLBACK_PEAKS["hbm_gbs"]))
    line = {"metric": "chained block hashing, tokens/s (64 requests x 200K tokens)", "value": tokens.numel() / (ms * 1e-3),
            "unit": "tokens/s", "n_gpus": 1, "steps": steps, "warmup": max(3, args.warmup), "ms_per_step": ms,
            "higher_is_better": True, "vs_baseline": None, "dtype": "u64", "data": "synthetic", "gpu_launches": 2 * steps,
            "config": {"workload": "64 requests of 200,000 tokens, 64-token blocks, first 100,000 tokens common"},
            "roofline": {"bound": "hbm", "kernel": "wpp_block_digest_kernel + wpp_hash_chain_kernel",
                         "achieved": nbytes / (ms * 1e-3) / 1e9, "peak": hbm, "unit": "GB/s",
                         "frac": nbytes / (ms * 1e-3) / 1e9 / hbm, "peak_source": f"of {peak_kind} (copy bandwidth)",
                         "traffic": None},
            "probe": {"mean_us_per_request": t_probe * 1e6, "mean_index_lookups": float(np.mean([p for _, p in res])),
                      "eligible_blocks": n_tok // B, "index_keys": len(idx),
                      "how": "host, through the Python binding; gallop then bisect"}}
    print(json.dumps(line))


def run_kda(args):
    """The recurrent-state (KDA) layer of one wave (Section 3.1 update, Section 3.2 snapshots): `--kda-lanes`
    requests of `--kda-chunk` tokens, 32 state heads of 128 x 128, every request resuming from a snapshot and
    storing one at the chunk end.  Timed with CUDA events over back-to-back launches on inputs larger than L2;
    the library's choice (--kda-layout 0) is the chunk-parallel tensor-core form, bounded by the algorithmic bytes at
    HBM bandwidth; the token-by-token forms (--kda-layout 1, 2) are plain fp32 arithmetic: 7 flop per state element
    and token against 148 SMs x 128 lanes x 2 flop x the maximum SM clock."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import torch
    import paper_2609_35263_b200 as wpp
    import wpp_workloads as W
    from oracle import kda as O
    dev = torch.device("cuda", 0)
    ctx = wpp.Context(0)
    w = W.kda_wave(args.kda_lanes, args.kda_chunk)
    t = w.tensors()
    d = {k: v.to(dev) for k, v in t.items()}
    i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev)
    ro, s_in, s_out = torch.from_numpy(w.row_offsets).to(dev), i32(w.state_in), i32(w.state_out)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    out = torch.empty((w.total_tokens, w.num_heads, w.d_v), dtype=torch.bfloat16, device=dev)
    P_dev = i32(w.prefix_lens)
    ws = torch.empty(wpp.wpp_kda_workspace_bytes(int(w.chunk_lens.size), w.num_heads, w.total_tokens), dtype=torch.uint8,
                     device=dev) if args.kda_layout in (0, 3) else None
    step = lambda: wpp.wpp_kda_chunk(ctx, d["q"], d["k"], d["v"], d["alpha"], d["beta"], ro, d["state_pool"], s_in, s_out,
                                     out=out, prefix_lens=P_dev, status=status, layout=args.kda_layout, workspace=ws)
    warm, steps = max(3, args.warmup), max(1, args.steps)
    for _ in range(warm):
        step()
    torch.cuda.synchronize()
    sampler = ClockSampler(0)
    sampler.start()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(steps):
        step()
    b.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = a.elapsed_time(b) / steps
    if int(status.item()) != 0:
        raise SystemExit(f"wpp_kda_chunk reported status {int(status.item())}")
    # parity on one chain, and the oracle's own speed on it
    req, head = w.chunk_lens.size - 1, w.num_heads - 1
    sl = slice(int(w.row_offsets[req]), int(w.row_offsets[req + 1]))
    f = lambda x: x[sl, head:head + 1].double().numpy()
    pool = t["state_pool"][:, head:head + 1].double().numpy().copy()
    t0 = time.perf_counter()
    ref = O.kda_chunk(f(t["q"]), f(t["k"]), f(t["v"]), f(t["alpha"]), f(t["beta"]), [sl.stop - sl.start], pool,
                      w.state_in[req:req + 1], w.state_out[req:req + 1])
    t_cpu = time.perf_counter() - t0
    got = out[sl, head:head + 1].float().cpu().double().numpy()
    err = float(np.abs(got - ref).max())
    if not np.all(np.abs(got - ref) <= 2.0 ** -8 * np.abs(ref) + 1e-4 * np.abs(ref).max()):
        raise SystemExit(f"wpp_kda_chunk disagrees with the oracle (max |delta| {err:.3e})")
    T, Hh = w.total_tokens, w.num_heads
    flops = 7.0 * w.d_k * w.d_v * T * Hh             # the method's work: 7 flop per state element, token and head
    nbytes = T * Hh * (2 * w.d_k * 2 + 2 * w.d_v * 2 + 4 * w.d_k + 4) + 2 * w.chunk_lens.size * Hh * w.d_k * w.d_v * 4
    peaks, peak_kind = load_peaks()
    hbm = float(peaks.get("hbm_gbs", FALLBACK_PEAKS["hbm_gbs"]))
    tensor_form = args.kda_layout == 3 or (args.kda_layout == 0 and T >= 64 * int(w.chunk_lens.size))
    if tensor_form:
        # Chunk-parallel form: the algorithmic bytes (q, k, v, alpha, beta in, outputs and states out) at the copy
        # bandwidth bound it from below (7 d_k d_v flop per token and head are 0.04 ms of tensor time for the default
        # wave, the bytes 0.13 ms); what it actually moves is three times that, because the preparation kernel hands
        # its per-block operands to the chain kernel through the workspace.
        roofline = {"bound": "hbm", "kernel": "kda_tc_prep_kernel + kda_tc_chain_kernel",
                    "achieved": nbytes / (ms * 1e-3) / 1e9, "peak": hbm, "unit": "GB/s",
                    "frac": nbytes / (ms * 1e-3) / 1e9 / hbm, "peak_source": f"of {peak_kind} (copy bandwidth)",
                    "algorithmic_bytes": nbytes, "flop_per_token_head": 7 * w.d_k * w.d_v,
                    "tflops_algorithmic": flops / (ms * 1e-3) / 1e12,
                    "traffic": KDA_TC_DRAM_BYTES_PER_TOKEN_HEAD * T * Hh,
                    "traffic_source": "estimate: dram read + write bytes of one preparation and one chain launch on the "
                                      "8 x 2,048-token wave (ncu), per (token, head), x this wave's pairs; not measured "
                                      "in this run"}
    else:
        peak = 148 * 128 * 2 * 1965e6 / 1e12
        roofline = {"bound": "alu", "kernel": "wpp_kda_chunk_kernel", "achieved": flops / (ms * 1e-3) / 1e12,
                    "peak": peak, "unit": "TFLOP/s", "frac": flops / (ms * 1e-3) / 1e12 / peak,
                    "peak_source": "derived: 148 SMs x 128 fp32 lanes x 2 flop x 1965 MHz",
                    "flop_per_token_head": 7 * w.d_k * w.d_v, "traffic": KDA_DRAM_BYTES_PER_TOKEN_HEAD * T * Hh,
                    "traffic_source": "estimate from an ncu capture of the default wave, scaled by (token, head) pairs",
                    "hbm_gbs_algorithmic": nbytes / (ms * 1e-3) / 1e9}
    line = {"metric": "recurrent-state (KDA) layer, new tokens/s through one layer", "value": T / (ms * 1e-3),
            "unit": "tokens/s", "n_gpus": 1, "steps": steps, "warmup": warm, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16 x 2 terms, fp32 accumulate" if tensor_form else "f32",
            "data": "synthetic", "gpu_launches": steps * (3 if tensor_form else 1),
            "config": {"workload": w.name, "requests": int(w.chunk_lens.size), "chunk": int(w.chunk_lens[0]),
                       "state_heads": Hh, "d_k": w.d_k, "d_v": w.d_v, "layout": args.kda_layout,
                       "form": "chunk-parallel on tensor cores" if tensor_form else "token by token on CUDA cores",
                       "l2": "inputs larger than L2"},
            "clocks": clocks, "roofline": roofline,
            "cpu_baseline": {"value": (sl.stop - sl.start) / t_cpu / Hh, "unit": "tokens/s", "cores": 1, "kind": "oracle",
                             "sample": f"one (request, head) chain of {sl.stop - sl.start} tokens, scaled to {Hh} heads"},
            "parity": {"checked": f"request {req}, head {head}: all outputs against the fp64 oracle", "max_abs_err": err}}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", default="cfg3")
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-yardsticks", action="store_true", help="skip the in-run matmul and copy timings")
    ap.add_argument("--rescale-mode", type=int, default=2, choices=[0, 1, 2],
                    help="where a moved row reference rescales the accumulator: 0 before the exponentials (the "
                         "library's default), 1 after them, 2 the library chooses from what its kernels counted")
    ap.add_argument("--no-other-configs", action="store_true",
                    help="skip the short runs of further workloads reported under other_configs")
    ap.add_argument("--force-kv-splits", type=int, default=0)
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    ap.add_argument("--plan-order", type=int, default=0, help="0: stream order (default), 1: longest tile first")
    ap.add_argument("--max-ctas", type=int, default=0, help="persistent CTAs to launch (0: one per SM)")
    ap.add_argument("--shape", type=int, default=0, help="attention kernel: 0 planner's choice, 1 SM-wide two-half CTAs, "
                                                         "2 small single-half CTAs (two per SM)")
    ap.add_argument("--waves", action="store_true", help="time the wave-budget planner (host only) instead")
    ap.add_argument("--waves-sim", action="store_true", help="wave planner + kernels: simulated pipeline fill")
    ap.add_argument("--hints", action="store_true", help="chained block hashing on the GPU and the hint probe")
    ap.add_argument("--kda", action="store_true", help="the recurrent-state (KDA) layer of one wave")
    ap.add_argument("--kda-lanes", type=int, default=8)
    ap.add_argument("--kda-chunk", type=int, default=2048)
    ap.add_argument("--kda-layout", type=int, default=0, help="0: library chooses, 1: one CTA per (request, head), 2: four, 3: chunk-parallel on tensor cores")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "native" else args.warmup

    if args.waves:
        run_waves(args)
        return
    if args.waves_sim:
        run_waves_sim(args)
        return
    if args.hints:
        run_hints(args)
        return
    if args.kda:
        run_kda(args)
        return
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import paper_2609_35263_b200 as wpp
    from paper_2609_35263_b200 import replicas

    rank, local_rank, world = replicas.env_ranks()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback for the product path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    replicas.init("nccl", dev)

    peaks, peak_kind = load_peaks()
    w = build_workload(args.config)
    ctx = wpp.Context(local_rank)
    ctx.set_rescale_mode(args.rescale_mode)
    desc = wpp.make_desc(w.num_requests, w.num_q_heads, w.num_kv_heads, w.head_dim, w.page_size,
                         w.max_blocks_per_req, w.num_pages)
    opts = wpp.PlanOpts(0, 0, args.force_kv_splits, args.max_ctas, args.plan_order, args.shape)
    T = w.total_new_tokens

    # ---- resident state and inputs on the device
    q, k_new, v_new = w.q(dev), w.k_new(dev), w.v_new(dev)
    k_pool, v_pool = w.k_pool(dev), w.v_pool(dev)
    bt_h = torch.from_numpy(w.block_tables).pin_memory()
    P_h = torch.from_numpy(w.prefix_lens).pin_memory()
    C_h = torch.from_numpy(w.chunk_lens).pin_memory()
    bt, P, C = bt_h.to(dev), P_h.to(dev), C_h.to(dev)
    out = torch.empty(T, w.num_q_heads, w.head_dim, dtype=torch.bfloat16, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)

    plan_bytes = wpp.wpp_plan_tiles(ctx, desc, w.prefix_lens, w.chunk_lens, opts=opts).info
    ring = 3
    plan_host = [torch.empty(int(plan_bytes.plan_bytes) + 4096, dtype=torch.uint8).pin_memory() for _ in range(ring)]
    plan_dev = [torch.empty(int(plan_bytes.plan_bytes) + 4096, dtype=torch.uint8, device=dev) for _ in range(ring)]
    plan_free = [torch.cuda.Event() for _ in range(ring)]
    ws = torch.empty(max(256, int(plan_bytes.workspace_bytes)), dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()

    # Inputs smaller than twice the 126 MB L2 would stay cached from one timed step to the next: such workloads get
    # the L2 flushed between steps (a 256 MB buffer is overwritten), and the step time is then the sum of the
    # steps' own event times, not the bracket around the loop, so that the flush is not counted.
    touched = (2 * T * w.num_q_heads * w.head_dim * 2 +
               w.unique_kv_pages() * w.num_kv_heads * w.page_size * w.head_dim * 2 * 2)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if touched < 2 * (126 << 20) else None

    def one_step(i, attn_events=None, qd=q, knd=k_new, vnd=v_new, btd=bt, Pd=P, Cd=C):
        s = i % ring
        if flush is not None:
            flush.fill_(i & 0xFF)
        plan_free[s].synchronize()                       # the copy that last used this buffer has run
        t_plan = time.perf_counter()
        plan = wpp.wpp_plan_tiles(ctx, desc, w.prefix_lens, w.chunk_lens, opts=opts, out=plan_host[s])
        t_plan = time.perf_counter() - t_plan
        plan.to_device(out=plan_dev[s])
        plan_free[s].record(stream)
        if attn_events is not None:
            a0, a, b = (torch.cuda.Event(enable_timing=True) for _ in range(3))
            a0.record(stream)
        wpp.wpp_kv_append(ctx, desc, knd, vnd, k_pool, v_pool, btd, Pd, Cd, plan, status=status)
        if attn_events is not None:
            a.record(stream)
        wpp.wpp_prefill_attention_varlen(ctx, desc, qd, out, None, k_pool, v_pool, btd, Pd, Cd, plan,
                                         workspace=ws, status=status)
        if attn_events is not None:
            b.record(stream)
            attn_events.append((a, b, a0, t_plan))
        return plan

    barrier = replicas.barrier

    def max_over_ranks(x):
        return replicas.max_over_ranks(x, dev)

    # ---- device-resident timing
    for i in range(args.warmup):
        plan = one_step(i)
    barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    launches0 = ctx.launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    attn_events = []
    ev0.record(stream)
    for i in range(args.steps):
        plan = one_step(args.warmup + i, attn_events)
    ev1.record(stream)
    barrier()
    launches = ctx.launch_count() - launches0
    clocks = sampler.stop()
    ms_step = ev0.elapsed_time(ev1) / args.steps
    if flush is not None:
        ms_step = statistics.mean(a0.elapsed_time(b) for _, b, a0, _ in attn_events)
    ms_step = max_over_ranks(ms_step)
    attn_ms = statistics.mean(a.elapsed_time(b) for a, b, _, _ in attn_events)
    phases = {"plan_host_ms": 1e3 * statistics.median(t for _, _, _, t in attn_events),
              "plan_host_ms_max": 1e3 * max(t for _, _, _, t in attn_events),
              "append_ms": statistics.mean(a0.elapsed_time(a) for a, _, a0, _ in attn_events),
              "attention_ms": attn_ms,
              "note": "the host plans the next wave while the GPU runs the current one; append and attention are "
                      "CUDA-event times on the launching stream"}
    if int(status.item()) != 0:
        raise SystemExit(f"device status {int(status.item())} after the timed region")
    info = plan.info
    flops = float(info.flops)
    tokens_per_s = world * T / (ms_step * 1e-3)
    r_steps, r_moves, r_late = ctx.rescale_stats()
    rescale_note = {"mode": ["before the exponentials", "after the exponentials", "chosen from the kernels' counters"][args.rescale_mode],
                    "in_use": "after" if r_late else "before",
                    "share_of_key_steps_that_rescaled": (r_moves / r_steps) if r_steps else None}

    roof_peak = float(peaks.get("bf16_tflops", FALLBACK_PEAKS["bf16_tflops"]))
    roof_sus = float(peaks.get("bf16_tflops_sustained", FALLBACK_PEAKS["bf16_tflops_sustained"]))
    achieved = flops / (attn_ms * 1e-3) / 1e12
    # the bound is the slower of FLOPs at the tensor peak and compulsory bytes at HBM bandwidth
    t_flops, t_bytes, kv_bytes, qo_bytes = roofline_times(w, flops, peaks)
    traffic = DRAM_BYTES_PER_KEY_STEP * float(info.key_steps)
    roofline = {"bound": "tensor" if t_flops >= t_bytes else "hbm", "kernel": "wpp_attn_kernel",
                "achieved": achieved, "peak": roof_peak, "unit": "TFLOP/s", "frac": achieved / roof_peak,
                "peak_source": f"of {peak_kind} (burst bf16 matmul)", "frac_of_sustained": achieved / roof_sus,
                "traffic": traffic, "traffic_source": DRAM_SOURCE, "compulsory_bytes": kv_bytes + qo_bytes,
                "flops_per_launch": flops, "kernel_ms": attn_ms,
                "roofline_ms": max(t_flops, t_bytes), "frac_of_roofline_time": max(t_flops, t_bytes) / attn_ms}

    roofline["frac_of_nominal"] = achieved / NOMINAL_BF16_TFLOPS
    if not args.no_yardsticks:
        roofline["yardsticks_this_run"] = measure_yardsticks(dev)

    # the append alone, back to back (the per-step bracket above includes the gap to the previous kernel)
    n_app = 20
    a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a0.record(stream)
    for _ in range(n_app):
        wpp.wpp_kv_append(ctx, desc, k_new, v_new, k_pool, v_pool, bt, P, C, plan, status=status)
    a1.record(stream)
    a1.synchronize()
    app_ms = a0.elapsed_time(a1) / n_app
    app_bytes = 2 * 2 * T * w.num_kv_heads * w.head_dim * 2           # K and V, read and written
    hbm = float(peaks.get("hbm_gbs", FALLBACK_PEAKS["hbm_gbs"]))
    phases["append_back_to_back"] = {"launches": n_app, "ms": app_ms, "gb_per_s": app_bytes / (app_ms * 1e-3) / 1e9,
                                     "frac_of_hbm_copy_peak": app_bytes / (app_ms * 1e-3) / 1e9 / hbm}

    # ---- end to end through host buffers
    e2e = None
    if not args.no_e2e:
        # Host buffers in, host buffer out, every step: q / k_new / v_new / block tables / lengths come from pinned
        # host memory and `out` goes back to pinned host memory.  The C ABI takes the stream to work on, so a
        # caller pipelines the three phases on three streams with two sets of device buffers: while wave i runs,
        # wave i+1's inputs are on their way in and wave i-1's output on its way out.
        hb = dict(q=q, k_new=k_new, v_new=v_new)
        host_in = {k: torch.empty(v.shape, dtype=v.dtype).pin_memory() for k, v in hb.items()}
        for k in hb:
            host_in[k].copy_(hb[k])
        out_h = [torch.empty(out.shape, dtype=out.dtype).pin_memory() for _ in range(2)]
        dev_in = [{k: torch.empty_like(v) for k, v in hb.items()} for _ in range(2)]
        dev_meta = [(torch.empty_like(bt), torch.empty_like(P), torch.empty_like(C)) for _ in range(2)]
        dev_out = [out, torch.empty_like(out)]
        h2d = sum(x.numel() * x.element_size() for x in list(host_in.values()) + [bt_h, P_h, C_h]) + int(info.plan_bytes)
        d2h = out.numel() * out.element_size()
        s_in, s_run, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
        in_done = [torch.cuda.Event() for _ in range(2)]
        run_done = [torch.cuda.Event() for _ in range(2)]
        out_done = [torch.cuda.Event() for _ in range(2)]

        def e2e_step(i):
            b2 = i % 2
            sl = i % ring
            # the plan is an input like the others: it is made first and travels on the input stream, ahead of the
            # large copies (a small copy issued later from the compute stream would queue behind the next wave's
            # 4.5 GB query copy on the one host-to-device engine and stall the kernels for 100 ms)
            plan_free[sl].synchronize()                  # the copy that last read this pinned buffer has run
            plan = wpp.wpp_plan_tiles(ctx, desc, w.prefix_lens, w.chunk_lens, opts=opts, out=plan_host[sl])
            with torch.cuda.stream(s_in):
                s_in.wait_event(run_done[b2])            # wave i-2 (and so wave i-3, which used this plan buffer) is done
                plan.to_device(out=plan_dev[sl])
                plan_free[sl].record(s_in)
                for k in hb:
                    dev_in[b2][k].copy_(host_in[k], non_blocking=True)
                for dst, src in zip(dev_meta[b2], (bt_h, P_h, C_h)):
                    dst.copy_(src, non_blocking=True)
                in_done[b2].record(s_in)
            with torch.cuda.stream(s_run):
                s_run.wait_event(in_done[b2])
                s_run.wait_event(out_done[b2])           # wave i-2's output has left this output buffer
                btd, Pd, Cd = dev_meta[b2]
                wpp.wpp_kv_append(ctx, desc, dev_in[b2]["k_new"], dev_in[b2]["v_new"], k_pool, v_pool, btd, Pd, Cd,
                                  plan, status=status, stream=s_run)
                wpp.wpp_prefill_attention_varlen(ctx, desc, dev_in[b2]["q"], dev_out[b2], None, k_pool, v_pool, btd,
                                                 Pd, Cd, plan, workspace=ws, status=status, stream=s_run)
                run_done[b2].record(s_run)
            with torch.cuda.stream(s_out):
                s_out.wait_event(run_done[b2])
                out_h[b2].copy_(dev_out[b2], non_blocking=True)
                out_done[b2].record(s_out)

        # Two waves fill the pipeline; the timed region then runs from the moment wave 1's output has reached the
        # host to the moment the last wave's output has: K waves leave the pipeline in it, each with its own
        # H2D copy, library calls and D2H copy (throughput of the full pipeline).  "cold" is the same run
        # measured from an idle device, fill and drain included.
        e2e_steps = max(4, min(args.steps, 8))
        torch.cuda.synchronize()
        barrier()
        c0, e0, e1 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        c0.record(s_in)
        for i in range(2):
            e2e_step(i)
        e0.record(s_out)
        for i in range(e2e_steps):
            e2e_step(2 + i)
        e1.record(s_out)
        s_out.synchronize()
        s_run.synchronize()
        s_in.synchronize()
        barrier()
        e2e_ms = max_over_ranks(e0.elapsed_time(e1) / e2e_steps)
        cold_ms = max_over_ranks(c0.elapsed_time(e1) / (e2e_steps + 2))
        if int(status.item()) != 0:
            raise SystemExit(f"device status {int(status.item())} after the end-to-end region")
        e2e = {"value": world * T / (e2e_ms * 1e-3), "unit": "tokens/s", "h2d_bytes_per_step": int(h2d),
               "d2h_bytes_per_step": int(d2h), "ms_per_step": e2e_ms, "steps": e2e_steps,
               "cold": {"ms_per_step": cold_ms, "steps": e2e_steps + 2,
                        "value": world * T / (cold_ms * 1e-3)},
               "how": "pinned host buffers; H2D, the C-ABI calls and D2H on three streams, two device buffer sets; "
                      "timed from wave 1's output on the host to the last wave's output on the host"}
        del host_in, out_h, dev_in, dev_out

    del q, k_new, v_new, k_pool, v_pool, out
    if not args.no_e2e:
        del hb
    torch.cuda.empty_cache()
    others = None
    if rank == 0 and world == 1 and not args.no_other_configs and args.config == "cfg3":
        others = []
        for name in OTHER_CONFIGS:
            others.append(measure_other_config(name, ctx, dev, peaks))
            torch.cuda.empty_cache()
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = OracleSampler(w, True).sample(args.cpu_seconds)

    if rank == 0:
        line = {
            "metric": METRIC, "value": tokens_per_s, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": dict(describe_config(w, world),
                           l2=(f"inputs larger than L2: Q+O {qo_bytes / 1e9:.2f} GB + unique KV {kv_bytes / 1e9:.2f} GB "
                              "touched per step vs 126 MB of L2; no explicit flush" if flush is None else
                              f"inputs ({touched / 1e6:.1f} MB touched per step) fit L2: a 256 MB buffer is overwritten "
                              "between steps; ms_per_step is the sum of append and attention event times"),
                           step="wpp_plan_tiles + plan H2D + wpp_kv_append + wpp_prefill_attention_varlen",
                           tiles=int(info.num_tiles), ctas=int(info.num_ctas), key_steps=int(info.key_steps),
                           kernel_shape=int(info.shape), rescale=rescale_note),
            "tflops": flops / (ms_step * 1e-3) / 1e12 * world,
            "served_tokens_per_s": world * float((w.prefix_lens.astype(np.int64) + w.chunk_lens).sum()) / (ms_step * 1e-3),
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline, "cpu_baseline": cpu,
            "phases": phases, "other_configs": others,
        }
        print(json.dumps(line))
    replicas.finalize()


if __name__ == "__main__":
    main()
