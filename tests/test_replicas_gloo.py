"""The N > 1 path on CPU: two gloo ranks meet at the barrier and agree on max-over-ranks timing."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import torch
    from paper_2609_35263_b200 import replicas
    import paper_2609_35263_b200 as wpp
    import wpp_workloads as W
    rank, local_rank, world = replicas.init(backend="gloo")
    assert world == 2 and torch.distributed.get_backend() == "gloo"
    # every replica plans the same wave on the host: identical plans, no exchange needed
    w = W.cfg1()
    d = wpp.make_desc(w.num_requests, w.num_q_heads, w.num_kv_heads, w.head_dim, w.page_size,
                      w.max_blocks_per_req, w.num_pages)
    plan = wpp.wpp_plan_tiles(None, d, w.prefix_lens, w.chunk_lens, pin=False)
    digest = float(sum(plan.host_bytes()) %% 1000003)
    assert replicas.max_over_ranks(digest) == digest == -replicas.max_over_ranks(-digest)
    replicas.barrier(sync_cuda=False)
    local_ms = 10.0 + 5.0 * rank                  # rank 1 is the slow one
    value, ms = replicas.aggregate_throughput(w.total_new_tokens, local_ms)
    replicas.barrier(sync_cuda=False)
    if rank == 0:
        print(json.dumps({"value": value, "ms": ms, "world": world}))
    replicas.finalize()
""") % ROOT


def test_two_gloo_ranks_report_max_time_and_aggregate_tokens(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29533", WORLD_SIZE="2", OMP_NUM_THREADS="1")
    procs = [subprocess.Popen([sys.executable, str(script)], env=dict(env, RANK=str(r), LOCAL_RANK=str(r)),
                              stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True) for r in range(2)]
    outs = [p.communicate(timeout=180) for p in procs]
    assert all(p.returncode == 0 for p in procs), [o[1][-2000:] for o in outs]
    import json
    line = json.loads(outs[0][0].strip().splitlines()[-1])
    assert line["world"] == 2 and line["ms"] == 15.0
    assert abs(line["value"] - 2 * 128 / 15e-3) < 1e-6
