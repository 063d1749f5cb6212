"""The stage hand-off on CPU: three gloo ranks (first, middle and last stage).  Stage 0 plans waves and sends spans
and activations; the middle stage receives them one wave ahead of its compute (header and activations are both
posted before the current wave is processed), checks every span against what it has materialised itself (Section
4.6), transforms the activations and forwards the wave; the last stage does the same checks.  A span that does not
start where a stage's cache ends fails that wave on that stage."""
import json
import os
import subprocess
import sys
import textwrap

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import torch
    import torch.distributed as dist
    import paper_2609_35263_b200 as wpp
    from paper_2609_35263_b200 import replicas
    from paper_2609_35263_b200.stages import StageLink, check_spans

    rank, _, world = replicas.init(backend="gloo")
    HID, LANES, M = 32, 4, 2048
    link = StageLink(rank, world, HID, LANES, M, dtype=torch.bfloat16)
    acts = lambda wave, n, stage: ((torch.arange(n * HID, dtype=torch.float32).reshape(n, HID) %% 251 + wave) %% 61
                                   + stage).to(torch.bfloat16)
    STOP = -1
    if rank == 0:
        cfg = wpp.WaveConfig(world, 2, 64, LANES, M, 256)
        st = wpp.WaveState()
        remaining, done, wave = [5000, 300, 3000], [0, 0, 0], 0
        while sum(remaining):
            chunks, info = wpp.wpp_plan_waves(cfg, st, remaining, [])
            spans = [(i, done[i], int(c)) for i, c in enumerate(chunks) if c]
            link.send_wave(wave, spans, acts(wave, int(info.wave_tokens), 0))
            for i, c in enumerate(chunks):
                remaining[i] -= int(c); done[i] += int(c)
            wave += 1
        link.send_wave(wave, [], acts(wave, 0, 0))                              # an empty wave is legal
        link.send_wave(wave + 1, [(0, done[0] + 1, 10)], acts(wave + 1, 10, 0))    # starts one token too far
        link.flush()
        print(json.dumps({"waves": wave}))
    else:
        cached, waves, tokens, failed, posted_ahead = {}, 0, 0, None, 0
        link.post_recv()
        while True:
            wave_id, spans, a = link.recv_wave()
            if wave_id == STOP:
                break
            link.post_recv()                          # header AND activations of the next wave travel from here on
            posted_ahead += int(link._posted is not None and len(link._posted) == 3)
            try:
                check_spans(spans, cached)
            except wpp.WppError as e:
                failed = (wave_id, e.status)
                if link.next is not None:
                    link.send_wave(STOP, [], a[:0])   # the wave failed here: the later stages are told to stop
                break
            assert wave_id == waves and torch.equal(a, acts(wave_id, a.shape[0], rank - 1))
            if link.next is not None:
                link.send_wave(wave_id, spans, a + 1)                           # this stage's "layers"
            waves += 1; tokens += a.shape[0]
        if link.next is not None:
            link.flush()
        print(json.dumps({"waves": waves, "tokens": tokens, "failed": failed, "cached": cached,
                          "posted_ahead": posted_ahead}))
    dist.barrier()
    os._exit(0)        # receives may still be posted: leave without waiting for them
""") % ROOT


def test_three_stages_hand_waves_over_and_reject_a_wrong_span(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29547", WORLD_SIZE="3", OMP_NUM_THREADS="1")
    procs = [subprocess.Popen([sys.executable, str(script)], env=dict(env, RANK=str(r), LOCAL_RANK=str(r)),
                              stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True) for r in range(3)]
    outs = [p.communicate(timeout=180) for p in procs]
    assert all(p.returncode == 0 for p in procs), [o[1][-2000:] for o in outs]
    sent = json.loads(outs[0][0].strip().splitlines()[-1])
    mid = json.loads(outs[1][0].strip().splitlines()[-1])
    last = json.loads(outs[2][0].strip().splitlines()[-1])
    for got in (mid, last):
        assert got["waves"] == sent["waves"] + 1 and got["tokens"] == 8300      # every wave and the empty one
        assert got["cached"] == {"0": 5000, "1": 300, "2": 3000}
        assert got["posted_ahead"] >= got["waves"]           # both receives of wave w+1 were posted before wave w ran
    assert mid["failed"] == [sent["waves"] + 1, 4]                              # WPP_ERR_POSITION_MISMATCH
    assert last["failed"] is None                                              # it was told to stop instead


def test_check_spans_without_a_process_group():
    import paper_2609_35263_b200 as wpp
    from paper_2609_35263_b200.stages import check_spans
    cached = {7: 128}
    check_spans([(7, 128, 64), (9, 0, 10)], cached)
    assert cached == {7: 192, 9: 10}
    with pytest.raises(wpp.WppError) as e:
        check_spans([(9, 10, 5), (7, 191, 1)], cached)
    assert e.value.status == 4 and cached == {7: 192, 9: 10}                    # a failed wave advances nothing
