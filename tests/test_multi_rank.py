"""The multi-GPU form of the benchmark is "replicas only": every rank decodes its own sequences
with its own copy of the weights and nothing crosses ranks on the data path.  What ranks do share
is checked here with two gloo ranks on the CPU: each rank derives different prompts and interleave
phases from its rank, the job's time is the slowest rank's, and throughput adds up."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import json, os, sys
    sys.path.insert(0, %r)
    import torch.distributed as dist
    import bench
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo")
    wl, dims, prompts, phi, off = bench.workload_setup("cfg3_step_b64", rank)
    ms_local = 10.0 + 5.0 * rank                       # rank 1 is the slow one
    ms = bench.max_over_ranks(ms_local, world, "cpu")
    tok = wl["batch"] * 5
    out = {"rank": rank, "ms": ms, "value": bench.job_tokens_per_s(tok, ms, world),
           "first_prompt": [int(x) for x in prompts[0][:8]], "phi": [int(x) for x in phi[:8]],
           "lens": [len(p) for p in prompts[:8]]}
    print("RESULT " + json.dumps(out), flush=True)
    dist.destroy_process_group()
""") % ROOT


def test_two_ranks_share_only_the_clock(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29613", WORLD_SIZE="2")
    procs = [subprocess.Popen([sys.executable, str(script)], env=dict(env, RANK=str(r)), stdout=subprocess.PIPE,
                              stderr=subprocess.PIPE, text=True) for r in range(2)]
    outs = []
    for p in procs:
        so, se = p.communicate(timeout=240)
        assert p.returncode == 0, se[-2000:]
        line = [l for l in so.splitlines() if l.startswith("RESULT ")][0]
        import json
        outs.append(json.loads(line[7:]))
    outs.sort(key=lambda o: o["rank"])
    assert outs[0]["ms"] == outs[1]["ms"] == 15.0                 # the slowest rank's time
    assert outs[0]["value"] == outs[1]["value"] == 2 * 64 * 5 / 0.015
    assert outs[0]["first_prompt"] != outs[1]["first_prompt"]     # each rank has its own sequences
    assert outs[0]["phi"] != outs[1]["phi"] or outs[0]["lens"] != outs[1]["lens"]
