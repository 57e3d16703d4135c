"""The N > 1 mode of bench.py is "replicas": one independent batch per rank, no collective on the data
path.  Its host-side logic (per-rank batches, max-over-ranks timing, whole-job throughput, the reference
arm running on rank 0 only) is checked here with two gloo ranks on CPU."""
import json
import os
import subprocess
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, os.environ["HA_ROOT"])
import torch, torch.distributed as dist
import bench
from paper_2609_32114_b200 import synth
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
w = synth.shrink(synth.WORKLOADS["gdn_layer_4k"], seq_lens=[96], hk=1, hv=1)
inp = synth.make_inputs(w, seed=bench.rank_seed(rank))
local_ms = 10.0 + 5.0 * rank                      # pretend rank 1 is slower
ms = bench.max_over_ranks(dist, local_ms, torch.device("cpu"))
val = bench.job_throughput(world, inp["T"], ms)
chk = torch.tensor([float(inp["q"].sum())], dtype=torch.float64)
gathered = [torch.zeros_like(chk) for _ in range(world)]
dist.all_gather(gathered, chk)
if rank == 0:
    print(json.dumps({"ms": ms, "value": val, "sums": [float(g.item()) for g in gathered]}))
dist.destroy_process_group()
"""


def test_two_gloo_ranks_replica_logic(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, HA_ROOT=ROOT, MASTER_ADDR="127.0.0.1", MASTER_PORT="29533", WORLD_SIZE="2")
    procs = []
    for r in range(2):
        e = dict(env, RANK=str(r), LOCAL_RANK=str(r))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=e, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=120) for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    d = json.loads(outs[0][0].strip().splitlines()[-1])
    assert d["ms"] == 15.0                                   # the slowest rank sets the step time
    assert np.isclose(d["value"], 2 * 96 / 0.015)            # whole-job tokens over that time
    assert d["sums"][0] != d["sums"][1]                      # the two ranks drew different batches


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT="29534")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""      # other ranks exit 0 without work
