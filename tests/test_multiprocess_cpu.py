"""The N > 1 path of the benchmark on CPU (gloo, world size 2): every rank draws its own sequences
(the path has no cross-sequence exchange, so ranks are replicas over different data), the job's time
is the max over ranks, and only rank 0 runs the CPU reference arm."""
import os
import socket
import subprocess
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r'''
import os, sys, json
import numpy as np
sys.path.insert(0, os.environ["RADAR_ROOT"])
import torch, torch.distributed as dist
import bench
from paper_2512_14069_b200 import workloads as W
rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo")
cfg = W.CONFIGS[1]
inp = bench.host_inputs(cfg, rank)
# rank r holds sequences r * B .. r * B + B - 1 of the configuration's generator
want = np.stack([W.draft_logits(W.shrink(cfg, B=cfg.B * world), rank * cfg.B + b) for b in range(cfg.B)])
ok_data = bool(np.array_equal(inp["draft"], want))
first = torch.tensor(inp["draft"][0, 0, :8].astype(np.float64))
got = [torch.zeros_like(first) for _ in range(world)]
dist.all_gather(got, first)
distinct = not bool(torch.equal(got[0], got[1]))
times = bench.reduce_max([10.0 + rank, 1.0 - 0.25 * rank], torch.device("cpu"))
value = bench.whole_job_value(world, 100, times[0])
print(json.dumps({"rank": rank, "ok_data": ok_data, "distinct": distinct, "times": times, "value": value}))
dist.destroy_process_group()
'''


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_ranks_shard_sequences_and_take_the_max_time():
    import json
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), RADAR_ROOT=ROOT)
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=300)
        assert p.returncode == 0, err[-2000:]
        outs.append(json.loads(out.strip().splitlines()[-1]))
    for o in outs:
        assert o["ok_data"] and o["distinct"]
        assert o["times"] == [11.0, 1.0]                       # the slowest rank, on every rank
        assert abs(o["value"] - 2 * 100 * 1000.0 / 11.0) < 1e-9


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1", MASTER_ADDR="127.0.0.1", MASTER_PORT="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0", "--config", "1"], env=env, capture_output=True, text=True,
                       timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
