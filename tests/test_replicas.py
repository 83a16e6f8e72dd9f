"""The N > 1 logic of the benchmark (independent replicas, max-over-ranks timing) on CPU with gloo, world size 2."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r'''
import json, os, sys
sys.path.insert(0, os.environ["TL_ROOT"])
import torch
import torch.distributed as dist
import bench
rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo")
dist.barrier()
ms = bench.max_over_ranks(10.0 + 5.0 * rank, torch.device("cpu"), world)        # rank 1 is the slower replica
value = bench.whole_job_value(world, 4, 10 ** 9, ms)
dist.barrier()
if rank == 0:
    print(json.dumps({"ms": ms, "value": value}), flush=True)
dist.destroy_process_group()
'''


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_replicas_report_the_slowest_rank_and_the_sum_of_their_work():
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), TL_ROOT=ROOT)
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE,
                                      text=True))
    outs = [p.communicate(timeout=180) for p in procs]
    assert all(p.returncode == 0 for p in procs), [o[1][-2000:] for o in outs]
    assert outs[1][0].strip() == ""                                   # only rank 0 prints
    line = json.loads(outs[0][0].strip().splitlines()[-1])
    assert line["ms"] == 15.0                                         # the maximum over ranks, not rank 0's 10 ms
    assert abs(line["value"] - 2 * 4 * 1e9 / 15e-3 / 1e12) < 1e-12    # both replicas' bytes over the slowest time


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(_free_port()))
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
