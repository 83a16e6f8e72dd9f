"""Sharded GEMM on the GPU: every rank's launch goes through the C ABI on its own slice; the ranks are run one after
another on cuda:0 (independent launches, nothing waits on a peer) and their results are combined the way the exchange
step combines them.  Integer-valued inputs make every partial sum exact, so the comparison is bit for bit."""
import os
import socket
import subprocess
import sys

import numpy as np
import pytest
import torch

import oracle as tlo
from paper_2607_04031_b200 import inputs, shard

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _oracle_rows(A, W_rowmajor, M, N, K):
    return tlo.matmul(inputs.bits(A), inputs.bits(W_rowmajor), tlo.ROW_MAJOR, 0, 0, M, N, K)[0]


@pytest.mark.parametrize("mode", ["n", "k"])
@pytest.mark.parametrize("world", [2, 3])
@pytest.mark.parametrize("blk", [(16, 128), (64, 32), (0, 0)])
@pytest.mark.parametrize("M", [3, 200])
def test_ranks_run_serially_reproduce_the_unsharded_product(mode, world, blk, M):
    br, bc = blk
    N, K, G = 1280, 1152, 4096
    A = inputs.bf16_integers((M, K), -4, 4, seed=11)
    W = inputs.bf16_integers((K, N), -3, 3, seed=12)
    want = _oracle_rows(A, W, M, N, K)
    shards = shard.plan(mode, N, K, br, bc, world)
    parts = []
    for s in shards:
        Wl = shard.ShardedWeight(shard.local_weight(W, s).to(DEV), s, G, br, bc)
        parts.append(shard.gemm_local(shard.local_activations(A, s).to(DEV), Wl))
    torch.cuda.synchronize()
    if mode == "n":
        assert [p.shape[1] for p in parts] == [s.n1 - s.n0 for s in shards]
        C = torch.cat(parts, dim=1)
    else:
        C = torch.stack(parts).sum(dim=0)
    assert np.array_equal(C.cpu().numpy().astype(np.float64), want)


@pytest.mark.parametrize("world", [2, 4])
def test_expert_shards_run_serially_reproduce_the_grouped_product(world):
    E, K, N, br, bc, G = 6, 256, 512, 16, 128, 4096
    offsets, counts, _ = inputs.zipf_topk_routing(50, E, 2, 1.1, seed=5)
    rows = int(offsets[-1])
    X = inputs.bf16_integers((rows, K), -4, 4, seed=21)
    WE = inputs.bf16_integers((E, K, N), -3, 3, seed=22)
    want = np.concatenate([_oracle_rows(X[int(offsets[e]):int(offsets[e + 1])], WE[e],
                                        int(offsets[e + 1] - offsets[e]), N, K) for e in range(E) if counts[e]])
    full = torch.zeros((rows, N), dtype=torch.float32, device=DEV)
    for s in shard.plan("expert", N, K, br, bc, world, E):
        Wl = shard.ShardedWeight(shard.local_weight(WE, s).to(DEV), s, G, br, bc)
        Xl = shard.local_activations(X, s, offsets).to(DEV)
        full[int(offsets[s.e0]):int(offsets[s.e1])] += shard.gemm_grouped_local(Xl, Wl, offsets)   # its rows, no others
    torch.cuda.synchronize()
    assert np.array_equal(full.cpu().numpy().astype(np.float64), want)


NCCL_WORKER = r'''
import os, sys
sys.path.insert(0, os.environ["TL_ROOT"])
import numpy as np, torch
import torch.distributed as dist
import oracle as tlo
from paper_2607_04031_b200 import inputs, shard
torch.cuda.set_device(0)
dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda:0"))
M, N, K, br, bc, G = 8, 512, 256, 16, 128, 4096
A = inputs.bf16_integers((M, K), -4, 4, seed=1)
W = inputs.bf16_integers((K, N), -3, 3, seed=2)
want = tlo.matmul(inputs.bits(A), inputs.bits(W), tlo.ROW_MAJOR, 0, 0, M, N, K)[0]
for mode in ("n", "k"):
    shards = shard.plan(mode, N, K, br, bc, 1)
    Wl = shard.ShardedWeight(shard.local_weight(W, shards[0]).to("cuda:0"), shards[0], G, br, bc)
    C = shard.gemm(shard.local_activations(A, shards[0]).to("cuda:0"), Wl, shards)
    C2 = C.clone()
    dist.all_reduce(C2)                      # the collective the k-split issues when there are peers, on NCCL
    torch.cuda.synchronize()
    assert np.array_equal(C.cpu().numpy().astype(np.float64), want), mode
    assert np.array_equal(C2.cpu().numpy().astype(np.float64), want), mode
dist.destroy_process_group()
print("ok")
'''


def test_one_rank_process_group_on_nccl_runs_the_sharded_call():
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    env = dict(os.environ, RANK="0", WORLD_SIZE="1", LOCAL_RANK="0", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port),
               TL_ROOT=ROOT, NCCL_NVLS_ENABLE="0")
    r = subprocess.run([sys.executable, "-c", NCCL_WORKER], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip().endswith("ok"), r.stderr[-3000:]
