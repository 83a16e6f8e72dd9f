"""Sharding the GEMM over ranks: the plan, shard-locality of the tile-major layout (Section 3), and the exchange
step on CPU with gloo, world size 2 (local results come from the oracle; the exchange code is the product's)."""
import json
import os
import socket
import subprocess
import sys

import numpy as np
import pytest
import torch

import oracle as tlo
from paper_2607_04031_b200 import inputs, shard

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.parametrize("mode", ["n", "k", "expert"])
@pytest.mark.parametrize("world", [1, 2, 3, 8])
@pytest.mark.parametrize("blk", [(16, 128), (32, 64), (4, 512), (2, 1024), (0, 0)])
def test_plan_covers_everything_once_on_block_boundaries(mode, world, blk):
    br, bc = blk
    N, K, E = 9 * 1024, 1280, 11
    shards = shard.plan(mode, N, K, br, bc, world, E)
    assert [s.rank for s in shards] == list(range(world)) and all(s.world == world and s.mode == mode for s in shards)
    dim = {"n": ("n0", "n1", N), "k": ("k0", "k1", K), "expert": ("e0", "e1", E)}[mode]
    lo = [getattr(s, dim[0]) for s in shards]
    hi = [getattr(s, dim[1]) for s in shards]
    assert lo[0] == 0 and hi[-1] == dim[2] and lo[1:] == hi[:-1]            # contiguous, disjoint, complete
    assert all(h > l for l, h in zip(lo, hi))                               # nobody is idle
    unit = {"n": bc if br else 64, "k": max(br, 8) if br else 8, "expert": 1}[mode]
    assert all(v % unit == 0 for v in lo + hi)
    sizes = [(h - l) // unit for l, h in zip(lo, hi)]
    assert max(sizes) - min(sizes) <= 1                                     # balanced to one block
    for s in shards:                                                        # the uncut dimensions stay whole
        if mode != "n": assert (s.n0, s.n1) == (0, N)
        if mode != "k": assert (s.k0, s.k1) == (0, K)
        if mode != "expert": assert (s.e0, s.e1) == (0, E)


def test_plan_refuses_what_it_cannot_cut():
    with pytest.raises(ValueError): shard.plan("n", 256, 256, 16, 128, 3)    # two block columns, three ranks
    with pytest.raises(ValueError): shard.plan("k", 256, 100, 16, 128, 2)    # K is not whole blocks
    with pytest.raises(ValueError): shard.plan("x", 256, 256, 16, 128, 2)
    with pytest.raises(ValueError): shard.plan("expert", 256, 256, 16, 128, 4, E=3)


@pytest.mark.parametrize("mode,world", [("n", 3), ("k", 2), ("k", 5)])
@pytest.mark.parametrize("blk", [(16, 128), (64, 32), (8, 256)])
def test_tile_major_image_of_a_shard_is_the_shards_blocks_of_the_full_image(mode, world, blk):
    """Blocks never straddle a shard boundary: re-laying-out a rank's slice gives exactly the blocks (kb, nb) of the
    full tile-major buffer that fall inside the slice, in the same block order (Eq. 1-2 with the slice's extents)."""
    br, bc = blk
    K, N = 640, 1280
    W = inputs.bf16_normal((K, N), 1.0, seed=7)
    full = tlo.relayout(inputs.bits(W).view(np.uint8), K, N, 2, br, bc, tlo.TO_TILE_MAJOR).view(np.uint16)
    blocks = full.reshape(K // br, N // bc, br * bc)                        # [K/br][N/bc][one G-byte block]
    for s in shard.plan(mode, N, K, br, bc, world):
        Wl = shard.local_weight(W, s)
        img = tlo.relayout(inputs.bits(Wl).view(np.uint8), s.k1 - s.k0, s.n1 - s.n0, 2, br, bc,
                           tlo.TO_TILE_MAJOR).view(np.uint16)
        want = blocks[s.k0 // br:s.k1 // br, s.n0 // bc:s.n1 // bc].reshape(-1)
        assert np.array_equal(img, want)


WORKER = r'''
import json, os, sys
sys.path.insert(0, os.environ["TL_ROOT"])
import numpy as np, torch
import torch.distributed as dist
import oracle as tlo
from paper_2607_04031_b200 import inputs, shard
rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo")
M, N, K, br, bc, E = 5, 384, 96, 16, 128, 5
A = inputs.bf16_normal((M, K), 1.0, seed=1)
W = inputs.bf16_normal((K, N), 0.05, seed=2)
def mm(a, w):   # local result from the oracle, row-major operand
    m, k = a.shape; n = w.shape[1]
    return torch.from_numpy(tlo.matmul(inputs.bits(a), inputs.bits(w), tlo.ROW_MAJOR, 0, 0, m, n, k)[0])
full = mm(A, W)
out = {}
for mode in ("n", "k"):
    shards = shard.plan(mode, N, K, br, bc, world)
    s = shards[rank]
    C_local = mm(shard.local_activations(A, s), shard.local_weight(W, s))
    C = shard.combine_n(C_local, shards) if mode == "n" else shard.combine_k(C_local)
    out[mode] = float((C - full).abs().max())
    out[mode + "_shape"] = list(C.shape)
# experts: rows of unequal counts, one expert without tokens
offsets = [0, 3, 3, 10, 11, 16]
X = inputs.bf16_normal((offsets[-1], K), 1.0, seed=3)
WE = inputs.bf16_normal((E, K, N), 0.05, seed=4)
full_e = torch.cat([mm(X[offsets[e]:offsets[e + 1]], WE[e]) for e in range(E)])
s = shard.plan("expert", N, K, br, bc, world, E)[rank]
Xl, Wl, offs = shard.local_activations(X, s, offsets), shard.local_weight(WE, s), shard.local_offsets(offsets, s)
rows = [mm(Xl[offs[i]:offs[i + 1]], Wl[i]) for i in range(s.e1 - s.e0)]
C = shard.combine_expert(torch.cat(rows), s, offsets, offsets[-1])
out["expert"] = float((C - full_e).abs().max())
out["expert_offs"] = offs
dist.barrier()
print(json.dumps(out), flush=True)
dist.destroy_process_group()
'''


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_exchange_step_on_two_gloo_ranks_reproduces_the_unsharded_product():
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), TL_ROOT=ROOT)
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=240) for p in procs]
    assert all(p.returncode == 0 for p in procs), [o[1][-2000:] for o in outs]
    lines = [json.loads(o[0].strip().splitlines()[-1]) for o in outs]
    for line in lines:                                                     # every rank holds the full result
        assert line["n"] == 0.0 and line["n_shape"] == [5, 384]            # concatenation moves values, no arithmetic
        assert line["k"] < 1e-12 and line["k_shape"] == [5, 384]           # fp64 partial sums: rounding order only
        assert line["expert"] == 0.0                                       # x + 0 is exact
    assert lines[0]["expert_offs"] == [0, 3, 3] and lines[1]["expert_offs"] == [0, 7, 8, 13]


def test_sharded_calls_fail_loudly_without_the_cuda_library(monkeypatch):
    """The launches go through the C-ABI binding; there is no host fallback behind them."""
    from paper_2607_04031_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", os.path.join(ROOT, "no_such_dir", "libtilelens.so"))
    s = shard.plan("n", 256, 64, 0, 0, 1)[0]
    W = shard.ShardedWeight(torch.zeros((64, 256), dtype=torch.bfloat16), s, 4096, 0, 0)
    with pytest.raises(RuntimeError, match="is missing"):
        shard.gemm_local(torch.zeros((4, 64), dtype=torch.bfloat16), W)
