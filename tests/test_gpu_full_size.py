"""Full-size parity (GPU): the benchmark's own shapes in the library's own launch configuration.

The oracle cannot form these products in full (Llama gate_up at M = 4096 is 1.9 T multiply-adds), so the products
are compared on a sample that leaves no output tile unvisited: for EVERY 128 x 128 tile of C sixteen seeded
elements, plus eight full rows, eight full columns and the four corner tiles in full.  A fault confined to a few
tiles of the grid (a wave remainder, a band of the tile order, a ragged last tile) cannot pass it.  The relayouts of
the same weights are compared with the oracle byte for byte, in both directions.
"""
import numpy as np
import pytest
import torch

import oracle as tlo
from paper_2607_04031_b200 import inputs

pytestmark = pytest.mark.gpu
TILE = tlo.TILE_MAJOR
BR, BC, G = 16, 128, 4096


def per_tile_sample(M, N, seed, per_tile=16, lines=8, tile=128):
    """Index arrays (ii, jj): `per_tile` seeded elements of every tile x tile block of an M x N matrix, `lines`
    full rows and columns, and the four corner blocks in full."""
    rng = np.random.default_rng(seed)
    tm, tn = -(-M // tile), -(-N // tile)
    ti, tj = np.meshgrid(np.arange(tm), np.arange(tn), indexing="ij")
    ti, tj = np.repeat(ti.reshape(-1), per_tile), np.repeat(tj.reshape(-1), per_tile)
    hi_i = np.minimum(tile, M - ti * tile)
    hi_j = np.minimum(tile, N - tj * tile)
    ii = [ti * tile + (rng.integers(0, 1 << 30, ti.size) % hi_i)]
    jj = [tj * tile + (rng.integers(0, 1 << 30, tj.size) % hi_j)]
    for r in rng.choice(M, size=min(lines, M), replace=False):            # full rows
        ii.append(np.full(N, r)); jj.append(np.arange(N))
    for c in rng.choice(N, size=min(lines, N), replace=False):            # full columns
        ii.append(np.arange(M)); jj.append(np.full(M, c))
    for r0 in {0, (tm - 1) * tile}:                                        # corner blocks
        for c0 in {0, (tn - 1) * tile}:
            r, c = np.meshgrid(np.arange(r0, min(r0 + tile, M)), np.arange(c0, min(c0 + tile, N)), indexing="ij")
            ii.append(r.reshape(-1)); jj.append(c.reshape(-1))
    return np.concatenate(ii).astype(np.int64), np.concatenate(jj).astype(np.int64)


def test_the_sample_visits_every_tile():
    ii, jj = per_tile_sample(300, 700, seed=1)
    seen = np.zeros((3, 6), dtype=np.int64)
    np.add.at(seen, (ii // 128, jj // 128), 1)
    assert seen.min() >= 16 and ii.max() == 299 and jj.max() == 699


@pytest.mark.parametrize("name,K,N", inputs.LLAMA70B_PROJ)
def test_llama_prefill_every_tile_sampled(name, K, N):
    from gpu_util import DEV, run_gemm, tl
    M = inputs.LLAMA_PREFILL_M
    A = inputs.bf16_normal((M, K), 1.0, seed=41, device=DEV)
    B = inputs.bf16_normal((K, N), 0.02, seed=42, device=DEV)
    Bt = torch.empty_like(B)
    tl.relayout(B, Bt, K, N, 2, G, BR, BC, tl.TO_TILE_MAJOR)
    del B
    C = run_gemm(A, Bt, M, N, K, BR, BC)
    plan = tl.gemm_last_plan()
    assert plan.pair_kernel == 1 and plan.cta_m == 512                   # the configuration bench.py times
    assert torch.isfinite(C).all()
    ii, jj = per_tile_sample(M, N, seed=K + N)
    got = C[torch.from_numpy(ii).to(DEV), torch.from_numpy(jj).to(DEV)].cpu().numpy().astype(np.float64)
    del C
    ref, S = tlo.matmul_at(inputs.bits(A), inputs.bits(Bt.reshape(-1)), TILE, BR, BC, M, N, K, ii, jj)
    err = np.abs(got - ref)
    assert np.all(err <= 1e-3 * S), f"max err/S = {np.max(err / np.maximum(S, 1e-300)):.3e}"
    assert float(np.max(err / np.maximum(S, 1e-300))) <= 1e-4


# Between decode and prefill the library picks the tile and the schedule from the shape: each kind once at full size.
MID_CASES = [
    ("gate_up", 128, "wide"),          # 128 x 256 x 64, whole tiles on 112 CTAs
    ("qkv", 128, "wide_clusters"),     # the same tile, split-K inside clusters of 3
    ("gate_up", 256, "two_blocks"),    # 256 x 256 x 64: two token blocks per weight slab
    ("down", 384, "cut"),              # 128 x 128 x 128 with the stream-K cut and its reduction kernel
    ("qkv", 640, "two_blocks"),        # 120 tiles on 120 CTAs instead of two waves of pairs
    ("gate_up", 768, "pairs_256"),     # CTA pairs on 256-token tiles only (512-token tiles would be half empty)
    ("down", 1024, "two_blocks"),      # 128 tiles on 128 CTAs
]


@pytest.mark.parametrize("proj,M,kind", MID_CASES)
def test_llama_between_decode_and_prefill_every_tile_sampled(proj, M, kind):
    from gpu_util import DEV, run_gemm, tl
    K, N = next((k, n) for name, k, n in inputs.LLAMA70B_PROJ if name == proj)
    A = inputs.bf16_normal((M, K), 1.0, seed=43, device=DEV)
    B = inputs.bf16_normal((K, N), 0.02, seed=44, device=DEV)
    Bt = torch.empty_like(B)
    tl.relayout(B, Bt, K, N, 2, G, BR, BC, tl.TO_TILE_MAJOR)
    del B
    C = run_gemm(A, Bt, M, N, K, BR, BC)
    p = tl.gemm_last_plan()
    if kind == "wide":
        assert (p.cta, p.stream_k, p.cluster_k) == ((128, 256, 64), 0, 1)
    elif kind == "wide_clusters":
        assert (p.cta, p.stream_k, p.cluster_k) == ((128, 256, 64), 0, 3)
    elif kind == "two_blocks":
        assert (p.cta, p.pair_kernel, p.stream_k, p.cluster_k) == ((256, 256, 64), 0, 0, 1)
    elif kind == "cut":
        assert (p.cta, p.stream_k) == ((128, 128, 128), 1)
    else:
        assert (p.pair_kernel, p.pair_tiles_512) == (1, 0)
    assert torch.isfinite(C).all()
    ii, jj = per_tile_sample(M, N, seed=K + N + M, per_tile=8, lines=4)
    got = C[torch.from_numpy(ii).to(DEV), torch.from_numpy(jj).to(DEV)].cpu().numpy().astype(np.float64)
    del C
    ref, S = tlo.matmul_at(inputs.bits(A), inputs.bits(Bt.reshape(-1)), TILE, BR, BC, M, N, K, ii, jj)
    err = np.abs(got - ref)
    assert np.all(err <= 1e-3 * S), f"max err/S = {np.max(err / np.maximum(S, 1e-300)):.3e}"
    assert float(np.max(err / np.maximum(S, 1e-300))) <= 1e-4


@pytest.mark.parametrize("name,K,N", inputs.QWEN_MOE_PROJ)
def test_qwen_moe_every_tile_sampled(name, K, N):
    from gpu_util import DEV, guarded_out, tl
    q = inputs.QWEN_MOE
    E = q["experts"]
    offsets, counts, expert_of_row = inputs.zipf_topk_routing(q["tokens"], E, q["topk"], q["zipf_alpha"], seed=0)
    rows = int(offsets[-1])
    A = inputs.bf16_normal((rows, K), 1.0, seed=1)
    B = inputs.bf16_normal((E, K, N), 0.02, seed=2, device=DEV)
    Bt = torch.empty_like(B)
    tl.relayout(B, Bt, E * K, N, 2, G, BR, BC, tl.TO_TILE_MAJOR)        # experts laid end to end
    g = guarded_out((rows, N), torch.float32)
    tl.gemm_grouped(A.to(DEV), Bt, g.t, torch.from_numpy(offsets).to(DEV), E, rows, N, K, G, BR, BC)
    tl.device_status()
    Ch = g.check().cpu().numpy().astype(np.float64)
    assert np.all(np.isfinite(Ch))
    ii, jj = per_tile_sample(rows, N, seed=K)
    A_bits, worst = inputs.bits(A), 0.0
    owner = expert_of_row[ii]
    for e in np.unique(owner):
        sel = owner == e
        r0, r1 = int(offsets[e]), int(offsets[e + 1])
        ref, S = tlo.matmul_at(A_bits[r0:r1], inputs.bits(Bt[e].reshape(-1)), TILE, BR, BC, r1 - r0, N, K,
                               ii[sel] - r0, jj[sel])
        err = np.abs(Ch[ii[sel], jj[sel]] - ref)
        assert np.all(err <= 1e-3 * S), f"expert {e}"
        worst = max(worst, float(np.max(err / np.maximum(S, 1e-300))))
    assert worst <= 1e-4


FULL_SIZE_WEIGHTS = [
    ("llama_gate_up", 8192, 57344), ("llama_down", 28672, 8192), ("llama_qkv", 8192, 10240),
    ("qwen_gate_up_128_experts", 128 * 2048, 1536), ("qwen_down_128_experts", 128 * 768, 2048),
]


@pytest.mark.parametrize("name,rows,cols", FULL_SIZE_WEIGHTS)
def test_relayout_of_full_size_weights_every_byte(name, rows, cols):
    from gpu_util import DEV, Guarded, tl
    B = inputs.bf16_normal((rows, cols), 0.02, seed=rows % 1009 + cols, device=DEV)
    host = inputs.bits(B).view(np.uint8).reshape(-1)
    want = tlo.relayout(host, rows, cols, 2, BR, BC, tlo.TO_TILE_MAJOR)
    gt = Guarded((rows, cols), torch.bfloat16)
    tl.relayout(B, gt.t, rows, cols, 2, G, BR, BC, tl.TO_TILE_MAJOR)
    tiled = gt.check()
    assert np.array_equal(tiled.cpu().view(torch.uint8).numpy().reshape(-1), want)
    # back, from the oracle's tile-major bytes (not from the bytes the library just wrote)
    src = torch.from_numpy(want).to(DEV)
    gb = Guarded((rows, cols), torch.bfloat16)
    tl.relayout(src, gb.t, rows, cols, 2, G, BR, BC, tl.TO_ROW_MAJOR)
    assert np.array_equal(gb.check().cpu().view(torch.uint8).numpy().reshape(-1), host)
    tl.device_status()


def test_layer_batch_relayout_every_byte():
    # the four Llama weights in one launch, as the benchmark step does it
    from gpu_util import DEV, Guarded, tl
    srcs, guards, shapes = [], [], []
    for i, (_, K, N) in enumerate(inputs.LLAMA70B_PROJ):
        srcs.append(inputs.bf16_normal((K, N), 0.02, seed=300 + i, device=DEV))
        guards.append(Guarded((K, N), torch.bfloat16))
        shapes.append((K, N))
    tl.relayout_batch(srcs, [g.t for g in guards], shapes, 2, G, BR, BC, tl.TO_TILE_MAJOR)
    tl.device_status()
    for src, g, (K, N) in zip(srcs, guards, shapes):
        want = tlo.relayout(inputs.bits(src).view(np.uint8).reshape(-1), K, N, 2, BR, BC, tlo.TO_TILE_MAJOR)
        assert np.array_equal(g.check().cpu().view(torch.uint8).numpy().reshape(-1), want), (K, N)
