"""Read-amplification kernel vs the oracle's brute force: bit-exact (GPU)."""
import numpy as np
import pytest
import torch

import oracle as tlo
from paper_2607_04031_b200 import inputs

pytestmark = pytest.mark.gpu
ROW, COL, TILE = 0, 1, 2

from test_oracle_readamp import TINY  # the same tiny cases the oracle is pinned on


@pytest.mark.parametrize("M,N,K,BM,BN,BK,layout,G,br,bc,s", TINY)
def test_tiny_cases(M, N, K, BM, BN, BK, layout, G, br, bc, s):
    from gpu_util import tl
    assert tl.read_amp(M, N, K, (BM, BN, BK), layout, G, br, bc, s) == \
        tlo.read_amp(M, N, K, BM, BN, BK, layout, G, br, bc, s)


def test_non_power_of_two_blocks_are_counted_too():
    from gpu_util import tl
    # the counter uses division, so any block shape works (only the kernels that move data need powers of two)
    assert tl.read_amp(3, 36, 30, (3, 10, 7), TILE, 48, 2, 6, 4) == tlo.read_amp(3, 36, 30, 3, 10, 7, TILE, 48, 2, 6, 4)


def test_config1():
    from gpu_util import tl
    for G, cases in ((4096, [(ROW, 0, 0), (COL, 0, 0), (TILE, 16, 128), (TILE, 32, 64)]),
                     (32, [(ROW, 0, 0), (TILE, 1, 16), (TILE, 2, 8)])):
        for layout, br, bc in cases:
            got = tl.read_amp(16, 512, 512, (64, 64, 64), layout, G, br, bc, 2)
            assert got == tlo.read_amp(16, 512, 512, 64, 64, 64, layout, G, br, bc, 2)
    assert tl.read_amp(16, 512, 512, (64, 64, 64), ROW, 4096, 0, 0, 2)[:2] == (4194304, 524288)
    assert tl.read_amp(16, 512, 512, (64, 64, 64), TILE, 4096, 16, 128, 2)[:2] == (1048576, 524288)
    assert tl.read_amp(16, 512, 512, (64, 128, 64), TILE, 4096, 16, 128, 2)[:2] == (524288, 524288)


@pytest.mark.parametrize("G", [32, 256, 1024, 4096, 16384])
def test_config5_sweep(G):
    from gpu_util import tl
    K = N = 8192
    for cta in ((64, 64, 64), (128, 128, 64), (256, 128, 64), (128, 256, 128)):
        for M in (1, 128):
            got = tl.read_amp(M, N, K, cta, ROW, G, 0, 0, 2)
            assert got == tlo.read_amp(M, N, K, *cta, ROW, G, 0, 0, 2)
        for r in (1, 8, 16, 32):
            bc = G // (2 * r)
            if bc < 1:
                continue
            got = tl.read_amp(16, N, K, cta, TILE, G, r, bc, 2)
            assert got == tlo.read_amp(16, N, K, *cta, TILE, G, r, bc, 2)
            # RA == 1 exactly when the memory tile divides the compute tile
            if cta[2] % r == 0 and cta[1] % bc == 0:
                assert got[0] == got[1]
    got = tl.read_amp(16, N, K, (64, 64, 64), COL, G, 0, 0, 2)
    assert got == tlo.read_amp(16, N, K, 64, 64, 64, COL, G, 0, 0, 2)


def test_llama_and_qwen_shapes_default_tile():
    from gpu_util import tl
    for name, K, N in inputs.LLAMA70B_PROJ:
        for layout, br, bc in ((ROW, 0, 0), (TILE, 16, 128)):
            for M in (1, 32, 4096):
                cta = (min(256, max(16, M)), 128, 64)
                assert tl.read_amp(M, N, K, cta, layout, 4096, br, bc, 2) == \
                    tlo.read_amp(M, N, K, *cta, layout, 4096, br, bc, 2), name
    # Section 6.5: the paper's 128 x 256 weight tile on the Qwen expert weights
    offsets, counts, _ = inputs.zipf_topk_routing(256, 128, 8, 1.1, seed=0)
    for name, K, N in inputs.QWEN_MOE_PROJ:
        for layout, br, bc in ((ROW, 0, 0), (TILE, 16, 128), (TILE, 32, 64)):
            got = tl.read_amp_grouped(offsets, N, K, (256, 256, 128), layout, 4096, br, bc, 2)
            assert got == tlo.read_amp_grouped(offsets, N, K, 256, 256, 128, layout, 4096, br, bc, 2), name
            if layout == TILE:
                assert got[0] == got[1]


def test_odd_sizes_and_pitches():
    from gpu_util import tl
    rng = np.random.default_rng(3)
    for _ in range(40):
        s = int(rng.choice([1, 2, 4]))
        N, K = int(rng.integers(1, 300)), int(rng.integers(1, 300))
        BN, BK, BM = int(rng.integers(1, 130)), int(rng.integers(1, 130)), int(rng.integers(1, 70))
        M = int(rng.integers(0, 200))
        G = int(rng.choice([4, 8, 12, 32, 48, 100, 256, 4096])) * s
        for layout in (ROW, COL):
            assert tl.read_amp(M, N, K, (BM, BN, BK), layout, G, 0, 0, s) == \
                tlo.read_amp(M, N, K, BM, BN, BK, layout, G, 0, 0, s), (M, N, K, BM, BN, BK, layout, G, s)
        br, bc = int(rng.integers(1, 9)), int(rng.integers(1, 17))
        N2, K2 = bc * int(rng.integers(1, 20)), br * int(rng.integers(1, 20))
        assert tl.read_amp(M, N2, K2, (BM, BN, BK), TILE, br * bc * s, br, bc, s) == \
            tlo.read_amp(M, N2, K2, BM, BN, BK, TILE, br * bc * s, br, bc, s)


def test_per_cta_arrays():
    from gpu_util import DEV, tl
    M, N, K, cta = 40, 200, 96, (16, 64, 32)
    mt, nt = 3, 4
    f = torch.zeros(mt * nt, dtype=torch.int64, device=DEV)
    u = torch.zeros_like(f)
    tl.read_amp_per_cta(M, N, K, cta, ROW, 128, 0, 0, 2, f, u)
    torch.cuda.synchronize()
    F, U, Q, pf, pu = tlo.read_amp(M, N, K, *cta, ROW, 128, 0, 0, 2, per_tile=True)
    assert np.array_equal(f.cpu().numpy().view(np.uint64), pf)
    assert np.array_equal(u.cpu().numpy().view(np.uint64), pu)


def test_empty_and_errors():
    from gpu_util import tl
    assert tl.read_amp(0, 512, 512, (64, 64, 64), ROW, 4096, 0, 0, 2) == (0, 0, 0)
    with pytest.raises(tl.TileLensError):
        tl.read_amp(1, 512, 512, (64, 64, 64), TILE, 4096, 16, 64, 2)


# ------------------------------------------------------------------ requests shared between co-resident CTAs
SHARED_CASES = [  # M, N, K, cta, G, layout, br, bc, s
    (70, 96, 64, (32, 24, 16), 128, "row", 0, 0, 2),
    (70, 96, 64, (32, 24, 16), 128, "col", 0, 0, 2),
    (70, 96, 64, (32, 24, 16), 128, "tile", 4, 16, 2),
    (70, 96, 64, (32, 24, 16), 128, "tile_k", 8, 8, 2),
    (300, 1000, 520, (128, 256, 128), 4096, "row", 0, 0, 2),
    (300, 1000, 520, (128, 256, 128), 4096, "col", 0, 0, 1),
    (512, 1536, 2048, (128, 256, 128), 4096, "tile", 32, 64, 2),
    (512, 1536, 2048, (128, 256, 128), 4096, "tile_k", 32, 64, 2),
    (512, 1536, 2048, (128, 256, 128), 4096, "row", 0, 0, 2),
]


@pytest.mark.parametrize("case", SHARED_CASES)
@pytest.mark.parametrize("P", [1, 2, 5, 8, 148, 100000])
def test_shared_request_count_matches_the_oracle(case, P):
    from gpu_util import tl
    M, N, K, cta, G, layout, br, bc, s = case
    lt = {"row": tl.LAYOUT_ROW_MAJOR, "col": tl.LAYOUT_COL_MAJOR, "tile": tl.LAYOUT_TILE_MAJOR, "tile_k": tl.LAYOUT_TILE_MAJOR_K}[layout]
    lo = {"row": tlo.ROW_MAJOR, "col": tlo.COL_MAJOR, "tile": tlo.TILE_MAJOR, "tile_k": tlo.TILE_MAJOR_K}[layout]
    assert tl.read_amp_shared(M, N, K, cta, P, lt, G, br, bc, s) == tlo.read_amp_shared(M, N, K, *cta, P, lo, G, br, bc, s)


def test_shared_request_count_full_size_properties():
    # Llama gate_up, prefill tiles, one wave = 148 CTAs.  Too large for the brute force: properties that hold at any
    # size -- never above the unshared count, never below what is needed, tile-major exactly what is needed.
    from gpu_util import tl
    M, N, K, cta, G = 4096, 57344, 8192, (256, 256, 64), 4096
    plain = tl.read_amp(M, N, K, cta, tl.LAYOUT_ROW_MAJOR, G, 0, 0, 2)
    f, u, q = tl.read_amp_shared(M, N, K, cta, 148, tl.LAYOUT_ROW_MAJOR, G, 0, 0, 2)
    assert u <= f <= plain[0] and f == q * G
    ft, ut, _ = tl.read_amp_shared(M, N, K, cta, 148, tl.LAYOUT_TILE_MAJOR, G, 16, 128, 2)
    assert ft == ut
    # 16 m-tiles share each n-tile: a wave of 148 tiles spans 10 n-tiles, so sharing cuts the row-major traffic
    assert f * 4 < plain[0]


def test_per_cta_counts_k_contiguous_flavour():
    import torch
    from gpu_util import DEV, tl
    M, N, K, cta, G, b, a = 300, 1024, 512, (128, 256, 128), 4096, 32, 64
    mt, nt = -(-M // cta[0]), -(-N // cta[1])
    f = torch.zeros(mt * nt, dtype=torch.int64, device=DEV)
    u = torch.zeros(mt * nt, dtype=torch.int64, device=DEV)
    tl.read_amp_per_cta(M, N, K, cta, tl.LAYOUT_TILE_MAJOR_K, G, b, a, 2, f, u)
    torch.cuda.synchronize()
    _, _, _, pf, pu = tlo.read_amp(M, N, K, *cta, tlo.TILE_MAJOR_K, G, b, a, 2, per_tile=True)
    assert np.array_equal(f.cpu().numpy().astype(np.uint64), pf) and np.array_equal(u.cpu().numpy().astype(np.uint64), pu)


def test_async_totals_match_the_waiting_call_when_queued_back_to_back():
    import torch
    from gpu_util import DEV, tl
    cases = [(8, 10240, 8192, (16, 128, 64), tl.LAYOUT_TILE_MAJOR, 16, 128), (32, 8192, 8192, (32, 128, 64), tl.LAYOUT_ROW_MAJOR, 0, 0),
             (300, 1000, 520, (128, 256, 128), tl.LAYOUT_COL_MAJOR, 0, 0), (0, 512, 512, (16, 128, 64), tl.LAYOUT_ROW_MAJOR, 0, 0),
             (1, 57344, 8192, (16, 256, 64), tl.LAYOUT_TILE_MAJOR_K, 32, 64)]
    out = torch.full((len(cases), 3), -1, dtype=torch.int64, device=DEV)
    for i, (M, N, K, cta, layout, br, bc) in enumerate(cases):          # all queued before any result is read
        tl.read_amp_async(M, N, K, cta, layout, 4096, br, bc, 2, out[i])
    got = out.cpu().numpy()
    for i, (M, N, K, cta, layout, br, bc) in enumerate(cases):
        assert tuple(int(x) for x in got[i]) == tl.read_amp(M, N, K, cta, layout, 4096, br, bc, 2)


def test_batched_counters_match_the_single_calls():
    import torch
    from gpu_util import DEV, tl
    cases = [(8, 10240, 8192, (16, 128, 64), tl.LAYOUT_TILE_MAJOR, 4096, 16, 128, 2),
             (32, 8192, 8192, (32, 128, 64), tl.LAYOUT_ROW_MAJOR, 4096, 0, 0, 2),
             (300, 1000, 520, (128, 256, 128), tl.LAYOUT_COL_MAJOR, 4096, 0, 0, 1),
             (0, 512, 512, (16, 128, 64), tl.LAYOUT_ROW_MAJOR, 4096, 0, 0, 2),
             (1, 57344, 8192, (16, 256, 64), tl.LAYOUT_TILE_MAJOR_K, 4096, 32, 64, 2),
             (70, 96, 64, (32, 24, 16), tl.LAYOUT_ROW_MAJOR, 128, 0, 0, 2)] * 2 + [(4096, 8192, 28672, (256, 128, 64), tl.LAYOUT_ROW_MAJOR, 4096, 0, 0, 2)]
    out = torch.full((len(cases), 3), -1, dtype=torch.int64, device=DEV)
    for rep in range(3):                                   # back to back: the accumulators must come back to zero
        tl.read_amp_batch(tl.read_amp_cfgs(cases), out)
    got = out.cpu().numpy()
    for i, (M, N, K, cta, layout, G, br, bc, s) in enumerate(cases):
        assert tuple(int(x) for x in got[i]) == tl.read_amp(M, N, K, cta, layout, G, br, bc, s), i
    with pytest.raises(tl.TileLensError):
        tl.read_amp_batch(tl.read_amp_cfgs(cases + cases), torch.zeros((26, 3), dtype=torch.int64, device=DEV))    # more than 16
