"""Pins for the oracle's read-amplification count (CPU only)."""
import json
import os

import numpy as np
import pytest

import oracle as tlo

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_values.json")))
ROW, COL, TILE = tlo.ROW_MAJOR, tlo.COL_MAJOR, tlo.TILE_MAJOR


def _element_positions(K, N, layout, br, bc):
    """Element index -> position in the buffer, built with numpy reshapes only (no offset formula)."""
    ids = np.arange(K * N).reshape(K, N)
    if layout == ROW:
        buf = ids.reshape(-1)
    elif layout == COL:
        buf = ids.T.reshape(-1)
    else:
        buf = ids.reshape(K // br, br, N // bc, bc).transpose(0, 2, 1, 3).reshape(-1)
    pos = np.empty(K * N, dtype=np.int64)
    pos[buf] = np.arange(K * N)
    return pos.reshape(K, N)


def _python_count(M, N, K, BM, BN, BK, layout, G, br, bc, s):
    """Set of G-blocks per tile load, byte by byte."""
    pos = _element_positions(K, N, layout, br, bc)
    fetched = used = requests = 0
    for n0 in range(0, N, BN):
        for k0 in range(0, K, BK):
            rect = pos[k0:min(k0 + BK, K), n0:min(n0 + BN, N)].reshape(-1)
            blocks = set()
            for p in rect:
                for byte in range(s):
                    blocks.add((int(p) * s + byte) // G)
            fetched += len(blocks) * G
            requests += len(blocks)
            used += rect.size * s
    mt = -(-M // BM)
    return fetched * mt, used * mt, requests * mt


def test_printed_requests_per_compute_tile():
    g = GOLD["requests_per_tile"]
    BK, BN, s, G = g["tile_rows"], g["tile_cols"], g["elem_bytes"], g["G"]
    a, b = g["tile_major_memory_tile_a_b"]          # a = contiguous extent -> bc, b -> br
    K, N = BK, 2048 * 2                             # one K iteration; row pitch 8 KB >= G
    _, _, q_row = tlo.read_amp(1, BN, K, 1, BN, BK, ROW, G, 0, 0, s)          # N = BN: pitch 512 B < G
    f, u, q = tlo.read_amp(1, N, K, 1, BN, BK, ROW, G, 0, 0, s)
    loads = N // BN
    assert q == g["row_major_requests"] * loads
    ft, ut, qt = tlo.read_amp(1, N, K, 1, BN, BK, TILE, G, b, a, s)
    assert qt == g["tile_major_requests"] * loads
    assert (q - qt) // loads == g["extra_requests"]
    assert (q - qt) // loads * G == g["extra_bytes_KB"] * 1024
    assert ft == ut == BK * BN * s * loads
    assert q_row == BK * BN * s // G                # a matrix exactly as wide as the tile wastes nothing


def test_printed_granularity_ratios():
    r = GOLD["granularity_ratio"]
    assert r["G_lgms"] // r["G_hbm"] == r["ratio"]
    # a tile row of w useful bytes on a pitch >= G fetches one whole block: RA = G / w
    for w, want in ((32, 128), (128, 32)):
        s, BK = 1, 8
        f, u, _ = tlo.read_amp(1, 8192, BK, 1, w // s, BK, ROW, 4096, 0, 0, s)
        assert f == want * u
    a = GOLD["amplification_32x"]
    assert a["sms"] * a["smem_KB"] * a["factor"] == a["total_MB"] * 1024
    f, u, _ = tlo.read_amp(1, 8192, 64, 1, 128, 64, ROW, 4096, 0, 0, 1)       # FP8, 128-B-wide strip
    assert f == a["factor"] * u


def test_fp8_64x64_memory_tile_fits_compute_tiles():
    # Figure 1(c), Section 3.1: a 64 x 64 FP8 memory tile inside 64x64, 128x128, 256x256 compute tiles.
    for t in (64, 128, 256):
        f, u, q = tlo.read_amp(1, 512, 512, 1, t, t, TILE, 4096, 64, 64, 1)
        assert f == u == 512 * 512
    f, u, _ = tlo.read_amp(1, 8192, 64, 1, 64, 64, ROW, 4096, 0, 0, 1)        # (1, 4096) strip
    assert f == 64 * u
    f, u, _ = tlo.read_amp(1, 64, 8192, 1, 64, 64, COL, 4096, 0, 0, 1)        # (4096, 1) strip
    assert f == 64 * u


@pytest.mark.parametrize("br,bc,BK,BN", [(16, 128, 64, 128), (32, 64, 64, 64), (8, 256, 128, 256),
                                         (16, 128, 16, 128), (1, 2048, 64, 2048), (32, 64, 128, 256)])
def test_no_amplification_when_memory_tile_divides_compute_tile(br, bc, BK, BN):
    K, N, s = 256, 4096, 2
    f, u, q = tlo.read_amp(100, N, K, 64, BN, BK, TILE, br * bc * s, br, bc, s)
    assert f == u == 2 * K * N * s                  # two m-tiles
    assert q * br * bc * s == f


TINY = [  # M, N, K, BM, BN, BK, layout, G, br, bc, s
    (1, 40, 48, 1, 16, 16, ROW, 32, 0, 0, 1),
    (1, 40, 48, 1, 16, 16, COL, 32, 0, 0, 1),
    (1, 40, 48, 1, 16, 16, TILE, 32, 4, 8, 1),
    (5, 40, 48, 2, 24, 20, ROW, 64, 0, 0, 2),       # tiles overhang N and K; P = 80 B, G = 64 B
    (5, 40, 48, 2, 24, 20, COL, 64, 0, 0, 2),       # column pitch 96 B vs G = 64 B
    (5, 40, 48, 2, 24, 20, TILE, 64, 4, 8, 2),
    (3, 36, 30, 3, 10, 7, ROW, 48, 0, 0, 4),        # nothing divides anything
    (3, 36, 30, 3, 10, 7, COL, 48, 0, 0, 4),
    (3, 36, 30, 3, 10, 7, TILE, 48, 2, 6, 4),
    (7, 64, 64, 4, 32, 16, TILE, 128, 16, 4, 2),    # tall block, wider than nothing
    (7, 64, 64, 4, 8, 64, TILE, 256, 2, 64, 2),     # block wider than the tile
    (1, 64, 64, 1, 64, 64, ROW, 4096, 0, 0, 2),     # G larger than the whole pitch
]


@pytest.mark.parametrize("M,N,K,BM,BN,BK,layout,G,br,bc,s", TINY)
def test_matches_python_sets_on_tiny_inputs(M, N, K, BM, BN, BK, layout, G, br, bc, s):
    assert tlo.read_amp(M, N, K, BM, BN, BK, layout, G, br, bc, s) == \
        _python_count(M, N, K, BM, BN, BK, layout, G, br, bc, s)


@pytest.mark.parametrize("G", [32, 256, 1024, 4096, 16384])
@pytest.mark.parametrize("BN", [64, 128])
def test_closed_forms_under_power_of_two_alignment(G, BN):
    K, N, s, BK = 256, 8192, 2, 64
    P, w = N * s, BN * s
    f, u, _ = tlo.read_amp(1, N, K, 1, BN, BK, ROW, G, 0, 0, s)
    assert f * w == u * max(w, min(G, P))                           # RA_row = min(G, P) / w (>= 1)
    f, u, _ = tlo.read_amp(1, N, K, 1, BN, BK, COL, G, 0, 0, s)
    assert f * (BK * s) == u * max(BK * s, min(G, K * s))           # RA_col = min(G, K s) / (BK s)
    for br in (1, 8, 16, 32):
        bc = G // (br * s)
        if bc < 1 or bc > N or K % br:
            continue
        f, u, _ = tlo.read_amp(1, N, K, 1, BN, BK, TILE, G, br, bc, s)
        assert f * (BK * BN) == u * max(BK, br) * max(BN, bc)       # RA_tile


def test_config1_values():
    # 512 x 512 bf16, 64 x 64 x 64 CTA tile, M = 16: pitch 1 KB, so one 4 KB block holds 4 rows:
    # 64 rows -> 16 blocks = 64 KB fetched for 8 KB used, 64 tile loads.
    assert tlo.read_amp(16, 512, 512, 64, 64, 64, ROW, 4096, 0, 0, 2) == (4194304, 524288, 1024)
    f, u, _ = tlo.read_amp(16, 512, 512, 64, 64, 64, TILE, 4096, 16, 128, 2)    # block twice as wide as the tile
    assert (f, u) == (1048576, 524288)
    f, u, _ = tlo.read_amp(16, 512, 512, 64, 64, 64, TILE, 4096, 32, 64, 2)
    assert f == u == 524288
    f, u, _ = tlo.read_amp(16, 512, 512, 64, 128, 64, TILE, 4096, 16, 128, 2)
    assert f == u == 524288
    for layout, br, bc in ((ROW, 0, 0), (TILE, 1, 16), (TILE, 2, 8)):
        f, u, _ = tlo.read_amp(16, 512, 512, 64, 64, 64, layout, 32, br, bc, 2)
        assert f == u == 524288


@pytest.mark.parametrize("layout,br,bc", [(ROW, 0, 0), (COL, 0, 0), (TILE, 8, 32), (TILE, 32, 8)])
def test_invariants(layout, br, bc):
    N, K, BN, BK, G, s = 192, 160, 48, 40, 512, 2
    f1, u1, q1 = tlo.read_amp(1, N, K, 16, BN, BK, layout, G, br, bc, s)
    assert f1 >= u1 and f1 % G == 0 and f1 == q1 * G and u1 == K * N * s
    for M in (16, 17, 64, 65):
        mt = -(-M // 16)
        assert tlo.read_amp(M, N, K, 16, BN, BK, layout, G, br, bc, s) == (f1 * mt, u1 * mt, q1 * mt)
    assert tlo.read_amp(0, N, K, 16, BN, BK, layout, G, br, bc, s) == (0, 0, 0)


def test_tile_major_count_is_invariant_under_transposition():
    N, K, BN, BK, br, bc, s = 192, 160, 48, 40, 8, 32, 2
    a = tlo.read_amp(1, N, K, 1, BN, BK, TILE, br * bc * s, br, bc, s)
    b = tlo.read_amp(1, K, N, 1, BK, BN, TILE, br * bc * s, bc, br, s)
    assert a == b


def test_row_and_column_major_are_transposes_of_each_other():
    N, K, BN, BK, G, s = 192, 160, 48, 40, 256, 2
    assert tlo.read_amp(1, N, K, 1, BN, BK, ROW, G, 0, 0, s) == tlo.read_amp(1, K, N, 1, BK, BN, COL, G, 0, 0, s)


def test_per_tile_arrays_sum_to_totals():
    f, u, q, pf, pu = tlo.read_amp(40, 200, 96, 16, 64, 32, ROW, 128, 0, 0, 2, per_tile=True)
    assert pf.size == 3 * 4 and int(pf.sum()) == f and int(pu.sum()) == u
    assert np.array_equal(pf[:4], pf[4:8]) and np.array_equal(pu[:4], pu[8:])
    assert pu[3] == 96 * (200 - 192) * 2            # the last n-tile is clipped


def test_grouped_is_the_sum_over_experts_with_tokens():
    N, K, BM, BN, BK, G, br, bc, s = 256, 128, 16, 128, 64, 4096, 16, 128, 2
    offsets = np.array([0, 5, 5, 40, 41, 41, 100], dtype=np.int32)
    for layout in (ROW, TILE):
        want = [0, 0, 0]
        for e in range(offsets.size - 1):
            Me = int(offsets[e + 1] - offsets[e])
            got = tlo.read_amp(Me, N, K, BM, BN, BK, layout, G, br, bc, s)
            want = [x + y for x, y in zip(want, got)]
        assert list(tlo.read_amp_grouped(offsets, N, K, BM, BN, BK, layout, G, br, bc, s)) == want


def test_bad_arguments_are_rejected():
    with pytest.raises(ValueError):
        tlo.read_amp(1, 64, 64, 1, 64, 64, TILE, 4096, 16, 64, 2)      # 16*64*2 != 4096
    with pytest.raises(ValueError):
        tlo.read_amp(1, 60, 64, 1, 64, 64, TILE, 256, 8, 16, 2)        # N not a multiple of bc


def test_k_contiguous_flavour_counts_like_the_transposed_problem():
    # The paper's own example again (Section 6.5), now literally: K contiguous, memory tile (a, b) = (64, 32):
    # a 128 (K) x 256 (N) compute tile of a K = 4096 weight needs 16 requests; column-major needs 256
    # (one 4 KB block per column, pitch 8 KB).
    K, N, s, G = 4096, 512, 2, 4096
    f, u, q = tlo.read_amp(1, N, K, 1, 256, 128, tlo.TILE_MAJOR_K, G, 32, 64, s)
    loads = (N // 256) * (K // 128)
    assert q == 16 * loads and f == u
    assert tlo.read_amp(1, N, K, 1, 256, 128, COL, G, 0, 0, s)[2] == 256 * loads
    # transposition invariance ties the two flavours together
    # (the K x N weight with K contiguous IS an N x K matrix with its columns contiguous: same blocks, tile loads
    # with their two extents exchanged)
    assert tlo.read_amp(3, N, K, 2, 96, 80, tlo.TILE_MAJOR_K, 512, 8, 32, s) == \
        tlo.read_amp(3, K, N, 2, 80, 96, TILE, 512, 8, 32, s)


# ------------------------------------------------------------------ requests shared between co-resident CTAs
def test_shared_count_with_one_cta_per_wave_is_the_plain_count():
    for layout, br, bc in ((tlo.ROW_MAJOR, 0, 0), (tlo.COL_MAJOR, 0, 0), (tlo.TILE_MAJOR, 4, 16), (tlo.TILE_MAJOR_K, 8, 8)):
        M, N, K, cta, G, s = 70, 96, 64, (32, 24, 16), 128, 2
        f, u, q = tlo.read_amp(M, N, K, *cta, layout, G, br, bc, s)
        assert tlo.read_amp_shared(M, N, K, *cta, 1, layout, G, br, bc, s) == (f, u, q)


def test_shared_count_hand_worked_row_major():
    # 4 x 16 matrix of bytes, G = 8: every row is two blocks.  CTA tiles 4 columns wide, 2 rows deep, one m-tile.
    # Alone, each of the 4 n-tiles fetches 2 rows x 1 block per K step: 4 tiles x 2 steps x 2 = 16 blocks.
    # Two tiles per wave: tiles 0,1 both live in columns 0-7 -> the same block per row: 2 waves x 2 steps x 2 = 8.
    # All four together: each row's two blocks once: 2 steps x 2 rows x 2 blocks = 8 as well.
    args = (1, 16, 4, 1, 4, 2)
    assert tlo.read_amp_shared(*args, 1, tlo.ROW_MAJOR, 8, 0, 0, 1) == (16 * 8, 4 * 16, 16)
    assert tlo.read_amp_shared(*args, 2, tlo.ROW_MAJOR, 8, 0, 0, 1) == (8 * 8, 4 * 16, 8)
    assert tlo.read_amp_shared(*args, 4, tlo.ROW_MAJOR, 8, 0, 0, 1) == (8 * 8, 4 * 16, 8)
    # three m-tiles over the same weights, wave of 3 = one n-tile's three CTAs: fetched once, not three times
    assert tlo.read_amp_shared(3, 16, 4, 1, 4, 2, 3, tlo.ROW_MAJOR, 8, 0, 0, 1) == (16 * 8, 4 * 16, 16)
    assert tlo.read_amp(3, 16, 4, 1, 4, 2, tlo.ROW_MAJOR, 8, 0, 0, 1)[0] == 3 * 16 * 8


@pytest.mark.parametrize("P", [1, 3, 8, 1000])
def test_shared_count_closed_forms(P):
    M, N, K, s, G = 256, 1024, 256, 2, 4096
    cta = (128, 256, 128)
    # tile-major with tiles inside the CTA tile: every fetched byte is needed, however the waves fall
    f, u, q = tlo.read_amp_shared(M, N, K, *cta, P, tlo.TILE_MAJOR, G, 16, 128, s)
    assert f == u
    f, u, q = tlo.read_amp_shared(M, N, K, *cta, P, tlo.TILE_MAJOR_K, G, 32, 64, s)
    assert f == u
    # row-major, pitch 2 KB: a 4 KB block is two whole rows.  A wave covering every n-tile needs whole rows: ratio 1.
    f, u, q = tlo.read_amp_shared(M, N, K, *cta, P, tlo.ROW_MAJOR, G, 0, 0, s)
    if P >= 8:
        assert f == u == K * N * s
    else:
        assert u < f <= tlo.read_amp(M, N, K, *cta, tlo.ROW_MAJOR, G, 0, 0, s)[0]
    # never more than without sharing, never less than what is needed
    for layout, br, bc in ((tlo.ROW_MAJOR, 0, 0), (tlo.COL_MAJOR, 0, 0)):
        fs, us, _ = tlo.read_amp_shared(M, N, K, *cta, P, layout, G, br, bc, s)
        assert us <= fs <= tlo.read_amp(M, N, K, *cta, layout, G, br, bc, s)[0]


def test_prefetch_degree_satisfies_the_inequality_it_is_derived_from():
    # Eq. 6: the largest d with p_wave * d <= B*L (so that p_wave * (d + 1) >= B*L), capped at K / TILE_K
    B, L, G = 4.9e12, 5e-6, 4096
    BL = B * L / G
    for n_sm, c_sm, p_tile, K, tk in [(132, 1, 16, 2048, 128), (132, 1, 128, 2048, 128), (148, 2, 16, 8192, 64),
                                      (8, 1, 4, 65536, 64), (1, 1, 1, 1 << 20, 64)]:
        p_wave = n_sm * c_sm * p_tile
        d = tlo.prefetch_degree(B, L, G, n_sm, c_sm, p_tile, K, tk)
        cap = K // tk
        assert 0 <= d <= cap
        if d < cap:
            assert p_wave * d <= BL < p_wave * (d + 1)
        else:
            assert p_wave * cap <= BL
        assert tlo.prefetch_degree(B, L, G, n_sm, c_sm, p_tile, K, tk, 2.0) >= d      # "in practice": first term doubled
    # as thread blocks retire p_wave shrinks and d grows (Section 5.2)
    ds = [tlo.prefetch_degree(B, L, G, n, 1, 16, 1 << 20, 64) for n in (132, 66, 33, 8, 1)]
    assert ds == sorted(ds) and ds[0] < ds[-1]
    # 8x more requests per tile (row-major, Section 6.5) leaves no room for prefetching on the same bus
    assert tlo.prefetch_degree(B, L, G, 132, 1, 128, 2048, 128) == 0 < tlo.prefetch_degree(B, L, G, 132, 1, 16, 2048, 128)
