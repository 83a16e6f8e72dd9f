"""Pins for the oracle's layout map and relayout (CPU only).

Each test ties the oracle to something other than itself: an equation of the
paper evaluated by hand, a printed example, an invariant, or a special case
that reduces to a plain copy.
"""
import json
import os

import numpy as np
import pytest

import oracle as tlo
from paper_2607_04031_b200 import inputs

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_values.json")))

CASES = [  # rows, cols, s, br, bc
    (8, 8, 1, 2, 4),
    (32, 64, 2, 16, 16),
    (48, 40, 1, 4, 8),
    (64, 256, 2, 16, 128),
    (96, 192, 4, 32, 32),
    (12, 20, 2, 3, 5),          # the oracle itself does not need powers of two
    (64, 64, 2, 8, 2),
    (64, 64, 2, 16, 1),
]


@pytest.mark.parametrize("rows,cols,s,br,bc", CASES)
def test_tile_map_is_a_bijection_onto_the_buffer(rows, cols, s, br, bc):
    offs = np.array([[tlo.off_tile(r, c, rows, cols, br, bc, s) for c in range(cols)] for r in range(rows)])
    assert offs.min() == 0 and offs.max() == (rows * cols - 1) * s
    assert np.all(offs % s == 0)
    assert np.unique(offs).size == rows * cols


@pytest.mark.parametrize("rows,cols,s,br,bc", CASES)
def test_every_G_block_is_one_br_by_bc_rectangle(rows, cols, s, br, bc):
    # Section 3: the contiguous G-byte unit is a 2-D rectangle of the matrix.
    G = br * bc * s
    members = {}
    for r in range(rows):
        for c in range(cols):
            members.setdefault(tlo.off_tile(r, c, rows, cols, br, bc, s) // G, []).append((r, c))
    assert len(members) == (rows // br) * (cols // bc)
    for q, rc in members.items():
        rs = sorted({r for r, _ in rc})
        cs = sorted({c for _, c in rc})
        assert len(rc) == br * bc
        assert rs == list(range(rs[0], rs[0] + br)) and rs[0] % br == 0
        assert cs == list(range(cs[0], cs[0] + bc)) and cs[0] % bc == 0
        # tiles are packed along the contiguous direction first
        assert q == (rs[0] // br) * (cols // bc) + cs[0] // bc


def test_hand_worked_offsets_of_eq2():
    # Eq. 2 by hand for the 8 x 8 example of Figure 4(a): K = N = 8, memory tile a x b = 4 x 2, s = 1.
    # (i,j)=(0,0): tile 0, intra 0 -> 0.     (1,0): intra i'=1 -> 1.
    # (0,1): j'=1 -> 1*4 = 4.                (4,0): T_i=1 -> tile 1 -> 8.
    # (0,2): T_j=1 -> tile (1*2+0)=2 -> 16.  (5,3): T_i=1,i'=1,T_j=1,j'=1 -> (1*2+1)*8 + (1*4+1) = 29.
    # (7,7): T_i=1,i'=3,T_j=3,j'=1 -> (3*2+1)*8 + (4+3) = 63.
    hand = {(0, 0): 0, (1, 0): 1, (0, 1): 4, (4, 0): 8, (0, 2): 16, (5, 3): 29, (7, 7): 63}
    for (i, j), want in hand.items():
        assert tlo.eq2(i, j, 8, 8, 4, 2, 1) == want
        # the exchanged (N-contiguous) flavour on the transposed problem gives the same bytes
        assert tlo.off_tile(j, i, 8, 8, 2, 4, 1) == want
    # with s = 2 every offset doubles
    assert tlo.eq2(5, 3, 8, 8, 4, 2, 2) == 58


def test_hand_worked_offsets_row_flavour():
    # 4 x 8 matrix, memory tile 2 rows x 4 contiguous columns, s = 2 (G = 16 B):
    # tiles are [rows 0-1 | cols 0-3], [rows 0-1 | cols 4-7], [rows 2-3 | cols 0-3], [rows 2-3 | cols 4-7].
    # (r,c)=(1,5): tile 1, intra (1,1) -> 1*16 + (1*4+1)*2 = 26.   (3,2): tile 2, intra (1,2) -> 32 + 12 = 44.
    assert tlo.off_tile(1, 5, 4, 8, 2, 4, 2) == 26
    assert tlo.off_tile(3, 2, 4, 8, 2, 4, 2) == 44
    assert tlo.off_row(3, 2, 4, 8, 2) == (3 * 8 + 2) * 2
    assert tlo.off_col(3, 2, 4, 8, 2) == (2 * 4 + 3) * 2


@pytest.mark.parametrize("K,N,a,b,s", [(8, 8, 4, 2, 1), (64, 32, 16, 8, 2), (384, 128, 128, 64, 1), (24, 18, 6, 3, 4)])
def test_eq2_literal_equals_exchanged_flavour_and_eq3(K, N, a, b, s):
    # Section 3.2: "the same approach applies to row-major, with rows and columns swapped".
    for i in range(K):
        for j in range(0, N, max(1, N // 16)):
            e2 = tlo.eq2(i, j, K, N, a, b, s)
            assert e2 == tlo.off_tile(j, i, N, K, b, a, s)
            assert e2 == tlo.eq3(i, j, K, N, a, b, s)          # Eq. 3: 4-D coordinate . stride


def test_eq4_tile_base_closed_form():
    # Eq. 4: for i a multiple of a and j a multiple of b, offset = (K*j + i*b)*s.
    K, N, a, b, s = 256, 128, 32, 16, 2
    for i in range(0, K, a):
        for j in range(0, N, b):
            assert tlo.eq2(i, j, K, N, a, b, s) == (K * j + i * b) * s


def test_printed_view_example():
    v = GOLD["view_example"]
    i, j = v["coord_2d"]
    assert list(tlo.eq1(i, j, v["a"], v["b"])) == v["coord_4d"]
    assert [v["a"], v["b"], v["K"] // v["a"], v["N"] // v["b"]] == v["shape_4d"]


def test_printed_case2_bit_layout():
    # Section 4.3, Case 2: inside a 128 x 32 FP8 memory tile the 12 offset bits are col(5) | sub-tile(2) | row(5):
    # the 7-bit intra-tile row index i' splits into sub-tile (high 2) and row (low 5).
    g = GOLD["case2_bit_layout"]
    a, b, s = g["a"], g["b"], g["elem_bytes"]
    assert a * b * s == 4096
    K, N = 4 * a, 2 * b
    for ip in (0, 1, 31, 32, 0b1100101, 127):
        for jp in (0, 1, 0b10011, 31):
            col, sub, row = jp, ip >> 5, ip & 31
            want = (col << 7) | (sub << 5) | row
            assert tlo.eq2(ip, jp, K, N, a, b, s) == want                 # tile (0,0)
            assert tlo.eq2(a + ip, b + jp, K, N, a, b, s) % 4096 == want  # any tile: low 12 bits
    assert ((0b10011 << 7) | (0b11 << 5) | 0b00101) == 2533
    assert tlo.eq2(0b1100101, 0b10011, K, N, a, b, s) == 2533


def test_fp8_extreme_shapes_are_row_and_column_major():
    # Section 3.1: for FP8, (1, 4096) is row-major and (4096, 1) column-major.
    rows, cols, s = 4096, 4096, 1
    pts = [(0, 0), (1, 0), (0, 1), (17, 4095), (4095, 33), (2048, 2048)]
    for r, c in pts:
        assert tlo.off_tile(r, c, rows, cols, 1, 4096, s) == tlo.off_row(r, c, rows, cols, s)
        # a 4096 x 1 tile: each tile is one column's worth of 4096 rows -> column-major
        # only when the tiles themselves run down the columns; with tiles ordered along
        # the contiguous direction first the tile index is T_r*cols + c, here T_r = 0.
        assert tlo.off_tile(r, c, rows, cols, 4096, 1, s) == c * 4096 + r == tlo.off_col(r, c, rows, cols, s)


@pytest.mark.parametrize("rows,cols,s,br,bc", CASES)
def test_round_trip_is_identity(rows, cols, s, br, bc):
    src = inputs.random_bytes(rows * cols * s, seed=rows * 131 + cols)
    tiled = tlo.relayout(src, rows, cols, s, br, bc, tlo.TO_TILE_MAJOR)
    back = tlo.relayout(tiled, rows, cols, s, br, bc, tlo.TO_ROW_MAJOR)
    assert np.array_equal(back, src)
    assert np.array_equal(np.sort(tiled), np.sort(src))
    if br > 1 and bc < cols:
        assert not np.array_equal(tiled, src)


@pytest.mark.parametrize("rows,cols,s", [(16, 64, 2), (5, 48, 1), (7, 12, 4)])
def test_degenerate_tiles_reduce_to_a_plain_copy(rows, cols, s):
    src = inputs.random_bytes(rows * cols * s, seed=99)
    for bc in (cols, cols // 2, cols // 4):       # one-row tiles: the layout is row-major
        assert np.array_equal(tlo.relayout(src, rows, cols, s, 1, bc, tlo.TO_TILE_MAJOR), src)
    # full-width tiles of any height: also row-major
    assert np.array_equal(tlo.relayout(src, rows, cols, s, rows, cols, tlo.TO_TILE_MAJOR), src)


def test_relayout_matches_numpy_block_transpose():
    # A tile-major buffer is the 4-D array [rows/br][cols/bc][br][bc]; numpy's reshape/transpose
    # builds it without any offset arithmetic.
    rows, cols, br, bc = 64, 96, 16, 32
    src = np.arange(rows * cols, dtype=np.uint16)
    want = src.reshape(rows // br, br, cols // bc, bc).transpose(0, 2, 1, 3).reshape(-1)
    got = tlo.relayout(src.view(np.uint8), rows, cols, 2, br, bc, tlo.TO_TILE_MAJOR).view(np.uint16)
    assert np.array_equal(got, want)


def test_relayout_rejects_non_divisible_shapes():
    src = np.zeros(10 * 10, dtype=np.uint8)
    with pytest.raises(ValueError):
        tlo.relayout(src, 10, 10, 1, 4, 2, tlo.TO_TILE_MAJOR)


def test_k_contiguous_flavour_is_eq2_and_the_transposed_relayout():
    # Layout code TILE_MAJOR_K: the weight exactly as the paper prints it (K contiguous, a along K, b along N).
    K, N, a, b, s = 64, 48, 16, 8, 2
    for i in (0, 1, 15, 16, 63):
        for j in (0, 7, 8, 47):
            assert tlo.off(tlo.TILE_MAJOR_K, i, j, K, N, b, a, s) == tlo.eq2(i, j, K, N, a, b, s)
    # relayout of the [N][K] array (K contiguous) with blocks of b rows x a columns produces that buffer
    w = np.arange(K * N, dtype=np.uint16).reshape(N, K)            # w[j][i]: element (i, j)
    buf = tlo.relayout(w.view(np.uint8), N, K, 2, b, a, tlo.TO_TILE_MAJOR).view(np.uint16)
    for i in range(0, K, 5):
        for j in range(0, N, 7):
            assert buf[tlo.off(tlo.TILE_MAJOR_K, i, j, K, N, b, a, s) // 2] == w[j, i]
