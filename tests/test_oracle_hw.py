"""Pins for the oracle's TileLens-HW address generation (Section 4.3; CPU only).

The emulator produces addresses with counters, the way the section describes the engine; the pins compare them
with Eq. 2 evaluated element by element (itself pinned by hand-worked values in test_oracle_layout.py), with the
closed form of Eq. 4, with the printed views and with the printed Case-2 bit layout.
"""
import itertools
import json
import os

import numpy as np
import pytest

import oracle as tlo

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_values.json")))


def eq2_addresses(dims, strides, box, coords, K, N, a, b, s):
    """Eq. 2 at the logical (i, j) of every element of the box, dimension 0 fastest."""
    out = []
    for x in itertools.product(*[range(v) for v in reversed(box)]):
        x = x[::-1]
        lin = sum((c + xi) * st for c, xi, st in zip(coords, x, strides))      # element offset in the column-major matrix
        i, j = lin % K, lin // K
        assert j < N
        out.append(tlo.eq2(i, j, K, N, a, b, s))
    return np.array(out, dtype=np.int64)


def test_the_three_printed_views_generate_the_same_eq2_addresses():
    v = GOLD["view_example"]
    K, N, a, b, s = v["K"], v["N"], v["a"], v["b"], 1
    traces = []
    for name in ("2d", "3d", "4d"):
        w = v["views"][name]
        d = tlo.hw_desc(w["tensor"], w["strides_derived"], w["tile"], s, a, b, K)
        got = tlo.hw_box_offsets(d, w["coords"])
        want = eq2_addresses(w["tensor"], w["strides_derived"], w["tile"], w["coords"], K, N, a, b, s)
        assert np.array_equal(got, want)
        traces.append(got)
    assert np.array_equal(traces[0], traces[1]) and np.array_equal(traces[0], traces[2])
    # a == u and v == b: the 128 x 64 box is exactly one memory tile, read front to back
    assert np.array_equal(traces[0], traces[0][0] + np.arange(128 * 64))
    # Eq. 4 at the printed coordinates: (K*j + i*b)*s
    assert traces[0][0] == (384 * 64 + 256 * 64) * 1


@pytest.mark.parametrize("s", [1, 2, 4])
def test_tile_base_is_eq4(s):
    K, N, a, b = 512, 256, 64, 16
    d = tlo.hw_desc([K, N], [1, K], [a, b], s, a, b, K)
    for i in range(0, K, a):
        for j in range(0, N, 4 * b):
            assert tlo.hw_box_offsets(d, [i, j])[0] == (K * j + i * b) * s


def test_case2_printed_bit_permutation():
    g = GOLD["case2_bit_layout"]
    a, b, s = g["a"], g["b"], g["elem_bytes"]
    u, v = g["tma_tile"]
    K, N = 4 * a, 2 * b
    d = tlo.hw_desc([K, N], [1, K], [u, v], s, a, b, K)
    # the TMA tile that is sub-tile 3 of memory tile (T_i, T_j) = (1, 1)
    sub, Ti, Tj = 3, 1, 1
    got = tlo.hw_box_offsets(d, [Ti * a + sub * u, Tj * b])
    want = eq2_addresses([K, N], [1, K], [u, v], [Ti * a + sub * u, Tj * b], K, N, a, b, s)
    assert np.array_equal(got, want)
    # element (row 5, col 19) of that TMA tile: low 12 bits are (col | sub-tile | row) = 10011 11 00101
    t = 19 * u + 5                                   # counter order: dimension 0 (rows of the tile) fastest
    assert got[t] % 4096 == ((19 << 7) | (3 << 5) | 5) == 2533
    # without the permutation the engine, working as if tiles were 32 x 32, would have produced (sub | col | row)
    as_if = tlo.hw_box_offsets(tlo.hw_desc([K, N], [1, K], [u, v], s, u, b, K), [Ti * a + sub * u, Tj * b])
    assert as_if[t] % 4096 == ((3 << 10) | (19 << 5) | 5)


def _random_view(rng, K, N, a, b, u):
    """A random view of the column-major K x N matrix: rows split into (u-chunk, chunks), columns into (b-groups...)."""
    # row direction: dim 0 holds r0 rows (multiple of u), an optional second row dimension the chunks
    r0 = int(rng.choice([x for x in (u, 2 * u, 4 * u, K) if x <= K and K % x == 0]))
    c0 = int(rng.choice([x for x in (b, 2 * b, N) if x <= N and N % x == 0]))
    dims, strides = [r0, c0], [1, K]
    if r0 < K:
        dims.append(K // r0); strides.append(r0)
    if c0 < N:
        dims.append(N // c0); strides.append(c0 * K)
    order = [0] + list(rng.permutation(np.arange(1, len(dims))))
    dims, strides = [dims[k] for k in order], [strides[k] for k in order]
    box, coords = [], []
    for dm, st in zip(dims, strides):
        if st == 1:
            box.append(u); coords.append(int(rng.integers(0, dm // u)) * u)
        elif st == K:
            v = b * int(rng.integers(1, dm // b + 1)); box.append(v)
            coords.append(int(rng.integers(0, (dm - v) // b + 1)) * b)
        else:
            e = int(rng.integers(1, dm + 1)); box.append(e); coords.append(int(rng.integers(0, dm - e + 1)))
    return dims, strides, box, coords


def test_brute_force_random_views_against_eq2():
    rng = np.random.default_rng(7)
    n_case2 = 0
    for _ in range(300):
        a = int(rng.choice([4, 8, 16])); b = int(rng.choice([2, 4, 8])); s = int(rng.choice([1, 2, 4]))
        u = int(rng.choice([x for x in (2, 4, 8, 16) if x <= a]))
        K = a * int(rng.integers(1, 5)); N = b * int(rng.integers(1, 5))
        dims, strides, box, coords = _random_view(rng, K, N, a, b, u)
        # row-direction coordinates must land on memory-tile boundaries of the pretended u x b tile: they do
        d = tlo.hw_desc(dims, strides, box, s, a, b, K)
        got = tlo.hw_box_offsets(d, coords)
        want = eq2_addresses(dims, strides, box, coords, K, N, a, b, s)
        assert np.array_equal(got, want), (dims, strides, box, coords, a, b, u, s)
        n_case2 += u < a
    assert n_case2 > 50


def test_aligned_box_touches_only_its_own_blocks():
    # Case 1, 4 KB tiles: a box of u x v elements reads exactly u*v*s/G whole blocks (read amplification 1);
    # every run of u elements is one contiguous request.
    K, N, a, b, s = 1024, 256, 128, 16, 2
    d = tlo.hw_desc([K, N], [1, K], [128, 64], s, a, b, K)
    off = tlo.hw_box_offsets(d, [256, 128])
    blocks = np.unique(off // 4096)
    assert blocks.size == 128 * 64 * s // 4096
    rows = off.reshape(64, 128)
    assert np.all(np.diff(rows, axis=1) == s)


def test_descriptors_the_section_does_not_cover_are_rejected():
    K, N, a, b = 256, 64, 32, 8
    ok = tlo.hw_desc([K, N], [1, K], [32, 16], 1, a, b, K)
    tlo.hw_box_offsets(ok, [32, 8])
    with pytest.raises(ValueError):
        tlo.hw_box_offsets(tlo.hw_desc([K, N], [1, K], [64, 16], 1, a, b, K), [0, 0])      # u > a
    with pytest.raises(ValueError):
        tlo.hw_box_offsets(tlo.hw_desc([K, N], [1, K], [32, 12], 1, a, b, K), [0, 0])      # v not a multiple of b
    with pytest.raises(ValueError):
        tlo.hw_box_offsets(ok, [16, 8])                                                    # row not tile-aligned
    with pytest.raises(ValueError):
        tlo.hw_box_offsets(ok, [32, 4])                                                    # column not tile-aligned
    with pytest.raises(ValueError):                                                        # stride 2K with b = 8
        tlo.hw_box_offsets(tlo.hw_desc([K, 2, N // 2], [1, K, 2 * K], [32, 2, 4], 1, a, b, K), [0, 0, 0])
