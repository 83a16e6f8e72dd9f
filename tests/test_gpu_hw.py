"""Tile-major aware box loads (Section 4.3) through the C ABI vs the oracle (GPU): offsets bit-exact, loaded bytes
equal to the logical tile of the column-major matrix."""
import json
import os

import numpy as np
import pytest
import torch

import oracle as tlo
from paper_2607_04031_b200 import inputs

pytestmark = pytest.mark.gpu
GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_values.json")))


def _offsets(dims, strides, box, s, a, b, K, coords_list):
    from gpu_util import DEV, tl
    d = tl.hw_desc(dims, strides, box, s, a, b, K)
    c = torch.tensor(coords_list, dtype=torch.int32, device=DEV).reshape(len(coords_list), len(dims))
    n = int(np.prod(box))
    out = torch.empty(len(coords_list) * n, dtype=torch.int64, device=DEV)
    tl.hw_box_offsets(d, c, out)
    tl.device_status()
    return out.cpu().numpy().reshape(len(coords_list), n)


def test_printed_views_offsets_match_the_oracle():
    v = GOLD["view_example"]
    K, a, b = v["K"], v["a"], v["b"]
    for name in ("2d", "3d", "4d"):
        w = v["views"][name]
        got = _offsets(w["tensor"], w["strides_derived"], w["tile"], 1, a, b, K, [w["coords"]])[0]
        want = tlo.hw_box_offsets(tlo.hw_desc(w["tensor"], w["strides_derived"], w["tile"], 1, a, b, K), w["coords"])
        assert np.array_equal(got, want)


def test_case2_offsets_match_the_oracle():
    g = GOLD["case2_bit_layout"]
    a, b, s = g["a"], g["b"], g["elem_bytes"]
    u, v = g["tma_tile"]
    K, N = 4 * a, 2 * b
    coords = [[Ti * a + sub * u, Tj * b] for Ti in range(4) for sub in range(4) for Tj in range(2)]
    got = _offsets([K, N], [1, K], [u, v], s, a, b, K, coords)
    d = tlo.hw_desc([K, N], [1, K], [u, v], s, a, b, K)
    for c, row in zip(coords, got):
        assert np.array_equal(row, tlo.hw_box_offsets(d, c))


def _views(rng, n):
    out = []
    while len(out) < n:
        a = int(rng.choice([16, 32, 64, 128])); b = int(rng.choice([4, 8, 16, 32])); s = int(rng.choice([1, 2, 4]))
        u = int(rng.choice([x for x in (8, 16, 32, 64, 128) if x <= a]))
        K = a * int(rng.integers(2, 6)); N = b * int(rng.integers(2, 6))
        rows0 = int(rng.choice([x for x in (u, 2 * u, K) if K % x == 0]))
        cols0 = int(rng.choice([x for x in (b, 2 * b, N) if N % x == 0]))
        dims, strides = [rows0, cols0], [1, K]
        if rows0 < K:
            dims.append(K // rows0); strides.append(rows0)
        if cols0 < N:
            dims.append(N // cols0); strides.append(cols0 * K)
        order = [0] + list(rng.permutation(np.arange(1, len(dims))))
        dims, strides = [dims[k] for k in order], [strides[k] for k in order]
        box = []
        for dm, st in zip(dims, strides):
            box.append(u if st == 1 else (b * int(rng.integers(1, dm // b + 1)) if st == K else int(rng.integers(1, dm + 1))))
        coords = []
        for _ in range(5):
            c = []
            for dm, st, bx in zip(dims, strides, box):
                if st == 1:
                    c.append(int(rng.integers(0, dm // u)) * u)
                elif st == K:
                    c.append(int(rng.integers(0, (dm - bx) // b + 1)) * b)
                else:
                    c.append(int(rng.integers(0, dm - bx + 1)))
            coords.append(c)
        out.append((dims, strides, box, s, a, b, K, N, coords))
    return out


def test_random_views_offsets_and_loaded_bytes():
    from gpu_util import DEV, tl
    rng = np.random.default_rng(11)
    for dims, strides, box, s, a, b, K, N, coords in _views(rng, 60):
        got = _offsets(dims, strides, box, s, a, b, K, coords)
        od = tlo.hw_desc(dims, strides, box, s, a, b, K)
        for c, row in zip(coords, got):
            assert np.array_equal(row, tlo.hw_box_offsets(od, c)), (dims, strides, box, c, a, b, s)
        # the loads: tile-major buffer made by the library's relayout from the [N][K] array
        mat = inputs.random_bytes(N * K * s, seed=K + N)                    # column-major K x N = [N][K] bytes
        src = torch.from_numpy(mat).to(DEV)
        tiled = torch.empty_like(src)
        tl.relayout(src, tiled, N, K, s, a * b * s, b, a, tl.TO_TILE_MAJOR)
        n = int(np.prod(box))
        dst = torch.full((len(coords) * n * s,), 0xEE, dtype=torch.uint8, device=DEV)
        cd = torch.tensor(coords, dtype=torch.int32, device=DEV)
        tl.hw_box_load(tl.hw_desc(dims, strides, box, s, a, b, K), tiled, cd, dst)
        tl.device_status()
        dst = dst.cpu().numpy().reshape(len(coords), n, s)
        elems = mat.reshape(N * K, s)
        for ci, c in enumerate(coords):
            # logical element offsets of the box in the column-major matrix, dimension 0 fastest
            grid = np.zeros([1] * len(dims), dtype=np.int64)
            for dm in range(len(dims)):
                shape = [1] * len(dims)
                shape[len(dims) - 1 - dm] = box[dm]
                grid = grid + ((c[dm] + np.arange(box[dm])) * strides[dm]).reshape(shape)
            want = elems[grid.reshape(-1)]
            assert np.array_equal(dst[ci], want)


def test_gemm_schedule_boxes_full_size():
    # every weight-tile load of a 128 (K) x 256 (N) compute tile over the Qwen gate_up weight, bf16, (64, 32) tiles:
    # 2 boxes of u = 64 per tile row-block... here as 64 x 256 boxes (case 1, v = 8 memory tiles)
    from gpu_util import DEV, tl
    K, N, s, a, b = 2048, 1536, 2, 64, 32
    w = inputs.bf16_normal((N, K), 0.02, seed=9, device=DEV)                # [N][K]
    tiled = torch.empty_like(w)
    tl.relayout(w, tiled, N, K, s, 4096, b, a, tl.TO_TILE_MAJOR)
    box = [64, 256]
    coords = [[i, j] for j in range(0, N, 256) for i in range(0, K, 64)]
    cd = torch.tensor(coords, dtype=torch.int32, device=DEV)
    dst = torch.empty((len(coords), 256, 64), dtype=torch.bfloat16, device=DEV)
    tl.hw_box_load(tl.hw_desc([K, N], [1, K], box, s, a, b, K), tiled, cd, dst)
    tl.device_status()
    want = w.reshape(N // 256, 256, K // 64, 64).permute(0, 2, 1, 3).reshape(len(coords), 256, 64)
    assert torch.equal(dst, want)


def test_bad_coordinates_raise_the_status_word_and_unsupported_descriptors_are_refused():
    from gpu_util import DEV, tl
    K, N, a, b = 256, 64, 32, 8
    d = tl.hw_desc([K, N], [1, K], [32, 16], 1, a, b, K)
    c = torch.tensor([[16, 8], [32, 8]], dtype=torch.int32, device=DEV)     # first box: row not tile-aligned
    out = torch.zeros(2 * 32 * 16, dtype=torch.int64, device=DEV)
    tl.hw_box_offsets(d, c, out)
    with pytest.raises(tl.TileLensError) as e:
        tl.device_status()
    assert e.value.status == 5 and "0x900" in str(e.value)
    o = out.cpu().numpy().reshape(2, -1)
    assert np.all(o[0] == -1)
    assert np.array_equal(o[1], tlo.hw_box_offsets(tlo.hw_desc([K, N], [1, K], [32, 16], 1, a, b, K), [32, 8]))
    tl.device_status()                                                      # the word was cleared
    with pytest.raises(tl.TileLensError) as e:
        tl.hw_box_offsets(tl.hw_desc([K, N], [1, K], [64, 16], 1, a, b, K), c, out)      # u > a
    assert e.value.status == 2
    with pytest.raises(tl.TileLensError) as e:
        tl.hw_box_offsets(tl.hw_desc([K, N], [1, K], [32, 12], 1, a, b, K), c, out)      # v not a multiple of b
    assert e.value.status == 2
