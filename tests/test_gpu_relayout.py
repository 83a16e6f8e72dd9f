"""Relayout kernel vs the oracle: bit-exact (GPU)."""
import numpy as np
import pytest
import torch

import oracle as tlo
from paper_2607_04031_b200 import inputs

pytestmark = pytest.mark.gpu

CASES = [  # rows, cols, s, br, bc
    (512, 512, 2, 16, 128),        # config 1
    (512, 512, 2, 32, 64),
    (512, 512, 2, 8, 256),
    (512, 512, 2, 1, 2048 // 4),   # one-row blocks: identity
    (256, 1024, 1, 64, 64),        # FP8 64 x 64 (Figure 1c)
    (256, 1024, 4, 8, 128),
    (96, 640, 2, 16, 16),          # 32-byte runs
    (512, 256, 2, 256, 8),         # 16-byte runs of a 4 KB tile: shared-memory kernel, not the copy engine
    (1056, 2176, 1, 32, 16),       # 16-byte runs, tiles overhang both edges
    (64, 256, 2, 8, 2),            # 4-byte runs: vectors gathered from 4 block rows
    (64, 256, 2, 16, 1),           # 2-byte runs
    (64, 256, 1, 32, 1),           # 1-byte runs
    (128, 64, 4, 32, 2),           # 8-byte runs
    (48, 40, 1, 4, 8),             # 40-byte pitch: element-wise fallback
    (24, 20, 2, 4, 2),             # G = 16, pitch 40 B
    (16, 8, 2, 2, 2),              # G = 8 < 16: element-wise
    (1056, 2176, 2, 32, 64),       # tiles overhang both edges (1056 = 33*32, 2176 = 17*128)
    (32, 8192, 2, 1, 2048),        # block row of 4 KB, wider than a tile
    (64, 16384, 2, 32, 8192 // 2 // 1),  # 16 KB rows: bc = 4096 -> G = 256 KB
    (8192, 16, 1, 4096, 1),        # column-major-like: 4096 x 1 blocks
]


@pytest.mark.parametrize("rows,cols,s,br,bc", CASES)
def test_both_directions_match_oracle(rows, cols, s, br, bc):
    from gpu_util import DEV, Guarded, dev_bytes, tl
    G = br * bc * s
    src = inputs.random_bytes(rows * cols * s, seed=rows + 7 * cols + s)
    want = tlo.relayout(src, rows, cols, s, br, bc, tlo.TO_TILE_MAJOR)
    d_src = dev_bytes(src)
    g_dst = Guarded((rows * cols * s,), torch.uint8)       # outputs sit between guard blocks, checked after the call
    tl.relayout(d_src, g_dst.t, rows, cols, s, G, br, bc, tl.TO_TILE_MAJOR)
    d_dst = g_dst.check()
    got = d_dst.cpu().numpy()
    assert np.array_equal(got, want)
    g_back = Guarded((rows * cols * s,), torch.uint8)
    tl.relayout(d_dst, g_back.t, rows, cols, s, G, br, bc, tl.TO_ROW_MAJOR)
    assert np.array_equal(g_back.check().cpu().numpy(), src)
    # the inverse direction on its own, from the oracle's tile-major bytes
    d_t = dev_bytes(want)
    g_r = Guarded((rows * cols * s,), torch.uint8)
    tl.relayout(d_t, g_r.t, rows, cols, s, G, br, bc, tl.TO_ROW_MAJOR)
    assert np.array_equal(g_r.check().cpu().numpy(), tlo.relayout(want, rows, cols, s, br, bc, tlo.TO_ROW_MAJOR))


def test_unaligned_pointers_take_the_elementwise_path():
    from gpu_util import DEV, dev_bytes, tl
    rows, cols, s, br, bc = 64, 128, 2, 16, 64
    src = inputs.random_bytes(rows * cols * s, seed=5)
    buf = torch.zeros(rows * cols * s + 64, dtype=torch.uint8, device=DEV)
    d_src = buf[2:2 + rows * cols * s]
    d_src.copy_(torch.from_numpy(src))
    d_dst = torch.zeros(rows * cols * s, dtype=torch.uint8, device=DEV)
    tl.relayout(d_src, d_dst, rows, cols, s, br * bc * s, br, bc, tl.TO_TILE_MAJOR)
    assert np.array_equal(d_dst.cpu().numpy(), tlo.relayout(src, rows, cols, s, br, bc, tlo.TO_TILE_MAJOR))


def test_full_size_llama_weight_matches_oracle():
    from gpu_util import DEV, tl
    K, N, br, bc = 8192, 8192, 16, 128
    B = inputs.bf16_normal((K, N), 0.02, seed=21, device=DEV)
    out = torch.empty_like(B)
    tl.relayout(B, out, K, N, 2, 4096, br, bc, tl.TO_TILE_MAJOR)
    want = tlo.relayout(inputs.bits(B).view(np.uint8), K, N, 2, br, bc, tlo.TO_TILE_MAJOR)
    assert np.array_equal(out.cpu().view(torch.uint8).numpy().reshape(-1), want)
    back = torch.empty_like(B)
    tl.relayout(out, back, K, N, 2, 4096, br, bc, tl.TO_ROW_MAJOR)
    assert torch.equal(back, B)


def test_errors():
    from gpu_util import DEV, tl
    a = torch.zeros(64 * 64 * 2, dtype=torch.uint8, device=DEV)
    b = torch.zeros_like(a)
    with pytest.raises(tl.TileLensError) as e:
        tl.relayout(a, b, 64, 64, 2, 4096, 16, 64, tl.TO_TILE_MAJOR)
    assert e.value.status == 1
    with pytest.raises(tl.TileLensError) as e:
        tl.relayout(a, a, 64, 64, 2, 2048, 16, 64, tl.TO_TILE_MAJOR)     # in place
    assert e.value.status == 1


@pytest.mark.parametrize("direction", [0, 1])
def test_batch_of_matrices_in_one_launch_matches_oracle(direction):
    # eleven matrices of unequal shapes: a run of eight in one launch, then three; the tile is 16 x 128 bf16
    from gpu_util import DEV, Guarded, tl
    br, bc, s = 16, 128, 2
    shapes = [(512, 512), (1056, 2176), (16, 128), (48, 1280), (2048, 256), (32, 8192), (640, 384), (16, 256),
              (4096, 128), (64, 1024), (528, 640)]
    srcs, guards, wants = [], [], []
    for i, (rows, cols) in enumerate(shapes):
        host = inputs.random_bytes(rows * cols * s, seed=100 + i)
        srcs.append(torch.from_numpy(host).to(DEV))
        guards.append(Guarded((rows * cols * s,), torch.uint8))
        guards[-1].t.fill_(0xEE)
        wants.append(tlo.relayout(host, rows, cols, s, br, bc, direction))
    tl.relayout_batch(srcs, [g.t for g in guards], shapes, s, br * bc * s, br, bc, direction)
    tl.device_status()
    for i, (g, w) in enumerate(zip(guards, wants)):
        assert np.array_equal(g.check().cpu().numpy(), w), shapes[i]


def test_batch_falls_back_per_matrix_and_reports_argument_errors():
    from gpu_util import DEV, tl
    # 8-byte block rows cannot take the copy engine: every matrix goes through the single call
    br, bc, s = 64, 8, 1
    shapes = [(128, 64), (64, 256)]
    hosts = [inputs.random_bytes(r * c * s, seed=7 + i) for i, (r, c) in enumerate(shapes)]
    srcs = [torch.from_numpy(h).to(DEV) for h in hosts]
    dsts = [torch.empty_like(t) for t in srcs]
    tl.relayout_batch(srcs, dsts, shapes, s, br * bc * s, br, bc, tl.TO_TILE_MAJOR)
    tl.device_status()
    for h, d, (r, c) in zip(hosts, dsts, shapes):
        assert np.array_equal(d.cpu().numpy(), tlo.relayout(h, r, c, s, br, bc, tlo.TO_TILE_MAJOR))
    # a matrix whose rows are not whole blocks ends the call with the single call's error
    with pytest.raises(tl.TileLensError):
        tl.relayout_batch(srcs, dsts, [(128, 64), (60, 256)], s, br * bc * s, br, bc, tl.TO_TILE_MAJOR)
    tl.relayout_batch([], [], [], 2, 4096, 16, 128, tl.TO_TILE_MAJOR)          # empty list: no-op
