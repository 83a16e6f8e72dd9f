"""Maximum sizes: buffers whose element counts and byte offsets do not fit 32 bits.  Sampled against the oracle
(its index functions and dot products are 64-bit throughout) plus properties that hold at any size."""
import numpy as np
import pytest
import torch

import oracle as tlo
from paper_2607_04031_b200 import inputs

pytestmark = pytest.mark.gpu


def _sample_rc(rows, cols, n, seed, br, bc):
    rng = np.random.default_rng(seed)
    r = rng.integers(0, rows, n)
    c = rng.integers(0, cols, n)
    # corners, and the first and last element of the last memory tile (offsets just under rows*cols)
    r[:6] = [0, 0, rows - 1, rows - 1, rows - br, rows - 1]
    c[:6] = [0, cols - 1, 0, cols - 1, cols - bc, cols - 1]
    return r, c


def test_weight_of_more_than_2_to_31_elements_relayout_and_decode_gemm():
    from gpu_util import DEV, check_against_oracle, run_gemm, sample_indices, tl
    K, N, br, bc, G = 16384, 147456, 16, 128, 4096                 # 2.42e9 elements, 4.83 GB: offsets pass 2^32
    assert K * N > 2 ** 31 and K * N * 2 > 2 ** 32
    B = inputs.bf16_normal((K, N), 0.02, seed=77, device=DEV)
    Bt = torch.empty_like(B)
    tl.relayout(B, Bt, K, N, 2, G, br, bc, tl.TO_TILE_MAJOR)
    # sampled elements: where Eq. 1-2 (the oracle's index function) says element (r, c) lives
    r, c = _sample_rc(K, N, 4000, 5, br, bc)
    offs = np.array([tlo.off_tile(int(a), int(b), K, N, br, bc, 2) for a, b in zip(r, c)], dtype=np.int64)
    assert offs.max() > 2 ** 32
    got = Bt.reshape(-1).view(torch.int16)[torch.from_numpy(offs // 2).to(DEV)]
    want = B.view(torch.int16)[torch.from_numpy(r).to(DEV), torch.from_numpy(c).to(DEV)]
    assert torch.equal(got, want)
    # round trip
    back = torch.empty_like(B)
    tl.relayout(Bt, back, K, N, 2, G, br, bc, tl.TO_ROW_MAJOR)
    assert torch.equal(back, B)
    del back
    # decode product: sampled outputs against the oracle reading the tile-major bits, and the row-major comparator
    M = 4
    A = inputs.bf16_normal((M, K), 1.0, seed=78)
    C = run_gemm(A, Bt, M, N, K, br, bc)
    ii, jj = sample_indices(M, N, 400, seed=9)
    jj[4:8] = [N - 2, N - 129, N // 2, N // 2 + 1]                 # the far end of the buffer
    check_against_oracle(C, A, Bt, tlo.TILE_MAJOR, br, bc, M, N, K, idx=(ii, jj))
    assert torch.equal(run_gemm(A, B, M, N, K, 0, 0), C)


def test_output_of_more_than_2_to_31_elements_prefill_gemm():
    from gpu_util import DEV, sample_indices, tl
    M, N, K, br, bc = 32768, 73728, 256, 16, 128                   # C: 2.42e9 floats, 9.7 GB
    assert M * N > 2 ** 31
    A = inputs.bf16_normal((M, K), 1.0, seed=81)
    B = inputs.bf16_normal((K, N), 0.05, seed=82, device=DEV)
    Bt = torch.empty_like(B)
    tl.relayout(B, Bt, K, N, 2, 4096, br, bc, tl.TO_TILE_MAJOR)
    C = torch.full((M, N), float("nan"), dtype=torch.float32, device=DEV)
    tl.gemm(A.to(DEV), Bt, C, M, N, K, 4096, br, bc)
    tl.device_status()
    assert not bool(torch.isnan(C[M - 4096:]).any()) and not bool(torch.isnan(C[:4096]).any())   # both ends written
    ii, jj = sample_indices(M, N, 600, seed=10)
    ii[4:8] = [M - 1, M - 2, M - 257, M // 2]
    jj[4:8] = [N - 1, N - 129, 1, N // 2]
    got = C[torch.from_numpy(ii).to(DEV), torch.from_numpy(jj).to(DEV)].cpu().numpy().astype(np.float64)
    ref, S = tlo.matmul_at(inputs.bits(A), inputs.bits(Bt.reshape(-1)), tlo.TILE_MAJOR, br, bc, M, N, K, ii, jj)
    assert np.all(np.abs(got - ref) <= 1e-3 * S), float(np.max(np.abs(got - ref) / np.maximum(S, 1e-300)))


def test_box_loads_from_a_buffer_of_more_than_4_GiB():
    from gpu_util import DEV, tl
    K, N, s, a, b = 16384, 147456, 2, 64, 32                       # [N][K] weight in (64, 32) memory tiles, 4.83 GB
    w = inputs.bf16_normal((N, K), 0.02, seed=91, device=DEV)
    tiled = torch.empty_like(w)
    tl.relayout(w, tiled, N, K, s, 4096, b, a, tl.TO_TILE_MAJOR)
    rng = np.random.default_rng(3)
    coords = [[int(i) * 64, int(j) * 256] for i, j in zip(rng.integers(0, K // 64, 60), rng.integers(0, N // 256, 60))]
    coords[:3] = [[0, 0], [K - 64, N - 256], [0, N - 256]]         # the last box starts 4.83e9 bytes into the buffer
    desc_args = ([K, N], [1, K], [64, 256], s, a, b, K)
    # offsets of the far boxes against the oracle's address generation
    cd = torch.tensor(coords, dtype=torch.int32, device=DEV)
    offs = torch.empty((len(coords), 64 * 256), dtype=torch.int64, device=DEV)
    tl.hw_box_offsets(tl.hw_desc(*desc_args), cd, offs)
    tl.device_status()
    od = tlo.hw_desc(*desc_args)
    for ci in (0, 1, 2, 17):
        want = tlo.hw_box_offsets(od, coords[ci])
        assert np.array_equal(offs[ci].cpu().numpy().astype(np.uint64), want.astype(np.uint64))
    assert int(offs[1].max()) > 2 ** 32
    # the loads: every box equals the slice of the matrix it names
    dst = torch.empty((len(coords), 256, 64), dtype=torch.bfloat16, device=DEV)
    tl.hw_box_load(tl.hw_desc(*desc_args), tiled, cd, dst)
    tl.device_status()
    for ci, (i, j) in enumerate(coords):
        assert torch.equal(dst[ci], w[j:j + 256, i:i + 64]), (ci, i, j)
