"""Pins for the oracle's fp64 product (CPU only)."""
import numpy as np
import pytest
import torch

import oracle as tlo
from paper_2607_04031_b200 import inputs


def _to_f64(t):
    return t.to(torch.float64).numpy()


def test_bf16_decoding_matches_torch_for_every_bit_pattern():
    allbits = np.arange(65536, dtype=np.uint16)
    want = torch.from_numpy(allbits.view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()
    got = np.array([tlo.bf16_to_double(int(h)) for h in allbits])
    finite = np.isfinite(want)
    assert np.array_equal(got[finite], want[finite])
    assert np.array_equal(np.isnan(got), np.isnan(want))
    assert np.array_equal(np.isinf(got), np.isinf(want))


def test_tiny_product_matches_pure_python_loops():
    M, N, K = 3, 8, 8
    A = inputs.bf16_normal((M, K), 1.0, seed=1)
    B = inputs.bf16_uniform((K, N), -1.0, 1.0, seed=2)
    a, b = _to_f64(A), _to_f64(B)
    C, S = tlo.matmul(inputs.bits(A), inputs.bits(B), tlo.ROW_MAJOR, 0, 0, M, N, K)
    for i in range(M):
        for j in range(N):
            acc = 0.0
            sab = 0.0
            for k in range(K):
                acc += float(a[i, k]) * float(b[k, j])
                sab += abs(float(a[i, k]) * float(b[k, j]))
            assert C[i, j] == acc
            assert S[i, j] == sab


@pytest.mark.parametrize("M,N,K,br,bc", [(16, 512, 512, 16, 128), (5, 96, 64, 8, 32), (33, 64, 128, 32, 64)])
def test_product_matches_numpy_for_every_layout_of_B(M, N, K, br, bc):
    A = inputs.bf16_normal((M, K), 1.0, seed=3)
    B = inputs.bf16_uniform((K, N), -1.0, 1.0, seed=4)
    want = _to_f64(A) @ _to_f64(B)
    want_S = np.abs(_to_f64(A)) @ np.abs(_to_f64(B))
    Bb = inputs.bits(B)
    B_tile = tlo.relayout(Bb.view(np.uint8), K, N, 2, br, bc, tlo.TO_TILE_MAJOR).view(np.uint16)
    B_col = np.ascontiguousarray(Bb.T)            # K contiguous: element (k, n) at n*K + k
    for layout, buf in ((tlo.ROW_MAJOR, Bb), (tlo.TILE_MAJOR, B_tile), (tlo.COL_MAJOR, B_col)):
        C, S = tlo.matmul(inputs.bits(A), buf, layout, br, bc, M, N, K)
        # same products, different summation order inside BLAS: a few ulps of the absolute sum
        assert np.all(np.abs(C - want) <= 1e-13 * want_S + 1e-300)
        assert np.all(np.abs(S - want_S) <= 1e-13 * want_S + 1e-300)
    # the three layouts must agree with each other exactly (same loop, same operands)
    C_row, _ = tlo.matmul(inputs.bits(A), Bb, tlo.ROW_MAJOR, 0, 0, M, N, K)
    C_tile, _ = tlo.matmul(inputs.bits(A), B_tile, tlo.TILE_MAJOR, br, bc, M, N, K)
    assert np.array_equal(C_row, C_tile)


def test_integer_inputs_give_exact_integers():
    M, N, K = 7, 64, 256
    A = inputs.bf16_integers((M, K), -8, 8, seed=5)
    B = inputs.bf16_integers((K, N), -8, 8, seed=6)
    want = A.to(torch.int64) @ B.to(torch.int64)
    C, S = tlo.matmul(inputs.bits(A), inputs.bits(B), tlo.ROW_MAJOR, 0, 0, M, N, K)
    assert np.array_equal(C, want.numpy().astype(np.float64))
    assert np.array_equal(S, (A.to(torch.int64).abs() @ B.to(torch.int64).abs()).numpy().astype(np.float64))


def test_one_hot_rows_select_rows_of_B():
    M, N, K, br, bc = 9, 128, 64, 16, 64
    A, ks = inputs.one_hot_rows(M, K, seed=7)
    B = inputs.bf16_normal((K, N), 0.02, seed=8)
    B_tile = tlo.relayout(inputs.bits(B).view(np.uint8), K, N, 2, br, bc, tlo.TO_TILE_MAJOR).view(np.uint16)
    C, _ = tlo.matmul(inputs.bits(A), B_tile, tlo.TILE_MAJOR, br, bc, M, N, K)
    assert np.array_equal(C, _to_f64(B)[ks.numpy()])


def test_all_ones_B_gives_row_sums():
    M, N, K = 4, 32, 128
    A = inputs.bf16_normal((M, K), 1.0, seed=9)
    B = torch.ones((K, N), dtype=torch.bfloat16)
    C, _ = tlo.matmul(inputs.bits(A), inputs.bits(B), tlo.ROW_MAJOR, 0, 0, M, N, K)
    sums = np.array([sum(float(x) for x in row) for row in _to_f64(A)])     # sequential, like the oracle
    assert np.array_equal(C, np.repeat(sums[:, None], N, axis=1))


def test_sampled_product_equals_full_product():
    M, N, K, br, bc = 16, 256, 128, 16, 128
    A = inputs.bf16_normal((M, K), 1.0, seed=10)
    B = inputs.bf16_normal((K, N), 0.02, seed=11)
    B_tile = tlo.relayout(inputs.bits(B).view(np.uint8), K, N, 2, br, bc, tlo.TO_TILE_MAJOR).view(np.uint16)
    C, S = tlo.matmul(inputs.bits(A), B_tile, tlo.TILE_MAJOR, br, bc, M, N, K)
    rng = np.random.default_rng(0)
    ii, jj = rng.integers(0, M, 50), rng.integers(0, N, 50)
    Cs, Ss = tlo.matmul_at(inputs.bits(A), B_tile, tlo.TILE_MAJOR, br, bc, M, N, K, ii, jj)
    assert np.array_equal(Cs, C[ii, jj]) and np.array_equal(Ss, S[ii, jj])
    with pytest.raises(ValueError):
        tlo.matmul_at(inputs.bits(A), B_tile, tlo.TILE_MAJOR, br, bc, M, N, K, [M], [0])


def test_k_contiguous_tile_major_gives_the_same_product():
    M, N, K, a, b = 5, 96, 128, 64, 32                   # the paper's (64, 32) memory tile
    A = inputs.bf16_normal((M, K), 1.0, seed=21)
    B = inputs.bf16_normal((K, N), 0.02, seed=22)
    want, _ = tlo.matmul(inputs.bits(A), inputs.bits(B), tlo.ROW_MAJOR, 0, 0, M, N, K)
    w_nk = np.ascontiguousarray(inputs.bits(B).T)        # [N][K], K contiguous
    buf = tlo.relayout(w_nk.view(np.uint8), N, K, 2, b, a, tlo.TO_TILE_MAJOR).view(np.uint16)
    got, _ = tlo.matmul(inputs.bits(A), buf, tlo.TILE_MAJOR_K, b, a, M, N, K)
    assert np.array_equal(got, want)


# ------------------------------------------------------------------ FP8 (E4M3)
def test_fp8_decoding_matches_torch_for_every_bit_pattern_and_known_values():
    allbits = np.arange(256, dtype=np.uint8)
    want = torch.from_numpy(allbits).view(inputs.FP8).to(torch.float64).numpy()
    got = np.array([tlo.fp8_e4m3_to_double(int(h)) for h in allbits])
    ok = ~np.isnan(want)
    assert np.array_equal(got[ok], want[ok]) and np.array_equal(np.isnan(got), np.isnan(want))
    assert np.isnan(got).sum() == 2 and not np.isinf(got).any()          # S.1111.111 only; no infinities
    # the format's landmarks, written out: 1.0, -1.0, largest finite 448, smallest subnormal 2^-9, smallest normal 2^-6
    assert tlo.fp8_e4m3_to_double(0x38) == 1.0 and tlo.fp8_e4m3_to_double(0xB8) == -1.0
    assert tlo.fp8_e4m3_to_double(0x7E) == 448.0 and tlo.fp8_e4m3_to_double(0x01) == 2.0 ** -9
    assert tlo.fp8_e4m3_to_double(0x08) == 2.0 ** -6 and tlo.fp8_e4m3_to_double(0x00) == 0.0
    assert tlo.fp8_e4m3_to_double(0x55) == 13.0                          # 0 1010 101: 1.101b x 2^(10-7)


def test_fp8_product_matches_numpy_and_exact_integers_in_every_layout():
    M, N, K, b, a = 6, 128, 256, 64, 64                       # the 64 x 64 FP8 memory tile of Figure 1(c)
    A = inputs.fp8_normal((M, K), 1.0, seed=31)
    B = inputs.fp8_normal((K, N), 0.5, seed=32)
    a64, b64 = A.to(torch.float64).numpy(), B.to(torch.float64).numpy()
    want, want_S = a64 @ b64, np.abs(a64) @ np.abs(b64)
    ii, jj = np.repeat(np.arange(M), N), np.tile(np.arange(N), M)
    w_nk = np.ascontiguousarray(inputs.bits8(B).T)            # [N][K]
    tiled = tlo.relayout(w_nk, N, K, 1, b, a, tlo.TO_TILE_MAJOR)
    for layout, buf, br, bc in ((tlo.ROW_MAJOR, inputs.bits8(B), 0, 0), (tlo.COL_MAJOR, w_nk, 0, 0),
                                (tlo.TILE_MAJOR_K, tiled, b, a)):
        C, S = tlo.matmul_at_fp8(inputs.bits8(A), buf, layout, br, bc, M, N, K, ii, jj)
        assert np.all(np.abs(C.reshape(M, N) - want) <= 1e-13 * want_S + 1e-300)
        assert np.all(np.abs(S.reshape(M, N) - want_S) <= 1e-13 * want_S + 1e-300)
    Ai = inputs.fp8_integers((M, K), -8, 8, seed=33)
    Bi = inputs.fp8_integers((K, N), -8, 8, seed=34)
    wi = Ai.to(torch.float32).to(torch.int64) @ Bi.to(torch.float32).to(torch.int64)
    tiled_i = tlo.relayout(np.ascontiguousarray(inputs.bits8(Bi).T), N, K, 1, b, a, tlo.TO_TILE_MAJOR)
    C, _ = tlo.matmul_at_fp8(inputs.bits8(Ai), tiled_i, tlo.TILE_MAJOR_K, b, a, M, N, K, ii, jj)
    assert np.array_equal(C.reshape(M, N), wi.numpy().astype(np.float64))
