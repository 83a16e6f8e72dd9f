"""The K-contiguous flavour (weights stored [N][K], Eq. 2 as printed) through the C ABI vs the oracle (GPU)."""
import numpy as np
import pytest
import torch

import oracle as tlo
from paper_2607_04031_b200 import inputs

pytestmark = pytest.mark.gpu


def _weights_nk(B_kn: torch.Tensor, N, K, tile_n, tile_k):
    """[K][N] logical weight -> the [N][K] array, then tile-major with tile_n x tile_k tiles (library relayout)."""
    from gpu_util import DEV, tl
    w = B_kn.t().contiguous().to(DEV)                       # [N][K], K contiguous
    if tile_n == 0:
        return w
    out = torch.empty_like(w)
    tl.relayout(w, out, N, K, 2, tile_n * tile_k * 2, tile_n, tile_k, tl.TO_TILE_MAJOR)
    return out


def _run(A, W, M, N, K, tile_n, tile_k, cta=(0, 0, 0)):
    from gpu_util import DEV, guarded_out, tl
    g = guarded_out((M, N), torch.float32)
    C = g.t
    tl.gemm_kmajor(A.to(DEV).contiguous(), W, C, M, N, K, tile_n * tile_k * 2, tile_n, tile_k, cta)
    tl.device_status()
    return g.check()


TILES = [(32, 64), (16, 128), (8, 256), (64, 64), (1, 2048 // 2), (4, 512), (0, 0), (64, 32), (128, 16)]     # (tile_n, tile_k); (32, 64) = the paper's (a, b) = (64, 32)


@pytest.mark.parametrize("tile_n,tile_k", TILES)
@pytest.mark.parametrize("cta", [(0, 0, 0), (64, 128, 64), (128, 256, 64), (32, 128, 128), (256, 128, 64), (16, 64, 64)])
def test_one_hot_rows_copy_rows_of_B_exactly(tile_n, tile_k, cta):
    M, N, K = 40, 1024, 1024
    A, ks = inputs.one_hot_rows(M, K, seed=7)
    B = inputs.bf16_normal((K, N), 0.02, seed=8)
    C = _run(A, _weights_nk(B, N, K, tile_n, tile_k), M, N, K, tile_n, tile_k, cta)
    assert torch.equal(C.cpu(), B.float()[ks])


@pytest.mark.parametrize("M,N,K", [(1, 512, 512), (33, 640, 1024), (64, 256, 8192), (300, 1152, 640), (16, 8192, 1024)])
@pytest.mark.parametrize("tile_n,tile_k", [(32, 64), (16, 128), (0, 0)])
def test_integer_inputs_match_the_oracle_exactly(M, N, K, tile_n, tile_k):
    A = inputs.bf16_integers((M, K), -8, 8, seed=M + N)
    B = inputs.bf16_integers((K, N), -8, 8, seed=K)
    W = _weights_nk(B, N, K, tile_n, tile_k)
    C = _run(A, W, M, N, K, tile_n, tile_k)
    rng = np.random.default_rng(1)
    ii, jj = rng.integers(0, M, 3000), rng.integers(0, N, 3000)
    ii[:2], jj[:2] = [0, M - 1], [0, N - 1]
    if tile_n:
        ref, _ = tlo.matmul_at(inputs.bits(A), inputs.bits(W.reshape(-1)), tlo.TILE_MAJOR_K, tile_n, tile_k, M, N, K, ii, jj)
    else:       # the plain [N][K] array is the column-major K x N matrix
        ref, _ = tlo.matmul_at(inputs.bits(A), inputs.bits(W.reshape(-1)), tlo.COL_MAJOR, 0, 0, M, N, K, ii, jj)
    assert np.array_equal(C.cpu().numpy()[ii, jj].astype(np.float64), ref)
    assert torch.isfinite(C).all()


@pytest.mark.parametrize("name,K,N", inputs.LLAMA70B_PROJ)
def test_llama_decode_and_prefill_full_size_sampled(name, K, N):
    from gpu_util import DEV, sample_indices, tl
    W_nk = inputs.bf16_normal((N, K), 0.02, seed=(K % 997) + (N % 991), device=DEV)     # [N][K]
    Wt = torch.empty_like(W_nk)
    tl.relayout(W_nk, Wt, N, K, 2, 4096, 32, 64, tl.TO_TILE_MAJOR)
    for M in (8, 4096):
        A = inputs.bf16_normal((M, K), 1.0, seed=31 + M, device=DEV)
        C = _run(A, Wt, M, N, K, 32, 64)
        ii, jj = sample_indices(M, N, 500, seed=M)
        ref, S = tlo.matmul_at(inputs.bits(A.cpu()), inputs.bits(Wt.reshape(-1)), tlo.TILE_MAJOR_K, 32, 64, M, N, K, ii, jj)
        got = C[torch.from_numpy(ii).to(DEV), torch.from_numpy(jj).to(DEV)].cpu().numpy().astype(np.float64)
        err = np.abs(got - ref)
        assert np.all(err <= 1e-3 * S) and float(np.max(err / np.maximum(S, 1e-300))) <= 1e-4
        # the untiled [N][K] array through the same kernel gives the same bits
        assert torch.equal(_run(A, W_nk, M, N, K, 0, 0), C)


def test_grouped_small_integer_exact():
    from gpu_util import DEV, tl
    E, K, N, tile_n, tile_k = 8, 256, 384, 32, 64
    offsets, counts, _ = inputs.zipf_topk_routing(40, E, 3, 1.1, seed=3)
    rows = int(offsets[-1])
    A = inputs.bf16_integers((rows, K), -8, 8, seed=4)
    B = inputs.bf16_integers((E, N, K), -8, 8, seed=5)           # per expert [N][K]
    Bd = B.to(DEV)
    Bt = torch.empty_like(Bd)
    tl.relayout(Bd, Bt, E * N, K, 2, tile_n * tile_k * 2, tile_n, tile_k, tl.TO_TILE_MAJOR)
    C = torch.full((rows, N), float("nan"), dtype=torch.float32, device=DEV)
    tl.gemm_grouped_kmajor(A.to(DEV), Bt, C, torch.from_numpy(offsets).to(DEV), E, rows, N, K, tile_n * tile_k * 2,
                           tile_n, tile_k)
    tl.device_status()
    want = torch.cat([A[int(offsets[e]):int(offsets[e + 1])].float() @ B[e].float().t() for e in range(E)])
    ref_rows = np.arange(rows)
    # oracle on every expert's first and last row, all columns
    Ch = C.cpu().numpy().astype(np.float64)
    for e in range(E):
        r0, r1 = int(offsets[e]), int(offsets[e + 1])
        if r1 == r0:
            continue
        for r in (r0, r1 - 1):
            jj = np.arange(N)
            ref, _ = tlo.matmul_at(inputs.bits(A[r:r + 1]), inputs.bits(Bt[e].reshape(-1)), tlo.TILE_MAJOR_K, tile_n, tile_k,
                                   1, N, K, np.zeros(N, dtype=np.int64), jj)
            assert np.array_equal(Ch[r], ref)
    assert torch.equal(C.cpu(), want)            # exact integers: also equal to the fp32 product


def test_read_amp_counter_k_contiguous_flavour():
    from gpu_util import tl
    cases = [(16, 512, 4096, (16, 256, 128), 4096, 32, 64), (3, 512, 4096, (2, 96, 80), 512, 8, 32),
             (4096, 8192, 8192, (256, 128, 64), 4096, 32, 64), (8, 10240, 8192, (16, 256, 64), 4096, 16, 128)]
    for M, N, K, cta, G, b, a in cases:
        got = tl.read_amp(M, N, K, cta, tl.LAYOUT_TILE_MAJOR_K, G, b, a, 2)
        assert got == tlo.read_amp(M, N, K, *cta, tlo.TILE_MAJOR_K, G, b, a, 2)
    # Section 6.5, literally: 128 (K) x 256 (N) weight tile, (a, b) = (64, 32): 16 requests per load, RA = 1
    f, u, q = tl.read_amp(1, 512, 4096, (1, 256, 128), tl.LAYOUT_TILE_MAJOR_K, 4096, 32, 64, 2)
    assert f == u and q == 16 * (512 // 256) * (4096 // 128)


def test_errors():
    from gpu_util import DEV, tl
    A = torch.zeros((8, 512), dtype=torch.bfloat16, device=DEV)
    W = torch.zeros((512, 512), dtype=torch.bfloat16, device=DEV)
    C = torch.zeros((8, 512), dtype=torch.float32, device=DEV)
    with pytest.raises(tl.TileLensError) as e:
        tl.gemm_kmajor(A, W, C, 8, 512, 512, 4096, 256, 8)        # tile rows of 16 bytes: no path in this flavour
    assert e.value.status == 2
    with pytest.raises(tl.TileLensError) as e:
        tl.gemm_kmajor(A, W, C, 8, 512, 512, 2048, 32, 64)        # G != tile_n * tile_k * 2
    assert e.value.status == 1
