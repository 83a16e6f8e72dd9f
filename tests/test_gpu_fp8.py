"""FP8 (E4M3) products on K-contiguous tile-major weights through the C ABI vs the oracle (GPU)."""
import numpy as np
import pytest
import torch

import oracle as tlo
from paper_2607_04031_b200 import inputs

pytestmark = pytest.mark.gpu


def _weights_nk(B_kn: torch.Tensor, N, K, tile_n, tile_k):
    """[K][N] logical FP8 weight -> [N][K] bytes, tile-major with tile_n x tile_k tiles (library relayout)."""
    from gpu_util import DEV, tl
    w = B_kn.view(torch.uint8).t().contiguous().to(DEV)
    if tile_n == 0:
        return w
    out = torch.empty_like(w)
    tl.relayout(w, out, N, K, 1, tile_n * tile_k, tile_n, tile_k, tl.TO_TILE_MAJOR)
    return out


def _run(A, W, M, N, K, tile_n, tile_k, cta=(0, 0, 0)):
    from gpu_util import DEV, guarded_out, tl
    g = guarded_out((M, N), torch.float32)
    C = g.t
    tl.gemm_fp8_kmajor(A.view(torch.uint8).to(DEV).contiguous(), W, C, M, N, K, tile_n * tile_k, tile_n, tile_k, cta)
    tl.device_status()
    return g.check()


TILES = [(64, 64), (32, 128), (16, 256), (128, 32), (8, 512), (0, 0)]        # (64, 64): Figure 1(c)


@pytest.mark.parametrize("tile_n,tile_k", TILES)
@pytest.mark.parametrize("cta", [(0, 0, 0), (64, 128, 128), (128, 256, 128), (32, 128, 256), (256, 128, 128), (16, 64, 128)])
def test_one_hot_rows_copy_rows_of_B_exactly(tile_n, tile_k, cta):
    M, N, K = 40, 1024, 1024
    ks = torch.randint(0, K, (M,), generator=torch.Generator().manual_seed(5))
    A = torch.zeros((M, K), dtype=torch.float32)
    A[torch.arange(M), ks] = 1.0
    A = A.to(inputs.FP8)
    B = inputs.fp8_normal((K, N), 0.5, seed=8)
    C = _run(A, _weights_nk(B, N, K, tile_n, tile_k), M, N, K, tile_n, tile_k, cta)
    assert torch.equal(C.cpu(), B.float()[ks])


@pytest.mark.parametrize("M,N,K", [(1, 512, 512), (33, 640, 1024), (64, 256, 8192), (300, 1152, 640), (16, 8192, 1024),
                                   (2560, 2048, 1024)])
@pytest.mark.parametrize("tile_n,tile_k", [(64, 64), (32, 128), (0, 0)])
def test_integer_inputs_match_the_oracle_exactly(M, N, K, tile_n, tile_k):
    if tile_n == 0 and K % 128:
        pytest.skip("the plain array needs K % 128 == 0")
    A = inputs.fp8_integers((M, K), -8, 8, seed=M + N)
    B = inputs.fp8_integers((K, N), -8, 8, seed=K)
    W = _weights_nk(B, N, K, tile_n, tile_k)
    C = _run(A, W, M, N, K, tile_n, tile_k)
    rng = np.random.default_rng(1)
    ii, jj = rng.integers(0, M, 3000), rng.integers(0, N, 3000)
    ii[:2], jj[:2] = [0, M - 1], [0, N - 1]
    layout = tlo.TILE_MAJOR_K if tile_n else tlo.COL_MAJOR
    ref, _ = tlo.matmul_at_fp8(inputs.bits8(A), W.cpu().numpy().reshape(-1), layout, tile_n, tile_k, M, N, K, ii, jj)
    assert np.array_equal(C.cpu().numpy()[ii, jj].astype(np.float64), ref)
    assert torch.isfinite(C).all()


@pytest.mark.parametrize("name,K,N", inputs.LLAMA70B_PROJ)
def test_llama_shapes_full_size_sampled(name, K, N):
    from gpu_util import DEV, sample_indices, tl
    W_nk = inputs.fp8_normal((N, K), 0.05, seed=(K % 997) + (N % 991), device=DEV).view(torch.uint8)
    Wt = torch.empty_like(W_nk)
    tl.relayout(W_nk, Wt, N, K, 1, 4096, 64, 64, tl.TO_TILE_MAJOR)
    for M in (8, 4096):
        A = inputs.fp8_normal((M, K), 1.0, seed=31 + M, device=DEV)
        C = _run(A, Wt, M, N, K, 64, 64)
        ii, jj = sample_indices(M, N, 400, seed=M)
        ref, S = tlo.matmul_at_fp8(inputs.bits8(A), Wt.cpu().numpy().reshape(-1), tlo.TILE_MAJOR_K, 64, 64, M, N, K, ii, jj)
        got = C[torch.from_numpy(ii).to(DEV), torch.from_numpy(jj).to(DEV)].cpu().numpy().astype(np.float64)
        err = np.abs(got - ref)
        assert np.all(err <= 1e-3 * S) and float(np.max(err / np.maximum(S, 1e-300))) <= 1e-4
        assert torch.equal(_run(A, W_nk, M, N, K, 0, 0), C)       # the untiled array gives the same bits


def test_grouped_small_integer_exact():
    from gpu_util import DEV, tl
    E, K, N, tile_n, tile_k = 8, 256, 384, 64, 64
    offsets, counts, _ = inputs.zipf_topk_routing(40, E, 3, 1.1, seed=3)
    rows = int(offsets[-1])
    A = inputs.fp8_integers((rows, K), -8, 8, seed=4)
    B = inputs.fp8_integers((E, N, K), -8, 8, seed=5)                 # per expert [N][K]
    Bd = B.view(torch.uint8).to(DEV)
    Bt = torch.empty_like(Bd)
    tl.relayout(Bd, Bt, E * N, K, 1, tile_n * tile_k, tile_n, tile_k, tl.TO_TILE_MAJOR)
    C = torch.full((rows, N), float("nan"), dtype=torch.float32, device=DEV)
    tl.gemm_grouped_fp8_kmajor(A.view(torch.uint8).to(DEV), Bt, C, torch.from_numpy(offsets).to(DEV), E, rows, N, K,
                               tile_n * tile_k, tile_n, tile_k)
    tl.device_status()
    want = torch.cat([A[int(offsets[e]):int(offsets[e + 1])].float() @ B[e].float().t() for e in range(E)])
    assert torch.equal(C.cpu(), want)
    r = int(offsets[np.argmax(counts)])                               # one row against the oracle, all columns
    e = int(np.argmax(counts))
    ref, _ = tlo.matmul_at_fp8(inputs.bits8(A[r:r + 1]), Bt[e].cpu().numpy().reshape(-1), tlo.TILE_MAJOR_K, tile_n, tile_k,
                               1, N, K, np.zeros(N, dtype=np.int64), np.arange(N))
    assert np.array_equal(C[r].cpu().numpy().astype(np.float64), ref)


def test_read_amp_counter_fp8_tiles():
    from gpu_util import tl
    # Figure 1(c): with 64 x 64 FP8 memory tiles every fetched byte of a 128 x 256 weight tile is used;
    # Section 3.1: the one-dimensional extremes (1, 4096) and (4096, 1) are not.
    for M, N, K, cta, b, a in [(16, 512, 4096, (16, 256, 128), 64, 64), (5, 1024, 8192, (16, 128, 256), 32, 128),
                               (16, 512, 8192, (16, 256, 128), 1, 4096), (16, 8192, 4096, (16, 256, 128), 4096, 1)]:
        got = tl.read_amp(M, N, K, cta, tl.LAYOUT_TILE_MAJOR_K, 4096, b, a, 1)
        assert got == tlo.read_amp(M, N, K, *cta, tlo.TILE_MAJOR_K, 4096, b, a, 1)
        if (b, a) == (64, 64):
            assert got[0] == got[1]
        if b == 1 or a == 1:
            assert got[0] > got[1]


def test_errors():
    from gpu_util import DEV, tl
    A = torch.zeros((8, 512), dtype=torch.uint8, device=DEV)
    W = torch.zeros((512, 512), dtype=torch.uint8, device=DEV)
    C = torch.zeros((8, 512), dtype=torch.float32, device=DEV)
    with pytest.raises(tl.TileLensError) as e:
        tl.gemm_fp8_kmajor(A, W, C, 8, 512, 512, 4096, 256, 16)       # 16-byte tile rows
    assert e.value.status == 2
    with pytest.raises(tl.TileLensError) as e:
        tl.gemm_fp8_kmajor(A, W, C, 8, 512, 512, 8192, 64, 64)        # G != tile_n * tile_k
    assert e.value.status == 1
    with pytest.raises(tl.TileLensError) as e:
        tl.gemm_fp8_kmajor(A, W, C, 8, 512, 512, 4096, 64, 64, (16, 256, 64))     # cta_k counts elements: 128 or 256
    assert e.value.status == 2
