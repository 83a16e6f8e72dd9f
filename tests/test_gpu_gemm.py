"""tcgen05 GEMM (dense, decode/stream-K, grouped) vs the oracle (GPU).

Tolerance (from the arithmetic): inputs are exact in fp64, the kernel accumulates in fp32, so
|C - C_ref| <= 1e-3 * sum_k |A_ik B_kj| with a wide margin; integer-valued and one-hot inputs
must come out bit-exact in every variant because every partial sum is an exact fp32 integer.
"""
import numpy as np
import pytest
import torch

import oracle as tlo
from paper_2607_04031_b200 import inputs

pytestmark = pytest.mark.gpu
ROW, TILE = tlo.ROW_MAJOR, tlo.TILE_MAJOR


def _oracle_full(A, B_dev_buf, layout, br, bc, M, N, K):
    return tlo.matmul(inputs.bits(A), inputs.bits(B_dev_buf.reshape(-1)), layout, br, bc, M, N, K)


def test_config1_tiny_tile_major_and_row_major():
    from gpu_util import DEV, check_against_oracle, run_gemm, tile_major_on_device
    M, N, K, br, bc = 16, 512, 512, 16, 128
    A = inputs.bf16_normal((M, K), 1.0, seed=101)
    B = inputs.bf16_uniform((K, N), -1.0, 1.0, seed=102)
    Bt = tile_major_on_device(B, K, N, br, bc)
    C = run_gemm(A, Bt, M, N, K, br, bc)
    check_against_oracle(C, A, Bt, TILE, br, bc, M, N, K)
    C_row = run_gemm(A, B.to(DEV), M, N, K, 0, 0)
    check_against_oracle(C_row, A, B.to(DEV), ROW, 0, 0, M, N, K)
    # same kernel, same K order: the two layouts give the same bits
    assert torch.equal(C, C_row)


# TMA-boxable tiles, row-major, one-row tiles (= row-major), and tiles only the generic-address path can read
BLOCKS = [(16, 128), (32, 64), (8, 256), (64, 64), (16, 512), (0, 0), (1, 1024), (1, 128),
          (8, 2), (16, 1), (8, 16), (16, 8), (32, 4), (16, 32), (32, 16), (2, 64), (4, 128), (64, 8),
          (8, 8), (8, 1), (64, 1), (128, 1), (4, 8), (8, 4), (16, 2), (64, 4), (64, 2), (128, 2), (128, 4), (4, 4),
          (2, 1024), (4, 512), (2, 256), (64, 32), (128, 16), (4, 32), (256, 16)]


@pytest.mark.parametrize("br,bc", BLOCKS)
@pytest.mark.parametrize("cta", [(0, 0, 0), (64, 128, 64), (128, 256, 64), (32, 128, 128), (128, 256, 128),
                                 (64, 64, 64), (16, 64, 128)])
def test_one_hot_rows_copy_rows_of_B_exactly(br, bc, cta):
    # No arithmetic at all: catches any error in the tensor-map view, the swizzle or the descriptors.
    from gpu_util import DEV, run_gemm, tile_major_on_device
    M, N, K = 40, 1024, 512
    A, ks = inputs.one_hot_rows(M, K, seed=7)
    B = inputs.bf16_normal((K, N), 0.02, seed=8)
    Bd = tile_major_on_device(B, K, N, br, bc) if br else B.to(DEV)
    hand_addressed = br > 1 and bc < 16          # rows shorter than 32 bytes; everything else is TMA-boxable
    cta_n, cta_k = (cta[1] or 128), (cta[2] or 64)
    # of those, single-column tiles of at least 8 rows are read as a K-major operand and tiles with 16-byte rows as
    # they are (if the CTA tile holds whole memory tiles); the rest is permuted in shared memory
    as_stored = hand_addressed and br >= 8 and (bc == 1 or (bc == 8 and br <= cta_k))
    # tiles with 8- or 4-byte rows are fetched as stored too and then transposed in place, 2 or 4 tiles at a time
    in_place = hand_addressed and br >= 8 and br <= cta_k and ((bc == 4 and br <= 64) or bc == 2)
    if hand_addressed and not as_stored and not in_place and (bc > cta_n or br > cta_k or cta_n * cta_k >= 256 * 128):
        # documented limits of the generic-address path: the memory tile must fit inside the CTA tile, and two
        # operand stages plus two raw stage images must fit in shared memory (not with 64 KB of weights per stage)
        from gpu_util import tl
        with pytest.raises(tl.TileLensError) as e:
            run_gemm(A, Bd, M, N, K, br, bc, cta)
        assert e.value.status == 2
        return
    C = run_gemm(A, Bd, M, N, K, br, bc, cta)
    assert torch.equal(C.cpu(), B.float()[ks])
    if hand_addressed:
        from gpu_util import tl
        assert tl.gemm_last_plan().generic_path == (2 if as_stored else 3 if in_place else 1)
        if (as_stored or in_place) and cta_n * cta_k < 256 * 128 and br <= cta_k:
            with tl.option(tl.OPT_GENERIC_RAW, 0):            # the same tiles through the permuting path
                assert torch.equal(run_gemm(A, Bd, M, N, K, br, bc, cta).cpu(), B.float()[ks])
                assert tl.gemm_last_plan().generic_path == 1


def test_short_tiles_wider_than_the_cta_tile_and_hand_addressed_tiles_taller_than_it():
    from gpu_util import run_gemm, tile_major_on_device, tl
    M, N, K = 24, 512, 256
    A, ks = inputs.one_hot_rows(M, K, seed=3)
    B = inputs.bf16_normal((K, N), 0.02, seed=4)
    Bd = tile_major_on_device(B, K, N, 4, 256)                 # 4-row tiles are TMA-boxable: part of a tile per CTA tile is fine
    assert torch.equal(run_gemm(A, Bd, M, N, K, 4, 256, (32, 256, 64)).cpu(), B.float()[ks])
    assert torch.equal(run_gemm(A, Bd, M, N, K, 4, 256, (32, 128, 64)).cpu(), B.float()[ks])
    Bd = tile_major_on_device(B, K, N, 128, 8)                 # 16-byte rows: hand-addressed, the tile must fit the CTA tile
    assert torch.equal(run_gemm(A, Bd, M, N, K, 128, 8, (32, 128, 128)).cpu(), B.float()[ks])
    with pytest.raises(tl.TileLensError) as e:
        run_gemm(A, Bd, M, N, K, 128, 8, (32, 128, 64))        # 128 rows do not fit 64
    assert e.value.status == 2


AS_STORED = [(16, 8), (8, 8), (64, 8), (16, 1), (8, 1), (32, 1), (64, 1), (128, 1),
             (32, 4), (8, 4), (64, 4), (8, 2), (16, 2), (32, 2), (64, 2)]


@pytest.mark.parametrize("br,bc", AS_STORED)
def test_tiles_read_as_stored_ragged_edges_grouped_and_prefill(br, bc):
    # Memory tiles with 16-byte rows (raw tiles = core matrices of the no-swizzle operand), single-column tiles (a
    # K-major operand in panels) and tiles with 8- or 4-byte rows (fetched as stored, 2 or 4 neighbours transposed in
    # place into a tile with 16-byte rows): ragged N and K against the oracle, a grouped product, a prefill-sized product on the
    # CTA-pair kernel; integer data, so everything is exact; the permuting path must give the same bits.
    from gpu_util import DEV, guarded_out, run_gemm, tile_major_on_device, tl
    G = br * bc * 2
    for M, N, K, cta in ((40, 1160, 1152, (0, 0, 0)), (130, 1096, 640, (128, 128, 128)), (300, 648, 384, (0, 0, 0)),
                         (9, 2056, 2176, (64, 256, 64)), (24, 1156, 512, (0, 0, 0))):
        if N % bc:
            continue                                        # (1156 columns: only for tiles of 1, 2 or 4 columns; the last
                                                            #  group of 2 or 4 neighbouring tiles is then incomplete)
        if K % br:
            K += br - K % br
        A = inputs.bf16_integers((M, K), -8, 8, seed=M + br)
        B = inputs.bf16_integers((K, N), -8, 8, seed=N + bc)
        Bd = tile_major_on_device(B, K, N, br, bc)
        want = (A.double() @ B.double()).float()
        if cta[2] and br > cta[2] and bc != 1:
            continue                                        # the memory tile must fit the CTA tile
        C = run_gemm(A, Bd, M, N, K, br, bc, cta)
        assert tl.gemm_last_plan().generic_path == ((3 if bc in (2, 4) else 2) if (bc == 1 or br <= tl.gemm_last_plan().cta_k) else 1)
        assert torch.equal(C.cpu(), want), (M, N, K, cta)
        ref, _ = _oracle_full(A, Bd, TILE, br, bc, M, N, K)
        assert np.array_equal(C.cpu().numpy().astype(np.float64), ref)
    # grouped: 12 experts, ragged row counts
    E, N, K = 12, 768, 512
    offsets, _, _ = inputs.zipf_topk_routing(64, E, 4, 1.0, seed=br + bc)
    rows = int(offsets[-1])
    A = inputs.bf16_integers((rows, K), -8, 8, seed=31)
    B = inputs.bf16_integers((E * K, N), -8, 8, seed=32)
    Bd = tile_major_on_device(B, E * K, N, br, bc)
    want = torch.empty((rows, N), dtype=torch.float32)
    for e in range(E):
        r0, r1 = int(offsets[e]), int(offsets[e + 1])
        want[r0:r1] = (A[r0:r1].double() @ B[e * K:(e + 1) * K].double()).float()
    g = guarded_out((rows, N), torch.float32)
    tl.gemm_grouped(A.to(DEV), Bd, g.t, torch.from_numpy(offsets).to(DEV), E, rows, N, K, G, br, bc)
    tl.device_status()
    assert tl.gemm_last_plan().generic_path == (3 if bc in (2, 4) else 2)
    assert torch.equal(g.check().cpu(), want)
    # prefill-sized: the CTA-pair kernel reads the same operand image
    M, N, K = 700, 9600, 256
    A = inputs.bf16_integers((M, K), -8, 8, seed=41)
    B = inputs.bf16_integers((K, N), -8, 8, seed=42)
    Bd = tile_major_on_device(B, K, N, br, bc)
    C = run_gemm(A, Bd, M, N, K, br, bc)
    plan = tl.gemm_last_plan()
    if bc in (2, 4):
        assert plan.pair_kernel == 0 and plan.generic_path == 3           # the pair kernel has no warps for the fix-up
    elif bc == 1 or br <= 64:
        assert plan.pair_kernel == 1 and plan.generic_path == 2
    assert torch.equal(C.cpu(), (A.double() @ B.double()).float())


SHAPES = [  # M, N, K
    (1, 512, 512), (8, 1024, 2048), (33, 640, 1024), (64, 256, 8192), (100, 384, 320),
    (300, 1152, 576), (257, 128, 64), (16, 8192, 1024),
]


@pytest.mark.parametrize("M,N,K", SHAPES)
@pytest.mark.parametrize("br,bc", [(16, 128), (32, 64), (0, 0), (8, 2), (16, 32), (1, 64)])
def test_integer_inputs_are_bit_exact(M, N, K, br, bc):
    from gpu_util import DEV, run_gemm, tile_major_on_device
    A = inputs.bf16_integers((M, K), -8, 8, seed=M + N)
    B = inputs.bf16_integers((K, N), -8, 8, seed=K)
    Bd = tile_major_on_device(B, K, N, br, bc) if br else B.to(DEV)
    layout = TILE if br else ROW
    C = run_gemm(A, Bd, M, N, K, br, bc)
    ref, _ = _oracle_full(A, Bd, layout, br, bc, M, N, K) if M * N * K <= 2 ** 28 else (None, None)
    if ref is None:
        ii, jj = np.divmod(np.arange(0, M * N, max(1, M * N // 20000)), N)
        ref_s, _ = tlo.matmul_at(inputs.bits(A), inputs.bits(Bd.reshape(-1)), layout, br, bc, M, N, K, ii, jj)
        assert np.array_equal(C.cpu().numpy()[ii, jj].astype(np.float64), ref_s)
    else:
        assert np.array_equal(C.cpu().numpy().astype(np.float64), ref)


@pytest.mark.parametrize("cta", [(16, 128, 64), (32, 128, 64), (64, 128, 128), (128, 128, 64), (256, 128, 64),
                                 (128, 256, 64), (64, 256, 128), (256, 128, 128), (64, 64, 64), (256, 64, 64),
                                 (128, 64, 128)])
def test_every_cta_tile_random_data(cta):
    from gpu_util import check_against_oracle, run_gemm, tile_major_on_device
    M, N, K, br, bc = 200, 768, 1024, 16, 128
    A = inputs.bf16_normal((M, K), 1.0, seed=11)
    B = inputs.bf16_normal((K, N), 0.02, seed=12)
    Bt = tile_major_on_device(B, K, N, br, bc)
    C = run_gemm(A, Bt, M, N, K, br, bc, cta)
    check_against_oracle(C, A, Bt, TILE, br, bc, M, N, K)


def _sweep_layouts():
    """Config 5: G x aspect (block rows 1, 8, 16, 32; block columns G / (2 rows)); invalid combinations skipped."""
    out = []
    for G in (32, 256, 1024, 4096, 16384):
        for br in (1, 8, 16, 32):
            bc = G // (2 * br)
            if bc >= 1:
                out.append((G, br, bc))
    return out


@pytest.mark.parametrize("G,br,bc", _sweep_layouts())
def test_granularity_sweep_layouts_every_cta_tile(G, br, bc):
    # Same layouts, CTA tiles, M and the full 8192 x 8192 weight of the benchmark's sweep; integer data, so
    # every sampled output must match the oracle exactly.
    from gpu_util import DEV, run_gemm, tile_major_on_device, tl
    K, N = 8192, 8192
    B = inputs.bf16_integers((K, N), -8, 8, seed=G + br, device=DEV)
    Bd = tile_major_on_device(B, K, N, br, bc)
    for M in (1, 16, 128):
        A = inputs.bf16_integers((M, K), -8, 8, seed=M)
        rng = np.random.default_rng(M)
        ii, jj = rng.integers(0, M, 150), rng.integers(0, N, 150)
        ii[:2], jj[:2] = [0, M - 1], [0, N - 1]
        ref, _ = tlo.matmul_at(inputs.bits(A), inputs.bits(Bd.reshape(-1)), TILE, br, bc, M, N, K, ii, jj)
        for cta in ((64, 64, 128), (128, 128, 128), (256, 128, 64), (64, 64, 64)):
            C = run_gemm(A, Bd, M, N, K, br, bc, cta)
            assert np.array_equal(C.cpu().numpy()[ii, jj].astype(np.float64), ref), (M, cta)
            assert torch.isfinite(C).all()


@pytest.mark.parametrize("br,bc", [(16, 128), (32, 64), (64, 64), (0, 0)])
def test_cta_pair_kernel_ragged_shapes(br, bc):
    # Large dense problems run on CTA pairs (256 x 256 tiles, cta_group::2 MMAs).  700 rows leave a 188-row
    # tail tile; 9600 columns are 37.5 pair tiles, so the last pair has only its first CTA in range.
    from gpu_util import DEV, run_gemm, tile_major_on_device
    M, N, K = 700, 9600, 320
    B = inputs.bf16_integers((K, N), -8, 8, seed=3)
    Bd = tile_major_on_device(B, K, N, br, bc) if br else B.to(DEV)
    A = inputs.bf16_integers((M, K), -8, 8, seed=4)
    C = run_gemm(A, Bd, M, N, K, br, bc)
    assert torch.isfinite(C).all()
    rng = np.random.default_rng(0)
    ii = np.concatenate([rng.integers(0, M, 3000), np.full(64, M - 1), np.arange(M)])
    jj = np.concatenate([rng.integers(0, N, 3000), np.arange(N - 64, N), np.full(M, N - 1)])
    ref, _ = tlo.matmul_at(inputs.bits(A), inputs.bits(Bd.reshape(-1)), TILE if br else ROW, br, bc, M, N, K, ii, jj)
    assert np.array_equal(C.cpu().numpy()[ii, jj].astype(np.float64), ref)
    A1, ks = inputs.one_hot_rows(M, K, seed=5)
    assert torch.equal(run_gemm(A1, Bd, M, N, K, br, bc).cpu(), B.float()[ks])


@pytest.mark.parametrize("M,N", [(1800, 5120), (1224, 7680), (4096, 2560)])
def test_cta_pair_kernel_512_token_tiles_and_their_remainder(M, N):
    # Whole waves of clusters take 512-token tiles, what is left of the tile grid runs as 256-token tiles; the last
    # 512-row m-tile is ragged (264 rows: eight in its second block; 200 rows: second block absent).
    from gpu_util import run_gemm, tile_major_on_device
    K, br, bc = 384, 16, 128
    B = inputs.bf16_integers((K, N), -8, 8, seed=13)
    Bd = tile_major_on_device(B, K, N, br, bc)
    A = inputs.bf16_integers((M, K), -8, 8, seed=14)
    C = run_gemm(A, Bd, M, N, K, br, bc)
    want = (A.to(torch.float64) @ B.to(torch.float64)).to(torch.float32)          # exact integers
    rng = np.random.default_rng(2)
    ii, jj = rng.integers(0, M, 2000), rng.integers(0, N, 2000)
    ref, _ = tlo.matmul_at(inputs.bits(A), inputs.bits(Bd.reshape(-1)), TILE, br, bc, M, N, K, ii, jj)
    assert np.array_equal(C.cpu().numpy()[ii, jj].astype(np.float64), ref)
    assert torch.equal(C.cpu(), want)                                             # every element, against the exact product


def test_all_ones_B_gives_row_sums():
    from gpu_util import DEV, run_gemm, tile_major_on_device
    M, N, K = 8, 256, 4096
    A = inputs.bf16_integers((M, K), -3, 3, seed=5)
    B = torch.ones((K, N), dtype=torch.bfloat16)
    C = run_gemm(A, tile_major_on_device(B, K, N, 16, 128), M, N, K, 16, 128)
    want = A.float().sum(dim=1, keepdim=True).expand(M, N)
    assert torch.equal(C.cpu(), want)


def test_results_are_reproducible_run_to_run():
    from gpu_util import run_gemm, tile_major_on_device
    M, N, K = 32, 1024, 8192          # stream-K with partial tiles
    A = inputs.bf16_normal((M, K), 1.0, seed=1)
    Bt = tile_major_on_device(inputs.bf16_normal((K, N), 0.02, seed=2), K, N, 16, 128)
    C0 = run_gemm(A, Bt, M, N, K, 16, 128)
    for _ in range(5):
        assert torch.equal(run_gemm(A, Bt, M, N, K, 16, 128), C0)


@pytest.mark.parametrize("name,K,N", inputs.LLAMA70B_PROJ)
@pytest.mark.parametrize("M", inputs.LLAMA_DECODE_M)
def test_llama_decode_full_size_sampled(name, K, N, M):
    # Same sizes and launch configuration (library heuristic) as the benchmark; 600 sampled outputs.
    from gpu_util import DEV, check_against_oracle, run_gemm, sample_indices
    from gpu_util import tl
    A = inputs.bf16_normal((M, K), 1.0, seed=31 + M)
    B = inputs.bf16_normal((K, N), 0.02, seed=(K % 997) + (N % 991), device=DEV)
    Bt = torch.empty_like(B)
    tl.relayout(B, Bt, K, N, 2, 4096, 16, 128, tl.TO_TILE_MAJOR)
    C = run_gemm(A, Bt, M, N, K, 16, 128)
    check_against_oracle(C, A, Bt, TILE, 16, 128, M, N, K, idx=sample_indices(M, N, 600, seed=M))
    # property that holds at any size: the row-major comparator gives the same bits
    assert torch.equal(run_gemm(A, B, M, N, K, 0, 0), C)


@pytest.mark.parametrize("name,K,N", inputs.LLAMA70B_PROJ)
def test_llama_prefill_full_size_sampled(name, K, N):
    from gpu_util import DEV, check_against_oracle, run_gemm, sample_indices, tl
    M = inputs.LLAMA_PREFILL_M
    A = inputs.bf16_normal((M, K), 1.0, seed=41, device=DEV)
    B = inputs.bf16_normal((K, N), 0.02, seed=42, device=DEV)
    Bt = torch.empty_like(B)
    tl.relayout(B, Bt, K, N, 2, 4096, 16, 128, tl.TO_TILE_MAJOR)
    C = run_gemm(A, Bt, M, N, K, 16, 128)
    ii, jj = sample_indices(M, N, 1500, seed=4)
    # plus one full column and a strided row through every tile
    cols = np.arange(0, N, 7)
    ii = np.concatenate([ii, np.full(cols.size, 1234), np.arange(M)])
    jj = np.concatenate([jj, cols, np.full(M, 4321)])
    Cs = C[torch.from_numpy(ii).to(DEV), torch.from_numpy(jj).to(DEV)]
    assert torch.isfinite(C).all()
    ref, S = tlo.matmul_at(inputs.bits(A.cpu()), inputs.bits(Bt.reshape(-1)), TILE, 16, 128, M, N, K, ii, jj)
    err = np.abs(Cs.cpu().numpy().astype(np.float64) - ref)
    assert np.all(err <= 1e-3 * S) and float(np.max(err / np.maximum(S, 1e-300))) <= 1e-4


def _grouped_case(E, tokens, topk, K, N, br, bc, seed, cta=(0, 0, 0), integer=False):
    from gpu_util import DEV, tl
    offsets, counts, _ = inputs.zipf_topk_routing(tokens, E, topk, 1.1, seed=seed)
    rows = int(offsets[-1])
    gen = (lambda shape, s: inputs.bf16_integers(shape, -8, 8, seed=s)) if integer else \
        (lambda shape, s: inputs.bf16_normal(shape, 1.0 if len(shape) == 2 else 0.02, seed=s))
    A = gen((rows, K), seed + 1)
    B = gen((E, K, N), seed + 2)
    Bd = B.to(DEV)
    if br:
        Bt = torch.empty_like(Bd)
        # experts are separate matrices laid end to end: relayout each (equal to one stacked E*K x N relayout)
        tl.relayout(Bd, Bt, E * K, N, 2, br * bc * 2, br, bc, tl.TO_TILE_MAJOR)
        Bd = Bt
    from gpu_util import guarded_out
    g = guarded_out((rows, N), torch.float32)
    tl.gemm_grouped(A.to(DEV), Bd, g.t, torch.from_numpy(offsets).to(DEV), E, rows, N, K,
                    br * bc * 2, br, bc, cta)
    tl.device_status()
    return offsets, counts, A, Bd, g.check()


def _check_grouped(offsets, A, Bd, C, E, K, N, br, bc, samples_per_expert, exact):
    layout = TILE if br else ROW
    Ch = C.cpu().numpy().astype(np.float64)
    assert np.all(np.isfinite(Ch))
    rng = np.random.default_rng(0)
    worst = 0.0
    for e in range(E):
        r0, r1 = int(offsets[e]), int(offsets[e + 1])
        if r1 == r0:
            continue
        Me = r1 - r0
        Be = inputs.bits(Bd[e].reshape(-1))
        Ae = inputs.bits(A[r0:r1])
        ii = rng.integers(0, Me, samples_per_expert)
        jj = rng.integers(0, N, samples_per_expert)
        ii[:2] = [0, Me - 1]
        jj[:2] = [0, N - 1]
        ref, S = tlo.matmul_at(Ae, Be, layout, br, bc, Me, N, K, ii, jj)
        got = Ch[r0 + ii, jj]
        if exact:
            assert np.array_equal(got, ref), f"expert {e}"
        else:
            assert np.all(np.abs(got - ref) <= 1e-3 * S), f"expert {e}"
            worst = max(worst, float(np.max(np.abs(got - ref) / np.maximum(S, 1e-300))))
    assert worst <= 1e-4


@pytest.mark.parametrize("br,bc", [(16, 128), (32, 64), (0, 0), (8, 16), (16, 1)])
def test_grouped_small_integer_exact(br, bc):
    E, K, N = 8, 256, 384
    offsets, counts, A, Bd, C = _grouped_case(E, 40, 3, K, N, br, bc, seed=3, integer=True)
    _check_grouped(offsets, A, Bd, C, E, K, N, br, bc, samples_per_expert=400, exact=True)


def test_grouped_with_empty_experts_and_small_tile_cap():
    from gpu_util import DEV, tl
    E, K, N = 6, 128, 256
    offsets = np.array([0, 0, 70, 70, 71, 200, 200], dtype=np.int32)
    A = inputs.bf16_integers((200, K), -8, 8, seed=1)
    B = inputs.bf16_integers((E, K, N), -8, 8, seed=2)
    Bt = torch.empty((E, K, N), dtype=torch.bfloat16, device=DEV)
    tl.relayout(B.to(DEV), Bt, E * K, N, 2, 4096, 16, 128, tl.TO_TILE_MAJOR)
    C = torch.full((200, N), float("nan"), dtype=torch.float32, device=DEV)
    tl.gemm_grouped(A.to(DEV), Bt, C, torch.from_numpy(offsets).to(DEV), E, 200, N, K, 4096, 16, 128, (32, 128, 64))
    tl.device_status()
    _check_grouped(offsets, A, Bt, C, E, K, N, 16, 128, samples_per_expert=300, exact=True)


@pytest.mark.parametrize("name,K,N", inputs.QWEN_MOE_PROJ)
def test_qwen_moe_full_size_sampled(name, K, N):
    q = inputs.QWEN_MOE
    offsets, counts, A, Bd, C = _grouped_case(q["experts"], q["tokens"], q["topk"], K, N, 16, 128, seed=0)
    assert int(offsets[-1]) == q["tokens"] * q["topk"]
    _check_grouped(offsets, A, Bd, C, q["experts"], K, N, 16, 128, samples_per_expert=48, exact=False)


@pytest.mark.parametrize("tokens,want_cta", [(512, (64, 256, 64)), (1024, (128, 256, 64))])
@pytest.mark.parametrize("name,K,N", inputs.QWEN_MOE_PROJ)
def test_qwen_moe_with_more_tokens_runs_larger_tiles(name, K, N, tokens, want_cta):
    # more rows per expert than the benchmark's routing leaves: the library's grouped tile grows with the average
    from gpu_util import tl
    q = inputs.QWEN_MOE
    offsets, counts, A, Bd, C = _grouped_case(q["experts"], tokens, q["topk"], K, N, 16, 128, seed=1, integer=True)
    p = tl.gemm_last_plan()
    assert p.cta == want_cta and p.stream_k == 0
    _check_grouped(offsets, A, Bd, C, q["experts"], K, N, 16, 128, samples_per_expert=64, exact=True)
    # every element of the busiest and of the smallest expert against the exact integer product
    order = np.argsort(counts)
    for e in (int(order[-1]), int(order[np.nonzero(counts[order])[0][0]])):
        r0, r1 = int(offsets[e]), int(offsets[e + 1])
        want = A[r0:r1].double() @ inputs_from_tile_major(Bd[e], K, N).double()
        assert torch.equal(C[r0:r1].cpu().double(), want)


def inputs_from_tile_major(Bt_e, K, N):
    """One expert's K x N weights back in row-major order (host side, for exact checks)."""
    return Bt_e.cpu().reshape(K // 16, N // 128, 16, 128).permute(0, 2, 1, 3).reshape(K, N)


@pytest.mark.parametrize("name,K,N", inputs.QWEN_ATTN_PROJ)
def test_qwen_attention_projections(name, K, N):
    from gpu_util import check_against_oracle, run_gemm, sample_indices, tile_major_on_device
    M = 256
    A = inputs.bf16_normal((M, K), 1.0, seed=51)
    Bt = tile_major_on_device(inputs.bf16_normal((K, N), 0.02, seed=52), K, N, 16, 128)
    C = run_gemm(A, Bt, M, N, K, 16, 128)
    check_against_oracle(C, A, Bt, TILE, 16, 128, M, N, K, idx=sample_indices(M, N, 4000, seed=5))


def test_host_buffer_entry_point():
    from gpu_util import DEV, tl
    M, N, K = 8, 512, 1024
    A = inputs.bf16_integers((M, K), -8, 8, seed=1).pin_memory()
    B = inputs.bf16_integers((K, N), -8, 8, seed=2).pin_memory()
    C = torch.empty((M, N), dtype=torch.float32).pin_memory()
    scratch = torch.empty(tl.gemm_host_scratch_bytes(M, N, K), dtype=torch.uint8, device=DEV)
    tl.gemm_host(A, B, C, M, N, K, scratch)
    ref, _ = tlo.matmul(inputs.bits(A), inputs.bits(B), ROW, 0, 0, M, N, K)
    assert np.array_equal(C.numpy().astype(np.float64), ref)


def test_caller_workspace_and_errors():
    from gpu_util import DEV, run_gemm, tile_major_on_device, tl
    M, N, K = 16, 2304, 28672              # 9 tiles of long K, 132 MB of weights: cut stream-K fashion, through a workspace
    A = inputs.bf16_integers((M, K), -8, 8, seed=1)
    Bt = tile_major_on_device(inputs.bf16_integers((K, N), -8, 8, seed=2), K, N, 16, 128)
    want = run_gemm(A, Bt, M, N, K, 16, 128)
    assert tl.gemm_last_plan().stream_k == 1 and tl.gemm_last_plan().workspace_bytes > 0
    need = tl.gemm_workspace_bytes(M, N, K)
    assert need > 0
    ws = torch.empty(need, dtype=torch.uint8, device=DEV)
    tl.set_workspace(ws)
    try:
        assert torch.equal(run_gemm(A, Bt, M, N, K, 16, 128), want)
        small = torch.empty(1024, dtype=torch.uint8, device=DEV)
        tl.set_workspace(small)
        with pytest.raises(tl.TileLensError) as e:
            run_gemm(A, Bt, M, N, K, 16, 128)
        assert e.value.status == 6
    finally:
        tl.set_workspace(None)
    with pytest.raises(tl.TileLensError) as e:
        run_gemm(A, Bt, M, N, K, 16, 128, cta=(48, 128, 64))
    assert e.value.status == 2
    C = torch.zeros((0, N), dtype=torch.float32, device=DEV)
    tl.gemm(A.to(DEV)[:0], Bt, C, 0, N, K, 4096, 16, 128)          # no rows: no-op


def test_products_on_two_streams_with_their_own_workspaces_match_serial_runs():
    # The header's rule for concurrent calls: each needs its own split-K workspace (the pointer travels with the
    # launch).  Two decode-shaped products on two streams, repeated, must give the bits of the serial runs.
    from gpu_util import DEV, tile_major_on_device, tl
    shapes = [(8, 1280, 28672), (32, 2304, 28672)]                      # (M, N, K): both cut stream-K fashion
    A, Bt, want, ws = [], [], [], []
    for i, (M, N, K) in enumerate(shapes):
        A.append(inputs.bf16_normal((M, K), 1.0, seed=40 + i).to(DEV))
        Bt.append(tile_major_on_device(inputs.bf16_normal((K, N), 0.02, seed=50 + i), K, N, 16, 128))
        C = torch.empty((M, N), dtype=torch.float32, device=DEV)
        tl.gemm(A[i], Bt[i], C, M, N, K, 4096, 16, 128)
        assert tl.gemm_last_plan().stream_k == 1 and tl.gemm_last_plan().workspace_bytes > 0
        want.append(C)
        ws.append(torch.empty(tl.gemm_workspace_bytes(M, N, K) + 256, dtype=torch.uint8, device=DEV))
    tl.device_status()
    streams = [torch.cuda.Stream(device=DEV) for _ in shapes]
    torch.cuda.synchronize()
    try:
        for rep in range(10):
            got = [torch.full_like(w, float("nan")) for w in want]
            for i, (M, N, K) in enumerate(shapes):
                tl.set_workspace(ws[i])
                for _ in range(3):                                       # keep both streams busy at the same time
                    tl.gemm(A[i], Bt[i], got[i], M, N, K, 4096, 16, 128, stream=streams[i])
            torch.cuda.synchronize()
            for g, w in zip(got, want):
                assert torch.equal(g, w)
    finally:
        tl.set_workspace(None)
    tl.device_status()
