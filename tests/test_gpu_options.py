"""Code paths behind the library's switches, the plan query, the give-up path and concurrent host threads (GPU).

Every switch selects between two ways of computing the same thing, so each test flips one switch in-process
(tl_set_option), runs a product or a relayout whose result is exact (integer-valued or one-hot inputs, bytes), and
compares it with the oracle and with the default path, bit for bit.
"""
import threading

import numpy as np
import pytest
import torch

import oracle as tlo
from paper_2607_04031_b200 import inputs

pytestmark = pytest.mark.gpu
ROW, TILE = tlo.ROW_MAJOR, tlo.TILE_MAJOR


def _int_case(M, N, K, br, bc, seed):
    from gpu_util import DEV, tile_major_on_device
    A = inputs.bf16_integers((M, K), -8, 8, seed=seed)
    B = inputs.bf16_integers((K, N), -8, 8, seed=seed + 1)
    Bd = tile_major_on_device(B, K, N, br, bc) if br else B.to(DEV)
    want = (A.to(torch.float64) @ B.to(torch.float64)).to(torch.float32)     # exact: integers below 2^24
    return A, Bd, want


@pytest.mark.parametrize("M,N,K,want_plan", [
    (128, 256 * 112, 512, ((128, 256, 64), 0, 1, 112)),       # whole wide tiles on 112 CTAs
    (200, 10240, 4608, ((128, 128, 128), 1, 1, 148)),         # 80 wide tiles would have to be cut: the narrow tile (also cut)
    (100, 10240, 4096, ((128, 256, 64), 0, 3, 120)),          # 40 wide tiles, split-K in clusters of 3
    (300, 4096, 4096, ((128, 256, 64), 0, 2, 96)),            # 48 wide tiles in clusters of 2 against a cut of the narrow ones
    (256, 512, 2048, ((128, 128, 128), 0, 4, 32)),            # small weights: the narrow tile
])
def test_products_between_decode_and_prefill_are_exact_on_the_tile_the_library_picks(M, N, K, want_plan):
    from gpu_util import run_gemm, tl
    A, Bd, want = _int_case(M, N, K, 16, 128, seed=M + N)
    got = run_gemm(A, Bd, M, N, K, 16, 128)
    p = tl.gemm_last_plan()
    assert (p.cta, p.stream_k, p.cluster_k, p.grid) == want_plan, p.as_dict()
    assert torch.equal(got.cpu(), want)
    for cta in ((128, 256, 64), (128, 128, 128)):             # and both candidates give the same bits (exact integers)
        assert torch.equal(run_gemm(A, Bd, M, N, K, 16, 128, cta).cpu(), want)


@pytest.mark.parametrize("M,N,K", [(256, 256 * 112, 512), (200, 256 * 112, 320), (130, 256 * 148, 64), (300, 256 * 148, 256),
                                   (512, 256 * 74, 192), (257, 256 * 148 + 128, 128)])
def test_tiles_of_two_token_blocks_are_exact(M, N, K):
    # 256 x 256 x 64 in the weights-on-N kernel: one weight slab per stage, two 128-row token blocks, both accumulators
    # owned by the tile.  Whole, ragged and single-block last tiles; fp32 and bf16 C; the [N][K] flavour and FP8.
    from gpu_util import DEV, guarded_out, run_gemm, tl
    A, Bd, want = _int_case(M, N, K, 16, 128, seed=M + K)
    got = run_gemm(A, Bd, M, N, K, 16, 128, (256, 256, 64))
    p = tl.gemm_last_plan()
    assert p.cta == (256, 256, 64) and p.stream_k == 0 and p.cluster_k == 1 and p.pair_kernel == 0 and p.weights_on_n == 1
    assert torch.equal(got.cpu(), want)
    g = guarded_out((M, N), torch.bfloat16)
    tl.gemm_bf16(A.to(DEV), Bd, g.t, M, N, K, 4096, 16, 128, (256, 256, 64))
    tl.device_status()
    assert torch.equal(g.check().cpu(), want.to(torch.bfloat16))
    if M <= 256:                  # the library's own choice for 129 to 256 rows and a short K loop: CTA pairs
        got = run_gemm(A, Bd, M, N, K, 16, 128)
        assert tl.gemm_last_plan().pair_kernel == 1 and tl.gemm_last_plan().pair_tiles_512 == 0
        assert torch.equal(got.cpu(), want)
    # K-contiguous weights, bf16 and FP8
    Bh = inputs.bf16_integers((K, N), -8, 8, seed=M + K + 1)
    Wnk = Bh.t().contiguous().to(DEV)
    C = guarded_out((M, N), torch.float32)
    tl.gemm_kmajor(A.to(DEV), Wnk, C.t, M, N, K, 0, 0, 0, (256, 256, 64))
    tl.device_status()
    assert tl.gemm_last_plan().cta == (256, 256, 64) and torch.equal(C.check().cpu(), want)
    if K % 128 != 0:                                          # (the plain FP8 array wants whole 128-byte rows)
        return
    A8, B8 = inputs.fp8_integers((M, K), -6, 6, seed=M), inputs.fp8_integers((K, N), -6, 6, seed=N)
    C = guarded_out((M, N), torch.float32)
    tl.gemm_fp8_kmajor(A8.to(DEV), B8.t().contiguous().to(DEV), C.t, M, N, K, 0, 0, 0, (256, 256, 128))
    tl.device_status()
    assert torch.equal(C.check().cpu().double(), A8.double() @ B8.double())


@pytest.mark.parametrize("M,N,K,want", [(1024, 8192, 256, ("two", 128)),     # 128 tiles: one wave of two-block tiles
                                        (640, 10240, 192, ("two", 120)),
                                        (768, 256 * 74, 2176, ("pair", 0)),    # two waves of half-empty 512-token tiles: small only
                                        (1024, 256 * 224, 64, ("pair", 444))])
def test_a_few_waves_above_512_rows_are_exact_on_the_schedule_the_library_picks(M, N, K, want):
    from gpu_util import run_gemm, tl
    A, Bd, exact = _int_case(M, N, K, 16, 128, seed=M + N)
    got = run_gemm(A, Bd, M, N, K, 16, 128)
    p = tl.gemm_last_plan()
    if want[0] == "two":
        assert (p.pair_kernel, p.cta, p.grid) == (0, (256, 256, 64), want[1])
    else:
        assert p.pair_kernel == 1 and p.pair_tiles_512 == want[1]
    assert torch.equal(got.cpu(), exact)


def test_a_tile_of_two_token_blocks_is_refused_where_it_would_be_cut():
    from gpu_util import run_gemm, tl
    A, Bd, _ = _int_case(200, 1024, 512, 16, 128, seed=9)
    with pytest.raises(tl.TileLensError) as e:
        run_gemm(A, Bd, 200, 1024, 512, 16, 128, (256, 256, 64))          # 4 tiles: clusters or a cut, neither of which it has
    assert e.value.status == 2


def test_one_box_per_memory_tile_gives_the_same_bits():
    from gpu_util import run_gemm, tl
    M, N, K = 40, 1024, 1024
    for br, bc in ((16, 128), (32, 64), (8, 256)):
        A, Bd, want = _int_case(M, N, K, br, bc, seed=br)
        with tl.option(tl.OPT_BOX_PER_BLOCK, 1):
            got = run_gemm(A, Bd, M, N, K, br, bc, (64, 256, 64))          # 2 x 4 memory tiles of 16 x 128 per stage
            assert tl.get_option(tl.OPT_BOX_PER_BLOCK) == 1
        assert torch.equal(got.cpu(), want)
        assert torch.equal(run_gemm(A, Bd, M, N, K, br, bc, (64, 256, 64)).cpu(), want)
    # random data: same K order on both paths, so the same bits
    from gpu_util import tile_major_on_device
    A = inputs.bf16_normal((M, K), 1.0, seed=1)
    Bt = tile_major_on_device(inputs.bf16_normal((K, N), 0.02, seed=2), K, N, 16, 128)
    ref = run_gemm(A, Bt, M, N, K, 16, 128)
    with tl.option(tl.OPT_BOX_PER_BLOCK, 1):
        assert torch.equal(run_gemm(A, Bt, M, N, K, 16, 128), ref)


def test_256_token_pair_tiles_are_what_small_prefill_runs():
    # M <= 512 with at least 74 pair tiles: too few 512-token tiles to fill a wave of clusters, so the pair kernel
    # runs its 256-token instantiation by itself (no switch involved).
    from gpu_util import run_gemm, tl
    M, N, K = 512, 9728, 256
    A, Bd, want = _int_case(M, N, K, 16, 128, seed=5)
    got = run_gemm(A, Bd, M, N, K, 16, 128)
    plan = tl.gemm_last_plan()
    assert plan.pair_kernel == 1 and plan.cta_m == 256 and plan.pair_tiles_512 == 0
    assert torch.equal(got.cpu(), want)
    A1, ks = inputs.one_hot_rows(M, K, seed=6)
    B = inputs.bf16_normal((K, N), 0.02, seed=7)
    from gpu_util import tile_major_on_device
    assert torch.equal(run_gemm(A1, tile_major_on_device(B, K, N, 16, 128), M, N, K, 16, 128).cpu(), B.float()[ks])


@pytest.mark.parametrize("opt_name,value", [("OPT_PAIR_KERNEL", 0), ("OPT_PAIR_512", 0), ("OPT_PDL", 0),
                                            ("OPT_MAX_STAGES", 2), ("OPT_PREFETCH_STAGES", 0),
                                            ("OPT_PAIR_TMA_STORE", 0)])
def test_prefill_switches_give_the_exact_product(opt_name, value):
    from gpu_util import run_gemm, tl
    M, N, K = 1800, 5120, 384                      # 512-token tiles and their 256-token remainder by default
    A, Bd, want = _int_case(M, N, K, 16, 128, seed=11)
    with tl.option(getattr(tl, opt_name), value):
        got = run_gemm(A, Bd, M, N, K, 16, 128)
        plan = tl.gemm_last_plan()
    assert torch.equal(got.cpu(), want)
    if opt_name == "OPT_PAIR_KERNEL":
        assert plan.pair_kernel == 0 and plan.cta == (256, 128, 64)
    if opt_name == "OPT_PAIR_512":
        assert plan.pair_kernel == 1 and plan.cta_m == 256
    if opt_name == "OPT_MAX_STAGES":
        assert plan.pair_kernel == 1 and plan.stages == 2
    if opt_name == "OPT_PAIR_TMA_STORE":
        assert plan.pair_kernel == 1 and plan.pair_tiles_512 > 0 and plan.pair_tiles_256 > 0


@pytest.mark.parametrize("M,N,K", [(700, 9600, 320), (1800, 5120, 384), (385, 256 * 74, 64)])
def test_pair_kernel_store_paths_write_the_same_bits(M, N, K):
    # C through shared memory and tiled bulk stores (default) against plain stores from the accumulator registers:
    # fp32 and bf16 C, ragged rows and columns, nothing outside C touched (guard blocks on both sides).
    from gpu_util import DEV, guarded_out, run_gemm, tile_major_on_device, tl
    A = inputs.bf16_normal((M, K), 1.0, seed=M)
    Bt = tile_major_on_device(inputs.bf16_normal((K, N), 0.02, seed=N), K, N, 16, 128)
    got = {}
    for mode in (1, 0):
        with tl.option(tl.OPT_PAIR_TMA_STORE, mode):
            got[mode] = run_gemm(A, Bt, M, N, K, 16, 128, (256, 128, 64)).clone()      # (the pair kernel's tile, by name)
            assert tl.gemm_last_plan().pair_kernel == 1
            g = guarded_out((M, N), torch.bfloat16)
            tl.gemm_bf16(A.to(DEV), Bt, g.t, M, N, K, 4096, 16, 128, (256, 128, 64))
            tl.device_status()
            got[mode, "bf16"] = g.check().clone()
    assert torch.equal(got[1], got[0]) and torch.equal(got[1, "bf16"], got[0, "bf16"])
    assert torch.equal(got[1].to(torch.bfloat16), got[1, "bf16"])


@pytest.mark.parametrize("no_scratch", [1, 0])
@pytest.mark.parametrize("opt_name,value", [("OPT_UMMA_M128", 1), ("OPT_MAX_STAGES", 2), ("OPT_PREFETCH_STAGES", 0),
                                            ("OPT_PREFETCH_STAGES", 8), ("OPT_PDL", 0), ("OPT_REDUCE_SPLIT", 0)])
def test_decode_switches_give_the_same_bits(opt_name, value, no_scratch):
    # no_scratch = 1: the library's own choice (cluster split-K or whole tiles where such a plan exists);
    # no_scratch = 0: the stream-K cut with its reduction kernel.  A switch never changes the bits of either.
    from gpu_util import run_gemm, tile_major_on_device, tl
    with tl.option(tl.OPT_NO_SCRATCH_PLANS, no_scratch):
        for M, N, K in ((8, 2048, 4096), (32, 1024, 8192), (100, 640, 2048), (16, 8192, 2048)):
            A = inputs.bf16_normal((M, K), 1.0, seed=M)
            Bt = tile_major_on_device(inputs.bf16_normal((K, N), 0.02, seed=N), K, N, 16, 128)
            ref = run_gemm(A, Bt, M, N, K, 16, 128)
            with tl.option(getattr(tl, opt_name), value):
                got = run_gemm(A, Bt, M, N, K, 16, 128)
                if opt_name == "OPT_MAX_STAGES":
                    assert tl.gemm_last_plan().stages == 2
            assert torch.equal(got, ref), (M, N, K)
            Ai, Bi, want = _int_case(M, N, K, 16, 128, seed=K)
            with tl.option(getattr(tl, opt_name), value):
                assert torch.equal(run_gemm(Ai, Bi, M, N, K, 16, 128).cpu(), want)


CLUSTER_CASES = [  # M, N, K, expected cluster size on a 148-SM part (0: some other schedule)
    # (64 x 6144 x 512: too few tiles to fill the SMs with clusters, but only 6 MB of weights: clusters all the same;
    #  16 tiles: 15 clusters of 8 CTAs can be resident, 22 of 6; 37 tiles: 33 clusters of 4, 45 of 3)
    (1, 8192, 8192, 4), (8, 10240, 8192, 3), (32, 8192, 28672, 4), (16, 4096, 1024, 6), (64, 6144, 512, 4),
    (8, 5120, 64, 0), (40, 9472, 2048, 3), (8, 8192, 192, 0), (24, 57344, 1024, 0), (3, 18944, 3584, 2),
    (8, 10112, 4096, 3),
]


@pytest.mark.parametrize("M,N,K,want_s", CLUSTER_CASES)
@pytest.mark.parametrize("br,bc", [(16, 128), (0, 0), (32, 64)])
def test_cluster_split_k_against_the_oracle_and_the_stream_k_cut(M, N, K, want_s, br, bc):
    # One tile per cluster, the K loop split over its CTAs, partial tiles added through distributed shared memory in
    # rank (= K) order: exact on integers, inside the tolerance on random data, bit-reproducible, ragged K shares
    # (K / 64 not a multiple of the cluster size), clipped last tiles (N not a multiple of 256), bf16 output.
    from gpu_util import DEV, check_against_oracle, guarded_out, run_gemm, sample_indices, tile_major_on_device, tl
    layout = TILE if br else ROW
    A, Bd, want = _int_case(M, N, K, br, bc, seed=M + K)
    got = run_gemm(A, Bd, M, N, K, br, bc)
    plan = tl.gemm_last_plan()
    if torch.cuda.get_device_properties(0).multi_processor_count == 148:
        assert plan.cluster_k == (want_s if want_s else 1), plan.as_dict()
        assert plan.workspace_bytes == 0 or want_s == 0
    assert torch.equal(got.cpu(), want)
    Ar = inputs.bf16_normal((M, K), 1.0, seed=1)
    Br = inputs.bf16_normal((K, N), 0.02, seed=2)
    Brd = tile_major_on_device(Br, K, N, br, bc) if br else Br.to(DEV)
    C = run_gemm(Ar, Brd, M, N, K, br, bc)
    check_against_oracle(C, Ar, Brd, layout, br, bc, M, N, K, idx=sample_indices(M, N, 3000, seed=3))
    for _ in range(3):
        assert torch.equal(run_gemm(Ar, Brd, M, N, K, br, bc), C)
    g = guarded_out((M, N), torch.bfloat16)
    tl.gemm_bf16(Ar.to(DEV), Brd, g.t, M, N, K, br * bc * 2, br, bc)
    tl.device_status()
    assert torch.equal(g.check(), C.to(torch.bfloat16))                 # the same fp32 sums, rounded once


@pytest.mark.parametrize("limit", [100, 37, 1])
def test_sm_limit_caps_the_grid_and_keeps_the_product_exact(limit):
    from gpu_util import run_gemm, tl
    for M, N, K in ((8, 2048, 4096), (200, 1024, 512), (1800, 5120, 384)):
        A, Bd, want = _int_case(M, N, K, 16, 128, seed=M)
        with tl.option(tl.OPT_SM_LIMIT, limit):
            got = run_gemm(A, Bd, M, N, K, 16, 128)
            plan = tl.gemm_last_plan()
        assert torch.equal(got.cpu(), want)
        assert plan.pair_kernel == 1 or plan.grid <= limit, plan.as_dict()      # (the CTA-pair kernel keeps its own grid)


@pytest.mark.parametrize("cap", [16, 64, 128])
def test_grouped_row_cap_keeps_the_products_exact(cap):
    # tiles of up to 128 token rows per expert: 128-row MMAs for the large experts, 64-row ones for the rest
    from gpu_util import DEV, guarded_out, tl
    E, K, N = 12, 512, 768
    offsets, counts, expert_of_row = inputs.zipf_topk_routing(160, E, 3, 1.1, seed=7)
    rows = int(offsets[-1])
    assert counts.max() > 64                                                      # at least one expert needs the 128-row path
    A = inputs.bf16_integers((rows, K), -8, 8, seed=1)
    B = inputs.bf16_integers((E, K, N), -8, 8, seed=2)
    Bt = torch.empty((E, K, N), dtype=torch.bfloat16, device=DEV)
    tl.relayout(B.to(DEV), Bt, E * K, N, 2, 4096, 16, 128, tl.TO_TILE_MAJOR)
    want = torch.empty((rows, N), dtype=torch.float32)
    for e in range(E):
        r0, r1 = int(offsets[e]), int(offsets[e + 1])
        want[r0:r1] = (A[r0:r1].double() @ B[e].double()).float()
    with tl.option(tl.OPT_MOE_ROW_CAP, cap):
        g = guarded_out((rows, N), torch.float32)
        tl.gemm_grouped(A.to(DEV), Bt, g.t, torch.from_numpy(offsets).to(DEV), E, rows, N, K, 4096, 16, 128)
        assert tl.gemm_last_plan().cta_m == cap
        tl.device_status()
    assert torch.equal(g.check().cpu(), want)


def test_grouped_tables_built_ahead_of_the_wait_are_checked_and_rebuilt():
    # A grouped kernel reads the expert offsets and builds its tile tables while its predecessor in the stream may still
    # be running, then reads the offsets again after waiting for it and rebuilds the tables if one differs.
    # (a) test hook: the provisional tables come from offsets 7 rows off; (b) the offsets really are written by the
    # kernel just before the product in the stream, over a stale routing.  Both must give the exact product.
    from gpu_util import DEV, guarded_out, tile_major_on_device, tl
    E, N, K = 24, 1024, 512
    offsets, counts, _ = inputs.zipf_topk_routing(96, E, 4, 1.1, seed=3)
    stale, _, _ = inputs.zipf_topk_routing(96, E, 4, 0.3, seed=9)
    rows = int(offsets[-1])
    assert int(stale[-1]) == rows and not np.array_equal(stale, offsets)
    A = inputs.bf16_integers((rows, K), -8, 8, seed=21)
    B = inputs.bf16_integers((E * K, N), -8, 8, seed=22)
    Bt = tile_major_on_device(B, E * K, N, 16, 128)
    want = torch.empty((rows, N), dtype=torch.float32)
    for e in range(E):
        r0, r1 = int(offsets[e]), int(offsets[e + 1])
        want[r0:r1] = (A[r0:r1].double() @ B[e * K:(e + 1) * K].double()).float()
    Ad, d_new = A.to(DEV), torch.from_numpy(offsets).to(DEV)
    d_off = d_new.clone()
    tl.set_option(tl.OPT_STALL_ONCE, 4)
    g = guarded_out((rows, N), torch.float32)
    tl.gemm_grouped(Ad, Bt, g.t, d_off, E, rows, N, K, 4096, 16, 128)
    assert tl.get_option(tl.OPT_STALL_ONCE) == 0
    tl.device_status()
    assert torch.equal(g.check().cpu(), want)
    for _ in range(5):
        d_off.copy_(torch.from_numpy(stale).to(DEV))
        torch.cuda.synchronize()
        g = guarded_out((rows, N), torch.float32)
        d_off.copy_(d_new)                                   # the product's stream predecessor writes the offsets
        tl.gemm_grouped(Ad, Bt, g.t, d_off, E, rows, N, K, 4096, 16, 128)
        tl.device_status()
        assert torch.equal(g.check().cpu(), want)


@pytest.mark.parametrize("E,rows_per_expert,K,N,host_cut", [(16, 128, 512, 1024, 0),    # the host rules the cut out
                                                            (96, 1, 512, 1024, 1),      # the kernel does, from 384 tiles
                                                            (12, 8, 512, 1024, 1),      # 48 tiles: cut over all CTAs
                                                            (96, 1, 4096, 1024, 1)])    # 64-stage tiles: cut
def test_grouped_products_with_and_without_the_cut_are_exact(E, rows_per_expert, K, N, host_cut):
    # Short tiles in sufficient number are handed out whole (no partial tiles, no reduction); otherwise what is left after
    # the whole rounds is cut along K.  Which of the two runs is decided from the tile count, by the host where the
    # row count alone settles it, else by the kernel (the reduction kernel then finds nothing to add).  Integer data:
    # every case must be exact.
    from gpu_util import DEV, guarded_out, tile_major_on_device, tl
    offsets = (np.arange(E + 1) * rows_per_expert).astype(np.int32)
    rows = int(offsets[-1])
    A = inputs.bf16_integers((rows, K), -8, 8, seed=E)
    B = inputs.bf16_integers((E * K, N), -8, 8, seed=K)
    Bt = tile_major_on_device(B, E * K, N, 16, 128)
    want = torch.empty((rows, N), dtype=torch.float32)
    for e in range(E):
        r0, r1 = int(offsets[e]), int(offsets[e + 1])
        want[r0:r1] = (A[r0:r1].double() @ B[e * K:(e + 1) * K].double()).float()
    g = guarded_out((rows, N), torch.float32)
    tl.gemm_grouped(A.to(DEV), Bt, g.t, torch.from_numpy(offsets).to(DEV), E, rows, N, K, 4096, 16, 128)
    assert tl.gemm_last_plan().stream_k == host_cut
    tl.device_status()
    assert torch.equal(g.check().cpu(), want)


def test_relayout_without_the_copy_engine_matches_the_oracle():
    from gpu_util import Guarded, dev_bytes, tl
    for rows, cols, s, br, bc in ((512, 512, 2, 16, 128), (1056, 2176, 2, 32, 64), (256, 1024, 1, 64, 64)):
        src = inputs.random_bytes(rows * cols * s, seed=rows + cols)
        want = tlo.relayout(src, rows, cols, s, br, bc, tlo.TO_TILE_MAJOR)
        with tl.option(tl.OPT_RELAYOUT_TMA, 0):
            g = Guarded((rows * cols * s,), torch.uint8)
            tl.relayout(dev_bytes(src), g.t, rows, cols, s, br * bc * s, br, bc, tl.TO_TILE_MAJOR)
            assert np.array_equal(g.check().cpu().numpy(), want)
            gb = Guarded((rows * cols * s,), torch.uint8)
            tl.relayout(dev_bytes(want), gb.t, rows, cols, s, br * bc * s, br, bc, tl.TO_ROW_MAJOR)
            assert np.array_equal(gb.check().cpu().numpy(), src)
            # a batch falls back to one call per matrix
            g2 = [Guarded((rows * cols * s,), torch.uint8) for _ in range(2)]
            tl.relayout_batch([dev_bytes(src)] * 2, [x.t for x in g2], [(rows, cols)] * 2, s, br * bc * s, br, bc)
            for x in g2:
                assert np.array_equal(x.check().cpu().numpy(), want)
    tl.device_status()


def test_set_option_rejects_what_it_does_not_know():
    from gpu_util import tl
    L = tl.lib()
    assert L.tl_set_option(99, 1) == 1 and L.tl_set_option(-1, 0) == 1
    assert L.tl_set_option(tl.OPT_PDL, 2) == 1
    assert L.tl_set_option(tl.OPT_WAIT_LIMIT_US, 5) == 1
    assert L.tl_set_option(tl.OPT_MAX_STAGES, 1) == 1
    assert L.tl_get_option(99) == -1
    assert tl.get_option(tl.OPT_WAIT_LIMIT_US) == 2_000_000


# ------------------------------------------------------------------------------------------------ the plan query

PLAN_CASES = [  # M, N, K, block, cta, E, flavour
    (1, 8192, 8192, (16, 128), (0, 0, 0), 0, 0), (8, 10240, 8192, (16, 128), (0, 0, 0), 0, 0),
    (32, 57344, 8192, (16, 128), (0, 0, 0), 0, 0), (32, 8192, 28672, (0, 0), (0, 0, 0), 0, 0),
    (128, 8192, 8192, (32, 64), (128, 128, 64), 0, 0), (16, 8192, 8192, (8, 2), (64, 64, 64), 0, 0),
    (4096, 8192, 8192, (16, 128), (0, 0, 0), 0, 0), (256, 4096, 2048, (16, 128), (0, 0, 0), 0, 0),
    (2048, 1536, 2048, (16, 128), (0, 0, 0), 128, 0), (2048, 2048, 768, (16, 128), (0, 0, 0), 128, 0),
    (8, 10240, 8192, (32, 64), (0, 0, 0), 0, 1), (8, 10240, 8192, (64, 64), (0, 0, 0), 0, 2),
]


@pytest.mark.parametrize("M,N,K,block,cta,E,flavour", PLAN_CASES)
def test_plan_query_equals_what_the_launch_ran(M, N, K, block, cta, E, flavour):
    from gpu_util import DEV, tl
    br, bc = block
    es = 1 if flavour == 2 else 2
    G = br * bc * es
    plan = tl.gemm_plan(M, N, K, G, br, bc, cta, E, flavour)
    A = torch.zeros((M, K), dtype=torch.uint8 if es == 1 else torch.bfloat16, device=DEV)
    W = torch.zeros((max(E, 1) * K * N,), dtype=torch.uint8 if es == 1 else torch.bfloat16, device=DEV)
    C = torch.empty((M, N), dtype=torch.float32, device=DEV)
    if E:
        # equal shares of the rows; the schedule on the host side depends on the totals only
        off = torch.tensor(np.linspace(0, M, E + 1).astype(np.int32), device=DEV)
        tl.gemm_grouped(A, W, C, off, E, M, N, K, G, br, bc, cta)
    elif flavour == 0:
        tl.gemm(A, W, C, M, N, K, G, br, bc, cta)
    elif flavour == 1:
        tl.gemm_kmajor(A, W, C, M, N, K, G, br, bc, cta)
    else:
        tl.gemm_fp8_kmajor(A, W, C, M, N, K, G, br, bc, cta)
    tl.device_status()
    assert tl.gemm_last_plan().as_dict() == plan.as_dict()
    assert plan.grid >= 1 and plan.stages >= 2
    if cta != (0, 0, 0):
        assert plan.cta == cta


def test_default_plans_of_the_benchmark_shapes():
    from gpu_util import tl
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    if sms != 148:
        pytest.skip("the expected grids below are those of a 148-SM B200")
    # decode: schedules without partial tiles in global memory
    p = tl.gemm_plan(8, 10240, 8192)                  # 40 tiles, clusters of 3 CTAs split K
    assert p.cta == (16, 256, 64) and (p.stream_k, p.cluster_k, p.grid, p.workspace_bytes) == (0, 3, 120, 0)
    p = tl.gemm_plan(32, 8192, 28672)                 # 32 tiles, clusters of 4
    assert p.cta == (32, 256, 64) and (p.stream_k, p.cluster_k, p.grid, p.workspace_bytes) == (0, 4, 128, 0)
    p = tl.gemm_plan(32, 57344, 8192)                 # 224 whole tiles on 112 CTAs
    assert p.cta == (32, 256, 64) and (p.stream_k, p.cluster_k, p.grid, p.workspace_bytes) == (0, 1, 112, 0)
    with tl.option(tl.OPT_NO_SCRATCH_PLANS, 0):       # the stream-K cut over every SM
        p = tl.gemm_plan(8, 10240, 8192)
        assert (p.stream_k, p.cluster_k, p.grid) == (1, 1, sms) and p.workspace_bytes == 2 * sms * 16 * 256 * 4
    p = tl.gemm_plan(4096, 57344, 8192)
    assert p.pair_kernel == 1 and p.cta == (512, 128, 64) and p.workspace_bytes == 0 and p.grid % 2 == 0
    assert 2 * p.pair_tiles_512 + p.pair_tiles_256 == 16 * 224
    # grouped, short tiles (at most 32 stages) and at least 64 m-tiles whatever the routing: whole tiles, nothing is cut
    for N, K in ((1536, 2048), (2048, 768)):
        p = tl.gemm_plan(2048, N, K, E=128)
        assert p.cta == (32, 256, 64) and (p.stream_k, p.cluster_k, p.grid, p.workspace_bytes) == (0, 1, sms, 0)
    # too few rows for the host to rule the cut out (the kernel decides from the tile count), and long tiles
    p = tl.gemm_plan(64, 1536, 2048, E=128)
    assert p.stream_k == 1 and p.workspace_bytes > 0
    p = tl.gemm_plan(2048, 2048, 8192, E=128)
    assert p.stream_k == 1 and p.workspace_bytes > 0


def test_workspace_bound_covers_many_small_experts():
    # 32 rows over 128 experts: every expert may add a ragged tile, so the grouped grid is far larger than the row
    # count suggests; the size the header promises for "any number of experts" must cover it.
    from gpu_util import tl
    M, N, K, E = 32, 128, 128, 128
    need = tl.gemm_plan(M, N, K, 4096, 16, 128, (0, 0, 0), E).workspace_bytes
    assert tl.gemm_workspace_bytes(M, N, K) >= need > 0


# ------------------------------------------------------------------------------------------------ giving up

def test_gemm_wait_that_runs_out_is_reported_and_the_next_call_is_clean():
    # The launch arms its first pipeline stage for 16 bytes more than its copies deliver (test hook): the wait of
    # the MMA warp on that stage runs out after the shortened limit, every role leaves its loop, the copies in flight
    # are waited for, tensor memory is freed and the kernel returns.  Nothing faults and nothing waits unbounded.
    from gpu_util import DEV, run_gemm, tile_major_on_device, tl
    M, N, K = 16, 512, 512
    A = inputs.bf16_integers((M, K), -8, 8, seed=1)
    B = inputs.bf16_integers((K, N), -8, 8, seed=2)
    Bt = tile_major_on_device(B, K, N, 16, 128)
    want, _ = tlo.matmul(inputs.bits(A), inputs.bits(Bt.reshape(-1)), TILE, 16, 128, M, N, K)
    tl.device_status()
    C = torch.zeros((M, N), dtype=torch.float32, device=DEV)
    with tl.option(tl.OPT_WAIT_LIMIT_US, 2000):
        tl.set_option(tl.OPT_STALL_ONCE, 1)
        tl.gemm(A.to(DEV), Bt, C, M, N, K, 4096, 16, 128)
        assert tl.get_option(tl.OPT_STALL_ONCE) == 0                     # consumed by that launch
        with pytest.raises(tl.TileLensError) as e:
            tl.device_status()
        # (the MMA warp's wait for the stage, or the epilogue's wait for the accumulator behind it: whichever looked
        # at the clock first)
        assert e.value.status == 5 and ("detail=0x200" in str(e.value) or "detail=0x400" in str(e.value))
    tl.device_status()                                                    # the flag was cleared by the report
    got = run_gemm(A, Bt, M, N, K, 16, 128)
    assert np.array_equal(got.cpu().numpy().astype(np.float64), want)
    # The other weight paths give up the same way: the permuting generic-address path (a second arrival on the same
    # barrier), tiles read as stored, and tiles fixed up in place (the copies land on a barrier of their own, on which
    # the four fix-up warps wait).
    for br, bc, raw, path in ((16, 8, 0, 1), (16, 8, 1, 2), (32, 4, 1, 3), (8, 2, 1, 3)):
        Bg = tile_major_on_device(B, K, N, br, bc)
        with tl.option(tl.OPT_WAIT_LIMIT_US, 2000), tl.option(tl.OPT_GENERIC_RAW, raw):
            tl.set_option(tl.OPT_STALL_ONCE, 1)
            tl.gemm(A.to(DEV), Bg, C, M, N, K, br * bc * 2, br, bc)
            assert tl.gemm_last_plan().generic_path == path
            with pytest.raises(tl.TileLensError) as e:
                tl.device_status()
            assert e.value.status == 5
            assert np.array_equal(run_gemm(A, Bg, M, N, K, br, bc).cpu().numpy().astype(np.float64), want)


def test_two_block_tiles_give_up_the_same_way():
    # The tile of two token blocks owns both accumulators and hands them back on one barrier: a stage that never fills
    # must end its MMA and epilogue roles like any other launch, and the next launch on the same tile must be exact.
    from gpu_util import DEV, run_gemm, tl
    M, N, K = 256, 256 * 112, 128
    A, Bd, want = _int_case(M, N, K, 16, 128, seed=77)
    C = torch.zeros((M, N), dtype=torch.float32, device=DEV)
    tl.device_status()
    with tl.option(tl.OPT_WAIT_LIMIT_US, 2000):
        tl.set_option(tl.OPT_STALL_ONCE, 1)
        tl.gemm(A.to(DEV), Bd, C, M, N, K, 4096, 16, 128, (256, 256, 64))
        assert tl.gemm_last_plan().cta == (256, 256, 64) and tl.get_option(tl.OPT_STALL_ONCE) == 0
        with pytest.raises(tl.TileLensError) as e:
            tl.device_status()
        assert e.value.status == 5
    tl.device_status()
    assert torch.equal(run_gemm(A, Bd, M, N, K, 16, 128, (256, 256, 64)).cpu(), want)


def test_relayout_wait_that_runs_out_is_reported_and_the_next_call_is_clean():
    from gpu_util import DEV, Guarded, dev_bytes, tl
    rows, cols, s, br, bc = 512, 512, 2, 16, 128
    src = inputs.random_bytes(rows * cols * s, seed=3)
    want = tlo.relayout(src, rows, cols, s, br, bc, tlo.TO_TILE_MAJOR)
    d_src = dev_bytes(src)
    tl.device_status()
    for direction, a, b in ((tl.TO_TILE_MAJOR, d_src, want), (tl.TO_ROW_MAJOR, dev_bytes(want), src)):
        scratch = torch.zeros(rows * cols * s, dtype=torch.uint8, device=DEV)
        with tl.option(tl.OPT_WAIT_LIMIT_US, 2000):
            tl.set_option(tl.OPT_STALL_ONCE, 2)
            tl.relayout(a, scratch, rows, cols, s, br * bc * s, br, bc, direction)
            assert tl.get_option(tl.OPT_STALL_ONCE) == 0
            with pytest.raises(tl.TileLensError) as e:
                tl.device_status()
            assert e.value.status == 5 and "detail=0x600" in str(e.value)
        g = Guarded((rows * cols * s,), torch.uint8)
        tl.relayout(a, g.t, rows, cols, s, br * bc * s, br, bc, direction)
        tl.device_status()
        assert np.array_equal(g.check().cpu().numpy(), b)


# ------------------------------------------------------------------------------------------------ PDL ordering

def test_chained_products_wait_for_the_whole_predecessor():
    # gate_up with K == cta_k has no tile cut along K: no reduction CTA has anything to add.  The down product that
    # follows in the stream must still see all of H (every reduction CTA waits for the GEMM grid before it leaves).
    from gpu_util import DEV, tl
    E, hidden, inter = 16, 128, 512
    offsets, counts, _ = inputs.zipf_topk_routing(96, E, 4, 1.1, seed=4)
    rows = int(offsets[-1])
    X = inputs.bf16_normal((rows, hidden), 1.0, seed=1, device=DEV)
    Wgu = inputs.bf16_normal((E, hidden, 2 * inter), 0.05, seed=2, device=DEV)
    Wd = inputs.bf16_normal((E, inter, hidden), 0.05, seed=3, device=DEV)
    Wgu_t, Wd_t = torch.empty_like(Wgu), torch.empty_like(Wd)
    tl.relayout(Wgu, Wgu_t, E * hidden, 2 * inter, 2, 4096, 16, 128, tl.TO_TILE_MAJOR)
    tl.relayout(Wd, Wd_t, E * inter, hidden, 2, 4096, 16, 128, tl.TO_TILE_MAJOR)
    d_off = torch.from_numpy(offsets).to(DEV)

    def chain():
        H = torch.zeros((rows, inter), dtype=torch.bfloat16, device=DEV)
        Y = torch.full((rows, hidden), float("nan"), dtype=torch.float32, device=DEV)
        for _ in range(20):                                   # back to back, so that launches overlap their ends
            H.zero_()
            tl.moe_ffn(X, Wgu_t, Wd_t, H, Y, d_off, E, rows, hidden, inter, 4096, 16, 128)
        tl.device_status()
        return H.clone(), Y.clone()

    H1, Y1 = chain()
    with tl.option(tl.OPT_PDL, 0):
        H0, Y0 = chain()
    assert torch.equal(H1, H0) and torch.equal(Y1, Y0)
    check = np.arange(rows)
    Hr, Yr, Sr = tlo.moe_ffn_rows(inputs.bits(X), inputs.bits(Wgu_t.reshape(-1)), inputs.bits(Wd_t.reshape(-1)), offsets,
                                  hidden, inter, tlo.TILE_MAJOR, 16, 128, check)
    assert np.all(np.abs(Y1.cpu().numpy().astype(np.float64) - Yr) <= 2e-2 * Sr + 1e-6)      # h itself is bf16-rounded


# ------------------------------------------------------------------------------------------------ host threads

def test_two_host_threads_with_their_own_streams_and_workspaces():
    from gpu_util import DEV, tile_major_on_device, tl
    shapes = [(8, 1280, 4096), (32, 2048, 2304)]
    A, Bt, want = [], [], []
    for i, (M, N, K) in enumerate(shapes):
        A.append(inputs.bf16_normal((M, K), 1.0, seed=60 + i).to(DEV))
        Bt.append(tile_major_on_device(inputs.bf16_normal((K, N), 0.02, seed=70 + i), K, N, 16, 128))
        C = torch.empty((M, N), dtype=torch.float32, device=DEV)
        tl.gemm(A[i], Bt[i], C, M, N, K, 4096, 16, 128)
        want.append(C)
    tl.device_status()
    errors, results = [], [None, None]

    def worker(i):
        try:
            torch.cuda.set_device(0)
            M, N, K = shapes[i]
            stream = torch.cuda.Stream(device=DEV)
            ws = torch.empty(tl.gemm_workspace_bytes(M, N, K) + 256, dtype=torch.uint8, device=DEV)
            tl.set_workspace(ws)                               # this thread's workspace and stream only
            tl.set_stream(stream)
            outs = []
            for rep in range(40):
                C = torch.full((M, N), float("nan"), dtype=torch.float32, device=DEV)
                tl.gemm(A[i], Bt[i], C, M, N, K, 4096, 16, 128, stream=stream)
                outs.append(C)
            stream.synchronize()
            results[i] = outs
            tl.set_workspace(None)
        except Exception as exc:                               # noqa: BLE001 -- reported by the main thread
            errors.append(exc)

    threads = [threading.Thread(target=worker, args=(i,)) for i in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    torch.cuda.synchronize()
    for i in range(2):
        for C in results[i]:
            assert torch.equal(C, want[i])
    tl.device_status()
