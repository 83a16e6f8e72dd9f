"""Host-side arithmetic of the library that needs no GPU (CPU only)."""
import pytest

import oracle as tlo
from paper_2607_04031_b200 import binding as tl


def test_prefetch_degree_matches_the_oracle_over_a_sweep():
    for B in (1.0e12, 4.9e12, 8.0e12):
        for L in (1e-6, 5e-6, 20e-6):
            for n_sm, c_sm in ((132, 1), (148, 1), (148, 2), (7, 1)):
                for p_tile in (1, 16, 128):
                    for K, tk in ((2048, 128), (8192, 64), (1 << 20, 64)):
                        for c in (1.0, 2.0):
                            assert tl.prefetch_degree(B, L, 4096, n_sm, c_sm, p_tile, K, tk, c) == \
                                tlo.prefetch_degree(B, L, 4096, n_sm, c_sm, p_tile, K, tk, c)


def test_prefetch_degree_rejects_bad_arguments():
    import pytest
    with pytest.raises(ValueError):
        tl.prefetch_degree(1e12, 1e-6, 4096, 0, 1, 16, 2048, 128)
    with pytest.raises(ValueError):
        tl.prefetch_degree(1e12, 1e-6, 4096, 132, 1, 16, 2048, 0)


def test_tile_arrival_latency_matches_the_oracle():
    # host arithmetic of the library (summation by parts, double) against the oracle (probability masses, long double)
    import numpy as np
    import pytest
    rng = np.random.default_rng(3)
    for N in (1, 2, 17, 1000, 50_000):
        for kind in ("lognormal", "uniform", "ties"):
            x = {"lognormal": 5.0 + rng.lognormal(-1.0, 1.2, N), "uniform": rng.uniform(0.0, 10.0, N),
                 "ties": rng.integers(0, 4, N).astype(np.float64)}[kind]
            for n in (1, 2, 16, 128, 4096):
                t = float(np.quantile(x, 0.9))
                got = tl.tile_arrival_latency(x, n, t)
                want = tlo.tile_arrival(x, n, t)
                for g, w in zip(got, want):
                    assert g == pytest.approx(w, rel=1e-10, abs=1e-12), (N, kind, n)


def test_tile_arrival_latency_of_the_printed_request_counts():
    # Section 6.5: 128 requests per 128 x 256 tile in row-major against 16 in tile-major.  On any long-tailed sample
    # the last arrival of 128 requests sits further in the tail than that of 16.
    import numpy as np
    rng = np.random.default_rng(11)
    lat = 5.0 + rng.lognormal(-1.0, 1.0, 10_000)
    f16, l16, _ = tl.tile_arrival_latency(lat, 16)
    f128, l128, _ = tl.tile_arrival_latency(lat, 128)
    assert l128 > l16 > f16 >= f128 >= lat.min()


def test_tile_arrival_latency_rejects_bad_arguments():
    import ctypes
    import numpy as np
    L = tl.lib()
    x = np.array([1.0, 2.0])
    a, b = ctypes.c_double(), ctypes.c_double()
    assert L.tl_tile_arrival_latency(x.ctypes.data, 2, 0, 0.0, ctypes.byref(a), ctypes.byref(b), None) == 1
    assert L.tl_tile_arrival_latency(x.ctypes.data, 0, 4, 0.0, ctypes.byref(a), ctypes.byref(b), None) == 1
    assert L.tl_tile_arrival_latency(None, 2, 4, 0.0, ctypes.byref(a), ctypes.byref(b), None) == 1
    bad = np.array([1.0, float("nan")])
    assert L.tl_tile_arrival_latency(bad.ctypes.data, 2, 4, 0.0, ctypes.byref(a), ctypes.byref(b), None) == 1


# ---- the planning rules, asked as if the device were a 148-SM B200 (test hook: no CUDA call is made)

def _plans_as_if(sms):
    return tl.option(tl.OPT_PLAN_AS_IF_SMS, sms)


def test_plans_of_the_benchmark_shapes_without_a_gpu():
    with _plans_as_if(148):
        # decode: schedules without partial tiles in global memory
        p = tl.gemm_plan(8, 10240, 8192)                  # 40 tiles, clusters of 3 CTAs split K (45 such clusters fit)
        assert p.cta == (16, 256, 64) and (p.stream_k, p.cluster_k, p.grid, p.workspace_bytes) == (0, 3, 120, 0)
        p = tl.gemm_plan(32, 8192, 28672)                 # 32 tiles, clusters of 4 (33 fit)
        assert p.cta == (32, 256, 64) and (p.stream_k, p.cluster_k, p.grid, p.workspace_bytes) == (0, 4, 128, 0)
        p = tl.gemm_plan(1, 57344, 8192)                  # 224 whole tiles on 112 CTAs
        assert p.cta == (16, 256, 64) and (p.stream_k, p.cluster_k, p.grid, p.workspace_bytes) == (0, 1, 112, 0)
        # prefill: CTA pairs, 512-token tiles in whole waves of 74 clusters, the rest as 256-token tiles
        p = tl.gemm_plan(4096, 8192, 8192)
        assert p.pair_kernel == 1 and p.cta == (512, 128, 64) and p.grid == 148
        assert (p.pair_tiles_512, p.pair_tiles_256) == (222, 68) and p.workspace_bytes == 0
        # Qwen expert products: short tiles, at least 64 m-tiles whatever the routing: whole tiles, nothing is cut
        for N, K in ((1536, 2048), (2048, 768)):
            p = tl.gemm_plan(2048, N, K, E=128)
            assert p.cta == (32, 256, 64) and (p.stream_k, p.cluster_k, p.grid, p.workspace_bytes) == (0, 1, 148, 0)
    assert tl.get_option(tl.OPT_PLAN_AS_IF_SMS) == 0


def test_cluster_plans_respect_how_many_clusters_can_be_resident():
    with _plans_as_if(148):
        # 16 tiles: 16 clusters of 8 CTAs would fill 128 SMs, but only 15 can be resident at once: 6 CTAs per cluster
        assert tl.gemm_plan(16, 4096, 1024).cluster_k == 6
        # 37 tiles: 33 clusters of 4 fit, 45 of 3
        p = tl.gemm_plan(40, 9472, 2048)
        assert (p.cluster_k, p.grid) == (3, 111)
        # 18 tiles x 8 = 144 CTAs does not fit either
        p = tl.gemm_plan(8, 4608, 4096)
        assert (p.stream_k, p.cluster_k, p.grid) == (0, 6, 108)
    with _plans_as_if(64):                                # a smaller part: 64 / S clusters of S CTAs
        p = tl.gemm_plan(8, 2048, 8192)                   # 8 tiles x 8 CTAs = 64
        assert (p.stream_k, p.cluster_k, p.grid) == (0, 8, 64)


def test_when_the_k_loops_are_cut_over_all_sms():
    with _plans_as_if(148):
        # few tiles of very long K and many bytes: neither whole tiles nor under-filled clusters are worth it
        p = tl.gemm_plan(16, 2304, 28672)
        assert (p.stream_k, p.cluster_k, p.grid) == (1, 1, 148) and p.workspace_bytes == 2 * 148 * 16 * 256 * 4
        # the same tiles with fewer bytes: clusters, although they fill only 72 SMs
        p = tl.gemm_plan(16, 2304, 8192)
        assert (p.stream_k, p.cluster_k, p.grid) == (0, 8, 72)
        # a few MB of weights: clusters, however few
        p = tl.gemm_plan(256, 512, 2048)
        assert (p.stream_k, p.cluster_k, p.grid, p.cta) == (0, 4, 32, (128, 128, 128))
        # grouped: too few rows for the host to rule the cut out (the kernel decides from the tile count); long tiles
        assert tl.gemm_plan(64, 1536, 2048, E=128).stream_k == 1
        assert tl.gemm_plan(2048, 2048, 8192, E=128).stream_k == 1
        # with the no-scratch schedules switched off: always the cut
        with tl.option(tl.OPT_NO_SCRATCH_PLANS, 0):
            p = tl.gemm_plan(8, 10240, 8192)
            assert (p.stream_k, p.cluster_k, p.grid) == (1, 1, 148)


def test_tile_of_dense_products_between_decode_and_prefill():
    with _plans_as_if(148):
        plan = lambda M, N, K: tl.gemm_plan(M, N, K)
        # enough tiles either way: 256 weight columns per tile halve the share of token rows in what an SM loads
        p = plan(128, 57344, 8192)
        assert (p.cta, p.stream_k, p.cluster_k, p.grid) == ((128, 256, 64), 0, 1, 112)
        p = plan(128, 10240, 8192)                        # 40 wide tiles in clusters of 3; the narrow tile would be cut
        assert (p.cta, p.stream_k, p.cluster_k, p.grid) == ((128, 256, 64), 0, 3, 120)
        # 129 to 256 rows with enough tiles for whole-tile schedules: both 128-row blocks on one weight slab per stage
        p = plan(256, 57344, 8192)
        assert (p.cta, p.pair_kernel, p.stream_k, p.cluster_k, p.grid, p.stages) == ((256, 256, 64), 0, 0, 1, 112, 3)
        p = plan(256, 57344, 4096)                        # a shorter K loop: CTA pairs on 256-token tiles
        assert (p.pair_kernel, p.pair_tiles_512, p.pair_tiles_256) == (1, 0, 224)
        p = plan(256, 8192, 28672)                        # 32 such tiles would have to be cut: the wide tile in clusters
        assert (p.cta, p.stream_k, p.cluster_k) == ((128, 256, 64), 0, 2)
        # where the default would be the CTA-pair kernel: the wide tile up to 384 rows
        p = plan(384, 57344, 8192)
        assert (p.cta, p.pair_kernel, p.stream_k) == ((128, 256, 64), 0, 0)
        # the two-block tile is refused outright where its schedule would leave partial tiles
        with pytest.raises(tl.TileLensError):
            tl.gemm_plan(256, 8192, 28672, 4096, 16, 128, (256, 256, 64))
        p = plan(512, 57344, 8192)
        assert p.pair_kernel == 1
        # small weights: more, smaller tiles win (latency, not bandwidth)
        assert plan(128, 512, 2048).cta == (128, 128, 128) and plan(256, 4096, 2048).cta == (128, 128, 128)
        # the wide tile only where it needs no partial tiles in global memory
        p = plan(384, 8192, 28672)
        assert (p.cta, p.stream_k) == ((128, 128, 128), 1)
        # a cut of the narrow tile against clusters of the wide one
        p = plan(384, 4096, 4096)
        assert (p.cta, p.stream_k, p.cluster_k) == ((128, 256, 64), 0, 2)
        # decode and prefill sizes are not touched
        assert plan(64, 57344, 8192).cta == (64, 256, 64) and plan(4096, 8192, 8192).pair_kernel == 1


def test_schedules_of_a_few_waves_above_512_rows():
    with _plans_as_if(148):
        plan = lambda M, N, K: tl.gemm_plan(M, N, K)
        # prefill proper: whole waves of 512-token pair tiles, 256-token tiles for the rest
        p = plan(4096, 10240, 8192)
        assert (p.pair_kernel, p.pair_tiles_512, p.pair_tiles_256) == (1, 296, 48)
        p = plan(1024, 57344, 8192)
        assert (p.pair_kernel, p.pair_tiles_512, p.pair_tiles_256) == (1, 444, 8)
        # M leaves every other 512-token tile half empty and there are ten waves: 256-token tiles alone
        p = plan(768, 57344, 8192)
        assert (p.pair_kernel, p.cta, p.pair_tiles_512, p.pair_tiles_256) == (1, (256, 128, 64), 0, 672)
        # 128 tiles: two waves of pairs, or one wave of two-block tiles on 128 CTAs
        p = plan(1024, 8192, 28672)
        assert (p.pair_kernel, p.cta, p.stream_k, p.cluster_k, p.grid) == (0, (256, 256, 64), 0, 1, 128)
        p = plan(640, 10240, 8192)                        # 120 tiles on 120 CTAs
        assert (p.pair_kernel, p.cta, p.grid) == (0, (256, 256, 64), 120)
        # the pair kernel switched off: none of this applies
        with tl.option(tl.OPT_PAIR_KERNEL, 0):
            assert plan(1024, 8192, 28672).cta == (256, 128, 64)


def test_grouped_tile_grows_with_the_rows_per_expert():
    with _plans_as_if(148):
        grouped = lambda rows, E, N, K: tl.gemm_plan(rows, N, K, 4096, 16, 128, (0, 0, 0), E)
        # the Qwen-3 routing of the benchmark: 16 rows per expert on average
        p = grouped(2048, 128, 1536, 2048)
        assert (p.cta, p.stream_k, p.grid, p.workspace_bytes) == ((32, 256, 64), 0, 148, 0)
        assert grouped(3072, 128, 1536, 2048).cta == (32, 256, 64)           # 24 rows
        assert grouped(4096, 128, 1536, 2048).cta == (64, 256, 64)           # 32 rows
        assert grouped(8192, 128, 1536, 2048).cta == (128, 256, 64)          # 64 rows
        assert grouped(32768, 128, 2048, 768).cta == (128, 256, 64)
        # many rows per expert but few tiles: the small tile, which needs no cut
        p = grouped(2048, 16, 1024, 512)
        assert (p.cta, p.stream_k) == ((32, 256, 64), 0)
        # a fixed row cap switches the rule off
        with tl.option(tl.OPT_MOE_ROW_CAP, 32):
            assert grouped(32768, 128, 1536, 2048).cta == (32, 256, 64)
        # what tl_gemm_workspace_bytes reports covers the larger tiles too
        for rows, E, N, K in ((8192, 128, 1536, 2048), (700, 4, 512, 8192), (40000, 100, 2048, 768)):
            assert tl.gemm_workspace_bytes(rows, N, K) >= grouped(rows, E, N, K).workspace_bytes


def test_the_reported_workspace_covers_every_plan():
    # tl_gemm_workspace_bytes is what a caller sizes its own workspace from: never less than the plan of that call
    with _plans_as_if(148):
        seen = 0
        for M in (1, 8, 16, 32, 48, 64, 100, 128, 256, 700, 4096):
            for N in (256, 1280, 2304, 8192, 10240, 57344):
                for K in (64, 512, 2048, 8192, 28672):
                    plan = tl.gemm_plan(M, N, K)
                    assert tl.gemm_workspace_bytes(M, N, K) >= plan.workspace_bytes, (M, N, K)
                    assert (plan.workspace_bytes > 0) == (plan.stream_k == 1), (M, N, K)
                    seen += plan.stream_k
        assert seen > 0                                   # the cut is among the schedules looked at


def test_weight_paths_by_memory_tile_shape():
    with _plans_as_if(148):
        path = lambda br, bc, cta=(0, 0, 0): tl.gemm_plan(16, 8192, 8192, br * bc * 2, br, bc, cta).generic_path
        assert path(16, 128) == 0 and path(32, 16) == 0 and path(16, 32) == 0           # TMA boxes
        assert path(16, 8) == 2 and path(8, 8) == 2 and path(64, 8) == 2                 # 16-byte rows: as stored
        assert path(16, 1) == 2 and path(8, 1) == 2 and path(128, 1) == 2                # single-column tiles: K-major panels
        assert path(32, 4) == 3 and path(8, 2) == 3 and path(8, 4) == 3                  # 8- and 4-byte rows: in place
        assert path(64, 4) == 3 and path(64, 2) == 3 and path(128, 2, (32, 128, 128)) == 3
        with pytest.raises(tl.TileLensError):                                             # a 128-row tile does not fit 64-row stages
            path(128, 2)
        assert path(4, 8) == 1 and path(4, 4) == 1                                        # fewer than 8 rows: permuted
        with tl.option(tl.OPT_GENERIC_RAW, 0):
            assert path(16, 8) == 1 and path(32, 4) == 1 and path(16, 1) == 1


def test_launches_are_refused_while_the_planning_hook_is_on():
    with _plans_as_if(148):
        assert tl.lib().tl_gemm(1 << 12, 1 << 13, 1 << 14, 16, 512, 512, 4096, 16, 128, 0, 0, 0, None) == 1
