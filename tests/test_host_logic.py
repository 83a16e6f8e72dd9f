"""Host-side arithmetic of the library that needs no GPU (CPU only)."""
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
