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
