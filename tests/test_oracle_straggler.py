"""Pins of the oracle's tile-arrival model (Section 6.5, "Straggler-Induced CTA Stalls"): CPU only.

The oracle takes a sample of per-request latencies from the caller (the paper shows its distribution only in
figures, so none is built in) and returns the expected time to the first and to the last arrival of the n requests of
a compute tile.  Pinned by the definition enumerated on tiny inputs, by closed forms of order statistics for
distributions whose quantiles are handed in as the sample, and by the properties the section states.
"""
import itertools
import math

import numpy as np
import pytest

import oracle as tlo


def test_enumeration_of_every_draw_on_tiny_samples():
    # the definition: n independent draws, each sample value with probability 1/N
    rng = np.random.default_rng(1)
    for N, n in ((4, 3), (5, 2), (3, 5), (6, 1), (2, 7)):
        x = rng.uniform(1.0, 9.0, N)
        draws = list(itertools.product(x, repeat=n))
        want_last = sum(max(d) for d in draws) / len(draws)
        want_first = sum(min(d) for d in draws) / len(draws)
        t = float(np.median(x))
        want_late = sum(1 for d in draws if max(d) > t) / len(draws)
        first, last, late = tlo.tile_arrival(x, n, t)
        assert first == pytest.approx(want_first, rel=1e-12)
        assert last == pytest.approx(want_last, rel=1e-12)
        assert late == pytest.approx(want_late, abs=1e-12)


def test_one_request_sees_the_mean_and_equal_latencies_have_no_straggler():
    x = np.array([5.0, 7.0, 6.0, 15.0])
    first, last, _ = tlo.tile_arrival(x, 1)
    assert first == pytest.approx(x.mean()) and last == pytest.approx(x.mean())
    first, last, late = tlo.tile_arrival(np.full(100, 5.0), 128, 5.0)
    assert first == 5.0 and last == 5.0 and late == 0.0


def test_closed_forms_of_order_statistics():
    # exponential latencies (rate 1): E[max of n] = H_n, E[min of n] = 1/n; uniform on (0, 1): n/(n+1), 1/(n+1).
    # The sample is the distribution's quantile grid, fine enough that the discretisation is below the tolerance.
    N = 400_000
    u = (np.arange(N) + 0.5) / N
    expo = -np.log1p(-u)
    for n in (1, 2, 16, 128):
        first, last, late = tlo.tile_arrival(expo, n, 3.0)
        assert last == pytest.approx(sum(1.0 / k for k in range(1, n + 1)), rel=2e-3)
        assert first == pytest.approx(1.0 / n, rel=2e-3)
        assert late == pytest.approx(1.0 - (1.0 - math.exp(-3.0)) ** n, abs=1e-4)
        first, last, _ = tlo.tile_arrival(u, n)
        assert last == pytest.approx(n / (n + 1.0), rel=1e-4) and first == pytest.approx(1.0 / (n + 1.0), rel=1e-3)


def test_more_outstanding_requests_wait_longer_for_the_last_one():
    # the section's point: 128 requests per tile (row-major) against 16 (tile-major) on the same long-tailed
    # distribution -- the last arrival moves into the tail, the first one hardly moves
    rng = np.random.default_rng(7)
    lat = 5.0 + rng.lognormal(mean=-1.0, sigma=1.0, size=20000)          # a long tail above a 5 us floor (any sample would do)
    prev_last, prev_first = 0.0, 1e9
    for n in (1, 2, 8, 16, 64, 128, 1024):
        first, last, late = tlo.tile_arrival(lat, n, float(np.quantile(lat, 0.99)))
        assert last >= prev_last and first <= prev_first and lat.min() <= first <= last <= lat.max()
        assert late == pytest.approx(1.0 - 0.99 ** n, abs=2e-3)
        prev_last, prev_first = last, first
    f16, l16, _ = tlo.tile_arrival(lat, 16)
    f128, l128, _ = tlo.tile_arrival(lat, 128)
    assert (l128 - f128) > (l16 - f16) and l128 > l16


def test_rejects_bad_arguments():
    with pytest.raises(ValueError):
        tlo.tile_arrival(np.array([]), 4)
    with pytest.raises(ValueError):
        tlo.tile_arrival(np.array([1.0, 2.0]), 0)
