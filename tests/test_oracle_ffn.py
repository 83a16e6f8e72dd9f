"""Pins for the oracle's expert-FFN chain (CPU only): bf16 rounding, silu, and the chain against numpy/torch."""
import math

import numpy as np
import torch

import oracle as tlo
from paper_2607_04031_b200 import inputs


def test_bf16_rounding_matches_torch_and_ties_go_to_even():
    rng = np.random.default_rng(3)
    xs = np.concatenate([rng.normal(0, 1, 4000), rng.normal(0, 1e-3, 1000), rng.normal(0, 1e4, 1000),
                         [0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.0e38, -3.0e38, 1e-40, float("inf")]])
    want = torch.tensor(xs, dtype=torch.float64).to(torch.float32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = np.array([tlo.double_to_bf16(float(x)) for x in xs], dtype=np.uint16)
    assert np.array_equal(got, want)
    # ties, by hand: 1 + 2^-8 lies exactly between 1.0 (0x3F80, even) and 1 + 2^-7 (0x3F81): goes to 0x3F80;
    # 1 + 3*2^-8 lies between 0x3F81 and 0x3F82 (even): goes to 0x3F82
    assert tlo.double_to_bf16(1.0 + 2.0 ** -8) == 0x3F80
    assert tlo.double_to_bf16(1.0 + 3 * 2.0 ** -8) == 0x3F82
    assert tlo.double_to_bf16(1.0 + 2.0 ** -8 + 2.0 ** -20) == 0x3F81            # just above the tie
    assert tlo.bf16_to_double(tlo.double_to_bf16(-2.5)) == -2.5


def test_silu_identities():
    assert tlo.silu(0.0) == 0.0
    for x in (0.1, 1.0, 2.5, 7.0, 30.0):
        assert abs((tlo.silu(x) - tlo.silu(-x)) - x) <= 1e-15 * x           # x*s(x) - (-x)*s(-x) = x*(s(x) + s(-x)) = x
        assert abs(tlo.silu(x) - x * (0.5 + 0.5 * math.tanh(x / 2))) <= 1e-15 * x
    assert tlo.silu(40.0) == 40.0 / (1.0 + math.exp(-40.0)) and abs(tlo.silu(-40.0)) < 1e-15
    assert abs(tlo.silu(1.0) - 0.7310585786300049) < 1e-16                  # 1 / (1 + 1/e)


def test_chain_matches_numpy_on_a_small_problem_in_both_layouts():
    E, hidden, inter = 3, 64, 32
    offsets = np.array([0, 5, 5, 9], dtype=np.int32)                        # the middle expert has no rows
    rows = int(offsets[-1])
    X = inputs.bf16_normal((rows, hidden), 1.0, seed=1)
    Wgu = inputs.bf16_normal((E, hidden, 2 * inter), 0.2, seed=2)           # columns 2j = gate_j, 2j+1 = up_j
    Wd = inputs.bf16_normal((E, inter, hidden), 0.2, seed=3)
    x64, g64, d64 = X.double().numpy(), Wgu.double().numpy(), Wd.double().numpy()
    want_H = np.empty((rows, inter)); want_Y = np.empty((rows, hidden))
    for r in range(rows):
        e = 0 if r < 5 else 2
        gu = x64[r] @ g64[e]
        g, u = gu[0::2], gu[1::2]
        h = torch.tensor(g / (1 + np.exp(-g)) * u).to(torch.float32).to(torch.bfloat16).double().numpy()
        want_H[r] = h
        want_Y[r] = h @ d64[e]
    H, Y, S = tlo.moe_ffn_rows(inputs.bits(X), inputs.bits(Wgu), inputs.bits(Wd), offsets, hidden, inter, tlo.ROW_MAJOR, 0, 0,
                               np.arange(rows))
    Hd = torch.from_numpy(H.view(np.int16)).view(torch.bfloat16).double().numpy()
    # the two sides sum in different orders: h may differ by one bf16 step where the fp64 value sits on a boundary
    assert np.all(np.abs(Hd - want_H) <= 2.0 ** -7 * np.abs(want_H) + 1e-30)
    assert np.mean(Hd == want_H) > 0.99
    w_of_row = np.stack([d64[0 if r < 5 else 2] for r in range(rows)])            # [rows, inter, hidden]
    assert np.all(np.abs(Y - np.einsum("rj,rjc->rc", Hd, w_of_row)) <= 1e-12 * S + 1e-300)   # y from the oracle's own h
    assert np.all(np.abs(S - np.einsum("rj,rjc->rc", np.abs(Hd), np.abs(w_of_row))) <= 1e-12 * S + 1e-300)
    # tile-major weights (16 x 16 tiles here) give the same numbers as row-major ones
    gt = np.stack([tlo.relayout(inputs.bits(Wgu[e]).view(np.uint8), hidden, 2 * inter, 2, 16, 16, tlo.TO_TILE_MAJOR).view(np.uint16) for e in range(E)])
    dt = np.stack([tlo.relayout(inputs.bits(Wd[e]).view(np.uint8), inter, hidden, 2, 16, 16, tlo.TO_TILE_MAJOR).view(np.uint16) for e in range(E)])
    H2, Y2, S2 = tlo.moe_ffn_rows(inputs.bits(X), gt, dt, offsets, hidden, inter, tlo.TILE_MAJOR, 16, 16, np.arange(rows))
    assert np.array_equal(H2, H) and np.array_equal(Y2, Y) and np.array_equal(S2, S)
