"""Randomised exactness sweep over shapes, memory tiles, flavours and CTA tiles (GPU).

Integer-valued inputs make every product and partial sum exact in fp32, so the result must equal the oracle's
fp64 product bit for bit whatever the tile schedule, the split of K between CTAs or the order of the reduction.
"""
import numpy as np
import pytest
import torch

import oracle as tlo
from paper_2607_04031_b200 import inputs

pytestmark = pytest.mark.gpu

CTAS = [(0, 0, 0), (16, 256, 64), (32, 128, 128), (64, 64, 64), (64, 128, 64), (128, 128, 128), (128, 256, 64), (256, 128, 64),
        (16, 64, 128), (256, 64, 64)]


def _pick(rng, xs):
    return xs[int(rng.integers(0, len(xs)))]


# memory tiles with rows of 16 bytes and less: read as stored, transposed in place, K-major panels, or permuted
NARROW = [(8, 8), (16, 8), (32, 8), (64, 8), (128, 8), (8, 4), (16, 4), (32, 4), (64, 4), (8, 2), (16, 2), (32, 2), (64, 2),
          (128, 2), (8, 1), (16, 1), (32, 1), (64, 1), (128, 1), (4, 8), (4, 4), (2, 8), (4, 16)]


def _case(rng, narrow=False):
    flavour = "n" if narrow else _pick(rng, ["n", "n", "k", "fp8"])
    s = 1 if flavour == "fp8" else 2
    if narrow:
        br, bc = _pick(rng, NARROW)
        k_unit, n_unit = max(br, 64), 64
    elif flavour == "n":
        br, bc = _pick(rng, [(0, 0), (1, 256), (2, 128), (4, 64), (8, 64), (16, 128), (32, 64), (64, 32), (128, 16), (16, 16),
                             (8, 8), (32, 4), (2, 1024), (64, 64), (8, 512)])
        k_unit, n_unit = max(br, 64), max(bc, 64)
    else:
        min_cols = 32 // s                               # a tile row of the [N][K] array is at least 32 bytes
        br, bc = _pick(rng, [(0, 0), (64, 64), (32, 128), (16, 256), (8, 128), (128, 32), (256, 16), (4, 256), (1, 512)])
        if br and bc < min_cols:
            bc = min_cols
        n_unit, k_unit = max(br, 64), max(bc, 128 if s == 1 else 64)
    M = int(_pick(rng, [1, 3, 8, 17, 32, 40, 100, 129, 256, 300, 515]))
    N = n_unit * int(rng.integers(1, 1 + max(1, 1536 // n_unit)))
    K = k_unit * int(rng.integers(1, 1 + max(1, 2048 // k_unit)))
    cta = _pick(rng, CTAS)
    if flavour == "fp8" and cta[2]:
        cta = (cta[0], cta[1], cta[2] * 2)              # cta_k counts elements
    return flavour, s, br, bc, M, N, K, cta


@pytest.mark.parametrize("seed", range(160))
def test_random_configuration_is_exact(seed):
    rng = np.random.default_rng(1000 + seed)
    _run(seed, rng, _case(rng))


@pytest.mark.parametrize("seed", range(120))
def test_random_narrow_tile_configuration_is_exact(seed):
    rng = np.random.default_rng(5000 + seed)
    _run(seed, rng, _case(rng, narrow=True))


def _run(seed, rng, case):
    from gpu_util import DEV, tl
    flavour, s, br, bc, M, N, K, cta = case
    G = br * bc * s
    if flavour == "fp8":
        A = inputs.fp8_integers((M, K), -6, 6, seed=seed)
        B = inputs.fp8_integers((K, N), -6, 6, seed=seed + 1)
        a_bits, b_kn = inputs.bits8(A), inputs.bits8(B)
    else:
        A = inputs.bf16_integers((M, K), -6, 6, seed=seed)
        B = inputs.bf16_integers((K, N), -6, 6, seed=seed + 1)
        a_bits, b_kn = inputs.bits(A), inputs.bits(B)
    Ad = torch.from_numpy(a_bits.copy()).to(DEV)
    C = torch.full((M, N), float("nan"), dtype=torch.float32, device=DEV)
    if flavour == "n":
        W = torch.from_numpy(b_kn.copy()).to(DEV)                       # [K][N]
        if br:
            Wt = torch.empty_like(W)
            tl.relayout(W, Wt, K, N, 2, G, br, bc, tl.TO_TILE_MAJOR)
            W = Wt
        layout = tlo.TILE_MAJOR if br else tlo.ROW_MAJOR
        call = lambda: tl.gemm(Ad, W, C, M, N, K, G, br, bc, cta)
    else:
        W = torch.from_numpy(np.ascontiguousarray(b_kn.T)).to(DEV)      # [N][K]
        if br:
            Wt = torch.empty_like(W)
            tl.relayout(W, Wt, N, K, s, G, br, bc, tl.TO_TILE_MAJOR)
            W = Wt
        layout = tlo.TILE_MAJOR_K if br else tlo.COL_MAJOR
        fn = tl.gemm_fp8_kmajor if flavour == "fp8" else tl.gemm_kmajor
        call = lambda: fn(Ad, W, C, M, N, K, G, br, bc, cta)
    try:
        call()
    except tl.TileLensError as e:
        # the only refusals allowed here: a hand-addressed tile that does not fit the CTA tile, or a tile shape
        # this flavour does not instantiate
        assert e.status == 2, (flavour, br, bc, M, N, K, cta, str(e))
        hand = flavour == "n" and br > 1 and bc < 16
        assert hand or (cta[1] == 256 and cta[0] > 128), (flavour, br, bc, M, N, K, cta)
        return
    tl.device_status()
    ii, jj = rng.integers(0, M, 400), rng.integers(0, N, 400)
    ii[:4], jj[:4] = [0, 0, M - 1, M - 1], [0, N - 1, 0, N - 1]
    w_bits = W.cpu().numpy().reshape(-1)
    if flavour == "fp8":
        ref, _ = tlo.matmul_at_fp8(a_bits, w_bits, layout, br, bc, M, N, K, ii, jj)
    else:
        ref, _ = tlo.matmul_at(a_bits, w_bits.view(np.uint16), layout, br, bc, M, N, K, ii, jj)
    got = C.cpu().numpy()
    assert np.all(np.isfinite(got)), (flavour, br, bc, M, N, K, cta)
    assert np.array_equal(got[ii, jj].astype(np.float64), ref), (flavour, br, bc, M, N, K, cta)
    # every element against the exact integer product
    want = (A.to(torch.float64) @ B.to(torch.float64)).numpy()
    assert np.array_equal(got.astype(np.float64), want), (flavour, br, bc, M, N, K, cta)
