"""Gated expert FFN (gate_up -> silu*mul -> down) through the C ABI vs the oracle (GPU)."""
import numpy as np
import pytest
import torch

import oracle as tlo
from paper_2607_04031_b200 import inputs

pytestmark = pytest.mark.gpu


def _bf16_steps(a_bits: np.ndarray, b_bits: np.ndarray) -> np.ndarray:
    """Distance in bf16 steps between two arrays of bit patterns (sign-magnitude -> ordered integers)."""
    def key(x):
        x = x.astype(np.int32)
        return np.where(x & 0x8000, -(x & 0x7FFF), x & 0x7FFF)
    return np.abs(key(a_bits) - key(b_bits))


def _run_case(E, hidden, inter, tokens, topk, br, bc, n_check, seed, want_chained=0):
    from gpu_util import DEV, tl
    offsets, counts, _ = inputs.zipf_topk_routing(tokens, E, topk, 1.1, seed=seed)
    rows = int(offsets[-1])
    X = inputs.bf16_normal((rows, hidden), 1.0, seed=seed + 1, device=DEV)
    Wgu = inputs.bf16_normal((E, hidden, 2 * inter), 0.02, seed=seed + 2, device=DEV)      # columns 2j gate, 2j+1 up
    Wd = inputs.bf16_normal((E, inter, hidden), 0.02, seed=seed + 3, device=DEV)
    G = br * bc * 2 if br else 0
    if br:
        Wgu_t, Wd_t = torch.empty_like(Wgu), torch.empty_like(Wd)
        tl.relayout(Wgu, Wgu_t, E * hidden, 2 * inter, 2, G, br, bc, tl.TO_TILE_MAJOR)
        tl.relayout(Wd, Wd_t, E * inter, hidden, 2, G, br, bc, tl.TO_TILE_MAJOR)
    else:
        Wgu_t, Wd_t = Wgu, Wd
    from gpu_util import guarded_out
    gH, gY = guarded_out((rows, inter), torch.bfloat16), guarded_out((rows, hidden), torch.float32)
    tl.moe_ffn(X, Wgu_t, Wd_t, gH.t, gY.t, torch.from_numpy(offsets).to(DEV), E, rows, hidden, inter, G, br, bc)
    assert tl.gemm_last_plan().chained == want_chained
    tl.device_status()
    H, Y = gH.check(), gY.check()
    assert torch.isfinite(H.float()).all() and torch.isfinite(Y).all()
    rng = np.random.default_rng(seed)
    check = np.unique(np.concatenate([[0, rows - 1], offsets[:-1][counts > 0], rng.integers(0, rows, n_check)]))
    layout = tlo.TILE_MAJOR if br else tlo.ROW_MAJOR
    Hr, Yr, Sr = tlo.moe_ffn_rows(inputs.bits(X), inputs.bits(Wgu_t.reshape(-1)), inputs.bits(Wd_t.reshape(-1)), offsets,
                                  hidden, inter, layout, br, bc, check)
    Hg = inputs.bits(H[torch.from_numpy(check).to(DEV)])
    to_f64 = lambda bits_: torch.from_numpy(bits_.view(np.int16)).view(torch.bfloat16).double().numpy()
    h_ref, h_got = to_f64(Hr), to_f64(Hg)
    # The two sides round the same real number h = silu(g) * u once to bf16, but from g and u that carry the
    # products' own tolerance (|dg| <= tol * S_g, S = sum_k |x_k w_k|; fp32 against fp64 accumulation).  First order:
    #   |dh| <= 2^-8 |h| (one bf16 step) + tol * (|silu'(g)| |u| S_g + |silu(g)| S_u),  |silu'| <= 1.1.
    # Where g or u cancels to almost nothing, h is tiny and several of ITS steps apart while the absolute error
    # stays at the scale of the sums; tol is asserted at 1e-4, ten times tighter than the GEMM's own bound.
    bound_abs = np.zeros_like(h_ref)
    Xb = inputs.bits(X)
    for t, r in enumerate(check):
        e = int(np.searchsorted(offsets, r, side="right") - 1)
        gu, S_gu = tlo.matmul_at(Xb[r:r + 1], inputs.bits(Wgu_t[e].reshape(-1)), layout, br, bc, 1, 2 * inter, hidden,
                                 np.zeros(2 * inter, dtype=np.int64), np.arange(2 * inter))
        g, u, Sg, Su = gu[0::2], gu[1::2], S_gu[0::2], S_gu[1::2]
        bound_abs[t] = 1e-4 * (1.1 * np.abs(u) * Sg + np.abs(g / (1 + np.exp(-g))) * Su)
    dh = np.abs(h_got - h_ref)
    assert np.all(dh <= 2.0 ** -8 * np.abs(h_ref) + bound_abs + 1e-30), float(np.max(dh - 2.0 ** -8 * np.abs(h_ref) - bound_abs))
    assert np.mean(_bf16_steps(Hg, Hr) == 0) > 0.97
    # y: the oracle multiplies ITS h.  |dy| <= 1e-3 * S_y (the product's own bound) + sum_j |dh_j| |w_jc|
    Yg = Y[torch.from_numpy(check).to(DEV)].cpu().numpy().astype(np.float64)
    err = np.abs(Yg - Yr)
    Wd_abs = np.abs(Wd.double().cpu().numpy())                                # logical [E, inter, hidden]
    dh_bound = 2.0 ** -8 * np.abs(h_ref) + bound_abs
    carry = np.stack([dh_bound[t] @ Wd_abs[int(np.searchsorted(offsets, r, side="right") - 1)] for t, r in enumerate(check)])
    assert np.all(err <= 1e-3 * Sr + carry + 1e-30)
    assert float(np.median(err / np.maximum(Sr, 1e-300))) <= 2e-4
    return rows


@pytest.mark.parametrize("br,bc", [(16, 128), (32, 64), (0, 0)])
def test_small_expert_ffn(br, bc):
    _run_case(E=8, hidden=256, inter=128, tokens=64, topk=2, br=br, bc=bc, n_check=24, seed=5)


def test_qwen3_30b_a3b_expert_ffn_full_size_sampled():
    q = inputs.QWEN_MOE
    rows = _run_case(E=q["experts"], hidden=q["hidden"], inter=q["inter"], tokens=q["tokens"], topk=q["topk"], br=16, bc=128,
                     n_check=12, seed=0)
    assert rows == q["tokens"] * q["topk"]


def test_gated_epilogue_alone_exact_on_constructed_inputs():
    # x = one-hot rows: g and u are single weights, so h = bf16(silu(w_g) * w_u) can be checked value by value
    from gpu_util import DEV, tl
    E, hidden, inter = 4, 128, 64
    offsets = np.array([0, 3, 3, 20, 33], dtype=np.int32)
    rows = 33
    X, ks = inputs.one_hot_rows(rows, hidden, seed=2)
    Wgu = inputs.bf16_normal((E, hidden, 2 * inter), 1.0, seed=3)
    H = torch.full((rows, inter), float("nan"), dtype=torch.bfloat16, device=DEV)
    tl.gemm_grouped_swiglu(X.to(DEV), Wgu.to(DEV), H, torch.from_numpy(offsets).to(DEV), E, rows, 2 * inter, hidden, 0, 0, 0)
    tl.device_status()
    Hg = inputs.bits(H)
    for r in range(rows):
        e = int(np.searchsorted(offsets, r, side="right") - 1)
        w = Wgu[e, int(ks[r])].double().numpy()
        want = np.array([tlo.double_to_bf16(tlo.silu(float(g)) * float(u)) for g, u in zip(w[0::2], w[1::2])], dtype=np.uint16)
        assert np.all(_bf16_steps(Hg[r], want) <= 1)
        assert np.mean(Hg[r] == want) > 0.9


def test_unsupported_and_invalid():
    from gpu_util import DEV, tl
    X = torch.zeros((300, 128), dtype=torch.bfloat16, device=DEV)
    W = torch.zeros((1, 128, 128), dtype=torch.bfloat16, device=DEV)
    H = torch.zeros((300, 64), dtype=torch.bfloat16, device=DEV)
    off = torch.tensor([0, 300], dtype=torch.int32, device=DEV)
    with pytest.raises(tl.TileLensError) as e:
        tl.gemm_grouped_swiglu(X, W, H, off, 1, 300, 128, 128, 0, 0, 0, (256, 128, 64))     # 256-row tiles: weights on the M side
    assert e.value.status == 2
    with pytest.raises(tl.TileLensError) as e:
        tl.gemm_grouped_swiglu(X, W, H, off, 1, 300, 96, 128, 0, 0, 0)                      # N not a multiple of 64
    assert e.value.status == 1


@pytest.mark.parametrize("E,hidden,inter,tokens,topk", [(8, 256, 128, 64, 2), (128, 2048, 768, 256, 8), (16, 128, 512, 96, 4),
                                                       (3, 4096, 64, 700, 1)])
def test_one_launch_and_two_launches_give_the_same_bits(E, hidden, inter, tokens, topk):
    # With TL_OPT_FFN_ONE_LAUNCH = 1 tl_moe_ffn runs both products as two phases of one cooperative launch (a
    # grid-wide barrier between them, the first product's split tiles summed inside the kernel) instead of two
    # launches.  Same tiles, same K ranges, same order of every sum: H and Y must agree bit for bit, repeatedly.
    from gpu_util import DEV, guarded_out, tl
    offsets, counts, _ = inputs.zipf_topk_routing(tokens, E, topk, 1.1, seed=3)
    rows = int(offsets[-1])
    X = inputs.bf16_normal((rows, hidden), 1.0, seed=1, device=DEV)
    Wgu = inputs.bf16_normal((E, hidden, 2 * inter), 0.05, seed=2, device=DEV)
    Wd = inputs.bf16_normal((E, inter, hidden), 0.05, seed=3, device=DEV)
    Wgu_t, Wd_t = torch.empty_like(Wgu), torch.empty_like(Wd)
    tl.relayout(Wgu, Wgu_t, E * hidden, 2 * inter, 2, 4096, 16, 128, tl.TO_TILE_MAJOR)
    tl.relayout(Wd, Wd_t, E * inter, hidden, 2, 4096, 16, 128, tl.TO_TILE_MAJOR)
    d_off = torch.from_numpy(offsets).to(DEV)

    def run():
        gH, gY = guarded_out((rows, inter), torch.bfloat16), guarded_out((rows, hidden), torch.float32)
        tl.moe_ffn(X, Wgu_t, Wd_t, gH.t, gY.t, d_off, E, rows, hidden, inter, 4096, 16, 128)
        chained = tl.gemm_last_plan().chained
        tl.device_status()
        return gH.check().clone(), gY.check().clone(), chained

    H0, Y0, chained0 = run()
    assert chained0 == 0
    for rep in range(3):
        with tl.option(tl.OPT_FFN_ONE_LAUNCH, 1):
            H1, Y1, chained1 = run()
        assert chained1 == 1, "the one-launch form was not taken"
        assert torch.equal(H1.view(torch.int16), H0.view(torch.int16)) and torch.equal(Y1, Y0), rep
    assert torch.isfinite(Y1).all()


@pytest.mark.parametrize("case", [dict(E=8, hidden=256, inter=128, tokens=64, topk=2, n_check=24, seed=5),
                                  dict(E=16, hidden=128, inter=512, tokens=96, topk=4, n_check=24, seed=6),
                                  dict(E=3, hidden=4096, inter=64, tokens=700, topk=1, n_check=12, seed=7),
                                  dict(E=128, hidden=2048, inter=768, tokens=256, topk=8, n_check=12, seed=0)])
def test_one_launch_with_per_m_tile_counters_against_the_oracle(case):
    # TL_OPT_FFN_ONE_LAUNCH = 2: one cooperative launch without grid barriers.  The first product runs whole tiles only
    # (so H may differ from the two-launch form in the order of a sum, never by more than the bound below), every
    # epilogue warp counts the m-tile it has stored, and the second product's producer waits for the m-tile it loads.
    # Checked against the oracle with the two-launch form's bounds, and for run-to-run reproducibility.
    from gpu_util import DEV, tl
    with tl.option(tl.OPT_FFN_ONE_LAUNCH, 2):
        _run_case(br=16, bc=128, want_chained=2, **case)
    E, hidden, inter = case["E"], case["hidden"], case["inter"]
    offsets, counts, _ = inputs.zipf_topk_routing(case["tokens"], E, case["topk"], 1.1, seed=case["seed"])
    rows = int(offsets[-1])
    X = inputs.bf16_normal((rows, hidden), 1.0, seed=11, device=DEV)
    Wgu = inputs.bf16_normal((E, hidden, 2 * inter), 0.05, seed=12, device=DEV)
    Wd = inputs.bf16_normal((E, inter, hidden), 0.05, seed=13, device=DEV)
    d_off = torch.from_numpy(offsets).to(DEV)
    outs = []
    for mode in (2, 2, 0):
        H = torch.zeros((rows, inter), dtype=torch.bfloat16, device=DEV)
        Y = torch.zeros((rows, hidden), dtype=torch.float32, device=DEV)
        with tl.option(tl.OPT_FFN_ONE_LAUNCH, mode):
            tl.moe_ffn(X, Wgu, Wd, H, Y, d_off, E, rows, hidden, inter, 0, 0, 0)
            tl.device_status()
        outs.append((H, Y))
    assert torch.equal(outs[0][0].view(torch.int16), outs[1][0].view(torch.int16)) and torch.equal(outs[0][1], outs[1][1])
    # against the two-launch form: a sum in another order now and then (one bf16 step of h, or a few steps of an h that
    # is tiny because g or u cancelled, see _run_case)
    steps = _bf16_steps(inputs.bits(outs[0][0]), inputs.bits(outs[2][0]))
    assert np.mean(steps == 0) > 0.99
    h_scale = float(outs[2][0].float().abs().max())
    assert float((outs[0][0].float() - outs[2][0].float()).abs().max()) <= 2.0 ** -7 * h_scale
    scale = float(outs[2][1].abs().max())
    assert float((outs[0][1] - outs[2][1]).abs().max()) <= 2e-3 * scale


def test_m_tile_counter_wait_that_runs_out_is_reported_and_the_next_call_is_clean():
    # Counter form: CTA 0 keeps the arrivals of its tiles to itself (test hook), the producers that need those m-tiles wait
    # out the shortened limit, the kernel terminates, the status reads TL_ERR_TIMEOUT (detail 0x900), the next call is clean.
    from gpu_util import DEV, tl
    E, hidden, inter = 16, 128, 512
    offsets, counts, _ = inputs.zipf_topk_routing(96, E, 4, 1.1, seed=4)
    rows = int(offsets[-1])
    X = inputs.bf16_normal((rows, hidden), 1.0, seed=1, device=DEV)
    Wgu = inputs.bf16_normal((E, hidden, 2 * inter), 0.05, seed=2, device=DEV)
    Wd = inputs.bf16_normal((E, inter, hidden), 0.05, seed=3, device=DEV)
    d_off = torch.from_numpy(offsets).to(DEV)
    H = torch.zeros((rows, inter), dtype=torch.bfloat16, device=DEV)
    Y = torch.zeros((rows, hidden), dtype=torch.float32, device=DEV)
    with tl.option(tl.OPT_FFN_ONE_LAUNCH, 2):
        tl.moe_ffn(X, Wgu, Wd, H, Y, d_off, E, rows, hidden, inter, 0, 0, 0)
        tl.device_status()
        H0, Y0 = H.clone(), Y.clone()
        with tl.option(tl.OPT_WAIT_LIMIT_US, 2000):
            tl.set_option(tl.OPT_STALL_ONCE, 3)
            tl.moe_ffn(X, Wgu, Wd, H, Y, d_off, E, rows, hidden, inter, 0, 0, 0)
            assert tl.get_option(tl.OPT_STALL_ONCE) == 0 and tl.gemm_last_plan().chained == 2
            with pytest.raises(tl.TileLensError) as e:
                tl.device_status()
            assert e.value.status == 5 and "detail=0x900" in str(e.value)
        tl.device_status()
        for _ in range(2):
            H.zero_(); Y.zero_()
            tl.moe_ffn(X, Wgu, Wd, H, Y, d_off, E, rows, hidden, inter, 0, 0, 0)
            assert tl.gemm_last_plan().chained == 2
            tl.device_status()
            assert torch.equal(H.view(torch.int16), H0.view(torch.int16)) and torch.equal(Y, Y0)


def test_grid_barrier_wait_that_runs_out_is_reported_and_the_next_call_is_clean():
    # One-launch form: CTA 0 stays away from the first grid barrier (test hook), every CTA's bounded wait runs out
    # after the shortened limit, the kernel still terminates, the status reads TL_ERR_TIMEOUT (detail 0x800), the
    # arrival counter is reset by the report, and the next call gives the bits of the two-launch form.
    from gpu_util import DEV, tl
    E, hidden, inter = 16, 128, 512
    offsets, counts, _ = inputs.zipf_topk_routing(96, E, 4, 1.1, seed=4)
    rows = int(offsets[-1])
    X = inputs.bf16_normal((rows, hidden), 1.0, seed=1, device=DEV)
    Wgu = inputs.bf16_normal((E, hidden, 2 * inter), 0.05, seed=2, device=DEV)
    Wd = inputs.bf16_normal((E, inter, hidden), 0.05, seed=3, device=DEV)
    d_off = torch.from_numpy(offsets).to(DEV)
    H = torch.zeros((rows, inter), dtype=torch.bfloat16, device=DEV)
    Y = torch.zeros((rows, hidden), dtype=torch.float32, device=DEV)
    tl.moe_ffn(X, Wgu, Wd, H, Y, d_off, E, rows, hidden, inter, 0, 0, 0)          # two launches: the reference bits
    tl.device_status()
    H0, Y0 = H.clone(), Y.clone()
    with tl.option(tl.OPT_FFN_ONE_LAUNCH, 1), tl.option(tl.OPT_WAIT_LIMIT_US, 2000):
        tl.set_option(tl.OPT_STALL_ONCE, 3)
        tl.moe_ffn(X, Wgu, Wd, H, Y, d_off, E, rows, hidden, inter, 0, 0, 0)
        assert tl.get_option(tl.OPT_STALL_ONCE) == 0 and tl.gemm_last_plan().chained == 1
        with pytest.raises(tl.TileLensError) as e:
            tl.device_status()
        assert e.value.status == 5 and "detail=0x800" in str(e.value)
        tl.device_status()
        for _ in range(2):
            H.zero_(); Y.zero_()
            tl.moe_ffn(X, Wgu, Wd, H, Y, d_off, E, rows, hidden, inter, 0, 0, 0)
            assert tl.gemm_last_plan().chained == 1
            tl.device_status()
            assert torch.equal(H.view(torch.int16), H0.view(torch.int16)) and torch.equal(Y, Y0)
