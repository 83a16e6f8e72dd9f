"""bf16 output option of the GEMM (fp32 accumulation, one rounding) through the C ABI vs the oracle (GPU)."""
import numpy as np
import pytest
import torch

import oracle as tlo
from paper_2607_04031_b200 import inputs

pytestmark = pytest.mark.gpu

SHAPES = [(8, 1024, 2048, (0, 0, 0)),        # decode: stream-K, reduction kernel writes C
          (40, 1024, 512, (64, 128, 64)),    # weights-on-N whole tiles
          (300, 1152, 576, (0, 0, 0)),       # 256-token tiles, single-CTA kernel, ragged rows
          (700, 9600, 320, (0, 0, 0)),       # CTA-pair kernel, ragged rows and columns
          (1800, 5120, 384, (0, 0, 0))]      # CTA-pair kernel with 512-token tiles


@pytest.mark.parametrize("M,N,K,cta", SHAPES)
def test_one_hot_rows_copy_rows_of_B_exactly(M, N, K, cta):
    from gpu_util import DEV, guarded_out, tile_major_on_device, tl
    A, ks = inputs.one_hot_rows(M, K, seed=7)
    B = inputs.bf16_normal((K, N), 0.02, seed=8)
    Bd = tile_major_on_device(B, K, N, 16, 128)
    g = guarded_out((M, N), torch.bfloat16)
    tl.gemm_bf16(A.to(DEV), Bd, g.t, M, N, K, 4096, 16, 128, cta)
    tl.device_status()
    C = g.check()
    assert torch.equal(C.cpu(), B[ks])                   # every value is a bf16 already: the rounding changes nothing


@pytest.mark.parametrize("M,N,K,cta", SHAPES)
def test_random_inputs_are_the_rounded_oracle_product(M, N, K, cta):
    from gpu_util import DEV, guarded_out, sample_indices, tile_major_on_device, tl
    A = inputs.bf16_normal((M, K), 1.0, seed=M)
    B = inputs.bf16_normal((K, N), 0.02, seed=N)
    Bd = tile_major_on_device(B, K, N, 16, 128)
    g = guarded_out((M, N), torch.bfloat16)
    tl.gemm_bf16(A.to(DEV), Bd, g.t, M, N, K, 4096, 16, 128, cta)
    tl.device_status()
    C = g.check()
    assert torch.isfinite(C.float()).all()
    ii, jj = sample_indices(M, N, 3000, seed=K)
    ref, S = tlo.matmul_at(inputs.bits(A), inputs.bits(Bd.reshape(-1)), tlo.TILE_MAJOR, 16, 128, M, N, K, ii, jj)
    got = C.cpu().double().numpy()[ii, jj]
    # one rounding to bf16 (half a step: 2^-9 relative) on top of the product's own tolerance
    assert np.all(np.abs(got - ref) <= 2.0 ** -9 * np.abs(ref) + 1e-3 * S + 1e-30)
    want_bits = np.array([tlo.double_to_bf16(float(x)) for x in ref], dtype=np.uint16)
    got_bits = inputs.bits(C.cpu())[ii, jj]
    assert np.mean(got_bits == want_bits) > 0.97         # the rest sit on a rounding boundary of the fp32 sum


def test_grouped_bf16_output():
    from gpu_util import DEV, guarded_out, tile_major_on_device, tl
    E, K, N = 8, 256, 384
    offsets, counts, _ = inputs.zipf_topk_routing(40, E, 3, 1.1, seed=3)
    rows = int(offsets[-1])
    A, ks = inputs.one_hot_rows(rows, K, seed=4)
    B = inputs.bf16_normal((E, K, N), 0.5, seed=5)
    Bt = tile_major_on_device(B.reshape(E * K, N), E * K, N, 16, 128)
    g = guarded_out((rows, N), torch.bfloat16)
    tl.gemm_grouped_bf16(A.to(DEV), Bt, g.t, torch.from_numpy(offsets).to(DEV), E, rows, N, K, 4096, 16, 128)
    tl.device_status()
    C = g.check()
    expert = np.searchsorted(offsets, np.arange(rows), side="right") - 1
    want = torch.stack([B[int(e), int(k)] for e, k in zip(expert, ks)])
    assert torch.equal(C.cpu(), want)


def test_invalid_arguments():
    from gpu_util import DEV, tl
    A = torch.zeros((8, 512), dtype=torch.bfloat16, device=DEV)
    W = torch.zeros((512, 516), dtype=torch.bfloat16, device=DEV)
    C = torch.zeros((8, 516), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(tl.TileLensError) as e:
        tl.gemm_bf16(A, W, C, 8, 516, 512, 0, 0, 0)          # N not a multiple of 8
    assert e.value.status == 1
