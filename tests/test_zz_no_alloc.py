"""tl_gemm_noalloc: the GEMM for callers that may not allocate device memory (GPU).

Some hosts of this library cannot call cudaMalloc once they are running: an inference server that
gave all of HBM to its own pool at start-up, a sandbox that forbids allocation after initialisation.
For them the split-K scratch lives in a fixed array inside the library.  This file checks that the
entry point, called through the C ABI, gives what tl_gemm gives (bit for bit on integer data, within
the GEMM tolerance otherwise), twice in a row (the array
keeps the first call's contents, so the second call proves the clean-up), and that it refuses
problems whose scratch does not fit.  It is collected last so that a failure here cannot hide
another test's result; it does not depend on any other test having run.
"""
import numpy as np
import pytest
import torch

import oracle as tlo
from paper_2607_04031_b200 import inputs

pytestmark = pytest.mark.gpu


def _case(M, N, K, seed, integer):
    from gpu_util import DEV, tile_major_on_device
    if integer:
        A = inputs.bf16_integers((M, K), -8, 8, seed=seed)
        B = inputs.bf16_integers((K, N), -8, 8, seed=seed + 1)
    else:
        A = inputs.bf16_normal((M, K), 1.0, seed=seed)
        B = inputs.bf16_normal((K, N), 0.02, seed=seed + 1)
    # bound of the GEMM tests' tolerance: 1e-3 * sum_k |A_ik B_kj| (fp32 is plenty for a bound)
    S = A.to(DEV).float().abs() @ B.to(DEV).float().abs()
    return A.to(DEV).contiguous(), tile_major_on_device(B, K, N, 16, 128), S


@pytest.mark.parametrize("M,N,K,integer", [(8, 1024, 8192, True), (32, 2048, 4096, False), (1, 512, 2048, False)])
def test_matches_tl_gemm_on_two_calls_in_a_row(M, N, K, integer):
    from gpu_util import DEV, tl
    A, Bt, S = _case(M, N, K, seed=70 + M, integer=integer)
    want = torch.full((M, N), float("nan"), dtype=torch.float32, device=DEV)
    tl.gemm(A, Bt, want, M, N, K, 4096, 16, 128)          # existing entry point (allocating workspace)
    tl.device_status()
    flag = torch.zeros(1, dtype=torch.int32, device=DEV)
    # against the oracle directly (exact integers), not only against the other entry point
    exact = None
    if integer:
        exact, _ = tlo.matmul(inputs.bits(A), inputs.bits(Bt.reshape(-1)), tlo.TILE_MAJOR, 16, 128, M, N, K)
    outs = [torch.full((M, N), float("nan"), dtype=torch.float32, device=DEV) for _ in range(2)]
    for call in range(2):
        got = outs[call]
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        tl.gemm_noalloc(A, Bt, got, M, N, K, 4096, 16, 128, timeout_flag=flag)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        if call == 1:
            # the second call cannot even have loaded a module: the device's free memory is what it was
            assert free_after == free_before, "tl_gemm_noalloc changed the amount of free device memory"
        assert int(flag.item()) == 0, "a bounded wait expired inside the kernel"
        if exact is not None:
            assert np.array_equal(got.cpu().numpy().astype(np.float64), exact), f"call {call} against the oracle"
        # Same kernel; the fixed scratch may make the library pick a narrower tile, hence another split of
        # the K sums.  Integer inputs are exact in any order; otherwise both results lie within the GEMM
        # tests' tolerance of 1e-3 * sum|a b| of the true product, so within twice that of each other.
        if integer:
            assert torch.equal(got, want), f"call {call}"
        else:
            assert bool(((got - want).abs() <= 2e-3 * S).all()), f"call {call}"
            assert float((got - want).abs().max()) <= 1e-4 * float(S.max())
    # a different problem right after, then the first one again: stale partial tiles must not leak
    A2, Bt2, _ = _case(16, 768, 2048, seed=5, integer=True)
    want2 = torch.empty((16, 768), dtype=torch.float32, device=DEV)
    tl.gemm(A2, Bt2, want2, 16, 768, 2048, 4096, 16, 128)
    got2 = torch.empty_like(want2)
    tl.gemm_noalloc(A2, Bt2, got2, 16, 768, 2048, 4096, 16, 128)
    got = torch.empty_like(want)
    tl.gemm_noalloc(A, Bt, got, M, N, K, 4096, 16, 128)
    torch.cuda.synchronize()
    assert torch.equal(got2, want2)
    assert torch.equal(got, want) if integer else bool(((got - want).abs() <= 2e-3 * S).all())


def test_large_products_that_need_no_scratch_are_not_refused():
    # Prefill-sized products run on CTA pairs, which keep nothing in scratch memory: the size limit of the fixed
    # array does not apply to them, whatever the split-K plan of the single-CTA kernel would have asked for.
    from gpu_util import DEV, tile_major_on_device, tl
    M, N, K = 1800, 5120, 384
    A = inputs.bf16_integers((M, K), -8, 8, seed=3)
    B = inputs.bf16_integers((K, N), -8, 8, seed=4)
    Bt = tile_major_on_device(B, K, N, 16, 128)
    want = (A.to(torch.float64) @ B.to(torch.float64)).to(torch.float32)
    for call in range(2):
        got = torch.full((M, N), float("nan"), dtype=torch.float32, device=DEV)
        tl.gemm_noalloc(A.to(DEV), Bt, got, M, N, K, 4096, 16, 128)
        torch.cuda.synchronize()
        assert tl.gemm_last_plan().pair_kernel == 1
        assert torch.equal(got.cpu(), want), f"call {call}"


def test_refuses_scratch_beyond_the_fixed_array():
    from gpu_util import DEV, tl
    # 5 tiles of very long K and 37 MB of weights: neither whole tiles nor clusters (at most 40 CTAs) are worth it, so the
    # K loops are cut over all SMs and the partial tiles need 2 * SMs * 64 * 128 * 4 bytes > 8 MiB on a B200
    M, N, K = 64, 640, 28672
    A, Bt, _ = _case(M, N, K, seed=9, integer=True)
    C = torch.zeros((M, N), dtype=torch.float32, device=DEV)
    need = tl.gemm_workspace_bytes(M, N, K)
    if need <= (8 << 20) - 256:
        pytest.skip("this GPU has few enough SMs for the scratch to fit")
    with pytest.raises(tl.TileLensError) as e:
        tl.gemm_noalloc(A, Bt, C, M, N, K, 4096, 16, 128)
    assert e.value.status == 6
    torch.cuda.synchronize()
    assert float(C.abs().sum()) == 0.0                     # nothing was enqueued
