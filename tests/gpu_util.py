"""Helpers shared by the GPU parity tests (not a test module)."""
import numpy as np
import torch

import oracle as tlo
from paper_2607_04031_b200 import binding as tl
from paper_2607_04031_b200 import inputs

DEV = "cuda:0"


def dev_bytes(arr: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(arr).view(np.uint8).reshape(-1).copy()).to(DEV)


def tile_major_on_device(B_row: torch.Tensor, K: int, N: int, br: int, bc: int) -> torch.Tensor:
    """Relayout with the CUDA library (the product path); returns the tile-major bf16 buffer."""
    B_row = B_row.to(DEV).contiguous()
    out = torch.empty_like(B_row)
    tl.relayout(B_row, out, K, N, 2, br * bc * 2, br, bc, tl.TO_TILE_MAJOR)
    return out


def run_gemm(A: torch.Tensor, B_dev: torch.Tensor, M, N, K, br, bc, cta=(0, 0, 0)) -> torch.Tensor:
    A = A.to(DEV).contiguous()
    C = torch.full((M, N), float("nan"), dtype=torch.float32, device=DEV)
    tl.gemm(A, B_dev, C, M, N, K, br * bc * 2, br, bc, cta)
    tl.device_status()
    return C


def check_against_oracle(C: torch.Tensor, A: torch.Tensor, B_buf_dev: torch.Tensor, layout, br, bc, M, N, K,
                         idx=None, tol=1e-3, warn=1e-4):
    """|C - C_ref| <= tol * sum_k |A_ik B_kj| at every (sampled) element; returns the worst ratio."""
    A_bits = inputs.bits(A)
    B_bits = inputs.bits(B_buf_dev.reshape(-1))
    Ch = C.cpu().numpy().astype(np.float64)
    if idx is None:
        ref, S = tlo.matmul(A_bits, B_bits, layout, br, bc, M, N, K)
        got = Ch
    else:
        ii, jj = idx
        ref, S = tlo.matmul_at(A_bits, B_bits, layout, br, bc, M, N, K, ii, jj)
        got = Ch[ii, jj]
    assert np.all(np.isfinite(got)), "non-finite output (an element was never written?)"
    err = np.abs(got - ref)
    assert np.all(err <= tol * S), f"max err/S = {np.max(err / np.maximum(S, 1e-300)):.3e}"
    assert np.all(got[S == 0] == 0)
    worst = float(np.max(err / np.maximum(S, 1e-300)))
    assert worst <= warn, f"inside the tolerance but unexpectedly large: {worst:.3e}"
    return worst


def sample_indices(M, N, n, seed):
    rng = np.random.default_rng(seed)
    ii = rng.integers(0, M, n)
    jj = rng.integers(0, N, n)
    # always include the corners
    ii[:4] = [0, 0, M - 1, M - 1]
    jj[:4] = [0, N - 1, 0, N - 1]
    return ii, jj
