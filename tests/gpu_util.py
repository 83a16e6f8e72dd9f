"""Helpers shared by the GPU parity tests (not a test module)."""
import numpy as np
import torch

import oracle as tlo
from paper_2607_04031_b200 import binding as tl
from paper_2607_04031_b200 import inputs

DEV = "cuda:0"


# Output buffers of the parity tests sit between two guard blocks holding a fixed bit pattern, checked after every
# call: a kernel that writes outside its output (the kind of fault a memory checker would report) changes a guard
# word and fails the test, while the NaN fill of the payload catches elements that were never written.
GUARD_BYTES = 4096
GUARD_WORD = 0x5AC3E1D7


class Guarded:
    """A CUDA tensor of `shape` / `dtype` with GUARD_BYTES of known words before and after it."""

    def __init__(self, shape, dtype, fill=None):
        item = torch.empty((), dtype=dtype).element_size()
        n = int(np.prod(shape)) if len(shape) else 1
        self.payload_bytes = n * item
        pad_tail = (-self.payload_bytes) % 4
        self.raw = torch.empty(GUARD_BYTES + self.payload_bytes + pad_tail + GUARD_BYTES, dtype=torch.uint8, device=DEV)
        words = self.raw.view(torch.int32)
        words.fill_(GUARD_WORD)
        self.t = self.raw[GUARD_BYTES:GUARD_BYTES + self.payload_bytes].view(dtype).view(shape)
        if fill is not None:
            self.t.fill_(fill)
        self._front = words[:GUARD_BYTES // 4]
        self._back = words[(GUARD_BYTES + self.payload_bytes + pad_tail) // 4:]

    def check(self):
        torch.cuda.synchronize()
        assert bool((self._front == GUARD_WORD).all()), "write before the start of the output buffer"
        assert bool((self._back == GUARD_WORD).all()), "write past the end of the output buffer"
        return self.t


def guarded_out(shape, dtype, fill=float("nan")):
    g = Guarded(shape, dtype, fill if dtype.is_floating_point else None)
    return g


def dev_bytes(arr: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(arr).view(np.uint8).reshape(-1).copy()).to(DEV)


def tile_major_on_device(B_row: torch.Tensor, K: int, N: int, br: int, bc: int) -> torch.Tensor:
    """Relayout with the CUDA library (the product path); returns the tile-major bf16 buffer."""
    B_row = B_row.to(DEV).contiguous()
    g = Guarded(tuple(B_row.shape), B_row.dtype)
    tl.relayout(B_row, g.t, K, N, 2, br * bc * 2, br, bc, tl.TO_TILE_MAJOR)
    return g.check()


def run_gemm(A: torch.Tensor, B_dev: torch.Tensor, M, N, K, br, bc, cta=(0, 0, 0)) -> torch.Tensor:
    A = A.to(DEV).contiguous()
    g = guarded_out((M, N), torch.float32)
    tl.gemm(A, B_dev, g.t, M, N, K, br * bc * 2, br, bc, cta)
    tl.device_status()
    return g.check()


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
