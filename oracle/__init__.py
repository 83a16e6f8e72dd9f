"""ctypes front end of the TileLens ORACLE (test infrastructure only).

The arithmetic lives in ``tlo.c``; this file only compiles it with gcc, loads
it and marshals numpy arrays.  Nothing here imports, or is imported by, the
CUDA package.  Callers: the tests, the smoke check and the CPU-baseline leg of
the benchmark.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tlo.c")
_HDR = os.path.join(_HERE, "tlo.h")
_LIB = os.path.join(_HERE, "libtlo.so")

ROW_MAJOR, COL_MAJOR, TILE_MAJOR, TILE_MAJOR_K = 0, 1, 2, 3
TO_TILE_MAJOR, TO_ROW_MAJOR = 0, 1


def build(force: bool = False) -> str:
    """Compile tlo.c into libtlo.so (plain -O2, OpenMP, no SIMD flags)."""
    stale = (not os.path.exists(_LIB)
             or os.path.getmtime(_LIB) < max(os.path.getmtime(_SRC), os.path.getmtime(_HDR)))
    if force or stale:
        tmp = f"{_LIB}.{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-shared", "-fPIC",
                               "-Wall", "-Wextra", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class HwDesc(ctypes.Structure):
    """Mirror of tlo_hw_desc (Section 4.3: a tensor view plus the memory tile (a, b) and the leading stride K)."""
    _fields_ = [("rank", ctypes.c_int32), ("s", ctypes.c_int32), ("dims", ctypes.c_int64 * 5),
                ("strides", ctypes.c_int64 * 5), ("box", ctypes.c_int64 * 5), ("a", ctypes.c_int64),
                ("b", ctypes.c_int64), ("K", ctypes.c_int64)]


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        i64, u64p, vp = ctypes.c_int64, ctypes.POINTER(ctypes.c_uint64), ctypes.c_void_p
        for name in ("tlo_off_row", "tlo_off_col"):
            getattr(L, name).restype = i64
            getattr(L, name).argtypes = [i64] * 5
        L.tlo_off_tile.restype = i64
        L.tlo_off_tile.argtypes = [i64] * 7
        L.tlo_off.restype = i64
        L.tlo_off.argtypes = [ctypes.c_int] + [i64] * 7
        L.tlo_eq1.restype = None
        L.tlo_eq1.argtypes = [i64] * 4 + [ctypes.POINTER(i64)]
        for name in ("tlo_eq2", "tlo_eq3"):
            getattr(L, name).restype = i64
            getattr(L, name).argtypes = [i64] * 7
        L.tlo_relayout.restype = ctypes.c_int
        L.tlo_relayout.argtypes = [vp, vp, i64, i64, i64, i64, i64, ctypes.c_int]
        L.tlo_bf16_to_double.restype = ctypes.c_double
        L.tlo_bf16_to_double.argtypes = [ctypes.c_uint16]
        L.tlo_matmul_at.restype = ctypes.c_int
        L.tlo_matmul_at.argtypes = [vp, vp, ctypes.c_int, i64, i64, i64, i64, i64, i64, vp, vp, vp, vp]
        L.tlo_fp8_e4m3_to_double.restype = ctypes.c_double
        L.tlo_fp8_e4m3_to_double.argtypes = [ctypes.c_uint8]
        L.tlo_matmul_at_fp8.restype = ctypes.c_int
        L.tlo_matmul_at_fp8.argtypes = [vp, vp, ctypes.c_int, i64, i64, i64, i64, i64, i64, vp, vp, vp, vp]
        L.tlo_matmul.restype = ctypes.c_int
        L.tlo_matmul.argtypes = [vp, vp, ctypes.c_int, i64, i64, i64, i64, i64, vp, vp]
        L.tlo_read_amp.restype = ctypes.c_int
        L.tlo_read_amp.argtypes = [i64] * 6 + [ctypes.c_int] + [i64] * 4 + [u64p, u64p, u64p, vp, vp]
        L.tlo_read_amp_grouped.restype = ctypes.c_int
        L.tlo_read_amp_grouped.argtypes = ([vp, ctypes.c_int] + [i64] * 5 + [ctypes.c_int] + [i64] * 4
                                           + [u64p, u64p, u64p])
        L.tlo_read_amp_shared.restype = ctypes.c_int
        L.tlo_read_amp_shared.argtypes = [i64] * 7 + [ctypes.c_int] + [i64] * 4 + [u64p, u64p, u64p]
        L.tlo_prefetch_degree.restype = i64
        L.tlo_prefetch_degree.argtypes = [ctypes.c_double, ctypes.c_double, i64, i64, i64, i64, i64, i64, ctypes.c_double]
        L.tlo_tile_arrival.restype = ctypes.c_int
        L.tlo_tile_arrival.argtypes = [vp, i64, i64, ctypes.c_double, ctypes.POINTER(ctypes.c_double),
                                       ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double)]
        L.tlo_double_to_bf16.restype = ctypes.c_uint16
        L.tlo_double_to_bf16.argtypes = [ctypes.c_double]
        L.tlo_silu.restype = ctypes.c_double
        L.tlo_silu.argtypes = [ctypes.c_double]
        L.tlo_moe_ffn_rows.restype = ctypes.c_int
        L.tlo_moe_ffn_rows.argtypes = [vp, vp, vp, vp, ctypes.c_int, i64, i64, ctypes.c_int, i64, i64, i64, vp, vp, vp, vp]
        L.tlo_hw_box_offsets.restype = ctypes.c_int
        L.tlo_hw_box_offsets.argtypes = [ctypes.POINTER(HwDesc), vp, vp]
        L.tlo_num_threads.restype = ctypes.c_int
        L.tlo_num_threads.argtypes = []
        _lib = L
    return _lib


def num_threads() -> int:
    return int(lib().tlo_num_threads())


def _ptr(a: np.ndarray) -> ctypes.c_void_p:
    return ctypes.c_void_p(a.ctypes.data)


def off_row(r, c, rows, cols, s):
    return int(lib().tlo_off_row(r, c, rows, cols, s))


def off_col(r, c, rows, cols, s):
    return int(lib().tlo_off_col(r, c, rows, cols, s))


def off_tile(r, c, rows, cols, br, bc, s):
    return int(lib().tlo_off_tile(r, c, rows, cols, br, bc, s))


def off(layout, r, c, rows, cols, br, bc, s):
    return int(lib().tlo_off(layout, r, c, rows, cols, br, bc, s))


def eq1(i, j, a, b):
    out = (ctypes.c_int64 * 4)()
    lib().tlo_eq1(i, j, a, b, out)
    return tuple(int(x) for x in out)


def eq2(i, j, K, N, a, b, s):
    return int(lib().tlo_eq2(i, j, K, N, a, b, s))


def eq3(i, j, K, N, a, b, s):
    return int(lib().tlo_eq3(i, j, K, N, a, b, s))


def relayout(src: np.ndarray, rows: int, cols: int, s: int, br: int, bc: int, direction: int) -> np.ndarray:
    """src: contiguous uint8 array of rows*cols*s bytes.  Returns the permuted bytes."""
    src = np.ascontiguousarray(src).view(np.uint8).reshape(-1)
    assert src.size == rows * cols * s
    dst = np.empty_like(src)
    rc = lib().tlo_relayout(_ptr(src), _ptr(dst), rows, cols, s, br, bc, direction)
    if rc != 0:
        raise ValueError(f"tlo_relayout rejected its arguments (rc={rc})")
    return dst


def bf16_to_double(h: int) -> float:
    return float(lib().tlo_bf16_to_double(h))


def matmul(A_bits: np.ndarray, B_bits: np.ndarray, layout: int, br: int, bc: int, M: int, N: int, K: int):
    """A_bits: uint16 [M,K] row-major; B_bits: uint16 buffer of K*N in `layout`.  Returns (C, S) fp64 [M,N]."""
    A_bits = np.ascontiguousarray(A_bits, dtype=np.uint16)
    B_bits = np.ascontiguousarray(B_bits, dtype=np.uint16)
    assert A_bits.size == M * K and B_bits.size == K * N
    C = np.empty((M, N), dtype=np.float64)
    S = np.empty((M, N), dtype=np.float64)
    rc = lib().tlo_matmul(_ptr(A_bits), _ptr(B_bits), layout, br, bc, M, N, K, _ptr(C), _ptr(S))
    if rc != 0:
        raise ValueError(f"tlo_matmul rejected its arguments (rc={rc})")
    return C, S


def matmul_at(A_bits, B_bits, layout, br, bc, M, N, K, idx_i, idx_j):
    """The product at the listed (i, j) only.  Returns (C, S) fp64 vectors."""
    A_bits = np.ascontiguousarray(A_bits, dtype=np.uint16)
    B_bits = np.ascontiguousarray(B_bits, dtype=np.uint16)
    assert A_bits.size == M * K and B_bits.size == K * N
    ii = np.ascontiguousarray(idx_i, dtype=np.int64)
    jj = np.ascontiguousarray(idx_j, dtype=np.int64)
    assert ii.shape == jj.shape and ii.ndim == 1
    C = np.empty(ii.size, dtype=np.float64)
    S = np.empty(ii.size, dtype=np.float64)
    rc = lib().tlo_matmul_at(_ptr(A_bits), _ptr(B_bits), layout, br, bc, M, N, K, ii.size,
                             _ptr(ii), _ptr(jj), _ptr(C), _ptr(S))
    if rc != 0:
        raise ValueError(f"tlo_matmul_at rejected its arguments (rc={rc})")
    return C, S


def fp8_e4m3_to_double(h: int) -> float:
    return float(lib().tlo_fp8_e4m3_to_double(h))


def matmul_at_fp8(A_bits, B_bits, layout, br, bc, M, N, K, idx_i, idx_j):
    """FP8 (E4M3) operands as uint8 bit patterns; otherwise as matmul_at."""
    A_bits = np.ascontiguousarray(A_bits, dtype=np.uint8)
    B_bits = np.ascontiguousarray(B_bits, dtype=np.uint8)
    assert A_bits.size == M * K and B_bits.size == K * N
    ii = np.ascontiguousarray(idx_i, dtype=np.int64)
    jj = np.ascontiguousarray(idx_j, dtype=np.int64)
    assert ii.shape == jj.shape and ii.ndim == 1
    C = np.empty(ii.size, dtype=np.float64)
    S = np.empty(ii.size, dtype=np.float64)
    rc = lib().tlo_matmul_at_fp8(_ptr(A_bits), _ptr(B_bits), layout, br, bc, M, N, K, ii.size,
                                 _ptr(ii), _ptr(jj), _ptr(C), _ptr(S))
    if rc != 0:
        raise ValueError(f"tlo_matmul_at_fp8 rejected its arguments (rc={rc})")
    return C, S


def read_amp(M, N, K, BM, BN, BK, layout, G, br, bc, s, per_tile=False):
    """Returns (fetched, used, requests) or, with per_tile, also the two per-CTA-tile arrays."""
    f, u, q = ctypes.c_uint64(), ctypes.c_uint64(), ctypes.c_uint64()
    pf = pu = None
    a = b = ctypes.c_void_p(None)
    if per_tile:
        mt, nt = -(-M // BM), -(-N // BN)
        pf = np.zeros(mt * nt, dtype=np.uint64)
        pu = np.zeros(mt * nt, dtype=np.uint64)
        a, b = _ptr(pf), _ptr(pu)
    rc = lib().tlo_read_amp(M, N, K, BM, BN, BK, layout, G, br, bc, s,
                            ctypes.byref(f), ctypes.byref(u), ctypes.byref(q), a, b)
    if rc != 0:
        raise ValueError(f"tlo_read_amp rejected its arguments (rc={rc})")
    if per_tile:
        return int(f.value), int(u.value), int(q.value), pf, pu
    return int(f.value), int(u.value), int(q.value)


def read_amp_shared(M, N, K, BM, BN, BK, P, layout, G, br, bc, s):
    """(fetched, needed, requests) when the P co-resident CTA tiles share the blocks they want at the same K step."""
    f, u, q = ctypes.c_uint64(), ctypes.c_uint64(), ctypes.c_uint64()
    rc = lib().tlo_read_amp_shared(M, N, K, BM, BN, BK, P, layout, G, br, bc, s,
                                   ctypes.byref(f), ctypes.byref(u), ctypes.byref(q))
    if rc != 0:
        raise ValueError(f"tlo_read_amp_shared rejected its arguments (rc={rc})")
    return int(f.value), int(u.value), int(q.value)


def tile_arrival(samples, requests: int, threshold: float = 0.0):
    """(E[first arrival], E[last arrival], P(last arrival > threshold)) of `requests` independent draws from the sample."""
    x = np.ascontiguousarray(samples, dtype=np.float64)
    first, last, late = ctypes.c_double(), ctypes.c_double(), ctypes.c_double()
    if lib().tlo_tile_arrival(_ptr(x), x.size, requests, threshold, ctypes.byref(first), ctypes.byref(last),
                              ctypes.byref(late)) != 0:
        raise ValueError("tlo_tile_arrival rejected its arguments")
    return first.value, last.value, late.value


def prefetch_degree(bandwidth, latency, G, n_sm, ctas_per_sm, p_tile, K, tile_k, collision_factor=1.0) -> int:
    d = int(lib().tlo_prefetch_degree(bandwidth, latency, G, n_sm, ctas_per_sm, p_tile, K, tile_k, collision_factor))
    if d < 0:
        raise ValueError("tlo_prefetch_degree rejected its arguments")
    return d


def double_to_bf16(x: float) -> int:
    return int(lib().tlo_double_to_bf16(x))


def silu(x: float) -> float:
    return float(lib().tlo_silu(x))


def moe_ffn_rows(X_bits, Wgu_bits, Wd_bits, offsets, hidden, inter, layout, br, bc, rows):
    """Returns (H bf16 bits [n, inter], Y fp64 [n, hidden], S fp64 [n, hidden]) for the listed rows."""
    X_bits = np.ascontiguousarray(X_bits, dtype=np.uint16)
    Wgu_bits = np.ascontiguousarray(Wgu_bits, dtype=np.uint16)
    Wd_bits = np.ascontiguousarray(Wd_bits, dtype=np.uint16)
    offs = np.ascontiguousarray(offsets, dtype=np.int32)
    E = offs.size - 1
    assert Wgu_bits.size == E * hidden * 2 * inter and Wd_bits.size == E * inter * hidden
    rr = np.ascontiguousarray(rows, dtype=np.int64)
    H = np.empty((rr.size, inter), dtype=np.uint16)
    Y = np.empty((rr.size, hidden), dtype=np.float64)
    S = np.empty((rr.size, hidden), dtype=np.float64)
    rc = lib().tlo_moe_ffn_rows(_ptr(X_bits), _ptr(Wgu_bits), _ptr(Wd_bits), _ptr(offs), E, hidden, inter, layout, br, bc,
                                rr.size, _ptr(rr), _ptr(H), _ptr(Y), _ptr(S))
    if rc != 0:
        raise ValueError(f"tlo_moe_ffn_rows rejected its arguments (rc={rc})")
    return H, Y, S


def hw_desc(dims, strides, box, s, a, b, K) -> HwDesc:
    d = HwDesc()
    d.rank, d.s, d.a, d.b, d.K = len(dims), s, a, b, K
    for k in range(len(dims)):
        d.dims[k], d.strides[k], d.box[k] = dims[k], strides[k], box[k]
    return d


def hw_box_offsets(desc: HwDesc, coords) -> np.ndarray:
    """Source byte offsets of one box load in counter order (Section 4.3)."""
    c = np.ascontiguousarray(coords, dtype=np.int64)
    assert c.size == desc.rank
    n = 1
    for k in range(desc.rank):
        n *= int(desc.box[k])
    out = np.empty(n, dtype=np.int64)
    rc = lib().tlo_hw_box_offsets(ctypes.byref(desc), _ptr(c), _ptr(out))
    if rc != 0:
        raise ValueError(f"tlo_hw_box_offsets rejected its arguments (rc={rc})")
    return out


def read_amp_grouped(offsets, N, K, BM, BN, BK, layout, G, br, bc, s):
    offs = np.ascontiguousarray(offsets, dtype=np.int32)
    f, u, q = ctypes.c_uint64(), ctypes.c_uint64(), ctypes.c_uint64()
    rc = lib().tlo_read_amp_grouped(_ptr(offs), offs.size - 1, N, K, BM, BN, BK, layout, G, br, bc, s,
                                    ctypes.byref(f), ctypes.byref(u), ctypes.byref(q))
    if rc != 0:
        raise ValueError(f"tlo_read_amp_grouped rejected its arguments (rc={rc})")
    return int(f.value), int(u.value), int(q.value)
