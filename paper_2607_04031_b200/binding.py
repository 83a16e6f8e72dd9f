"""Thin Python binding of the tilelens C ABI (``include/tilelens.h``): argument marshalling only.

Every step of the path runs inside ``libtilelens.so``.  torch is used for device
memory and streams, nothing else.  There is no fallback: if the library has not
been built, or a call returns a non-zero status, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtilelens.so")

TL_OK = 0
TO_TILE_MAJOR, TO_ROW_MAJOR = 0, 1
LAYOUT_ROW_MAJOR, LAYOUT_COL_MAJOR, LAYOUT_TILE_MAJOR, LAYOUT_TILE_MAJOR_K = 0, 1, 2, 3

# Every symbol include/tilelens.h declares: (name, restype, argtypes)
_i64, _int, _vp, _sz = ctypes.c_int64, ctypes.c_int, ctypes.c_void_p, ctypes.c_size_t
_u64p = ctypes.POINTER(ctypes.c_uint64)
_SIGNATURES = {
    "tl_status_string": (ctypes.c_char_p, [_int]),
    "tl_last_cuda_error": (_int, []),
    "tl_set_stream": (_int, [_vp]),
    "tl_device_status": (_int, [ctypes.POINTER(ctypes.c_uint32)]),
    "tl_set_option": (_int, [_int, _i64]),
    "tl_get_option": (_i64, [_int]),
    "tl_gemm_plan": (_int, [_i64, _i64, _i64, _i64, _int, _int, _int, _int, _int, _int, _int, _vp]),
    "tl_gemm_last_plan": (_int, [_vp]),
    "tl_relayout": (_int, [_vp, _vp, _i64, _i64, _int, _i64, _int, _int, _int]),
    "tl_relayout_on": (_int, [_vp, _vp, _i64, _i64, _int, _i64, _int, _int, _int, _vp]),
    "tl_relayout_batch": (_int, [_int, _vp, _vp, _vp, _vp, _int, _i64, _int, _int, _int, _vp]),
    "tl_gemm": (_int, [_vp, _vp, _vp, _i64, _i64, _i64, _i64, _int, _int, _int, _int, _int, _vp]),
    "tl_gemm_grouped": (_int, [_vp, _vp, _vp, _vp, _int, _i64, _i64, _i64, _i64, _int, _int, _int, _int, _int, _vp]),
    "tl_gemm_bf16": (_int, [_vp, _vp, _vp, _i64, _i64, _i64, _i64, _int, _int, _int, _int, _int, _vp]),
    "tl_gemm_grouped_bf16": (_int, [_vp, _vp, _vp, _vp, _int, _i64, _i64, _i64, _i64, _int, _int, _int, _int, _int, _vp]),
    "tl_gemm_grouped_swiglu": (_int, [_vp, _vp, _vp, _vp, _int, _i64, _i64, _i64, _i64, _int, _int, _int, _int, _int,
                                      _vp]),
    "tl_moe_ffn": (_int, [_vp, _vp, _vp, _vp, _vp, _vp, _int, _i64, _i64, _i64, _i64, _int, _int, _vp]),
    "tl_gemm_kmajor": (_int, [_vp, _vp, _vp, _i64, _i64, _i64, _i64, _int, _int, _int, _int, _int, _vp]),
    "tl_gemm_grouped_kmajor": (_int, [_vp, _vp, _vp, _vp, _int, _i64, _i64, _i64, _i64, _int, _int, _int, _int, _int,
                                      _vp]),
    "tl_gemm_fp8_kmajor": (_int, [_vp, _vp, _vp, _i64, _i64, _i64, _i64, _int, _int, _int, _int, _int, _vp]),
    "tl_gemm_grouped_fp8_kmajor": (_int, [_vp, _vp, _vp, _vp, _int, _i64, _i64, _i64, _i64, _int, _int, _int, _int,
                                          _int, _vp]),
    "tl_read_amp_async": (_int, [_i64, _i64, _i64, _int, _int, _int, _int, _i64, _int, _int, _int, _vp, _vp]),
    "tl_read_amp_batch": (_int, [_vp, _int, _vp, _vp]),
    "tl_read_amp_shared": (_int, [_i64, _i64, _i64, _int, _int, _int, _i64, _int, _i64, _int, _int, _int, _vp, _vp, _vp]),
    "tl_prefetch_degree": (_i64, [ctypes.c_double, ctypes.c_double, _i64, _i64, _i64, _i64, _i64, _i64, ctypes.c_double]),
    "tl_tile_arrival_latency": (_int, [_vp, _i64, _i64, ctypes.c_double, ctypes.POINTER(ctypes.c_double),
                                       ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double)]),
    "tl_hw_box_offsets": (_int, [_vp, _vp, _i64, _vp, _vp]),
    "tl_hw_box_load": (_int, [_vp, _vp, ctypes.c_uint64, _vp, _i64, _vp, _vp]),
    "tl_gemm_workspace_bytes": (_sz, [_i64, _i64, _i64, _int, _int, _int]),
    "tl_set_workspace": (_int, [_vp, _sz]),
    "tl_gemm_host": (_int, [_vp, _vp, _vp, _i64, _i64, _i64, _i64, _int, _int, _int, _int, _int, _vp, _sz, _vp]),
    "tl_gemm_host_scratch_bytes": (_sz, [_i64, _i64, _i64]),
    "tl_gemm_noalloc": (_int, [_vp, _vp, _vp, _i64, _i64, _i64, _i64, _int, _int, _int, _int, _int, _vp, _vp]),
    "tl_read_amp": (_int, [_i64, _i64, _i64, _int, _int, _int, _int, _i64, _int, _int, _int, _u64p, _u64p, _u64p]),
    "tl_read_amp_grouped": (_int, [_vp, _int, _i64, _i64, _int, _int, _int, _int, _i64, _int, _int, _int,
                                   _u64p, _u64p, _u64p]),
    "tl_read_amp_per_cta": (_int, [_i64, _i64, _i64, _int, _int, _int, _int, _i64, _int, _int, _int, _vp, _vp, _vp]),
}

# tl_option
(OPT_PDL, OPT_PREFETCH_STAGES, OPT_PAIR_KERNEL, OPT_PAIR_512, OPT_BOX_PER_BLOCK, OPT_MAX_STAGES, OPT_UMMA_M128,
 OPT_RELAYOUT_TMA, OPT_LOG, OPT_WAIT_LIMIT_US, OPT_STALL_ONCE, OPT_MOE_ROW_CAP, OPT_REDUCE_SPLIT, OPT_SM_LIMIT,
 OPT_NO_SCRATCH_PLANS, OPT_FFN_ONE_LAUNCH, OPT_GENERIC_RAW, OPT_PAIR_TMA_STORE, OPT_PLAN_AS_IF_SMS) = range(19)
FLAVOUR_N_BF16, FLAVOUR_K_BF16, FLAVOUR_K_FP8 = 0, 1, 2

_lib = None


class TileLensError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().tl_status_string(status).decode()
        extra = f" (cuda error {lib().tl_last_cuda_error()})" if status == 4 else ""
        super().__init__(f"{where}: {msg}{extra}")


def lib() -> ctypes.CDLL:
    """Loads libtilelens.so; raises if it has not been built (no CPU fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2607_04031_b200.build` "
                "(nvcc, sm_100a). The CUDA library is the only implementation of this path.")
        L = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(L, name)          # AttributeError if the library lacks a declared symbol
            fn.restype = res
            fn.argtypes = args
        _lib = L
    return _lib


def declared_symbols():
    return list(_SIGNATURES)


def _check(status: int, where: str):
    if status != TL_OK:
        raise TileLensError(status, where)


def _dev_ptr(t: torch.Tensor) -> int:
    if not t.is_cuda:
        raise ValueError("expected a CUDA tensor")
    if not t.is_contiguous():
        raise ValueError("expected a contiguous tensor")
    return t.data_ptr()


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream


def status_string(status: int) -> str:
    return lib().tl_status_string(status).decode()


def set_stream(stream=None):
    _check(lib().tl_set_stream(_stream_ptr(stream)), "tl_set_stream")


def device_status():
    """Synchronises; raises TileLensError(TL_ERR_TIMEOUT) if a kernel abandoned a bounded wait."""
    detail = ctypes.c_uint32(0)
    st = lib().tl_device_status(ctypes.byref(detail))
    if st != TL_OK:
        raise TileLensError(st, f"tl_device_status detail=0x{detail.value:x}")


def set_option(option: int, value: int):
    _check(lib().tl_set_option(option, value), "tl_set_option")


def get_option(option: int) -> int:
    return int(lib().tl_get_option(option))


class option:
    """with option(OPT_x, v): ... sets a library switch for the block and restores the previous value afterwards."""

    def __init__(self, opt: int, value: int):
        self.opt, self.value = opt, value

    def __enter__(self):
        self.old = get_option(self.opt)
        set_option(self.opt, self.value)
        return self

    def __exit__(self, *exc):
        set_option(self.opt, self.old)
        return False


class GemmPlan(ctypes.Structure):
    """tl_gemm_plan_info"""
    _fields_ = [("cta_m", ctypes.c_int32), ("cta_n", ctypes.c_int32), ("cta_k", ctypes.c_int32),
                ("pair_kernel", ctypes.c_int32), ("stream_k", ctypes.c_int32), ("grid", ctypes.c_int32),
                ("stages", ctypes.c_int32), ("weights_on_n", ctypes.c_int32), ("generic_path", ctypes.c_int32),
                ("cluster_k", ctypes.c_int32), ("pair_tiles_512", ctypes.c_int64), ("pair_tiles_256", ctypes.c_int64),
                ("chained", ctypes.c_int32), ("reserved", ctypes.c_int32),
                ("workspace_bytes", ctypes.c_uint64)]

    def as_dict(self):
        return {name: int(getattr(self, name)) for name, _ in self._fields_ if name != "reserved"}

    @property
    def cta(self):
        return (int(self.cta_m), int(self.cta_n), int(self.cta_k))


def gemm_plan(M: int, N: int, K: int, G: int = 4096, block_rows: int = 16, block_cols: int = 128, cta=(0, 0, 0),
              E: int = 0, flavour: int = FLAVOUR_N_BF16) -> GemmPlan:
    """The schedule a GEMM call with these sizes runs (host only, nothing is enqueued)."""
    out = GemmPlan()
    _check(lib().tl_gemm_plan(M, N, K, G, block_rows, block_cols, cta[0], cta[1], cta[2], E, flavour,
                              ctypes.addressof(out)), "tl_gemm_plan")
    return out


def gemm_last_plan() -> GemmPlan:
    """What this thread's most recent GEMM launch ran."""
    out = GemmPlan()
    _check(lib().tl_gemm_last_plan(ctypes.addressof(out)), "tl_gemm_last_plan")
    return out


def relayout(src: torch.Tensor, dst: torch.Tensor, rows: int, cols: int, elem_bytes: int, G: int,
             block_rows: int, block_cols: int, direction: int, stream=None):
    _check(lib().tl_relayout_on(_dev_ptr(src), _dev_ptr(dst), rows, cols, elem_bytes, G, block_rows, block_cols,
                                direction, _stream_ptr(stream)), "tl_relayout")


def relayout_batch(srcs, dsts, shapes, elem_bytes: int, G: int, block_rows: int, block_cols: int,
                   direction: int = TO_TILE_MAJOR, stream=None):
    """srcs, dsts: lists of CUDA tensors; shapes: list of (rows, cols).  One launch for the whole list where possible."""
    n = len(srcs)
    ptr_arr, i64_arr = ctypes.c_void_p * n, ctypes.c_int64 * n
    _check(lib().tl_relayout_batch(n, ptr_arr(*[_dev_ptr(t) for t in srcs]), ptr_arr(*[_dev_ptr(t) for t in dsts]),
                                   i64_arr(*[int(r) for r, _ in shapes]), i64_arr(*[int(c) for _, c in shapes]),
                                   elem_bytes, G, block_rows, block_cols, direction, _stream_ptr(stream)),
           "tl_relayout_batch")


def gemm(A: torch.Tensor, B: torch.Tensor, C: torch.Tensor, M: int, N: int, K: int, G: int = 4096,
         block_rows: int = 16, block_cols: int = 128, cta=(0, 0, 0), stream=None):
    """C (fp32 [M,N]) = A (bf16 [M,K]) x B (bf16, tile-major blocks; block_rows == 0: row-major [K,N])."""
    _check(lib().tl_gemm(_dev_ptr(A), _dev_ptr(B), _dev_ptr(C), M, N, K, G, block_rows, block_cols,
                         cta[0], cta[1], cta[2], _stream_ptr(stream)), "tl_gemm")


def gemm_grouped(A: torch.Tensor, B: torch.Tensor, C: torch.Tensor, offsets: torch.Tensor, E: int,
                 total_rows: int, N: int, K: int, G: int = 4096, block_rows: int = 16, block_cols: int = 128,
                 cta=(0, 0, 0), stream=None):
    _check(lib().tl_gemm_grouped(_dev_ptr(A), _dev_ptr(B), _dev_ptr(C), _dev_ptr(offsets), E, total_rows, N, K, G,
                                 block_rows, block_cols, cta[0], cta[1], cta[2], _stream_ptr(stream)),
           "tl_gemm_grouped")


def gemm_bf16(A: torch.Tensor, B: torch.Tensor, C_bf16: torch.Tensor, M: int, N: int, K: int, G: int = 4096,
              block_rows: int = 16, block_cols: int = 128, cta=(0, 0, 0), stream=None):
    """tl_gemm with a bf16 C."""
    _check(lib().tl_gemm_bf16(_dev_ptr(A), _dev_ptr(B), _dev_ptr(C_bf16), M, N, K, G, block_rows, block_cols,
                              cta[0], cta[1], cta[2], _stream_ptr(stream)), "tl_gemm_bf16")


def gemm_grouped_bf16(A: torch.Tensor, B: torch.Tensor, C_bf16: torch.Tensor, offsets: torch.Tensor, E: int,
                      total_rows: int, N: int, K: int, G: int = 4096, block_rows: int = 16, block_cols: int = 128,
                      cta=(0, 0, 0), stream=None):
    _check(lib().tl_gemm_grouped_bf16(_dev_ptr(A), _dev_ptr(B), _dev_ptr(C_bf16), _dev_ptr(offsets), E, total_rows, N, K,
                                      G, block_rows, block_cols, cta[0], cta[1], cta[2], _stream_ptr(stream)),
           "tl_gemm_grouped_bf16")


def gemm_grouped_swiglu(A: torch.Tensor, B_gate_up: torch.Tensor, H: torch.Tensor, offsets: torch.Tensor, E: int,
                        total_rows: int, N: int, K: int, G: int = 4096, block_rows: int = 16, block_cols: int = 128,
                        cta=(0, 0, 0), stream=None):
    """H (bf16 [rows, N/2]) = silu(gate) * up, gate/up = columns 2j / 2j+1 of A x B."""
    _check(lib().tl_gemm_grouped_swiglu(_dev_ptr(A), _dev_ptr(B_gate_up), _dev_ptr(H), _dev_ptr(offsets), E, total_rows,
                                        N, K, G, block_rows, block_cols, cta[0], cta[1], cta[2], _stream_ptr(stream)),
           "tl_gemm_grouped_swiglu")


def moe_ffn(X: torch.Tensor, W_gate_up: torch.Tensor, W_down: torch.Tensor, H: torch.Tensor, Y: torch.Tensor,
            offsets: torch.Tensor, E: int, total_rows: int, hidden: int, inter: int, G: int = 4096,
            block_rows: int = 16, block_cols: int = 128, stream=None):
    _check(lib().tl_moe_ffn(_dev_ptr(X), _dev_ptr(W_gate_up), _dev_ptr(W_down), _dev_ptr(H), _dev_ptr(Y),
                            _dev_ptr(offsets), E, total_rows, hidden, inter, G, block_rows, block_cols,
                            _stream_ptr(stream)), "tl_moe_ffn")


def gemm_kmajor(A: torch.Tensor, B_nk: torch.Tensor, C: torch.Tensor, M: int, N: int, K: int, G: int = 4096,
                tile_n: int = 32, tile_k: int = 64, cta=(0, 0, 0), stream=None):
    """Weights stored [N][K] (K contiguous), tile-major as Eq. 2 prints it; tile_n == 0: the plain [N][K] array."""
    _check(lib().tl_gemm_kmajor(_dev_ptr(A), _dev_ptr(B_nk), _dev_ptr(C), M, N, K, G, tile_n, tile_k,
                                cta[0], cta[1], cta[2], _stream_ptr(stream)), "tl_gemm_kmajor")


def gemm_grouped_kmajor(A: torch.Tensor, B_nk: torch.Tensor, C: torch.Tensor, offsets: torch.Tensor, E: int,
                        total_rows: int, N: int, K: int, G: int = 4096, tile_n: int = 32, tile_k: int = 64,
                        cta=(0, 0, 0), stream=None):
    _check(lib().tl_gemm_grouped_kmajor(_dev_ptr(A), _dev_ptr(B_nk), _dev_ptr(C), _dev_ptr(offsets), E, total_rows,
                                        N, K, G, tile_n, tile_k, cta[0], cta[1], cta[2], _stream_ptr(stream)),
           "tl_gemm_grouped_kmajor")


def gemm_fp8_kmajor(A: torch.Tensor, B_nk: torch.Tensor, C: torch.Tensor, M: int, N: int, K: int, G: int = 4096,
                    tile_n: int = 64, tile_k: int = 64, cta=(0, 0, 0), stream=None):
    """FP8 (E4M3) A [M,K] and weights [N,K] (tile-major tile_n x tile_k bytes, or plain when tile_n == 0); C fp32."""
    _check(lib().tl_gemm_fp8_kmajor(_dev_ptr(A), _dev_ptr(B_nk), _dev_ptr(C), M, N, K, G, tile_n, tile_k,
                                    cta[0], cta[1], cta[2], _stream_ptr(stream)), "tl_gemm_fp8_kmajor")


def gemm_grouped_fp8_kmajor(A: torch.Tensor, B_nk: torch.Tensor, C: torch.Tensor, offsets: torch.Tensor, E: int,
                            total_rows: int, N: int, K: int, G: int = 4096, tile_n: int = 64, tile_k: int = 64,
                            cta=(0, 0, 0), stream=None):
    _check(lib().tl_gemm_grouped_fp8_kmajor(_dev_ptr(A), _dev_ptr(B_nk), _dev_ptr(C), _dev_ptr(offsets), E, total_rows,
                                            N, K, G, tile_n, tile_k, cta[0], cta[1], cta[2], _stream_ptr(stream)),
           "tl_gemm_grouped_fp8_kmajor")


def gemm_workspace_bytes(M: int, N: int, K: int, cta=(0, 0, 0)) -> int:
    return int(lib().tl_gemm_workspace_bytes(M, N, K, cta[0], cta[1], cta[2]))


def set_workspace(buf: torch.Tensor | None):
    if buf is None:
        _check(lib().tl_set_workspace(None, 0), "tl_set_workspace")
    else:
        _check(lib().tl_set_workspace(_dev_ptr(buf), buf.numel() * buf.element_size()), "tl_set_workspace")


def gemm_host_scratch_bytes(M: int, N: int, K: int) -> int:
    return int(lib().tl_gemm_host_scratch_bytes(M, N, K))


def gemm_host(A_host: torch.Tensor, B_rowmajor_host: torch.Tensor, C_host: torch.Tensor, M: int, N: int, K: int,
              scratch: torch.Tensor, G: int = 4096, block_rows: int = 16, block_cols: int = 128, cta=(0, 0, 0),
              stream=None):
    """Host buffers in, host buffer out: H2D copies, relayout, GEMM and D2H copy all inside the call."""
    for t in (A_host, B_rowmajor_host, C_host):
        if t.is_cuda or not t.is_contiguous():
            raise ValueError("gemm_host takes contiguous host tensors")
    _check(lib().tl_gemm_host(A_host.data_ptr(), B_rowmajor_host.data_ptr(), C_host.data_ptr(), M, N, K, G,
                              block_rows, block_cols, cta[0], cta[1], cta[2], _dev_ptr(scratch),
                              scratch.numel() * scratch.element_size(), _stream_ptr(stream)), "tl_gemm_host")


def gemm_noalloc(A: torch.Tensor, B: torch.Tensor, C: torch.Tensor, M: int, N: int, K: int, G: int = 4096,
                 block_rows: int = 16, block_cols: int = 128, cta=(0, 0, 0), timeout_flag: torch.Tensor | None = None,
                 stream=None):
    """tl_gemm for processes that may not allocate device memory: split-K scratch is a fixed array
    inside the library (8 MiB per GPU).  `timeout_flag`: optional zeroed uint32/int32 CUDA tensor."""
    flag = _dev_ptr(timeout_flag) if timeout_flag is not None else None
    _check(lib().tl_gemm_noalloc(_dev_ptr(A), _dev_ptr(B), _dev_ptr(C), M, N, K, G, block_rows, block_cols,
                                 cta[0], cta[1], cta[2], flag, _stream_ptr(stream)), "tl_gemm_noalloc")


class HwDesc(ctypes.Structure):
    """tl_hw_desc: a tensor view of the column-major K x N matrix plus the memory tile (a, b) and the leading stride."""
    _fields_ = [("rank", ctypes.c_int32), ("elem_bytes", ctypes.c_int32), ("dims", ctypes.c_int64 * 5),
                ("strides", ctypes.c_int64 * 5), ("box", ctypes.c_int32 * 5), ("tile_a", ctypes.c_int32),
                ("tile_b", ctypes.c_int32), ("leading_stride", ctypes.c_int64)]


def hw_desc(dims, strides, box, elem_bytes: int, tile_a: int, tile_b: int, leading_stride: int) -> HwDesc:
    d = HwDesc()
    d.rank, d.elem_bytes, d.tile_a, d.tile_b, d.leading_stride = len(dims), elem_bytes, tile_a, tile_b, leading_stride
    for k in range(min(len(dims), 5)):
        d.dims[k], d.strides[k], d.box[k] = dims[k], strides[k], box[k]
    return d


def hw_box_offsets(desc: HwDesc, coords: torch.Tensor, offsets: torch.Tensor, stream=None):
    """coords: int32 CUDA tensor [n_boxes, rank]; offsets: uint64/int64 CUDA tensor [n_boxes * prod(box)]."""
    _check(lib().tl_hw_box_offsets(ctypes.addressof(desc), _dev_ptr(coords), coords.shape[0], _dev_ptr(offsets),
                                   _stream_ptr(stream)), "tl_hw_box_offsets")


def hw_box_load(desc: HwDesc, src: torch.Tensor, coords: torch.Tensor, dst: torch.Tensor, stream=None):
    """src: the tile-major buffer; dst: n_boxes dense boxes."""
    _check(lib().tl_hw_box_load(ctypes.addressof(desc), _dev_ptr(src), src.numel() * src.element_size(),
                                _dev_ptr(coords), coords.shape[0], _dev_ptr(dst), _stream_ptr(stream)),
           "tl_hw_box_load")


def read_amp(M: int, N: int, K: int, cta, layout: int, G: int, block_rows: int = 0, block_cols: int = 0,
             elem_bytes: int = 2):
    """Returns (bytes_fetched, bytes_used, requests), exact integers."""
    f, u, q = ctypes.c_uint64(), ctypes.c_uint64(), ctypes.c_uint64()
    _check(lib().tl_read_amp(M, N, K, cta[0], cta[1], cta[2], layout, G, block_rows, block_cols, elem_bytes,
                             ctypes.byref(f), ctypes.byref(u), ctypes.byref(q)), "tl_read_amp")
    return int(f.value), int(u.value), int(q.value)


def read_amp_async(M: int, N: int, K: int, cta, layout: int, G: int, block_rows: int, block_cols: int, elem_bytes: int,
                   totals: torch.Tensor, stream=None):
    """totals: CUDA tensor of 3 int64/uint64 that receives (bytes_fetched, bytes_used, requests); no wait."""
    _check(lib().tl_read_amp_async(M, N, K, cta[0], cta[1], cta[2], layout, G, block_rows, block_cols, elem_bytes,
                                   _dev_ptr(totals), _stream_ptr(stream)), "tl_read_amp_async")


class ReadAmpCfg(ctypes.Structure):
    """tl_read_amp_cfg"""
    _fields_ = [("M", ctypes.c_int64), ("N", ctypes.c_int64), ("K", ctypes.c_int64), ("cta_m", ctypes.c_int32),
                ("cta_n", ctypes.c_int32), ("cta_k", ctypes.c_int32), ("layout", ctypes.c_int32), ("G", ctypes.c_int64),
                ("block_rows", ctypes.c_int32), ("block_cols", ctypes.c_int32), ("elem_bytes", ctypes.c_int32),
                ("reserved", ctypes.c_int32)]


def read_amp_cfgs(cfgs):
    """cfgs: iterable of (M, N, K, cta, layout, G, block_rows, block_cols, elem_bytes) -> ctypes array for read_amp_batch."""
    cfgs = list(cfgs)
    arr = (ReadAmpCfg * len(cfgs))()
    for a, (M, N, K, cta, layout, G, br, bc, s) in zip(arr, cfgs):
        a.M, a.N, a.K, a.cta_m, a.cta_n, a.cta_k, a.layout, a.G = M, N, K, cta[0], cta[1], cta[2], layout, G
        a.block_rows, a.block_cols, a.elem_bytes = br, bc, s
    return arr


def read_amp_batch(cfg_array, totals: torch.Tensor, stream=None):
    """One launch for up to 16 configurations; totals: CUDA int64/uint64 tensor [n, 3]; no wait."""
    _check(lib().tl_read_amp_batch(ctypes.addressof(cfg_array), len(cfg_array), _dev_ptr(totals), _stream_ptr(stream)),
           "tl_read_amp_batch")


def read_amp_shared(M: int, N: int, K: int, cta, wave_ctas: int, layout: int, G: int, block_rows: int = 0,
                    block_cols: int = 0, elem_bytes: int = 2):
    """(bytes_fetched, bytes_needed, requests) when the wave_ctas co-resident CTA tiles share blocks per K step."""
    f, u, q = ctypes.c_uint64(), ctypes.c_uint64(), ctypes.c_uint64()
    _check(lib().tl_read_amp_shared(M, N, K, cta[0], cta[1], cta[2], wave_ctas, layout, G, block_rows, block_cols,
                                    elem_bytes, ctypes.byref(f), ctypes.byref(u), ctypes.byref(q)), "tl_read_amp_shared")
    return int(f.value), int(u.value), int(q.value)


def prefetch_degree(bandwidth_bytes_per_s: float, latency_s: float, G: int, n_sm: int, ctas_per_sm: int,
                    requests_per_tile: int, K: int, cta_k: int, collision_factor: float = 1.0) -> int:
    d = int(lib().tl_prefetch_degree(bandwidth_bytes_per_s, latency_s, G, n_sm, ctas_per_sm, requests_per_tile, K,
                                     cta_k, collision_factor))
    if d < 0:
        raise ValueError("tl_prefetch_degree: bad arguments")
    return d


def tile_arrival_latency(latencies, requests: int, threshold: float = 0.0):
    """(E[first arrival], E[last arrival], P(last arrival > threshold)) for `requests` requests per tile whose
    latencies are independent draws from the sample `latencies` (host arithmetic, Section 6.5)."""
    import numpy as np
    x = np.ascontiguousarray(latencies, dtype=np.float64)
    first, last, late = ctypes.c_double(), ctypes.c_double(), ctypes.c_double()
    _check(lib().tl_tile_arrival_latency(x.ctypes.data, x.size, requests, threshold, ctypes.byref(first),
                                         ctypes.byref(last), ctypes.byref(late)), "tl_tile_arrival_latency")
    return first.value, last.value, late.value


def read_amp_grouped(offsets_host, N: int, K: int, cta, layout: int, G: int, block_rows: int = 0,
                     block_cols: int = 0, elem_bytes: int = 2):
    import numpy as np
    offs = np.ascontiguousarray(offsets_host, dtype=np.int32)
    f, u, q = ctypes.c_uint64(), ctypes.c_uint64(), ctypes.c_uint64()
    _check(lib().tl_read_amp_grouped(offs.ctypes.data, offs.size - 1, N, K, cta[0], cta[1], cta[2], layout, G,
                                     block_rows, block_cols, elem_bytes, ctypes.byref(f), ctypes.byref(u),
                                     ctypes.byref(q)), "tl_read_amp_grouped")
    return int(f.value), int(u.value), int(q.value)


def read_amp_per_cta(M: int, N: int, K: int, cta, layout: int, G: int, block_rows: int, block_cols: int,
                     elem_bytes: int, fetched: torch.Tensor, used: torch.Tensor, stream=None):
    _check(lib().tl_read_amp_per_cta(M, N, K, cta[0], cta[1], cta[2], layout, G, block_rows, block_cols, elem_bytes,
                                     _dev_ptr(fetched), _dev_ptr(used), _stream_ptr(stream)), "tl_read_amp_per_cta")
