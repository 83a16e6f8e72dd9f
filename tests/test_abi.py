"""The C-ABI library loads without a GPU and exports every symbol the header declares (CPU only).

Only argument checks that return before any CUDA call are exercised here; no kernel runs.
"""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def tl():
    from paper_2607_04031_b200 import build
    build.build()
    from paper_2607_04031_b200 import binding
    return binding


def _declared_in_header():
    text = open(os.path.join(ROOT, "include", "tilelens.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(tl_[a-z_0-9]+)\s*\(", text)))


def test_header_symbols_are_exported_and_bound(tl):
    declared = _declared_in_header()
    assert "tl_relayout" in declared and "tl_gemm" in declared and "tl_read_amp" in declared
    raw = ctypes.CDLL(tl.LIB_PATH)
    for name in declared:
        assert hasattr(raw, name), f"{name} declared in tilelens.h but not exported"
    assert sorted(tl.declared_symbols()) == declared
    tl.lib()            # sets restype/argtypes for every symbol; raises if one is missing


def test_status_strings(tl):
    assert tl.status_string(0) == "TL_OK"
    for code in range(1, 7):
        assert tl.status_string(code).startswith("TL_ERR_")
    assert "unknown" in tl.status_string(99)


def test_relayout_argument_checks_need_no_device(tl):
    L = tl.lib()
    bogus_a, bogus_b = ctypes.c_void_p(0x10000), ctypes.c_void_p(0x90000)
    # G must equal block_rows * block_cols * elem_bytes
    assert L.tl_relayout(bogus_a, bogus_b, 64, 64, 2, 4096, 16, 64, 0) == 1
    # element sizes other than 1, 2, 4
    assert L.tl_relayout(bogus_a, bogus_b, 64, 64, 3, 16 * 64 * 3, 16, 64, 0) == 1
    # matrix not divisible by the memory tile
    assert L.tl_relayout(bogus_a, bogus_b, 60, 64, 2, 2048, 16, 64, 0) == 1
    # non-power-of-two memory tile
    assert L.tl_relayout(bogus_a, bogus_b, 48, 48, 2, 12 * 12 * 2, 12, 12, 0) == 2
    # bad direction
    assert L.tl_relayout(bogus_a, bogus_b, 64, 64, 2, 2048, 16, 64, 7) == 1
    # empty matrix: nothing to do
    assert L.tl_relayout(None, None, 0, 64, 2, 2048, 16, 64, 0) == 0
    # overlapping buffers
    assert L.tl_relayout(bogus_a, ctypes.c_void_p(0x10100), 64, 64, 2, 2048, 16, 64, 0) == 1


def test_relayout_batch_argument_checks_need_no_device(tl):
    L = tl.lib()
    P2, I2 = ctypes.c_void_p * 2, ctypes.c_int64 * 2
    srcs, dsts = P2(0x10000, 0x200000), P2(0x90000, 0x300000)
    # nothing to do; negative count; missing arrays
    assert L.tl_relayout_batch(0, None, None, None, None, 2, 4096, 16, 128, 0, None) == 0
    assert L.tl_relayout_batch(-1, srcs, dsts, I2(64, 64), I2(128, 128), 2, 4096, 16, 128, 0, None) == 1
    assert L.tl_relayout_batch(2, None, dsts, I2(64, 64), I2(128, 128), 2, 4096, 16, 128, 0, None) == 1
    # the first bad matrix ends the call with tl_relayout's own error: G mismatch, indivisible rows, odd tile
    assert L.tl_relayout_batch(2, srcs, dsts, I2(64, 64), I2(128, 128), 2, 2048, 16, 128, 0, None) == 1
    assert L.tl_relayout_batch(2, srcs, dsts, I2(60, 64), I2(128, 128), 2, 4096, 16, 128, 0, None) == 1
    assert L.tl_relayout_batch(2, srcs, dsts, I2(48, 48), I2(48, 48), 2, 12 * 12 * 2, 12, 12, 0, None) == 2
    # empty matrices are skipped one by one
    assert L.tl_relayout_batch(2, srcs, dsts, I2(0, 0), I2(128, 128), 2, 4096, 16, 128, 0, None) == 0


def test_read_amp_argument_checks_need_no_device(tl):
    L = tl.lib()
    f, u = ctypes.c_uint64(), ctypes.c_uint64()
    args = lambda **kw: [kw.get("M", 16), kw.get("N", 512), kw.get("K", 512), 64, 64, 64, kw.get("layout", 2),
                         kw.get("G", 4096), kw.get("br", 16), kw.get("bc", 128), kw.get("s", 2),
                         ctypes.byref(f), ctypes.byref(u), None]
    assert L.tl_read_amp(*args(G=2048)) == 1                 # G != br*bc*s
    assert L.tl_read_amp(*args(N=500)) == 1                  # N % bc
    assert L.tl_read_amp(*args(layout=5)) == 1
    assert L.tl_read_amp(*args(s=3)) == 1
    assert L.tl_read_amp(*args(M=-1)) == 1


def test_gemm_argument_checks_need_no_device(tl):
    L = tl.lib()
    p = ctypes.c_void_p(0x10000)
    call = lambda M=16, N=512, K=512, G=4096, br=16, bc=128, A=p, B=p, C=p: L.tl_gemm(
        A, B, C, M, N, K, G, br, bc, 0, 0, 0, None)
    assert call(M=0) == 0                                    # no rows: no-op
    assert call(M=-1) == 1
    assert call(A=None) == 1
    assert call(G=2048) == 1                                 # G != br*bc*2
    assert call(K=520) == 1                                  # K % br
    assert call(br=12, bc=128, G=12 * 128 * 2) == 2          # not a power of two
    assert call(br=256, bc=8) == 2                           # hand-addressed tiles (rows under 32 bytes) must fit inside the CTA tile
    assert call(B=ctypes.c_void_p(0x10010)) == 3             # tile-major operand must be 128-byte aligned
    assert L.tl_gemm_host_scratch_bytes(16, 512, 512) >= 16 * 512 * 2 + 2 * 512 * 512 * 2 + 16 * 512 * 4


def test_output_rows_must_hold_whole_16_byte_vectors(tl):
    # fp32 C is written in 16-byte vectors; the hand-addressed memory tiles of one or two columns would otherwise
    # admit an N that is not a multiple of four
    L = tl.lib()
    p = ctypes.c_void_p(0x10000)
    assert L.tl_gemm(p, p, p, 16, 1022, 512, 64, 16, 2, 0, 0, 0, None) == 2
    assert L.tl_gemm(p, p, p, 16, 1021, 512, 32, 16, 1, 0, 0, 0, None) == 2
    assert L.tl_gemm_kmajor(p, p, p, 16, 1022, 512, 4096, 2, 1024, 0, 0, 0, None) == 2


def test_noalloc_argument_checks_need_no_device(tl):
    L = tl.lib()
    p = ctypes.c_void_p(0x10000)
    call = lambda M=16, N=512, K=512, A=p, B=p, C=p: L.tl_gemm_noalloc(A, B, C, M, N, K, 4096, 16, 128, 0, 0, 0, None, None)
    assert call(M=0) == 0
    assert call(M=-1) == 1
    assert call(N=0) == 1


def test_options_and_plan_argument_checks(tl):
    L = tl.lib()
    assert L.tl_set_option(99, 0) == 1 and L.tl_get_option(99) == -1
    assert L.tl_set_option(tl.OPT_PDL, 7) == 1
    old = tl.get_option(tl.OPT_MAX_STAGES)
    with tl.option(tl.OPT_MAX_STAGES, 3):
        assert tl.get_option(tl.OPT_MAX_STAGES) == 3
    assert tl.get_option(tl.OPT_MAX_STAGES) == old
    out = tl.GemmPlan()
    assert L.tl_gemm_plan(16, 512, 512, 4096, 16, 128, 0, 0, 0, 0, 0, None) == 1          # no result buffer
    assert L.tl_gemm_plan(16, 512, 512, 4096, 16, 128, 0, 0, 0, 0, 5, ctypes.addressof(out)) == 1
    assert L.tl_gemm_plan(16, 512, 512, 2048, 16, 128, 0, 0, 0, 0, 0, ctypes.addressof(out)) == 1     # G mismatch
    assert L.tl_gemm_plan(16, 1022, 512, 64, 16, 2, 0, 0, 0, 0, 0, ctypes.addressof(out)) == 2       # N % 4
    assert L.tl_gemm_last_plan(None) == 1


def test_host_threads_may_call_concurrently(tl):
    # Argument-check paths only (no device here): two threads hammer the entry points, each with its own stream and
    # workspace settings; every call must return the code the single-threaded call returns.
    import threading
    L = tl.lib()
    p = ctypes.c_void_p(0x10000)
    bad = []

    def worker(k):
        L.tl_set_stream(ctypes.c_void_p(0x1000 * (k + 1)))
        L.tl_set_workspace(ctypes.c_void_p(0x100000 * (k + 1)), 1 << 20)
        for i in range(3000):
            if L.tl_gemm(p, p, p, -1, 512, 512, 4096, 16, 128, 0, 0, 0, None) != 1: bad.append(("gemm", k, i))
            if L.tl_relayout(p, ctypes.c_void_p(0x90000), 60, 64, 2, 2048, 16, 64, 0) != 1: bad.append(("relayout", k, i))
            if L.tl_set_option(tl.OPT_MAX_STAGES, 2 + (i + k) % 3) != 0: bad.append(("opt", k, i))
            if not 2 <= L.tl_get_option(tl.OPT_MAX_STAGES) <= 4: bad.append(("get", k, i))
            if L.tl_set_workspace(ctypes.c_void_p(0x100000 * (k + 1) + 8), 64) != 3: bad.append(("ws", k, i))
        L.tl_set_workspace(None, 0)
        L.tl_set_stream(None)

    threads = [threading.Thread(target=worker, args=(k,)) for k in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    L.tl_set_option(tl.OPT_MAX_STAGES, 0)
    assert not bad, bad[:5]


def test_binding_refuses_to_run_without_the_library(tl, monkeypatch):
    monkeypatch.setattr(tl, "_lib", None)
    monkeypatch.setattr(tl, "LIB_PATH", os.path.join(ROOT, "does_not_exist.so"))
    with pytest.raises(RuntimeError, match="missing"):
        tl.lib()
