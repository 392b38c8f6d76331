"""The C-ABI boundary without a GPU: libhif4.so loads, exports every function that include/hif4.h
declares (and the Python binding lists the same names), and its host-only entry points answer as the
header says.  No kernel is launched here."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "hif4.h")


def declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    text = re.sub(r"typedef\s+enum\s*\{.*?\}\s*\w+\s*;", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(hif4_\w+)\s*\(", text)))


@pytest.fixture(scope="module")
def cdll():
    import importlib.util
    spec = importlib.util.spec_from_file_location("_hif4_build", os.path.join(ROOT, "paper_2602_11287_b200", "build.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return ctypes.CDLL(mod.build())


def test_header_declares_the_calls_of_the_hot_path():
    names = declared_functions()
    for must in ("hif4_quantize", "hif4_dequantize", "hif4_gemm", "hif4_grouped_gemm", "hif4_packed_bytes",
                 "hif4_gemm_workspace", "hif4_grouped_gemm_workspace", "hif4_last_device_status", "hif4_status_string"):
        assert must in names


def test_library_exports_every_declared_symbol(cdll):
    for name in declared_functions():
        assert hasattr(cdll, name), f"libhif4.so does not export {name}"


def test_binding_lists_the_same_names():
    import paper_2602_11287_b200 as hif4
    assert sorted(hif4.EXPORTED_SYMBOLS) == declared_functions()


def test_host_only_entry_points(cdll):
    i64, sz = ctypes.c_int64, ctypes.c_size_t
    cdll.hif4_packed_bytes.restype = sz
    cdll.hif4_packed_bytes.argtypes = [i64, i64]
    assert cdll.hif4_packed_bytes(3, 128) == 3 * 2 * 36            # 288 bits per 64 values (Section II-A)
    assert cdll.hif4_packed_bytes(1, 64) * 8 == 288
    assert cdll.hif4_packed_bytes(3, 100) == 0 and cdll.hif4_packed_bytes(-1, 64) == 0
    cdll.hif4_status_string.restype = ctypes.c_char_p
    seen = {cdll.hif4_status_string(c) for c in range(9)}
    assert len(seen) == 9 and all(s for s in seen)
    n = sz(123)
    cdll.hif4_gemm_workspace.argtypes = [i64, i64, i64, ctypes.POINTER(sz)]
    assert cdll.hif4_gemm_workspace(16, 16, 128, ctypes.byref(n)) == 0
    assert cdll.hif4_gemm_workspace(16, 16, 100, ctypes.byref(n)) == 2          # K % 64
    assert cdll.hif4_gemm_workspace(16, 16, 128, None) == 1
    cdll.hif4_grouped_gemm_workspace.argtypes = [ctypes.c_int, i64, i64, i64, ctypes.POINTER(sz)]
    assert cdll.hif4_grouped_gemm_workspace(4, 1000, 256, 512, ctypes.byref(n)) == 0
    assert n.value >= (1000 // 128 + 4) * 16 and n.value % 256 == 0
    assert cdll.hif4_grouped_gemm_workspace(-1, 10, 64, 64, ctypes.byref(n)) == 2


def test_gemm_workspace_follows_the_kernel_choice_and_tile_schedule(cdll):
    """hif4_gemm_workspace is host logic: it picks the kernel by M and plans the tile schedule.  Sizes worked out
    by hand for 148 SMs = 74 CTA pairs (what the library assumes without a device, and what a B200 has)."""
    i64, sz = ctypes.c_int64, ctypes.c_size_t
    cdll.hif4_gemm_workspace.argtypes = [i64, i64, i64, ctypes.POINTER(sz)]
    n = sz(0)
    want = {
        # M <= 32: decoded activation rows, 2 bytes x K x (8, 16 or 32 rows)
        (1, 4096, 4096): 2 * 4096 * 8, (16, 14336, 4096): 2 * 4096 * 16, (32, 4096, 14336): 2 * 14336 * 32,
        # 33..128 rows: 56 weight tiles on 74 pairs are not sliced; 16 tiles x 4 K slices x 8 completion words
        (64, 14336, 4096): 0, (128, 4096, 14336): 16 * 4 * 8 * 4,
        # pair kernel, several rounds with a partial one: (74 + 1) flag rows x 2 x 8 words, rounded up to 256 bytes
        (4096, 14336, 4096): 4864, (4096, 4096, 4096): 4864,
        # a whole number of rounds, or one round that is not worth slicing: nothing
        (256 * 74, 256, 1024): 0, (4096, 1024, 4096): 0, (4096, 4096, 192): 0,
        # one round of 32 tiles x 2 slices, of 8 tiles x 4 slices
        (2048, 1024, 8192): 32 * 2 * 8 * 4, (1024, 512, 16384): 8 * 4 * 8 * 4,
    }
    for (M, N, K), bytes_ in want.items():
        assert cdll.hif4_gemm_workspace(M, N, K, ctypes.byref(n)) == 0
        assert n.value == bytes_, (M, N, K, n.value, bytes_)


def test_argument_errors_are_found_before_any_launch(cdll):
    """Shape / dtype / null checks come before the first CUDA call, so they answer without a GPU."""
    i64, vp, ci = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int
    cdll.hif4_quantize.argtypes = [vp, ci, i64, i64, i64, vp, ci, vp]
    cdll.hif4_debug_launch_count.restype = ctypes.c_uint64
    before = cdll.hif4_debug_launch_count()
    assert cdll.hif4_quantize(None, 0, 4, 100, 100, None, 0, None) == 2     # cols % 64
    assert cdll.hif4_quantize(None, 5, 4, 128, 128, None, 0, None) == 4     # dtype
    assert cdll.hif4_quantize(None, 0, 4, 128, 128, None, 9, None) == 4     # rounding mode
    assert cdll.hif4_quantize(None, 0, 4, 128, 64, None, 0, None) == 2      # ld < cols
    assert cdll.hif4_quantize(None, 0, 4, 128, 128, None, 0, None) == 1     # null
    assert cdll.hif4_quantize(None, 0, 0, 128, 128, None, 0, None) == 0     # empty: no-op
    cdll.hif4_gemm.argtypes = [vp, vp, vp, i64, i64, i64, i64, vp, ctypes.c_size_t, vp]
    assert cdll.hif4_gemm(None, None, None, 4, 4, 100, 4, None, 0, None) == 2
    assert cdll.hif4_gemm(None, None, None, 0, 4, 64, 4, None, 0, None) == 0
    assert cdll.hif4_debug_launch_count() == before


def test_launch_count_helper_of_the_tests_states_the_limits_of_the_source():
    """tests/kernel_choice.py restates, for the launch-count expectations of the GPU tests, when the weight-streaming
    kernel builds its tokens itself; its numbers must be the ones compiled into the library."""
    import re
    from tests.kernel_choice import tokens_stay_in_shared_memory
    src = open(os.path.join(ROOT, "paper_2602_11287_b200", "csrc", "hif4_gemv.cu")).read()
    units = int(re.search(r"kResidentMaxElemsUnits = (\d+)", src).group(1))
    bf16 = int(re.search(r"kResidentMaxElemsBf16 = (\d+)", src).group(1))
    max_bytes = int(re.search(r"kResidentMaxBytes = (\d+) \* 1024", src).group(1)) * 1024
    assert min(units, bf16) * 2 <= max_bytes
    for (M, rows) in ((1, 1), (2, 2), (3, 4), (4, 4), (5, 8), (8, 8), (9, 16), (16, 16)):
        for limit, from_bf16 in ((units, False), (bf16, True)):
            k_fit = limit // rows // 256 * 256
            if k_fit * rows * 2 <= max_bytes:
                assert tokens_stay_in_shared_memory(M, k_fit, from_bf16) and not tokens_stay_in_shared_memory(M, k_fit + 256, from_bf16)
    assert not tokens_stay_in_shared_memory(17, 256)
