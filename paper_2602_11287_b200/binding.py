"""Thin ctypes binding of libhif4.so: argument marshalling only.

Every step of the path runs in the CUDA kernels behind the C ABI declared in ``include/hif4.h``;
PyTorch supplies device memory and the current stream.  There is no CPU fallback: if the library has
not been built, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libhif4.so")

UNIT_ELEMS, UNIT_BYTES = 64, 36
HIF4_BF16, HIF4_FP32, HIF4_FP16 = 0, 1, 2
HIF4_RNE, HIF4_RHA = 0, 1
HIF4_FMT_HIF4, HIF4_FMT_MXFP4, HIF4_FMT_NVFP4, HIF4_FMT_NVFP4_PTS = 0, 1, 2, 3
HIF4_OK = 0

EXPORTED_SYMBOLS = [
    "hif4_packed_bytes", "hif4_quantize", "hif4_dequantize", "hif4_gemm_workspace", "hif4_gemm",
    "hif4_grouped_gemm_workspace", "hif4_grouped_gemm", "hif4_last_device_status", "hif4_status_string",
    "hif4_debug_launch_count", "hif4_debug_set_gemm_path", "hif4_grouped_gemm_noalloc", "hif4_grouped_gemm_noalloc_capacity",
    "hif4_linear", "hif4_linear_workspace", "hif4_quantize_transposed", "hif4_debug_wait_timeout",
    "hif4_mse_workspace", "hif4_mse_roundtrip",
]


class Hif4Error(RuntimeError):
    def __init__(self, call: str, code: int):
        self.code = code
        super().__init__(f"{call} failed: {status_string(code)} (status {code})")


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2602_11287_b200.build` "
            "(there is no CPU fallback)")
    L = ctypes.CDLL(LIB_PATH)
    i64, vp, ci, sz = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    L.hif4_packed_bytes.restype = sz
    L.hif4_packed_bytes.argtypes = [i64, i64]
    L.hif4_quantize.restype = ci
    L.hif4_quantize.argtypes = [vp, ci, i64, i64, i64, vp, ci, vp]
    L.hif4_quantize_transposed.restype = ci
    L.hif4_quantize_transposed.argtypes = [vp, ci, i64, i64, i64, vp, ci, vp]
    L.hif4_dequantize.restype = ci
    L.hif4_dequantize.argtypes = [vp, i64, i64, vp, ci, i64, vp]
    L.hif4_gemm_workspace.restype = ci
    L.hif4_gemm_workspace.argtypes = [i64, i64, i64, ctypes.POINTER(sz)]
    L.hif4_gemm.restype = ci
    L.hif4_gemm.argtypes = [vp, vp, vp, i64, i64, i64, i64, vp, sz, vp]
    L.hif4_grouped_gemm_workspace.restype = ci
    L.hif4_grouped_gemm_workspace.argtypes = [ci, i64, i64, i64, ctypes.POINTER(sz)]
    L.hif4_grouped_gemm.restype = ci
    L.hif4_grouped_gemm.argtypes = [vp, vp, vp, vp, ci, i64, i64, i64, i64, vp, sz, vp]
    L.hif4_grouped_gemm_noalloc.restype = ci
    L.hif4_grouped_gemm_noalloc.argtypes = [vp, vp, vp, vp, ci, i64, i64, i64, i64, vp]
    L.hif4_grouped_gemm_noalloc_capacity.restype = sz
    L.hif4_grouped_gemm_noalloc_capacity.argtypes = []
    L.hif4_linear_workspace.restype = ci
    L.hif4_linear_workspace.argtypes = [i64, i64, i64, ctypes.POINTER(sz)]
    L.hif4_linear.restype = ci
    L.hif4_linear.argtypes = [vp, ci, i64, vp, vp, i64, i64, i64, i64, ci, vp, sz, vp]
    L.hif4_mse_workspace.restype = ci
    L.hif4_mse_workspace.argtypes = [i64, ci, ctypes.POINTER(sz)]
    L.hif4_mse_roundtrip.restype = ci
    L.hif4_mse_roundtrip.argtypes = [vp, i64, ci, vp, vp, vp, sz, vp]
    L.hif4_last_device_status.restype = ci
    L.hif4_last_device_status.argtypes = [vp]
    L.hif4_status_string.restype = ctypes.c_char_p
    L.hif4_status_string.argtypes = [ci]
    L.hif4_debug_set_gemm_path.restype = ci
    L.hif4_debug_set_gemm_path.argtypes = [ci]
    L.hif4_debug_launch_count.restype = ctypes.c_uint64
    L.hif4_debug_launch_count.argtypes = []
    L.hif4_debug_wait_timeout.restype = ci
    L.hif4_debug_wait_timeout.argtypes = [ctypes.c_uint64, vp]
    return L


lib = _load()


def status_string(code: int) -> str:
    return lib.hif4_status_string(int(code)).decode()


def _check(call: str, code: int) -> None:
    if code != HIF4_OK:
        raise Hif4Error(call, code)


def _stream(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _dtype_code(dt: torch.dtype) -> int:
    if dt == torch.bfloat16:
        return HIF4_BF16
    if dt == torch.float32:
        return HIF4_FP32
    if dt == torch.float16:
        return HIF4_FP16                                  # source type only: the library rejects it as a destination
    raise TypeError(f"HiF4 conversion takes bfloat16, float32 or (as a source) float16, not {dt}")


def _need_cuda(*tensors: torch.Tensor) -> None:
    for t in tensors:
        if t is not None and not t.is_cuda:
            raise ValueError("the HiF4 library takes device tensors only (no CPU path exists)")


def launch_count() -> int:
    return int(lib.hif4_debug_launch_count())


def hif4_packed_bytes(rows: int, cols: int) -> int:
    return int(lib.hif4_packed_bytes(rows, cols))


def hif4_quantize(src: torch.Tensor, mode: int = HIF4_RNE, out: Optional[torch.Tensor] = None,
                  stream=None) -> torch.Tensor:
    """[rows, cols] BF16/FP32 (row stride = src.stride(0)) -> uint8 units [rows, cols // 64, 36]."""
    _need_cuda(src, out)
    assert src.dim() == 2 and src.stride(1) == 1
    rows, cols = src.shape
    if out is None:
        out = torch.empty((rows, cols // UNIT_ELEMS if cols % UNIT_ELEMS == 0 else 0, UNIT_BYTES),
                          dtype=torch.uint8, device=src.device)
    ld = src.stride(0) if rows > 1 else max(cols, src.stride(0))
    _check("hif4_quantize", lib.hif4_quantize(src.data_ptr(), _dtype_code(src.dtype), rows, cols, ld,
                                              out.data_ptr(), mode, _stream(stream)))
    return out


def hif4_quantize_transposed(src: torch.Tensor, mode: int = HIF4_RNE, out: Optional[torch.Tensor] = None,
                             stream=None) -> torch.Tensor:
    """[rows, cols] BF16 / FP32 / FP16 -> uint8 units [cols, rows // 64, 36]: the units of src.T without transposing."""
    _need_cuda(src, out)
    assert src.dim() == 2 and src.stride(1) == 1
    rows, cols = src.shape
    if out is None:
        out = torch.empty((cols, rows // UNIT_ELEMS if rows % UNIT_ELEMS == 0 else 0, UNIT_BYTES),
                          dtype=torch.uint8, device=src.device)
    ld = src.stride(0) if rows > 1 else max(cols, src.stride(0))
    _check("hif4_quantize_transposed", lib.hif4_quantize_transposed(src.data_ptr(), _dtype_code(src.dtype), rows, cols, ld,
                                                                    out.data_ptr(), mode, _stream(stream)))
    return out


def hif4_dequantize(units: torch.Tensor, dtype: torch.dtype = torch.bfloat16, out: Optional[torch.Tensor] = None,
                    stream=None) -> torch.Tensor:
    """uint8 units [rows, upr, 36] -> [rows, upr * 64] of `dtype` (Eq. 2)."""
    _need_cuda(units, out)
    assert units.dtype == torch.uint8 and units.dim() == 3 and units.shape[2] == UNIT_BYTES and units.is_contiguous()
    rows, upr, _ = units.shape
    cols = upr * UNIT_ELEMS
    if out is None:
        out = torch.empty((rows, cols), dtype=dtype, device=units.device)
    assert out.stride(1) == 1
    ld = out.stride(0) if rows > 1 else max(cols, out.stride(0))
    _check("hif4_dequantize", lib.hif4_dequantize(units.data_ptr(), rows, cols, out.data_ptr(),
                                                  _dtype_code(out.dtype), ld, _stream(stream)))
    return out


def hif4_gemm_workspace(M: int, N: int, K: int) -> int:
    n = ctypes.c_size_t(0)
    _check("hif4_gemm_workspace", lib.hif4_gemm_workspace(M, N, K, ctypes.byref(n)))
    return int(n.value)


def hif4_gemm(a_units: torch.Tensor, b_units: torch.Tensor, out: Optional[torch.Tensor] = None,
              workspace: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """C[M, N] (FP32) = A[M, K] @ B[N, K]^T on HiF4 units ([M, K/64, 36] and [N, K/64, 36])."""
    _need_cuda(a_units, b_units, out, workspace)
    assert a_units.dtype == torch.uint8 and b_units.dtype == torch.uint8
    assert a_units.dim() == 3 and b_units.dim() == 3 and a_units.shape[1] == b_units.shape[1]
    assert a_units.is_contiguous() and b_units.is_contiguous()
    M, upr, _ = a_units.shape
    N = b_units.shape[0]
    K = upr * UNIT_ELEMS
    if out is None:
        out = torch.empty((M, N), dtype=torch.float32, device=a_units.device)
    assert out.dtype == torch.float32 and out.stride(1) == 1
    need = hif4_gemm_workspace(M, N, K)
    if workspace is None and need:
        workspace = torch.empty(need, dtype=torch.uint8, device=a_units.device)
    ldc = out.stride(0) if M > 1 else max(N, out.stride(0))
    _check("hif4_gemm", lib.hif4_gemm(a_units.data_ptr(), b_units.data_ptr(), out.data_ptr(), M, N, K, ldc,
                                      workspace.data_ptr() if workspace is not None else None,
                                      workspace.numel() if workspace is not None else 0, _stream(stream)))
    return out


def hif4_linear_workspace(M: int, N: int, K: int) -> int:
    n = ctypes.c_size_t(0)
    _check("hif4_linear_workspace", lib.hif4_linear_workspace(M, N, K, ctypes.byref(n)))
    return int(n.value)


def hif4_linear(x: torch.Tensor, w_units: torch.Tensor, out: Optional[torch.Tensor] = None, mode: int = HIF4_RNE,
                workspace: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Y[M, N] (FP32) = HiF4(X[M, K]) @ W[N, K]^T: activations quantized on the fly (Algorithm 1), weights
    given as HiF4 units [N, K/64, 36]."""
    _need_cuda(x, w_units, out, workspace)
    assert x.dim() == 2 and x.stride(1) == 1 and w_units.dtype == torch.uint8 and w_units.dim() == 3
    assert w_units.is_contiguous() and w_units.shape[2] == UNIT_BYTES
    M, K = x.shape
    N = w_units.shape[0]
    assert w_units.shape[1] * UNIT_ELEMS == K
    if out is None:
        out = torch.empty((M, N), dtype=torch.float32, device=x.device)
    assert out.dtype == torch.float32 and out.stride(1) == 1
    need = hif4_linear_workspace(M, N, K)
    if workspace is None and need:
        workspace = torch.empty(need, dtype=torch.uint8, device=x.device)
    ld_x = x.stride(0) if M > 1 else max(K, x.stride(0))
    ldy = out.stride(0) if M > 1 else max(N, out.stride(0))
    _check("hif4_linear", lib.hif4_linear(x.data_ptr(), _dtype_code(x.dtype), ld_x, w_units.data_ptr(), out.data_ptr(),
                                          M, N, K, ldy, mode, workspace.data_ptr() if workspace is not None else None,
                                          workspace.numel() if workspace is not None else 0, _stream(stream)))
    return out


def hif4_grouped_gemm_workspace(num_groups: int, total_rows: int, N: int, K: int) -> int:
    n = ctypes.c_size_t(0)
    _check("hif4_grouped_gemm_workspace",
           lib.hif4_grouped_gemm_workspace(num_groups, total_rows, N, K, ctypes.byref(n)))
    return int(n.value)


def hif4_grouped_gemm(a_units: torch.Tensor, b_units: torch.Tensor, group_offsets: torch.Tensor,
                      out: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                      stream=None) -> torch.Tensor:
    """Per group g: C[off[g]:off[g+1]] = A[off[g]:off[g+1]] @ B[g]^T; B is [G, N, K/64, 36] and
    `group_offsets` a device int64 tensor of G+1 prefix sums."""
    _need_cuda(a_units, b_units, group_offsets, out, workspace)
    assert a_units.dtype == torch.uint8 and b_units.dtype == torch.uint8 and group_offsets.dtype == torch.int64
    assert a_units.dim() == 3 and b_units.dim() == 4 and a_units.shape[1] == b_units.shape[2]
    assert a_units.is_contiguous() and b_units.is_contiguous() and group_offsets.is_contiguous()
    total, upr, _ = a_units.shape
    G, N = b_units.shape[0], b_units.shape[1]
    assert group_offsets.numel() == G + 1
    K = upr * UNIT_ELEMS
    if out is None:
        out = torch.empty((total, N), dtype=torch.float32, device=a_units.device)
    need = hif4_grouped_gemm_workspace(G, total, N, K)
    if workspace is None and need:
        workspace = torch.empty(need, dtype=torch.uint8, device=a_units.device)
    ldc = out.stride(0) if total > 1 else max(N, out.stride(0))
    _check("hif4_grouped_gemm",
           lib.hif4_grouped_gemm(a_units.data_ptr(), b_units.data_ptr(), out.data_ptr(), group_offsets.data_ptr(),
                                 G, total, N, K, ldc, workspace.data_ptr() if workspace is not None else None,
                                 workspace.numel() if workspace is not None else 0, _stream(stream)))
    return out


def hif4_grouped_gemm_noalloc_capacity() -> int:
    """Bytes of the scratch array built into the library for `hif4_grouped_gemm_noalloc`."""
    return int(lib.hif4_grouped_gemm_noalloc_capacity())


def hif4_grouped_gemm_noalloc(a_units: torch.Tensor, b_units: torch.Tensor, group_offsets: torch.Tensor,
                              out: torch.Tensor, stream=None) -> torch.Tensor:
    """`hif4_grouped_gemm` for callers that may not allocate on the device: the output must be passed
    in, and the kernel's tile table sits in a fixed array inside the library instead of a workspace.
    Problems whose table does not fit are refused (Hif4Error, status 5).  All calls on a GPU share
    that array, so calls that could overlap on the GPU must be ordered by the caller."""
    _need_cuda(a_units, b_units, group_offsets, out)
    assert a_units.dtype == torch.uint8 and b_units.dtype == torch.uint8 and group_offsets.dtype == torch.int64
    assert a_units.dim() == 3 and b_units.dim() == 4 and a_units.shape[1] == b_units.shape[2]
    assert a_units.is_contiguous() and b_units.is_contiguous() and group_offsets.is_contiguous()
    total, upr, _ = a_units.shape
    G, N = b_units.shape[0], b_units.shape[1]
    assert group_offsets.numel() == G + 1
    assert out.dtype == torch.float32 and out.stride(1) == 1 and out.shape == (total, N)
    ldc = out.stride(0) if total > 1 else max(N, out.stride(0))
    _check("hif4_grouped_gemm_noalloc",
           lib.hif4_grouped_gemm_noalloc(a_units.data_ptr(), b_units.data_ptr(), out.data_ptr(),
                                         group_offsets.data_ptr(), G, total, N, upr * UNIT_ELEMS, ldc, _stream(stream)))
    return out


def hif4_debug_set_gemm_path(path: int) -> None:
    """Test hook: 0 = by shape, 1 = CUDA-core kernel, 2 = single-CTA tensor-core kernel, 3 = CTA-pair kernel,
    4 = weight-streaming kernel (each whenever legal)."""
    _check("hif4_debug_set_gemm_path", lib.hif4_debug_set_gemm_path(path))


def hif4_mse_workspace(n: int, fmt: int) -> int:
    b = ctypes.c_size_t(0)
    _check("hif4_mse_workspace", lib.hif4_mse_workspace(n, fmt, ctypes.byref(b)))
    return int(b.value)


def hif4_mse_roundtrip(src: torch.Tensor, fmt: int, want_image: bool = True, workspace: Optional[torch.Tensor] = None,
                       stream=None):
    """BF16 tensor -> (FP32 image after a round trip through the 4-bit format `fmt` or None, one-element FP64 device
    tensor holding the summed squared error): the quantization-error experiment of Section III-A."""
    _need_cuda(src, workspace)
    assert src.dtype == torch.bfloat16 and src.is_contiguous()
    n = src.numel()
    image = torch.empty(src.shape, dtype=torch.float32, device=src.device) if want_image else None
    err = torch.empty(1, dtype=torch.float64, device=src.device)
    need = hif4_mse_workspace(n, fmt)
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=src.device)
    _check("hif4_mse_roundtrip", lib.hif4_mse_roundtrip(src.data_ptr(), n, fmt, image.data_ptr() if want_image else None,
                                                        err.data_ptr(), workspace.data_ptr(), workspace.numel(), _stream(stream)))
    return image, err


def hif4_debug_wait_timeout(budget_ns: int, stream=None) -> None:
    """Test hook: a kernel whose bounded wait (budget_ns) runs out on purpose; see include/hif4.h."""
    _check("hif4_debug_wait_timeout", lib.hif4_debug_wait_timeout(int(budget_ns), _stream(stream)))


def hif4_last_device_status(stream=None) -> int:
    return int(lib.hif4_last_device_status(_stream(stream)))
