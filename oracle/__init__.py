"""CPU oracle for HiF4 -- TEST INFRASTRUCTURE ONLY.

Thin ctypes loader around ``hif4_ref.cpp`` (plain C++17, written from the paper: Eq. 2, Algorithm 1,
Eq. 3).  Only the test-suite, the smoke check and the benchmark's CPU-baseline leg may import this
package; the CUDA library and its Python binding never do, and share no code with it.

Arrays are numpy: BF16 data travels as ``uint16`` bit patterns, FP32 as ``float32``, packed units as
``uint8`` of shape ``[rows, cols // 64, 36]``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hif4_ref.cpp")
_LIB = os.path.join(_HERE, "libhif4_ref.so")

BF16, FP32, FP64 = 0, 1, 2
RNE, RHA = 0, 1
UNIT_ELEMS, UNIT_BYTES = 64, 36


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (no fast-math, no FMA contraction) and return the .so path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = f"{_LIB}.{os.getpid()}.tmp"       # several processes may build at once: each its own file, then an atomic rename
        cmd = ["g++", "-O2", "-std=c++17", "-fPIC", "-shared", "-ffp-contract=off", "-fno-fast-math",
               "-pthread", "-Wall", "-Wextra", "-o", tmp, _SRC]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        i64, dbl, vp, ci, cu = ctypes.c_int64, ctypes.c_double, ctypes.c_void_p, ctypes.c_int, ctypes.c_uint
        L.hif4_ref_packed_bytes.restype = i64
        L.hif4_ref_packed_bytes.argtypes = [i64, i64]
        L.hif4_ref_e6m2_value.restype = dbl
        L.hif4_ref_e6m2_value.argtypes = [cu]
        L.hif4_ref_e6m2_from_value.restype = cu
        L.hif4_ref_e6m2_from_value.argtypes = [dbl, ci]
        L.hif4_ref_e6m2_reciprocal.restype = dbl
        L.hif4_ref_e6m2_reciprocal.argtypes = [cu, ci]
        L.hif4_ref_round_to.restype = dbl
        L.hif4_ref_round_to.argtypes = [dbl, ci]
        L.hif4_ref_quantize.restype = ci
        L.hif4_ref_quantize.argtypes = [vp, ci, i64, i64, i64, vp, ci, ci]
        L.hif4_ref_dequantize.restype = ci
        L.hif4_ref_dequantize.argtypes = [vp, i64, i64, vp, ci, i64, ci]
        L.hif4_ref_gemm_f64.restype = ci
        L.hif4_ref_gemm_f64.argtypes = [vp, vp, vp, vp, i64, i64, i64, ci]
        L.hif4_ref_gemm_sampled_f64.restype = ci
        L.hif4_ref_gemm_sampled_f64.argtypes = [vp, vp, i64, i64, i64, vp, vp, i64, vp, vp]
        L.hif4_ref_grouped_gemm_f64.restype = ci
        L.hif4_ref_grouped_gemm_f64.argtypes = [vp, vp, vp, vp, vp, ci, i64, i64, ci]
        L.hif4_ref_dot_eq3.restype = dbl
        L.hif4_ref_dot_eq3.argtypes = [vp, vp]
        L.hif4_ref_best_unit.restype = dbl
        L.hif4_ref_best_unit.argtypes = [vp, vp]
        L.hif4_ref_hardware_threads.restype = ci
        flt, fp = ctypes.c_float, ctypes.c_void_p
        L.hif4_ref_e2m1_round.restype = flt
        L.hif4_ref_e2m1_round.argtypes = [flt]
        L.hif4_ref_e4m3_round.restype = flt
        L.hif4_ref_e4m3_round.argtypes = [flt]
        L.hif4_ref_pts_gain.restype = flt
        L.hif4_ref_pts_gain.argtypes = [fp, i64]
        L.hif4_ref_mxfp4_roundtrip.restype = ci
        L.hif4_ref_mxfp4_roundtrip.argtypes = [fp, i64, fp]
        L.hif4_ref_nvfp4_roundtrip.restype = ci
        L.hif4_ref_nvfp4_roundtrip.argtypes = [fp, i64, flt, fp]
        _lib = L
    return _lib


def _ptr(a: np.ndarray) -> ctypes.c_void_p:
    return ctypes.c_void_p(a.ctypes.data)


def _check(rc: int, what: str) -> None:
    if rc != 0:
        raise ValueError(f"{what}: oracle rejected the arguments (code {rc})")


def hardware_threads() -> int:
    return int(lib().hif4_ref_hardware_threads())


def e6m2_value(byte: int) -> float:
    return float(lib().hif4_ref_e6m2_value(byte))


def e6m2_from_value(sf: float, mode: int = RNE) -> int:
    return int(lib().hif4_ref_e6m2_from_value(float(sf), mode))


def e6m2_reciprocal(byte: int, dt: int = BF16) -> float:
    return float(lib().hif4_ref_e6m2_reciprocal(byte, dt))


def round_to(v: float, dt: int) -> float:
    return float(lib().hif4_ref_round_to(float(v), dt))


def quantize(src: np.ndarray, mode: int = RNE, nthreads: int = 1) -> np.ndarray:
    """Algorithm 1 on a 2-D array: ``uint16`` = BF16 bit patterns, ``float32`` = FP32, ``float16`` = FP16.

    Section II-B extends the conversion to FP32 and FP16 sources without further detail.  FP16 arithmetic
    cannot hold the reciprocal of an E6M2 scale (up to 2^48), so an FP16 source is read as: widen every
    element to FP32 (a storage conversion, exact) and run the FP32 form of Algorithm 1."""
    assert src.ndim == 2 and src.shape[1] % UNIT_ELEMS == 0
    if src.dtype == np.uint16:
        dt = BF16
    elif src.dtype == np.float32:
        dt = FP32
    elif src.dtype == np.float16:
        dt = FP32
        src = src.astype(np.float32)
    else:
        raise TypeError("quantize takes uint16 (BF16 bits), float32 or float16")
    src = np.ascontiguousarray(src)
    rows, cols = src.shape
    out = np.zeros((rows, cols // UNIT_ELEMS, UNIT_BYTES), dtype=np.uint8)
    if rows and cols:
        _check(lib().hif4_ref_quantize(_ptr(src), dt, rows, cols, cols, _ptr(out), mode, nthreads), "quantize")
    return out


def dequantize(units: np.ndarray, dt: int = FP64, nthreads: int = 1) -> np.ndarray:
    """Eq. 2 on ``[rows, upr, 36]`` units -> ``[rows, upr*64]`` (uint16 BF16 bits, float32 or float64)."""
    assert units.dtype == np.uint8 and units.ndim == 3 and units.shape[2] == UNIT_BYTES
    units = np.ascontiguousarray(units)
    rows, upr, _ = units.shape
    cols = upr * UNIT_ELEMS
    out = np.zeros((rows, cols), dtype={BF16: np.uint16, FP32: np.float32, FP64: np.float64}[dt])
    if rows and cols:
        _check(lib().hif4_ref_dequantize(_ptr(units), rows, cols, _ptr(out), dt, cols, nthreads), "dequantize")
    return out


def gemm_f64(a_units: np.ndarray, b_units: np.ndarray, nthreads: int = 1, want_abs: bool = True):
    """FP64 ``A @ B.T`` on decoded operands, plus ``sum_k |a||b|`` for the tolerance."""
    a_units = np.ascontiguousarray(a_units)
    b_units = np.ascontiguousarray(b_units)
    M, upr, _ = a_units.shape
    N, upr_b, _ = b_units.shape
    assert upr == upr_b
    C = np.zeros((M, N), dtype=np.float64)
    Cabs = np.zeros((M, N), dtype=np.float64) if want_abs else None
    _check(lib().hif4_ref_gemm_f64(_ptr(a_units), _ptr(b_units), _ptr(C), _ptr(Cabs) if want_abs else None,
                                   M, N, upr * UNIT_ELEMS, nthreads), "gemm_f64")
    return C, Cabs


def gemm_sampled_f64(a_units: np.ndarray, b_units: np.ndarray, rows: np.ndarray, cols: np.ndarray):
    a_units = np.ascontiguousarray(a_units)
    b_units = np.ascontiguousarray(b_units)
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    cols = np.ascontiguousarray(cols, dtype=np.int64)
    M, upr, _ = a_units.shape
    N = b_units.shape[0]
    out = np.zeros(rows.shape[0], dtype=np.float64)
    out_abs = np.zeros(rows.shape[0], dtype=np.float64)
    _check(lib().hif4_ref_gemm_sampled_f64(_ptr(a_units), _ptr(b_units), M, N, upr * UNIT_ELEMS, _ptr(rows),
                                           _ptr(cols), rows.shape[0], _ptr(out), _ptr(out_abs)), "gemm_sampled_f64")
    return out, out_abs


def grouped_gemm_f64(a_units: np.ndarray, b_units: np.ndarray, offsets: np.ndarray, nthreads: int = 1):
    """``b_units`` is ``[G, N, upr, 36]``; rows ``offsets[g]:offsets[g+1]`` of A meet weight g."""
    a_units = np.ascontiguousarray(a_units)
    b_units = np.ascontiguousarray(b_units)
    offsets = np.ascontiguousarray(offsets, dtype=np.int64)
    total, upr, _ = a_units.shape
    G, N = b_units.shape[0], b_units.shape[1]
    assert offsets.shape[0] == G + 1 and offsets[-1] == total
    C = np.zeros((total, N), dtype=np.float64)
    Cabs = np.zeros((total, N), dtype=np.float64)
    _check(lib().hif4_ref_grouped_gemm_f64(_ptr(a_units), _ptr(b_units), _ptr(C), _ptr(Cabs), _ptr(offsets), G, N,
                                           upr * UNIT_ELEMS, nthreads), "grouped_gemm_f64")
    return C, Cabs


def dot_eq3(unit_a: np.ndarray, unit_b: np.ndarray) -> float:
    unit_a = np.ascontiguousarray(unit_a, dtype=np.uint8)
    unit_b = np.ascontiguousarray(unit_b, dtype=np.uint8)
    assert unit_a.size == UNIT_BYTES and unit_b.size == UNIT_BYTES
    return float(lib().hif4_ref_dot_eq3(_ptr(unit_a), _ptr(unit_b)))


def best_unit(x: np.ndarray):
    """Brute-force MSE-optimal unit for 64 finite doubles -> (sum of squared errors, unit bytes)."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    assert x.size == UNIT_ELEMS
    out = np.zeros(UNIT_BYTES, dtype=np.uint8)
    err = float(lib().hif4_ref_best_unit(_ptr(x), _ptr(out)))
    return err, out


# ---- comparison formats of the quantization-error study (Section III-A)
def e2m1_round(q: float) -> float:
    return float(lib().hif4_ref_e2m1_round(float(q)))


def e4m3_round(v: float) -> float:
    return float(lib().hif4_ref_e4m3_round(float(v)))


def pts_gain(x: np.ndarray) -> float:
    """2688 / max|x| (one FP32 division): the per-tensor scaling that precedes NVFP4 in the study."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    return float(lib().hif4_ref_pts_gain(_ptr(x), x.size))


def mxfp4_roundtrip(x: np.ndarray) -> np.ndarray:
    """float32 array (size a multiple of 32) -> its MXFP4 quantize-dequantize image, float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    out = np.empty_like(x)
    _check(lib().hif4_ref_mxfp4_roundtrip(_ptr(x), x.size, _ptr(out)), "mxfp4_roundtrip")
    return out


def nvfp4_roundtrip(x: np.ndarray, gain: float = 1.0) -> np.ndarray:
    """float32 array (size a multiple of 16) -> its NVFP4 image; gain = pts_gain(x) applies per-tensor scaling."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    out = np.empty_like(x)
    _check(lib().hif4_ref_nvfp4_roundtrip(_ptr(x), x.size, float(np.float32(gain)), _ptr(out)), "nvfp4_roundtrip")
    return out


# ---- small numpy conveniences for BF16 bit patterns (storage conversion only, no method arithmetic)
def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def f32_to_bf16_bits_exact(x: np.ndarray) -> np.ndarray:
    """Bit patterns of float32 values that are already BF16-representable (asserted)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    assert np.all((u & 0xFFFF) == 0), "value is not exactly a BF16"
    return (u >> 16).astype(np.uint16)
