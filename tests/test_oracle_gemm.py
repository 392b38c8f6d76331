"""Pins of the oracle's dot product (Eq. 3) and FP64 GEMM reference."""
import numpy as np

import oracle
from tests.test_oracle_encode import to_bf16_bits
from tests.test_oracle_format import make_unit


def _random_units(rng, rows, upr, nan_rate=0.0):
    u = rng.integers(0, 256, size=(rows, upr, 36), dtype=np.uint8)
    # keep E6M2 in a moderate range so FP64 sums stay far from overflow, avoid the NaN byte
    u[..., 0] = rng.integers(0x80, 0xF0, size=(rows, upr), dtype=np.uint8)
    if nan_rate:
        u[..., 0] = np.where(rng.random((rows, upr)) < nan_rate, 0xFF, u[..., 0])
    return u


def test_eq3_integer_flow_equals_flat_sum_of_eq2_products():
    rng = np.random.default_rng(10)
    ua = _random_units(rng, 400, 1)[:, 0]
    ub = _random_units(rng, 400, 1)[:, 0]
    va = oracle.dequantize(ua.reshape(-1, 1, 36))
    vb = oracle.dequantize(ub.reshape(-1, 1, 36))
    for a, b, xa, xb in zip(ua, ub, va, vb):
        # 64 products of <= 12 significant bits on one common exponent: the FP64 sum is exact
        assert oracle.dot_eq3(a, b) == float(np.dot(xa, xb))


def test_eq3_hand_case():
    # A: E6M2 = 1.25 (0xC1), group 0 shifted by level 2, elements 0..3 = 1.75 ; B: E6M2 = 2 (0xC4),
    # level-3 group 0 shifted, elements 0..3 = -0.5, element 8 = 1.0 against A's element 8 = 0.25
    a = make_unit(0xC1, 0b1, 0, [7, 7, 7, 7, 0, 0, 0, 0, 1])
    b = make_unit(0xC4, 0, 0b1, [0xA, 0xA, 0xA, 0xA, 0, 0, 0, 0, 4])
    want = 1.25 * 2.0 * (4 * (1.75 * 2) * (-0.5 * 2) + 0.25 * 1.0)
    assert oracle.dot_eq3(a, b) == want
    nan = make_unit(0xFF)
    assert np.isnan(oracle.dot_eq3(a, nan)) and np.isnan(oracle.dot_eq3(nan, b))


def test_gemm_f64_against_numpy_matmul_and_eq3():
    rng = np.random.default_rng(11)
    M, N, upr = 9, 13, 3
    A, B = _random_units(rng, M, upr), _random_units(rng, N, upr)
    C, Cabs = oracle.gemm_f64(A, B)
    Ad, Bd = oracle.dequantize(A), oracle.dequantize(B)
    ref = Ad @ Bd.T                                     # library routine on the decoded operands
    refabs = np.abs(Ad) @ np.abs(Bd).T
    assert np.allclose(C, ref, rtol=0, atol=1e-13 * refabs.max())
    assert np.allclose(Cabs, refabs, rtol=1e-13)
    # transposition mistakes would show: A and B have different row counts and contents
    assert C.shape == (M, N)
    # unit-pair sums of Eq. 3 add up to the same thing
    for i in (0, M - 1):
        for j in (0, N - 1):
            s = sum(oracle.dot_eq3(A[i, k], B[j, k]) for k in range(upr))
            assert abs(s - C[i, j]) <= 1e-13 * Cabs[i, j]
    # multi-threaded run is identical
    C2, _ = oracle.gemm_f64(A, B, nthreads=3)
    assert np.array_equal(C, C2)


def test_gemm_sampled_matches_full():
    rng = np.random.default_rng(12)
    A, B = _random_units(rng, 20, 2), _random_units(rng, 17, 2)
    C, Cabs = oracle.gemm_f64(A, B)
    rows = rng.integers(0, 20, 50); cols = rng.integers(0, 17, 50)
    s, sabs = oracle.gemm_sampled_f64(A, B, rows, cols)
    assert np.array_equal(s, C[rows, cols]) and np.array_equal(sabs, Cabs[rows, cols])


def test_gemm_nan_units_poison_their_row_or_column():
    rng = np.random.default_rng(13)
    A, B = _random_units(rng, 4, 2), _random_units(rng, 5, 2)
    A[2, 1, 0] = 0xFF
    B[3, 0, 0] = 0xFF
    C, _ = oracle.gemm_f64(A, B)
    mask = np.zeros((4, 5), bool); mask[2, :] = True; mask[:, 3] = True
    assert np.array_equal(np.isnan(C), mask)


def test_grouped_gemm_is_per_group_gemm():
    rng = np.random.default_rng(14)
    G, N, upr = 5, 6, 2
    counts = np.array([3, 0, 7, 1, 0])
    off = np.concatenate([[0], np.cumsum(counts)]).astype(np.int64)
    A = _random_units(rng, int(off[-1]), upr)
    B = _random_units(rng, G * N, upr).reshape(G, N, upr, 36)
    C, Cabs = oracle.grouped_gemm_f64(A, B, off)
    for g in range(G):
        if counts[g]:
            Cg, Cg_abs = oracle.gemm_f64(A[off[g]:off[g + 1]], B[g])
            assert np.array_equal(C[off[g]:off[g + 1]], Cg) and np.array_equal(Cabs[off[g]:off[g + 1]], Cg_abs)


def test_quantized_linear_tracks_the_bf16_linear():
    """End-to-end sanity of quantize -> gemm: relative error of the W4A4 product against the
    unquantised product is at the level a 3-bit significand gives (a few percent), not garbage."""
    rng = np.random.default_rng(15)
    X = to_bf16_bits(rng.standard_normal((16, 256)).astype(np.float32))
    W = to_bf16_bits((rng.standard_normal((24, 256)) * 0.02).astype(np.float32))
    C, _ = oracle.gemm_f64(oracle.quantize(X), oracle.quantize(W))
    ref = oracle.bf16_bits_to_f64(X) @ oracle.bf16_bits_to_f64(W).T
    rel = np.linalg.norm(C - ref) / np.linalg.norm(ref)
    assert rel < 0.15
