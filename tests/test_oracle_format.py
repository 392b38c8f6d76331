"""Pins of the oracle's decoder (Eq. 2) and of the unit layout against what the paper prints."""
import math
from fractions import Fraction

import numpy as np
import pytest

import oracle
from tests import paper_constants


def make_unit(byte=0xC0, e8=0, e16=0, codes=None):
    """Assemble one unit from fields, following the layout stated in include/hif4.h."""
    u = np.zeros(36, dtype=np.uint8)
    meta = (byte & 0xFF) | ((e8 & 0xFF) << 8) | ((e16 & 0xFFFF) << 16)
    u[0:4] = np.frombuffer(np.uint32(meta).tobytes(), dtype=np.uint8)
    if codes is not None:
        for i, c in enumerate(codes):
            u[4 + i // 2] |= (c & 0xF) << (4 * (i & 1))
    return u


def decode1(u, dt=oracle.FP64):
    return oracle.dequantize(u.reshape(1, 1, 36), dt)[0]


@pytest.fixture(scope="module")
def paper(golden_dir):
    return paper_constants.load(golden_dir)


def test_unit_size_is_288_bits(paper):
    bits = paper["unit_metadata_bits"] + paper["unit_elements"] * paper["unit_element_bits"]
    assert bits == 288
    assert oracle.UNIT_BYTES * 8 == bits
    assert oracle.lib().hif4_ref_unit_bytes() * 8 == bits
    assert Fraction(bits, paper["unit_elements"]) == paper["bits_per_value"]
    assert oracle.lib().hif4_ref_packed_bytes(3, 128) == 3 * 2 * 36
    assert oracle.lib().hif4_ref_packed_bytes(3, 100) == 0


def test_e6m2_table1(paper):
    assert Fraction(oracle.e6m2_value(paper["e6m2_max_byte"])) == paper["e6m2_max_value"]
    assert Fraction(oracle.e6m2_value(paper["e6m2_min_byte"])) == paper["e6m2_min_value"]
    assert math.isnan(oracle.e6m2_value(paper["e6m2_nan_byte"]))
    bias = paper["e6m2_exponent_bias"]
    for byte in range(255):
        E, M = (byte >> 2) - bias, byte & 3
        assert paper["e6m2_unbiased_exp_min"] <= E <= paper["e6m2_unbiased_exp_max"]
        # Eq. 1: X = 2^E * 1.M, hidden bit 1, no zero, no infinity, normal only
        assert Fraction(oracle.e6m2_value(byte)) == Fraction(2) ** E * Fraction(4 + M, 4)
    vals = [oracle.e6m2_value(b) for b in range(255)]
    assert all(b > a for a, b in zip(vals, vals[1:])), "E6M2 bytes are monotone in value"


def test_exhaustive_decode_all_code_and_metadata_combinations(paper):
    """Every E6M2 byte x level-2 bit x level-3 bit x 4-bit code, against integer arithmetic:
    value = (+-) (4+M) * m * 2^(E - 48 + e8 + e16 - 4)."""
    bias = paper["e6m2_exponent_bias"]
    distinct = set()
    largest, smallest = Fraction(0), None
    for byte in range(255):
        units = []
        for e8 in (0, 1):
            for e16 in (0, 1):
                # element 0 sits in level-2 group 0 and level-3 group 0; sweep its 16 codes through
                # all 64 positions' worth of units in one call
                for code in range(16):
                    units.append(make_unit(byte, e8, e16, [code]))
        arr = np.stack(units).reshape(len(units), 1, 36)
        v64 = oracle.dequantize(arr, oracle.FP64)[:, 0]
        v32 = oracle.dequantize(arr, oracle.FP32)[:, 0]
        v16 = oracle.bf16_bits_to_f64(oracle.dequantize(arr, oracle.BF16)[:, 0])
        n = 0
        E, M = (byte >> 2) - bias, byte & 3
        for e8 in (0, 1):
            for e16 in (0, 1):
                for code in range(16):
                    m, s = code & 7, code >> 3
                    want = Fraction((4 + M) * m) * Fraction(2) ** (E + e8 + e16 - 4)
                    got = Fraction(float(v64[n]))
                    assert abs(got) == want, (byte, e8, e16, code)
                    assert math.copysign(1.0, v64[n]) == (-1.0 if s else 1.0)
                    # exactly representable in FP32 and BF16 (what lets a BF16 tensor core hold it)
                    assert float(v32[n]) == float(v64[n]) and float(v16[n]) == float(v64[n])
                    if m:
                        distinct.add(want)
                        largest = max(largest, want)
                        smallest = want if smallest is None else min(smallest, want)
                    n += 1
    assert largest == paper["hif4_max_positive"] == 344064
    assert smallest == paper["hif4_min_positive"]
    top = math.floor(math.log2(largest)); bottom = math.floor(math.log2(smallest))
    assert (bottom, top) == (-50, 18) and top - bottom + 1 == paper["global_binades"]
    # every magnitude needs at most 6 significand bits: (4+M)*m <= 49
    for v in distinct:
        num = v.numerator
        while num % 2 == 0:
            num //= 2
        assert num < 64


def test_intra_group_range_and_s1p2(paper):
    # E6M2 = 1.0 (byte 0xC0): the "blue part" of Eq. 2
    hi = decode1(make_unit(0xC0, 1, 1, [7]))[0]
    lo = decode1(make_unit(0xC0, 0, 0, [1]))[0]
    assert Fraction(hi) == paper["intra_group_max"] and Fraction(lo) == paper["intra_group_min"]
    assert round(math.log2(hi / lo), 2) == float(paper["local_dynamic_range"])
    assert Fraction(decode1(make_unit(0xC0, 0, 0, [7]))[0]) == paper["s1p2_max_value"]
    assert Fraction(decode1(make_unit(0xC0, 0, 0, [1]))[0]) == paper["s1p2_min_value"]
    # 3-bit significand: the 8 magnitudes are k/4
    mags = [decode1(make_unit(0xC0, 0, 0, [c]))[0] for c in range(8)]
    assert mags == [k / 4 for k in range(8)]
    # sign-magnitude: +0 and -0 both exist
    z = decode1(make_unit(0xC0, 0, 0, [0, 8]))
    assert z[0] == 0 and not np.signbit(z[0]) and z[1] == 0 and np.signbit(z[1])


def test_layout_positions():
    """Element i <-> nibble i; level-2 bit j covers 8j..8j+7; level-3 bit k covers 4k..4k+3."""
    for i in range(64):
        codes = [0] * 64
        codes[i] = 4  # 1.0
        v = decode1(make_unit(0xC0, 0, 0, codes))
        assert v[i] == 1.0 and np.count_nonzero(v) == 1
    ones = [4] * 64
    for j in range(8):
        v = decode1(make_unit(0xC0, 1 << j, 0, ones))
        want = np.ones(64); want[8 * j:8 * j + 8] = 2.0
        assert np.array_equal(v, want)
    for k in range(16):
        v = decode1(make_unit(0xC0, 0, 1 << k, ones))
        want = np.ones(64); want[4 * k:4 * k + 4] = 2.0
        assert np.array_equal(v, want)
    # level 2 and level 3 multiply (Eq. 2: exponents add)
    v = decode1(make_unit(0xC0, 0b00000001, 0b0000000000000010, ones))
    assert list(v[:8]) == [2, 2, 2, 2, 4, 4, 4, 4] and np.all(v[8:] == 1)
    # metadata is a little-endian 32-bit word: E6M2 in the first byte
    u = make_unit(0xB5, 0x12, 0x3456, None)
    assert list(u[:4]) == [0xB5, 0x12, 0x56, 0x34]


def test_nan_unit_decodes_to_all_nan():
    rng = np.random.default_rng(0)
    u = make_unit(0xFF, 0xA5, 0x1234, list(rng.integers(0, 16, 64)))
    for dt in (oracle.FP64, oracle.FP32):
        assert np.all(np.isnan(decode1(u, dt)))
    bits = decode1(u, oracle.BF16)
    assert np.all(bits == 0x7FC0)
