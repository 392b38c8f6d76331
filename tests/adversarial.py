"""Adversarial quantizer inputs (bit patterns only, no format arithmetic): every BF16 magnitude as
an element under many different unit peaks, exponent extremes, signed zeros, subnormals, NaN, Inf."""
import numpy as np


def bf16_sweep_units(peaks_bits, lo_bits=0x0000, hi_bits=0x7F80, seed=0):
    """For each peak pattern: units whose element 0 (or a random slot) holds the peak and whose other
    63 slots walk through consecutive BF16 patterns in [lo_bits, hi_bits), with random signs."""
    rng = np.random.default_rng(seed)
    pats = np.arange(lo_bits, hi_bits, dtype=np.uint32)
    n_units = -(-len(pats) // 63)
    pad = n_units * 63 - len(pats)
    pats = np.concatenate([pats, pats[:pad]])
    out = []
    for p in peaks_bits:
        body = np.minimum(pats, p).reshape(n_units, 63)       # never exceed the peak
        unit = np.empty((n_units, 64), dtype=np.uint32)
        slot = rng.integers(0, 64, n_units)
        mask = np.ones((n_units, 64), bool)
        mask[np.arange(n_units), slot] = False
        unit[mask] = body.reshape(-1)
        unit[np.arange(n_units), slot] = p
        unit |= (rng.integers(0, 2, unit.shape, dtype=np.uint32) << 15)
        out.append(unit)
    return np.concatenate(out).astype(np.uint16)


def bf16_special_units():
    """Hand-picked units: zeros, negative zeros, NaN, +-Inf, largest finite, subnormals, smallest
    scales, single spikes."""
    rows = []

    def unit(**kw):
        u = np.zeros(64, dtype=np.uint16)
        for k, v in kw.items():
            u[int(k[1:])] = v
        rows.append(u)

    unit()                                           # all +0
    unit(e3=0x8000, e10=0x8000)                      # some -0
    unit(e17=0x7FC0, e0=0x3F80)                      # NaN
    unit(e63=0xFFC1)                                 # negative NaN payload
    unit(e9=0xFF80, e0=0x3F80, e8=0x4000)            # -Inf with finite neighbours
    unit(e0=0x7F80, e1=0x7F7F)                       # +Inf and max finite
    unit(e0=0x7F7F, e5=0xFF7F, e6=0x7E80)            # max finite
    unit(e0=0x0001, e1=0x8001, e2=0x007F)            # subnormals
    unit(e0=0x0080, e1=0x0100)                       # smallest normals
    for ebits in range(0x25, 0x2B):                  # around 2^-52 .. 2^-46: bottom of the E6M2 range
        for mant in (0x00, 0x20, 0x40, 0x60, 0x7F):
            unit(e0=(ebits << 7) | mant, e1=((ebits - 1) << 7) | 0x40, e9=0x8000 | ((ebits - 2) << 7))
    for ebits in range(0x8E, 0x95):                  # around 2^15 .. 2^21: top of the E6M2 range
        for mant in (0x00, 0x20, 0x40, 0x60, 0x7F):
            unit(e0=(ebits << 7) | mant, e1=((ebits - 1) << 7) | 0x40, e9=0x8000 | ((ebits - 3) << 7))
    for i in (0, 7, 8, 31, 32, 63):                  # single spike in a quiet unit
        u = np.full(64, 0x3C00, dtype=np.uint16)     # 2^-7
        u[i] = 0x4480                                # 1024
        rows.append(u)
    return np.stack(rows)


def fp32_adversarial(seed=0, n_units=6000):
    """FP32 units: BF16-exact values (they sit on the rounding ties of the scaled domain), their
    1-ulp neighbours, wide exponent spread, specials."""
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((n_units, 64)).astype(np.float32)
    x[: n_units // 3] = (x[: n_units // 3].view(np.uint32) & 0xFFFF0000).view(np.float32)
    third = slice(n_units // 3, 2 * n_units // 3)
    base = (x[third].view(np.uint32) & 0xFFFF0000).astype(np.int64)
    x[third] = (base + rng.integers(-1, 2, base.shape)).astype(np.uint32).view(np.float32)
    x *= np.exp2(rng.integers(-60, 30, (n_units, 1))).astype(np.float32)
    x[0, :] = 0.0
    x[1, 5] = -0.0
    x[2, 7] = np.nan
    x[3, 1] = np.inf
    x[4, 2] = -np.inf
    x[5, :] = np.float32(3.4028235e38)
    x[6, :] = np.float32(1e-45)
    x[7, 0] = 7.0; x[7, 1:] = 0.125
    return x
