"""GPU parity, bit-exact: hif4_quantize / hif4_dequantize through the C ABI against the CPU oracle."""
import numpy as np
import pytest
import torch

import hif4_workloads as wl
import oracle
from tests import adversarial

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def hif4():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    import paper_2602_11287_b200 as lib
    return lib


def _gpu_quantize_bits(hif4, bits_u16, mode=0):
    t = wl.u16_numpy_to_bf16(bits_u16, "cuda")
    return hif4.hif4_quantize(t, mode).cpu().numpy()


def _compare_units(got, want, what):
    if np.array_equal(got, want):
        return
    bad = np.argwhere((got != want).any(axis=-1))
    r, u = bad[0]
    raise AssertionError(f"{what}: {len(bad)} of {got.shape[0] * got.shape[1]} units differ; first at row {r} unit {u}: "
                         f"gpu {got[r, u].tobytes().hex()} oracle {want[r, u].tobytes().hex()}")


@pytest.mark.parametrize("mode", [0, 1])
def test_quantize_bf16_every_magnitude_under_many_peaks(hif4, mode):
    peaks = [0x4000 | m for m in range(0, 128, 3)] + [0x3F80, 0x3FFF, 0x40E0, 0x4100]
    bits = adversarial.bf16_sweep_units(peaks, 0x0000, 0x4200, seed=mode)
    got = _gpu_quantize_bits(hif4, bits, mode)
    want = oracle.quantize(bits, mode, nthreads=8)
    _compare_units(got, want, f"bf16 sweep mode {mode}")


@pytest.mark.parametrize("mode", [0, 1])
def test_quantize_bf16_specials_and_extremes(hif4, mode):
    bits = adversarial.bf16_special_units()
    got = _gpu_quantize_bits(hif4, bits, mode)
    want = oracle.quantize(bits, mode)
    _compare_units(got, want, "bf16 specials")
    # whole-range sweep with huge / tiny peaks
    bits = adversarial.bf16_sweep_units([0x7F7F, 0x7F80, 0x4780, 0x2A00, 0x0100, 0x0040], 0, 0x7F80, seed=3)
    _compare_units(_gpu_quantize_bits(hif4, bits, mode), oracle.quantize(bits, mode, nthreads=8), "bf16 extremes")


@pytest.mark.parametrize("mode", [0, 1])
def test_quantize_fp32_adversarial(hif4, mode):
    x = adversarial.fp32_adversarial(seed=mode)
    got = hif4.hif4_quantize(torch.from_numpy(x).cuda(), mode).cpu().numpy()
    want = oracle.quantize(x, mode, nthreads=8)
    _compare_units(got, want, f"fp32 adversarial mode {mode}")


def test_quantize_workload_distributions(hif4):
    x, w = wl.single_layer(device="cuda")
    for t in (x, w):
        _compare_units(hif4.hif4_quantize(t).cpu().numpy(), oracle.quantize(wl.bf16_to_u16_numpy(t), nthreads=8), "cfg1")
    t = wl.llama_activations(48, 4096, device="cuda")
    _compare_units(hif4.hif4_quantize(t).cpu().numpy(), oracle.quantize(wl.bf16_to_u16_numpy(t), nthreads=8), "cfg2")
    t = wl.quantize_sweep(2 ** 20, device="cuda")
    _compare_units(hif4.hif4_quantize(t).cpu().numpy(), oracle.quantize(wl.bf16_to_u16_numpy(t), nthreads=8), "cfg3")
    t32 = wl.quantize_sweep(2 ** 18, device="cuda", dtype=torch.float32)
    _compare_units(hif4.hif4_quantize(t32).cpu().numpy(), oracle.quantize(t32.cpu().numpy(), nthreads=8), "cfg3 fp32")
    t = wl.prefill_activations(64, 5120, device="cuda")
    _compare_units(hif4.hif4_quantize(t).cpu().numpy(), oracle.quantize(wl.bf16_to_u16_numpy(t), nthreads=8), "cfg4")


def test_quantize_ragged_sizes_strided_rows_and_guard_bands(hif4):
    g = torch.Generator(device="cuda"); g.manual_seed(5)
    for rows, cols, ld in [(1, 64, 64), (3, 64, 72), (5, 192, 192), (7, 320, 384), (33, 448, 448), (130, 64, 64),
                           (1, 4096, 4096), (17, 1088, 1096)]:
        for dtype in (torch.bfloat16, torch.float32):
            buf = torch.randn(rows, ld, generator=g, device="cuda", dtype=torch.float32).to(dtype)
            src = buf[:, :cols]
            upr = cols // 64
            out = torch.full((rows * upr * 36 + 128,), 0xAB, dtype=torch.uint8, device="cuda")
            view = out[64:64 + rows * upr * 36].view(rows, upr, 36)
            hif4.hif4_quantize(src, out=view)
            host = src.contiguous().cpu()
            ref = oracle.quantize(wl.bf16_to_u16_numpy(host) if dtype == torch.bfloat16 else host.numpy())
            _compare_units(view.cpu().numpy(), ref, f"ragged {rows}x{cols} ld {ld} {dtype}")
            o = out.cpu().numpy()
            assert (o[:64] == 0xAB).all() and (o[64 + rows * upr * 36:] == 0xAB).all(), "guard band overwritten"


def test_quantize_empty_and_bad_arguments(hif4):
    e = torch.empty(0, 128, dtype=torch.bfloat16, device="cuda")
    assert hif4.hif4_quantize(e).shape == (0, 2, 36)
    x = torch.zeros(4, 100, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(hif4.Hif4Error) as ei:
        hif4.hif4_quantize(x, out=torch.empty(4, 1, 36, dtype=torch.uint8, device="cuda"))
    assert ei.value.code == 2
    x = torch.zeros(4, 136, dtype=torch.bfloat16, device="cuda")[:, 4:132]     # rows not 16-byte aligned
    with pytest.raises(hif4.Hif4Error) as ei:
        hif4.hif4_quantize(x)
    assert ei.value.code == 3
    with pytest.raises(hif4.Hif4Error) as ei:
        hif4.hif4_quantize(torch.zeros(2, 64, dtype=torch.bfloat16, device="cuda"), mode=7)
    assert ei.value.code == 4
    with pytest.raises(TypeError):
        hif4.hif4_quantize(torch.zeros(2, 64, dtype=torch.float64, device="cuda"))
    with pytest.raises(ValueError):
        hif4.hif4_quantize(torch.zeros(2, 64, dtype=torch.bfloat16))
    assert hif4.hif4_last_device_status() == 0


def test_dequantize_every_code_and_metadata_value(hif4):
    rng = np.random.default_rng(6)
    # all 256 level-1 bytes (incl. NaN) x random micro-exponents and codes, plus fully random units
    u = rng.integers(0, 256, size=(256 * 8, 3, 36), dtype=np.uint8)
    u[:, :, 0] = (np.arange(256 * 8) % 256)[:, None]
    # make sure every (e8, e16, code) combination occurs under every byte: structured units
    s = np.zeros((256, 4, 36), dtype=np.uint8)
    for b in range(256):
        for v, (e8, e16) in enumerate([(0, 0), (0, 0xFFFF), (0xFF, 0), (0xFF, 0xFFFF)]):
            s[b, v, 0] = b; s[b, v, 1] = e8; s[b, v, 2] = e16 & 0xFF; s[b, v, 3] = e16 >> 8
            s[b, v, 4:] = np.tile(np.array([0x10, 0x32, 0x54, 0x76, 0x98, 0xBA, 0xDC, 0xFE], dtype=np.uint8), 4)
    for units in (u, s):
        dev = torch.from_numpy(units).cuda()
        got16 = hif4.hif4_dequantize(dev, torch.bfloat16)
        got32 = hif4.hif4_dequantize(dev, torch.float32)
        want16 = oracle.dequantize(units, oracle.BF16)
        want32 = oracle.dequantize(units, oracle.FP32)
        assert np.array_equal(wl.bf16_to_u16_numpy(got16), want16)
        assert np.array_equal(got32.cpu().numpy().view(np.uint32), want32.view(np.uint32))


def test_dequantize_strided_output_and_roundtrip(hif4):
    t = wl.llama_activations(19, 1088, device="cuda")
    units = hif4.hif4_quantize(t)
    buf = torch.full((19, 1100), 7.0, dtype=torch.float32, device="cuda")
    hif4.hif4_dequantize(units, out=buf[:, :1088])
    ref = oracle.dequantize(oracle.quantize(wl.bf16_to_u16_numpy(t)), oracle.FP32)
    assert np.array_equal(buf[:, :1088].cpu().numpy().view(np.uint32), ref.view(np.uint32))
    assert (buf[:, 1088:] == 7.0).all()
    # the "simulated 4-bit" tensor stays close to the source (3-bit significand, shared scales)
    rel = (buf[:, :1088] - t.float()).norm() / t.float().norm()
    assert rel < 0.15


@pytest.mark.parametrize("mode", [0, 1])
def test_quantize_random_bit_patterns(hif4, mode):
    """Uniformly random BF16 and FP32 bit patterns (every exponent, NaN and Inf included), plus units that
    mix a narrow range of exponents so that the finite path is exercised as well."""
    rng = np.random.default_rng(100 + mode)
    # BF16
    wild = rng.integers(0, 1 << 16, size=(512, 1024), dtype=np.uint32).astype(np.uint16)
    expo = rng.integers(100, 150, size=(512, 16, 1), dtype=np.uint32)                  # per unit: base exponent
    mant = rng.integers(0, 1 << 7, size=(512, 16, 64), dtype=np.uint32)
    sign = rng.integers(0, 2, size=(512, 16, 64), dtype=np.uint32) << 15
    spread = rng.integers(0, 7, size=(512, 16, 64), dtype=np.uint32)
    tame = (sign | ((expo - spread) << 7) | mant).astype(np.uint16).reshape(512, 1024)
    for bits in (wild, tame):
        got = _gpu_quantize_bits(hif4, bits, mode)
        _compare_units(got, oracle.quantize(bits, mode, nthreads=8), f"random bf16 bits mode {mode}")
    # FP32
    wild32 = rng.integers(0, 1 << 32, size=(256, 1024), dtype=np.uint64).astype(np.uint32).view(np.float32)
    expo = rng.integers(90, 160, size=(256, 16, 1), dtype=np.uint32)
    mant = rng.integers(0, 1 << 23, size=(256, 16, 64), dtype=np.uint32)
    sign = rng.integers(0, 2, size=(256, 16, 64), dtype=np.uint32) << 31
    spread = rng.integers(0, 7, size=(256, 16, 64), dtype=np.uint32)
    tame32 = (sign | ((expo - spread) << 23) | mant).astype(np.uint32).reshape(256, 1024).view(np.float32)
    for x in (wild32, tame32):
        got = hif4.hif4_quantize(torch.from_numpy(x.copy()).cuda(), mode).cpu().numpy()
        _compare_units(got, oracle.quantize(x, mode, nthreads=8), f"random fp32 bits mode {mode}")


@pytest.mark.parametrize("mode", [0, 1])
def test_quantize_fp16_source(hif4, mode):
    """FP16 sources (widened exactly to FP32, then Algorithm 1 in FP32 arithmetic): every FP16 bit pattern
    (subnormals, Inf and NaN included), units of a narrow exponent range, a strided source, and the one-call
    linear layer on FP16 activations."""
    rng = np.random.default_rng(300 + mode)
    every = np.arange(1 << 16, dtype=np.uint16)
    rng.shuffle(every)
    wild = every.reshape(64, 1024).view(np.float16)
    expo = rng.integers(3, 28, size=(256, 16, 1), dtype=np.uint32)
    mant = rng.integers(0, 1 << 10, size=(256, 16, 64), dtype=np.uint32)
    sign = rng.integers(0, 2, size=(256, 16, 64), dtype=np.uint32) << 15
    spread = rng.integers(0, 4, size=(256, 16, 64), dtype=np.uint32)
    tame = (sign | (np.maximum(expo - spread, 0) << 10) | mant).astype(np.uint16).reshape(256, 1024).view(np.float16)
    for x in (wild, tame):
        got = hif4.hif4_quantize(torch.from_numpy(x.copy()).cuda(), mode).cpu().numpy()
        _compare_units(got, oracle.quantize(x, mode, nthreads=8), f"fp16 bits mode {mode}")
    # strided source: columns [64, 64 + 320) of a wider tensor, guard band around the output
    wide = torch.from_numpy(tame.copy()).cuda()
    view = wide[:37, 64:384]
    out = torch.full((39, 5, 36), 0xAB, dtype=torch.uint8, device="cuda")
    hif4.hif4_quantize(view, mode, out=out[1:38])
    _compare_units(out[1:38].cpu().numpy(), oracle.quantize(np.ascontiguousarray(tame[:37, 64:384]), mode), "fp16 strided")
    assert (out[0] == 0xAB).all() and (out[38] == 0xAB).all()
    with pytest.raises(hif4.Hif4Error):
        hif4.hif4_dequantize(out[1:38].contiguous(), dtype=torch.float16)     # FP16 is a source type only
    # hif4_linear on FP16 activations = quantize + GEMM
    g = torch.Generator(device="cuda"); g.manual_seed(9 + mode)
    x16 = torch.randn(24, 512, generator=g, device="cuda").to(torch.float16)
    w = hif4.hif4_quantize((torch.randn(96, 512, generator=g, device="cuda") * 0.05).to(torch.bfloat16))
    y = hif4.hif4_linear(x16, w, mode=mode)
    assert torch.equal(y, hif4.hif4_gemm(hif4.hif4_quantize(x16, mode), w))


@pytest.mark.parametrize("mode", [0, 1])
def test_quantize_transposed_is_quantize_of_the_transpose(hif4, mode):
    """Units down the columns: bit-identical to the oracle's Algorithm 1 on the transposed matrix, for ragged column
    counts, a strided source, random bit patterns (NaN and Inf included) and the workload mix."""
    rng = np.random.default_rng(500 + mode)
    cases = []
    for (rows, cols) in ((64, 8), (128, 72), (192, 136), (640, 1000), (1024, 2048), (448, 264)):
        expo = rng.integers(100, 150, size=(1, cols), dtype=np.uint32)                 # per column: base exponent
        mant = rng.integers(0, 1 << 7, size=(rows, cols), dtype=np.uint32)
        sign = rng.integers(0, 2, size=(rows, cols), dtype=np.uint32) << 15
        spread = rng.integers(0, 7, size=(rows, cols), dtype=np.uint32)
        cases.append((sign | ((expo - spread) << 7) | mant).astype(np.uint16))
    cases.append(rng.integers(0, 1 << 16, size=(256, 512), dtype=np.uint32).astype(np.uint16))      # every kind of value
    cases.append(wl.bf16_to_u16_numpy(wl.quantize_sweep(2 ** 20, device="cuda")))                   # [256, 4096] workload mix
    for bits in cases:
        rows, cols = bits.shape
        x = wl.u16_numpy_to_bf16(bits, "cuda")
        out = torch.full((cols + 2, rows // 64, 36), 0xCD, dtype=torch.uint8, device="cuda")
        hif4.hif4_quantize_transposed(x, mode, out=out[1:cols + 1])
        want = oracle.quantize(np.ascontiguousarray(bits.T), mode, nthreads=8)
        _compare_units(out[1:cols + 1].cpu().numpy(), want, f"transposed {rows}x{cols} mode {mode}")
        assert (out[0] == 0xCD).all() and (out[cols + 1] == 0xCD).all()
        assert torch.equal(out[1:cols + 1], hif4.hif4_quantize(x.t().contiguous(), mode)), "differs from quantizing the transpose"
    # strided source
    wide = wl.u16_numpy_to_bf16(cases[3], "cuda")
    view = wide[:, 8:808]
    got = hif4.hif4_quantize_transposed(view, mode).cpu().numpy()
    _compare_units(got, oracle.quantize(np.ascontiguousarray(cases[3][:, 8:808].T), mode, nthreads=8), "transposed, strided")
    # argument checks
    with pytest.raises(hif4.Hif4Error) as ei:
        hif4.hif4_quantize_transposed(torch.zeros(100, 64, dtype=torch.bfloat16, device="cuda"))
    assert ei.value.code == 2                                                                      # rows % 64
    with pytest.raises(hif4.Hif4Error) as ei:
        hif4.hif4_quantize_transposed(torch.zeros(64, 60, dtype=torch.float32, device="cuda"))
    assert ei.value.code == 2                                                                      # cols % 8
    assert hif4.hif4_quantize_transposed(torch.zeros(0, 64, dtype=torch.bfloat16, device="cuda")).shape == (64, 0, 36)
    assert hif4.hif4_last_device_status() == 0


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("dtype", [torch.float32, torch.float16])
def test_quantize_transposed_fp32_and_fp16_sources(hif4, mode, dtype):
    """Units down the columns of FP32 and FP16 matrices: bit-identical to the oracle's P = FP32 steps on the
    transposed matrix (ragged column counts, a strided source, special values, values between BF16 neighbours)."""
    rng = np.random.default_rng(900 + mode)
    np_dt = np.float32 if dtype == torch.float32 else np.float16
    cases = []
    for (rows, cols) in ((64, 8), (128, 72), (192, 136), (640, 1000), (512, 2048), (448, 264)):
        scale = np.exp2(rng.integers(-12, 12, size=(1, cols))) if dtype == torch.float32 else np.exp2(rng.integers(-6, 6, size=(1, cols)))
        x = rng.standard_normal((rows, cols)) * scale * np.exp2(-rng.integers(0, 6, size=(rows, cols)))
        cases.append(x.astype(np_dt))
    special = rng.standard_normal((256, 256)).astype(np_dt)
    special[5, 7] = np.nan; special[70, 9] = np.inf; special[130, 11] = -np.inf; special[:, 13] = 0.0
    special[64:128, 15] = -0.0; special[3, 17] = np.finfo(np_dt).max; special[200, 19] = np.finfo(np_dt).tiny / 4
    cases.append(special)
    for x_np in cases:
        rows, cols = x_np.shape
        x = torch.from_numpy(x_np).cuda()
        out = torch.full((cols + 2, rows // 64, 36), 0xCD, dtype=torch.uint8, device="cuda")
        hif4.hif4_quantize_transposed(x, mode, out=out[1:cols + 1])
        want = oracle.quantize(np.ascontiguousarray(x_np.T), mode, nthreads=8)
        _compare_units(out[1:cols + 1].cpu().numpy(), want, f"transposed {dtype} {rows}x{cols} mode {mode}")
        assert (out[0] == 0xCD).all() and (out[cols + 1] == 0xCD).all()
        assert torch.equal(out[1:cols + 1], hif4.hif4_quantize(x.t().contiguous(), mode)), "differs from quantizing the transpose"
    wide = torch.from_numpy(cases[3]).cuda()
    got = hif4.hif4_quantize_transposed(wide[:, 8:808], mode).cpu().numpy()
    _compare_units(got, oracle.quantize(np.ascontiguousarray(cases[3][:, 8:808].T), mode, nthreads=8), "transposed, strided")
    assert hif4.hif4_last_device_status() == 0
