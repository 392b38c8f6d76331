"""GPU parity for hif4_mse_roundtrip (the quantization-error study of Section III-A) through the C ABI: the FP32
image of every format is bit-identical to the oracle's, the FP64 error sum agrees to summation rounding, and the
study's ratios come out as the paper prints them."""
import numpy as np
import pytest
import torch

import hif4_workloads as wl
import oracle
from tests import paper_constants

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def hif4():
    assert torch.cuda.is_available()
    import paper_2602_11287_b200 as lib
    return lib


def _oracle_images(bits):
    """The four images of a BF16 tensor (uint16 bit patterns, 2-D) from the oracle, as float32."""
    xf = oracle.bf16_bits_to_f64(bits).astype(np.float32)
    flat = xf.reshape(-1)
    return xf, {
        0: oracle.dequantize(oracle.quantize(bits.reshape(1, -1), nthreads=8), oracle.FP32).reshape(xf.shape),
        1: oracle.mxfp4_roundtrip(flat).reshape(xf.shape),
        2: oracle.nvfp4_roundtrip(flat).reshape(xf.shape),
        3: oracle.nvfp4_roundtrip(flat, oracle.pts_gain(flat)).reshape(xf.shape),
    }


def _check_all_formats(hif4, x, what):
    bits = wl.bf16_to_u16_numpy(x)
    xf, want = _oracle_images(bits)
    for fmt in (0, 1, 2, 3):
        image, err = hif4.hif4_mse_roundtrip(x, fmt)
        got = image.cpu().numpy()
        assert np.array_equal(got.view(np.uint32), want[fmt].view(np.uint32)), \
            f"{what}, format {fmt}: {int((got.view(np.uint32) != want[fmt].view(np.uint32)).sum())} elements differ"
        ref = float(np.sum((want[fmt].astype(np.float64) - xf.astype(np.float64)) ** 2))
        assert abs(float(err.item()) - ref) <= 1e-12 * max(ref, 1e-300), (what, fmt, float(err.item()), ref)
        _, err_only = hif4.hif4_mse_roundtrip(x, fmt, want_image=False)          # error without an image buffer
        assert float(err_only.item()) == float(err.item())
    assert hif4.hif4_last_device_status() == 0


@pytest.mark.parametrize("xexp", [0, 9, 17])
def test_gaussian_matrices_of_the_study(hif4, xexp):
    g = torch.Generator(device="cuda"); g.manual_seed(300 + xexp)
    x = (torch.randn(1024, 1024, generator=g, device="cuda") * (0.01 * 2.0 ** xexp)).to(torch.bfloat16)
    _check_all_formats(hif4, x, f"sigma = 0.01 * 2^{xexp}")


def test_rounding_ties_saturation_zero_blocks_and_a_ragged_grid(hif4):
    """Values on the E2M1 ties under a scale of one, block peaks that saturate the E4M3 scale and the E2M1 element,
    all-zero and negative-zero blocks, E4M3-subnormal scales; 64 * 1237 elements, so the last thread blocks are partly idle."""
    rng = np.random.default_rng(5)
    x = rng.standard_normal((1237, 64)).astype(np.float32)
    ties = np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, 6.0, 7.5, 0.5, 3.0, -2.5, -0.25, 1.0, 4.0, -6.0], dtype=np.float32)
    x[0, :16] = ties; x[0, 16:32] = ties[::-1]; x[0, 32:] = 0.0
    x[1, :] = 0.0; x[1, 3] = -0.0
    x[2, :] = 1e-4; x[2, 7] = 3e-3                       # NVFP4 scales in the E4M3 subnormal range
    x[3, :] = 2.0 ** -30                                 # below E4M3: the direct cast flushes the block
    x[4, :] = 100.0; x[4, 0] = 3000.0; x[4, 17] = -40000.0   # scale saturation at 448
    x[5:9] *= 1000.0
    t = torch.from_numpy(x).to(torch.bfloat16).cuda()
    _check_all_formats(hif4, t, "edge cases")


def test_ratios_of_the_study(hif4, golden_dir):
    """HiF4 : NVFP4 (with per-tensor scaling) : MXFP4 = 1 : 1.32 : 1.89 on Gaussian 1024 x 1024 matrices."""
    paper = paper_constants.load(golden_dir)
    nv, mx = [], []
    for xexp in (0, 5, 9, 13, 17):
        g = torch.Generator(device="cuda"); g.manual_seed(900 + xexp)
        x = (torch.randn(1024, 1024, generator=g, device="cuda") * (0.01 * 2.0 ** xexp)).to(torch.bfloat16)
        errs = [float(hif4.hif4_mse_roundtrip(x, fmt, want_image=False)[1].item()) for fmt in (0, 1, 3)]
        nv.append(errs[2] / errs[0]); mx.append(errs[1] / errs[0])
    assert abs(np.mean(nv) - float(paper["mse_ratio_nvfp4"])) < 0.03, nv
    assert abs(np.mean(mx) - float(paper["mse_ratio_mxfp4"])) < 0.03, mx


def test_arguments(hif4):
    x = torch.zeros(100, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(hif4.Hif4Error) as ei:
        hif4.hif4_mse_roundtrip(x, 0)
    assert ei.value.code == 2                               # n % 64
    with pytest.raises(hif4.Hif4Error) as ei:
        hif4.hif4_mse_workspace(64, 7)
    assert ei.value.code == 4
    x = torch.zeros(128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(hif4.Hif4Error) as ei:
        hif4.hif4_mse_roundtrip(x, 1, workspace=torch.empty(256, dtype=torch.uint8, device="cuda"))
    assert ei.value.code == 5
    image, err = hif4.hif4_mse_roundtrip(x, 3)
    assert float(err.item()) == 0.0 and not image.any()
