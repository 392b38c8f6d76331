"""GPU parity for hif4_gemm / hif4_grouped_gemm through the C ABI:
max |C_gpu - C_ref| <= 1e-5 * sum_k |a_ik| |b_jk| against the FP64 oracle on the decoded operands."""
import numpy as np
import pytest
import torch

import hif4_workloads as wl
import oracle
from tests.kernel_choice import tokens_stay_in_shared_memory

pytestmark = pytest.mark.gpu
TOL = 1e-5


@pytest.fixture(scope="module")
def hif4():
    assert torch.cuda.is_available()
    import paper_2602_11287_b200 as lib
    return lib


def check_full(hif4, a_units, b_units, what, out=None):
    C = hif4.hif4_gemm(a_units, b_units, out=out)
    ref, refabs = oracle.gemm_f64(a_units.cpu().numpy(), b_units.cpu().numpy(), nthreads=8)
    got = C.cpu().numpy().astype(np.float64)
    err = np.abs(got - ref)
    bound = TOL * refabs
    assert np.all(err <= bound + 1e-300), f"{what}: worst ratio {np.max(err / np.maximum(bound, 1e-300)):.3g}"
    return C


def check_sampled(hif4, a_units, b_units, what, n=600, seed=0, C=None):
    if C is None:
        C = hif4.hif4_gemm(a_units, b_units)
    M, N = C.shape
    rng = np.random.default_rng(seed)
    rows = np.concatenate([rng.integers(0, M, n), [0, M - 1, 0, M - 1]])
    cols = np.concatenate([rng.integers(0, N, n), [0, 0, N - 1, N - 1]])
    ref, refabs = oracle.gemm_sampled_f64(a_units.cpu().numpy(), b_units.cpu().numpy(), rows, cols)
    got = C[torch.from_numpy(rows).cuda(), torch.from_numpy(cols).cuda()].cpu().numpy().astype(np.float64)
    err = np.abs(got - ref)
    assert np.all(err <= TOL * refabs + 1e-300), f"{what}: worst ratio {np.max(err / np.maximum(TOL * refabs, 1e-300)):.3g}"
    return C


def test_single_layer_config(hif4):
    x, w = wl.single_layer(device="cuda")
    check_full(hif4, hif4.hif4_quantize(x), hif4.hif4_quantize(w), "cfg1 128x512x512")


@pytest.mark.parametrize("M,N,K", [(1, 64, 64), (1, 1, 64), (3, 5, 128), (64, 64, 64), (65, 63, 192), (130, 257, 320),
                                   (16, 200, 1024), (200, 16, 256), (129, 300, 768), (257, 513, 256)])
def test_small_and_ragged_shapes(hif4, M, N, K):
    g = torch.Generator(device="cuda"); g.manual_seed(M * 1000 + N)
    a = torch.randn(M, K, generator=g, device="cuda").to(torch.bfloat16)
    b = (torch.randn(N, K, generator=g, device="cuda") * 0.05).to(torch.bfloat16)
    check_full(hif4, hif4.hif4_quantize(a), hif4.hif4_quantize(b), f"{M}x{N}x{K}")


@pytest.mark.parametrize("M,N,K", [(33, 300, 256), (40, 257, 768), (100, 1000, 1024), (128, 512, 2048), (65, 31, 256),
                                   (40, 500, 4096), (100, 1000, 2048), (128, 4096, 4096), (64, 2100, 3072)])
def test_few_rows_default_path(hif4, M, N, K):
    """33 <= M <= 128 with K % 256 == 0 goes to the CTA-pair kernel with swapped operands; with few weight tiles and a
    long K every tile is cut into up to four K slices that are added in slice order (the last four shapes)."""
    g = torch.Generator(device="cuda"); g.manual_seed(M * 13 + N)
    a = hif4.hif4_quantize(torch.randn(M, K, generator=g, device="cuda").to(torch.bfloat16))
    b = hif4.hif4_quantize((torch.randn(N, K, generator=g, device="cuda") * 0.05).to(torch.bfloat16))
    out = torch.full((M + 2, N + 5), -5.0, dtype=torch.float32, device="cuda")
    before = hif4.launch_count()
    C = check_full(hif4, a, b, f"few rows {M}x{N}x{K}", out=out[1:M + 1, 2:N + 2])
    assert hif4.launch_count() - before == 1
    assert (out[0] == -5.0).all() and (out[M + 1] == -5.0).all() and (out[:, :2] == -5.0).all() and (out[:, N + 2:] == -5.0).all()
    assert torch.equal(C.contiguous(), hif4.hif4_gemm(a, b)), "two runs differ"
    assert hif4.hif4_last_device_status() == 0


def test_random_units_all_scales_and_strided_c(hif4):
    rng = np.random.default_rng(21)
    M, N, upr = 70, 90, 4
    A = rng.integers(0, 256, (M, upr, 36), dtype=np.uint8)
    B = rng.integers(0, 256, (N, upr, 36), dtype=np.uint8)
    A[..., 0] = rng.integers(0x60, 0xE0, (M, upr)); B[..., 0] = rng.integers(0x60, 0xE0, (N, upr))
    out = torch.full((M, 96), -5.0, dtype=torch.float32, device="cuda")
    check_full(hif4, torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda(), "random units", out=out[:, :N])
    assert (out[:, N:] == -5.0).all()


@pytest.mark.parametrize("M,N,ld,K", [(300, 90, 96, 256), (300, 257, 260, 512), (513, 258, 260, 256), (300, 259, 260, 256),
                                      (70, 90, 96, 256), (128, 1030, 1032, 1024), (16, 90, 96, 256), (2500, 1298, 1300, 1280),
                                      (1000, 4098, 4100, 512), (70, 24, 28, 256), (100, 8, 8, 512), (128, 36, 40, 256),
                                      (300, 8, 12, 256)])
def test_c_inside_a_wider_buffer_with_a_column_count_that_is_not_a_multiple_of_four(hif4, M, N, ld, K):
    """C as the left columns of a wider, 16-byte aligned buffer (ldc % 4 == 0) with N % 4 != 0: a store path that clips
    in 16-byte pieces would write the columns between N and the next multiple of four.  Nothing right of column N may
    change, on any kernel (pair kernel with whole and shared tiles, swapped pair kernel, weight streaming).  The last
    shapes have fewer columns than the store boxes are wide."""
    g = torch.Generator(device="cuda"); g.manual_seed(M + N)
    a = hif4.hif4_quantize(torch.randn(M, K, generator=g, device="cuda").to(torch.bfloat16))
    b = hif4.hif4_quantize((torch.randn(N, K, generator=g, device="cuda") * 0.05).to(torch.bfloat16))
    out = torch.full((M + 2, ld), -5.0, dtype=torch.float32, device="cuda")
    check_full(hif4, a, b, f"{M}x{N} in a buffer of {ld} columns", out=out[1:M + 1, :N])
    assert (out[:, N:] == -5.0).all() and (out[0] == -5.0).all() and (out[M + 1] == -5.0).all()
    assert hif4.hif4_last_device_status() == 0


def test_grouped_c_inside_a_wider_buffer_with_a_column_count_that_is_not_a_multiple_of_four(hif4):
    rng = np.random.default_rng(23)
    counts = [300, 0, 17, 64, 130]
    total, N, ld, upr = sum(counts), 90, 96, 4
    A = rng.integers(0, 256, (total, upr, 36), dtype=np.uint8)
    B = rng.integers(0, 256, (len(counts), N, upr, 36), dtype=np.uint8)
    A[..., 0] = rng.integers(0x60, 0xE0, (total, upr)); B[..., 0] = rng.integers(0x60, 0xE0, (len(counts), N, upr))
    off_h = np.concatenate([[0], np.cumsum(counts)]).astype(np.int64)
    out = torch.full((total + 2, ld), -5.0, dtype=torch.float32, device="cuda")
    C = hif4.hif4_grouped_gemm(torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda(), torch.from_numpy(off_h).cuda(),
                               out=out[1:total + 1, :N])
    ref, refabs = oracle.grouped_gemm_f64(A, B, off_h, nthreads=8)
    assert np.all(np.abs(C.cpu().numpy().astype(np.float64) - ref) <= TOL * refabs + 1e-300)
    assert (out[:, N:] == -5.0).all() and (out[0] == -5.0).all() and (out[total + 1] == -5.0).all()


def test_nan_units_and_determinism(hif4):
    rng = np.random.default_rng(22)
    A = rng.integers(0, 256, (66, 4, 36), dtype=np.uint8); A[..., 0] = 0xC0
    B = rng.integers(0, 256, (70, 4, 36), dtype=np.uint8); B[..., 0] = 0xB0
    A[5, 2, 0] = 0xFF
    B[69, 0, 0] = 0xFF
    a, b = torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda()
    C = hif4.hif4_gemm(a, b)
    nan = torch.isnan(C).cpu().numpy()
    want = np.zeros((66, 70), bool); want[5, :] = True; want[:, 69] = True
    assert np.array_equal(nan, want)
    C2 = hif4.hif4_gemm(a, b)
    assert torch.equal(torch.nan_to_num(C), torch.nan_to_num(C2)), "two runs differ"


def test_llama_shapes_sampled(hif4):
    for (name, K, N) in wl.LLAMA3_8B_LINEARS:
        w = hif4.hif4_quantize(wl.gaussian(N, K, 0.02, seed=2000 + N + K, device="cuda"))
        for M in (1, 16, 512):
            x = hif4.hif4_quantize(wl.llama_activations(M, K, device="cuda"))
            check_sampled(hif4, x, w, f"llama {name} M={M}", n=300)


def test_empty_and_bad_arguments(hif4):
    a = torch.zeros(0, 2, 36, dtype=torch.uint8, device="cuda")
    b = torch.zeros(5, 2, 36, dtype=torch.uint8, device="cuda")
    assert hif4.hif4_gemm(a, b).shape == (0, 5)
    a = torch.zeros(3, 0, 36, dtype=torch.uint8, device="cuda")
    b = torch.zeros(5, 0, 36, dtype=torch.uint8, device="cuda")
    out = torch.ones(3, 8, dtype=torch.float32, device="cuda")
    hif4.hif4_gemm(a, b, out=out[:, :5])          # K == 0: zero fill of the [M, N] window only
    assert (out[:, :5] == 0).all() and (out[:, 5:] == 1).all()
    import ctypes
    n = ctypes.c_size_t(0)
    assert hif4.lib.hif4_gemm_workspace(4, 4, 100, ctypes.byref(n)) == 2
    assert hif4.lib.hif4_gemm(None, None, None, 4, 4, 64, 4, None, 0, None) == 1
    c = torch.zeros(4, 6, dtype=torch.float32, device="cuda")
    au = torch.zeros(4, 1, 36, dtype=torch.uint8, device="cuda")
    assert hif4.lib.hif4_gemm(au.data_ptr() + 2, au.data_ptr(), c.data_ptr(), 4, 4, 64, 6, None, 0, None) == 3   # A % 4
    assert hif4.lib.hif4_gemm(au.data_ptr(), au.data_ptr(), c.data_ptr(), 4, 4, 64, 2, None, 0, None) == 2   # ldc < N


def _grouped_case(hif4, counts, N, K, seed):
    g = torch.Generator(device="cuda"); g.manual_seed(seed)
    G = len(counts)
    off = torch.zeros(G + 1, dtype=torch.int64)
    off[1:] = torch.cumsum(torch.tensor(counts), 0)
    total = int(off[-1])
    a = hif4.hif4_quantize(torch.randn(max(total, 1), K, generator=g, device="cuda").to(torch.bfloat16))[:total]
    b = hif4.hif4_quantize((torch.randn(G * N, K, generator=g, device="cuda") * 0.02).to(torch.bfloat16)).view(G, N, K // 64, 36)
    out = torch.full((total, N), 3.0, dtype=torch.float32, device="cuda")
    if total:
        hif4.hif4_grouped_gemm(a, b, off.cuda(), out=out)
    ref, refabs = oracle.grouped_gemm_f64(a.cpu().numpy(), b.cpu().numpy(), off.numpy(), nthreads=8)
    err = np.abs(out.cpu().numpy().astype(np.float64) - ref)
    assert np.all(err <= TOL * refabs + 1e-300)


def test_grouped_gemm_with_empty_and_ragged_groups(hif4):
    _grouped_case(hif4, [3, 0, 70, 1, 0, 129, 64, 0], N=96, K=256, seed=31)
    _grouped_case(hif4, [0, 0, 5], N=64, K=64, seed=32)
    _grouped_case(hif4, [200], N=130, K=512, seed=33)


def test_grouped_gemm_small_and_large_token_tiles_odd_weight_tile_count(hif4):
    """Token tiles of at most 64 rows take two weight tiles per work record, larger ones one: groups on both sides of
    that limit (64 / 65 rows, a 256 + 40 row group whose last tile is small, single rows, empty groups), with three
    weight tiles (the last record of a small tile has no second weight tile and must not touch the next group's rows)
    and with four, over several K chunks.  Every entry against the oracle; the guard value around C stays."""
    for (N, K, seed) in ((700, 768, 51), (1024, 512, 52), (257, 256, 53)):
        _grouped_case(hif4, [64, 65, 0, 296, 1, 33, 0, 130, 32], N=N, K=K, seed=seed)


def test_grouped_gemm_moe_routing_sampled(hif4):
    r = wl.moe_routing(tokens=512, experts=32, topk=4, device="cuda")
    off = r["offsets"]
    total = int(off[-1])
    K, N, G = 512, 256, 32
    a = hif4.hif4_quantize(wl.outlier_channel_activations(total, K, seed=41, device="cuda"))
    b = hif4.hif4_quantize(wl.gaussian(G * N, K, 0.02, seed=42, device="cuda")).view(G, N, K // 64, 36)
    out = hif4.hif4_grouped_gemm(a, b, off)
    ref, refabs = oracle.grouped_gemm_f64(a.cpu().numpy(), b.cpu().numpy(), off.cpu().numpy(), nthreads=8)
    err = np.abs(out.cpu().numpy().astype(np.float64) - ref)
    assert np.all(err <= TOL * refabs + 1e-300)


def test_grouped_gemm_many_small_groups_wide_n(hif4):
    """Many experts with few rows and a wide N (8192 rows, 140 groups of 1..130 rows + empty ones, N = 8192 + 40:
    33 weight tiles per token tile, the last one ragged): thousands of small work units per launch.  Compared
    entry by entry with the single-CTA kernel, and sampled against the oracle."""
    rng = np.random.default_rng(77)
    sizes = list(rng.integers(1, 131, 140))
    sizes[5] = 0; sizes[60] = 0
    sizes[-1] += 8192 - sum(sizes) if sum(sizes) < 8192 else 0
    G, K, N = len(sizes), 256, 8192 + 40
    off = torch.tensor(np.concatenate([[0], np.cumsum(sizes)]), dtype=torch.int64, device="cuda")
    total = int(off[-1])
    g = torch.Generator(device="cuda"); g.manual_seed(78)
    a = hif4.hif4_quantize(torch.randn(total, K, generator=g, device="cuda").to(torch.bfloat16))
    b = hif4.hif4_quantize((torch.randn(G * N, K, generator=g, device="cuda") * 0.05).to(torch.bfloat16)).view(G, N, K // 64, 36)
    out = hif4.hif4_grouped_gemm(a, b, off)
    assert torch.equal(out, hif4.hif4_grouped_gemm(a, b, off)), "two runs differ"
    hif4.hif4_debug_set_gemm_path(2)
    try:
        ref1 = hif4.hif4_grouped_gemm(a, b, off)
    finally:
        hif4.hif4_debug_set_gemm_path(0)
    assert (out - ref1).abs().max().item() <= 1e-5 * K * ref1.abs().max().item()
    off_h = off.cpu().numpy()
    for gsel in (0, 7, 60, 61, G - 1):
        lo, hi = int(off_h[gsel]), int(off_h[gsel + 1])
        if hi > lo:
            check_sampled(hif4, a[lo:hi], b[gsel], f"group {gsel}", n=400, seed=gsel, C=out[lo:hi])
    assert hif4.hif4_last_device_status() == 0


# ------------------------------------------------------------------ tensor-core (tcgen05) kernel
@pytest.fixture(params=[2, 3], ids=["one_cta", "cta_pair"])
def tc_path(hif4, request):
    """2 = single-CTA 128 x 256 kernel, 3 = CTA-pair 256 x 256 kernel, forced whatever the shape."""
    hif4.hif4_debug_set_gemm_path(request.param)
    yield hif4
    hif4.hif4_debug_set_gemm_path(0)
    assert hif4.hif4_last_device_status() == 0, "a bounded wait inside the kernel ran out"


@pytest.mark.parametrize("M,N,K", [(128, 256, 256), (128, 256, 512), (1, 64, 256), (130, 257, 768), (300, 700, 1024),
                                   (64, 2000, 256), (1000, 130, 2048), (256, 256, 256), (513, 385, 512),
                                   (2500, 1300, 1280)])
def test_tensor_core_kernel_full_compare(tc_path, M, N, K):
    hif4 = tc_path
    g = torch.Generator(device="cuda"); g.manual_seed(M * 7 + N)
    a = torch.randn(M, K, generator=g, device="cuda").to(torch.bfloat16)
    b = (torch.randn(N, K, generator=g, device="cuda") * 0.05).to(torch.bfloat16)
    before = hif4.launch_count()
    C = check_full(hif4, hif4.hif4_quantize(a), hif4.hif4_quantize(b), f"tc {M}x{N}x{K}")
    assert hif4.launch_count() - before == 3
    C2 = hif4.hif4_gemm(hif4.hif4_quantize(a), hif4.hif4_quantize(b))
    assert torch.equal(C, C2), "two runs of the tensor-core kernel differ"


def test_tensor_core_kernel_random_units_nan_and_guard_bands(tc_path):
    hif4 = tc_path
    rng = np.random.default_rng(51)
    M, N, upr = 150, 280, 8
    A = rng.integers(0, 256, (M, upr, 36), dtype=np.uint8)
    B = rng.integers(0, 256, (N, upr, 36), dtype=np.uint8)
    A[..., 0] = rng.integers(0x00, 0xFF, (M, upr)); B[..., 0] = rng.integers(0x40, 0xC0, (N, upr))
    A[77, 3, 0] = 0xFF
    B[279, 7, 0] = 0xFF
    out = torch.full((M + 2, 288), -5.0, dtype=torch.float32, device="cuda")
    a, b = torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda()
    C = hif4.hif4_gemm(a, b, out=out[1:M + 1, :N])
    ref, refabs = oracle.gemm_f64(A, B, nthreads=8)
    got = C.cpu().numpy().astype(np.float64)
    nan = np.isnan(ref)
    assert np.array_equal(np.isnan(got), nan)
    err = np.abs(got - ref)[~nan]
    assert np.all(err <= TOL * refabs[~nan] + 1e-300)
    assert (out[0] == -5.0).all() and (out[M + 1] == -5.0).all() and (out[:, N:] == -5.0).all()


def test_cta_pair_kernel_few_columns_in_the_last_tile_repeated(hif4):
    """A last column tile with 8 valid columns leaves 15 of its 16 staged slabs unused; the staging
    buffers of the TMA-store epilogue must not be reused while a store still reads them."""
    hif4.hif4_debug_set_gemm_path(3)
    try:
        for (M, N, K) in [(300, 520, 1024), (257, 264, 256), (512, 1032, 512)]:
            g = torch.Generator(device="cuda"); g.manual_seed(M + N + K)
            a = hif4.hif4_quantize(torch.randn(M, K, generator=g, device="cuda").to(torch.bfloat16))
            b = hif4.hif4_quantize((torch.randn(N, K, generator=g, device="cuda") * 0.05).to(torch.bfloat16))
            C = check_full(hif4, a, b, f"pair kernel {M}x{N}x{K}")
            for _ in range(20):
                assert torch.equal(C, hif4.hif4_gemm(a, b)), "runs differ"
    finally:
        hif4.hif4_debug_set_gemm_path(0)
    assert hif4.hif4_last_device_status() == 0


@pytest.mark.parametrize("M,N,K", [(2560, 2048, 16384), (2500, 2000, 8192), (19 * 256, 4 * 256 + 8, 8192), (2560, 2048, 2048),
                                   (512, 2048, 4096), (300, 1000, 2048), (2304, 4096, 256), (3000, 3000, 768),
                                   (130, 20000, 1024)])
def test_cta_pair_kernel_k_sliced_last_round(hif4, M, N, K):
    """More tiles than CTA pairs with a partial last round (80 and 95 tiles on 74 pairs): the K chunks of the last
    whole round and the partial one are dealt out in equal runs, so most of those tiles are computed by two pairs,
    the end of the tile stored first and the beginning added to it.  A single round with fewer tiles than half the
    pairs is cut into K slices that are added to C in slice order (16 tiles x 4, 8 tiles x 2)."""
    assert hif4.hif4_gemm_workspace(M, N, K) > 0, "the K-sliced round needs its completion words"
    g = torch.Generator(device="cuda"); g.manual_seed(M + N + K)
    a = hif4.hif4_quantize(torch.randn(M, K, generator=g, device="cuda").to(torch.bfloat16))
    b = hif4.hif4_quantize((torch.randn(N, K, generator=g, device="cuda") * 0.05).to(torch.bfloat16))
    out = torch.full((M + 2, N + 4), -3.0, dtype=torch.float32, device="cuda")
    C = check_sampled(hif4, a, b, f"k-sliced {M}x{N}x{K}", n=1500, seed=K, C=hif4.hif4_gemm(a, b, out=out[1:M + 1, :N]))
    assert (out[0] == -3.0).all() and (out[M + 1] == -3.0).all() and (out[:, N:] == -3.0).all()
    # every entry of the tail tiles against the kernel that never slices (different FP32 summation order)
    hif4.hif4_debug_set_gemm_path(2)
    try:
        C1 = hif4.hif4_gemm(a, b)
    finally:
        hif4.hif4_debug_set_gemm_path(0)
    scale = (C1.abs().max() + 1e-30).item()
    assert (C.contiguous() - C1).abs().max().item() <= 1e-5 * scale * K
    for _ in range(3):
        assert torch.equal(hif4.hif4_gemm(a, b), C.contiguous()), "K-sliced tiles are not reproducible"
    with pytest.raises(hif4.Hif4Error) as ei:
        hif4.hif4_gemm(a, b, workspace=torch.empty(64, dtype=torch.uint8, device="cuda"))
    assert ei.value.code == 5
    assert hif4.hif4_last_device_status() == 0


def test_cta_pair_kernel_random_shapes_against_the_single_cta_kernel(hif4):
    """Seeded random shapes around the schedule's case distinctions (fewer tiles than CTA pairs with and without K
    slices, whole rounds, a partial round balanced chunk by chunk, ragged edges, K of one to sixteen chunks): every
    entry against the single-CTA kernel, which never splits a tile, plus sampled entries against FP64."""
    rng = np.random.default_rng(20260211)
    shapes = [(int(rng.integers(129, 5000)), int(rng.integers(8, 5000)), 256 * int(rng.integers(1, 17))) for _ in range(14)]
    shapes += [(256 * 74, 256, 512), (256 * 37, 512, 768), (257, 256 * 74 + 8, 256)]      # exactly one and two rounds, one more tile
    for M, N, K in shapes:
        g = torch.Generator(device="cuda"); g.manual_seed(M * 7 + N * 3 + K)
        a = hif4.hif4_quantize(torch.randn(M, K, generator=g, device="cuda").to(torch.bfloat16))
        b = hif4.hif4_quantize((torch.randn(N, K, generator=g, device="cuda") * 0.05).to(torch.bfloat16))
        C = check_sampled(hif4, a, b, f"random shape {M}x{N}x{K}", n=300, seed=M + N)
        hif4.hif4_debug_set_gemm_path(2)
        try:
            C1 = hif4.hif4_gemm(a, b)
        finally:
            hif4.hif4_debug_set_gemm_path(0)
        scale = (C1.abs().max() + 1e-30).item()
        assert (C - C1).abs().max().item() <= 1e-5 * scale * K, (M, N, K)
    assert hif4.hif4_last_device_status() == 0


def test_tensor_core_kernel_c_rows_not_16_byte_aligned(tc_path):
    """ldc odd and a base that is only 4-byte aligned: the kernels fall back from vector / TMA stores."""
    hif4 = tc_path
    M, N, K = 300, 333, 512
    g = torch.Generator(device="cuda"); g.manual_seed(77)
    a = hif4.hif4_quantize(torch.randn(M, K, generator=g, device="cuda").to(torch.bfloat16))
    b = hif4.hif4_quantize((torch.randn(N, K, generator=g, device="cuda") * 0.05).to(torch.bfloat16))
    buf = torch.full((M + 2, N + 2), -5.0, dtype=torch.float32, device="cuda")
    check_full(hif4, a, b, "unaligned C", out=buf[1:M + 1, 1:N + 1])
    assert (buf[0] == -5.0).all() and (buf[M + 1] == -5.0).all() and (buf[:, 0] == -5.0).all() and (buf[:, N + 1] == -5.0).all()


def test_tensor_core_grouped(tc_path):
    """Path 2 = single-CTA kernel with 128-row tiles, path 3 = CTA pairs with swapped operands."""
    hif4 = tc_path
    _grouped_case(hif4, [3, 0, 70, 1, 0, 129, 64, 0, 300], N=300, K=256, seed=61)
    _grouped_case(hif4, [0, 0, 5], N=64, K=512, seed=62)
    _grouped_case(hif4, [513], N=256, K=256, seed=63)
    _grouped_case(hif4, [31, 32, 33, 255, 256, 257, 0, 16, 700], N=520, K=768, seed=64)
    _grouped_case(hif4, [1] * 40, N=257, K=256, seed=65)


def test_tensor_core_prefill_shape_sampled(tc_path):
    hif4 = tc_path
    K, N, M = 4096, 4096, 4096
    w = hif4.hif4_quantize(wl.gaussian(N, K, 0.02, seed=71, device="cuda"))
    x = hif4.hif4_quantize(wl.llama_activations(M, K, device="cuda"))
    check_sampled(hif4, x, w, "tc llama qo M=4096", n=400)


# ------------------------------------------------------------------ weight-streaming kernel (M <= 16)
@pytest.fixture()
def gemv_path(hif4):
    hif4.hif4_debug_set_gemm_path(4)
    yield hif4
    hif4.hif4_debug_set_gemm_path(0)
    assert hif4.hif4_last_device_status() == 0, "a bounded wait inside the kernel ran out"


@pytest.mark.parametrize("M,N,K", [(1, 1, 256), (1, 64, 256), (2, 33, 512), (7, 200, 1024), (8, 4096, 256), (9, 130, 768),
                                   (16, 1000, 2304), (16, 64, 4096), (5, 9475, 256), (3, 31, 5120), (12, 77, 14336),
                                   (1, 40003, 256), (16, 2376, 1024), (10, 1192, 512), (4, 19000, 256),
                                   (17, 300, 256), (32, 1000, 1024), (25, 4200, 512), (31, 77, 4096), (20, 14336, 256),
                                   (8, 300, 6144), (8, 300, 6400), (5, 14336, 4096), (1, 1030, 4096),
                                   (1, 300, 14336), (2, 300, 14336), (3, 200, 8192), (4, 200, 16384), (8, 300, 8192),
                                   (8, 300, 8448), (16, 300, 4096), (16, 300, 4352), (12, 14336, 4096), (1, 9, 65536)])
def test_weight_streaming_kernel_full_compare(gemv_path, M, N, K):
    hif4 = gemv_path
    g = torch.Generator(device="cuda"); g.manual_seed(M * 11 + N)
    a = hif4.hif4_quantize(torch.randn(M, K, generator=g, device="cuda").to(torch.bfloat16))
    b = hif4.hif4_quantize((torch.randn(N, K, generator=g, device="cuda") * 0.05).to(torch.bfloat16))
    assert hif4.hif4_gemm_workspace(M, N, K) >= (8 if M <= 8 else 16 if M <= 16 else 32) * K * 2   # the decoded tokens (or more, if another kernel for this shape needs more)
    before = hif4.launch_count()
    out = torch.full((M + 2, N + 3), -5.0, dtype=torch.float32, device="cuda")
    C = check_full(hif4, a, b, f"gemv {M}x{N}x{K}", out=out[1:M + 1, 1:N + 1])
    one_launch = tokens_stay_in_shared_memory(M, K)      # few tokens, short K: the streaming kernel decodes the tokens itself
    assert hif4.launch_count() - before == (1 if one_launch else 2), "token preparation + streaming kernel, or the latter alone"
    assert (out[0] == -5.0).all() and (out[M + 1] == -5.0).all() and (out[:, 0] == -5.0).all() and (out[:, N + 1:] == -5.0).all()
    C2 = hif4.hif4_gemm(a, b)
    assert torch.equal(C.contiguous(), C2), "two runs of the weight-streaming kernel differ"


def test_weight_streaming_kernel_random_units_and_nan(gemv_path):
    hif4 = gemv_path
    rng = np.random.default_rng(81)
    M, N, upr = 11, 150, 8
    A = rng.integers(0, 256, (M, upr, 36), dtype=np.uint8)
    B = rng.integers(0, 256, (N, upr, 36), dtype=np.uint8)
    A[..., 0] = rng.integers(0x00, 0xFF, (M, upr)); B[..., 0] = rng.integers(0x40, 0xC0, (N, upr))
    A[3, 5, 0] = 0xFF
    B[149, 0, 0] = 0xFF
    C = hif4.hif4_gemm(torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda())
    ref, refabs = oracle.gemm_f64(A, B, nthreads=8)
    got = C.cpu().numpy().astype(np.float64)
    nan = np.isnan(ref)
    assert nan[3].all() and nan[:, 149].all() and np.array_equal(np.isnan(got), nan)
    assert np.all(np.abs(got - ref)[~nan] <= TOL * refabs[~nan] + 1e-300)


@pytest.fixture()
def fp8_path(hif4):
    """5 = the weight-streaming kernel on Eq. 3's factorisation: E4M3 operands, level-1 scales per unit pair."""
    hif4.hif4_debug_set_gemm_path(5)
    yield hif4
    hif4.hif4_debug_set_gemm_path(0)
    assert hif4.hif4_last_device_status() == 0, "a bounded wait inside the kernel ran out"


@pytest.mark.parametrize("M,N,K", [(1, 1, 256), (2, 33, 512), (7, 200, 1024), (8, 4096, 256), (9, 130, 768), (16, 1000, 2304),
                                   (3, 31, 5120), (12, 77, 14336), (1, 40003, 256), (17, 300, 256), (32, 1000, 1024),
                                   (25, 4200, 512), (5, 14336, 4096)])
def test_fp8_operand_kernel_full_compare(fp8_path, M, N, K):
    """Section III-B's flow (small signed operands, one scale product per unit pair) on tensor-core FP8 operands gives
    the product within the same tolerance as the kernels that fold the level-1 scale into BF16 operands."""
    hif4 = fp8_path
    g = torch.Generator(device="cuda"); g.manual_seed(M * 11 + N)
    a = hif4.hif4_quantize(torch.randn(M, K, generator=g, device="cuda").to(torch.bfloat16))
    b = hif4.hif4_quantize((torch.randn(N, K, generator=g, device="cuda") * 0.05).to(torch.bfloat16))
    before = hif4.launch_count()
    out = torch.full((M + 2, N + 3), -5.0, dtype=torch.float32, device="cuda")
    C = check_full(hif4, a, b, f"fp8 gemv {M}x{N}x{K}", out=out[1:M + 1, 1:N + 1])
    assert hif4.launch_count() - before == 2, "token preparation + streaming kernel"
    assert (out[0] == -5.0).all() and (out[M + 1] == -5.0).all() and (out[:, 0] == -5.0).all() and (out[:, N + 1:] == -5.0).all()
    assert torch.equal(C.contiguous(), hif4.hif4_gemm(a, b)), "two runs differ"


def test_fp8_operand_kernel_random_units_and_nan(fp8_path):
    hif4 = fp8_path
    rng = np.random.default_rng(82)
    M, N, upr = 11, 150, 8
    A = rng.integers(0, 256, (M, upr, 36), dtype=np.uint8)
    B = rng.integers(0, 256, (N, upr, 36), dtype=np.uint8)
    A[..., 0] = rng.integers(0x00, 0xFF, (M, upr)); B[..., 0] = rng.integers(0x40, 0xC0, (N, upr))
    A[3, 5, 0] = 0xFF
    B[149, 0, 0] = 0xFF
    C = hif4.hif4_gemm(torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda())
    ref, refabs = oracle.gemm_f64(A, B, nthreads=8)
    got = C.cpu().numpy().astype(np.float64)
    nan = np.isnan(ref)
    assert nan[3].all() and nan[:, 149].all() and np.array_equal(np.isnan(got), nan)
    assert np.all(np.abs(got - ref)[~nan] <= TOL * refabs[~nan] + 1e-300)


def test_weight_streaming_kernel_needs_its_workspace(gemv_path):
    hif4 = gemv_path
    a = torch.zeros(4, 4, 36, dtype=torch.uint8, device="cuda")
    b = torch.zeros(64, 4, 36, dtype=torch.uint8, device="cuda")
    c = torch.zeros(4, 64, dtype=torch.float32, device="cuda")
    before = hif4.launch_count()
    assert hif4.lib.hif4_gemm(a.data_ptr(), b.data_ptr(), c.data_ptr(), 4, 64, 256, 64, None, 0, None) == 5
    ws = torch.empty(1024, dtype=torch.uint8, device="cuda")
    assert hif4.lib.hif4_gemm(a.data_ptr(), b.data_ptr(), c.data_ptr(), 4, 64, 256, 64, ws.data_ptr(), 1024, None) == 5
    assert hif4.launch_count() == before


# ------------------------------------------------------------------ exactness of the in-kernel decoders
def _exhaustive_units(K):
    """Rows of K/64 units covering every E6M2 byte below NaN x both values of both micro-exponents x all
    16 codes at every position parity: row r uses byte r % 255, unit u the micro-exponent pattern u % 4,
    element i the code (i + r + u) % 16 (so each code meets each (byte, e8, e16) at many positions)."""
    upr = K // 64
    rows = 255 * 2
    A = np.zeros((rows, upr, 36), dtype=np.uint8)
    for r in range(rows):
        for u in range(upr):
            pat = (u + r // 255) % 4
            meta = (r % 255) | ((0xFF if pat & 1 else 0) << 8) | ((0xFFFF if pat & 2 else 0) << 16)
            if u % 5 == 4:                       # mixed micro-exponents inside one unit
                meta = (r % 255) | (0xA5 << 8) | (0x3C5A << 16)
            A[r, u, 0:4] = np.frombuffer(np.uint32(meta).tobytes(), dtype=np.uint8)
            codes = (np.arange(64) + r + u) % 16
            A[r, u, 4:] = (codes[0::2] | (codes[1::2] << 4)).astype(np.uint8)
    return A


def _one_hot_units(K):
    """K rows; row j decodes to 1.0 at position j and 0 elsewhere (E6M2 = 1.0, code 4 = 1.00)."""
    upr = K // 64
    B = np.zeros((K, upr, 36), dtype=np.uint8)
    B[:, :, 0] = 0xC0
    for j in range(K):
        B[j, j // 64, 4 + (j % 64) // 2] = 4 << (4 * (j % 2))
    return B


@pytest.mark.parametrize("path,rows", [(1, 510), (2, 510), (3, 510), (0, 100), (4, 16), (4, 7), (5, 16), (5, 7)])
def test_every_code_under_every_scale_passes_through_the_gemm_exactly(hif4, path, rows):
    """C = A * B^T with one-hot rows in B returns the decoded elements of A themselves: each in-kernel
    decoder (CUDA cores, single CTA, CTA pair, swapped pair for few rows, weight streaming) must give
    exactly the values of Eq. 2, as A operand and as B operand."""
    K = 256
    A_all = _exhaustive_units(K)
    Bh = _one_hot_units(K)
    want_all = oracle.dequantize(A_all, oracle.FP32)
    assert np.array_equal(oracle.dequantize(Bh, oracle.FP32), np.eye(K, dtype=np.float32))
    hif4.hif4_debug_set_gemm_path(path)
    try:
        for start in range(0, A_all.shape[0], rows):
            A = A_all[start:start + rows]
            a, b = torch.from_numpy(A).cuda(), torch.from_numpy(Bh).cuda()
            got = hif4.hif4_gemm(a, b).cpu().numpy()                       # exhaustive units as the A operand
            assert np.array_equal(got.view(np.uint32) & 0x7FFFFFFF, want_all[start:start + rows].view(np.uint32) & 0x7FFFFFFF)
            nz = want_all[start:start + rows] != 0                           # sign of zero products is not defined by Eq. 3
            assert np.array_equal(np.signbit(got)[nz], np.signbit(want_all[start:start + rows])[nz])
            if path in (4, 5):                                               # (the streaming kernels take few rows only)
                continue
            got_t = hif4.hif4_gemm(b, a).cpu().numpy()                     # and as the B operand
            assert np.array_equal(np.abs(got_t.T), np.abs(want_all[start:start + rows]))
    finally:
        hif4.hif4_debug_set_gemm_path(0)
    assert hif4.hif4_last_device_status() == 0


@pytest.mark.parametrize("M,N,K,dtype", [(1, 300, 512, torch.bfloat16), (16, 64, 256, torch.float32), (70, 257, 768, torch.bfloat16),
                                          (300, 520, 1024, torch.bfloat16), (5, 33, 192, torch.bfloat16)])
def test_linear_is_quantize_then_gemm(hif4, M, N, K, dtype):
    """hif4_linear (one call for the W4A4 layer) gives the bits of the two separate calls, and those are
    within tolerance of the FP64 reference on the oracle's encodings."""
    g = torch.Generator(device="cuda"); g.manual_seed(M + N + K)
    x = torch.randn(M, K, generator=g, device="cuda").to(dtype)
    w = hif4.hif4_quantize((torch.randn(N, K, generator=g, device="cuda") * 0.05).to(torch.bfloat16))
    y = hif4.hif4_linear(x, w)
    xq = hif4.hif4_quantize(x)
    assert torch.equal(y, hif4.hif4_gemm(xq, w))
    src = wl.bf16_to_u16_numpy(x) if dtype == torch.bfloat16 else x.cpu().numpy()
    ref, refabs = oracle.gemm_f64(oracle.quantize(src), w.cpu().numpy(), nthreads=8)
    assert np.all(np.abs(y.cpu().numpy().astype(np.float64) - ref) <= TOL * refabs + 1e-300)
    assert hif4.lib.hif4_linear(x.data_ptr(), 0, K, w.data_ptr(), y.data_ptr(), M, N, K, N, 0, None, 0, None) == 5


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32, torch.float16])
@pytest.mark.parametrize("M,N,K", [(1, 4096, 4096), (16, 1000, 1024), (7, 260, 256), (9, 64, 2304), (16, 14336, 4096),
                                   (24, 520, 1024), (32, 64, 256), (2, 520, 14336), (3, 300, 8192), (13, 300, 4096),
                                   (2, 300, 4096), (3, 260, 2048), (1, 130, 14336)])
def test_linear_with_few_rows_quantizes_inside_the_token_preparation(hif4, M, N, K, dtype, mode):
    """M <= 32 rows of activations: hif4_linear runs two kernels (quantize-and-decode of the tokens, weight
    streaming) instead of three -- a single one for a few BF16 rows of moderate length -- and gives exactly the bits
    of hif4_quantize followed by hif4_gemm, on a strided source with spikes, a NaN and an Inf, for every source type
    and both rounding modes."""
    g = torch.Generator(device="cuda"); g.manual_seed(M * 3 + N + K + mode)
    wide = torch.randn(M, K + 64, generator=g, device="cuda").to(dtype)
    x = wide[:, 64:]                                      # row stride K + 64
    x[0, 5] = 1000.0
    if M > 2:
        x[1, 70] = float("nan")
        x[2, 129] = float("-inf")
    w = hif4.hif4_quantize((torch.randn(N, K, generator=g, device="cuda") * 0.05).to(torch.bfloat16))
    before = hif4.launch_count()
    y = hif4.hif4_linear(x, w, mode=mode)
    one_launch = dtype == torch.bfloat16 and tokens_stay_in_shared_memory(M, K, from_bf16=True)     # conversion, token decode and streaming in one kernel
    assert hif4.launch_count() - before == (1 if one_launch else 2)
    want = hif4.hif4_gemm(hif4.hif4_quantize(x, mode), w)
    assert torch.equal(y.view(torch.int32), want.view(torch.int32)), "fused token preparation differs from quantize + GEMM"
    assert hif4.hif4_last_device_status() == 0


@pytest.mark.parametrize("M,N,K", [(129, 300, 256), (300, 520, 1024), (1000, 257, 768), (513, 1024, 2048), (4096, 1024, 512)])
def test_linear_with_many_rows_can_convert_inside_the_pair_kernel(hif4, M, N, K):
    """M > 128 rows of BF16 activations, conversion forced into the CTA-pair kernel (the A-side decode threads run
    Algorithm 1 on the units they decode, once per column tile): one launch (plus the flag memset where tiles are
    split along K), and exactly the bits of hif4_quantize followed by hif4_gemm -- on a strided source with spikes,
    NaN and Inf rows and a ragged last row tile."""
    g = torch.Generator(device="cuda"); g.manual_seed(M + 7 * N + K)
    wide = torch.randn(M, K + 64, generator=g, device="cuda").to(torch.bfloat16)
    x = wide[:, 64:]                                      # row stride K + 64
    x[0, 5] = 1000.0
    x[M // 2, 70] = float("nan")
    x[M - 1, 129] = float("-inf")
    w = hif4.hif4_quantize((torch.randn(N, K, generator=g, device="cuda") * 0.05).to(torch.bfloat16))
    want = hif4.hif4_gemm(hif4.hif4_quantize(x), w)
    hif4.hif4_debug_set_gemm_path(6)
    try:
        before = hif4.launch_count()
        y = hif4.hif4_linear(x, w)
        assert hif4.launch_count() - before == 1, "conversion and GEMM in one kernel"
        y_rha = hif4.hif4_linear(x, w, mode=1)            # half-away rounding is not fused: two launches, same contract
    finally:
        hif4.hif4_debug_set_gemm_path(0)
    assert torch.equal(y.view(torch.int32), want.view(torch.int32)), "in-kernel conversion differs from quantize + GEMM"
    assert torch.equal(y_rha.view(torch.int32), hif4.hif4_gemm(hif4.hif4_quantize(x, 1), w).view(torch.int32))
    xq = oracle.quantize(wl.bf16_to_u16_numpy(x.contiguous()), nthreads=8)
    ref, refabs = oracle.gemm_f64(xq, w.cpu().numpy(), nthreads=8)
    got = y.cpu().numpy().astype(np.float64)
    nan = np.isnan(ref)
    assert np.array_equal(np.isnan(got), nan) and np.all(np.abs(got - ref)[~nan] <= TOL * refabs[~nan] + 1e-300)
    assert hif4.hif4_last_device_status() == 0


# ------------------------------------------------------------------ failure reporting
def test_a_bounded_wait_that_runs_out_is_reported_once_and_the_context_stays_usable(hif4):
    """A kernel waits, with the library's bounded-wait helper and a 1 ms budget, on an mbarrier that nobody arrives
    on (no copy or MMA in flight).  It gives up, raises the device error word and returns; the host reads
    HIF4_ERR_DEVICE_TIMEOUT (7) once, then HIF4_OK, and the next GEMM on the same context is correct."""
    assert hif4.hif4_last_device_status() == 0
    hif4.hif4_debug_wait_timeout(1_000_000)
    assert hif4.hif4_last_device_status() == 7
    assert hif4.status_string(7)
    assert hif4.hif4_last_device_status() == 0
    with pytest.raises(hif4.Hif4Error) as ei:
        hif4.hif4_debug_wait_timeout(10 ** 10)              # budgets beyond 0.1 s are refused, nothing is launched
    assert ei.value.code == 2
    x, w = wl.single_layer(device="cuda")
    check_full(hif4, hif4.hif4_quantize(x), hif4.hif4_quantize(w), "gemm after a reported timeout")
    assert hif4.hif4_last_device_status() == 0


def test_gemm_workspace_is_valid_under_every_path_override(hif4):
    """hif4_gemm_workspace reports one figure per shape that is enough whichever kernel the override selects."""
    g = torch.Generator(device="cuda"); g.manual_seed(77)
    try:
        for (M, N, K) in ((8, 520, 512), (100, 700, 1024), (300, 300, 2048)):
            a = hif4.hif4_quantize(torch.randn(M, K, generator=g, device="cuda").to(torch.bfloat16))
            b = hif4.hif4_quantize(torch.randn(N, K, generator=g, device="cuda").to(torch.bfloat16))
            hif4.hif4_debug_set_gemm_path(0)
            need = hif4.hif4_gemm_workspace(M, N, K)
            ws = torch.empty(max(need, 256), dtype=torch.uint8, device="cuda")
            ref, refabs = oracle.gemm_f64(a.cpu().numpy(), b.cpu().numpy(), nthreads=8)
            for path in (0, 1, 2, 3, 4, 5):
                hif4.hif4_debug_set_gemm_path(path)
                assert hif4.hif4_gemm_workspace(M, N, K) == need
                c = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
                rc = hif4.lib.hif4_gemm(a.data_ptr(), b.data_ptr(), c.data_ptr(), M, N, K, N, ws.data_ptr(), need, None)
                assert rc == 0, (M, N, K, path, rc)
                err = np.abs(c.cpu().numpy().astype(np.float64) - ref)
                assert np.all(err <= TOL * refabs + 1e-300), (M, N, K, path)
    finally:
        hif4.hif4_debug_set_gemm_path(0)


def test_grouped_gemm_refuses_row_counts_beyond_its_tile_table(hif4):
    off = torch.zeros(2, dtype=torch.int64, device="cuda")
    before = hif4.launch_count()
    rc = hif4.lib.hif4_grouped_gemm(off.data_ptr(), off.data_ptr(), off.data_ptr(), off.data_ptr(), 1, 2 ** 31, 64, 256, 64,
                                    None, 0, None)
    assert rc == 2 and hif4.launch_count() == before
    with pytest.raises(hif4.Hif4Error):
        hif4.hif4_grouped_gemm_workspace(1, 2 ** 31, 64, 256)
