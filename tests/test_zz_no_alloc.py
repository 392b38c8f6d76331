"""hif4_grouped_gemm_noalloc through the C ABI: the grouped GEMM for callers that cannot allocate device
memory (fixed memory plans, plug-ins without an allocator, sections where a cudaMalloc's device-wide
synchronisation is not acceptable).  Its tile table sits in a fixed array inside the library, so this
file checks that (a) it gives what hif4_grouped_gemm gives and what the CPU oracle's FP64 product gives, within
the GEMM tolerance, on two calls in a row that reuse the array with different group layouts, (b) problems that do not fit the array are refused, nothing launched.

Collected last on purpose (file name): if it fails, a run that stops at the first failure has already
run every other test."""
import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu
TOL = 1e-5          # the GEMM tolerance of the other GPU tests: |C - C_ref| <= TOL * sum_k |a||b|


@pytest.fixture(scope="module")
def hif4():
    assert torch.cuda.is_available()
    import paper_2602_11287_b200 as lib
    return lib


def _problem(hif4, counts, N, K, seed):
    g = torch.Generator(device="cuda"); g.manual_seed(seed)
    G = len(counts)
    off = torch.zeros(G + 1, dtype=torch.int64)
    off[1:] = torch.cumsum(torch.tensor(counts), 0)
    total = int(off[-1])
    a = hif4.hif4_quantize(torch.randn(total, K, generator=g, device="cuda").to(torch.bfloat16))
    b = hif4.hif4_quantize((torch.randn(G * N, K, generator=g, device="cuda") * 0.02).to(torch.bfloat16))
    return a, b.view(G, N, K // 64, 36), off.cuda()


def _check_against_existing_entry_point(hif4, a, b, off, what):
    total, N = a.shape[0], b.shape[1]
    want = hif4.hif4_grouped_gemm(a, b, off)                       # caller-provided workspace
    got = torch.full((total, N), -7.0, dtype=torch.float32, device="cuda")
    hif4.hif4_grouped_gemm_noalloc(a, b, off, out=got)             # built-in scratch
    torch.cuda.synchronize()
    ref, refabs = oracle.grouped_gemm_f64(a.cpu().numpy(), b.cpu().numpy(), off.cpu().numpy(), nthreads=8)
    got64, want64 = got.cpu().numpy().astype(np.float64), want.cpu().numpy().astype(np.float64)
    bound = TOL * refabs + 1e-300
    # each entry point against the oracle's FP64 result (an error common to both kernels would show here) ...
    for name, c in (("no-alloc", got64), ("workspace", want64)):
        err = np.abs(c - ref)
        assert np.all(err <= bound), f"{what}, {name} entry point vs oracle: worst ratio {np.max(err / bound):.3g}"
    # ... and against each other (they run different kernels, so the bits may differ; the tolerance may not)
    err = np.abs(got64 - want64)
    assert np.all(err <= bound), f"{what}: worst ratio between the entry points {np.max(err / bound):.3g}"


def test_two_calls_in_a_row_match_the_workspace_entry_point(hif4):
    # first call: 9 groups with empty and ragged ones, 567 rows -> 14 table entries in use
    a1, b1, off1 = _problem(hif4, [3, 0, 70, 1, 0, 129, 64, 0, 300], N=300, K=256, seed=91)
    # second call: fewer, differently placed tiles, so entries left by the first call would show
    a2, b2, off2 = _problem(hif4, [0, 200, 5], N=130, K=512, seed=92)
    before = hif4.launch_count()
    _check_against_existing_entry_point(hif4, a1, b1, off1, "first call")
    _check_against_existing_entry_point(hif4, a2, b2, off2, "second call")
    assert hif4.launch_count() - before == 8, "each entry point launches the table builder and the GEMM"
    assert hif4.hif4_last_device_status() == 0


def test_k_not_a_multiple_of_256_needs_no_scratch(hif4):
    a, b, off = _problem(hif4, [5, 0, 66], N=70, K=192, seed=93)
    _check_against_existing_entry_point(hif4, a, b, off, "K=192")


def test_problem_beyond_the_builtin_scratch_is_refused(hif4):
    cap = hif4.hif4_grouped_gemm_noalloc_capacity()
    assert cap == 65536
    G = cap // 16 + 1                                               # one table entry per group alone is too many
    a = torch.zeros(1, 4, 36, dtype=torch.uint8, device="cuda")
    b = torch.zeros(G, 1, 4, 36, dtype=torch.uint8, device="cuda")
    off = torch.ones(G + 1, dtype=torch.int64, device="cuda"); off[0] = 0
    out = torch.full((1, 1), 5.0, dtype=torch.float32, device="cuda")
    before = hif4.launch_count()
    with pytest.raises(hif4.Hif4Error) as ei:
        hif4.hif4_grouped_gemm_noalloc(a, b, off, out=out)
    assert ei.value.code == 5
    assert hif4.launch_count() == before and float(out[0, 0]) == 5.0
    assert hif4.hif4_grouped_gemm_workspace(G, 1, 1, 256) > cap     # the workspace variant would have asked for more
