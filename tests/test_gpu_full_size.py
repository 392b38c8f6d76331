"""GPU parity at the full configured sizes, in the launch configuration bench.py times (default kernel
selection).  The oracle cannot redo whole tensors of this size in seconds, so it recomputes sampled rows
(quantizer: bit-exact) and sampled output entries plus the four corners (GEMM: the stated tolerance)."""
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
    yield lib
    assert lib.hif4_last_device_status() == 0
    torch.cuda.empty_cache()


def _sampled_rows_match(hif4, x, n_rows, seed):
    q = hif4.hif4_quantize(x)
    rng = np.random.default_rng(seed)
    rows = np.unique(np.concatenate([rng.integers(0, x.shape[0], n_rows), [0, x.shape[0] - 1]]))
    idx = torch.from_numpy(rows).cuda()
    host = x[idx].cpu()
    src = wl.bf16_to_u16_numpy(host) if x.dtype == torch.bfloat16 else host.numpy()
    want = oracle.quantize(src, nthreads=8)
    got = q[idx].cpu().numpy()
    assert np.array_equal(got, want), f"{int((got != want).any(axis=-1).sum())} sampled units differ"
    return q


def test_quantize_sweep_sizes_sampled_rows(hif4):
    """Config 3: 2^20 .. 2^28 BF16 elements of the Gaussian / Student-t / uniform mix with spike units."""
    for log2n in (20, 24, 28):
        x = wl.quantize_sweep(2 ** log2n, device="cuda")
        q = _sampled_rows_match(hif4, x, 48, seed=log2n)
        assert q.shape == (2 ** log2n // 4096, 64, 36)
        del x, q
    x32 = wl.quantize_sweep(2 ** 24, device="cuda", dtype=torch.float32)
    _sampled_rows_match(hif4, x32, 48, seed=1)


def _sampled_entries(hif4, a_units, b_units, C, what, n=300, seed=0):
    M, N = C.shape
    rng = np.random.default_rng(seed)
    rows = np.concatenate([rng.integers(0, M, n), [0, M - 1, 0, M - 1]])
    cols = np.concatenate([rng.integers(0, N, n), [0, 0, N - 1, N - 1]])
    urows, rinv = np.unique(rows, return_inverse=True)
    ucols, cinv = np.unique(cols, return_inverse=True)
    a_host = a_units[torch.from_numpy(urows).cuda()].cpu().numpy()          # only the sampled rows travel to the host
    b_host = b_units[torch.from_numpy(ucols).cuda()].cpu().numpy()
    ref, refabs = oracle.gemm_sampled_f64(a_host, b_host, rinv, cinv)
    got = C[torch.from_numpy(rows).cuda(), torch.from_numpy(cols).cuda()].cpu().numpy().astype(np.float64)
    err = np.abs(got - ref)
    assert np.all(err <= TOL * refabs + 1e-300), f"{what}: worst ratio {np.max(err / np.maximum(TOL * refabs, 1e-300)):.3g}"


def _abs_bound_on_device(hif4, a_units, b_units):
    """sum_k |a_ik| |b_jk| for every entry, formed on the GPU from the decoded operands (FP32 matmul of magnitudes):
    only the scale of a tolerance between two GPU kernels, never an expected value."""
    a = hif4.hif4_dequantize(a_units, torch.float32).abs_()
    b = hif4.hif4_dequantize(b_units, torch.float32).abs_()
    prev = torch.backends.cuda.matmul.allow_tf32
    torch.backends.cuda.matmul.allow_tf32 = False
    try:
        return a @ b.t()
    finally:
        torch.backends.cuda.matmul.allow_tf32 = prev


def _whole_c_against_the_single_cta_kernel(hif4, a_units, b_units, C, what):
    """Every entry of the default path's C against the single-CTA tensor-core kernel's C (another tile shape, no
    tile shared between CTAs, another summation order): the two may differ by FP32 rounding only."""
    hif4.hif4_debug_set_gemm_path(2)
    try:
        other = hif4.hif4_gemm(a_units, b_units)
    finally:
        hif4.hif4_debug_set_gemm_path(0)
    bound = _abs_bound_on_device(hif4, a_units, b_units).mul_(2 * TOL)
    bad = (C - other).abs_() > bound
    assert not bool(bad.any()), f"{what}: {int(bad.sum())} entries differ between the pair kernel and the single-CTA kernel"


def _tile_against_oracle(hif4, a_units, b_units, C, m0, n0, what, rows=256, cols=256):
    """Every entry of C[m0:m0+rows, n0:n0+cols] against the oracle's FP64 product of those operand rows."""
    M, N = C.shape
    m1, n1 = min(M, m0 + rows), min(N, n0 + cols)
    ref, refabs = oracle.gemm_f64(a_units[m0:m1].cpu().numpy(), b_units[n0:n1].cpu().numpy(), nthreads=oracle.hardware_threads())
    err = np.abs(C[m0:m1, n0:n1].cpu().numpy().astype(np.float64) - ref)
    assert np.all(err <= TOL * refabs + 1e-300), f"{what} tile ({m0}, {n0}): worst ratio {np.max(err / np.maximum(TOL * refabs, 1e-300)):.3g}"


def _shared_tiles(M, N, pairs=74):
    """Origins of two 256 x 256 tiles that the balanced last rounds of the pair kernel split between two CTA pairs
    (the end of the tile stored by one pair, its beginning added by the next), for a device with `pairs` CTA pairs:
    tiles are numbered row-major; after floor(tiles / pairs) - 1 whole rounds the remaining tiles are dealt out in
    equal runs of K chunks, so all but a few of them are shared.  Also the last tile of the last row and column."""
    nt = -(-N // 256)
    tiles = -(-M // 256) * nt
    first = (tiles // pairs - 1) * pairs if tiles >= pairs and tiles % pairs else 0
    picks = [first + 1, (first + tiles) // 2, tiles - 1]
    return [((t // nt) * 256, (t % nt) * 256) for t in picks]


def test_llama_prefill_whole_c_and_whole_shared_tiles(hif4):
    """Config 2 at M = 4096, default dispatch: the whole C against the single-CTA kernel entry by entry, and whole
    256 x 256 tiles that two CTA pairs share (store, then reduce-add), plus the last tile, against the oracle."""
    M = 4096
    for (name, K, N) in wl.LLAMA3_8B_LINEARS:
        w = hif4.hif4_quantize(wl.gaussian(N, K, 0.02, seed=2000 + N + K, device="cuda"))
        x = hif4.hif4_quantize(wl.llama_activations(M, K, seed=1002 + M + K, device="cuda"))
        C = hif4.hif4_gemm(x, w)
        _whole_c_against_the_single_cta_kernel(hif4, x, w, C, f"llama {name} M={M}")
        for (m0, n0) in _shared_tiles(M, N):
            _tile_against_oracle(hif4, x, w, C, m0, n0, f"llama {name} M={M}")
        _tile_against_oracle(hif4, x, w, C, M - 32, 0, f"llama {name} last rows", rows=32, cols=N)
        del C, x, w
        torch.cuda.empty_cache()


def test_llama_linears_all_m(hif4):
    """Config 2 exactly as the benchmark runs it: every (M, K, N) through the default dispatch."""
    for (name, K, N) in wl.LLAMA3_8B_LINEARS:
        w = hif4.hif4_quantize(wl.gaussian(N, K, 0.02, seed=2000 + N + K, device="cuda"))
        for M in wl.LLAMA3_8B_M:
            x = hif4.hif4_quantize(wl.llama_activations(M, K, seed=1002 + M + K, device="cuda"))
            C = hif4.hif4_gemm(x, w)
            _sampled_entries(hif4, x, w, C, f"llama {name} M={M}", n=200, seed=M)
            del C
        del w


def test_llama_decode_linears_replayed_from_a_cuda_graph(hif4):
    """The benchmark replays the M = 1 and M = 16 linears (hif4_linear: token quantization + preparation, then
    weight streaming; shared workspace) from CUDA graphs: the same launches, captured once.  The replayed results
    are identical to hif4_quantize + hif4_gemm launched directly and are checked against the oracle like them."""
    shapes = [(M, K, N) for M in (1, 16) for (_, K, N) in wl.LLAMA3_8B_LINEARS]
    weights = {(K, N): hif4.hif4_quantize(wl.gaussian(N, K, 0.02, seed=2000 + N + K, device="cuda"))
               for (_, K, N) in wl.LLAMA3_8B_LINEARS}
    acts = {(M, K): wl.llama_activations(M, K, seed=1002 + M + K, device="cuda") for (M, K, _) in shapes}
    xq = {sh: hif4.hif4_quantize(acts[(sh[0], sh[1])]) for sh in shapes}
    cs = {sh: torch.empty(sh[0], sh[2], dtype=torch.float32, device="cuda") for sh in shapes}
    ws = torch.empty(max(max(hif4.hif4_linear_workspace(M, N, K) for (M, K, N) in shapes), 256), dtype=torch.uint8, device="cuda")
    direct = {sh: hif4.hif4_gemm(xq[sh], weights[(sh[1], sh[2])]) for sh in shapes}

    def run():
        for (M, K, N) in shapes:
            hif4.hif4_linear(acts[(M, K)], weights[(K, N)], out=cs[(M, K, N)], workspace=ws)

    run()                                               # direct launches (also the one-time kernel attributes)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    before = hif4.launch_count()
    with torch.cuda.graph(graph):
        run()
    want_launches = sum(1 if tokens_stay_in_shared_memory(M, K, from_bf16=True) else 2 for (M, K, N) in shapes)
    assert hif4.launch_count() - before == want_launches, "streaming kernel per linear, preceded by a token kernel where building the tokens in every CTA would cost more than that launch"
    for c in cs.values():
        c.fill_(-7.0)
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    assert hif4.hif4_last_device_status() == 0
    for sh in shapes:
        M, K, N = sh
        assert torch.equal(cs[sh], direct[sh]), f"replayed {sh} differs from hif4_quantize + hif4_gemm"
        _sampled_entries(hif4, xq[sh], weights[(K, N)], cs[sh], f"graph replay {sh}", n=100, seed=M + N)


def test_dense_prefill_m8192(hif4):
    """Config 4: M = 8192 tokens with per-token scales over 2^-4 .. 2^4."""
    for (name, K, N) in wl.DENSE_PREFILL_LINEARS:
        x = hif4.hif4_quantize(wl.prefill_activations(wl.DENSE_PREFILL_M, K, device="cuda"))
        w = hif4.hif4_quantize(wl.gaussian(N, K, 0.015, seed=4000 + N + K, device="cuda"))
        C = hif4.hif4_gemm(x, w)
        _sampled_entries(hif4, x, w, C, f"prefill {name}", n=300, seed=K)
        _whole_c_against_the_single_cta_kernel(hif4, x, w, C, f"prefill {name}")
        for (m0, n0) in _shared_tiles(wl.DENSE_PREFILL_M, N)[:2 if K > 8192 else 3]:
            _tile_against_oracle(hif4, x, w, C, m0, n0, f"prefill {name}")
        del x, w, C
        torch.cuda.empty_cache()


def _expert_weights(hif4, experts, N, K, seed):
    out = torch.empty(experts, N, K // 64, 36, dtype=torch.uint8, device="cuda")
    step = 16                                          # BF16 sources are drawn 16 experts at a time
    for e0 in range(0, experts, step):
        w = wl.gaussian(step * N, K, 0.02, seed=seed + e0, device="cuda")
        hif4.hif4_quantize(w, out=out[e0:e0 + step].view(step * N, K // 64, 36))
        del w
    return out


def test_moe_layer_grouped_full_size(hif4):
    """Config 5: 4096 tokens, top-8 of 256 experts under Zipf(1.1) popularity, both expert linears."""
    r = wl.moe_routing(device="cuda")
    off = r["offsets"]
    counts = r["counts"].cpu().numpy()
    total = int(off[-1])
    assert total == wl.MOE_TOKENS * wl.MOE_TOPK and len(counts) == wl.MOE_EXPERTS
    assert (counts > 0).sum() >= 250 and counts.max() > 2000 and np.median(counts) < 80, "Zipf-shaped expert loads"
    off_h = off.cpu().numpy()
    order = np.argsort(counts)
    picks = [int(order[-1]), int(order[0]), int(order[len(order) // 2]), int(order[-2]), int(order[len(order) // 4])]
    for (K, N, seed) in ((wl.MOE_HIDDEN, 2 * wl.MOE_INTER, 5100), (wl.MOE_INTER, wl.MOE_HIDDEN, 5200)):
        a = hif4.hif4_quantize(wl.outlier_channel_activations(total, K, seed=seed, device="cuda"))
        b = _expert_weights(hif4, wl.MOE_EXPERTS, N, K, seed + 1)
        C = hif4.hif4_grouped_gemm(a, b, off)
        for g in picks:
            lo, hi = int(off_h[g]), int(off_h[g + 1])
            if hi > lo:
                _sampled_entries(hif4, a[lo:hi], b[g], C[lo:hi], f"moe K={K} expert {g} ({hi - lo} rows)", n=60, seed=g)
        del a, b, C
        torch.cuda.empty_cache()
