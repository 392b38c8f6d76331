// hif4_gemm / hif4_grouped_gemm entry points: argument checks on the host, then kernel selection.
#include "hif4_common.cuh"
#include "hif4_gemm_internal.cuh"

using namespace hif4;

namespace {
// Test hook (hif4_debug_set_gemm_path): 0 = choose by shape, 1 = CUDA-core kernel only, 2 = single-CTA
// tensor-core kernel whenever it is legal, 3 = CTA-pair tensor-core kernel whenever it is legal,
// 4 = weight-streaming kernel whenever it is legal (M <= kGemvMaxM), 5 = the weight-streaming kernel on FP8 operands
// with Eq. 3's per-unit-pair scaling whenever it is legal (same shapes), 6 = hif4_linear converts BF16 activations
// inside the CTA-pair kernel whenever that is legal (hif4_gemm itself behaves as under 0).
int g_gemm_path = 0;
constexpr int64_t kPairMinM = 129;      // below that a 256-row pair tile would be half empty
constexpr int64_t kFuseMaxColumnTiles = 0;   // hif4_linear: in-kernel conversion for C with at most this many 256-column tiles
constexpr int64_t kGroupedMaxRows = (1ll << 31) - 257;   // tile tables keep row numbers (and row + tile height) in 32-bit ints

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

hif4_status check_common(const void* A, const void* B, const float* C, int64_t M, int64_t N, int64_t K,
                         int64_t ldc) {
  if (M < 0 || N < 0 || K < 0 || K % kUnitElems != 0 || ldc < N) return HIF4_ERR_SHAPE;
  if (M == 0 || N == 0) return HIF4_OK;
  if (!C || (K > 0 && (!A || !B))) return HIF4_ERR_NULL;
  if (!aligned(A, 4) || !aligned(B, 4) || !aligned(C, 4)) return HIF4_ERR_ALIGN;
  return HIF4_OK;
}
}  // namespace

extern "C" hif4_status hif4_gemm_workspace(int64_t M, int64_t N, int64_t K, size_t* bytes) {
  if (!bytes) return HIF4_ERR_NULL;
  if (M < 0 || N < 0 || K < 0 || K % kUnitElems != 0) return HIF4_ERR_SHAPE;
  // The largest need over every kernel that may serve this shape, whatever the path override says at call
  // time: decoded tokens of the weight-streaming path (M <= kGemvMaxM), completion words of the K slices of
  // the swapped pair kernel (few rows) and of the tiles that the pair kernel shares along K.
  *bytes = gemv_workspace_bytes(M, K);
  if (gemv8_workspace_bytes(M, K) > *bytes) *bytes = gemv8_workspace_bytes(M, K);
  if (M > kGemvMaxM && M < kPairMinM) {
    const size_t few_bytes = gemm_tc2_swapped_workspace_bytes(M, N, K);
    if (few_bytes > *bytes) *bytes = few_bytes;
  }
  const size_t pair_bytes = gemm_tc2_workspace_bytes(M, N, K);
  if (pair_bytes > *bytes) *bytes = pair_bytes;
  return HIF4_OK;
}

extern "C" hif4_status hif4_debug_set_gemm_path(int path) {
  if (path < 0 || path > 6) return HIF4_ERR_DTYPE;
  g_gemm_path = path;
  return HIF4_OK;
}

extern "C" hif4_status hif4_gemm(const void* A_units, const void* B_units, float* C, int64_t M, int64_t N,
                                 int64_t K, int64_t ldc, void* workspace, size_t workspace_bytes,
                                 void* stream) {
  const hif4_status chk = check_common(A_units, B_units, C, M, N, K, ldc);
  if (chk != HIF4_OK || M == 0 || N == 0) return chk;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (K == 0) {
    if (cudaMemset2DAsync(C, static_cast<size_t>(ldc) * 4, 0, static_cast<size_t>(N) * 4,
                          static_cast<size_t>(M), st) != cudaSuccess)
      return HIF4_ERR_CUDA;
    return HIF4_OK;
  }
  if ((g_gemm_path == 0 || g_gemm_path == 4) && gemv_supported(A_units, B_units, M, N, K)) {
    if (!workspace || workspace_bytes < gemv_workspace_bytes(M, K)) return HIF4_ERR_WORKSPACE;
    if (!aligned(workspace, 256)) return HIF4_ERR_ALIGN;
    return launch_gemv(A_units, B_units, C, M, N, K, ldc, workspace, st);
  }
  if (g_gemm_path == 5 && gemv_supported(A_units, B_units, M, N, K)) {
    if (!workspace || workspace_bytes < gemv8_workspace_bytes(M, K)) return HIF4_ERR_WORKSPACE;
    if (!aligned(workspace, 256)) return HIF4_ERR_ALIGN;
    return launch_gemv8(A_units, B_units, C, M, N, K, ldc, workspace, st);
  }
  const bool tc_ok = g_gemm_path != 1 && gemm_tc_supported(A_units, B_units, M, N, N, K);
  if (tc_ok && g_gemm_path != 2 && (g_gemm_path == 3 || M >= kPairMinM) && gemm_tc2_supported(A_units, B_units, M, N, K)) {
    if (workspace && !aligned(workspace, 256)) return HIF4_ERR_ALIGN;
    return launch_gemm_tc2(A_units, B_units, C, M, N, K, ldc, workspace, workspace_bytes, st);
  }
  // few rows: the pair kernel with the operands swapped pads them to 32 instead of 128
  if (tc_ok && g_gemm_path == 0 && M > kGemvMaxM && M < kPairMinM && gemm_tc2_supported(A_units, B_units, M, N, K)) {
    if (workspace && !aligned(workspace, 256)) return HIF4_ERR_ALIGN;
    return launch_gemm_tc2_swapped(A_units, B_units, C, M, N, K, ldc, workspace, workspace_bytes, st);
  }
  if (tc_ok && (g_gemm_path >= 2 || M > kGemvMaxM)) return launch_gemm_tc(A_units, B_units, C, M, N, K, ldc, st);
  return launch_gemm_simt(A_units, B_units, C, M, N, K, ldc, st);
}

extern "C" hif4_status hif4_grouped_gemm_workspace(int num_groups, int64_t total_rows, int64_t N, int64_t K,
                                                   size_t* bytes) {
  if (!bytes) return HIF4_ERR_NULL;
  if (num_groups < 0 || total_rows < 0 || total_rows > kGroupedMaxRows || N < 0 || K < 0 || K % kUnitElems != 0)
    return HIF4_ERR_SHAPE;
  // the tensor-core path keeps its tile table (one 16-byte entry per 128-row tile) here
  *bytes = 0;
  if (K > 0 && K % 256 == 0 && total_rows > 0 && num_groups > 0) {      // the larger of the two tensor-core kernels' tables
    const size_t single = grouped_tc_workspace_bytes(num_groups, total_rows);
    const size_t pairs = N > 0 ? grouped_tc2_workspace_bytes(num_groups, total_rows, N) : 0;
    *bytes = single > pairs ? single : pairs;
  }
  return HIF4_OK;
}

extern "C" hif4_status hif4_grouped_gemm(const void* A_units, const void* B_units, float* C,
                                         const int64_t* group_offsets_dev, int num_groups, int64_t total_rows,
                                         int64_t N, int64_t K, int64_t ldc, void* workspace,
                                         size_t workspace_bytes, void* stream) {
  if (num_groups < 0 || total_rows > kGroupedMaxRows) return HIF4_ERR_SHAPE;
  const hif4_status chk = check_common(A_units, B_units, C, total_rows, N, K, ldc);
  if (chk != HIF4_OK || total_rows == 0 || N == 0 || num_groups == 0) return chk;
  if (!group_offsets_dev) return HIF4_ERR_NULL;
  if (!aligned(group_offsets_dev, 8)) return HIF4_ERR_ALIGN;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (K == 0) {
    if (cudaMemset2DAsync(C, static_cast<size_t>(ldc) * 4, 0, static_cast<size_t>(N) * 4,
                          static_cast<size_t>(total_rows), st) != cudaSuccess)
      return HIF4_ERR_CUDA;
    return HIF4_OK;
  }
  const bool tc_ok = g_gemm_path != 1 &&
                     gemm_tc_supported(A_units, B_units, total_rows, static_cast<int64_t>(num_groups) * N, N, K);
  if (tc_ok && g_gemm_path != 2 && N < (1ll << 31) - 256 && static_cast<int64_t>(num_groups) * N < (1ll << 31) - 256) {
    // CTA pairs, swapped operands: padding of small experts costs 32 rows instead of 128
    if (!workspace || workspace_bytes < grouped_tc2_workspace_bytes(num_groups, total_rows, N)) return HIF4_ERR_WORKSPACE;
    if (!aligned(workspace, 256)) return HIF4_ERR_ALIGN;
    return launch_grouped_gemm_tc2(A_units, B_units, C, group_offsets_dev, num_groups, total_rows, N, K, ldc,
                                   workspace, st);
  }
  if (tc_ok) {
    const size_t need = grouped_tc_workspace_bytes(num_groups, total_rows);
    if (!workspace || workspace_bytes < need) return HIF4_ERR_WORKSPACE;
    if (!aligned(workspace, 256)) return HIF4_ERR_ALIGN;
    return launch_grouped_gemm_tc(A_units, B_units, C, group_offsets_dev, num_groups, total_rows, N, K, ldc,
                                  workspace, st);
  }
  return launch_grouped_gemm_simt(A_units, B_units, C, group_offsets_dev, num_groups, total_rows, N, K, ldc,
                                  st);
}

// ---------------------------------------------------------------------------------------- hif4_linear
namespace {
size_t round256(size_t n) { return (n + 255) / 256 * 256; }
}  // namespace

extern "C" hif4_status hif4_linear_workspace(int64_t M, int64_t N, int64_t K, size_t* bytes) {
  if (!bytes) return HIF4_ERR_NULL;
  size_t gemm_bytes = 0;
  const hif4_status st = hif4_gemm_workspace(M, N, K, &gemm_bytes);
  if (st != HIF4_OK) return st;
  *bytes = round256(hif4_packed_bytes(M, K)) + round256(gemm_bytes);
  return HIF4_OK;
}

extern "C" hif4_status hif4_linear(const void* X, hif4_dtype dt, int64_t ld_x, const void* W_units, float* Y,
                                   int64_t M, int64_t N, int64_t K, int64_t ldy, hif4_round mode, void* workspace,
                                   size_t workspace_bytes, void* stream) {
  size_t need = 0;
  const hif4_status ws = hif4_linear_workspace(M, N, K, &need);
  if (ws != HIF4_OK) return ws;
  if (M == 0 || N == 0) return (ldy < N) ? HIF4_ERR_SHAPE : HIF4_OK;
  if (need > 0 && (!workspace || workspace_bytes < need)) return HIF4_ERR_WORKSPACE;
  if (need > 0 && !aligned(workspace, 256)) return HIF4_ERR_ALIGN;
  const size_t x_bytes = round256(hif4_packed_bytes(M, K));
  uint8_t* x_units = static_cast<uint8_t*>(workspace);
  // Few rows of activations: quantized and decoded inside the token preparation of the weight-streaming kernel
  // (same encoder code, so the same bits), one launch fewer and no packed round trip.
  if ((dt == HIF4_BF16 || dt == HIF4_FP32 || dt == HIF4_FP16) && (mode == HIF4_RNE || mode == HIF4_RHA) && K > 0 &&
      (g_gemm_path == 0 || g_gemm_path == 4) && X && W_units && Y && ldy >= N && aligned(W_units, 4) && aligned(Y, 4) &&
      gemv_linear_supported(X, dt, ld_x, W_units, M, N, K))
    return launch_gemv_linear(X, dt, ld_x, mode == HIF4_RHA, W_units, Y, M, N, K, ldy, x_units + x_bytes,
                              static_cast<cudaStream_t>(stream));
  // Many rows: the conversion can also run inside the pair kernel's A-side decode threads (once per column tile of
  // C).  Measured against the two launches it loses on every shape, even with a single column tile (M = 4096,
  // K = 4096: N = 256 62 vs 44 us, N = 1024 100 vs 52 us, N = 14336 1149 vs 381 us): Algorithm 1 costs about 2.6 times
  // the decode per element and sits on the critical path of every K chunk.  kFuseMaxColumnTiles = 0 therefore keeps
  // the default on two launches; the test hook (path 6) still reaches the fused kernel, whose result is bit-identical.
  if (dt == HIF4_BF16 && mode == HIF4_RNE && K > 0 && M >= kPairMinM && X && W_units && Y && ldy >= N &&
      (g_gemm_path == 6 || (g_gemm_path == 0 && ceil_div64(N, 256) <= kFuseMaxColumnTiles)) && aligned(X, 16) &&
      ld_x >= K && (ld_x * 2) % 16 == 0 && aligned(W_units, 4) && aligned(Y, 4) &&
      gemm_tc2_supported(W_units, W_units, M, N, K)) {
    size_t pair_bytes = gemm_tc2_workspace_bytes(M, N, K);
    if (pair_bytes > workspace_bytes - x_bytes) return HIF4_ERR_WORKSPACE;
    return launch_gemm_tc2_fused_bf16(X, ld_x, W_units, Y, M, N, K, ldy, x_units + x_bytes, workspace_bytes - x_bytes,
                                      static_cast<cudaStream_t>(stream));
  }
  if (K > 0) {
    const hif4_status q = hif4_quantize(X, dt, M, K, ld_x, x_units, mode, stream);
    if (q != HIF4_OK) return q;
  }
  return hif4_gemm(x_units, W_units, Y, M, N, K, ldy, x_units + x_bytes, workspace_bytes - x_bytes, stream);
}
