// hif4_grouped_gemm_noalloc -- hif4_grouped_gemm for callers that have no way to hand over device
// scratch memory.
//
// The tensor-core grouped GEMM keeps a table of its row tiles (one 16-byte entry per 128-row tile of
// every expert) in device memory.  hif4_grouped_gemm takes that table's storage from the caller,
// which means somebody has to allocate it.  Some callers cannot: code that runs inside a fixed memory
// plan (an inference engine that sized every buffer at start-up and forbids later allocations), a
// plug-in that is handed tensors but no allocator, or a latency-critical section in which a
// cudaMalloc (which synchronises the device) is not acceptable.  For them the table lives here, in a
// file-scope __device__ array that the library's image carries: every GPU that loads the library
// holds these kNoAllocScratchBytes bytes from load until the process exits.
//
// Consequences the caller has to know:
//   * the problem must fit: ceil(total_rows / 128) + num_groups tile entries of 16 bytes, rounded up
//     to 256 bytes, may not exceed kNoAllocScratchBytes; larger problems are refused with
//     HIF4_ERR_WORKSPACE before anything is launched;
//   * all calls on one GPU share the one array.  Calls that are ordered on a stream are fine (every
//     call rewrites all the entries it uses, nothing has to start at zero); calls that can overlap
//     on the GPU (different streams without an event between them, different host threads) race on
//     it and compute garbage;
//   * in host code the array's name is only a handle, not a device pointer, so the device address is
//     looked up with cudaGetSymbolAddress, once per GPU, with that GPU current, by the first call
//     made on it.  That first call should therefore not sit inside a stream capture.
#include "hif4_common.cuh"
#include "hif4_gemm_internal.cuh"

namespace hif4 {
namespace {

constexpr size_t kNoAllocScratchBytes = HIF4_NOALLOC_SCRATCH_BYTES;
constexpr int kMaxDevices = 64;

static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

// Device address of g_noalloc_scratch on each GPU this process has used it on (nullptr = not yet
// looked up).  Not thread-safe for concurrent first calls on the same device.
void* g_scratch_addr[kMaxDevices] = {};

// Returns the device address of the scratch array on the current GPU, resolving it on first use.
hif4_status scratch_for_current_device(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0) return HIF4_ERR_CUDA;
  if (dev >= kMaxDevices) return HIF4_ERR_UNSUPPORTED;
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_noalloc_scratch) != cudaSuccess || !p) {
      (void)cudaGetLastError();
      return HIF4_ERR_CUDA;
    }
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return HIF4_OK;
}

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

}  // namespace
}  // namespace hif4

using namespace hif4;

extern "C" size_t hif4_grouped_gemm_noalloc_capacity(void) { return kNoAllocScratchBytes; }

extern "C" hif4_status hif4_grouped_gemm_noalloc(const void* A_units, const void* B_units, float* C,
                                                 const int64_t* group_offsets_dev, int num_groups,
                                                 int64_t total_rows, int64_t N, int64_t K, int64_t ldc,
                                                 void* stream) {
  // Same argument rules as hif4_grouped_gemm.
  if (num_groups < 0 || total_rows < 0 || N < 0 || K < 0 || K % kUnitElems != 0 || ldc < N) return HIF4_ERR_SHAPE;
  if (total_rows == 0 || N == 0 || num_groups == 0) return HIF4_OK;
  if (!C || !group_offsets_dev || (K > 0 && (!A_units || !B_units))) return HIF4_ERR_NULL;
  if (!aligned(A_units, 4) || !aligned(B_units, 4) || !aligned(C, 4) || !aligned(group_offsets_dev, 8))
    return HIF4_ERR_ALIGN;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (K == 0) {
    if (cudaMemset2DAsync(C, static_cast<size_t>(ldc) * 4, 0, static_cast<size_t>(N) * 4,
                          static_cast<size_t>(total_rows), st) != cudaSuccess)
      return HIF4_ERR_CUDA;
    return HIF4_OK;
  }
  if (!gemm_tc_supported(A_units, B_units, total_rows, static_cast<int64_t>(num_groups) * N, N, K)) {
    // K not a multiple of 256 or operands not 16-byte aligned: the CUDA-core kernel walks the
    // offsets itself and needs no scratch at all.
    return launch_grouped_gemm_simt(A_units, B_units, C, group_offsets_dev, num_groups, total_rows, N, K, ldc, st);
  }
  if (grouped_tc_workspace_bytes(num_groups, total_rows) > kNoAllocScratchBytes) return HIF4_ERR_WORKSPACE;
  void* scratch = nullptr;
  const hif4_status rs = scratch_for_current_device(&scratch);
  if (rs != HIF4_OK) return rs;
  return launch_grouped_gemm_tc(A_units, B_units, C, group_offsets_dev, num_groups, total_rows, N, K, ldc,
                                scratch, st);
}
