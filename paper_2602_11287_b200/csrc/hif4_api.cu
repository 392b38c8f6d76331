// Host-only parts of the HiF4 C ABI: sizes, status strings, the launch counter and the device
// error word that kernels with bounded waits report through.
#include <atomic>

#include "hif4_common.cuh"

namespace hif4 {
namespace {
std::atomic<uint64_t> g_launches{0};
__device__ unsigned int g_device_error = 0u;
}  // namespace

void note_launch(int n) { g_launches.fetch_add(static_cast<uint64_t>(n), std::memory_order_relaxed); }

unsigned int* device_error_word() {
  void* p = nullptr;
  if (cudaGetSymbolAddress(&p, g_device_error) != cudaSuccess) {
    (void)cudaGetLastError();
    return nullptr;
  }
  return static_cast<unsigned int*>(p);
}
}  // namespace hif4

extern "C" size_t hif4_packed_bytes(int64_t rows, int64_t cols) {
  if (rows < 0 || cols < 0 || cols % HIF4_UNIT_ELEMS != 0) return 0;
  return static_cast<size_t>(rows) * static_cast<size_t>(cols / HIF4_UNIT_ELEMS) * HIF4_UNIT_BYTES;
}

extern "C" const char* hif4_status_string(hif4_status s) {
  switch (s) {
    case HIF4_OK: return "ok";
    case HIF4_ERR_NULL: return "null pointer";
    case HIF4_ERR_SHAPE: return "bad shape (negative size, cols/K not a multiple of 64, or leading dimension too small)";
    case HIF4_ERR_ALIGN: return "pointer or leading dimension not aligned as documented";
    case HIF4_ERR_DTYPE: return "unknown dtype or rounding mode";
    case HIF4_ERR_WORKSPACE: return "workspace too small or misaligned";
    case HIF4_ERR_CUDA: return "CUDA call or kernel launch failed";
    case HIF4_ERR_DEVICE_TIMEOUT: return "a bounded wait inside a kernel ran out";
    case HIF4_ERR_UNSUPPORTED: return "not supported by this build";
  }
  return "unknown status";
}

extern "C" uint64_t hif4_debug_launch_count(void) { return hif4::g_launches.load(std::memory_order_relaxed); }

extern "C" hif4_status hif4_last_device_status(void* stream) {
  if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return HIF4_ERR_CUDA;
  unsigned int* word = hif4::device_error_word();
  if (!word) return HIF4_ERR_CUDA;
  unsigned int host = 0;
  if (cudaMemcpy(&host, word, sizeof(host), cudaMemcpyDeviceToHost) != cudaSuccess) return HIF4_ERR_CUDA;
  if (host != 0) {
    const unsigned int zero = 0;
    if (cudaMemcpy(word, &zero, sizeof(zero), cudaMemcpyHostToDevice) != cudaSuccess) return HIF4_ERR_CUDA;
    return HIF4_ERR_DEVICE_TIMEOUT;
  }
  return HIF4_OK;
}
