// Shared host/device helpers of the HiF4 CUDA library (sm_100a).  Nothing here is shared with the
// CPU oracle.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "hif4.h"

namespace hif4 {

constexpr int kUnitElems = HIF4_UNIT_ELEMS;
constexpr int kUnitBytes = HIF4_UNIT_BYTES;
constexpr int kUnitWords = kUnitBytes / 4;  // 9 x 32-bit: metadata word + 8 code words

// Host-side count of kernel launches issued by this library.
void note_launch(int n = 1);

// Device word that kernels set when a bounded wait runs out (0 = fine).  Returns its device address
// for the current device, or nullptr if the symbol cannot be resolved.
unsigned int* device_error_word();

inline hif4_status launch_status() {
  return cudaGetLastError() == cudaSuccess ? HIF4_OK : HIF4_ERR_CUDA;
}

// Kernels that need more than 48 KB of dynamic shared memory have to opt in; the setting belongs to
// the device, so it is made once per device and kernel (`done_mask`: one bit per device ordinal).
template <typename Kernel>
inline bool ensure_dynamic_smem(Kernel kernel, int bytes, uint64_t& done_mask) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return false;
  if (dev < 64 && ((done_mask >> dev) & 1ull)) return true;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return false;
  if (dev < 64) done_mask |= 1ull << dev;
  return true;
}

__host__ __device__ inline int64_t ceil_div64(int64_t a, int64_t b) { return (a + b - 1) / b; }

}  // namespace hif4
