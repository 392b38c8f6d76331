// Quantization-error study of Section III-A on the GPU: a BF16 tensor is converted to one of four 4-bit block
// formats and back, the image is written out as FP32 and the squared error against the source is summed.
//   HiF4       Algorithm 1 (hif4_quantize into the workspace), then Eq. 2 per element
//   MXFP4      blocks of 32, power-of-two scale 2^(floor(log2 amax) - 2), E2M1 elements
//   NVFP4      blocks of 16, E4M3 scale amax / 6, E2M1 elements (direct cast)
//   NVFP4+PTS  the same after scaling the tensor's peak magnitude to 2688 = 448 * 6, undone afterwards
// The two comparison formats are computed in FP32 with one IEEE round-to-nearest operation per step (division
// included), which is what the CPU oracle does, so the images agree bit for bit.  The error is summed in FP64:
// per thread, then per block in a fixed tree, then over the blocks in index order by a one-block kernel, so the
// sum does not depend on scheduling.
#include "hif4_common.cuh"

namespace hif4 {
namespace {

constexpr int kMseThreads = 256;

__device__ __forceinline__ float bf16_to_f32(uint16_t h) { return __uint_as_float(static_cast<uint32_t>(h) << 16); }

// Nearest E2M1 magnitude {0, 0.5, 1, 1.5, 2, 3, 4, 6}; a tie goes to the even code (0, 1, 2, 4); saturating.
__device__ __forceinline__ float e2m1_round(float q) {
  if (q <= 0.25f) return 0.0f;
  if (q < 0.75f) return 0.5f;
  if (q <= 1.25f) return 1.0f;
  if (q < 1.75f) return 1.5f;
  if (q <= 2.5f) return 2.0f;
  if (q < 3.5f) return 3.0f;
  if (q <= 5.0f) return 4.0f;
  return 6.0f;
}
// FP8 E4M3 of a non-negative finite value: 4-bit significand, subnormal step 2^-9, nearest-even, saturating at 448.
__device__ __forceinline__ float e4m3_round(float v) {
  if (v == 0.0f) return 0.0f;
  int e = static_cast<int>((__float_as_uint(v) >> 23) & 0xFFu) - 127;        // floor(log2 v) for a normal float
  if ((__float_as_uint(v) >> 23) == 0u) e = -127;                             // FP32 subnormal: far below 2^-6 anyway
  if (e < -6) e = -6;
  const float quantum = __uint_as_float(static_cast<uint32_t>(e - 3 + 127) << 23);
  const float r = __fmul_rn(rintf(__fdiv_rn(v, quantum)), quantum);           // rintf: ties to even
  return r > 448.0f ? 448.0f : r;
}

// Block-wide FP64 sum in a fixed tree; the result is valid in thread 0.
__device__ __forceinline__ double block_sum(double v, double* smem) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xFFFFFFFFu, v, o);
  if ((threadIdx.x & 31) == 0) smem[threadIdx.x >> 5] = v;
  __syncthreads();
  double s = 0.0;
  if (threadIdx.x == 0)
    for (int w = 0; w < kMseThreads / 32; ++w) s += smem[w];
  return s;
}

__global__ void __launch_bounds__(kMseThreads)
mse_amax_kernel(const uint16_t* __restrict__ x, int64_t n, unsigned int* __restrict__ amax_bits) {
  unsigned int m = 0u;
  for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < n; i += static_cast<int64_t>(gridDim.x) * blockDim.x)
    m = max(m, static_cast<unsigned int>(x[i] & 0x7FFFu));                    // |x| bit patterns order like the values
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_down_sync(0xFFFFFFFFu, m, o));
  if ((threadIdx.x & 31) == 0 && m) atomicMax(amax_bits, m);
}

// kBlock = 32 (MXFP4) or 16 (NVFP4); thread per block of elements.
template <int kBlock, bool kPts>
__global__ void __launch_bounds__(kMseThreads)
mse_block_format_kernel(const uint16_t* __restrict__ x, int64_t n, const unsigned int* __restrict__ amax_bits,
                        float* __restrict__ dst, double* __restrict__ partials) {
  __shared__ double red[kMseThreads / 32];
  const int64_t b = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  double err = 0.0;
  if (b * kBlock < n) {
    float gain = 1.0f;
    if (kPts) {
      const float tensor_amax = bf16_to_f32(static_cast<uint16_t>(*amax_bits));
      gain = tensor_amax > 0.0f ? __fdiv_rn(2688.0f, tensor_amax) : 1.0f;
    }
    float src[kBlock], v[kBlock];
    const uint4* p = reinterpret_cast<const uint4*>(x + b * kBlock);
#pragma unroll
    for (int c = 0; c < kBlock / 8; ++c) {
      const uint4 w = __ldg(p + c);
      const uint32_t ws[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        src[8 * c + 2 * k] = bf16_to_f32(static_cast<uint16_t>(ws[k] & 0xFFFFu));
        src[8 * c + 2 * k + 1] = bf16_to_f32(static_cast<uint16_t>(ws[k] >> 16));
      }
    }
    float amax = 0.0f;
#pragma unroll
    for (int i = 0; i < kBlock; ++i) {
      v[i] = __fmul_rn(src[i], gain);
      amax = fmaxf(amax, fabsf(v[i]));
    }
    float scale;
    if (kBlock == 32) {
      int e = static_cast<int>((__float_as_uint(amax) >> 23) & 0xFFu) - 127 - 2;    // floor(log2 amax) - 2 (BF16 normals)
      e = min(127, max(-127, e));
      scale = amax > 0.0f ? __uint_as_float(static_cast<uint32_t>(max(e + 127, 0)) << 23) : 0.0f;
      if (e == -127) scale = __uint_as_float(0x00400000u);                          // 2^-127 is an FP32 subnormal
    } else {
      scale = e4m3_round(__fdiv_rn(amax, 6.0f));
    }
#pragma unroll
    for (int i = 0; i < kBlock; ++i) {
      float d = 0.0f;
      if (scale > 0.0f) d = __fmul_rn(e2m1_round(__fdiv_rn(fabsf(v[i]), scale)), scale);
      const float out = __fdiv_rn(copysignf(d, src[i]), gain);
      if (dst) dst[b * kBlock + i] = out;
      const double diff = static_cast<double>(out) - static_cast<double>(src[i]);
      err += diff * diff;
    }
  }
  const double s = block_sum(err, red);
  if (threadIdx.x == 0) partials[blockIdx.x] = s;
}

// HiF4 image from the packed units (Eq. 2 in FP32, exact) and its error; thread per unit.
__global__ void __launch_bounds__(kMseThreads)
mse_hif4_kernel(const uint16_t* __restrict__ x, const uint32_t* __restrict__ units, int64_t n_units, float* __restrict__ dst,
                double* __restrict__ partials) {
  __shared__ double red[kMseThreads / 32];
  const int64_t u = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  double err = 0.0;
  if (u < n_units) {
    const uint32_t* unit = units + u * kUnitWords;
    const uint32_t meta = __ldg(unit);
    const uint32_t byte = meta & 0xFFu;
    const float e6m2 = byte == 0xFFu ? __uint_as_float(0x7FC00000u) : __uint_as_float((byte + 316u) << 21);   // Eq. 1
    for (int j = 0; j < 8; ++j) {
      const uint32_t w = __ldg(unit + 1 + j);
      const uint32_t e8 = (meta >> (8 + j)) & 1u;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const uint32_t c = (w >> (4 * i)) & 0xFu;
        const uint32_t sh = e8 + ((meta >> (16 + 2 * j + (i >> 2))) & 1u);
        float val = __fmul_rn(static_cast<float>((c & 7u) << sh) * 0.25f, e6m2);        // Eq. 2: exact in FP32
        if (c & 8u) val = -val;
        const int64_t e = u * kUnitElems + 8 * j + i;
        if (dst) dst[e] = val;
        const double diff = static_cast<double>(val) - static_cast<double>(bf16_to_f32(x[e]));
        err += diff * diff;
      }
    }
  }
  const double s = block_sum(err, red);
  if (threadIdx.x == 0) partials[blockIdx.x] = s;
}

__global__ void __launch_bounds__(kMseThreads)
mse_finish_kernel(const double* __restrict__ partials, int64_t count, double* __restrict__ out) {
  __shared__ double red[kMseThreads / 32];
  // thread t sums partials t, t + 256, ... in index order; then the fixed block tree
  double s = 0.0;
  for (int64_t i = threadIdx.x; i < count; i += kMseThreads) s += partials[i];
  const double total = block_sum(s, red);
  if (threadIdx.x == 0) *out = total;
}

size_t round256(size_t v) { return (v + 255) / 256 * 256; }
int64_t work_items(int64_t n, hif4_bfp4_format fmt) { return n / (fmt == HIF4_FMT_HIF4 ? 64 : fmt == HIF4_FMT_MXFP4 ? 32 : 16); }

}  // namespace
}  // namespace hif4

using namespace hif4;

extern "C" hif4_status hif4_mse_workspace(int64_t n, hif4_bfp4_format fmt, size_t* bytes) {
  if (!bytes) return HIF4_ERR_NULL;
  if (n < 0 || n % kUnitElems != 0) return HIF4_ERR_SHAPE;
  if (fmt < HIF4_FMT_HIF4 || fmt > HIF4_FMT_NVFP4_PTS) return HIF4_ERR_DTYPE;
  const size_t blocks = static_cast<size_t>(ceil_div64(work_items(n, fmt), kMseThreads));
  // [tensor peak word: 256 B][per-block partial sums][HiF4 only: the packed units]
  *bytes = 256 + round256(blocks * sizeof(double)) + (fmt == HIF4_FMT_HIF4 ? round256(hif4_packed_bytes(1, n)) : 0);
  return HIF4_OK;
}

extern "C" hif4_status hif4_mse_roundtrip(const void* src_bf16, int64_t n, hif4_bfp4_format fmt, float* dst,
                                          double* sq_err_sum, void* workspace, size_t workspace_bytes, void* stream) {
  size_t need = 0;
  const hif4_status ws = hif4_mse_workspace(n, fmt, &need);
  if (ws != HIF4_OK) return ws;
  if (!sq_err_sum) return HIF4_ERR_NULL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (n == 0) return cudaMemsetAsync(sq_err_sum, 0, sizeof(double), st) == cudaSuccess ? HIF4_OK : HIF4_ERR_CUDA;
  if (!src_bf16 || !workspace) return HIF4_ERR_NULL;
  if (workspace_bytes < need) return HIF4_ERR_WORKSPACE;
  if ((reinterpret_cast<uintptr_t>(src_bf16) & 15u) || (reinterpret_cast<uintptr_t>(workspace) & 255u) ||
      (reinterpret_cast<uintptr_t>(sq_err_sum) & 7u) || (reinterpret_cast<uintptr_t>(dst) & 3u))
    return HIF4_ERR_ALIGN;
  const int64_t items = work_items(n, fmt);
  const int64_t blocks = ceil_div64(items, kMseThreads);
  if (blocks > 0x7FFFFFFFll) return HIF4_ERR_SHAPE;
  uint8_t* base = static_cast<uint8_t*>(workspace);
  unsigned int* amax_bits = reinterpret_cast<unsigned int*>(base);
  double* partials = reinterpret_cast<double*>(base + 256);
  const uint16_t* x = static_cast<const uint16_t*>(src_bf16);
  const unsigned grid = static_cast<unsigned>(blocks);
  if (fmt == HIF4_FMT_HIF4) {
    void* units = base + 256 + round256(static_cast<size_t>(blocks) * sizeof(double));
    const hif4_status q = hif4_quantize(src_bf16, HIF4_BF16, 1, n, n, units, HIF4_RNE, stream);
    if (q != HIF4_OK) return q;
    mse_hif4_kernel<<<grid, kMseThreads, 0, st>>>(x, static_cast<const uint32_t*>(units), items, dst, partials);
  } else if (fmt == HIF4_FMT_MXFP4) {
    mse_block_format_kernel<32, false><<<grid, kMseThreads, 0, st>>>(x, n, amax_bits, dst, partials);
  } else if (fmt == HIF4_FMT_NVFP4) {
    mse_block_format_kernel<16, false><<<grid, kMseThreads, 0, st>>>(x, n, amax_bits, dst, partials);
  } else {
    if (cudaMemsetAsync(amax_bits, 0, sizeof(unsigned int), st) != cudaSuccess) return HIF4_ERR_CUDA;
    const unsigned agrid = static_cast<unsigned>(ceil_div64(n, kMseThreads * 16) < 1184 ? ceil_div64(n, kMseThreads * 16) : 1184);
    mse_amax_kernel<<<agrid, kMseThreads, 0, st>>>(x, n, amax_bits);
    note_launch();
    mse_block_format_kernel<16, true><<<grid, kMseThreads, 0, st>>>(x, n, amax_bits, dst, partials);
  }
  note_launch();
  if (cudaGetLastError() != cudaSuccess) return HIF4_ERR_CUDA;
  mse_finish_kernel<<<1, kMseThreads, 0, st>>>(partials, blocks, sq_err_sum);
  note_launch();
  return launch_status();
}
