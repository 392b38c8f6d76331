// Generic HiF4 x HiF4 -> FP32 GEMM on CUDA cores: the always-correct path of hif4_gemm /
// hif4_grouped_gemm for shapes the tensor-core kernel does not take (K not a multiple of 256,
// unaligned operands, tiny problems).  C = A * B^T, Eq. 3 summed over the K/64 unit pairs.
//
// One block computes a 64 x 64 tile of C.  Per 64-wide K step it decodes 64 units of A and 64 units
// of B (Eq. 2, exact in FP32) into shared memory, k-major, and every thread accumulates a 4 x 4
// micro-tile with FP32 FMAs (each product of two decoded values has at most 12 significant bits and
// is exact; only the accumulation rounds).
#include "hif4_common.cuh"
#include "hif4_gemm_internal.cuh"

namespace hif4 {
namespace {

constexpr int kTile = 64;
constexpr int kThreads = 256;
constexpr int kPad = 4;   // row stride 68 floats keeps float4 alignment

// Decodes 32 elements (4 code words starting at word `w0`) of one unit into dst[k * stride].
__device__ __forceinline__ void decode_half_unit(const uint32_t* unit, int w0, float* dst, int stride) {
  const uint32_t meta = unit[0];
  const uint32_t byte = meta & 0xFFu;
  const float mant = static_cast<float>(4u + (byte & 3u));
#pragma unroll
  for (int w = 0; w < 4; ++w) {
    const int j = w0 + w;                       // level-2 group
    const uint32_t word = unit[1 + j];
    const uint32_t e8 = (meta >> (8 + j)) & 1u;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const uint32_t e16 = (meta >> (16 + 2 * j + h)) & 1u;
      const float s = mant * __uint_as_float(((byte >> 2) + 75u + e8 + e16) << 23);
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const uint32_t c = (word >> (16 * h + 4 * e)) & 0xFu;
        float v = static_cast<float>(c & 7u) * s;
        v = __uint_as_float(__float_as_uint(v) | ((c & 8u) << 28));
        if (byte == 0xFFu) v = __uint_as_float(0x7FC00000u);
        dst[(8 * j + 4 * h + e - 8 * w0) * stride] = v;
      }
    }
  }
}

// blockIdx.x = m_tile * tiles_n + n_tile.  grouped == false: one problem, rows [0, M).
// grouped == true: m_tile enumerates 64-row tiles over all groups; each block finds its group by
// walking the device-side offsets.
template <bool kGrouped>
__global__ void __launch_bounds__(kThreads)
gemm_simt_kernel(const uint32_t* __restrict__ A, const uint32_t* __restrict__ B, float* __restrict__ C,
                 int64_t M, int64_t N, int64_t K, int64_t ldc, const int64_t* __restrict__ offsets,
                 int num_groups) {
  __shared__ __align__(16) float As[kTile][kTile + kPad];   // [k][m]
  __shared__ __align__(16) float Bs[kTile][kTile + kPad];   // [k][n]

  const int64_t upr = K / kUnitElems;
  const unsigned tiles_n = static_cast<unsigned>((N + kTile - 1) / kTile);
  int64_t row0, row_end;
  const uint32_t* Bg = B;
  if (kGrouped) {
    int64_t tile = blockIdx.x / tiles_n;
    int g = 0;
    int64_t lo = 0, hi = 0;
    for (; g < num_groups; ++g) {
      lo = offsets[g]; hi = offsets[g + 1];
      const int64_t tiles = (hi - lo + kTile - 1) / kTile;
      if (tile < tiles) break;
      tile -= tiles;
    }
    if (g == num_groups) return;
    row0 = lo + tile * kTile;
    row_end = hi;
    Bg = B + static_cast<int64_t>(g) * N * upr * kUnitWords;
  } else {
    row0 = static_cast<int64_t>(blockIdx.x / tiles_n) * kTile;
    row_end = M;
  }
  const int64_t col0 = static_cast<int64_t>(blockIdx.x % tiles_n) * kTile;

  const int t = threadIdx.x;
  const int ty = t >> 4, tx = t & 15;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.0f;

  // decode assignment: threads 0..127 -> A rows (2 threads per unit), 128..255 -> B rows
  const int dec_row = (t & 127) >> 1, dec_half = t & 1;
  for (int64_t ku = 0; ku < upr; ++ku) {
    {
      const bool isA = t < 128;
      const int64_t r = (isA ? row0 : col0) + dec_row;
      const bool valid = isA ? (r < row_end) : (r < N);
      float* dst = (isA ? &As[0][0] : &Bs[0][0]) + dec_half * 32 * (kTile + kPad) + dec_row;
      if (valid) {
        const uint32_t* unit = (isA ? A : Bg) + (r * upr + ku) * kUnitWords;
        decode_half_unit(unit, dec_half * 4, dst, kTile + kPad);
      } else {
#pragma unroll
        for (int k = 0; k < 32; ++k) dst[k * (kTile + kPad)] = 0.0f;
      }
    }
    __syncthreads();
#pragma unroll 8
    for (int k = 0; k < kTile; ++k) {
      const float4 a = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
      const float4 b = *reinterpret_cast<const float4*>(&Bs[k][tx * 4]);
      const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int64_t r = row0 + ty * 4 + i;
    if (r >= row_end) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int64_t c = col0 + tx * 4 + j;
      if (c < N) C[r * ldc + c] = acc[i][j];
    }
  }
}

}  // namespace

hif4_status launch_gemm_simt(const void* A, const void* B, float* C, int64_t M, int64_t N, int64_t K,
                             int64_t ldc, cudaStream_t st) {
  const int64_t gy = ceil_div64(M, kTile), gx = ceil_div64(N, kTile);
  if (gx > 0x7FFFFFFFll || gy > 0x7FFFFFFFll / gx) return HIF4_ERR_SHAPE;
  gemm_simt_kernel<false><<<dim3(static_cast<unsigned>(gx * gy)), kThreads, 0, st>>>(
      static_cast<const uint32_t*>(A), static_cast<const uint32_t*>(B), C, M, N, K, ldc, nullptr, 0);
  note_launch();
  return launch_status();
}

hif4_status launch_grouped_gemm_simt(const void* A, const void* B, float* C, const int64_t* offsets,
                                     int num_groups, int64_t total_rows, int64_t N, int64_t K, int64_t ldc,
                                     cudaStream_t st) {
  const int64_t gy = ceil_div64(total_rows, kTile) + num_groups, gx = ceil_div64(N, kTile);
  if (gx > 0x7FFFFFFFll || gy > 0x7FFFFFFFll / gx) return HIF4_ERR_SHAPE;
  gemm_simt_kernel<true><<<dim3(static_cast<unsigned>(gx * gy)), kThreads, 0, st>>>(
      static_cast<const uint32_t*>(A), static_cast<const uint32_t*>(B), C, total_rows, N, K, ldc, offsets,
      num_groups);
  note_launch();
  return launch_status();
}

}  // namespace hif4
