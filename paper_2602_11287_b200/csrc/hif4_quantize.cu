// hif4_quantize / hif4_dequantize -- Algorithm 1 (Section II-B) and Eq. 2 of the HiFloat4 paper as
// streaming CUDA kernels for sm_100a.  Both are bound by HBM traffic: 2 B (or 4 B) read and
// 0.5625 B written per element for the quantizer, the reverse for the dequantizer.
//
// BF16 quantizer, thread mapping: 2 consecutive lanes own one 64-element unit; lane l loads the
// 16 bytes of the level-2 groups l, l + 2, l + 4, l + 6 with four 128-bit loads, so a warp covers 16
// units per pass and each lane issues all its loads before it computes.  Algorithm 1 is written in BF16 arithmetic; packed bf16x2 instructions with
// round-to-nearest-even are exactly that arithmetic for two elements at a time:
//   - peak magnitudes are integer maxima of the |x| bit patterns (NaN patterns sort above Inf);
//   - SF = Vmax * (1/7)_BF16 is one mul.rn.bf16x2; rounding SF to the 3-bit-significand E6M2 byte is
//     an integer add/shift on its bit pattern (the carry runs into the exponent by itself);
//   - the E6M2 reciprocal is the 4-entry table on the mantissa plus an exponent subtraction;
//   - rounding is monotone, so max_i bf16(|x_i| * REC) == bf16(max_i |x_i| * REC): each element is
//     multiplied once and the micro-exponent thresholds are taken on maxima of the products;
//   - fma.rn.bf16x2(t, 4 * 2^-(e8+e16), 128) rounds t's quarter count to nearest-even in the low
//     mantissa bits (ulp is 1 in [128, 256)); an integer min clamps to 1.75 (and catches Inf).
// FP32 sources run the same steps in FP32 arithmetic with 4 lanes per unit (lane = four level-3
// groups of 4 elements).
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "hif4_common.cuh"
#include "hif4_quantize_device.cuh"

namespace hif4 {
namespace {

constexpr int kThreads = 256;
// units per 8-lane group and pass of the dequantizer: more loads in flight pay for BF16 output, not for FP32
constexpr int kUnrollDeqBf16 = 8, kUnrollDeqFp32 = 8;

// ----------------------------------------------------------------------------- streaming loads and stores
__device__ __forceinline__ void st_stream(uint32_t* p, uint32_t v) {
  asm volatile("st.global.cs.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void st_stream(uint4* p, uint4 v) {
  asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z),
               "r"(v.w)
               : "memory");
}
// Offset (in elements) of unit u of a [rows, upr*64] matrix with row stride ld.
template <bool kContig>
__device__ __forceinline__ int64_t unit_offset(int64_t u, int64_t upr, int64_t ld) {
  if (kContig) return u * kUnitElems;
  const int64_t r = u / upr;
  return r * ld + (u - r * upr) * kUnitElems;
}

// Two consecutive lanes own one unit: lane l loads the 16-byte chunks l, l + 2, l + 4, l + 6 of its 128
// bytes, i.e. the level-2 groups of that parity, so that each load instruction of a warp reads one
// full 32-byte sector per unit and the per-unit scalar work (scale, reciprocal, metadata) is shared
// by 32 elements.  A warp handles 16 units per pass and issues all 4 * kUnrollBf16 loads before it computes.
constexpr int kUnrollBf16 = 2;

template <bool kRHA, bool kContig>
__global__ void __launch_bounds__(kThreads)
quantize_bf16_kernel(const uint16_t* __restrict__ src, int64_t n_units, int64_t upr, int64_t ld_src,
                     uint32_t* __restrict__ dst) {
  const int lane = threadIdx.x & 31;
  const int l = lane & 1;
  const int64_t warp = (static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x) >> 5;
  const int64_t first = warp * (16 * kUnrollBf16) + (lane >> 1);
  uint4 v[kUnrollBf16][4];
#pragma unroll
  for (int i = 0; i < kUnrollBf16; ++i) {
    const int64_t u = first + 16 * i;
#pragma unroll
    for (int c = 0; c < 4; ++c) v[i][c] = make_uint4(0u, 0u, 0u, 0u);
    if (u < n_units) {
      const uint4* p = reinterpret_cast<const uint4*>(src + unit_offset<kContig>(u, upr, ld_src)) + l;
#pragma unroll
      for (int c = 0; c < 4; ++c) v[i][c] = ld_stream(p + 2 * c);
    }
  }

#pragma unroll
  for (int i = 0; i < kUnrollBf16; ++i) {
    const int64_t u = first + 16 * i;
    uint32_t codes[4], meta;
    encode_unit_bf16_pair<kRHA>(v[i], l, codes, meta);

    if (u < n_units) {
      uint32_t* out = dst + u * kUnitWords;
#pragma unroll
      for (int c = 0; c < 4; ++c) st_stream(out + 1 + 2 * c + l, codes[c]);
      if (l == 0) st_stream(out, meta);
    }
  }
}

// ----------------------------------------------------------------------------- BF16 quantizer, units down the columns
// One 64-thread block converts a tile of 64 rows x 128 columns: the rows are read as they lie (256 bytes each) and
// staged in shared memory with 16-byte stores; each pair of lanes (l and l + 16 of a warp) then takes four
// neighbouring columns (one 8-byte load per row) as its four units, lane l again the level-2 groups l, l + 2,
// l + 4, l + 6 of each.  The 16 lanes of a half warp read 128 consecutive bytes of one row: no bank conflicts,
// and a quarter of the shared-memory instructions that 4-byte accesses need.  Same encoder as above, so the
// units are those of hif4_quantize on the transposed matrix.
constexpr int kTileCols = 128;
constexpr int kTileThreads = 64;
constexpr int kTileRowWords = kTileCols / 2;

// Writes the `ncols` units of a tile (9 words each, one after the other in `units`) to their columns of dst: unit c
// goes to row tile blockIdx.x of column c0 + c.
__device__ __forceinline__ void flush_tile_units(const uint32_t* units, uint32_t* __restrict__ dst, int64_t c0, int ncols,
                                                 int64_t units_per_col) {
  for (int i = threadIdx.x; i < ncols * kUnitWords; i += kTileThreads) {
    const int c = i / kUnitWords, w = i - c * kUnitWords;
    st_stream(dst + ((c0 + c) * units_per_col + blockIdx.x) * kUnitWords + w, units[i]);
  }
}

template <bool kRHA>
__global__ void __launch_bounds__(kTileThreads)
quantize_bf16_transposed_kernel(const uint16_t* __restrict__ src, int64_t rows, int64_t cols, int64_t ld_src,
                                uint32_t* __restrict__ dst) {
  __shared__ __align__(16) uint32_t tile[kUnitElems * kTileRowWords];
  // consecutive blocks take consecutive row tiles of the same columns: their units are neighbours in dst
  const int64_t c0 = static_cast<int64_t>(blockIdx.y) * kTileCols;
  const int64_t r0 = static_cast<int64_t>(blockIdx.x) * kUnitElems;
  // 64 rows x 16 chunks of 8 elements; a chunk is inside the matrix or outside as a whole (cols % 8 == 0)
  constexpr int kChunks = kUnitElems * (kTileCols / 8) / kTileThreads;      // 16 per thread
  // asynchronous 16-byte copies straight into shared memory (no registers, one instruction per chunk instead of a
  // load and a store); chunks outside the matrix are filled with zeros
  const uint32_t tile_addr = static_cast<uint32_t>(__cvta_generic_to_shared(tile));
#pragma unroll
  for (int n = 0; n < kChunks; ++n) {
    const int i = n * kTileThreads + threadIdx.x, r = i >> 4, ch = i & 15;           // row i / 16, words 4 (i % 16) ..
    const bool inside = c0 + 8 * ch < cols;
    const uint16_t* p = inside ? src + (r0 + r) * ld_src + c0 + 8 * ch : src;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(tile_addr + 16u * i), "l"(p), "r"(inside ? 16 : 0) : "memory");
  }
  asm volatile("cp.async.commit_group;" ::: "memory");
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  __syncthreads();
  const int lane = threadIdx.x & 31, l = lane >> 4;
  const int cq = (threadIdx.x >> 5) * 16 + (lane & 15);                      // columns 4 cq .. 4 cq + 3 of the tile
  uint4 col[4][4];                                                           // [column][group l + 2c]
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    const uint32_t* p = tile + (8 * (l + 2 * c)) * kTileRowWords + 2 * cq;   // rows 8 g .. 8 g + 7, four columns
    uint32_t e[4][4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const uint2 a = *reinterpret_cast<const uint2*>(p + (2 * k) * kTileRowWords);
      const uint2 b2 = *reinterpret_cast<const uint2*>(p + (2 * k + 1) * kTileRowWords);
      e[0][k] = prmt(a.x, b2.x, 0x5410u);                     // low halves: column 0 of rows 2k, 2k + 1
      e[1][k] = prmt(a.x, b2.x, 0x7632u);                     // high halves: column 1
      e[2][k] = prmt(a.y, b2.y, 0x5410u);
      e[3][k] = prmt(a.y, b2.y, 0x7632u);
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) col[j][c] = make_uint4(e[j][0], e[j][1], e[j][2], e[j][3]);
  }
  const int64_t units_per_col = rows / kUnitElems;
  // The units of neighbouring columns lie a whole column apart in dst: written straight from the encoder's registers,
  // every 4-byte store of a warp would go to 32 different sectors.  They are collected in the tile's shared memory
  // instead (all its rows have been read) and written with nine consecutive lanes per unit.
  __syncthreads();
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    uint32_t codes[4], meta;
    encode_unit_bf16_pair<kRHA, 16>(col[j], l, codes, meta);
    uint32_t* out = tile + (4 * cq + j) * kUnitWords;
#pragma unroll
    for (int g = 0; g < 4; ++g) out[1 + 2 * g + l] = codes[g];
    if (l == 0) out[0] = meta;
  }
  __syncthreads();
  flush_tile_units(tile, dst, c0, static_cast<int>(cols - c0 < kTileCols ? cols - c0 : kTileCols), units_per_col);
}

// ----------------------------------------------------------------------------- FP32 quantizer
// 4 lanes per unit.  Lane l loads the level-3 groups l, l + 4, l + 8, l + 12 (4 elements each: 16-byte chunks
// of an FP32 unit, 8-byte chunks of an FP16 unit); lanes 2w', 2w'+1 together hold the level-2
// groups w' + 2c (c = 0..3).  A warp covers 8 units per pass.
constexpr int kUnrollFp32 = 2;

template <bool kRHA, bool kContig, typename Src>
__global__ void __launch_bounds__(kThreads)
quantize_fp32_kernel(const Src* __restrict__ src, int64_t n_units, int64_t upr, int64_t ld_src,
                     uint32_t* __restrict__ dst) {
  const int lane = threadIdx.x & 31;
  const int l = lane & 3;
  const int64_t warp = (static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x) >> 5;
  const int64_t first = warp * (8 * kUnrollFp32) + (lane >> 2);

  uint4 v[kUnrollFp32][4];
#pragma unroll
  for (int i = 0; i < kUnrollFp32; ++i) {
    const int64_t u = first + 8 * i;
#pragma unroll
    for (int c = 0; c < 4; ++c) v[i][c] = make_uint4(0u, 0u, 0u, 0u);
    if (u < n_units) {
      const Src* p = src + unit_offset<kContig>(u, upr, ld_src) + 4 * l;
#pragma unroll
      for (int c = 0; c < 4; ++c) v[i][c] = load_group_fp32(p + 16 * c);
    }
  }

#pragma unroll
  for (int i = 0; i < kUnrollFp32; ++i) {
    const int64_t u = first + 8 * i;
    uint32_t codes[4], meta;
    encode_unit_fp32_quad<kRHA>(v[i], l, codes, meta);

    if (u < n_units) {
      uint32_t* out = dst + u * kUnitWords;
      if ((l & 1) == 0) {
#pragma unroll
        for (int c = 0; c < 4; ++c) st_stream(out + 1 + (l >> 1) + 2 * c, codes[c]);
      }
      if (l == 0) st_stream(out, meta);
    }
  }
}

// ----------------------------------------------------------------------------- FP32 / FP16 quantizer, units down the columns
// Same plan as the BF16 kernel above on a tile of 64 rows x 64 columns held as FP32 words (FP16 elements are widened
// when they are staged): four lanes per unit, lanes l, l + 8, l + 16, l + 24 of a warp, each quad taking four
// neighbouring columns with one 16-byte load per row (the eight lanes of a quarter warp read 128 consecutive bytes).
constexpr int kTileCols32 = 64;

template <bool kRHA, typename Src>
__global__ void __launch_bounds__(kTileThreads)
quantize_fp32_transposed_kernel(const Src* __restrict__ src, int64_t rows, int64_t cols, int64_t ld_src,
                                uint32_t* __restrict__ dst) {
  __shared__ __align__(16) uint32_t tile[kUnitElems * kTileCols32];
  const int64_t c0 = static_cast<int64_t>(blockIdx.y) * kTileCols32;
  const int64_t r0 = static_cast<int64_t>(blockIdx.x) * kUnitElems;
  // 64 rows x 16 chunks of 4 elements; a chunk is inside the matrix or outside as a whole (cols % 8 == 0)
  constexpr int kChunks = kUnitElems * (kTileCols32 / 4) / kTileThreads;    // 16 per thread
  if constexpr (sizeof(Src) == 4) {
    // FP32 source: asynchronous 16-byte copies straight into shared memory, zeros outside the matrix
    const uint32_t tile_addr = static_cast<uint32_t>(__cvta_generic_to_shared(tile));
#pragma unroll
    for (int n = 0; n < kChunks; ++n) {
      const int i = n * kTileThreads + threadIdx.x, r = i >> 4, ch = i & 15;         // row i / 16, words 4 (i % 16) ..
      const bool inside = c0 + 4 * ch < cols;
      const Src* p = inside ? src + (r0 + r) * ld_src + c0 + 4 * ch : src;
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(tile_addr + 16u * i), "l"(p), "r"(inside ? 16 : 0) : "memory");
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    asm volatile("cp.async.wait_group 0;" ::: "memory");
  } else {
    uint4 in[kChunks];                                   // FP16 source: widened on the way
#pragma unroll
    for (int n = 0; n < kChunks; ++n) {
      const int i = n * kTileThreads + threadIdx.x, r = i >> 4, ch = i & 15;
      in[n] = make_uint4(0u, 0u, 0u, 0u);
      if (c0 + 4 * ch < cols) in[n] = load_group_fp32(src + (r0 + r) * ld_src + c0 + 4 * ch);
    }
#pragma unroll
    for (int n = 0; n < kChunks; ++n) {
      const int i = n * kTileThreads + threadIdx.x;
      *reinterpret_cast<uint4*>(tile + 4 * i) = in[n];                       // row i / 16, words 4 (i % 16) ..
    }
  }
  __syncthreads();
  const int lane = threadIdx.x & 31, l = lane >> 3;
  const int cq = (threadIdx.x >> 5) * 8 + (lane & 7);                        // columns 4 cq .. 4 cq + 3 of the tile
  uint32_t col[4][4][4];                                                     // [column][group l + 4c][row of the group]
#pragma unroll
  for (int c = 0; c < 4; ++c)
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const uint4 a = *reinterpret_cast<const uint4*>(tile + (4 * (l + 4 * c) + k) * kTileCols32 + 4 * cq);
      col[0][c][k] = a.x; col[1][c][k] = a.y; col[2][c][k] = a.z; col[3][c][k] = a.w;
    }
  const int64_t units_per_col = rows / kUnitElems;
  __syncthreads();                                       // the units are collected in the tile's shared memory, as above
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    uint4 v[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) v[c] = make_uint4(col[j][c][0], col[j][c][1], col[j][c][2], col[j][c][3]);
    uint32_t codes[4], meta;
    encode_unit_fp32_quad<kRHA, 8>(v, l, codes, meta);
    uint32_t* out = tile + (4 * cq + j) * kUnitWords;
    if ((l & 1) == 0) {
#pragma unroll
      for (int g = 0; g < 4; ++g) out[1 + (l >> 1) + 2 * g] = codes[g];
    }
    if (l == 0) out[0] = meta;
  }
  __syncthreads();
  flush_tile_units(tile, dst, c0, static_cast<int>(cols - c0 < kTileCols32 ? cols - c0 : kTileCols32), units_per_col);
}

template <typename Src>
void launch_quantize_fp32_transposed(const Src* x, bool rha, dim3 grid, cudaStream_t st, int64_t rows, int64_t cols,
                                     int64_t ld_src, uint32_t* dst) {
  if (rha) quantize_fp32_transposed_kernel<true, Src><<<grid, kTileThreads, 0, st>>>(x, rows, cols, ld_src, dst);
  else quantize_fp32_transposed_kernel<false, Src><<<grid, kTileThreads, 0, st>>>(x, rows, cols, ld_src, dst);
}

// ----------------------------------------------------------------------------- dequantizer (Eq. 2)
// BF16 output: 8 lanes per unit, lane j decodes code word j (elements 8j..8j+7, 16 bytes of output).  FP32 output:
// 16 lanes per unit, lane k decodes half k & 1 of code word k >> 1 (4 elements, again 16 bytes of output), so that
// every store instruction of a warp writes whole, consecutive sectors.  Each value is
// m * (4+M) * 2^(E-48-4+e8+e16): an integer below 64 times a power of two, exact in BF16 (and so in FP32).
template <bool kBF16Out, bool kContig>
__global__ void __launch_bounds__(kThreads)
dequantize_kernel(const uint32_t* __restrict__ src, int64_t n_units, int64_t upr, int64_t ld_dst,
                  void* __restrict__ dst) {
  constexpr int kLanes = kBF16Out ? 8 : 16;                   // lanes per unit
  constexpr int kUnroll = kBF16Out ? kUnrollDeqBf16 : kUnrollDeqFp32;
  const int lane = threadIdx.x & 31;
  const int k = lane & (kLanes - 1);
  const int j = kBF16Out ? k : k >> 1;                        // code word
  const int64_t warp = (static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x) >> 5;
  const int64_t first = warp * ((32 / kLanes) * kUnroll) + lane / kLanes;

  uint32_t meta[kUnroll], word[kUnroll];
#pragma unroll
  for (int i = 0; i < kUnroll; ++i) {
    const int64_t u = first + (32 / kLanes) * i;
    meta[i] = 0; word[i] = 0;
    if (u < n_units) {
      meta[i] = __ldg(src + u * kUnitWords);
      word[i] = __ldg(src + u * kUnitWords + 1 + j);
    }
  }
#pragma unroll
  for (int i = 0; i < kUnroll; ++i) {
    const int64_t u = first + (32 / kLanes) * i;
    if (u >= n_units) continue;
    const uint32_t byte = meta[i] & 0xFFu;
    const uint32_t e8 = (meta[i] >> (8 + j)) & 1u;
    const uint32_t e16a = (meta[i] >> (16 + 2 * j)) & 1u, e16b = (meta[i] >> (17 + 2 * j)) & 1u;
    // Packed BF16 arithmetic, two elements per instruction: S = E6M2 / 4 * 2^shift as BF16 bits is
    // ((byte + 308) << 5) + (shift << 7); (128 + m) * S - 128 * S in one fused multiply-add is m * S exactly; the
    // sign bit goes on afterwards so that a negative zero stays negative.
    const uint32_t base = (byte + 308u) << 5;
    const uint32_t S = (base + ((e8 + e16a) << 7)) | ((base + ((e8 + e16b) << 7)) << 16);   // (elements 0..3, elements 4..7)
    const uint32_t O = S + 0x83808380u;                                                     // -128 S
    const uint32_t w = word[i];
    uint32_t r[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {                                                           // elements e and e + 4
      const uint32_t c = w >> (4 * e);
      r[e] = fma_bf16x2((c & 0x00070007u) | 0x43004300u, S, O) | ((c << 12) & 0x80008000u);
      if (byte == 0xFFu) r[e] = 0x7FC07FC0u;                                                // NaN unit
    }
    if (kBF16Out) {
      const int64_t off = unit_offset<kContig>(u, upr, ld_dst) + 8 * j;
      uint4 o;
      o.x = prmt(r[0], r[1], 0x5410u);          // elements 0, 1
      o.y = prmt(r[2], r[3], 0x5410u);          // elements 2, 3
      o.z = prmt(r[0], r[1], 0x7632u);          // elements 4, 5
      o.w = prmt(r[2], r[3], 0x7632u);          // elements 6, 7
      st_stream(reinterpret_cast<uint4*>(static_cast<uint16_t*>(dst) + off), o);
    } else {                                    // a BF16 widens to FP32 by appending sixteen zero bits
      const int64_t off = unit_offset<kContig>(u, upr, ld_dst) + 4 * k;
      const uint4 o = (k & 1) ? make_uint4(r[0] & 0xFFFF0000u, r[1] & 0xFFFF0000u, r[2] & 0xFFFF0000u, r[3] & 0xFFFF0000u)
                              : make_uint4(r[0] << 16, r[1] << 16, r[2] << 16, r[3] << 16);
      st_stream(reinterpret_cast<uint4*>(static_cast<float*>(dst) + off), o);
    }
  }
}

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

template <typename Src>
void launch_quantize_fp32(const Src* x, bool rha, bool contig, dim3 grid, cudaStream_t st, int64_t n_units, int64_t upr,
                          int64_t ld_src, uint32_t* dst) {
  if (!rha && contig) quantize_fp32_kernel<false, true, Src><<<grid, kThreads, 0, st>>>(x, n_units, upr, ld_src, dst);
  else if (!rha) quantize_fp32_kernel<false, false, Src><<<grid, kThreads, 0, st>>>(x, n_units, upr, ld_src, dst);
  else if (contig) quantize_fp32_kernel<true, true, Src><<<grid, kThreads, 0, st>>>(x, n_units, upr, ld_src, dst);
  else quantize_fp32_kernel<true, false, Src><<<grid, kThreads, 0, st>>>(x, n_units, upr, ld_src, dst);
}

}  // namespace
}  // namespace hif4

using namespace hif4;

extern "C" hif4_status hif4_quantize(const void* src, hif4_dtype dt, int64_t rows, int64_t cols,
                                     int64_t ld_src, void* dst_units, hif4_round mode, void* stream) {
  if (dt != HIF4_BF16 && dt != HIF4_FP32 && dt != HIF4_FP16) return HIF4_ERR_DTYPE;
  if (mode != HIF4_RNE && mode != HIF4_RHA) return HIF4_ERR_DTYPE;
  if (rows < 0 || cols < 0 || cols % kUnitElems != 0 || ld_src < cols) return HIF4_ERR_SHAPE;
  if (rows == 0 || cols == 0) return HIF4_OK;
  if (!src || !dst_units) return HIF4_ERR_NULL;
  const size_t esz = dt == HIF4_FP32 ? 4 : 2;
  if (!aligned(src, 16) || (static_cast<size_t>(ld_src) * esz) % 16 != 0 || !aligned(dst_units, 4))
    return HIF4_ERR_ALIGN;
  const int64_t upr = cols / kUnitElems;
  const int64_t n_units = rows * upr;
  const bool contig = ld_src == cols;
  const int units_per_block = (kThreads / 32) * (dt == HIF4_BF16 ? 16 * kUnrollBf16 : 8 * kUnrollFp32);
  const int64_t blocks = ceil_div64(n_units, units_per_block);
  if (blocks > 0x7FFFFFFFll) return HIF4_ERR_SHAPE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint32_t* dst = static_cast<uint32_t*>(dst_units);
  const dim3 grid(static_cast<unsigned>(blocks));
  const bool rha = mode == HIF4_RHA;
  if (dt == HIF4_BF16) {
    const uint16_t* x = static_cast<const uint16_t*>(src);
    if (!rha && contig) quantize_bf16_kernel<false, true><<<grid, kThreads, 0, st>>>(x, n_units, upr, ld_src, dst);
    else if (!rha) quantize_bf16_kernel<false, false><<<grid, kThreads, 0, st>>>(x, n_units, upr, ld_src, dst);
    else if (contig) quantize_bf16_kernel<true, true><<<grid, kThreads, 0, st>>>(x, n_units, upr, ld_src, dst);
    else quantize_bf16_kernel<true, false><<<grid, kThreads, 0, st>>>(x, n_units, upr, ld_src, dst);
  } else if (dt == HIF4_FP32) {
    launch_quantize_fp32(static_cast<const float*>(src), rha, contig, grid, st, n_units, upr, ld_src, dst);
  } else {
    launch_quantize_fp32(static_cast<const __half*>(src), rha, contig, grid, st, n_units, upr, ld_src, dst);
  }
  note_launch();
  return launch_status();
}

extern "C" hif4_status hif4_quantize_transposed(const void* src, hif4_dtype dt, int64_t rows, int64_t cols,
                                                int64_t ld_src, void* dst_units, hif4_round mode, void* stream) {
  if (dt != HIF4_BF16 && dt != HIF4_FP32 && dt != HIF4_FP16) return HIF4_ERR_DTYPE;
  if (mode != HIF4_RNE && mode != HIF4_RHA) return HIF4_ERR_DTYPE;
  if (rows < 0 || cols < 0 || rows % kUnitElems != 0 || cols % 8 != 0 || ld_src < cols) return HIF4_ERR_SHAPE;
  if (rows == 0 || cols == 0) return HIF4_OK;
  if (!src || !dst_units) return HIF4_ERR_NULL;
  const size_t esz = dt == HIF4_FP32 ? 4 : 2;
  if (!aligned(src, 16) || (static_cast<size_t>(ld_src) * esz) % 16 != 0 || !aligned(dst_units, 4)) return HIF4_ERR_ALIGN;
  const int64_t col_tiles = ceil_div64(cols, dt == HIF4_BF16 ? kTileCols : kTileCols32), row_tiles = rows / kUnitElems;
  if (row_tiles > 0x7FFFFFFFll || col_tiles > 65535) return HIF4_ERR_SHAPE;
  const dim3 grid(static_cast<unsigned>(row_tiles), static_cast<unsigned>(col_tiles));
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint32_t* dst = static_cast<uint32_t*>(dst_units);
  const bool rha = mode == HIF4_RHA;
  if (dt == HIF4_BF16) {
    const uint16_t* x = static_cast<const uint16_t*>(src);
    if (rha) quantize_bf16_transposed_kernel<true><<<grid, kTileThreads, 0, st>>>(x, rows, cols, ld_src, dst);
    else quantize_bf16_transposed_kernel<false><<<grid, kTileThreads, 0, st>>>(x, rows, cols, ld_src, dst);
  } else if (dt == HIF4_FP32) {
    launch_quantize_fp32_transposed(static_cast<const float*>(src), rha, grid, st, rows, cols, ld_src, dst);
  } else {
    launch_quantize_fp32_transposed(static_cast<const __half*>(src), rha, grid, st, rows, cols, ld_src, dst);
  }
  note_launch();
  return launch_status();
}

extern "C" hif4_status hif4_dequantize(const void* src_units, int64_t rows, int64_t cols, void* dst,
                                       hif4_dtype dt, int64_t ld_dst, void* stream) {
  if (dt != HIF4_BF16 && dt != HIF4_FP32) return HIF4_ERR_DTYPE;
  if (rows < 0 || cols < 0 || cols % kUnitElems != 0 || ld_dst < cols) return HIF4_ERR_SHAPE;
  if (rows == 0 || cols == 0) return HIF4_OK;
  if (!src_units || !dst) return HIF4_ERR_NULL;
  const size_t esz = dt == HIF4_BF16 ? 2 : 4;
  if (!aligned(dst, 16) || (static_cast<size_t>(ld_dst) * esz) % 16 != 0 || !aligned(src_units, 4))
    return HIF4_ERR_ALIGN;
  const int64_t upr = cols / kUnitElems;
  const int64_t n_units = rows * upr;
  const bool contig = ld_dst == cols;
  const int64_t blocks = ceil_div64(n_units, (kThreads / 32) * (dt == HIF4_BF16 ? kUnrollDeqBf16 * 4 : kUnrollDeqFp32 * 2));
  if (blocks > 0x7FFFFFFFll) return HIF4_ERR_SHAPE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const uint32_t* in = static_cast<const uint32_t*>(src_units);
  const dim3 grid(static_cast<unsigned>(blocks));
  if (dt == HIF4_BF16) {
    if (contig) dequantize_kernel<true, true><<<grid, kThreads, 0, st>>>(in, n_units, upr, ld_dst, dst);
    else dequantize_kernel<true, false><<<grid, kThreads, 0, st>>>(in, n_units, upr, ld_dst, dst);
  } else {
    if (contig) dequantize_kernel<false, true><<<grid, kThreads, 0, st>>>(in, n_units, upr, ld_dst, dst);
    else dequantize_kernel<false, false><<<grid, kThreads, 0, st>>>(in, n_units, upr, ld_dst, dst);
  }
  note_launch();
  return launch_status();
}
