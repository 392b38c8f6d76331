// Tensor-core HiF4 x HiF4 -> FP32 GEMM for sm_100a: C = A * B^T (Eq. 3 summed over unit pairs).
//
// Every HiF4 value, level-1 scale included, is exactly a BF16 (at most 6 significant bits, exponent
// in [-50, 18]), and a product of two of them is exact in the FP32 accumulator, so the contraction
// runs as a BF16 tcgen05.mma (kind::f16) with accumulators in tensor memory.  Packed units never
// expand in HBM: a persistent, warp-specialised CTA
//   warp 0      TMA producer: raw units (4 units = 144 B per row, i.e. K = 256) -> shared memory
//   warps 6-17  decode: one thread per tile row turns one unit (Eq. 2) into 64 BF16 values and writes
//               them as one 128-byte row of a K-major SWIZZLE_128B operand tile
//   warp 1      issues tcgen05.mma (128 x 256 x 16, four per 64-wide K block) and commits to mbarriers
//   warps 2-5   epilogue: tcgen05.ld the finished accumulator and store FP32 rows of C
// with two raw stages, two decoded stages and two 256-column accumulators, so that the epilogue of a
// tile overlaps the main loop of the next.
//
// Decode arithmetic (per 32-bit code word = 8 elements = one level-2 group): a magnitude field m is
// OR-ed into the mantissa of the BF16 constant 128 (or 128 + 16 m for fields that sit four bits
// higher), and one fma.rn.bf16x2 with (S, -128 S) (or (S/16, -8 S)) yields m * S exactly, S being
// E6M2 * 2^(E1_8 + E1_16 - 2) for the element's level-3 group; the sign bit is XOR-ed in.  Elements k
// and k+4 of a word share a register, so inside a unit the K order is permuted; A and B use the same
// permutation and the contraction does not depend on it.
//
// Every wait on an mbarrier is bounded: when the budget runs out the kernel raises an error word,
// every role leaves its loop, tensor memory is released and the kernel returns.
#include "hif4_common.cuh"
#include "hif4_gemm_internal.cuh"
#include "hif4_tc_common.cuh"

namespace hif4 {
namespace {

constexpr int BM = 128;
constexpr int BN = 256;
constexpr int kRawABytes = BM * kRawRowBytes;         // 18432
constexpr int kRawBBytes = BN * kRawRowBytes;         // 36864
constexpr int kRawStageBytes = kRawABytes + kRawBBytes;
constexpr int kDecABytes = BM * 128;                  // 128 rows x 64 BF16
constexpr int kDecBBytes = BN * 128;
constexpr int kDecStageBytes = kDecABytes + kDecBBytes;
constexpr int kRawStages = 2;
constexpr int kDecStages = 2;
constexpr int kAccStages = 2;
constexpr int kTmemCols = 512;

constexpr int kEpilogueWarp0 = 2;
constexpr int kDecodeWarp0 = 6;
constexpr int kDecodeThreads = BM + BN;               // 384: one thread per tile row
constexpr int kThreads = kDecodeWarp0 * 32 + kDecodeThreads;   // 576

constexpr int kSmemBarriers = 16 * 8;
constexpr int kSmemBytes = 1024 /*alignment slack*/ + kDecStages * kDecStageBytes +
                           kRawStages * kRawStageBytes + kSmemBarriers + 64;

// Instruction descriptor of tcgen05.mma kind::f16: D = F32, A = B = BF16, both K-major, N/8, M/16.
constexpr uint32_t kInstrDesc = (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(BN >> 3) << 17) |
                                (static_cast<uint32_t>(BM >> 4) << 24);

struct MTile { int row0; int row_end; int group; int pad; };

struct GemmParams {
  float* C;
  int64_t ldc;
  int64_t M;            // rows of A (all groups)
  int64_t N;            // columns of C = rows of one B matrix
  int num_kc;           // K / 256
  int n_tiles;          // ceil(N / BN)
  int m_tiles;          // number of entries to walk (grouped: upper bound)
  const MTile* table;   // nullptr: dense problem
  unsigned int* error_word;
};

struct TileCoord { int m0; int m_end; int n0; int b_row0; bool valid; };

__device__ __forceinline__ TileCoord tile_coord(const GemmParams& p, int t) {
  TileCoord c;
  const int mt = t / p.n_tiles, nt = t - mt * p.n_tiles;
  c.n0 = nt * BN;
  if (p.table) {
    const MTile e = p.table[mt];
    c.valid = e.group >= 0;
    c.m0 = e.row0;
    c.m_end = e.row_end;
    c.b_row0 = static_cast<int>(e.group * p.N) + c.n0;
  } else {
    c.valid = true;
    c.m0 = mt * BM;
    c.m_end = static_cast<int>(p.M);
    c.b_row0 = c.n0;
  }
  return c;
}

__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t dec_base = smem_base;                                        // 1024-byte aligned stages
  const uint32_t raw_base = dec_base + kDecStages * kDecStageBytes;
  const uint32_t bar_base = raw_base + kRawStages * kRawStageBytes;
  const uint32_t raw_full = bar_base, raw_empty = bar_base + 16, dec_full = bar_base + 32,
                 dec_empty = bar_base + 48, tmem_full = bar_base + 64, tmem_empty = bar_base + 80;
  uint8_t* gen_base = smem_raw + (smem_base - smem_u32(smem_raw));
  volatile uint32_t* tmem_ptr_smem = reinterpret_cast<volatile uint32_t*>(gen_base + (bar_base - smem_base) + 96);
  volatile uint32_t* abort_flag = tmem_ptr_smem + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int total_tiles = p.m_tiles * p.n_tiles;

  if (threadIdx.x == 0) {
    for (int s = 0; s < 2; ++s) {
      mbar_init(raw_full + 8 * s, 1);
      mbar_init(raw_empty + 8 * s, kDecodeThreads);
      mbar_init(dec_full + 8 * s, kDecodeThreads);
      mbar_init(dec_empty + 8 * s, 1);
      mbar_init(tmem_full + 8 * s, 1);
      mbar_init(tmem_empty + 8 * s, 128);
    }
    *abort_flag = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(bar_base + 96),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_ptr_smem;

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer
    if (lane == 0) {
      uint32_t rc = 0;
      for (int t = blockIdx.x; t < total_tiles; t += gridDim.x) {
        const TileCoord tc = tile_coord(p, t);
        if (!tc.valid) continue;
        bool ok = true;
        for (int kc = 0; kc < p.num_kc; ++kc, ++rc) {
          const uint32_t s = rc & 1u, ph = (rc >> 1) & 1u;
          if (!(ok = mbar_wait(raw_empty + 8 * s, ph ^ 1u, abort_flag))) break;
          mbar_expect_tx(raw_full + 8 * s, kRawStageBytes);
          const uint32_t dst = raw_base + s * kRawStageBytes;
          tma_load_2d(dst, &tmA, kc * kRawRowBytes, tc.m0, raw_full + 8 * s);
          tma_load_2d(dst + kRawABytes, &tmB, kc * kRawRowBytes, tc.b_row0, raw_full + 8 * s);
        }
        if (!ok) break;
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      uint32_t dc = 0, tcount = 0;
      for (int t = blockIdx.x; t < total_tiles; t += gridDim.x) {
        const TileCoord tc = tile_coord(p, t);
        if (!tc.valid) continue;
        const uint32_t acc = tcount & 1u, aph = (tcount >> 1) & 1u;
        bool ok = mbar_wait(tmem_empty + 8 * acc, aph ^ 1u, abort_flag);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * BN;
        const int num_kb = p.num_kc * kRawUnits;
        for (int kb = 0; kb < num_kb; ++kb, ++dc) {
          const uint32_t s = dc & 1u, ph = (dc >> 1) & 1u;
          if (!(ok = mbar_wait(dec_full + 8 * s, ph, abort_flag))) break;
          tc_fence_after();
          const uint64_t adesc = make_desc(dec_base + s * kDecStageBytes);
          const uint64_t bdesc = make_desc(dec_base + s * kDecStageBytes + kDecABytes);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)
            tc_mma(d_tmem, adesc + 2 * kk, bdesc + 2 * kk, kInstrDesc, (kb | kk) != 0 ? 1u : 0u);
          tc_commit(dec_empty + 8 * s);          // arrives once these MMAs have read the stage
        }
        if (!ok) break;
        tc_commit(tmem_full + 8 * acc);          // accumulator complete
        ++tcount;
      }
    }
  } else if (warp < kDecodeWarp0) {
    // ---------------------------------------------------------------- epilogue
    const int q = warp & 3;                      // TMEM lane quadrant this warp may read
    uint32_t tcount = 0;
    const bool vec_ok = ((reinterpret_cast<uintptr_t>(p.C) & 15u) == 0) && (p.ldc % 4 == 0);
    for (int t = blockIdx.x; t < total_tiles; t += gridDim.x) {
      const TileCoord tc = tile_coord(p, t);
      if (!tc.valid) continue;
      const uint32_t acc = tcount & 1u, aph = (tcount >> 1) & 1u;
      if (!mbar_wait(tmem_full + 8 * acc, aph, abort_flag)) break;
      tc_fence_after();
      const int row = tc.m0 + q * 32 + lane;
      const bool row_ok = row < tc.m_end;
      float* crow = p.C + static_cast<int64_t>(row) * p.ldc + tc.n0;
#pragma unroll 1
      for (int c = 0; c < BN / 32; ++c) {
        uint32_t r[32];
        tc_ld32(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc * BN + c * 32, r);
        tc_wait_ld();
        const int64_t col0 = static_cast<int64_t>(tc.n0) + c * 32;
        if (row_ok && col0 < p.N) {
          if (vec_ok && col0 + 32 <= p.N) {
#pragma unroll
            for (int v = 0; v < 8; ++v)
              *reinterpret_cast<uint4*>(crow + c * 32 + 4 * v) = make_uint4(r[4 * v], r[4 * v + 1], r[4 * v + 2], r[4 * v + 3]);
          } else {
#pragma unroll
            for (int v = 0; v < 32; ++v)
              if (col0 + v < p.N) crow[c * 32 + v] = __uint_as_float(r[v]);
          }
        }
      }
      tc_fence_before();
      mbar_arrive(tmem_empty + 8 * acc);
      ++tcount;
    }
  } else {
    // ---------------------------------------------------------------- decode
    const int d = threadIdx.x - kDecodeWarp0 * 32;            // tile row: 0..127 A, 128..383 B
    const bool isA = d < BM;
    const uint32_t r7 = static_cast<uint32_t>(d) & 7u;
    const uint32_t raw_row = (isA ? 0u : static_cast<uint32_t>(kRawABytes)) +
                             static_cast<uint32_t>(isA ? d : d - BM) * kRawRowBytes;
    const uint32_t dec_row = (isA ? 0u : static_cast<uint32_t>(kDecABytes)) + static_cast<uint32_t>(isA ? d : d - BM) * 128u;
    uint32_t rc = 0, dc = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
      const TileCoord tc = tile_coord(p, t);
      if (!tc.valid) continue;
      for (int kc = 0; kc < p.num_kc && ok; ++kc, ++rc) {
        const uint32_t s = rc & 1u, ph = (rc >> 1) & 1u;
        if (!(ok = mbar_wait(raw_full + 8 * s, ph, abort_flag))) break;
        uint32_t w[36];
        const uint32_t src = raw_base + s * kRawStageBytes + raw_row;
#pragma unroll
        for (int i = 0; i < 9; ++i) {
          const uint4 v = lds128(src + 16 * i);
          w[4 * i] = v.x; w[4 * i + 1] = v.y; w[4 * i + 2] = v.z; w[4 * i + 3] = v.w;
        }
        // The stage is refilled through the async proxy (TMA) while it was read through the generic
        // proxy: the proxy fence orders these reads before the release, so that no load is still
        // in flight when the next copy lands.
        fence_proxy_async_smem();
        mbar_arrive(raw_empty + 8 * s);
#pragma unroll
        for (int u = 0; u < kRawUnits; ++u, ++dc) {
          const uint32_t ds = dc & 1u, dph = (dc >> 1) & 1u;
          if (!(ok = mbar_wait(dec_empty + 8 * ds, dph ^ 1u, abort_flag))) break;
          decode_unit_to_row(w[9 * u], &w[9 * u + 1], dec_base + ds * kDecStageBytes + dec_row, r7);
          fence_proxy_async_smem();                           // generic-proxy writes -> visible to the tensor core
          mbar_arrive(dec_full + 8 * ds);
        }
      }
    }
  }

  // ------------------------------------------------------------------ teardown
  __syncwarp();
  if (*abort_flag) {
    // Some wait gave up: give copies and MMAs that are still in flight time to land before the
    // shared and tensor memory they target is released.
    const uint64_t t0 = global_ns();
    while (global_ns() - t0 < 2000000ull) {}
    if (threadIdx.x == 0) atomicExch(p.error_word, 1u);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

// Builds the m-tile table of a grouped problem from the device-side offsets: one entry per 128-row
// tile of every non-empty group, then invalid entries up to `max_tiles`.
__global__ void build_mtile_table_kernel(const int64_t* __restrict__ offsets, int num_groups, MTile* table,
                                         int max_tiles) {
  __shared__ int s_total;
  if (threadIdx.x == 0) {
    int n = 0;
    for (int g = 0; g < num_groups; ++g) {
      const int64_t lo = offsets[g], hi = offsets[g + 1];
      for (int64_t r = lo; r < hi && n < max_tiles; r += BM) {
        table[n].row0 = static_cast<int>(r);
        table[n].row_end = static_cast<int>(hi);
        table[n].group = g;
        table[n].pad = 0;
        ++n;
      }
    }
    s_total = n;
  }
  __syncthreads();
  for (int i = s_total + threadIdx.x; i < max_tiles; i += blockDim.x) {
    table[i].row0 = 0; table[i].row_end = 0; table[i].group = -1; table[i].pad = 0;
  }
}

// ------------------------------------------------------------------------------------ host side
hif4_status launch_tc(const void* A, const void* B, int64_t a_rows, int64_t b_rows, GemmParams p, int64_t K,
                      cudaStream_t st) {
  static uint64_t smem_opt_in = 0;
  if (!ensure_dynamic_smem(gemm_tc_kernel, kSmemBytes, smem_opt_in)) return HIF4_ERR_CUDA;
  CUtensorMap tmA, tmB;
  const int64_t upr = K / kUnitElems;
  if (!make_unit_map(&tmA, A, a_rows, upr, BM) || !make_unit_map(&tmB, B, b_rows, upr, BN)) return HIF4_ERR_CUDA;
  p.error_word = device_error_word();
  if (!p.error_word) return HIF4_ERR_CUDA;
  const int64_t tiles = static_cast<int64_t>(p.m_tiles) * p.n_tiles;
  const int grid = static_cast<int>(tiles < sm_count() ? tiles : sm_count());
  gemm_tc_kernel<<<grid, kThreads, kSmemBytes, st>>>(tmA, tmB, p);
  note_launch();
  return launch_status();
}

}  // namespace

bool gemm_tc_supported(const void* A, const void* B, int64_t a_rows, int64_t b_rows, int64_t N, int64_t K) {
  if (K <= 0 || K % (kRawUnits * kUnitElems) != 0) return false;                 // TMA row pitch must be a multiple of 16 B
  if ((reinterpret_cast<uintptr_t>(A) | reinterpret_cast<uintptr_t>(B)) & 15u) return false;
  if (a_rows >= (1ll << 31) - BM || b_rows >= (1ll << 31) - BN || N >= (1ll << 31) - BN) return false;
  if ((K / kUnitElems) * kUnitBytes >= (1ll << 31)) return false;
  return encode_tiled_fn() != nullptr;
}

hif4_status launch_gemm_tc(const void* A, const void* B, float* C, int64_t M, int64_t N, int64_t K, int64_t ldc,
                           cudaStream_t st) {
  GemmParams p{};
  p.C = C; p.ldc = ldc; p.M = M; p.N = N;
  p.num_kc = static_cast<int>(K / (kRawUnits * kUnitElems));
  p.n_tiles = static_cast<int>(ceil_div64(N, BN));
  p.m_tiles = static_cast<int>(ceil_div64(M, BM));
  p.table = nullptr;
  return launch_tc(A, B, M, N, p, K, st);
}

size_t grouped_tc_workspace_bytes(int num_groups, int64_t total_rows) {
  const int64_t max_tiles = ceil_div64(total_rows, BM) + num_groups;
  return static_cast<size_t>((max_tiles * static_cast<int64_t>(sizeof(MTile)) + 255) / 256 * 256);
}

hif4_status launch_grouped_gemm_tc(const void* A, const void* B, float* C, const int64_t* offsets, int num_groups,
                                   int64_t total_rows, int64_t N, int64_t K, int64_t ldc, void* workspace,
                                   cudaStream_t st) {
  const int max_tiles = static_cast<int>(ceil_div64(total_rows, BM) + num_groups);
  MTile* table = static_cast<MTile*>(workspace);
  build_mtile_table_kernel<<<1, 256, 0, st>>>(offsets, num_groups, table, max_tiles);
  note_launch();
  if (cudaGetLastError() != cudaSuccess) return HIF4_ERR_CUDA;
  GemmParams p{};
  p.C = C; p.ldc = ldc; p.M = total_rows; p.N = N;
  p.num_kc = static_cast<int>(K / (kRawUnits * kUnitElems));
  p.n_tiles = static_cast<int>(ceil_div64(N, BN));
  p.m_tiles = max_tiles;
  p.table = table;
  return launch_tc(A, B, total_rows, static_cast<int64_t>(num_groups) * N, p, K, st);
}

}  // namespace hif4
