// Decode-shaped HiF4 GEMM (M <= 16 tokens): C = A * B^T with the weight matrix B streamed once from
// HBM.  The problem is bound by the 0.5625 bytes per weight element that have to cross the memory
// bus, so the kernel is organised around keeping many TMA copies of packed weight rows in flight,
// and the few tokens are prepared once.
//
//   1. gemv_prepare_tokens_kernel decodes the M rows of A (Eq. 2, exact BF16) into a small workspace
//      laid out per K = 256 chunk as the B fragments of mma.sync.m16n8k16 want them.
//   2. gemv_kernel: one CTA owns 16 * kRowGroups weight rows and the whole K range.  A producer warp
//      streams, per K = 256 chunk, the CTA's packed weight rows (one 2-D TMA box, 144 bytes per row) and
//      the tokens' chunk (one bulk copy, L2-resident) through a 4- or 8-stage ring.  Consumer warp (rg, ks)
//      owns 16 weight rows and unit ks of every kChunkWays-th chunk (8 or 16 K slices per row group, so
//      that even a narrow problem has enough warps in flight to hide the decode latency): lane (g, q) reads the metadata word and code words
//      2q, 2q+1 of rows g and g+8, decodes them in registers straight into the A fragments (weights are
//      the 16-row MMA operand), reads the matching token fragments from shared memory and issues four
//      BF16 MMAs with FP32 accumulators.  Inside a unit the K order is permuted the same way on both
//      operands.  The K slices are summed through shared memory in a fixed order.
// Results are deterministic (no atomics).  Every mbarrier wait is bounded.
#include "hif4_common.cuh"
#include "hif4_gemm_internal.cuh"
#include "hif4_tc_common.cuh"

namespace hif4 {
namespace {

constexpr int kTokChunkBytes = 512;                  // one token, K = 256, BF16

struct GemvParams {
  const uint32_t* A;        // [M, K/64] units (tokens)
  uint8_t* tokens;          // workspace: [K/256][m_pad][512 B]
  float* C;
  int64_t ldc;
  int M;
  int m_pad;                // 8 or 16
  int64_t N;
  int num_kc;               // K / 256
  unsigned int* error_word;
};

// One code word (8 elements of level-2 group j) -> four bf16x2 registers holding elements (0,4), (1,5),
// (2,6), (3,7) of the group.  base2 = BF16 bits of E6M2 / 4 in both halves.
__device__ __forceinline__ void decode_word_regs(uint32_t meta, uint32_t base2, int j, uint32_t wj, uint32_t (&r)[4]) {
  const uint32_t e8 = (meta >> (8 + j)) & 1u;
  const uint32_t e16 = (((meta >> (16 + 2 * j)) & 3u) * 0x00400080u) & 0x00800080u;   // E1_16[2j] bit 7, [2j+1] bit 23
  const uint32_t Sa = base2 + e16 + e8 * 0x00800080u;               // (S_lo, S_hi), S = E6M2 * 2^(e8 + e16 - 2)
  const uint32_t Sb = Sa - 0x02000200u;                             // S / 16
  const uint32_t Oa = Sa + 0x83808380u;                             // -128 S
  const uint32_t Ob = Sa + 0x81808180u;                             // -8 S
  const uint32_t wh = wj >> 8;
  r[0] = fma_bf16x2((wj & 0x00070007u) | 0x43004300u, Sa, Oa) ^ ((wj << 12) & 0x80008000u);
  r[1] = fma_bf16x2((wj & 0x00700070u) | 0x43004300u, Sb, Ob) ^ ((wj << 8) & 0x80008000u);
  r[2] = fma_bf16x2((wh & 0x00070007u) | 0x43004300u, Sa, Oa) ^ ((wj << 4) & 0x80008000u);
  r[3] = fma_bf16x2((wh & 0x00700070u) | 0x43004300u, Sb, Ob) ^ (wj & 0x80008000u);
}
// Words j and j+1 of one unit -> eight registers; a NaN unit (Eq. 2) gives NaN everywhere.
__device__ __forceinline__ void decode_two_words(uint32_t meta, int j, uint32_t w0, uint32_t w1, uint32_t (&r)[8]) {
  const uint32_t byte = meta & 0xFFu;
  if (byte == 0xFFu) {
#pragma unroll
    for (int i = 0; i < 8; ++i) r[i] = 0x7FC07FC0u;
    return;
  }
  const uint32_t base2 = byte * 0x00200020u + 0x26802680u;         // ((byte + 308) << 5) in both halves
  uint32_t lo[4], hi[4];
  decode_word_regs(meta, base2, j, w0, lo);
  decode_word_regs(meta, base2, j + 1, w1, hi);
#pragma unroll
  for (int i = 0; i < 4; ++i) { r[i] = lo[i]; r[4 + i] = hi[i]; }
}

__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void bulk_load_1d(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}

// Token workspace: chunk kc, token n: 512 bytes = 4 units x 8 words x 16 bytes, the 16-byte group of word W
// stored at position W ^ (n & 1) so that the fragment loads of a quarter-warp hit distinct banks.
__global__ void __launch_bounds__(128)
gemv_prepare_tokens_kernel(const uint32_t* __restrict__ A, int M, int m_pad, int64_t upr, uint8_t* __restrict__ tokens) {
  // the streaming kernel may be scheduled right away: it starts fetching weights and waits for this
  // grid (griddepcontrol.wait) only before it touches the tokens
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;     // (token n, unit U)
  if (idx >= static_cast<int64_t>(m_pad) * upr) return;
  const int n = static_cast<int>(idx / upr);
  const int64_t U = idx - static_cast<int64_t>(n) * upr;
  uint4* dst = reinterpret_cast<uint4*>(tokens + ((U >> 2) * m_pad + n) * kTokChunkBytes + (U & 3) * 128);
  if (n >= M) {
#pragma unroll
    for (int W = 0; W < 8; ++W) dst[W] = make_uint4(0u, 0u, 0u, 0u);
    return;
  }
  const uint32_t* unit = A + (static_cast<int64_t>(n) * upr + U) * kUnitWords;
  const uint32_t meta = __ldg(unit);
#pragma unroll
  for (int W = 0; W < 8; W += 2) {
    uint32_t r[8];
    decode_two_words(meta, W, __ldg(unit + 1 + W), __ldg(unit + 2 + W), r);
    dst[W ^ (n & 1)] = make_uint4(r[0], r[1], r[2], r[3]);
    dst[(W + 1) ^ (n & 1)] = make_uint4(r[4], r[5], r[6], r[7]);
  }
}

template <int kRowGroups, int kTokTiles, int kChunkWays, int kStages>
__global__ void __launch_bounds__((4 * kChunkWays * kRowGroups + 1) * 32)
gemv_kernel(const __grid_constant__ CUtensorMap tmB, const GemvParams p) {
  constexpr int kWarps = 4 * kChunkWays * kRowGroups;              // consumer warps
  constexpr int kRows = 16 * kRowGroups;
  constexpr int kWeightBytes = kRows * kRawRowBytes;
  constexpr int kTokBytes = 8 * kTokTiles * kTokChunkBytes;
  constexpr int kStageBytes = kWeightBytes + kTokBytes;            // multiples of 128
  constexpr int kRedBytes = kWarps * 32 * 4 * kTokTiles * 4;       // partial accumulators of every consumer warp
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 127u) & ~127u;
  const uint32_t bar_base = smem_base + kStages * kStageBytes + kRedBytes;
  const uint32_t full = bar_base, empty = bar_base + 8 * kStages;
  uint8_t* gen_base = smem_raw + (smem_base - smem_u32(smem_raw));
  float* red = reinterpret_cast<float*>(gen_base + kStages * kStageBytes);
  volatile uint32_t* abort_flag =
      reinterpret_cast<volatile uint32_t*>(gen_base + kStages * kStageBytes + kRedBytes + 16 * kStages);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t row0 = static_cast<int64_t>(blockIdx.x) * kRows;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(full + 8 * s, 1);
      mbar_init(empty + 8 * s, 4 * kRowGroups);          // the warps that read one chunk
    }
    *abort_flag = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  if (warp == kWarps) {
    // ---------------------------------------------------------------- producer
    if (lane == 0) {
      // Launched as a programmatic dependent of the token preparation: the weights of the first ring
      // of stages are requested first, then the preparation grid is waited for, then the tokens follow.
      const int head = p.num_kc < kStages ? p.num_kc : kStages;
      for (int kc = 0; kc < head; ++kc) {
        mbar_expect_tx(full + 8 * kc, kStageBytes);
        tma_load_2d(smem_base + kc * kStageBytes, &tmB, kc * kRawRowBytes, static_cast<int>(row0), full + 8 * kc);
      }
      asm volatile("griddepcontrol.wait;" ::: "memory");
      for (int kc = 0; kc < head; ++kc)
        bulk_load_1d(smem_base + kc * kStageBytes + kWeightBytes,
                     p.tokens + static_cast<int64_t>(kc) * p.m_pad * kTokChunkBytes, kTokBytes, full + 8 * kc);
      for (int kc = head; kc < p.num_kc; ++kc) {
        const uint32_t s = kc % kStages, ph = (kc / kStages) & 1u;
        if (!mbar_wait(empty + 8 * s, ph ^ 1u, abort_flag, 32)) break;
        mbar_expect_tx(full + 8 * s, kStageBytes);
        const uint32_t dst = smem_base + s * kStageBytes;
        tma_load_2d(dst, &tmB, kc * kRawRowBytes, static_cast<int>(row0), full + 8 * s);
        bulk_load_1d(dst + kWeightBytes, p.tokens + static_cast<int64_t>(kc) * p.m_pad * kTokChunkBytes, kTokBytes,
                     full + 8 * s);
      }
    }
  } else {
    // ---------------------------------------------------------------- consumers: 16 weight rows x one K slice per warp
    // row group, K slice: unit (slice & 3) of the chunks kc = slice / 4 (mod kChunkWays)
    const int rg = warp % kRowGroups, slice = warp / kRowGroups, ks = slice & 3, way = slice >> 2;
    const int g = lane >> 2, q = lane & 3;
    // two accumulator sets per token tile, so that consecutive MMAs do not wait on one another
    float acc[kTokTiles][4], acc2[kTokTiles][4];
#pragma unroll
    for (int t = 0; t < kTokTiles; ++t)
#pragma unroll
      for (int i = 0; i < 4; ++i) acc[t][i] = acc2[t][i] = 0.0f;
    const uint32_t w_off0 = static_cast<uint32_t>(16 * rg + g) * kRawRowBytes + ks * kUnitBytes;   // MMA row g
    const uint32_t w_off1 = w_off0 + 8 * kRawRowBytes;                                               // MMA row g + 8
    // token g (and g + 8): words 2q and 2q+1 of unit ks, 16-byte groups swizzled by the token's parity
    const uint32_t t_base = kWeightBytes + static_cast<uint32_t>(g) * kTokChunkBytes + ks * 128;
    const uint32_t t_lo = t_base + ((static_cast<uint32_t>(2 * q) ^ (g & 1u)) << 4);
    const uint32_t t_hi = t_base + ((static_cast<uint32_t>(2 * q + 1) ^ (g & 1u)) << 4);
    bool ok = true;
    for (int kc = way; kc < p.num_kc && ok; kc += kChunkWays) {
      const uint32_t s = kc % kStages, ph = (kc / kStages) & 1u;
      if (!(ok = __all_sync(0xFFFFFFFFu, mbar_wait(full + 8 * s, ph, abort_flag)))) break;
      const uint32_t st = smem_base + s * kStageBytes;
      uint32_t a[8], b[8];
      const uint32_t r0 = st + w_off0, r1 = st + w_off1;
      const uint32_t m0 = lds32(r0), w00 = lds32(r0 + 4 + 8 * q), w01 = lds32(r0 + 8 + 8 * q);
      const uint32_t m1 = lds32(r1), w10 = lds32(r1 + 4 + 8 * q), w11 = lds32(r1 + 8 + 8 * q);
      uint4 x[kTokTiles], y[kTokTiles];
#pragma unroll
      for (int t = 0; t < kTokTiles; ++t) {
        x[t] = lds128(st + t_lo + t * 8 * kTokChunkBytes);
        y[t] = lds128(st + t_hi + t * 8 * kTokChunkBytes);
      }
      fence_proxy_async_smem();                  // reads done before the async proxy refills the stage
      __syncwarp();
      if (lane == 0) mbar_arrive(empty + 8 * s);
      decode_two_words(m0, 2 * q, w00, w01, a);
      decode_two_words(m1, 2 * q, w10, w11, b);
#pragma unroll
      for (int t = 0; t < kTokTiles; ++t) {
        mma_bf16_16816(acc[t], a[0], b[0], a[1], b[1], x[t].x, x[t].y);
        mma_bf16_16816(acc2[t], a[2], b[2], a[3], b[3], x[t].z, x[t].w);
        mma_bf16_16816(acc[t], a[4], b[4], a[5], b[5], y[t].x, y[t].y);
        mma_bf16_16816(acc2[t], a[6], b[6], a[7], b[7], y[t].z, y[t].w);
      }
    }
#pragma unroll
    for (int t = 0; t < kTokTiles; ++t)
#pragma unroll
      for (int i = 0; i < 4; ++i) acc[t][i] += acc2[t][i];
    // Sum the K slices of every row group in a fixed order, then store.
    float* mine = red + (static_cast<size_t>(warp) * 32 + lane) * (4 * kTokTiles);
#pragma unroll
    for (int t = 0; t < kTokTiles; ++t)
#pragma unroll
      for (int i = 0; i < 4; ++i) mine[4 * t + i] = acc[t][i];
    asm volatile("bar.sync 1, %0;" ::"n"(kWarps * 32) : "memory");     // consumer warps only
    if (slice == 0 && !*abort_flag) {
      // acc[t]: {row g: tokens 2q, 2q+1; row g+8: tokens 2q, 2q+1} (+ 8 t)
      const int64_t n0 = row0 + 16 * rg + g;
#pragma unroll
      for (int t = 0; t < kTokTiles; ++t)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          float v = acc[t][i];
#pragma unroll
          for (int k = 1; k < 4 * kChunkWays; ++k)
            v += red[(static_cast<size_t>(k * kRowGroups + rg) * 32 + lane) * (4 * kTokTiles) + 4 * t + i];
          const int tok = 8 * t + 2 * q + (i & 1);
          const int64_t n = n0 + (i >> 1) * 8;
          if (tok < p.M && n < p.N) p.C[static_cast<int64_t>(tok) * p.ldc + n] = v;
        }
    }
  }
  __syncwarp();
  if (*abort_flag) {
    const uint64_t t0 = global_ns();
    while (global_ns() - t0 < 2000000ull) {}     // let copies that are still in flight land
    if (threadIdx.x == 0) atomicExch(p.error_word, 1u);
  }
}

template <int kRowGroups, int kTokTiles, int kChunkWays, int kStages>
hif4_status launch_gemv_t(const void* B, int64_t upr, const GemvParams& p, cudaStream_t st) {
  constexpr int kRows = 16 * kRowGroups;
  constexpr int smem = 128 + kStages * (kRows * kRawRowBytes + 8 * kTokTiles * kTokChunkBytes) +
                       4 * kChunkWays * kRowGroups * 32 * 4 * kTokTiles * 4 + 16 * kStages + 16;
  static uint64_t smem_opt_in = 0;
  if (!ensure_dynamic_smem(gemv_kernel<kRowGroups, kTokTiles, kChunkWays, kStages>, smem, smem_opt_in)) return HIF4_ERR_CUDA;
  CUtensorMap tmB;
  if (!make_unit_map(&tmB, B, p.N, upr, kRows)) return HIF4_ERR_CUDA;
  const int64_t blocks = ceil_div64(p.N, kRows);
  if (blocks > 0x7FFFFFFFll) return HIF4_ERR_SHAPE;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(blocks));
  cfg.blockDim = dim3((4 * kChunkWays * kRowGroups + 1) * 32);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;      // may start while the token preparation still runs
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, gemv_kernel<kRowGroups, kTokTiles, kChunkWays, kStages>, tmB, p) != cudaSuccess) {
    (void)cudaGetLastError();
    return HIF4_ERR_CUDA;
  }
  note_launch();
  return HIF4_OK;
}

}  // namespace

bool gemv_supported(const void* A, const void* B, int64_t M, int64_t N, int64_t K) {
  return M >= 1 && M <= kGemvMaxM && gemm_tc_supported(B, B, N, N, N, K) && (reinterpret_cast<uintptr_t>(A) & 3u) == 0;
}

size_t gemv_workspace_bytes(int64_t M, int64_t K) {
  if (M < 1 || M > kGemvMaxM || K <= 0 || K % 256 != 0) return 0;
  const int64_t m_pad = M <= 8 ? 8 : 16;
  return static_cast<size_t>(m_pad * K * 2);
}

hif4_status launch_gemv(const void* A, const void* B, float* C, int64_t M, int64_t N, int64_t K, int64_t ldc,
                        void* workspace, cudaStream_t st) {
  GemvParams p{};
  p.A = static_cast<const uint32_t*>(A);
  p.tokens = static_cast<uint8_t*>(workspace);
  p.C = C; p.ldc = ldc; p.M = static_cast<int>(M); p.m_pad = M <= 8 ? 8 : 16; p.N = N;
  p.num_kc = static_cast<int>(K / 256);
  p.error_word = device_error_word();
  if (!p.error_word) return HIF4_ERR_CUDA;
  const int64_t upr = K / kUnitElems;
  const int64_t prep = static_cast<int64_t>(p.m_pad) * upr;
  gemv_prepare_tokens_kernel<<<static_cast<unsigned>(ceil_div64(prep, 128)), 128, 0, st>>>(p.A, p.M, p.m_pad, upr, p.tokens);
  note_launch();
  if (cudaGetLastError() != cudaSuccess) return HIF4_ERR_CUDA;
  // 16 weight rows per CTA with 16 K slices for narrow problems (few CTAs, so each needs many warps),
  // 32 rows with 4 K slices per row group once that still gives every SM two CTAs
  const bool wide = N >= 64ll * sm_count();
  if (p.m_pad == 8) return wide ? launch_gemv_t<2, 1, 1, 4>(B, upr, p, st) : launch_gemv_t<1, 1, 4, 8>(B, upr, p, st);
  return wide ? launch_gemv_t<2, 2, 1, 4>(B, upr, p, st) : launch_gemv_t<1, 2, 4, 8>(B, upr, p, st);
}

}  // namespace hif4
