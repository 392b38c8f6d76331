// Decode-shaped HiF4 GEMM (M <= 32 tokens) on Eq. 3's own factorisation: C = A * B^T with the weight matrix B
// streamed once from HBM, the contraction of every unit pair done on FP8 (E4M3) tensor-core operands that
// hold only the "integer" part of the format, and the two level-1 scales applied to the FP32 partial sum of
// each 64-wide unit pair:
//
//     C[i][j] = sum over units k of  E6M2(A_ik) * E6M2(B_jk) * sum_{e<64} a_e * b_e,   a_e = +-S1P2 * 2^(E1_8 + E1_16)
//
// (Section III-B: the micro-exponents are absorbed into small integers, the 64 products are summed in an
// integer tree, one multiplication per unit pair applies the scales.)  An element a_e = +-(m/4) * 2^s with
// m <= 7, s <= 2 has at most three significant bits and lies in [2^-2, 7], so it is exactly an E4M3 number;
// the products are multiples of 1/16 below 49 and the sum of 32 of them is exact in the tensor core's
// accumulator (checked against the oracle for every code under every scale); only the accumulation over units
// rounds, in FP32, as in the other kernels.
//
// Why: the weight decode on the CUDA cores bounds this shape, not HBM.  Folding the level-1 scale into BF16
// operands costs a packed FMA per element pair plus the nibble extraction; an E4M3 operand byte is one byte
// permute away from the code nibble (`prmt` used as an eight-entry table on the 3-bit magnitude, four elements
// per instruction, the table pre-shifted by the group's micro-exponents), the sign is placed by a second
// permute in its sign-replicating mode, and mma.sync.m16n8k32 on E4M3 runs at twice the instruction rate and
// twice the K of the BF16 m16n8k16 form.
//
//   1. a token kernel turns the M rows of A (packed units) into E4M3 operand bytes laid out as the MMA's B
//      fragments, plus one FP32 scale per token and unit: 2176 bytes per 8 tokens and K = 256.
//   2. gemv8_kernel: one CTA per SM owns a contiguous run of 8-row blocks of B and the whole K range.  A producer
//      warp streams, per K = 256 chunk, the CTA's packed weight rows (one 2-D TMA box) and the tokens' chunk
//      through a ring of stages.  Consumer warp (pair, way) owns 16 weight rows and every `ways`-th chunk; lane
//      (g, q) decodes code words 2q and 2q + 1 of rows g and g + 8 of each unit (one word per MMA), so an MMA
//      never mixes units and its FP32 result can be scaled per row and token.  The K slices of a pair are
//      summed through shared memory in a fixed order: deterministic, no atomics.  Every mbarrier wait is bounded.
#include "hif4_common.cuh"
#include "hif4_gemm_internal.cuh"
#include "hif4_tc_common.cuh"

namespace hif4 {
namespace {

constexpr int kTok8OperandBytes = 2048;              // 8 tokens x 256 elements, one E4M3 byte each
constexpr int kTok8TileBytes = kTok8OperandBytes + 128;   // + 4 units x 8 tokens FP32 scales
constexpr int kBlockRows = 8;                        // granule of the row partition
constexpr int kBlockBytes = kBlockRows * kRawRowBytes;   // 1152 = 9 * 128
constexpr int kMaxBlocks = 16;                       // 8-row blocks per CTA (TMA box of up to 128 rows)
constexpr int kMaxStages = 16;
constexpr int kGemv8WarpsMany = 31, kGemv8WarpsFew = 24;   // consumer warps: 31 when a CTA owns five row pairs or more
constexpr int kRingBudget = 176 * 1024;              // bytes of shared memory given to the ring of stages
constexpr int kTableBytes = 1024 + 64 + 16 + 48;     // E6M2 values (256 floats), level-3 spread (16), level-2 spread (4), pad

// E4M3 bytes of m/4 for m = 0..7 (0, 0.25, 0.5, 0.75, 1, 1.25, 1.5, 1.75); a micro-exponent sum s adds s to the
// exponent field (bit 3 up) of the seven non-zero entries.
constexpr uint32_t kLutLo = 0x34302800u, kLutHi = 0x3E3C3A38u;
constexpr uint32_t kLutStepLo = 0x08080800u, kLutStepHi = 0x08080808u;

struct Gemv8Mul {            // runtime-valued on purpose (kernel parameters): the compiler keeps them as multiply-adds
  uint32_t m16, m256, m65536, m16777216;
};
inline Gemv8Mul make_gemv8_mul() { return Gemv8Mul{16u, 256u, 65536u, 16777216u}; }

struct Gemv8Params {
  uint8_t* tokens;          // workspace: [K/256][tiles][2176 bytes]
  float* C;
  int64_t ldc;
  int M;
  int64_t N;
  int num_kc;               // K / 256
  int num_blocks;           // ceil(N / 8)
  int max_blocks;           // 8-row blocks of the largest CTA; the others have one fewer
  int stages;
  Gemv8Mul mul;
  unsigned int* error_word;
};

// FP32 value of an E6M2 byte (Eq. 1: 2^(E - 48) * (1 + M/4)); 0xFF is NaN.
__device__ __forceinline__ uint32_t e6m2_float_bits(uint32_t byte) {
  return byte == 0xFFu ? 0x7FC00000u : (byte + 316u) << 21;      // ((E - 48 + 127) << 23) | (M << 21)
}

// One code word (8 elements: level-3 groups A = elements 0..3 and B = 4..7 of level-2 group j) -> two registers of
// four signed E4M3 bytes each, given the permute tables of the two groups (pre-shifted by their micro-exponents).
__device__ __forceinline__ void word_to_e4m3(uint32_t w, uint32_t loA, uint32_t hiA, uint32_t loB, uint32_t hiB,
                                             uint32_t w4, uint32_t& ra, uint32_t& rb) {
  const uint32_t w7 = w & 0x77777777u;                 // selector nibbles = magnitudes (bit 3 would mean "replicate sign")
  const uint32_t magA = prmt(loA, hiA, w7);            // elements 0..3: nibbles 0..3 of the word
  const uint32_t magB = prmt(loB, hiB, w7 >> 16);      // elements 4..7
  // sign bytes: element i's sign is bit 3 of nibble i = the top bit of byte i/2 of w (odd i) or of w << 4 (even i)
  const uint32_t sgA = prmt(w, w4, 0x9D8Cu);
  const uint32_t sgB = prmt(w, w4, 0xBFAEu);
  ra = magA | (sgA & 0x80808080u);
  rb = magB | (sgB & 0x80808080u);
}
// The same for the token kernels, micro-exponents taken straight from the metadata word.
__device__ __forceinline__ void token_word_to_e4m3(uint32_t meta, int W, uint32_t w, uint32_t& ra, uint32_t& rb) {
  const uint32_t e8 = (meta >> (8 + W)) & 1u;
  const uint32_t sA = e8 + ((meta >> (16 + 2 * W)) & 1u), sB = e8 + ((meta >> (17 + 2 * W)) & 1u);
  word_to_e4m3(w, kLutLo + sA * kLutStepLo, kLutHi + sA * kLutStepHi, kLutLo + sB * kLutStepLo, kLutHi + sB * kLutStepHi,
               w << 4, ra, rb);
}
// Where the eight operand bytes of code word W of unit U of token n go, and the unit's scale.
__device__ __forceinline__ uint8_t* token_tile(uint8_t* tokens, int n, int64_t U, int tiles) {
  return tokens + ((U >> 2) * tiles + (n >> 3)) * kTok8TileBytes;
}
__device__ __forceinline__ uint2* token_slot(uint8_t* tile, int n, int64_t U, int W) {
  return reinterpret_cast<uint2*>(tile + (2 * static_cast<int>(U & 3) + (W & 1)) * 256 + ((n & 7) * 4 + (W >> 1)) * 8);
}
__device__ __forceinline__ uint32_t* token_scale(uint8_t* tile, int n, int64_t U) {
  return reinterpret_cast<uint32_t*>(tile + kTok8OperandBytes + static_cast<int>(U & 3) * 32 + (n & 7) * 4);
}

__device__ __forceinline__ void mma_e4m3_16832(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k32.row.col.f32.e4m3.e4m3.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// First MMA of a unit: the accumulator starts from zero.
__device__ __forceinline__ void mma_e4m3_16832_zero(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                                    uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k32.row.col.f32.e4m3.e4m3.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
      : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(0.0f));
}
__device__ __forceinline__ void bulk_load_1d(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
__device__ __forceinline__ uint2 lds64(uint32_t addr) {
  uint2 v;
  asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
  return v;
}

int64_t gemv8_m_pad(int64_t M) { return M <= 8 ? 8 : M <= 16 ? 16 : 32; }

// ------------------------------------------------------------------------------------------ token kernels
// From packed units: thread (token n, unit U).
__global__ void __launch_bounds__(128)
gemv8_prepare_tokens_kernel(const uint32_t* __restrict__ A, int M, int m_pad, int64_t upr, uint8_t* __restrict__ tokens) {
  // the streaming kernel may be scheduled right away: it starts fetching weights and waits for this grid
  // (griddepcontrol.wait) only before it touches the tokens
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx >= static_cast<int64_t>(m_pad) * upr) return;
  const int n = static_cast<int>(idx / upr);
  const int64_t U = idx - static_cast<int64_t>(n) * upr;
  uint8_t* tile = token_tile(tokens, n, U, m_pad >> 3);
  if (n >= M) {
#pragma unroll
    for (int W = 0; W < 8; ++W) *token_slot(tile, n, U, W) = make_uint2(0u, 0u);
    *token_scale(tile, n, U) = 0u;
    return;
  }
  const uint32_t* unit = A + (static_cast<int64_t>(n) * upr + U) * kUnitWords;
  const uint32_t meta = __ldg(unit);
#pragma unroll
  for (int W = 0; W < 8; ++W) {
    uint32_t ra, rb;
    token_word_to_e4m3(meta, W, __ldg(unit + 1 + W), ra, rb);
    *token_slot(tile, n, U, W) = make_uint2(ra, rb);
  }
  *token_scale(tile, n, U) = e6m2_float_bits(meta & 0xFFu);
}

// A parity wait cannot tell a barrier that is one phase behind from one that is done, so a consumer first waits
// until the producer has announced the chunk it wants for that stage (the producer only announces it after every
// reader of the stage's previous chunk has arrived).  Bounded like mbar_wait.
__device__ __forceinline__ bool wait_announced8(const volatile int* slot, int kc, volatile uint32_t* abort_flag) {
  if (*slot >= kc) return true;
  const uint64_t t0 = global_ns();
  for (uint32_t it = 1;; ++it) {
    if (*slot >= kc) return true;
    __nanosleep(64);
    if ((it & 63u) == 0u) {
      if (*abort_flag) return false;
      if (global_ns() - t0 > kWaitBudgetNs) {
        *abort_flag = 1u;
        return false;
      }
    }
  }
}

// Per (weight row, unit): the row's level-1 scale as FP32 and the micro-exponent sums of this lane's four level-3
// groups (code words 2q and 2q + 1) as four bytes [A of word 2q, B of word 2q, A of word 2q+1, B of word 2q+1].
struct RowUnit {
  uint32_t s4;
  float ew;
};
__device__ __forceinline__ RowUnit prepare_row_unit(uint32_t meta, uint32_t tables, uint32_t sh16, uint32_t sh8) {
  RowUnit r;
  r.ew = __uint_as_float(lds32(tables + ((meta << 2) & 0x3FCu)));
  // 16-entry table: bit i of the lane's E1_16 nibble -> byte i; 4-entry table: E1_8 bit h -> bytes 2h, 2h + 1
  r.s4 = lds32(tables + 1024 + ((meta >> sh16) & 0x3Cu)) + lds32(tables + 1088 + ((meta >> sh8) & 0xCu));
  return r;
}

// Shared memory: [tables][partial sums][barriers, abort word, announced chunks: 384 B][ring of stages, 128-byte aligned]
template <int kTokTiles, int kWarps>
__global__ void __launch_bounds__((kWarps + 1) * 32, 1)
gemv8_kernel(const __grid_constant__ CUtensorMap tm_full, const __grid_constant__ CUtensorMap tm_short, const Gemv8Params p) {
  constexpr int kTokBytes = kTokTiles * kTok8TileBytes;
  constexpr int kRedBytes = kWarps * 32 * 4 * kTokTiles * 4;     // partial accumulators of every consumer warp
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 127u) & ~127u;
  uint8_t* gen_base = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t tables = smem_base;
  float* red = reinterpret_cast<float*>(gen_base + kTableBytes);
  const uint32_t bar_base = smem_base + kTableBytes + kRedBytes;
  const uint32_t full = bar_base, empty = bar_base + 8 * kMaxStages;
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(gen_base + kTableBytes + kRedBytes + 16 * kMaxStages);
  volatile int* announced = reinterpret_cast<volatile int*>(gen_base + kTableBytes + kRedBytes + 16 * kMaxStages + 16);
  const uint32_t ring = bar_base + 384;
  const uint32_t w_bytes_max = static_cast<uint32_t>(p.max_blocks) * kBlockBytes;
  const uint32_t stage_bytes = w_bytes_max + kTokBytes;

  // this CTA's run of 8-row blocks
  const int64_t blk_begin = static_cast<int64_t>(blockIdx.x) * p.num_blocks / gridDim.x;
  const int nblk = static_cast<int>(static_cast<int64_t>(blockIdx.x + 1) * p.num_blocks / gridDim.x - blk_begin);
  const int npairs = (nblk + 1) >> 1;
  const int ways = kWarps / npairs;              // >= 1: npairs <= kMaxBlocks / 2

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(full + 8 * s, 1);
      mbar_init(empty + 8 * s, npairs);                // the warps that read one chunk
      announced[s] = -1;
    }
    *abort_flag = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (threadIdx.x < 256) {
    uint32_t* t = reinterpret_cast<uint32_t*>(gen_base);
    t[threadIdx.x] = e6m2_float_bits(threadIdx.x);
    if (threadIdx.x < 16) {
      const uint32_t x = threadIdx.x;
      t[256 + x] = (x & 1u) | ((x & 2u) << 7) | ((x & 4u) << 14) | ((x & 8u) << 21);
    }
    if (threadIdx.x < 4) t[272 + threadIdx.x] = (threadIdx.x & 1u) * 0x0101u + (threadIdx.x >> 1) * 0x01010000u;
  }
  __syncthreads();

  if (warp == kWarps) {
    // ---------------------------------------------------------------- producer
    if (lane == 0) {
      const CUtensorMap* map = nblk == p.max_blocks ? &tm_full : &tm_short;
      const uint32_t tx = static_cast<uint32_t>(nblk) * kBlockBytes + kTokBytes;
      const int row0 = static_cast<int>(blk_begin * kBlockRows);
      // Launched as a programmatic dependent of the token kernel: the weights of the first ring of stages are
      // requested first, then the token grid is waited for, then the tokens follow.
      const int head = p.num_kc < p.stages ? p.num_kc : p.stages;
      for (int kc = 0; kc < head; ++kc) {
        announced[kc] = kc;
        mbar_expect_tx(full + 8 * kc, tx);
        tma_load_2d(ring + kc * stage_bytes, map, kc * kRawRowBytes, row0, full + 8 * kc);
      }
      asm volatile("griddepcontrol.wait;" ::: "memory");
      for (int kc = 0; kc < head; ++kc)
        bulk_load_1d(ring + kc * stage_bytes + w_bytes_max, p.tokens + static_cast<int64_t>(kc) * kTokBytes, kTokBytes,
                     full + 8 * kc);
      uint32_t s = 0, ph = 1;                          // stage and phase of chunk `head`
      for (int kc = head; kc < p.num_kc; ++kc) {
        if (!mbar_wait(empty + 8 * s, ph ^ 1u, abort_flag, 32)) break;
        announced[s] = kc;
        __threadfence_block();
        mbar_expect_tx(full + 8 * s, tx);
        const uint32_t dst = ring + s * stage_bytes;
        tma_load_2d(dst, map, kc * kRawRowBytes, row0, full + 8 * s);
        bulk_load_1d(dst + w_bytes_max, p.tokens + static_cast<int64_t>(kc) * kTokBytes, kTokBytes, full + 8 * s);
        if (++s == static_cast<uint32_t>(p.stages)) { s = 0; ph ^= 1u; }
      }
    }
  } else {
    // ---------------------------------------------------------------- consumers: 16 weight rows x one K slice per warp
    const int pair = warp % npairs, way = warp / npairs;
    const bool active = way < ways;
    const bool has_hi = 2 * pair + 1 < nblk;           // the pair's second block exists
    const int g = lane >> 2, q = lane & 3;
    float acc[kTokTiles][4];
#pragma unroll
    for (int t = 0; t < kTokTiles; ++t)
#pragma unroll
      for (int i = 0; i < 4; ++i) acc[t][i] = 0.0f;
    // words 2q, 2q + 1 of the unit; rows g (lo) and g + 8 (hi) of the pair
    const uint32_t off_lo = static_cast<uint32_t>(16 * pair + g) * kRawRowBytes;
    const uint32_t off_hi = off_lo + 8 * kRawRowBytes;
    const uint32_t off_word = 4u + 8u * static_cast<uint32_t>(q);
    const uint32_t off_tok = w_bytes_max + static_cast<uint32_t>(lane) * 8;
    const uint32_t off_scale = w_bytes_max + kTok8OperandBytes + static_cast<uint32_t>(q) * 8;
    const uint32_t sh16 = 14u + 4u * static_cast<uint32_t>(q);      // (meta >> sh16) & 0x3C = 4 * (E1_16 bits 4q .. 4q+3)
    const uint32_t sh8 = 6u + 2u * static_cast<uint32_t>(q);        // (meta >> sh8) & 0xC = 4 * (E1_8 bits 2q, 2q+1)
    if (active) {
      uint32_t s = static_cast<uint32_t>(way % p.stages), ph = static_cast<uint32_t>(way / p.stages) & 1u;
      const uint32_t s_step = static_cast<uint32_t>(ways % p.stages), ph_step = static_cast<uint32_t>(ways / p.stages);
      bool ok = true;
      for (int kc = way; kc < p.num_kc; kc += ways) {
        if (!(ok = __all_sync(0xFFFFFFFFu, wait_announced8(announced + s, kc, abort_flag) &&
                                               mbar_wait(full + 8 * s, ph, abort_flag))))
          break;
        const uint32_t st = ring + s * stage_bytes;
#pragma unroll 1
        for (int u = 0; u < kRawUnits; ++u) {
          const uint32_t ul = st + off_lo + u * kUnitBytes, uh = st + off_hi + u * kUnitBytes;
          const uint32_t ml = lds32(ul), mh = has_hi ? lds32(uh) : 0u;
          const RowUnit rl = prepare_row_unit(ml, tables, sh16, sh8), rh = prepare_row_unit(mh, tables, sh16, sh8);
          float part[kTokTiles][4];
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            const uint32_t wl = lds32(ul + off_word + 4 * h), wh = has_hi ? lds32(uh + off_word + 4 * h) : 0u;
            // micro-exponent sums of groups A and B of this word, rows lo and hi
            const uint32_t slA = (rl.s4 >> (16 * h)) & 0xFFu, slB = (rl.s4 >> (16 * h + 8)) & 0xFFu;
            const uint32_t shA = (rh.s4 >> (16 * h)) & 0xFFu, shB = (rh.s4 >> (16 * h + 8)) & 0xFFu;
            uint32_t a0, a1, a2, a3;
            word_to_e4m3(wl, slA * kLutStepLo + kLutLo, slA * kLutStepHi + kLutHi, slB * kLutStepLo + kLutLo,
                         slB * kLutStepHi + kLutHi, wl * p.mul.m16, a0, a2);
            word_to_e4m3(wh, shA * kLutStepLo + kLutLo, shA * kLutStepHi + kLutHi, shB * kLutStepLo + kLutLo,
                         shB * kLutStepHi + kLutHi, wh * p.mul.m16, a1, a3);
#pragma unroll
            for (int t = 0; t < kTokTiles; ++t) {
              const uint2 b = lds64(st + off_tok + t * kTok8TileBytes + (2 * u + h) * 256);
              if (h == 0) mma_e4m3_16832_zero(part[t], a0, a1, a2, a3, b.x, b.y);
              else mma_e4m3_16832(part[t], a0, a1, a2, a3, b.x, b.y);
            }
          }
          // Eq. 3: the unit pair's sum times the two level-1 scales
#pragma unroll
          for (int t = 0; t < kTokTiles; ++t) {
            const uint2 ex = lds64(st + off_scale + t * kTok8TileBytes + u * 32);
            const float e0 = __uint_as_float(ex.x), e1 = __uint_as_float(ex.y);
            acc[t][0] = fmaf(part[t][0], rl.ew * e0, acc[t][0]);
            acc[t][1] = fmaf(part[t][1], rl.ew * e1, acc[t][1]);
            acc[t][2] = fmaf(part[t][2], rh.ew * e0, acc[t][2]);
            acc[t][3] = fmaf(part[t][3], rh.ew * e1, acc[t][3]);
          }
        }
        fence_proxy_async_smem();                  // reads done before the async proxy refills the stage
        __syncwarp();
        if (lane == 0) mbar_arrive(empty + 8 * s);
        s += s_step; ph += ph_step;
        if (s >= static_cast<uint32_t>(p.stages)) { s -= p.stages; ++ph; }
        ph &= 1u;
      }
    }
    // Sum the K slices of every pair in a fixed order, then store.
    float* mine = red + (static_cast<size_t>(warp) * 32 + lane) * (4 * kTokTiles);
#pragma unroll
    for (int t = 0; t < kTokTiles; ++t)
#pragma unroll
      for (int i = 0; i < 4; ++i) mine[4 * t + i] = acc[t][i];
    asm volatile("bar.sync 1, %0;" ::"n"(kWarps * 32) : "memory");     // consumer warps only
    if (way == 0 && !*abort_flag) {
      // acc[t]: {row g: tokens 2q, 2q+1; row g+8: tokens 2q, 2q+1} (+ 8 t)
      const int64_t n0 = (blk_begin + 2 * pair) * kBlockRows + g;
#pragma unroll
      for (int t = 0; t < kTokTiles; ++t)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          float v = acc[t][i];
          for (int k = 1; k < ways; ++k)
            v += red[(static_cast<size_t>(k * npairs + pair) * 32 + lane) * (4 * kTokTiles) + 4 * t + i];
          const int tok = 8 * t + 2 * q + (i & 1);
          const int64_t n = n0 + (i >> 1) * 8;
          if (tok < p.M && n < p.N && ((i >> 1) == 0 || has_hi)) p.C[static_cast<int64_t>(tok) * p.ldc + n] = v;
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

template <int kTokTiles, int kWarps>
hif4_status launch_gemv8_t(const void* B, int64_t upr, Gemv8Params p, cudaStream_t st) {
  constexpr int kTokBytes = kTokTiles * kTok8TileBytes;
  constexpr int kFixed = 128 + kTableBytes + kWarps * 32 * 4 * kTokTiles * 4 + 384;
  // One CTA per SM (several rounds of them when a CTA would get more than kMaxBlocks blocks).
  const int64_t sms = sm_count();
  const int64_t rounds = ceil_div64(p.num_blocks, sms * kMaxBlocks);
  const int64_t grid = p.num_blocks < sms * rounds ? p.num_blocks : sms * rounds;
  if (grid > 0x7FFFFFFFll) return HIF4_ERR_SHAPE;
  p.max_blocks = static_cast<int>(ceil_div64(p.num_blocks, grid));
  const int stage_bytes = p.max_blocks * kBlockBytes + kTokBytes;
  p.stages = kRingBudget / stage_bytes;
  if (p.stages > kMaxStages) p.stages = kMaxStages;
  if (p.stages > p.num_kc) p.stages = p.num_kc;
  const int smem = kFixed + p.stages * stage_bytes;
  static uint64_t smem_opt_in = 0;
  if (!ensure_dynamic_smem(gemv8_kernel<kTokTiles, kWarps>, kFixed + kRingBudget, smem_opt_in)) return HIF4_ERR_CUDA;
  CUtensorMap tm_full, tm_short;
  if (!make_unit_map(&tm_full, B, p.N, upr, p.max_blocks * kBlockRows)) return HIF4_ERR_CUDA;
  if (!make_unit_map(&tm_short, B, p.N, upr, (p.max_blocks > 1 ? p.max_blocks - 1 : 1) * kBlockRows)) return HIF4_ERR_CUDA;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(grid));
  cfg.blockDim = dim3((kWarps + 1) * 32);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;      // may start while the token kernel still runs
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, gemv8_kernel<kTokTiles, kWarps>, tm_full, tm_short, p) != cudaSuccess) {
    (void)cudaGetLastError();
    return HIF4_ERR_CUDA;
  }
  note_launch();
  return HIF4_OK;
}


// Fills the launch parameters both entry points share; returns false when N is out of range.
bool gemv8_params(Gemv8Params& p, float* C, int64_t M, int64_t N, int64_t K, int64_t ldc, void* workspace) {
  p.tokens = static_cast<uint8_t*>(workspace);
  p.C = C; p.ldc = ldc; p.M = static_cast<int>(M); p.N = N;
  p.num_kc = static_cast<int>(K / 256);
  if (ceil_div64(N, kBlockRows) > 0x7FFFFFFFll) return false;
  p.num_blocks = static_cast<int>(ceil_div64(N, kBlockRows));
  p.mul = make_gemv8_mul();
  p.error_word = device_error_word();
  return true;
}
// The streaming kernel on tokens that the preceding launch in `st` has prepared.
hif4_status launch_gemv8_stream(const void* B, const Gemv8Params& p, int m_pad, int64_t upr, cudaStream_t st) {
  const int64_t sms = sm_count();
  const int64_t rounds = ceil_div64(p.num_blocks, sms * kMaxBlocks);
  const int64_t grid = p.num_blocks < sms * rounds ? p.num_blocks : sms * rounds;
  const bool many = ceil_div64(p.num_blocks, grid) >= 9;
  if (m_pad == 32) return launch_gemv8_t<4, kGemv8WarpsFew>(B, upr, p, st);
  if (m_pad == 8) return many ? launch_gemv8_t<1, kGemv8WarpsMany>(B, upr, p, st) : launch_gemv8_t<1, kGemv8WarpsFew>(B, upr, p, st);
  return many ? launch_gemv8_t<2, kGemv8WarpsMany>(B, upr, p, st) : launch_gemv8_t<2, kGemv8WarpsFew>(B, upr, p, st);
}
}  // namespace

size_t gemv8_workspace_bytes(int64_t M, int64_t K) {
  if (M < 1 || M > kGemvMaxM || K <= 0 || K % 256 != 0) return 0;
  return static_cast<size_t>((K / 256) * (gemv8_m_pad(M) / 8) * kTok8TileBytes);
}

hif4_status launch_gemv8(const void* A, const void* B, float* C, int64_t M, int64_t N, int64_t K, int64_t ldc,
                         void* workspace, cudaStream_t st) {
  Gemv8Params p{};
  if (!gemv8_params(p, C, M, N, K, ldc, workspace)) return HIF4_ERR_SHAPE;
  if (!p.error_word) return HIF4_ERR_CUDA;
  const int m_pad = static_cast<int>(gemv8_m_pad(M));
  const int64_t upr = K / kUnitElems;
  const int64_t prep = static_cast<int64_t>(m_pad) * upr;
  gemv8_prepare_tokens_kernel<<<static_cast<unsigned>(ceil_div64(prep, 128)), 128, 0, st>>>(
      static_cast<const uint32_t*>(A), p.M, m_pad, upr, p.tokens);
  note_launch();
  if (cudaGetLastError() != cudaSuccess) return HIF4_ERR_CUDA;
  return launch_gemv8_stream(B, p, m_pad, upr, st);
}

}  // namespace hif4
