// Decode-shaped HiF4 GEMM (M <= 32 tokens): C = A * B^T with the weight matrix B streamed once from
// HBM.  The few tokens are decoded once; the work per weight element is the register decode, so the
// kernel is organised around decoding with as few instructions per element as possible and around
// giving every SM the same number of weight rows.
//
//   1. gemv_prepare_tokens_kernel decodes the M rows of A (Eq. 2, exact BF16) into a small workspace
//      laid out per K = 256 chunk as the B fragments of mma.sync.m16n8k16 want them.
//   2. gemv_kernel: one CTA per SM owns a contiguous run of 8-row blocks of B (the runs differ by at
//      most one block) and the whole K range.  A producer warp streams, per K = 256 chunk, the CTA's
//      packed weight rows (one 2-D TMA box, 144 bytes per row) and the tokens' chunk (one bulk copy,
//      L2-resident) through a ring of stages.  Consumer warp (pair, way) owns two 8-row blocks (the 16
//      rows of the MMA's weight operand) and every `ways`-th chunk.  Lane (g, q) owns unit q of the
//      chunk for rows g and g + 8: it reads the two 36-byte units, prepares the unit's scales once, and
//      decodes word after word straight into the A fragments (k slots 2q, 2q+1, 2q+8, 2q+9 of every MMA
//      come from unit q on both operands, so the K order is permuted the same way on both sides).
//      The K slices of a pair are summed through shared memory in a fixed order.
//   3. Up to 16 tokens with few elements in all (kSrc 1, 2): no token kernel at all.  Every CTA decodes the few tokens
//      itself (from packed units, or from BF16 activations that it first converts with Algorithm 1) into a resident
//      block of shared memory before its main loop, while its producer warp is already streaming weights; one launch
//      per product instead of two, which is most of the time of the small shapes.  The resident block keeps 1, 2, 4 or
//      8 token rows per n-tile (the MMA lanes of the rows it leaves out read zeros); rows kept x K is limited to what
//      a CTA builds in less time than the second launch costs (one token from packed units: K up to 49152).
// Results are deterministic (no atomics).  Every mbarrier wait is bounded.
#include "hif4_common.cuh"
#include "hif4_gemm_internal.cuh"
#include "hif4_quantize_device.cuh"
#include "hif4_tc_common.cuh"

namespace hif4 {
namespace {

constexpr int kTokChunkBytes = 512;                  // one token, K = 256, BF16
constexpr int kTileChunkBytes = 8 * kTokChunkBytes;  // eight tokens (one MMA n-tile), K = 256
constexpr int kBlockRows = 8;                        // granule of the row partition
constexpr int kBlockBytes = kBlockRows * kRawRowBytes;   // 1152 = 9 * 128
constexpr int kMaxBlocks = 16;                       // 8-row blocks per CTA (TMA box of up to 128 rows)
constexpr int kMaxStages = 16;
// consumer warps per CTA: 31 when a CTA owns many rows (five row pairs or more share them evenly and hide
// more latency), 24 otherwise (fewer warps wait on the same few chunks)
constexpr int kGemvWarpsMany = 31, kGemvWarpsFew = 24;
constexpr int kRingBudget = 176 * 1024;              // bytes of shared memory given to the ring of stages

constexpr int kSrcWorkspace = 0, kSrcUnits = 1, kSrcBf16 = 2;   // where the streaming kernel gets its tokens from
constexpr int kResidentMaxBytes = 128 * 1024;         // resident tokens: K / 256 chunks of (n-tiles x 8 words x rows x 64) bytes

struct GemvParams {
  const uint32_t* A;        // [M, K/64] units (tokens)
  const uint16_t* X;        // kSrcBf16: [M, K] BF16 activations, row stride ld_x elements
  int64_t ld_x;
  int rha;                  // kSrcBf16: rounding mode of the conversion
  uint8_t* tokens;          // workspace: [K/256][tiles][8 words][8 tokens][4 units][16 B]
  float* C;
  int64_t ldc;
  int M;
  int64_t N;
  int num_kc;               // K / 256
  int num_blocks;           // ceil(N / 8)
  int max_blocks;           // 8-row blocks of the largest CTA; the others have one fewer
  int stages;
  int res_rows;             // resident tokens: token rows kept per n-tile (1, 2, 4 or 8)
  DecodeMul mul;
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

// Token workspace: chunk kc, n-tile t, word W: 512 bytes = 8 tokens x 4 units x 16 bytes, so that the 32
// lanes (token g, unit q) of a warp read one contiguous, conflict-free line per word.
__global__ void __launch_bounds__(128)
gemv_prepare_tokens_kernel(const uint32_t* __restrict__ A, int M, int m_pad, int64_t upr, uint8_t* __restrict__ tokens) {
  // the streaming kernel may be scheduled right away: it starts fetching weights and waits for this
  // grid (griddepcontrol.wait) only before it touches the tokens
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;     // (token n, unit U)
  if (idx >= static_cast<int64_t>(m_pad) * upr) return;
  const int n = static_cast<int>(idx / upr);
  const int64_t U = idx - static_cast<int64_t>(n) * upr;
  const int tiles = m_pad >> 3;
  uint8_t* dst = tokens + (((U >> 2) * tiles + (n >> 3)) * 8) * kTokChunkBytes + ((n & 7) * 4 + (U & 3)) * 16;
  if (n >= M) {
#pragma unroll
    for (int W = 0; W < 8; ++W) *reinterpret_cast<uint4*>(dst + W * kTokChunkBytes) = make_uint4(0u, 0u, 0u, 0u);
    return;
  }
  const uint32_t* unit = A + (static_cast<int64_t>(n) * upr + U) * kUnitWords;
  const uint32_t meta = __ldg(unit);
#pragma unroll
  for (int W = 0; W < 8; W += 2) {
    uint32_t r[8];
    decode_two_words(meta, W, __ldg(unit + 1 + W), __ldg(unit + 2 + W), r);
    *reinterpret_cast<uint4*>(dst + W * kTokChunkBytes) = make_uint4(r[0], r[1], r[2], r[3]);
    *reinterpret_cast<uint4*>(dst + (W + 1) * kTokChunkBytes) = make_uint4(r[4], r[5], r[6], r[7]);
  }
}

// The same preparation straight from BF16 activations: Algorithm 1 (the streaming quantizer's own code, two
// lanes per unit) followed by Eq. 2 of the unit just encoded, without the packed units ever going to memory.
// Used by the one-call linear layer for M <= 32 BF16 rows; the tokens written are bit-identical to quantizing first.
template <bool kRHA>
__global__ void __launch_bounds__(128)
gemv_quantize_tokens_kernel(const uint16_t* __restrict__ X, int64_t ld_x, int M, int m_pad, int64_t upr,
                            uint8_t* __restrict__ tokens) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;     // ((token n, unit U), lane l)
  const int l = static_cast<int>(idx & 1);
  const int64_t pair = idx >> 1;
  const bool in_range = pair < static_cast<int64_t>(m_pad) * upr;      // same for both lanes of a pair
  const int n = in_range ? static_cast<int>(pair / upr) : 0;
  const int64_t U = in_range ? pair - static_cast<int64_t>(n) * upr : 0;
  uint4 v[4];
#pragma unroll
  for (int c = 0; c < 4; ++c) v[c] = make_uint4(0u, 0u, 0u, 0u);
  if (in_range && n < M) {
    const uint4* src = reinterpret_cast<const uint4*>(X + static_cast<int64_t>(n) * ld_x + U * kUnitElems) + l;
#pragma unroll
    for (int c = 0; c < 4; ++c) v[c] = __ldg(src + 2 * c);
  }
  uint32_t codes[4], meta;
  encode_unit_bf16_pair<kRHA>(v, l, codes, meta);        // every lane of the warp takes part (pair-wise exchange)
  if (!in_range) return;
  const int tiles = m_pad >> 3;
  uint8_t* dst = tokens + (((U >> 2) * tiles + (n >> 3)) * 8) * kTokChunkBytes + ((n & 7) * 4 + (U & 3)) * 16;
  const uint32_t byte = meta & 0xFFu;
  const uint32_t base2 = byte * 0x00200020u + 0x26802680u;
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    const int W = l + 2 * c;                             // this lane's code words
    uint32_t r[4] = {0u, 0u, 0u, 0u};
    if (n < M) {
      if (byte == 0xFFu) r[0] = r[1] = r[2] = r[3] = 0x7FC07FC0u;
      else decode_word_regs(meta, base2, W, codes[c], r);
    }
    *reinterpret_cast<uint4*>(dst + W * kTokChunkBytes) = make_uint4(r[0], r[1], r[2], r[3]);
  }
}

// The same for FP32 and FP16 activations (Algorithm 1 in FP32 arithmetic, four lanes per unit; the even lanes hold
// the code words afterwards and decode them).
template <bool kRHA, typename Src>
__global__ void __launch_bounds__(128)
gemv_quantize_tokens32_kernel(const Src* __restrict__ X, int64_t ld_x, int M, int m_pad, int64_t upr,
                              uint8_t* __restrict__ tokens) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;     // ((token n, unit U), lane l)
  const int l = static_cast<int>(idx & 3);
  const int64_t quad = idx >> 2;
  const bool in_range = quad < static_cast<int64_t>(m_pad) * upr;      // same for the four lanes of a unit
  const int n = in_range ? static_cast<int>(quad / upr) : 0;
  const int64_t U = in_range ? quad - static_cast<int64_t>(n) * upr : 0;
  uint4 v[4];
#pragma unroll
  for (int c = 0; c < 4; ++c) v[c] = make_uint4(0u, 0u, 0u, 0u);
  if (in_range && n < M) {
    const Src* src = X + static_cast<int64_t>(n) * ld_x + U * kUnitElems + 4 * l;
#pragma unroll
    for (int c = 0; c < 4; ++c) v[c] = load_group_fp32(src + 16 * c);
  }
  uint32_t codes[4], meta;
  encode_unit_fp32_quad<kRHA>(v, l, codes, meta);        // every lane of the warp takes part
  if (!in_range || (l & 1)) return;
  const int tiles = m_pad >> 3;
  uint8_t* dst = tokens + (((U >> 2) * tiles + (n >> 3)) * 8) * kTokChunkBytes + ((n & 7) * 4 + (U & 3)) * 16;
  const uint32_t byte = meta & 0xFFu;
  const uint32_t base2 = byte * 0x00200020u + 0x26802680u;
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    const int W = (l >> 1) + 2 * c;                      // this lane's code words
    uint32_t r[4] = {0u, 0u, 0u, 0u};
    if (n < M) {
      if (byte == 0xFFu) r[0] = r[1] = r[2] = r[3] = 0x7FC07FC0u;
      else decode_word_regs(meta, base2, W, codes[c], r);
    }
    *reinterpret_cast<uint4*>(dst + W * kTokChunkBytes) = make_uint4(r[0], r[1], r[2], r[3]);
  }
}

// Resident tokens (`tiles` n-tiles of `rows` token rows each, all K): the consumer warps of a CTA build them before the
// main loop.  Layout: chunk, n-tile, word W: rows x 4 units x 16 bytes, so that lane (token g, unit q) of a warp reads
// at g * 64 + q * 16 of the word's line (lanes with g >= rows read nothing).  From packed units: task (token n, unit U).
__device__ __forceinline__ void build_tokens_from_units(const uint32_t* __restrict__ A, int M, int64_t upr, uint8_t* tok,
                                                        int tiles, int rows, int tid, int nthreads) {
  const int word_bytes = rows * 64;
  for (int64_t idx = tid; idx < static_cast<int64_t>(tiles) * rows * upr; idx += nthreads) {
    const int n = static_cast<int>(idx / upr);
    const int64_t U = idx - static_cast<int64_t>(n) * upr;
    const int t = n / rows, row = n - t * rows;
    uint8_t* dst = tok + (((U >> 2) * tiles + t) * 8) * word_bytes + (row * 4 + (U & 3)) * 16;
    if (n >= M) {
#pragma unroll
      for (int W = 0; W < 8; ++W) *reinterpret_cast<uint4*>(dst + W * word_bytes) = make_uint4(0u, 0u, 0u, 0u);
      continue;
    }
    const uint32_t* unit = A + (static_cast<int64_t>(n) * upr + U) * kUnitWords;
    const uint32_t meta = __ldg(unit);
#pragma unroll
    for (int W = 0; W < 8; W += 2) {
      uint32_t r[8];
      decode_two_words(meta, W, __ldg(unit + 1 + W), __ldg(unit + 2 + W), r);
      *reinterpret_cast<uint4*>(dst + W * word_bytes) = make_uint4(r[0], r[1], r[2], r[3]);
      *reinterpret_cast<uint4*>(dst + (W + 1) * word_bytes) = make_uint4(r[4], r[5], r[6], r[7]);
    }
  }
}
// From BF16 activations: Algorithm 1 with two lanes per unit (the streaming quantizer's own code), then Eq. 2 of the
// unit just encoded.  Whole warps take part (the encoder exchanges values between the two lanes of a unit): the task
// count is rounded up to a multiple of 32 and the surplus lanes encode zeros that they do not store.
template <bool kRHA>
__device__ __forceinline__ void build_tokens_from_bf16(const uint16_t* __restrict__ X, int64_t ld_x, int M, int64_t upr,
                                                       uint8_t* tok, int tiles, int rows, int tid, int nthreads) {
  const int word_bytes = rows * 64;
  const int64_t tasks = 2 * static_cast<int64_t>(tiles) * rows * upr;
  for (int64_t idx = tid; idx < ((tasks + 31) & ~static_cast<int64_t>(31)); idx += nthreads) {      // nthreads is a multiple of 32
    const bool valid = idx < tasks;
    const int l = static_cast<int>(idx & 1);
    const int64_t pair = idx >> 1;
    const int n = valid ? static_cast<int>(pair / upr) : M;
    const int64_t U = valid ? pair - static_cast<int64_t>(n) * upr : 0;
    const int t = n / rows, row = n - t * rows;
    uint4 v[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) v[c] = make_uint4(0u, 0u, 0u, 0u);
    if (n < M) {
      const uint4* src = reinterpret_cast<const uint4*>(X + static_cast<int64_t>(n) * ld_x + U * kUnitElems) + l;
#pragma unroll
      for (int c = 0; c < 4; ++c) v[c] = __ldg(src + 2 * c);
    }
    uint32_t codes[4], meta;
    encode_unit_bf16_pair<kRHA>(v, l, codes, meta);
    if (!valid) continue;
    uint8_t* dst = tok + (((U >> 2) * tiles + t) * 8) * word_bytes + (row * 4 + (U & 3)) * 16;
    const uint32_t byte = meta & 0xFFu;
    const uint32_t base2 = byte * 0x00200020u + 0x26802680u;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const int W = l + 2 * c;                             // this lane's code words
      uint32_t r[4] = {0u, 0u, 0u, 0u};
      if (n < M) {
        if (byte == 0xFFu) r[0] = r[1] = r[2] = r[3] = 0x7FC07FC0u;
        else decode_word_regs(meta, base2, W, codes[c], r);
      }
      *reinterpret_cast<uint4*>(dst + W * word_bytes) = make_uint4(r[0], r[1], r[2], r[3]);
    }
  }
}

// Per-unit part of the weight decode: the BF16 bits of E6M2 / 4 in both halves, the constant that is
// OR-ed into every element pair (128.0, or NaN for a NaN unit, Eq. 2), and E1_8[j] + E1_16[2j] /
// E1_16[2j+1] for all eight words as two-bit fields of the low / high half.
struct UnitPrep {
  uint32_t base2, or_k, sum;
};
__device__ __forceinline__ UnitPrep prepare_unit(uint32_t meta, uint32_t lut) {
  UnitPrep u;
  const uint32_t byte = meta & 0xFFu;
  u.or_k = byte == 0xFFu ? 0x7FC07FC0u : 0x43004300u;
  u.base2 = byte * 0x00200020u + 0x26802680u;                       // ((byte + 308) << 5) in both halves
  u.sum = (((meta >> 16) & 0x5555u) | ((meta >> 1) & 0x55550000u)) + lds32(lut + ((meta >> 6) & 0x3FCu));
  return u;
}
// Word j of the unit -> four bf16x2 registers holding elements (0,4), (1,5), (2,6), (3,7) of level-2
// group j.  Left shifts and most additions are written as multiply-adds with run-time multipliers so
// that they issue on the multiply-add pipe instead of the integer/logic pipe.
__device__ __forceinline__ void decode_word(const UnitPrep& u, int j, uint32_t wj, const DecodeMul& k, uint32_t (&r)[4]) {
  const uint32_t f = ((u.sum >> (2 * j)) * k.m128) & 0x01800180u;    // field j at the exponent's low bits
  const uint32_t Sa = f * k.one + u.base2;                          // (S_lo, S_hi), S = E6M2 * 2^(e8 + e16 - 2)
  const uint32_t Oa = mul_bf16x2(Sa, 0xC308C308u);                  // -136 S
  const uint32_t uj = offset_nibbles(wj, k);                        // nibbles 8 + value: no separate sign step
  r[0] = fma_bf16x2((uj & 0x000F000Fu) | u.or_k, Sa, Oa);           // (128 + u) S - 136 S
  r[1] = fma_bf16x2(((uj >> 4) & 0x000F000Fu) | u.or_k, Sa, Oa);
  r[2] = fma_bf16x2(((uj >> 8) & 0x000F000Fu) | u.or_k, Sa, Oa);
  r[3] = fma_bf16x2(((uj >> 12) & 0x000F000Fu) | u.or_k, Sa, Oa);
}

// A parity wait cannot tell a barrier that is one phase behind from one that is done, so a consumer
// first waits until the producer has announced the chunk it wants for that stage (the producer only
// announces it after every reader of the stage's previous chunk has arrived).  Bounded like mbar_wait.
__device__ __forceinline__ bool wait_announced(const volatile int* slot, int kc, volatile uint32_t* abort_flag) {
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

// Shared memory: [spread table 1 KB][partial sums][barriers, abort word, announced chunks: 384 B][resident tokens (kSrc 1, 2)]
// [ring of stages, 128-byte aligned]
template <int kTokTiles, int kGemvWarps, int kSrc>
__global__ void __launch_bounds__((kGemvWarps + 1) * 32, 1)
gemv_kernel(const __grid_constant__ CUtensorMap tm_full, const __grid_constant__ CUtensorMap tm_short, const GemvParams p) {
  constexpr bool kResident = kSrc != kSrcWorkspace;
  static_assert(!kResident || kTokTiles <= 2, "resident tokens: one or two n-tiles");
  constexpr int kTokBytes = kTokTiles * kTileChunkBytes;
  // bytes of one word's line of tokens (rows x 4 units x 16 bytes) and of one K = 256 chunk of them
  const uint32_t tok_word_bytes = kResident ? static_cast<uint32_t>(p.res_rows) * 64u : static_cast<uint32_t>(kTokChunkBytes);
  const uint32_t tok_chunk_bytes = kTokTiles * 8u * tok_word_bytes;
  constexpr int kRedBytes = kGemvWarps * 32 * 4 * kTokTiles * 4;     // partial accumulators of every consumer warp
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 127u) & ~127u;
  uint8_t* gen_base = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t lut = smem_base;
  float* red = reinterpret_cast<float*>(gen_base + 1024);
  const uint32_t bar_base = smem_base + 1024 + kRedBytes;
  const uint32_t full = bar_base, empty = bar_base + 8 * kMaxStages;
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(gen_base + 1024 + kRedBytes + 16 * kMaxStages);
  volatile int* announced = reinterpret_cast<volatile int*>(gen_base + 1024 + kRedBytes + 16 * kMaxStages + 16);   // chunk in each stage
  const uint32_t tok_res = bar_base + 384;                              // resident tokens: num_kc chunks of kTokBytes
  uint8_t* tok_res_gen = gen_base + 1024 + kRedBytes + 384;
  const uint32_t ring = tok_res + (kResident ? static_cast<uint32_t>(p.num_kc) * tok_chunk_bytes : 0u);
  const uint32_t w_bytes_max = static_cast<uint32_t>(p.max_blocks) * kBlockBytes;
  const uint32_t stage_bytes = w_bytes_max + (kResident ? 0 : kTokBytes);

  // this CTA's run of 8-row blocks
  const int64_t blk_begin = static_cast<int64_t>(blockIdx.x) * p.num_blocks / gridDim.x;
  const int nblk = static_cast<int>(static_cast<int64_t>(blockIdx.x + 1) * p.num_blocks / gridDim.x - blk_begin);
  const int npairs = (nblk + 1) >> 1;
  const int ways = kGemvWarps / npairs;              // >= 1: npairs <= kMaxBlocks / 2

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
  if (threadIdx.x < 256) reinterpret_cast<uint32_t*>(gen_base)[threadIdx.x] = spread_e8_entry(threadIdx.x);
  __syncthreads();

  if (warp == kGemvWarps) {
    // ---------------------------------------------------------------- producer
    if (lane == 0) {
      const CUtensorMap* map = nblk == p.max_blocks ? &tm_full : &tm_short;
      const uint32_t tx = static_cast<uint32_t>(nblk) * kBlockBytes + (kResident ? 0 : kTokBytes);
      const int row0 = static_cast<int>(blk_begin * kBlockRows);
      // Launched as a programmatic dependent of the token preparation: the weights of the first ring
      // of stages are requested first, then the preparation grid is waited for, then the tokens follow.
      const int head = p.num_kc < p.stages ? p.num_kc : p.stages;
      // With resident tokens the preceding launch in the stream is the caller's (it may have written the weights, the
      // tokens, or still read C): the CTA may be scheduled early, but nothing is read or written before that grid is done.
      if (kResident) asm volatile("griddepcontrol.wait;" ::: "memory");
      for (int kc = 0; kc < head; ++kc) {
        announced[kc] = kc;
        mbar_expect_tx(full + 8 * kc, tx);
        tma_load_2d(ring + kc * stage_bytes, map, kc * kRawRowBytes, row0, full + 8 * kc);
      }
      if (!kResident) {
        asm volatile("griddepcontrol.wait;" ::: "memory");
        for (int kc = 0; kc < head; ++kc)
          bulk_load_1d(ring + kc * stage_bytes + w_bytes_max, p.tokens + static_cast<int64_t>(kc) * kTokBytes, kTokBytes,
                       full + 8 * kc);
      }
      uint32_t s = 0, ph = 1;                          // stage and phase of chunk `head`
      for (int kc = head; kc < p.num_kc; ++kc) {
        if (!mbar_wait(empty + 8 * s, ph ^ 1u, abort_flag, 32)) break;
        announced[s] = kc;
        __threadfence_block();
        mbar_expect_tx(full + 8 * s, tx);
        const uint32_t dst = ring + s * stage_bytes;
        tma_load_2d(dst, map, kc * kRawRowBytes, row0, full + 8 * s);
        if (!kResident) bulk_load_1d(dst + w_bytes_max, p.tokens + static_cast<int64_t>(kc) * kTokBytes, kTokBytes, full + 8 * s);
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
    const uint32_t off_lo = static_cast<uint32_t>(16 * pair + g) * kRawRowBytes + q * kUnitBytes;   // MMA row g
    const uint32_t off_hi = off_lo + 8 * kRawRowBytes;                                                // MMA row g + 8
    const uint32_t off_tok = (kResident ? 0u : w_bytes_max) + static_cast<uint32_t>(lane) * 16;
    const bool tok_row_kept = !kResident || g < p.res_rows;       // resident tokens may keep fewer than eight rows per n-tile
    if (kResident) {
      asm volatile("griddepcontrol.wait;" ::: "memory");      // see the producer
      // every consumer thread helps to build the CTA's own copy of the tokens, then all of them meet
      const int64_t upr = static_cast<int64_t>(p.num_kc) * kRawUnits;
      if (kSrc == kSrcUnits) build_tokens_from_units(p.A, p.M, upr, tok_res_gen, kTokTiles, p.res_rows, threadIdx.x, kGemvWarps * 32);
      else if (p.rha) build_tokens_from_bf16<true>(p.X, p.ld_x, p.M, upr, tok_res_gen, kTokTiles, p.res_rows, threadIdx.x, kGemvWarps * 32);
      else build_tokens_from_bf16<false>(p.X, p.ld_x, p.M, upr, tok_res_gen, kTokTiles, p.res_rows, threadIdx.x, kGemvWarps * 32);
      asm volatile("bar.sync 1, %0;" ::"n"(kGemvWarps * 32) : "memory");
    }
    if (active) {
      uint32_t s = static_cast<uint32_t>(way % p.stages), ph = static_cast<uint32_t>(way / p.stages) & 1u;
      const uint32_t s_step = static_cast<uint32_t>(ways % p.stages), ph_step = static_cast<uint32_t>(ways / p.stages);
      bool ok = true;
      for (int kc = way; kc < p.num_kc; kc += ways) {
        if (!(ok = __all_sync(0xFFFFFFFFu, wait_announced(announced + s, kc, abort_flag) &&
                                               mbar_wait(full + 8 * s, ph, abort_flag))))
          break;
        const uint32_t st = ring + s * stage_bytes;
        const uint32_t tk = kResident ? tok_res + static_cast<uint32_t>(kc) * tok_chunk_bytes : st;      // this chunk's tokens
        const uint32_t ml = lds32(st + off_lo), mh = has_hi ? lds32(st + off_hi) : 0u;
        const UnitPrep ul = prepare_unit(ml, lut), uh = prepare_unit(mh, lut);
        // a short loop rather than eight unrolled words: the body stays small enough for the instruction cache
#pragma unroll 2
        for (int j = 0; j < 8; ++j) {
          uint4 x[kTokTiles];
#pragma unroll
          for (int t = 0; t < kTokTiles; ++t)
            x[t] = tok_row_kept ? lds128(tk + off_tok + (t * 8 + j) * tok_word_bytes) : make_uint4(0u, 0u, 0u, 0u);
          uint32_t a[4], b[4] = {0u, 0u, 0u, 0u};
          decode_word(ul, j, lds32(st + off_lo + 4 + 4 * j), p.mul, a);
          if (has_hi) decode_word(uh, j, lds32(st + off_hi + 4 + 4 * j), p.mul, b);
#pragma unroll
          for (int t = 0; t < kTokTiles; ++t) {
            mma_bf16_16816(acc[t], a[0], b[0], a[1], b[1], x[t].x, x[t].y);
            mma_bf16_16816(acc[t], a[2], b[2], a[3], b[3], x[t].z, x[t].w);
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
    asm volatile("bar.sync 1, %0;" ::"n"(kGemvWarps * 32) : "memory");     // consumer warps only
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

template <int kTokTiles, int kGemvWarps, int kSrc = kSrcWorkspace>
hif4_status launch_gemv_t(const void* B, int64_t upr, GemvParams p, cudaStream_t st) {
  constexpr bool kResident = kSrc != kSrcWorkspace;
  constexpr int kTokBytes = kTokTiles * kTileChunkBytes;
  const int resident_bytes = kResident ? p.num_kc * kTokTiles * 8 * p.res_rows * 64 : 0;
  constexpr int kFixed = 128 + 1024 + kGemvWarps * 32 * 4 * kTokTiles * 4 + 384;
  // One CTA per SM (several rounds of them when a CTA would get more than kMaxBlocks blocks).
  const int64_t sms = sm_count();
  const int64_t rounds = ceil_div64(p.num_blocks, sms * kMaxBlocks);
  const int64_t grid = p.num_blocks < sms * rounds ? p.num_blocks : sms * rounds;
  if (grid > 0x7FFFFFFFll) return HIF4_ERR_SHAPE;
  p.max_blocks = static_cast<int>(ceil_div64(p.num_blocks, grid));
  const int stage_bytes = p.max_blocks * kBlockBytes + (kResident ? 0 : kTokBytes);
  p.stages = (kRingBudget - resident_bytes) / stage_bytes;
  if (p.stages > kMaxStages) p.stages = kMaxStages;
  if (p.stages > p.num_kc) p.stages = p.num_kc;
  if (p.stages < 1) return HIF4_ERR_SHAPE;
  const int smem = kFixed + resident_bytes + p.stages * stage_bytes;
  static uint64_t smem_opt_in = 0;
  if (!ensure_dynamic_smem(gemv_kernel<kTokTiles, kGemvWarps, kSrc>, kFixed + kRingBudget, smem_opt_in)) return HIF4_ERR_CUDA;
  CUtensorMap tm_full, tm_short;
  if (!make_unit_map(&tm_full, B, p.N, upr, p.max_blocks * kBlockRows)) return HIF4_ERR_CUDA;
  if (!make_unit_map(&tm_short, B, p.N, upr, (p.max_blocks > 1 ? p.max_blocks - 1 : 1) * kBlockRows)) return HIF4_ERR_CUDA;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(grid));
  cfg.blockDim = dim3((kGemvWarps + 1) * 32);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;      // may start while the token preparation still runs
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, gemv_kernel<kTokTiles, kGemvWarps, kSrc>, tm_full, tm_short, p) != cudaSuccess) {
    (void)cudaGetLastError();
    return HIF4_ERR_CUDA;
  }
  note_launch();
  return HIF4_OK;
}

}  // namespace

// Token rows are padded to whole MMA n-tiles of 8: one, two or four of them.
static int64_t gemv_m_pad(int64_t M) { return M <= 8 ? 8 : M <= 16 ? 16 : 32; }

bool gemv_supported(const void* A, const void* B, int64_t M, int64_t N, int64_t K) {
  return M >= 1 && M <= kGemvMaxM && gemm_tc_supported(B, B, N, N, N, K) && (reinterpret_cast<uintptr_t>(A) & 3u) == 0;
}

size_t gemv_workspace_bytes(int64_t M, int64_t K) {
  if (M < 1 || M > kGemvMaxM || K <= 0 || K % 256 != 0) return 0;
  return static_cast<size_t>(gemv_m_pad(M) * K * 2);
}

namespace {
// Fills the launch parameters both entry points share; returns false when N is out of range.
bool gemv_params(GemvParams& p, float* C, int64_t M, int64_t N, int64_t K, int64_t ldc, void* workspace) {
  p.tokens = static_cast<uint8_t*>(workspace);
  p.C = C; p.ldc = ldc; p.M = static_cast<int>(M); p.N = N;
  p.num_kc = static_cast<int>(K / 256);
  if (ceil_div64(N, kBlockRows) > 0x7FFFFFFFll) return false;
  p.num_blocks = static_cast<int>(ceil_div64(N, kBlockRows));
  p.mul = make_decode_mul();
  p.error_word = device_error_word();
  return true;
}
// At most two n-tiles of tokens and few enough token elements: the streaming kernel builds them itself, in shared
// memory.  Returns the token rows kept per n-tile (the next power of two >= M, eight for two tiles), 0 when the
// two-launch form is the faster one.  Every CTA repeats the build before its main loop, so it pays only while it costs
// less than the launch it saves: measured break-even (rows kept x K) about 57 000 elements when the tokens are decoded
// from packed units and about 16 000 when they are first converted from BF16 with Algorithm 1.
constexpr int64_t kResidentMaxElemsUnits = 49152, kResidentMaxElemsBf16 = 16384;
int gemv_resident_rows(int64_t M, int num_kc, int64_t max_elems) {
  if (M > 16) return 0;
  const int tiles = M <= 8 ? 1 : 2;
  const int rows = M <= 1 ? 1 : M <= 2 ? 2 : M <= 4 ? 4 : 8;
  const int64_t elems = static_cast<int64_t>(num_kc) * 256 * tiles * rows;
  return elems <= max_elems && elems * 2 <= kResidentMaxBytes ? rows : 0;
}
template <int kSrc>
hif4_status launch_gemv_resident(const void* B, const GemvParams& p, int64_t upr, cudaStream_t st) {
  const int64_t sms = sm_count();
  const int64_t rounds = ceil_div64(p.num_blocks, sms * kMaxBlocks);
  const int64_t grid = p.num_blocks < sms * rounds ? p.num_blocks : sms * rounds;
  const bool many = ceil_div64(p.num_blocks, grid) >= 9;
  if (p.M > 8) return many ? launch_gemv_t<2, kGemvWarpsMany, kSrc>(B, upr, p, st) : launch_gemv_t<2, kGemvWarpsFew, kSrc>(B, upr, p, st);
  return many ? launch_gemv_t<1, kGemvWarpsMany, kSrc>(B, upr, p, st) : launch_gemv_t<1, kGemvWarpsFew, kSrc>(B, upr, p, st);
}
// The streaming kernel on tokens that the preceding launch in `st` has prepared.
hif4_status launch_gemv_stream(const void* B, const GemvParams& p, int m_pad, int64_t upr, cudaStream_t st) {
  // blocks of the largest CTA (same arithmetic as launch_gemv_t): nine or more are five row pairs or more
  const int64_t sms = sm_count();
  const int64_t rounds = ceil_div64(p.num_blocks, sms * kMaxBlocks);
  const int64_t grid = p.num_blocks < sms * rounds ? p.num_blocks : sms * rounds;
  const bool many = ceil_div64(p.num_blocks, grid) >= 9;
  if (m_pad == 32) return launch_gemv_t<4, kGemvWarpsFew>(B, upr, p, st);      // four token tiles: registers for 24 warps only
  if (m_pad == 8) return many ? launch_gemv_t<1, kGemvWarpsMany>(B, upr, p, st) : launch_gemv_t<1, kGemvWarpsFew>(B, upr, p, st);
  return many ? launch_gemv_t<2, kGemvWarpsMany>(B, upr, p, st) : launch_gemv_t<2, kGemvWarpsFew>(B, upr, p, st);
}
}  // namespace

hif4_status launch_gemv(const void* A, const void* B, float* C, int64_t M, int64_t N, int64_t K, int64_t ldc,
                        void* workspace, cudaStream_t st) {
  GemvParams p{};
  p.A = static_cast<const uint32_t*>(A);
  if (!gemv_params(p, C, M, N, K, ldc, workspace)) return HIF4_ERR_SHAPE;
  if (!p.error_word) return HIF4_ERR_CUDA;
  const int m_pad = static_cast<int>(gemv_m_pad(M));
  const int64_t upr = K / kUnitElems;
  p.res_rows = gemv_resident_rows(M, p.num_kc, kResidentMaxElemsUnits);
  if (p.res_rows > 0) return launch_gemv_resident<kSrcUnits>(B, p, upr, st);     // one launch
  const int64_t prep = static_cast<int64_t>(m_pad) * upr;
  gemv_prepare_tokens_kernel<<<static_cast<unsigned>(ceil_div64(prep, 128)), 128, 0, st>>>(p.A, p.M, m_pad, upr, p.tokens);
  note_launch();
  if (cudaGetLastError() != cudaSuccess) return HIF4_ERR_CUDA;
  return launch_gemv_stream(B, p, m_pad, upr, st);
}

bool gemv_linear_supported(const void* X, hif4_dtype dt, int64_t ld_x, const void* B, int64_t M, int64_t N, int64_t K) {
  const int64_t esz = dt == HIF4_FP32 ? 4 : 2;
  return M >= 1 && M <= kGemvMaxM && gemm_tc_supported(B, B, N, N, N, K) && (reinterpret_cast<uintptr_t>(X) & 15u) == 0 &&
         ld_x >= K && (ld_x * esz) % 16 == 0;
}

hif4_status launch_gemv_linear(const void* X, hif4_dtype dt, int64_t ld_x, int rha, const void* B, float* C, int64_t M,
                               int64_t N, int64_t K, int64_t ldc, void* workspace, cudaStream_t st) {
  GemvParams p{};
  if (!gemv_params(p, C, M, N, K, ldc, workspace)) return HIF4_ERR_SHAPE;
  if (!p.error_word) return HIF4_ERR_CUDA;
  const int m_pad = static_cast<int>(gemv_m_pad(M));
  const int64_t upr = K / kUnitElems;
  p.res_rows = dt == HIF4_BF16 ? gemv_resident_rows(M, p.num_kc, kResidentMaxElemsBf16) : 0;
  if (p.res_rows > 0) {        // one launch: conversion, decode and streaming
    p.X = static_cast<const uint16_t*>(X); p.ld_x = ld_x; p.rha = rha;
    return launch_gemv_resident<kSrcBf16>(B, p, upr, st);
  }
  const int lanes = dt == HIF4_BF16 ? 2 : 4;             // lanes per unit of the encoder
  const unsigned blocks = static_cast<unsigned>(ceil_div64(lanes * static_cast<int64_t>(m_pad) * upr, 128));
  if (dt == HIF4_BF16) {
    const uint16_t* x = static_cast<const uint16_t*>(X);
    if (rha) gemv_quantize_tokens_kernel<true><<<blocks, 128, 0, st>>>(x, ld_x, p.M, m_pad, upr, p.tokens);
    else gemv_quantize_tokens_kernel<false><<<blocks, 128, 0, st>>>(x, ld_x, p.M, m_pad, upr, p.tokens);
  } else if (dt == HIF4_FP32) {
    const float* x = static_cast<const float*>(X);
    if (rha) gemv_quantize_tokens32_kernel<true, float><<<blocks, 128, 0, st>>>(x, ld_x, p.M, m_pad, upr, p.tokens);
    else gemv_quantize_tokens32_kernel<false, float><<<blocks, 128, 0, st>>>(x, ld_x, p.M, m_pad, upr, p.tokens);
  } else {
    const __half* x = static_cast<const __half*>(X);
    if (rha) gemv_quantize_tokens32_kernel<true, __half><<<blocks, 128, 0, st>>>(x, ld_x, p.M, m_pad, upr, p.tokens);
    else gemv_quantize_tokens32_kernel<false, __half><<<blocks, 128, 0, st>>>(x, ld_x, p.M, m_pad, upr, p.tokens);
  }
  note_launch();
  if (cudaGetLastError() != cudaSuccess) return HIF4_ERR_CUDA;
  return launch_gemv_stream(B, p, m_pad, upr, st);
}

}  // namespace hif4
