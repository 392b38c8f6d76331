// Device and host helpers shared by the tensor-core HiF4 GEMM kernels (sm_100a): mbarrier, TMA,
// tcgen05 and shared-memory PTX wrappers, the Eq. 2 decoder that turns packed code words into exact
// BF16 pairs, and the tensor map of a packed-unit matrix.
#pragma once
#include <cuda.h>

#include "hif4_bf16x2.cuh"
#include "hif4_common.cuh"

namespace hif4 {
namespace {

// One TMA box row: 4 units = K 256 = 144 bytes (box rows and global pitch must be multiples of 16 bytes).
constexpr int kRawUnits = 4;
constexpr int kRawRowBytes = kRawUnits * kUnitBytes;

constexpr uint64_t kWaitBudgetNs = 2000000000ull;     // 2 s per wait, far beyond any legitimate one

// ------------------------------------------------------------------------------------ PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ uint64_t global_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false when the budget ran out or another thread has already given up.
// Roles that wait long (a whole tile, a whole raw chunk) pass `sleep_ns` > 0 and back off between
// polls, so that their spinning does not take issue slots from the decode warps.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                          uint32_t sleep_ns = 0, uint64_t budget_ns = kWaitBudgetNs) {
  if (mbar_try(bar, parity)) return true;
  const uint64_t t0 = global_ns();
  for (uint32_t it = 1;; ++it) {
    if (mbar_try(bar, parity)) return true;
    if (sleep_ns) __nanosleep(sleep_ns);
    if ((it & 63u) == 0u) {
      if (*abort_flag) return false;
      if (global_ns() - t0 > budget_ns) {
        *abort_flag = 1u;
        return false;
      }
    }
  }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                       uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// K-major SWIZZLE_128B operand descriptor: 128-byte rows, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr) {
  return static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4) | (1ull << 16) | (static_cast<uint64_t>(1024 >> 4) << 32) |
         (1ull << 46) | (2ull << 61);
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ void sts128(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

// Decodes one unit (metadata word + 8 code words) into one 128-byte operand row at `row_addr`;
// 16-byte chunk j of the row lands at position j ^ r7 (SWIZZLE_128B, r7 = row & 7).
__device__ __forceinline__ void decode_unit_to_row(uint32_t meta, const uint32_t* w, uint32_t row_addr, uint32_t r7) {
  const uint32_t byte = meta & 0xFFu;
  if (byte == 0xFFu) {                           // NaN unit (Eq. 2): every element is NaN
#pragma unroll
    for (int j = 0; j < 8; ++j)
      sts128(row_addr + ((static_cast<uint32_t>(j) ^ r7) << 4), 0x7FC07FC0u, 0x7FC07FC0u, 0x7FC07FC0u, 0x7FC07FC0u);
    return;
  }
  // BF16 bits of E6M2 / 4 (the S1P2 quarter): exponent field (byte >> 2) - 48 - 2 + 127, mantissa
  // (byte & 3) << 5, i.e. (byte + 308) << 5; replicated into both halves.
  const uint32_t base2 = ((byte + 308u) << 5) * 0x10001u;
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const uint32_t e8 = (meta >> (1 + j)) & 0x80u;                    // E1_8[j] at bit 7
    const uint32_t e16 = (((meta >> (16 + 2 * j)) & 3u) * 0x00400080u) & 0x00800080u;   // E1_16[2j] bit 7, [2j+1] bit 23
    const uint32_t Sa = base2 + e16 + e8 * 0x10001u;                  // (S_lo, S_hi)
    const uint32_t Sb = Sa - 0x02000200u;                             // S / 16
    const uint32_t Oa = Sa + 0x83808380u;                             // -128 S
    const uint32_t Ob = Sa + 0x81808180u;                             // -8 S
    const uint32_t wj = w[j], wh = wj >> 8;
    const uint32_t r0 = fma_bf16x2((wj & 0x00070007u) | 0x43004300u, Sa, Oa) ^ ((wj << 12) & 0x80008000u);  // elements 0, 4
    const uint32_t r1 = fma_bf16x2((wj & 0x00700070u) | 0x43004300u, Sb, Ob) ^ ((wj << 8) & 0x80008000u);   // elements 1, 5
    const uint32_t r2 = fma_bf16x2((wh & 0x00070007u) | 0x43004300u, Sa, Oa) ^ ((wj << 4) & 0x80008000u);   // elements 2, 6
    const uint32_t r3 = fma_bf16x2((wh & 0x00700070u) | 0x43004300u, Sb, Ob) ^ (wj & 0x80008000u);          // elements 3, 7
    sts128(row_addr + ((static_cast<uint32_t>(j) ^ r7) << 4), r0, r1, r2, r3);
  }
}

// ---- pipe-balanced decoder
// The decode is bound by instruction issue on the integer/logic pipe, while the pipe that runs integer
// multiply-adds and packed BF16 FMAs is mostly idle.  This variant moves every left shift and most
// additions onto that pipe by writing them as multiply-adds with multipliers that the compiler cannot
// see (kernel parameters), takes the sum of the micro-exponents of all eight level-2 groups at once
// (two-bit fields), and uses store addresses that are computed once per thread.
struct DecodeMul {            // runtime-valued on purpose: 1, 2, 7, 8, 32, 128
  uint32_t one, m2, m7, m8, m32, m128;
};
inline DecodeMul make_decode_mul() { return DecodeMul{1u, 2u, 7u, 8u, 32u, 128u}; }

// The eight sign-magnitude nibbles (s, m) of a code word -> offset nibbles u = 8 + value (1..15), all at
// once: u = c ^ 8 for s = 0 and 16 - c for s = 1, i.e. (c ^ (8 | 7s)) + s with no carry out of a nibble.
// An element then decodes as (128 + u) * S - 136 * S with no separate sign step (-0 decodes as +0).
__device__ __forceinline__ uint32_t offset_nibbles(uint32_t w, const DecodeMul& k) {
  const uint32_t s1 = (w & 0x88888888u) >> 3;                       // 1 in every negative nibble
  return (w ^ (s1 * k.m7 | 0x88888888u)) + s1 * k.one;
}

// 256-entry table in shared memory: bit i of the index spread to bit 2i, replicated in both halves.
__device__ __forceinline__ uint32_t spread_e8_entry(uint32_t x) {
  x = (x | (x << 4)) & 0x0F0Fu;
  x = (x | (x << 2)) & 0x3333u;
  x = (x | (x << 1)) & 0x5555u;
  return x * 0x10001u;
}
__device__ __forceinline__ uint32_t lds32(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
  return v;
}

// Decodes one unit into one 128-byte operand row; chunk_addr[j] is the shared-memory address of the
// 16-byte chunk that word j of this thread's row goes to (swizzle applied) inside stage 0, `stage_off`
// the byte offset of the target stage, `lut` the address of the spread table.
__device__ __forceinline__ void decode_unit_balanced(uint32_t meta, const uint32_t* w, const uint32_t (&chunk_addr)[8],
                                                     uint32_t stage_off, uint32_t lut, const DecodeMul& k) {
  const uint32_t byte = meta & 0xFFu;
  if (byte == 0xFFu) {                           // NaN unit (Eq. 2): every element is NaN
#pragma unroll
    for (int j = 0; j < 8; ++j)
      sts128(chunk_addr[j] + stage_off, 0x7FC07FC0u, 0x7FC07FC0u, 0x7FC07FC0u, 0x7FC07FC0u);
    return;
  }
  // BF16 bits of E6M2 / 4 in both halves: ((byte + 308) << 5) * 0x10001
  const uint32_t base2 = byte * 0x00200020u + 0x26802680u;
  // Two-bit fields: field j of the low half = E1_8[j] + E1_16[2j], of the high half = E1_8[j] + E1_16[2j+1]
  const uint32_t sum = (((meta >> 16) & 0x5555u) | ((meta >> 1) & 0x55550000u)) + lds32(lut + ((meta >> 6) & 0x3FCu));
  const uint32_t sumh = sum >> 8;
  const uint32_t mul[4] = {k.m128, k.m32, k.m8, k.m2};
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const uint32_t f = ((j < 4 ? sum : sumh) * mul[j & 3]) & 0x01800180u;       // field j at the exponent's low bits
    const uint32_t Sa = f * k.one + base2;                            // (S_lo, S_hi), S = E6M2 * 2^(e8 + e16 - 2)
    const uint32_t Oa = mul_bf16x2(Sa, 0xC308C308u);                  // -136 S
    const uint32_t uj = offset_nibbles(w[j], k);
    const uint32_t r0 = fma_bf16x2((uj & 0x000F000Fu) | 0x43004300u, Sa, Oa);           // elements 0, 4: (128 + u) S - 136 S
    const uint32_t r1 = fma_bf16x2(((uj >> 4) & 0x000F000Fu) | 0x43004300u, Sa, Oa);    // elements 1, 5
    const uint32_t r2 = fma_bf16x2(((uj >> 8) & 0x000F000Fu) | 0x43004300u, Sa, Oa);    // elements 2, 6
    const uint32_t r3 = fma_bf16x2(((uj >> 12) & 0x000F000Fu) | 0x43004300u, Sa, Oa);   // elements 3, 7
    sts128(chunk_addr[j] + stage_off, r0, r1, r2, r3);
  }
}

// ------------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = [] {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      sym = nullptr;
    return reinterpret_cast<EncodeTiledFn>(sym);
  }();
  return fn;
}

// Byte view of a unit matrix: [rows, upr * 36] uint8, box = 144 bytes x box_rows.
bool make_unit_map(CUtensorMap* map, const void* base, int64_t rows, int64_t upr, int box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(upr * kUnitBytes), static_cast<cuuint64_t>(rows)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(upr * kUnitBytes)};
  const cuuint32_t box[2] = {static_cast<cuuint32_t>(kRawRowBytes), static_cast<cuuint32_t>(box_rows)};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// SM count of the current device (cached per device ordinal: a process may drive several GPUs).
int sm_count() {
  static int cache[64] = {};
  int dev = 0, v = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 148;
  if (dev >= 0 && dev < 64 && cache[dev] > 0) return cache[dev];
  if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) return 148;
  if (dev >= 0 && dev < 64) cache[dev] = v;
  return v;
}

}  // namespace
}  // namespace hif4
