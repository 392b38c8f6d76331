// Device-side pieces of Algorithm 1 (Section II-B) in its BF16 and FP32 forms, shared by the streaming quantizer and
// by kernels that quantize a few activation rows on their way into a GEMM: both run exactly this code, so
// their encodings are the same bits.
#pragma once
#include <cuda_fp16.h>

#include "hif4_common.cuh"
#include "hif4_bf16x2.cuh"

namespace hif4 {
namespace {

__device__ __forceinline__ uint32_t umax2(uint32_t a, uint32_t b) { return __vmaxu2(a, b); }
__device__ __forceinline__ uint32_t hmax_halves(uint32_t m) { return max(m & 0xFFFFu, m >> 16); }

// E6M2 byte from the bit pattern of a non-negative, non-NaN float whose mantissa field has
// `kMant` bits and whose exponent bias is 127: round to 2 mantissa bits, then re-bias (127 -> 48)
// and saturate into [0x00, 0xFE].  Subnormals and everything below 2^-48 land on 0x00, Inf and
// everything from 1.75 * 2^15 up on 0xFE.
template <int kMant, bool kRHA>
__device__ __forceinline__ uint32_t e6m2_from_bits(uint32_t h) {
  constexpr int drop = kMant - 2;
  const uint32_t half = 1u << (drop - 1);
  const uint32_t q = kRHA ? (h + half) >> drop : (h + (half - 1) + ((h >> drop) & 1u)) >> drop;
  const int b = static_cast<int>(q) - ((127 - 48) << 2);
  return static_cast<uint32_t>(min(max(b, 0), 0xFE));
}

// Stage 3 of Algorithm 1 for one level-2 group (8 elements, magnitudes a0..a3 as bf16x2 pairs, source
// words x0..x3 for the signs): micro-exponents from the peaks of the products, S1P2 codes packed into
// one 32-bit word.  `e8`, `e16a`, `e16b` come back as 0/1.
template <bool kRHA>
__device__ __forceinline__ uint32_t encode_group_bf16(uint32_t x0, uint32_t x1, uint32_t x2, uint32_t x3,
                                                      uint32_t rec2, uint32_t& e8, uint32_t& e16a,
                                                      uint32_t& e16b) {
  const uint32_t t0 = mul_bf16x2(x0 & 0x7FFF7FFFu, rec2), t1 = mul_bf16x2(x1 & 0x7FFF7FFFu, rec2),
                 t2 = mul_bf16x2(x2 & 0x7FFF7FFFu, rec2), t3 = mul_bf16x2(x3 & 0x7FFF7FFFu, rec2);
  const uint32_t p16a = hmax_halves(umax2(t0, t1));     // elements 0..3 of the group
  const uint32_t p16b = hmax_halves(umax2(t2, t3));     // elements 4..7
  e8 = max(p16a, p16b) >= 0x4080u;                      // >= 4.0
  const uint32_t thr = 0x4000u + (e8 << 7);             // 2.0 * 2^e8
  e16a = p16a >= thr;
  e16b = p16b >= thr;
  uint32_t c0, c1, c2, c3;
  if (!kRHA) {
    // quarter counts 4 * t * 2^-(e8+e16) rounded to nearest-even in the low mantissa bits of 128 + q
    const uint32_t mula = 0x40804080u - (e8 + e16a) * 0x00800080u;
    const uint32_t mulb = 0x40804080u - (e8 + e16b) * 0x00800080u;
    c0 = __vminu2(fma_bf16x2(t0, mula, 0x43004300u), 0x43074307u);
    c1 = __vminu2(fma_bf16x2(t1, mula, 0x43004300u), 0x43074307u);
    c2 = __vminu2(fma_bf16x2(t2, mulb, 0x43004300u), 0x43074307u);
    c3 = __vminu2(fma_bf16x2(t3, mulb, 0x43004300u), 0x43074307u);
  } else {
    // round-half-away: widen to FP32 (exact), add one half, truncate
    const float fa = __uint_as_float((129u - (e8 + e16a)) << 23);
    const float fb = __uint_as_float((129u - (e8 + e16b)) << 23);
    auto rha = [](uint32_t t, float f) {
      const float lo = fminf(__uint_as_float(t << 16) * f, 8.0f);
      const float hi = fminf(__uint_as_float(t & 0xFFFF0000u) * f, 8.0f);
      const uint32_t ql = min(static_cast<uint32_t>(lo + 0.5f), 7u);
      const uint32_t qh = min(static_cast<uint32_t>(hi + 0.5f), 7u);
      return 0x43004300u | ql | (qh << 16);
    };
    c0 = rha(t0, fa); c1 = rha(t1, fa); c2 = rha(t2, fb); c3 = rha(t3, fb);
  }
  // Pack: low bytes of the four bf16x2 results hold the magnitudes; signs come from the top bit of
  // each source element.  Pairs are gathered in swapped order so that one multiply by 0x1001
  // drops (q_even | q_odd << 4) into bytes 1 and 3.
  uint32_t g0 = prmt(c0, c1, 0x4602u), g1 = prmt(c2, c3, 0x4602u);
  g0 |= prmt(x0, x1, 0xDF9Bu) & 0x08080808u;
  g1 |= prmt(x2, x3, 0xDF9Bu) & 0x08080808u;
  return prmt(g0 * 0x1001u, g1 * 0x1001u, 0x7531u);
}

// One unit held by two lanes, kPartner apart (consecutive by default): lane l (0 or 1) holds the level-2 groups l,
// l + 2, l + 4, l + 6 (16 bytes each) in v[0..3].  Returns the lane's four code words (groups l + 2c) and, in both
// lanes, the unit's metadata word.  Must be called by both lanes of the pair (it exchanges with lane ^ kPartner).
template <bool kRHA, int kPartner = 1>
__device__ __forceinline__ void encode_unit_bf16_pair(const uint4 (&v)[4], int l, uint32_t (&codes)[4], uint32_t& meta_out) {
  // metadata bit weights of this lane's groups g = 2i + l: E1_8 bit 8 + g, E1_16 bits 16 + 2g, 17 + 2g
  const uint32_t w8 = 0x100u << l, w16 = 0x10000u << (2 * l);
  // Stage 1: peak magnitude of the unit as an integer maximum of the |x| bit patterns (the group
  // peaks are taken on the products in encode_group_bf16).
  constexpr uint32_t kAbs = 0x7FFF7FFFu;
  uint32_t vm = 0u;
#pragma unroll
  for (int c = 0; c < 4; ++c)
    vm = umax2(vm, umax2(umax2(v[c].x & kAbs, v[c].y & kAbs), umax2(v[c].z & kAbs, v[c].w & kAbs)));
  vm = hmax_halves(vm);
  vm = max(vm, __shfl_xor_sync(0xFFFFFFFFu, vm, kPartner));
  const bool unit_nan = vm > 0x7F80u;

  // Stage 2: level-1 scale, its reciprocal.
  const uint32_t sf = mul_bf16x2(vm, 0x3E12u) & 0xFFFFu;             // Vmax * (1/7)_BF16
  const uint32_t byte = e6m2_from_bits<7, kRHA>(sf);
  // 1/1.M in BF16 is 3F80 3F4D 3F2B 3F12: low byte by table, then the exponent subtraction
  const uint32_t lut = prmt(0x122B4D80u, 0u, (byte & 3u) | 0x4440u);
  const uint32_t rec2 = (lut + 0x5700u - ((byte & 0xFCu) << 5)) * 0x10001u;

  uint32_t m8 = 0u, m16 = 0u;
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    uint32_t e8, e16a, e16b;
    codes[c] = encode_group_bf16<kRHA>(v[c].x, v[c].y, v[c].z, v[c].w, rec2, e8, e16a, e16b);
    m8 += e8 << (2 * c);
    m16 += (e16a + 2u * e16b) << (4 * c);
  }
  uint32_t meta = m8 * w8 + m16 * w16;
  meta |= __shfl_xor_sync(0xFFFFFFFFu, meta, kPartner);
  meta |= byte;
  if (unit_nan) {                                      // NaN unit: E6M2 = NaN, all else zero
    meta = 0xFFu;
#pragma unroll
    for (int c = 0; c < 4; ++c) codes[c] = 0u;
  }
  meta_out = meta;
}

// The same unit held by ONE thread: v[g] is level-2 group g (8 elements, 16 bytes).  Same steps, same helpers, so the
// same bits as the two-lane form; used where a GEMM's operand-decode thread converts the activations it is about to
// decode (one unit per thread and step), with no partner lane to share the work with.
template <bool kRHA>
__device__ __forceinline__ void encode_unit_bf16_single(const uint4 (&v)[8], uint32_t (&codes)[8], uint32_t& meta_out) {
  constexpr uint32_t kAbs = 0x7FFF7FFFu;
  uint32_t vm = 0u;
#pragma unroll
  for (int g = 0; g < 8; ++g)
    vm = umax2(vm, umax2(umax2(v[g].x & kAbs, v[g].y & kAbs), umax2(v[g].z & kAbs, v[g].w & kAbs)));
  vm = hmax_halves(vm);
  const bool unit_nan = vm > 0x7F80u;
  const uint32_t sf = mul_bf16x2(vm, 0x3E12u) & 0xFFFFu;             // Vmax * (1/7)_BF16
  const uint32_t byte = e6m2_from_bits<7, kRHA>(sf);
  const uint32_t lut = prmt(0x122B4D80u, 0u, (byte & 3u) | 0x4440u);
  const uint32_t rec2 = (lut + 0x5700u - ((byte & 0xFCu) << 5)) * 0x10001u;
  uint32_t meta = byte;
#pragma unroll
  for (int g = 0; g < 8; ++g) {
    uint32_t e8, e16a, e16b;
    codes[g] = encode_group_bf16<kRHA>(v[g].x, v[g].y, v[g].z, v[g].w, rec2, e8, e16a, e16b);
    meta |= (e8 << (8 + g)) | ((e16a + 2u * e16b) << (16 + 2 * g));
  }
  if (unit_nan) {                                      // NaN unit: E6M2 = NaN, all else zero
    meta = 0xFFu;
#pragma unroll
    for (int g = 0; g < 8; ++g) codes[g] = 0u;
  }
  meta_out = meta;
}

// ----------------------------------------------------------------------------- FP32 form (FP32 and FP16 sources)
__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.cs.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}
// Four consecutive source elements (one level-3 group) as FP32 bit patterns.  FP16 elements are widened,
// which is exact, so an FP16 tensor encodes like the FP32 tensor of the same values.
__device__ __forceinline__ uint4 load_group_fp32(const float* p) { return ld_stream(reinterpret_cast<const uint4*>(p)); }
__device__ __forceinline__ uint4 load_group_fp32(const __half* p) {
  uint2 h;
  asm volatile("ld.global.cs.v2.u32 {%0,%1}, [%2];" : "=r"(h.x), "=r"(h.y) : "l"(p));
  const float2 lo = __half22float2(*reinterpret_cast<const __half2*>(&h.x));
  const float2 hi = __half22float2(*reinterpret_cast<const __half2*>(&h.y));
  return make_uint4(__float_as_uint(lo.x), __float_as_uint(lo.y), __float_as_uint(hi.x), __float_as_uint(hi.y));
}

// Same steps as above in FP32 arithmetic: (1/7) and the reciprocal table are the nearest FP32 values,
// every product is a single mul.rn.f32.  One level-3 group (4 elements): micro-exponent from the peak
// of the products (e8 is passed in), codes as four nibbles in the low 16 bits.
template <bool kRHA>
__device__ __forceinline__ uint32_t encode_group_fp32(const uint32_t (&xb)[4], const float (&t)[4], uint32_t p16,
                                                      uint32_t e8, uint32_t& e16) {
  e16 = p16 >= 0x40000000u + (e8 << 23);                          // >= 2.0 * 2^e8
  const float mul = __uint_as_float((129u - (e8 + e16)) << 23);   // 4 * 2^-(e8+e16)
  uint32_t half = 0;
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    uint32_t m;
    if (!kRHA) {
      // t * mul is exact (power of two); adding 1.5 * 2^23 rounds it to an integer, nearest-even, in
      // the low mantissa bits; the integer minimum clamps to 7 and also catches Inf
      m = min(__float_as_uint(__fmaf_rn(t[e], mul, 12582912.0f)), 0x4B400007u) & 7u;
    } else {
      const float q = fminf(__fmul_rn(t[e], mul), 8.0f);
      const float fl = truncf(q);
      m = min(static_cast<uint32_t>(fl) + ((q - fl) >= 0.5f ? 1u : 0u), 7u);
    }
    half += (m | ((xb[e] >> 28) & 8u)) << (4 * e);
  }
  return half;
}

// One unit held by four lanes, kStride apart (consecutive by default), in FP32 bit patterns: lane l (0..3) holds the
// level-3 groups l, l + 4, l + 8, l + 12 (4 elements each) in v[0..3].  Returns, in the even lanes, the code words
// (l >> 1) + 2c and, in all four lanes, the unit's metadata word.  Must be called by all four lanes (it exchanges
// with lane ^ kStride, ^ 2 kStride).
template <bool kRHA, int kStride = 1>
__device__ __forceinline__ void encode_unit_fp32_quad(const uint4 (&v)[4], int l, uint32_t (&codes)[4], uint32_t& meta_out) {
  uint32_t xb[4][4], ab[4][4];
  uint32_t vm = 0u;
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    xb[c][0] = v[c].x; xb[c][1] = v[c].y; xb[c][2] = v[c].z; xb[c][3] = v[c].w;
#pragma unroll
    for (int e = 0; e < 4; ++e) { ab[c][e] = xb[c][e] & 0x7FFFFFFFu; vm = max(vm, ab[c][e]); }
  }
  vm = max(vm, __shfl_xor_sync(0xFFFFFFFFu, vm, kStride));
  vm = max(vm, __shfl_xor_sync(0xFFFFFFFFu, vm, 2 * kStride));
  const bool unit_nan = vm > 0x7F800000u;

  const float sf = __fmul_rn(__uint_as_float(vm), __uint_as_float(0x3E124925u));   // (1/7)_FP32
  const uint32_t byte = e6m2_from_bits<23, kRHA>(__float_as_uint(sf));
  const uint32_t M = byte & 3u;
  // nearest FP32 of 1, 0.8, 2/3, 4/7
  const uint32_t lut = M == 0 ? 0x3F800000u : M == 1 ? 0x3F4CCCCDu : M == 2 ? 0x3F2AAAABu : 0x3F124925u;
  const float rec = __uint_as_float(lut + (48u << 23) - ((byte >> 2) << 23));

  uint32_t half[4], meta = 0u;
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    float t[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) t[e] = __fmul_rn(__uint_as_float(ab[c][e]), rec);
    const uint32_t p16 = max(max(__float_as_uint(t[0]), __float_as_uint(t[1])),
                             max(__float_as_uint(t[2]), __float_as_uint(t[3])));
    // level-2 peak: this lane's level-3 group and its neighbour's
    const uint32_t e8 = max(p16, __shfl_xor_sync(0xFFFFFFFFu, p16, kStride)) >= 0x40800000u;    // >= 4.0
    uint32_t e16;
    half[c] = encode_group_fp32<kRHA>(xb[c], t, p16, e8, e16);
    // level-3 group l + 4c -> E1_16 bit 16 + l + 4c; its level-2 group (l >> 1) + 2c -> E1_8 bit, set by the even lane
    meta |= e16 << (16 + l + 4 * c);
    if ((l & 1) == 0) meta |= e8 << (8 + (l >> 1) + 2 * c);
  }
  // even lane: word (l >> 1) + 2c = its four nibbles | the odd neighbour's << 16
  const uint32_t mine01 = half[0] | (half[1] << 16), mine23 = half[2] | (half[3] << 16);
  const uint32_t other01 = __shfl_xor_sync(0xFFFFFFFFu, mine01, kStride), other23 = __shfl_xor_sync(0xFFFFFFFFu, mine23, kStride);
  const uint32_t packed[4] = {(mine01 & 0xFFFFu) | (other01 << 16), (mine01 >> 16) | (other01 & 0xFFFF0000u),
                       (mine23 & 0xFFFFu) | (other23 << 16), (mine23 >> 16) | (other23 & 0xFFFF0000u)};
  meta |= __shfl_xor_sync(0xFFFFFFFFu, meta, kStride);
  meta |= __shfl_xor_sync(0xFFFFFFFFu, meta, 2 * kStride);
  meta |= byte;
#pragma unroll
  for (int c = 0; c < 4; ++c) codes[c] = unit_nan ? 0u : packed[c];
  meta_out = unit_nan ? 0xFFu : meta;
}

}  // namespace
}  // namespace hif4
