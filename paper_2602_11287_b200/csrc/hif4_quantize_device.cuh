// Device-side pieces of the BF16 form of Algorithm 1 (Section II-B), shared by the streaming quantizer and
// by kernels that quantize a few activation rows on their way into a GEMM: both run exactly this code, so
// their encodings are the same bits.
#pragma once
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

// One unit held by two consecutive lanes: lane l (0 or 1) holds the level-2 groups l, l + 2, l + 4, l + 6 (16
// bytes each) in v[0..3].  Returns the lane's four code words (groups l + 2c) and, in both lanes, the
// unit's metadata word.  Must be called by both lanes of the pair (it exchanges with lane ^ 1).
template <bool kRHA>
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
  vm = max(vm, __shfl_xor_sync(0xFFFFFFFFu, vm, 1));
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
  meta |= __shfl_xor_sync(0xFFFFFFFFu, meta, 1);
  meta |= byte;
  if (unit_nan) {                                      // NaN unit: E6M2 = NaN, all else zero
    meta = 0xFFu;
#pragma unroll
    for (int c = 0; c < 4; ++c) codes[c] = 0u;
  }
  meta_out = meta;
}

}  // namespace
}  // namespace hif4
