// hif4_ref.cpp -- CPU oracle for the HiF4 format ("HiFloat4 Format for Language Model Inference").
//
// TEST INFRASTRUCTURE ONLY.  This is a plain, slow, obviously-correct restatement of what the
// paper defines: decode (Eq. 2), the BF16/FP32 -> HiF4 conversion (Algorithm 1, Section II-B),
// the dot product (Eq. 3), a flat FP64 GEMM on decoded values, and the MXFP4 / NVFP4 round trips that the
// quantization-error study of Section III-A compares HiF4 with.  It shares no code, table or
// constant with the CUDA library and must never be linked into or called from it; only the test
// suite, the smoke check and the benchmark's CPU-baseline leg use it.
//
// Every value is carried as a double that is exactly representable in the working precision P
// (BF16: 8-bit significand; FP32: 24-bit significand; both with exponent range [-126, 127] and
// gradual underflow).  rP() rounds an exactly formed double product to P once, to nearest-even,
// which is what "a BF16 multiply" (or "an FP32 multiply") is.  Products of two P values are exact
// in double (at most 48 significand bits).
//
// Parity pins (tests/test_oracle_*.py): Table I / Table II constants, exhaustive decode of all
// 255 x 2 x 2 x 16 combinations against integer arithmetic, hand-derived worked encodings, E6M2
// rounding vectors, sign/scale/permutation invariants, the paper's Gaussian MSE ratio, brute-force
// optimum as a lower bound, Eq. 3 against the flat sum.  The P = FP32 form of Algorithm 1 (FP32 and
// FP16 sources) is pinned separately: a restatement with numpy float32 products on thousands of
// units in both rounding modes, and hand-derived cases in which a BF16-precision (1/7), scale
// product, table entry or threshold product would change a byte, a micro-exponent or a code.
// Parity unpinned: the byte/bit order inside a unit and the choice of FP32 working precision for
// FP32/FP16 sources are conventions of this repository (the paper's unit figure is not available
// as text and it only says that those types are converted in a like manner); the paper prints no
// worked encoding, so the worked examples are derived by hand from Algorithm 1.

#include <cmath>
#include <cstdint>
#include <cstring>
#include <thread>
#include <vector>
#include <limits>
#include <algorithm>

namespace {

constexpr int kUnit = 64;        // elements per unit (Section II-A)
constexpr int kUnitBytes = 36;   // 32-bit metadata + 64 x 4 bit

enum { DT_BF16 = 0, DT_FP32 = 1, DT_FP64 = 2 };
enum { RND_RNE = 0, RND_RHA = 1 };

// ---------------------------------------------------------------- precision P
struct Prec { int sig_bits; int emin; int emax; };
const Prec kBF16{8, -126, 127};
const Prec kFP32{24, -126, 127};

// Round a double to the binary format `p` (round-to-nearest, ties-to-even, gradual underflow,
// overflow to infinity).  nearbyint() runs in the default rounding mode, which is ties-to-even.
double round_to(double v, const Prec& p) {
  if (v == 0.0 || !std::isfinite(v)) return v;
  int e = std::ilogb(v);
  if (e < p.emin) e = p.emin;
  const double quantum = std::ldexp(1.0, e - (p.sig_bits - 1));
  double r = std::nearbyint(v / quantum) * quantum;
  const double maxv = std::ldexp(2.0 - std::ldexp(1.0, -(p.sig_bits - 1)), p.emax);
  if (std::fabs(r) > maxv) r = std::copysign(std::numeric_limits<double>::infinity(), v);
  return r;
}

// Rounding of a non-negative value to an integer under the selectable mode (Section II-B:
// half-to-even or half-away-from-zero).
double round_int(double v, int mode) {
  return mode == RND_RHA ? std::floor(v + 0.5) : std::nearbyint(v);
}

// ---------------------------------------------------------------- storage helpers
double load_elem(const void* base, int dt, int64_t idx) {
  if (dt == DT_BF16) {
    uint16_t h = static_cast<const uint16_t*>(base)[idx];
    uint32_t u = static_cast<uint32_t>(h) << 16;
    float f;
    std::memcpy(&f, &u, 4);
    return static_cast<double>(f);
  }
  if (dt == DT_FP32) return static_cast<double>(static_cast<const float*>(base)[idx]);
  return static_cast<const double*>(base)[idx];
}

// v is exactly representable in the target type (decode results are), or NaN.
void store_elem(void* base, int dt, int64_t idx, double v) {
  if (dt == DT_FP64) { static_cast<double*>(base)[idx] = v; return; }
  float f = static_cast<float>(v);
  uint32_t u;
  if (std::isnan(v)) u = 0x7FC00000u; else std::memcpy(&u, &f, 4);
  if (dt == DT_FP32) { std::memcpy(static_cast<float*>(base) + idx, &u, 4); return; }
  static_cast<uint16_t*>(base)[idx] = static_cast<uint16_t>(u >> 16);
}

// ---------------------------------------------------------------- E6M2 (Table I, Eq. 1)
bool e6m2_is_nan(unsigned byte) { return byte == 0xFFu; }
double e6m2_value(unsigned byte) {
  if (e6m2_is_nan(byte)) return std::numeric_limits<double>::quiet_NaN();
  const int E = static_cast<int>(byte >> 2) - 48;   // bias 48
  const int M = static_cast<int>(byte & 3u);        // hidden bit 1
  return std::ldexp(1.0 + M / 4.0, E);
}

// BF16_to_E6M2 (Algorithm 1, level-1 scale factor step): keep a 3-bit significand, carry into the exponent on
// mantissa overflow, saturate into [0x00, 0xFE] (the format has no zero, no infinity, and 0xFF is
// reserved for NaN, so finite data never produces it).  sf >= 0 and not NaN.
unsigned e6m2_from_value(double sf, int mode) {
  if (std::isinf(sf)) return 0xFEu;
  if (sf <= 0.0) return 0x00u;
  int e = std::ilogb(sf);
  const double frac = std::ldexp(sf, -e);            // [1, 2), exact
  int q = static_cast<int>(round_int((frac - 1.0) * 4.0, mode));
  if (q == 4) { q = 0; e += 1; }
  if (e < -48) return 0x00u;
  if (e > 15 || (e == 15 && q == 3)) return 0xFEu;
  return static_cast<unsigned>(((e + 48) << 2) | q);
}

// E6M2_REC_to_BF16 (Algorithm 1, reciprocal step; Section II-B): four-entry table on the mantissa, entry =
// 1/1.M rounded to P, and an exponent subtraction (exact scaling by a power of two).
double e6m2_reciprocal(unsigned byte, const Prec& p) {
  const int E = static_cast<int>(byte >> 2) - 48;
  const int M = static_cast<int>(byte & 3u);
  const double entry = round_to(1.0 / (1.0 + M / 4.0), p);
  return std::ldexp(entry, -E);
}

// ---------------------------------------------------------------- unit access
uint32_t unit_meta(const uint8_t* u) {
  return static_cast<uint32_t>(u[0]) | (static_cast<uint32_t>(u[1]) << 8) |
         (static_cast<uint32_t>(u[2]) << 16) | (static_cast<uint32_t>(u[3]) << 24);
}
unsigned unit_code(const uint8_t* u, int i) {
  const uint8_t b = u[4 + i / 2];
  return (i & 1) ? (b >> 4) : (b & 0xF);
}

// Eq. 2: the 64 values of a unit.
void decode_unit(const uint8_t* u, double out[kUnit]) {
  const uint32_t meta = unit_meta(u);
  const unsigned byte = meta & 0xFFu;
  if (e6m2_is_nan(byte)) {
    for (int i = 0; i < kUnit; ++i) out[i] = std::numeric_limits<double>::quiet_NaN();
    return;
  }
  const double scale = e6m2_value(byte);
  for (int i = 0; i < kUnit; ++i) {
    const int e8 = (meta >> (8 + i / 8)) & 1u;
    const int e16 = (meta >> (16 + i / 4)) & 1u;
    const unsigned c = unit_code(u, i);
    const double s1p2 = (c & 7u) / 4.0;
    const double v = scale * std::ldexp(s1p2, e8 + e16);
    out[i] = (c & 8u) ? -v : v;
  }
}

// Algorithm 1, step by step, in working precision p.
void encode_unit(const double x[kUnit], const Prec& p, int mode, uint8_t out[kUnitBytes]) {
  std::memset(out, 0, kUnitBytes);
  for (int i = 0; i < kUnit; ++i) {
    if (std::isnan(x[i])) { out[0] = 0xFF; return; }   // NaN unit: E6M2 = NaN, rest zero
  }
  // Stage 1: three-level tree of peak magnitudes.
  double V16[16], V8[8], Vmax = 0.0;
  for (int k = 0; k < 16; ++k) {
    V16[k] = 0.0;
    for (int t = 0; t < 4; ++t) V16[k] = std::max(V16[k], std::fabs(x[4 * k + t]));
  }
  for (int j = 0; j < 8; ++j) V8[j] = std::max(V16[2 * j], V16[2 * j + 1]);
  for (int j = 0; j < 8; ++j) Vmax = std::max(Vmax, V8[j]);

  // Stage 2: level-1 scale, its reciprocal, the micro-exponents.
  const double c7 = round_to(1.0 / 7.0, p);                 // (1/7)_P
  const double SF = round_to(Vmax * c7, p);                 // high-precision scale factor
  const unsigned byte = e6m2_from_value(SF, mode);          // level-1 scale factor
  const double REC = e6m2_reciprocal(byte, p);              // reciprocal of E6M2
  int e8[8], e16[16];
  for (int j = 0; j < 8; ++j) e8[j] = round_to(V8[j] * REC, p) >= 4.0 ? 1 : 0;   // level 2
  for (int k = 0; k < 16; ++k)
    e16[k] = std::ldexp(round_to(V16[k] * REC, p), -e8[k / 2]) >= 2.0 ? 1 : 0;   // level 3

  uint32_t meta = byte;
  for (int j = 0; j < 8; ++j) meta |= static_cast<uint32_t>(e8[j]) << (8 + j);
  for (int k = 0; k < 16; ++k) meta |= static_cast<uint32_t>(e16[k]) << (16 + k);
  out[0] = meta & 0xFF; out[1] = (meta >> 8) & 0xFF; out[2] = (meta >> 16) & 0xFF; out[3] = meta >> 24;

  // Stage 3: scale each element, round to S1P2, clamp to 1.75, keep the sign.
  for (int i = 0; i < kUnit; ++i) {
    const double t = std::ldexp(round_to(x[i] * REC, p), -(e8[i / 8] + e16[i / 4]));
    double m = round_int(std::fabs(t) * 4.0, mode);         // S1P2 magnitude in quarters
    if (m > 7.0) m = 7.0;
    const unsigned code = static_cast<unsigned>(m) | (std::signbit(x[i]) ? 8u : 0u);
    out[4 + i / 2] |= static_cast<uint8_t>((i & 1) ? (code << 4) : code);
  }
}

template <class F>
void parallel_rows(int64_t rows, int nthreads, F&& body) {
  if (nthreads <= 1 || rows < 2) { body(int64_t{0}, rows); return; }
  nthreads = static_cast<int>(std::min<int64_t>(nthreads, rows));
  std::vector<std::thread> pool;
  const int64_t chunk = (rows + nthreads - 1) / nthreads;
  for (int t = 0; t < nthreads; ++t) {
    const int64_t r0 = t * chunk, r1 = std::min(rows, r0 + chunk);
    if (r0 >= r1) break;
    pool.emplace_back([=, &body] { body(r0, r1); });
  }
  for (auto& th : pool) th.join();
}

const Prec& prec_of(int dt) { return dt == DT_BF16 ? kBF16 : kFP32; }

// Integer part of Eq. 3 for one unit pair: level-3 micro-exponents absorbed into the elements
// (5-bit signed integers in quarters), 4-element sums, then the level-2 shifts.  The result is in
// units of 1/16 (product of two quarter-valued elements).
int64_t eq3_integer_sum(const uint8_t* ua, const uint8_t* ub) {
  const uint32_t ma = unit_meta(ua), mb = unit_meta(ub);
  int64_t total = 0;
  for (int i = 0; i < 8; ++i) {                       // level-2 groups
    int64_t s2 = 0;
    for (int j = 2 * i; j <= 2 * i + 1; ++j) {        // level-3 groups
      int64_t s3 = 0;
      for (int k = 4 * j; k < 4 * j + 4; ++k) {       // elements
        const unsigned ca = unit_code(ua, k), cb = unit_code(ub, k);
        const int a = (ca & 8u) ? -static_cast<int>(ca & 7u) : static_cast<int>(ca & 7u);
        const int b = (cb & 8u) ? -static_cast<int>(cb & 7u) : static_cast<int>(cb & 7u);
        s3 += a * b;
      }
      const int sh3 = ((ma >> (16 + j)) & 1u) + ((mb >> (16 + j)) & 1u);
      s2 += s3 * (int64_t{1} << sh3);                 // shift of a signed sum, written as a multiply
    }
    const int sh2 = ((ma >> (8 + i)) & 1u) + ((mb >> (8 + i)) & 1u);
    total += s2 * (int64_t{1} << sh2);
  }
  return total;
}

}  // namespace

// =====================================================================================
// C interface (host pointers everywhere).  Return 0 on success, non-zero on bad arguments.
// =====================================================================================
extern "C" {

int hif4_ref_unit_bytes(void) { return kUnitBytes; }

int64_t hif4_ref_packed_bytes(int64_t rows, int64_t cols) {
  if (rows < 0 || cols < 0 || cols % kUnit) return 0;
  return rows * (cols / kUnit) * kUnitBytes;
}

double hif4_ref_e6m2_value(unsigned byte) { return e6m2_value(byte & 0xFFu); }
unsigned hif4_ref_e6m2_from_value(double sf, int mode) { return e6m2_from_value(sf, mode); }
double hif4_ref_e6m2_reciprocal(unsigned byte, int dt) { return e6m2_reciprocal(byte & 0xFFu, prec_of(dt)); }
double hif4_ref_round_to(double v, int dt) { return round_to(v, prec_of(dt)); }

// Algorithm 1 over a [rows, cols] matrix of dtype dt (0 = BF16, 1 = FP32), row stride ld_src
// elements; writes rows*(cols/64) units.
int hif4_ref_quantize(const void* src, int dt, int64_t rows, int64_t cols, int64_t ld_src,
                      void* dst_units, int mode, int nthreads) {
  if (!src || !dst_units) return 1;
  if (rows < 0 || cols < 0 || cols % kUnit || ld_src < cols) return 2;
  if (dt != DT_BF16 && dt != DT_FP32) return 4;
  const int64_t upr = cols / kUnit;
  uint8_t* out = static_cast<uint8_t*>(dst_units);
  parallel_rows(rows, nthreads, [&](int64_t r0, int64_t r1) {
    double x[kUnit];
    for (int64_t r = r0; r < r1; ++r)
      for (int64_t u = 0; u < upr; ++u) {
        for (int i = 0; i < kUnit; ++i) x[i] = load_elem(src, dt, r * ld_src + u * kUnit + i);
        encode_unit(x, prec_of(dt), mode, out + (r * upr + u) * kUnitBytes);
      }
  });
  return 0;
}

// Eq. 2 over a matrix of units; dt may also be 2 (FP64 output).
int hif4_ref_dequantize(const void* src_units, int64_t rows, int64_t cols, void* dst, int dt,
                        int64_t ld_dst, int nthreads) {
  if (!src_units || !dst) return 1;
  if (rows < 0 || cols < 0 || cols % kUnit || ld_dst < cols) return 2;
  if (dt < DT_BF16 || dt > DT_FP64) return 4;
  const int64_t upr = cols / kUnit;
  const uint8_t* in = static_cast<const uint8_t*>(src_units);
  parallel_rows(rows, nthreads, [&](int64_t r0, int64_t r1) {
    double v[kUnit];
    for (int64_t r = r0; r < r1; ++r)
      for (int64_t u = 0; u < upr; ++u) {
        decode_unit(in + (r * upr + u) * kUnitBytes, v);
        for (int i = 0; i < kUnit; ++i) store_elem(dst, dt, r * ld_dst + u * kUnit + i, v[i]);
      }
  });
  return 0;
}

// C[i][j] = sum_k a_ik * b_jk in FP64 on decoded operands (flat definition of Eq. 3 summed over
// the K/64 unit pairs); Cabs (may be NULL) receives sum_k |a_ik| |b_jk| for the tolerance.
int hif4_ref_gemm_f64(const void* A_units, const void* B_units, double* C, double* Cabs, int64_t M,
                      int64_t N, int64_t K, int nthreads) {
  if (!A_units || !B_units || !C) return 1;
  if (M < 0 || N < 0 || K < 0 || K % kUnit) return 2;
  std::vector<double> A(static_cast<size_t>(M * K)), B(static_cast<size_t>(N * K));
  if (M > 0 && K > 0) hif4_ref_dequantize(A_units, M, K, A.data(), DT_FP64, K, nthreads);
  if (N > 0 && K > 0) hif4_ref_dequantize(B_units, N, K, B.data(), DT_FP64, K, nthreads);
  parallel_rows(M, nthreads, [&](int64_t r0, int64_t r1) {
    for (int64_t i = r0; i < r1; ++i)
      for (int64_t j = 0; j < N; ++j) {
        double s = 0.0, sa = 0.0;
        for (int64_t k = 0; k < K; ++k) {
          const double a = A[i * K + k], b = B[j * K + k];
          s += a * b;
          sa += std::fabs(a) * std::fabs(b);
        }
        C[i * N + j] = s;
        if (Cabs) Cabs[i * N + j] = sa;
      }
  });
  return 0;
}

// The same for `count` sampled entries (rows[s], cols[s]) of a large product.
int hif4_ref_gemm_sampled_f64(const void* A_units, const void* B_units, int64_t M, int64_t N,
                              int64_t K, const int64_t* rows, const int64_t* cols, int64_t count,
                              double* out, double* out_abs) {
  if (!A_units || !B_units || !rows || !cols || !out) return 1;
  if (M < 0 || N < 0 || K < 0 || K % kUnit) return 2;
  const int64_t upr = K / kUnit;
  const uint8_t* A = static_cast<const uint8_t*>(A_units);
  const uint8_t* B = static_cast<const uint8_t*>(B_units);
  double a[kUnit], b[kUnit];
  for (int64_t s = 0; s < count; ++s) {
    if (rows[s] < 0 || rows[s] >= M || cols[s] < 0 || cols[s] >= N) return 2;
    double acc = 0.0, acc_abs = 0.0;
    for (int64_t u = 0; u < upr; ++u) {
      decode_unit(A + (rows[s] * upr + u) * kUnitBytes, a);
      decode_unit(B + (cols[s] * upr + u) * kUnitBytes, b);
      for (int i = 0; i < kUnit; ++i) { acc += a[i] * b[i]; acc_abs += std::fabs(a[i]) * std::fabs(b[i]); }
    }
    out[s] = acc;
    if (out_abs) out_abs[s] = acc_abs;
  }
  return 0;
}

// Grouped form: rows off[g]..off[g+1] of A against weight matrix g of B ([G, N, K/64] units).
int hif4_ref_grouped_gemm_f64(const void* A_units, const void* B_units, double* C, double* Cabs,
                              const int64_t* offsets, int num_groups, int64_t N, int64_t K,
                              int nthreads) {
  if (!A_units || !B_units || !C || !offsets) return 1;
  if (num_groups < 0 || N < 0 || K < 0 || K % kUnit) return 2;
  const int64_t upr = K / kUnit;
  const uint8_t* A = static_cast<const uint8_t*>(A_units);
  const uint8_t* B = static_cast<const uint8_t*>(B_units);
  for (int g = 0; g < num_groups; ++g) {
    const int64_t r0 = offsets[g], r1 = offsets[g + 1];
    if (r1 < r0) return 2;
    if (r1 == r0) continue;
    int rc = hif4_ref_gemm_f64(A + r0 * upr * kUnitBytes, B + static_cast<int64_t>(g) * N * upr * kUnitBytes,
                               C + r0 * N, Cabs ? Cabs + r0 * N : nullptr, r1 - r0, N, K, nthreads);
    if (rc) return rc;
  }
  return 0;
}

// Eq. 3 for one pair of units, evaluated the way the paper's flow does: an integer sum with the
// micro-exponents as shifts, then one multiplication by the two level-1 scales.
double hif4_ref_dot_eq3(const void* unit_a, const void* unit_b) {
  const uint8_t* ua = static_cast<const uint8_t*>(unit_a);
  const uint8_t* ub = static_cast<const uint8_t*>(unit_b);
  const unsigned ba = unit_meta(ua) & 0xFFu, bb = unit_meta(ub) & 0xFFu;
  if (e6m2_is_nan(ba) || e6m2_is_nan(bb)) return std::numeric_limits<double>::quiet_NaN();
  const int64_t isum = eq3_integer_sum(ua, ub);
  return e6m2_value(ba) * e6m2_value(bb) * (static_cast<double>(isum) / 16.0);
}

// Exhaustive search for the unit (over every E6M2 byte, every micro-exponent setting and every
// code) that minimises the squared error to x[0..63].  The search decomposes: for a fixed level-1
// byte each level-2 group chooses its bit independently, inside it each level-3 group, inside that
// each element takes its nearest code.  Returns the minimum sum of squared errors and writes the
// minimising unit (ties: first found).  x must be finite.
double hif4_ref_best_unit(const double* x, void* best_unit) {
  double best = std::numeric_limits<double>::infinity();
  uint8_t bestu[kUnitBytes] = {0};
  for (unsigned byte = 0; byte < 0xFFu; ++byte) {
    const double scale = e6m2_value(byte);
    uint8_t cand[kUnitBytes] = {0};
    uint32_t meta = byte;
    double err = 0.0;
    for (int j = 0; j < 8; ++j) {
      double best2 = std::numeric_limits<double>::infinity();
      int best_e8 = 0, best_e16[2] = {0, 0};
      unsigned best_codes[8] = {0};
      for (int e8 = 0; e8 < 2; ++e8) {
        double err2 = 0.0;
        int pick16[2];
        unsigned codes[8];
        for (int h = 0; h < 2; ++h) {
          double best3 = std::numeric_limits<double>::infinity();
          for (int e16 = 0; e16 < 2; ++e16) {
            double err3 = 0.0;
            unsigned c3[4];
            for (int t = 0; t < 4; ++t) {
              const double xv = x[8 * j + 4 * h + t];
              double be = std::numeric_limits<double>::infinity();
              unsigned bc = 0;
              for (unsigned m = 0; m < 8; ++m) {
                const double v = scale * std::ldexp(m / 4.0, e8 + e16);
                const double d = std::fabs(xv) - v;
                if (d * d < be) { be = d * d; bc = m; }
              }
              c3[t] = bc | (std::signbit(xv) ? 8u : 0u);
              err3 += be;
            }
            if (err3 < best3) { best3 = err3; pick16[h] = e16; for (int t = 0; t < 4; ++t) codes[4 * h + t] = c3[t]; }
          }
          err2 += best3;
        }
        if (err2 < best2) {
          best2 = err2; best_e8 = e8; best_e16[0] = pick16[0]; best_e16[1] = pick16[1];
          for (int t = 0; t < 8; ++t) best_codes[t] = codes[t];
        }
      }
      err += best2;
      meta |= static_cast<uint32_t>(best_e8) << (8 + j);
      meta |= static_cast<uint32_t>(best_e16[0]) << (16 + 2 * j);
      meta |= static_cast<uint32_t>(best_e16[1]) << (16 + 2 * j + 1);
      for (int t = 0; t < 8; ++t) {
        const int i = 8 * j + t;
        cand[4 + i / 2] |= static_cast<uint8_t>((i & 1) ? (best_codes[t] << 4) : best_codes[t]);
      }
    }
    if (err < best) {
      best = err;
      cand[0] = meta & 0xFF; cand[1] = (meta >> 8) & 0xFF; cand[2] = (meta >> 16) & 0xFF; cand[3] = meta >> 24;
      std::memcpy(bestu, cand, kUnitBytes);
    }
  }
  if (best_unit) std::memcpy(best_unit, bestu, kUnitBytes);
  return best;
}

// ---------------------------------------------------------------- comparison formats of Section III-A
// The quantization-error study converts the same matrices to MXFP4 and NVFP4 as well.  Both are published
// formats; only what the study needs is restated here (quantize-then-dequantize of a flat array), in FP32
// arithmetic with IEEE round-to-nearest-even operations, one operation per step, so that a GPU kernel can be
// compared bit for bit.
//   E2M1 element: magnitudes {0, 0.5, 1, 1.5, 2, 3, 4, 6}, round to nearest, ties to the even code, saturating.
//   MXFP4: blocks of 32, power-of-two scale 2^(floor(log2 amax) - 2) (2 = the largest E2M1 exponent), exponent
//          clamped to [-127, 127]; elements round(x / scale), so values between 6 and 8 scales saturate to 6.
//   NVFP4: blocks of 16, scale = E4M3(amax / 6) (the group's peak lands on 6, the largest E2M1 magnitude), elements
//          round(x / scale).  With per-tensor scaling the tensor is first multiplied by gain = 2688 / max|x|
//          (2688 = 448 * 6) and the result divided by the gain again.
namespace {
const float kE2M1[8] = {0.0f, 0.5f, 1.0f, 1.5f, 2.0f, 3.0f, 4.0f, 6.0f};

float e2m1_round(float q) {                       // q >= 0
  int best = 0;
  for (int c = 1; c < 8; ++c) {
    const float d_best = std::fabs(q - kE2M1[best]), d_c = std::fabs(q - kE2M1[c]);
    if (d_c < d_best || (d_c == d_best && (c % 2 == 0))) best = c;     // nearest; a tie goes to the even code
  }
  return kE2M1[best];
}

// FP8 E4M3 (bias 7, 3 mantissa bits, subnormals in steps of 2^-9, largest value 448): nearest-even, saturating.
float e4m3_round(float v) {                       // v >= 0, finite
  if (v == 0.0f) return 0.0f;
  int e = std::ilogb(v);
  if (e < -6) e = -6;
  const float quantum = std::ldexp(1.0f, e - 3);
  const float r = std::nearbyint(v / quantum) * quantum;           // division by a power of two: exact
  return r > 448.0f ? 448.0f : r;
}
}  // namespace

float hif4_ref_e2m1_round(float q) { return e2m1_round(q); }
float hif4_ref_e4m3_round(float v) { return e4m3_round(v); }

// 2688 / max|x| in FP32 (one division); 1 for an all-zero tensor.
float hif4_ref_pts_gain(const float* x, int64_t n) {
  float amax = 0.0f;
  for (int64_t i = 0; i < n; ++i) amax = std::max(amax, std::fabs(x[i]));
  return amax > 0.0f ? 2688.0f / amax : 1.0f;
}

int hif4_ref_mxfp4_roundtrip(const float* x, int64_t n, float* out) {
  if (!x || !out) return 1;
  if (n < 0 || n % 32) return 2;
  for (int64_t b = 0; b < n; b += 32) {
    float amax = 0.0f;
    for (int i = 0; i < 32; ++i) amax = std::max(amax, std::fabs(x[b + i]));
    if (amax == 0.0f) { for (int i = 0; i < 32; ++i) out[b + i] = std::copysign(0.0f, x[b + i]); continue; }
    int e = std::ilogb(amax) - 2;
    e = std::min(127, std::max(-127, e));
    const float scale = std::ldexp(1.0f, e);
    for (int i = 0; i < 32; ++i) {
      const float q = std::fabs(x[b + i]) / scale;
      out[b + i] = std::copysign(e2m1_round(q) * scale, x[b + i]);
    }
  }
  return 0;
}

int hif4_ref_nvfp4_roundtrip(const float* x, int64_t n, float gain, float* out) {
  if (!x || !out) return 1;
  if (n < 0 || n % 16) return 2;
  for (int64_t b = 0; b < n; b += 16) {
    float v[16], amax = 0.0f;
    for (int i = 0; i < 16; ++i) { v[i] = x[b + i] * gain; amax = std::max(amax, std::fabs(v[i])); }
    const float scale = e4m3_round(amax / 6.0f);
    for (int i = 0; i < 16; ++i) {
      float d = 0.0f;
      if (scale > 0.0f) d = e2m1_round(std::fabs(v[i]) / scale) * scale;
      out[b + i] = std::copysign(d, x[b + i]) / gain;
    }
  }
  return 0;
}

int hif4_ref_hardware_threads(void) {
  unsigned n = std::thread::hardware_concurrency();
  return n ? static_cast<int>(n) : 1;
}

}  // extern "C"
