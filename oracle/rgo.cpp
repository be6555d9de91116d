// rgo — CPU oracle for descriptor-fixed GEMM and row reductions.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
// CUDA library is checked against.  Only tests, the smoke check and the
// benchmark's cpu_baseline / reference legs may build or call it; the product
// path never does.  It shares no code, header, table or constant generator
// with the CUDA sources.
//
// Every fp32 operation below is one IEEE-754 binary32 operation rounded to
// nearest-even (build with -O2 -ffp-contract=off, no fast-math, x86-64 SSE
// scalar arithmetic).  Citations name the paper's sections.
//
// What is defined here
//   * dependence trees over n leaves (Sec. 3.1): left fold and the balanced
//     "neighbours pair first" tree that the count-up butterfly of Sec. 5.1
//     (Fig. 3) builds;
//   * the matrix-instruction step ("atom", Sec. 3.2.1): three models,
//     EXACT_RN (the semantics the paper assumes), SEQ (scalar path, one
//     rounding per element with fma, two without) and ALIGN_TRUNC (a
//     finite-window family fitted to hardware by black-box probes; the paper
//     does not fix it: parity unpinned by the paper, pinned only by probes);
//   * plain and split-K GEMM (Sec. 3.2.2): parts from a zero accumulator,
//     atoms in ascending k, fp32 partials, merge tree, fused epilogue;
//   * row reductions: sum, RMSNorm, softmax normaliser (Sec. 5, App. F).
//
// Parity status: tree, SEQ, EXACT_RN, split/merge, epilogue, reductions are
// pinned by tests against printed examples, closed forms and brute force.
// ALIGN_TRUNC: parity unpinned (no statement in the paper fixes it).

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

// ---------------------------------------------------------------- bit helpers
inline float bits_f32(uint32_t u) { float f; std::memcpy(&f, &u, 4); return f; }
inline uint32_t f32_bits(float f) { uint32_t u; std::memcpy(&u, &f, 4); return u; }

// bf16 is the upper half of binary32: widening is exact.
inline float bf16_to_f32(uint16_t h) { return bits_f32(uint32_t(h) << 16); }

// Round-to-nearest-even narrowing binary32 -> bf16 ("where the rounding to the
// output type falls", Sec. 2 / Sec. 3.2.2: one rounding, at the very end).
inline uint16_t f32_to_bf16(float f) {
  uint32_t u = f32_bits(f);
  if ((u & 0x7fffffffu) > 0x7f800000u) return 0x7fffu;  // NaN: canonical quiet NaN
  uint32_t lsb = (u >> 16) & 1u;
  u += 0x7fffu + lsb;
  return uint16_t(u >> 16);
}

enum { DT_BF16 = 0, DT_F32 = 1, DT_F16 = 2, DT_F8E4M3 = 3 };

// IEEE binary16 (1-5-10): widening is exact.
inline float f16_to_f32(uint16_t h) {
  const uint32_t sign = uint32_t(h >> 15) << 31;
  const int e = (h >> 10) & 0x1f;
  const uint32_t m = h & 0x3ffu;
  if (e == 0x1f) return bits_f32(sign | 0x7f800000u | (m << 13));
  if (e == 0) {                                   // zero or subnormal: m * 2^-24
    const float v = float(m) * 0x1p-24f;          // exact
    return sign ? -v : v;
  }
  return bits_f32(sign | (uint32_t(e + 112) << 23) | (m << 13));
}

// Round-to-nearest-even narrowing binary32 -> binary16, subnormals kept, overflow to infinity.
inline uint16_t f32_to_f16(float f) {
  const uint32_t u = f32_bits(f);
  const uint16_t sign = uint16_t((u >> 16) & 0x8000u);
  const uint32_t a = u & 0x7fffffffu;
  if (a > 0x7f800000u) return 0x7fffu;                           // NaN: canonical quiet NaN
  if (a >= 0x47800000u) return uint16_t(sign | 0x7c00u);         // >= 65536 (or inf): infinity
  const int e = int(a >> 23) - 127;                               // unbiased exponent
  uint32_t mant = (a & 0x7fffffu) | 0x800000u;                    // 24-bit significand
  int shift;                                                      // bits dropped from the significand
  uint32_t base;
  if (e >= -14) { shift = 13; base = uint32_t(e + 15) << 10; }    // normal target
  else { shift = 13 + (-14 - e); base = 0; }                      // subnormal target
  if (a == 0) return sign;
  if (shift > 25) return sign;                                    // below half the smallest subnormal
  const uint32_t kept = mant >> shift;
  const uint32_t rem = mant & ((1u << shift) - 1u);
  const uint32_t half = 1u << (shift - 1);
  uint32_t r = (e >= -14) ? (base + (kept & 0x3ffu)) : kept;      // hidden bit folded into the exponent field
  if (rem > half || (rem == half && (r & 1u))) r += 1;            // a carry walks into the exponent: still correct
  return uint16_t(sign | r);                                      // 0x7c00 when it rounds up to infinity
}

// 8-bit float 1-4-3, bias 7, no infinities, NaN = S.1111.111, largest finite 448 (the e4m3 input
// type of Sec. 2's fp8 GEMMs).  Operands travel in 16-bit containers (value in the low byte).
inline float f8e4m3_to_f32(uint16_t h) {
  const int neg = (h >> 7) & 1;
  const int e = (h >> 3) & 0xf;
  const int m = h & 7;
  float v;
  if (e == 0xf && m == 7) v = std::numeric_limits<float>::quiet_NaN();
  else if (e == 0) v = std::ldexp(float(m), -9);          // zero or subnormal: m * 2^-9
  else v = std::ldexp(float(8 + m), e - 10);              // 1.m * 2^(e-7)
  return neg ? -v : v;
}

inline float in_to_f32(uint16_t h, int dtype) {
  return dtype == DT_F16 ? f16_to_f32(h) : dtype == DT_F8E4M3 ? f8e4m3_to_f32(h) : bf16_to_f32(h);
}

inline float load_elem(const void* p, int dtype, int64_t idx) {
  if (dtype == DT_BF16) return bf16_to_f32(static_cast<const uint16_t*>(p)[idx]);
  if (dtype == DT_F16) return f16_to_f32(static_cast<const uint16_t*>(p)[idx]);
  return static_cast<const float*>(p)[idx];
}
inline void store_elem(void* p, int dtype, int64_t idx, float v) {
  if (dtype == DT_BF16) static_cast<uint16_t*>(p)[idx] = f32_to_bf16(v);
  else if (dtype == DT_F16) static_cast<uint16_t*>(p)[idx] = f32_to_f16(v);
  else static_cast<float*>(p)[idx] = v;
}

// ------------------------------------------------------------------ the trees
// Sec. 3.1: a reduction order is a binary tree over the leaves, up to swapping
// an addition's two inputs.
//
// TREE_LEFT: ((v0 + v1) + v2) + ...  (the chain of length n-1).
// TREE_BALANCED: level by level, v'[t] = v[2t] + v[2t+1]; an unpaired last
// value moves up unchanged.  This is the tree a count-up butterfly (offsets
// 1, 2, 4, ...; Sec. 5.1, Fig. 3) builds over the logical element order; its
// height is ceil(log2 n).  The leaf order is the logical index, never a
// thread id.
enum { TREE_LEFT = 0, TREE_BALANCED = 1 };

float tree_reduce(std::vector<float>& v, int tree) {
  size_t n = v.size();
  if (n == 0) return 0.0f;
  if (tree == TREE_LEFT) {
    float acc = v[0];
    for (size_t t = 1; t < n; ++t) acc = acc + v[t];
    return acc;
  }
  while (n > 1) {
    size_t m = 0;
    for (size_t t = 0; 2 * t + 1 < n; ++t) v[m++] = v[2 * t] + v[2 * t + 1];
    if (n & 1) v[m++] = v[n - 1];
    n = m;
  }
  return v[0];
}

// The same trees with the running sum kept at `merge_dtype` (Sec. 3.2.2, split-K: "a finished part
// is written at one type and the running sum kept at another"): every add is an fp32 add whose
// result is then rounded to the merge type (for bf16 operands this equals the correctly rounded
// bf16 sum: the fp32 add is exact or its error lies far below half a bf16 ulp).
inline float round_to(float v, int dtype) {
  return dtype == DT_BF16 ? bf16_to_f32(f32_to_bf16(v)) : dtype == DT_F16 ? f16_to_f32(f32_to_f16(v)) : v;
}

float tree_reduce_at(std::vector<float>& v, int tree, int merge_dtype) {
  if (merge_dtype == DT_F32) return tree_reduce(v, tree);
  size_t n = v.size();
  if (n == 0) return 0.0f;
  if (tree == TREE_LEFT) {
    float acc = v[0];
    for (size_t t = 1; t < n; ++t) acc = round_to(acc + v[t], merge_dtype);
    return acc;
  }
  while (n > 1) {
    size_t m = 0;
    for (size_t t = 0; 2 * t + 1 < n; ++t) v[m++] = round_to(v[2 * t] + v[2 * t + 1], merge_dtype);
    if (n & 1) v[m++] = v[n - 1];
    n = m;
  }
  return v[0];
}

// --------------------------------------------------- exact long accumulator
// Fixed-point accumulator wide enough for any sum of bf16*bf16 products and
// binary32 values: bit i of the accumulator has weight 2^(i - BIAS).
struct LongAcc {
  static constexpr int LIMBS = 32;        // 32 * 32 = 1024 bits
  static constexpr int BIAS = 512;        // weights 2^-512 .. 2^511
  int64_t limb[LIMBS];                    // each holds a signed multiple of 2^(32*i)
  LongAcc() { std::memset(limb, 0, sizeof(limb)); }

  // add sign * mag * 2^exp, mag < 2^64
  void add(int sign, uint64_t mag, int exp) {
    if (mag == 0) return;
    int pos = exp + BIAS;                 // bit position of mag's bit 0
    // callers guarantee 0 <= pos and pos + 64 < LIMBS*32
    int li = pos >> 5, sh = pos & 31;
    unsigned __int128 w = (unsigned __int128)mag << sh;   // < 2^95
    for (int t = 0; t < 3; ++t) {
      int64_t piece = int64_t(uint32_t(w));
      limb[li + t] += sign < 0 ? -piece : piece;
      w >>= 32;
    }
  }
  void add_f32(float f) {
    uint32_t u = f32_bits(f);
    int e = int((u >> 23) & 0xff);
    uint32_t m = u & 0x7fffffu;
    int sign = (u >> 31) ? -1 : 1;
    if (e == 0) add(sign, m, -149);
    else add(sign, m | 0x800000u, e - 150);
  }
  // Canonical form: returns sign (-1, 0, +1) and fills mag[] with the
  // magnitude's 32-bit limbs.
  int canonical(uint32_t* mag) const {
    int64_t c[LIMBS + 1];
    int64_t carry = 0;
    for (int i = 0; i < LIMBS; ++i) {
      int64_t t = limb[i] + carry;
      int64_t lo = t & 0xffffffffLL;      // t mod 2^32, in [0, 2^32)
      carry = (t - lo) >> 32;             // exact arithmetic shift
      c[i] = lo;
    }
    c[LIMBS] = carry;                     // -1, 0 (or small positive, never here)
    int sign = 0;
    if (carry < 0) {
      sign = -1;                          // negate (two's complement over LIMBS limbs)
      int64_t b = 1;
      for (int i = 0; i < LIMBS; ++i) {
        int64_t t = (0xffffffffLL - c[i]) + b;
        mag[i] = uint32_t(t & 0xffffffffLL);
        b = t >> 32;
      }
    } else {
      for (int i = 0; i < LIMBS; ++i) { mag[i] = uint32_t(c[i]); if (c[i]) sign = 1; }
    }
    return sign;
  }
};

enum { ROUND_RZ = 0, ROUND_RN = 1 };

// Round the exact value sign * (mag limbs) * 2^-BIAS to binary32.
// `zero_result` is returned when the value is exactly zero.
float round_limbs_to_f32(int sign, const uint32_t* mag, int nl, int bias, int mode, float zero_result) {
  int top = -1;
  for (int i = nl - 1; i >= 0 && top < 0; --i)
    if (mag[i]) top = i * 32 + (31 - __builtin_clz(mag[i]));
  if (top < 0) return zero_result;
  auto bit = [&](int p) -> uint32_t { return p < 0 ? 0u : (mag[p >> 5] >> (p & 31)) & 1u; };
  int e = top - bias;                     // value in [2^e, 2^(e+1))
  // lsb position of the 24-bit significand (subnormals: fixed at 2^-149)
  int lsb_e = std::max(e - 23, -149);
  int lsb_p = lsb_e + bias;               // bit position of the result's lsb
  uint64_t sig = 0;
  for (int p = top; p >= lsb_p; --p) sig = (sig << 1) | bit(p);
  uint32_t guard = bit(lsb_p - 1);
  bool sticky = false;
  for (int p = lsb_p - 2; p >= 0 && !sticky; --p) {
    // skip whole zero limbs quickly
    if ((p & 31) == 31 && mag[p >> 5] == 0) { p -= 31; continue; }
    if (bit(p)) sticky = true;
  }
  if (mode == ROUND_RN && guard && (sticky || (sig & 1))) sig += 1;
  // sig * 2^lsb_e, sig <= 2^24
  double d = std::ldexp(double(sig), lsb_e);          // exact in double
  float r = d >= 0x1p128 ? (mode == ROUND_RN ? INFINITY : 0x1.fffffep127f) : float(d);  // float(d) exact here
  return sign < 0 ? -r : r;
}

float round_longacc(const LongAcc& L, int mode, float zero_result) {
  uint32_t mag[LongAcc::LIMBS];
  int sign = L.canonical(mag);
  if (sign == 0) return zero_result;
  return round_limbs_to_f32(sign, mag, LongAcc::LIMBS, LongAcc::BIAS, mode, zero_result);
}

// ------------------------------------------------------------------ the atom
// Sec. 3.2.1: one matrix instruction folds instruction_k products and the
// incoming accumulator.
struct AtomModel {
  int32_t model;          // 0 EXACT_RN, 1 SEQ, 2 ALIGN_TRUNC
  int32_t atom_k;         // instruction_k (16 for a 16-bit tensor-core step, App. E)
  int32_t fma;            // SEQ: 1 = fused multiply-add, 0 = multiply then add
  // ALIGN_TRUNC parameters (fitted by probes, not stated by the paper)
  int32_t group;          // products folded per internal step (divides atom_k)
  int32_t window_bits;    // F: bits kept below the largest exponent present
  int32_t exp_mode;       // 0: exponent of the normalised product; 1: Ea + Eb
  int32_t acc_in_window;  // 1: the accumulator is aligned/truncated like a product
  int32_t addend_round;   // 0: truncate toward zero; 1: floor (toward -inf)
  int32_t final_round;    // 0: RZ; 1: RN-even
  int32_t in_dtype;       // operand type of the products: DT_BF16, DT_F16 or DT_F8E4M3
};
enum { ATOM_EXACT_RN = 0, ATOM_SEQ = 1, ATOM_ALIGN_TRUNC = 2 };

struct Prod { int sign; uint32_t mag; int exp; int e_op; };  // value = sign*mag*2^exp ; e_op = Ea+Eb

inline void bf16_decode(uint16_t h, int& sign, uint32_t& mag, int& exp, int& e_lead) {
  sign = (h >> 15) ? -1 : 1;
  int e = (h >> 7) & 0xff;
  uint32_t m = h & 0x7f;
  if (e == 0) { mag = m; exp = -133; e_lead = -126; }       // subnormal: leading exponent fixed
  else { mag = m | 0x80; exp = e - 134; e_lead = e - 127; }
}
inline bool bf16_finite(uint16_t h) { return ((h >> 7) & 0xff) != 0xff; }
inline void f16_decode(uint16_t h, int& sign, uint32_t& mag, int& exp, int& e_lead) {
  sign = (h >> 15) ? -1 : 1;
  int e = (h >> 10) & 0x1f;
  uint32_t m = h & 0x3ff;
  if (e == 0) { mag = m; exp = -24; e_lead = -14; }
  else { mag = m | 0x400; exp = e - 25; e_lead = e - 15; }
}
inline bool f16_finite(uint16_t h) { return ((h >> 10) & 0x1f) != 0x1f; }
inline void f8e4m3_decode(uint16_t h, int& sign, uint32_t& mag, int& exp, int& e_lead) {
  sign = ((h >> 7) & 1) ? -1 : 1;
  int e = (h >> 3) & 0xf;
  uint32_t m = h & 7;
  if (e == 0) { mag = m; exp = -9; e_lead = -6; }
  else { mag = m | 8; exp = e - 10; e_lead = e - 7; }
}
inline bool f8e4m3_finite(uint16_t h) { return (h & 0x7f) != 0x7f; }
inline bool in_finite(uint16_t h, int dtype) {
  return dtype == DT_F16 ? f16_finite(h) : dtype == DT_F8E4M3 ? f8e4m3_finite(h) : bf16_finite(h);
}

inline Prod make_prod(uint16_t a, uint16_t b, int dtype) {
  int sa, sb, ea, eb, la, lb; uint32_t ma, mb;
  if (dtype == DT_F16) { f16_decode(a, sa, ma, ea, la); f16_decode(b, sb, mb, eb, lb); }
  else if (dtype == DT_F8E4M3) { f8e4m3_decode(a, sa, ma, ea, la); f8e4m3_decode(b, sb, mb, eb, lb); }
  else { bf16_decode(a, sa, ma, ea, la); bf16_decode(b, sb, mb, eb, lb); }
  Prod p; p.sign = sa * sb; p.mag = ma * mb; p.exp = ea + eb; p.e_op = la + lb;
  return p;
}

inline int ilog2_u64(uint64_t v) { return 63 - __builtin_clzll(v); }

float atom_seq(float acc, const uint16_t* a, const uint16_t* b, int n, int fma, int dtype) {
  // Sec. 3.2.1, scalar path: acc <- fma(a, b, acc), or two roundings unfused.
  for (int u = 0; u < n; ++u) {
    float x = in_to_f32(a[u], dtype), y = in_to_f32(b[u], dtype);
    if (fma) acc = std::fmaf(x, y, acc);
    else { float p = x * y; acc = acc + p; }
  }
  return acc;
}

float atom_exact_rn(float acc, const uint16_t* a, const uint16_t* b, int n, int dtype) {
  // Sec. 3.2.1: acc <- RN_fp32(acc + sum_j a_j*b_j), the sum formed exactly.
  LongAcc L;
  L.add_f32(acc);
  for (int u = 0; u < n; ++u) {
    Prod p = make_prod(a[u], b[u], dtype);
    L.add(p.sign, p.mag, p.exp);
  }
  // An exactly-zero sum: IEEE gives +0 under RN unless every addend is -0.
  bool all_neg_zero = (f32_bits(acc) == 0x80000000u);
  for (int u = 0; u < n && all_neg_zero; ++u) {
    Prod p = make_prod(a[u], b[u], dtype);
    if (!(p.mag == 0 && p.sign < 0)) all_neg_zero = false;
  }
  return round_longacc(L, ROUND_RN, all_neg_zero ? -0.0f : 0.0f);
}

// One internal step of the finite-window family: align every addend to the
// largest exponent present, keep window_bits below it, add exactly, round once.
float align_trunc_step(float acc, const uint16_t* a, const uint16_t* b, int n, const AtomModel& m) {
  Prod p[64];
  int emax = INT32_MIN;
  for (int u = 0; u < n; ++u) {
    p[u] = make_prod(a[u], b[u], m.in_dtype);
    if (p[u].mag) {
      int e = m.exp_mode ? p[u].e_op : (p[u].exp + ilog2_u64(p[u].mag));
      emax = std::max(emax, e);
    }
  }
  uint32_t ub = f32_bits(acc);
  int asign = (ub >> 31) ? -1 : 1;
  int ae = int((ub >> 23) & 0xff);
  uint32_t amag = ae ? ((ub & 0x7fffffu) | 0x800000u) : (ub & 0x7fffffu);
  int aexp = ae ? ae - 150 : -149;
  if (m.acc_in_window && amag) emax = std::max(emax, aexp + ilog2_u64(amag));
  if (emax == INT32_MIN) return acc;                 // nothing but zeros
  int q = emax - std::min(m.window_bits, 90);        // weight of the window's last bit
  auto align = [&](int sign, uint64_t mag, int exp) -> __int128 {
    if (!mag) return 0;
    int sh = exp - q;                                // <= window_bits, so no overflow below
    __int128 t;
    bool lost = false;
    if (sh >= 0) t = (__int128)mag << sh;
    else if (-sh >= 64) { t = 0; lost = true; }
    else { t = (__int128)(mag >> (-sh)); lost = (mag & ((uint64_t(1) << (-sh)) - 1)) != 0; }
    if (lost && m.addend_round == 1 && sign < 0) t += 1;   // floor of a negative value
    return sign < 0 ? -t : t;
  };
  __int128 S = 0;
  for (int u = 0; u < n; ++u) S += align(p[u].sign, p[u].mag, p[u].exp);
  LongAcc L;
  if (m.acc_in_window) S += align(asign, amag, aexp);
  else L.add_f32(acc);
  int ssign = S < 0 ? -1 : 1;
  unsigned __int128 SM = S < 0 ? (unsigned __int128)(-S) : (unsigned __int128)S;
  L.add(ssign, uint64_t(SM), q);
  L.add(ssign, uint64_t(SM >> 64), q + 64);
  return round_longacc(L, m.final_round, 0.0f);
}

float atom_step(float acc, const uint16_t* a, const uint16_t* b, int n, const AtomModel& m) {
  for (int u = 0; u < n; ++u)
    if (!in_finite(a[u], m.in_dtype) || !in_finite(b[u], m.in_dtype)) return atom_seq(acc, a, b, n, 1, m.in_dtype);
  if (!std::isfinite(acc)) return atom_seq(acc, a, b, n, 1, m.in_dtype);
  switch (m.model) {
    case ATOM_SEQ: return atom_seq(acc, a, b, n, m.fma, m.in_dtype);
    case ATOM_EXACT_RN: return atom_exact_rn(acc, a, b, n, m.in_dtype);
    default: {
      int g = m.group > 0 ? m.group : n;
      for (int u0 = 0; u0 < n; u0 += g) acc = align_trunc_step(acc, a + u0, b + u0, std::min(g, n - u0), m);
      return acc;
    }
  }
}

// ---------------------------------------------------------------- rg_expf
// The paper leaves the exponential to "the hardware's base-two exponential"
// (App. F), which no CPU reproduces.  This library instead fixes exp() as a
// sequence of IEEE operations so both sides agree bit for bit:
//   n = rint(x * log2(e));  r = x - n*ln2 (two-term Cody-Waite, fused);
//   p = degree-7 Taylor polynomial in r (Horner, fused);  result = p * 2^n,
//   the scaling split in two exact power-of-two factors.
float rg_expf(float x) {
  if (x != x) return x;
  if (x > 88.72284f) return INFINITY;
  if (x < -87.33655f) return 0.0f;
  float n = std::nearbyintf(x * 0x1.715476p+0f);
  float r = std::fmaf(n, -0x1.62e400p-1f, x);
  r = std::fmaf(n, -0x1.7f7d1cp-20f, r);
  float p = 0x1.a01a02p-13f;              // 1/5040
  p = std::fmaf(p, r, 0x1.6c16c2p-10f);   // 1/720
  p = std::fmaf(p, r, 0x1.111112p-7f);    // 1/120
  p = std::fmaf(p, r, 0x1.555556p-5f);    // 1/24
  p = std::fmaf(p, r, 0x1.555556p-3f);    // 1/6
  p = std::fmaf(p, r, 0.5f);
  p = std::fmaf(p, r, 1.0f);
  p = std::fmaf(p, r, 1.0f);
  int ni = int(n);
  int h = ni >> 1;                        // floor(n/2)
  float s1 = bits_f32(uint32_t(ni - h + 127) << 23);
  float s2 = bits_f32(uint32_t(h + 127) << 23);
  return (p * s1) * s2;
}

// Base-two exponential, fixed the same way (App. F: attention kernels fold log2 e into the score
// scale and take a base-two exponential): n = rint(x); f = x - n (exact, |f| <= 1/2);
// p = degree-7 Taylor polynomial of 2^f = exp(f ln 2) (Horner, fused); result = p * 2^n, an exact
// scaling.  2^x for x < -126 is 0 and for x >= 128 is +inf; integers give exact powers of two.
float rg_exp2f(float x) {
  if (x != x) return x;
  if (x >= 128.0f) return INFINITY;
  if (x < -126.0f) return 0.0f;
  float n = std::nearbyintf(x);
  float f = x - n;
  float p = 0x1.ffcbfcp-17f;              // (ln 2)^7 / 5040
  p = std::fmaf(p, f, 0x1.430912p-13f);   // (ln 2)^6 / 720
  p = std::fmaf(p, f, 0x1.5d87fep-10f);   // (ln 2)^5 / 120
  p = std::fmaf(p, f, 0x1.3b2ab6p-7f);    // (ln 2)^4 / 24
  p = std::fmaf(p, f, 0x1.c6b08ep-5f);    // (ln 2)^3 / 6
  p = std::fmaf(p, f, 0x1.ebfbe0p-3f);    // (ln 2)^2 / 2
  p = std::fmaf(p, f, 0x1.62e430p-1f);    // ln 2
  p = std::fmaf(p, f, 1.0f);
  return std::ldexp(p, int(n));           // exact: p in [0.70, 1.42], the result is a normal number
}

inline float silu(float v) { return v / (1.0f + rg_expf(-v)); }

// ------------------------------------------------------------------- GEMM
struct GemmDesc {
  AtomModel atom;
  int32_t tree;            // merge tree over the split-K partials
  int32_t n_cuts;          // interior cut points, strictly increasing, 0 < c < K
  const int64_t* cuts;
  // epilogue (fixed order: bias, activation, residual, one rounding)
  const void* bias; int32_t bias_dtype;
  int32_t act;             // 0 none, 1 SiLU
  const void* residual; int32_t residual_dtype; int64_t ldr;
  int32_t out_dtype;
  int32_t partial_dtype;   // type a finished part is written at (fp32 or bf16)
  int32_t merge_dtype;     // type the running sum of the parts is kept at
  int64_t inner_span;      // second level of the cut nest: 0 = none, else an accumulator is closed every inner_span k
};

// One output element, Sec. 3.2.2.  `partials_out` (nullable) receives the
// fp32 partial of each part.
float gemm_element(const GemmDesc& d, const uint16_t* arow, const uint16_t* brow, int64_t K,
                   int64_t i, int64_t j, float* partials_out) {
  int S = d.n_cuts + 1;
  std::vector<float> part(S);
  for (int s = 0; s < S; ++s) {
    int64_t k_lo = s == 0 ? 0 : d.cuts[s - 1];
    int64_t k_hi = s == S - 1 ? K : d.cuts[s];
    int ak = d.atom.model == ATOM_SEQ ? 1 : d.atom.atom_k;
    // Sec. 3.2.2: "some kernels cut again inside a part, closing an accumulator every so many
    // elements before the part is finished".  Each group of inner_span k runs its own chain from a
    // zero accumulator; the closed groups are added at fp32, in ascending order, into the part's
    // running sum (the first group starts it): one extra rounding per group (App. E, per-group
    // accumulation).
    const int64_t span = d.inner_span > 0 ? d.inner_span : (k_hi - k_lo);
    float acc = 0.0f;
    bool first_group = true;
    for (int64_t g_lo = k_lo; g_lo < k_hi; g_lo += span) {
      const int64_t g_hi = std::min(k_hi, g_lo + span);
      float gacc = 0.0f;                                // every group starts from zero
      for (int64_t k0 = g_lo; k0 < g_hi; k0 += ak) {    // ascending k, atoms relative to the group
        int n = int(std::min<int64_t>(ak, g_hi - k0));
        gacc = atom_step(gacc, arow + k0, brow + k0, n, d.atom);
      }
      acc = first_group ? gacc : acc + gacc;
      first_group = false;
    }
    // a finished part is written at partial_dtype only when the axis is split (Sec. 3.2.2, split-K:
    // "a finished part is written at one type"); a plain GEMM writes no part and keeps fp32
    part[s] = S > 1 ? round_to(acc, d.partial_dtype) : acc;
    if (partials_out) partials_out[s] = part[s];
  }
  float v = tree_reduce_at(part, d.tree, d.merge_dtype);  // merge in tree order, sum kept at merge_dtype
  if (d.bias) v = v + load_elem(d.bias, d.bias_dtype, j);
  if (d.act == 1) v = silu(v);
  if (d.residual) v = v + load_elem(d.residual, d.residual_dtype, i * d.ldr + j);
  return v;
}

}  // namespace

// =============================================================== C interface
extern "C" {

int rgo_num_threads() {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

float rgo_bf16_to_f32(uint16_t h) { return bf16_to_f32(h); }
uint16_t rgo_f32_to_bf16(float f) { return f32_to_bf16(f); }
float rgo_f16_to_f32(uint16_t h) { return f16_to_f32(h); }
float rgo_f8e4m3_to_f32(uint8_t h) { return f8e4m3_to_f32(h); }
uint16_t rgo_f32_to_f16(float f) { return f32_to_f16(f); }
float rgo_add_f32(float a, float b) { return a + b; }
float rgo_mul_f32(float a, float b) { return a * b; }
float rgo_expf(float x) { return rg_expf(x); }
float rgo_exp2f(float x) { return rg_exp2f(x); }
float rgo_silu(float x) { return silu(x); }
// the same two functions over an array (a loop around the scalar definitions, for the tests' sake)
void rgo_exp_array(const float* x, float* y, int64_t n, int base2) {
  for (int64_t i = 0; i < n; ++i) y[i] = base2 ? rg_exp2f(x[i]) : rg_expf(x[i]);
}
void rgo_silu_array(const float* x, float* y, int64_t n) {
  for (int64_t i = 0; i < n; ++i) y[i] = silu(x[i]);
}

// Tree-reduce n fp32 values (input is not modified).
float rgo_tree_sum(const float* v, int64_t n, int tree) {
  std::vector<float> w(v, v + n);
  return tree_reduce(w, tree);
}

// One atom step on n (<= 64) products.
float rgo_atom(const AtomModel* m, float acc, const uint16_t* a, const uint16_t* b, int n) {
  return atom_step(acc, a, b, n, *m);
}

// C[i,j] = epilogue(merge(parts of sum_k A[i,k]*B[j,k])) for all i<M, j<N.
// A is [M,K] bf16 row-major (lda), B is [N,K] bf16 row-major (ldb): C = A * B^T.
void rgo_gemm(const AtomModel* atom, int tree, int n_cuts, const int64_t* cuts,
              int64_t M, int64_t N, int64_t K,
              const uint16_t* A, int64_t lda, const uint16_t* B, int64_t ldb,
              void* C, int out_dtype, int64_t ldc,
              const void* bias, int bias_dtype, int act,
              const void* residual, int residual_dtype, int64_t ldr, int partial_dtype, int merge_dtype, int64_t inner_span) {
  GemmDesc d{*atom, tree, n_cuts, cuts, bias, bias_dtype, act, residual, residual_dtype, ldr, out_dtype, partial_dtype, merge_dtype, inner_span};
#pragma omp parallel for collapse(2) schedule(static)
  for (int64_t i = 0; i < M; ++i)
    for (int64_t j = 0; j < N; ++j) {
      float v = gemm_element(d, A + i * lda, B + j * ldb, K, i, j, nullptr);
      store_elem(C, out_dtype, i * ldc + j, v);
    }
}

// Same, for a list of (i, j) samples; out[t] is fp32 holding the value after
// the output rounding (a bf16 result is widened exactly).
void rgo_gemm_samples(const AtomModel* atom, int tree, int n_cuts, const int64_t* cuts,
                      int64_t K, const uint16_t* A, int64_t lda, const uint16_t* B, int64_t ldb,
                      int out_dtype,
                      const void* bias, int bias_dtype, int act,
                      const void* residual, int residual_dtype, int64_t ldr,
                      int64_t n_samples, const int64_t* si, const int64_t* sj, float* out,
                      int partial_dtype, int merge_dtype, int64_t inner_span) {
  GemmDesc d{*atom, tree, n_cuts, cuts, bias, bias_dtype, act, residual, residual_dtype, ldr, out_dtype, partial_dtype, merge_dtype, inner_span};
#pragma omp parallel for schedule(static)
  for (int64_t t = 0; t < n_samples; ++t) {
    float v = gemm_element(d, A + si[t] * lda, B + sj[t] * ldb, K, si[t], sj[t], nullptr);
    out[t] = round_to(v, out_dtype);
  }
}

// Partials of every part, [S][M][N], before the merge (fp32 holding the value at partial_dtype).
void rgo_gemm_partials(const AtomModel* atom, int n_cuts, const int64_t* cuts,
                       int64_t M, int64_t N, int64_t K,
                       const uint16_t* A, int64_t lda, const uint16_t* B, int64_t ldb, float* P, int partial_dtype, int64_t inner_span) {
  GemmDesc d{*atom, TREE_LEFT, n_cuts, cuts, nullptr, 0, 0, nullptr, 0, 0, DT_F32, partial_dtype, DT_F32, inner_span};
  int S = n_cuts + 1;
#pragma omp parallel for collapse(2) schedule(static)
  for (int64_t i = 0; i < M; ++i)
    for (int64_t j = 0; j < N; ++j) {
      std::vector<float> part(S);
      gemm_element(d, A + i * lda, B + j * ldb, K, i, j, part.data());
      for (int s = 0; s < S; ++s) P[(int64_t(s) * M + i) * N + j] = part[s];
    }
}

// GEMV family (Sec. 3.2.2 "GEMV"): no matrix instruction; `lanes` lanes share one output element.
// Each lane owns tiles of `tile` consecutive k and folds its elements in ascending k into one
// accumulator with a scalar multiply-add (Sec. 3.2.1: one rounding per element with fma, two
// without).  layout 0 (strided): lane l takes tiles l, l+lanes, l+2*lanes, ...; layout 1
// (contiguous): lane l takes the l-th run of ceil(tiles/lanes) consecutive tiles.  The lane totals are
// then folded by a butterfly: fold 0 counts the offsets up (1, 2, 4, ...), a balanced tree over the
// lanes in index order; fold 1 counts them down (lanes/2, ..., 1), a balanced tree over the lanes
// in bit-reversed order.  Then the same epilogue as the GEMM.
void rgo_gemv(int in_dtype, int fma, int lanes, int tile, int layout, int fold,
              int64_t M, int64_t N, int64_t K,
              const uint16_t* A, int64_t lda, const uint16_t* B, int64_t ldb,
              void* C, int out_dtype, int64_t ldc,
              const void* bias, int bias_dtype, int act,
              const void* residual, int residual_dtype, int64_t ldr) {
  const int64_t tiles = (K + tile - 1) / tile;
  const int64_t run = (tiles + lanes - 1) / lanes;
  int bits = 0;
  while ((1 << bits) < lanes) ++bits;
#pragma omp parallel for collapse(2) schedule(static)
  for (int64_t i = 0; i < M; ++i)
    for (int64_t j = 0; j < N; ++j) {
      const uint16_t* a = A + i * lda;
      const uint16_t* b = B + j * ldb;
      std::vector<float> tot(lanes);
      for (int l = 0; l < lanes; ++l) {
        float acc = 0.0f;
        for (int64_t t = 0; t < tiles; ++t) {
          const bool mine = layout == 0 ? (t % lanes == l) : (t / run == l);
          if (!mine) continue;
          for (int64_t k = t * tile; k < std::min<int64_t>(K, (t + 1) * tile); ++k) {
            const float x = in_to_f32(a[k], in_dtype), y = in_to_f32(b[k], in_dtype);
            if (fma) acc = std::fmaf(x, y, acc);
            else { const float p = x * y; acc = acc + p; }
          }
        }
        tot[l] = acc;
      }
      std::vector<float> order(lanes);
      for (int l = 0; l < lanes; ++l) {
        int src = l;
        if (fold == 1) {                                  // bit-reversed lane order
          src = 0;
          for (int q = 0; q < bits; ++q) src |= ((l >> q) & 1) << (bits - 1 - q);
        }
        order[l] = tot[src];
      }
      float v = tree_reduce(order, TREE_BALANCED);
      if (bias) v = v + load_elem(bias, bias_dtype, j);
      if (act == 1) v = silu(v);
      if (residual) v = v + load_elem(residual, residual_dtype, i * ldr + j);
      store_elem(C, out_dtype, i * ldc + j, v);
    }
}

// Row reductions.  op: 0 sum, 1 RMSNorm, 2 softmax normaliser.
//   sum:      out[r] = TREE(f32(x[r,:]))                                    (fp32 out)
//   rmsnorm:  ss = TREE(x*x) (fma=1: level-0 nodes are fma(x1,x1,x0*x0));
//             rinv = 1 / sqrt(ss / C + eps);  y = RN_out((x*rinv)*w)         ([R,C] out)
//   softmax:  m = max x;  out[r] = TREE(rg_expf(x - m));  aux[r] = m        (fp32 out)
void rgo_reduce_rows(int op, int tree, int fma, const void* x, int x_dtype,
                     int64_t R, int64_t C, int64_t ldx,
                     void* out, int out_dtype, int64_t ldo,
                     const void* weight, int w_dtype, float eps, float* aux) {
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < R; ++r) {
    std::vector<float> leaf;
    if (op == 0) {
      leaf.resize(C);
      for (int64_t c = 0; c < C; ++c) leaf[c] = load_elem(x, x_dtype, r * ldx + c);
      static_cast<float*>(out)[r * ldo] = tree_reduce(leaf, tree);
    } else if (op == 1) {
      if (fma && tree == TREE_BALANCED) {
        // the multiply of the second leaf of each level-0 pair fuses into the add
        leaf.resize((C + 1) / 2);
        for (int64_t t = 0; 2 * t < C; ++t) {
          float x0 = load_elem(x, x_dtype, r * ldx + 2 * t);
          float s = x0 * x0;
          if (2 * t + 1 < C) {
            float x1 = load_elem(x, x_dtype, r * ldx + 2 * t + 1);
            s = std::fmaf(x1, x1, s);
          }
          leaf[t] = s;
        }
      } else if (fma) {  // left fold: every step after the first is an fma
        float x0 = load_elem(x, x_dtype, r * ldx);
        float acc = x0 * x0;
        for (int64_t c = 1; c < C; ++c) {
          float xc = load_elem(x, x_dtype, r * ldx + c);
          acc = std::fmaf(xc, xc, acc);
        }
        leaf.assign(1, acc);
      } else {
        leaf.resize(C);
        for (int64_t c = 0; c < C; ++c) {
          float xc = load_elem(x, x_dtype, r * ldx + c);
          leaf[c] = xc * xc;
        }
      }
      float ss = tree_reduce(leaf, tree);
      float ms = ss / float(C);
      float rinv = 1.0f / std::sqrt(ms + eps);
      if (aux) aux[r] = rinv;
      for (int64_t c = 0; c < C; ++c) {
        float xc = load_elem(x, x_dtype, r * ldx + c);
        float wc = weight ? load_elem(weight, w_dtype, c) : 1.0f;
        float y = (xc * rinv) * wc;
        store_elem(out, out_dtype, r * ldo + c, y);
      }
    } else {
      float m = load_elem(x, x_dtype, r * ldx);
      for (int64_t c = 1; c < C; ++c) m = std::max(m, load_elem(x, x_dtype, r * ldx + c));
      leaf.resize(C);
      for (int64_t c = 0; c < C; ++c) leaf[c] = rg_expf(load_elem(x, x_dtype, r * ldx + c) - m);
      static_cast<float*>(out)[r * ldo] = tree_reduce(leaf, tree);
      if (aux) aux[r] = m;
    }
  }
}

// Reductions along the other axis (Sec. 6: "reductions on different dims/axes"; the column sum a
// matrix-multiply epilogue emits; the LayerNorm weight-gradient reduction): out[c] = TREE over the
// rows r = 0..R-1, in index order, of the leaf
//   op 0 (sum):  x[r][c]
//   op 1 (dot):  x[r][c] * y[r][c]   (one rounding per product; with fma and the balanced tree the
//                second product of each level-0 pair is fused into that pair's add, as for RMSNorm)
// The tree is the same "neighbours pair first" tree as along rows (Sec. 5.1).
void rgo_reduce_cols(int op, int tree, int fma, const void* x, int x_dtype, const void* y, int y_dtype,
                     int64_t R, int64_t C, int64_t ldx, int64_t ldy, float* out) {
#pragma omp parallel for schedule(static)
  for (int64_t c = 0; c < C; ++c) {
    std::vector<float> leaf;
    if (op == 0) {
      leaf.resize(R);
      for (int64_t r = 0; r < R; ++r) leaf[r] = load_elem(x, x_dtype, r * ldx + c);
    } else if (fma && tree == TREE_BALANCED) {
      leaf.resize((R + 1) / 2);
      for (int64_t t = 0; 2 * t < R; ++t) {
        float s = load_elem(x, x_dtype, 2 * t * ldx + c) * load_elem(y, y_dtype, 2 * t * ldy + c);
        if (2 * t + 1 < R) s = std::fmaf(load_elem(x, x_dtype, (2 * t + 1) * ldx + c), load_elem(y, y_dtype, (2 * t + 1) * ldy + c), s);
        leaf[t] = s;
      }
    } else if (fma) {
      float acc = load_elem(x, x_dtype, c) * load_elem(y, y_dtype, c);
      for (int64_t r = 1; r < R; ++r) acc = std::fmaf(load_elem(x, x_dtype, r * ldx + c), load_elem(y, y_dtype, r * ldy + c), acc);
      leaf.assign(1, acc);
    } else {
      leaf.resize(R);
      for (int64_t r = 0; r < R; ++r) leaf[r] = load_elem(x, x_dtype, r * ldx + c) * load_elem(y, y_dtype, r * ldy + c);
    }
    out[c] = tree_reduce(leaf, tree);
  }
}

// Attention with a fixed descriptor (App. F): one query row, keys cut into blocks of width w.
// Per block j, with everything below in binary32 unless noted:
//   s_t   = scale * (q . k_t)         the contraction is a chain of tensor-core steps over the head
//                                     dimension from a zero accumulator (Sec. 3.2.1), then one multiply
//   m_j   = max(m_{j-1}, max_t s_t)   a maximum rounds nothing
//   alpha = exp(m_{j-1} - m_j),  p_t = exp(s_t - m_j)          (exp as fixed by this library: base e,
//                                     or base two with log2 e folded into `scale` by the caller)
//   l_j   = alpha * l_{j-1} + TREE_t p_t                        (the block's row sum in the given tree)
//   P_t   = p_t narrowed to p_dtype                             (the operand type of the second product)
//   O_j   = alpha * O_{j-1} + (P . V)_block                     the block's product is a chain of steps
//                                                               over its keys from a zero accumulator
// and the answer is O_B / l_B, divided once at the end and rounded once to the output type.
// Keys past Nk in the last block are absent: their scores are -inf, their probabilities exactly 0.
// Causal masking (mask = 1, App. F "Masking puts the query block into the answer"): query row i sees
// keys t <= i.  The walk of a row in query tile [q0, q0 + block_m) stops at key q0 + block_m; the blocks
// from q0 on are the ones that straddle the diagonal, and there every score takes an offset before the
// maximum: 0 where t <= i, -1e6 where t > i (so those probabilities underflow to exactly 0).
// Vt is V transposed: [d, Nk], keys contiguous.
void rgo_attention(const AtomModel* atom, int block_n, int sum_tree, int p_dtype, int exp_base, int mask, int block_m, float scale,
                   int64_t Nq, int64_t Nk, int64_t d, const uint16_t* Q, int64_t ldq, const uint16_t* K, int64_t ldk,
                   const uint16_t* Vt, int64_t ldv, void* O, int o_dtype, int64_t ldo) {
  const int ak = atom->atom_k;
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < Nq; ++i) {
    const uint16_t* q = Q + i * ldq;
    float m = -INFINITY, l = 0.0f;
    std::vector<float> Oacc(d, 0.0f), s(block_n), pf(block_n);
    std::vector<uint16_t> pn(block_n);
    const int64_t tile0 = mask ? (i / block_m) * block_m : 0;
    const int64_t kend = mask ? std::min<int64_t>(Nk, tile0 + block_m) : Nk;
    for (int64_t t0 = 0; t0 < kend; t0 += block_n) {
      const int n = (int)std::min<int64_t>(block_n, kend - t0);
      const bool diagonal = mask && t0 >= tile0;
      float mb = -INFINITY;
      for (int t = 0; t < n; ++t) {
        const uint16_t* k = K + (t0 + t) * ldk;
        float acc = 0.0f;
        for (int64_t c0 = 0; c0 < d; c0 += ak) acc = atom_step(acc, q + c0, k + c0, (int)std::min<int64_t>(ak, d - c0), *atom);
        s[t] = acc * scale;
        if (diagonal) s[t] = s[t] + ((t0 + t) <= i ? 0.0f : -1.0e6f);
        mb = std::max(mb, s[t]);
      }
      const float m_new = std::max(m, mb);
      const float alpha = exp_base == 2 ? rg_exp2f(m - m_new) : rg_expf(m - m_new);
      std::vector<float> leaf(n);
      for (int t = 0; t < n; ++t) { pf[t] = exp_base == 2 ? rg_exp2f(s[t] - m_new) : rg_expf(s[t] - m_new); leaf[t] = pf[t]; }
      const float rowsum = tree_reduce(leaf, sum_tree);
      l = alpha * l + rowsum;
      for (int t = 0; t < n; ++t) pn[t] = p_dtype == DT_F16 ? f32_to_f16(pf[t]) : f32_to_bf16(pf[t]);
      AtomModel pm = *atom; pm.in_dtype = p_dtype == DT_F16 ? DT_F16 : DT_BF16;
      for (int64_t c = 0; c < d; ++c) {
        const uint16_t* v = Vt + c * ldv + t0;
        float acc = 0.0f;
        for (int u0 = 0; u0 < n; u0 += ak) acc = atom_step(acc, pn.data() + u0, v + u0, std::min(ak, n - u0), pm);
        Oacc[c] = alpha * Oacc[c] + acc;
      }
      m = m_new;
    }
    for (int64_t c = 0; c < d; ++c) store_elem(O, o_dtype, i * ldo + c, Oacc[c] / l);
  }
}

}  // extern "C"
