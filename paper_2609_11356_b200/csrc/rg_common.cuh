// Device-side scalar arithmetic shared by the GEMM epilogue, the split-K merge and the
// row reductions.  Every operation is an explicit round-to-nearest intrinsic so that the
// compiler can neither contract a multiply into an add nor reassociate: the dependence tree
// written here is the one that runs (Sec. 3.1).
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/rg.h"

namespace rg {

__device__ __forceinline__ float f_add(float a, float b) { return __fadd_rn(a, b); }
__device__ __forceinline__ float f_mul(float a, float b) { return __fmul_rn(a, b); }
__device__ __forceinline__ float f_fma(float a, float b, float c) { return __fmaf_rn(a, b, c); }

__device__ __forceinline__ float bf16_bits_to_f32(uint32_t h) { return __uint_as_float(h << 16); }

// Exponential fixed as a sequence of IEEE operations (the paper's kernels use the hardware's
// base-two exponential, App. F, which is not reproducible off the GPU): n = rint(x*log2 e),
// two-term Cody-Waite reduction with fused multiply-adds, degree-7 Taylor polynomial in
// Horner form, and an exact two-factor scaling by 2^n.
__device__ __forceinline__ float rg_exp(float x) {
  // straight-line code: the range checks are selects at the end, so independent calls overlap
  const float y = f_mul(x, 0x1.715476p+0f);
  const float t = f_add(y, 12582912.0f);                // round to nearest-even integer: same value as rint(y)
  const float n = f_add(t, -12582912.0f);               //   for |y| < 2^22, which the range checks guarantee
  float r = f_fma(n, -0x1.62e400p-1f, x);
  r = f_fma(n, -0x1.7f7d1cp-20f, r);
  float p = 0x1.a01a02p-13f;
  p = f_fma(p, r, 0x1.6c16c2p-10f);
  p = f_fma(p, r, 0x1.111112p-7f);
  p = f_fma(p, r, 0x1.555556p-5f);
  p = f_fma(p, r, 0x1.555556p-3f);
  p = f_fma(p, r, 0.5f);
  p = f_fma(p, r, 1.0f);
  p = f_fma(p, r, 1.0f);
  const int ni = __float_as_int(t) - 0x4B400000;        // the integer n, read from t's mantissa
  const int h = ni >> 1;
  const float s1 = __int_as_float((ni - h + 127) << 23);
  const float s2 = __int_as_float((h + 127) << 23);
  float e = f_mul(f_mul(p, s1), s2);
  e = x < -87.33655f ? 0.0f : e;
  e = x > 88.72284f ? __int_as_float(0x7f800000) : e;
  return x != x ? x : e;
}

// rg_exp for |x| <= 87 (and not NaN): no range select can fire, n lies in [-126, 126], so 2^n is a
// normal number, the result is normal, and the two-factor scaling of rg_exp (two exact
// multiplications there) equals one exact multiplication by 2^n.  Same bits as rg_exp on that domain.
__device__ __forceinline__ float rg_exp_inrange(float x) {
  const float y = f_mul(x, 0x1.715476p+0f);
  const float t = f_add(y, 12582912.0f);
  const float n = f_add(t, -12582912.0f);
  float r = f_fma(n, -0x1.62e400p-1f, x);
  r = f_fma(n, -0x1.7f7d1cp-20f, r);
  float p = 0x1.a01a02p-13f;
  p = f_fma(p, r, 0x1.6c16c2p-10f);
  p = f_fma(p, r, 0x1.111112p-7f);
  p = f_fma(p, r, 0x1.555556p-5f);
  p = f_fma(p, r, 0x1.555556p-3f);
  p = f_fma(p, r, 0.5f);
  p = f_fma(p, r, 1.0f);
  p = f_fma(p, r, 1.0f);
  return f_mul(p, __int_as_float((__float_as_int(t) << 23) + 0x3f800000));   // t's low mantissa bits hold n
}

// rg_exp_inrange(-v) for a pair of values with |v| <= 87, computed from v itself with packed fp32x2 instructions
// where that is safe.  Rounding to nearest is symmetric in sign, so with n' = rint(v * log2 e) = -n and
// r' = v - n' ln2 = -r every intermediate of rg_exp_inrange(-v) appears here with its sign flipped or not at
// all changed: the Horner steps in r' take the coefficients with alternating signs, and 2^n is 2^-n'.  Same
// bits as the scalar form.  The first multiply stays scalar: a packed multiply in front of the packed add that
// rounds to an integer is fused with it by the assembler (another n on a few arguments in a billion).
__device__ __forceinline__ float2 rg_exp_neg_inrange2(float2 v) {
  const float2 y = make_float2(f_mul(v.x, 0x1.715476p+0f), f_mul(v.y, 0x1.715476p+0f));
  const float2 t = __fadd2_rn(y, make_float2(12582912.0f, 12582912.0f));
  const float2 n = __fadd2_rn(t, make_float2(-12582912.0f, -12582912.0f));
  float2 r = __ffma2_rn(n, make_float2(-0x1.62e400p-1f, -0x1.62e400p-1f), v);
  r = __ffma2_rn(n, make_float2(-0x1.7f7d1cp-20f, -0x1.7f7d1cp-20f), r);
  float2 q = make_float2(-0x1.a01a02p-13f, -0x1.a01a02p-13f);                       // degree 7: odd, sign flipped
  q = __ffma2_rn(q, r, make_float2(0x1.6c16c2p-10f, 0x1.6c16c2p-10f));
  q = __ffma2_rn(q, r, make_float2(-0x1.111112p-7f, -0x1.111112p-7f));
  q = __ffma2_rn(q, r, make_float2(0x1.555556p-5f, 0x1.555556p-5f));
  q = __ffma2_rn(q, r, make_float2(-0x1.555556p-3f, -0x1.555556p-3f));
  q = __ffma2_rn(q, r, make_float2(0.5f, 0.5f));
  q = __ffma2_rn(q, r, make_float2(-1.0f, -1.0f));
  q = __ffma2_rn(q, r, make_float2(1.0f, 1.0f));
  // t's low mantissa bits hold n'; the scale is 2^-n'
  return __fmul2_rn(q, make_float2(__int_as_float(0x3f800000 - (__float_as_int(t.x) << 23)), __int_as_float(0x3f800000 - (__float_as_int(t.y) << 23))));
}

// largest magnitude of three values; NaN if any of them is NaN (one instruction on this architecture)
__device__ __forceinline__ float absmax3_nan(float a, float b, float c) {
  float r;
  asm("max.NaN.abs.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}

// Base-two exponential fixed the same way (attention folds log2 e into the score scale, App. F):
// n = rint(x), f = x - n (exact), degree-7 Taylor polynomial of 2^f in Horner form with fused
// multiply-adds, and an exact scaling by 2^n done on the exponent field (the polynomial lies in
// [0.70, 1.42] and n in [-126, 128], so the result is a normal number or overflows to the clamp).
__device__ __forceinline__ float rg_exp2(float x) {
  const float t = f_add(x, 12582912.0f);                // round to nearest-even integer
  const float n = f_add(t, -12582912.0f);
  const float f = f_add(x, -n);
  float p = 0x1.ffcbfcp-17f;
  p = f_fma(p, f, 0x1.430912p-13f);
  p = f_fma(p, f, 0x1.5d87fep-10f);
  p = f_fma(p, f, 0x1.3b2ab6p-7f);
  p = f_fma(p, f, 0x1.c6b08ep-5f);
  p = f_fma(p, f, 0x1.ebfbe0p-3f);
  p = f_fma(p, f, 0x1.62e430p-1f);
  p = f_fma(p, f, 1.0f);
  const int ni = __float_as_int(t) - 0x4B400000;        // the integer n, read from t's mantissa
  float e = __int_as_float(__float_as_int(p) + (ni << 23));
  e = x < -126.0f ? 0.0f : e;
  e = x >= 128.0f ? __int_as_float(0x7f800000) : e;
  return x != x ? x : e;
}

__device__ __forceinline__ float rg_silu(float v) { return __fdiv_rn(v, f_add(1.0f, rg_exp(-v))); }

// Epilogue operands, passed by value to kernels.
struct EpilogueArgs {
  const void* bias;
  const void* residual;
  int64_t ldr;
  int32_t bias_dtype;
  int32_t residual_dtype;
  int32_t act;
};

__device__ __forceinline__ float f16_bits_to_f32(uint32_t h) { return __half2float(__ushort_as_half((unsigned short)h)); }

__device__ __forceinline__ float load_scalar(const void* p, int dtype, int64_t idx) {
  if (dtype == RG_BF16) return bf16_bits_to_f32(static_cast<const uint16_t*>(p)[idx]);
  if (dtype == RG_F16) return f16_bits_to_f32(static_cast<const uint16_t*>(p)[idx]);
  return static_cast<const float*>(p)[idx];
}

// One rounding of an fp32 value to `dtype` and back (identity for fp32).
__device__ __forceinline__ float round_through(float v, int dtype) {
  if (dtype == RG_BF16) return __bfloat162float(__float2bfloat16_rn(v));
  if (dtype == RG_F16) return __half2float(__float2half_rn(v));
  return v;
}

__device__ __forceinline__ uint32_t pack_f16x2(float lo, float hi) {
  const __half2 v = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}
__device__ __forceinline__ uint32_t pack_16x2(float lo, float hi, int dtype);

// `n` (<= 32) consecutive elements starting at element index `idx` of a bf16 or fp32 array, widened
// to fp32; entries past n are zero.  Uses 16-byte loads when the segment is full and aligned.
__device__ __forceinline__ void load_row_segment(const void* base, int dtype, int64_t idx, int n, float (&out)[32]) {
  // the type is tested once, outside the unrolled loops
  if (dtype == RG_BF16) {
    const uint16_t* p = static_cast<const uint16_t*>(base) + idx;
    if (n == 32 && (reinterpret_cast<uintptr_t>(p) & 15) == 0) {
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const uint4 w = __ldg(reinterpret_cast<const uint4*>(p) + q);
        const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          out[8 * q + 2 * t] = bf16_bits_to_f32(ww[t] & 0xffffu);
          out[8 * q + 2 * t + 1] = bf16_bits_to_f32(ww[t] >> 16);
        }
      }
    } else {
#pragma unroll
      for (int c = 0; c < 32; ++c) out[c] = c < n ? bf16_bits_to_f32(p[c]) : 0.0f;
    }
  } else if (dtype == RG_F16) {
    const uint16_t* p = static_cast<const uint16_t*>(base) + idx;
    if (n == 32 && (reinterpret_cast<uintptr_t>(p) & 15) == 0) {
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const uint4 w = __ldg(reinterpret_cast<const uint4*>(p) + q);
        const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          out[8 * q + 2 * t] = f16_bits_to_f32(ww[t] & 0xffffu);
          out[8 * q + 2 * t + 1] = f16_bits_to_f32(ww[t] >> 16);
        }
      }
    } else {
#pragma unroll
      for (int c = 0; c < 32; ++c) out[c] = c < n ? f16_bits_to_f32(p[c]) : 0.0f;
    }
  } else {
    const float* p = static_cast<const float*>(base) + idx;
    if (n == 32 && (reinterpret_cast<uintptr_t>(p) & 15) == 0) {
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        const float4 w = __ldg(reinterpret_cast<const float4*>(p) + q);
        out[4 * q] = w.x; out[4 * q + 1] = w.y; out[4 * q + 2] = w.z; out[4 * q + 3] = w.w;
      }
    } else {
#pragma unroll
      for (int c = 0; c < 32; ++c) out[c] = c < n ? p[c] : 0.0f;
    }
  }
}

// bias -> activation -> residual, in that order, on one fp32 value (Sec. 2: the position of
// the output rounding is part of the order; it happens once, in the caller's store).
__device__ __forceinline__ float apply_epilogue(float v, const EpilogueArgs& e, int64_t i, int64_t j) {
  if (e.bias) v = f_add(v, load_scalar(e.bias, e.bias_dtype, j));
  if (e.act == 1) v = rg_silu(v);
  if (e.residual) v = f_add(v, load_scalar(e.residual, e.residual_dtype, i * e.ldr + j));
  return v;
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  // one cvt.rn.bf16x2.f32: each half is rounded to nearest even exactly as a single conversion is
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}

__device__ __forceinline__ uint32_t pack_16x2(float lo, float hi, int dtype) {
  return dtype == RG_F16 ? pack_f16x2(lo, hi) : pack_bf16x2(lo, hi);
}

// Store one fp32 value rounded once to a 16-bit or fp32 output element.
__device__ __forceinline__ void store_scalar(void* p, int dtype, int64_t idx, float v) {
  if (dtype == RG_BF16) static_cast<__nv_bfloat16*>(p)[idx] = __float2bfloat16_rn(v);
  else if (dtype == RG_F16) static_cast<__half*>(p)[idx] = __float2half_rn(v);
  else static_cast<float*>(p)[idx] = v;
}

}  // namespace rg
