// Device-side scalar arithmetic shared by the GEMM epilogue, the split-K merge and the
// row reductions.  Every operation is an explicit round-to-nearest intrinsic so that the
// compiler can neither contract a multiply into an add nor reassociate: the dependence tree
// written here is the one that runs (Sec. 3.1).
#pragma once
#include <cuda_bf16.h>
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
  if (x != x) return x;
  if (x > 88.72284f) return __int_as_float(0x7f800000);
  if (x < -87.33655f) return 0.0f;
  const float n = rintf(f_mul(x, 0x1.715476p+0f));
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
  const int ni = (int)n;
  const int h = ni >> 1;
  const float s1 = __int_as_float((ni - h + 127) << 23);
  const float s2 = __int_as_float((h + 127) << 23);
  return f_mul(f_mul(p, s1), s2);
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

__device__ __forceinline__ float load_scalar(const void* p, int dtype, int64_t idx) {
  if (dtype == RG_BF16) return bf16_bits_to_f32(static_cast<const uint16_t*>(p)[idx]);
  return static_cast<const float*>(p)[idx];
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
  const uint32_t l = __bfloat16_as_ushort(__float2bfloat16_rn(lo));
  const uint32_t h = __bfloat16_as_ushort(__float2bfloat16_rn(hi));
  return l | (h << 16);
}

}  // namespace rg
