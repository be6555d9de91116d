// Reductions along the other axis (Sec. 6: reductions on different axes; the column sum a
// matrix-multiply epilogue emits; the LayerNorm weight-gradient shape): one balanced "neighbours
// pair first" tree (Sec. 5.1) per column, over the rows in index order.
//
// A CTA of 8 warps owns 128 columns x 256 rows.  A lane owns 4 consecutive columns; a warp owns 32
// consecutive rows (an aligned block, so its total is a subtree): four groups of 8 rows, the 8 loads
// of a group in flight together, each group folded by the fixed tree on 8 leaves, the four group
// totals by the fixed tree on 4.  The 8 warp totals meet in shared memory and are folded by the
// fixed tree on 8.  Rows past the end are the additive identity -0.0f (x + -0 = x for every x), so
// "an unpaired value moves up unchanged" needs no special case.  With more than 256 rows the CTA
// totals are written as rows of a partial matrix and the same kernel folds that matrix: the blocks
// are aligned, so this is the upper part of the same tree.
#include "rg_common.cuh"
#include "rg_internal.h"

namespace rg {

namespace {

constexpr int COL_THREADS = 256;
constexpr int COL_TILE = 128;       // columns per CTA
constexpr int ROWS_PER_WARP = 32;
constexpr int ROWS_PER_CTA = 256;

struct ColParams {
  const void* x;
  const void* y;
  float* out;          // [gridDim.y][C]
  int64_t ldx, ldy;
  int64_t R, C;
};

__device__ __forceinline__ float4 add4(const float4& a, const float4& b) {
  return make_float4(f_add(a.x, b.x), f_add(a.y, b.y), f_add(a.z, b.z), f_add(a.w, b.w));
}

// four consecutive elements of one row, widened to fp32; columns past C and rows past R give `fill`
template <bool IN16>
__device__ __forceinline__ float4 load4(const void* base, int64_t ld, int64_t row, int64_t R, int64_t col0, int64_t C,
                                        bool vec_ok, float fill) {
  float4 v = make_float4(fill, fill, fill, fill);
  if (row >= R || col0 >= C) return v;
  if (IN16) {
    const uint16_t* p = static_cast<const uint16_t*>(base) + row * ld + col0;
    if (vec_ok && col0 + 4 <= C) {
      const uint2 w = __ldg(reinterpret_cast<const uint2*>(p));
      v = make_float4(bf16_bits_to_f32(w.x & 0xffffu), bf16_bits_to_f32(w.x >> 16), bf16_bits_to_f32(w.y & 0xffffu), bf16_bits_to_f32(w.y >> 16));
    } else {
      v.x = bf16_bits_to_f32(p[0]);
      if (col0 + 1 < C) v.y = bf16_bits_to_f32(p[1]);
      if (col0 + 2 < C) v.z = bf16_bits_to_f32(p[2]);
      if (col0 + 3 < C) v.w = bf16_bits_to_f32(p[3]);
    }
  } else {
    const float* p = static_cast<const float*>(base) + row * ld + col0;
    if (vec_ok && col0 + 4 <= C) {
      v = __ldg(reinterpret_cast<const float4*>(p));
    } else {
      v.x = p[0];
      if (col0 + 1 < C) v.y = p[1];
      if (col0 + 2 < C) v.z = p[2];
      if (col0 + 3 < C) v.w = p[3];
    }
  }
  return v;
}

// OP 0: sum of x; OP 1: sum of x*y.  FMA (OP 1 only): the second product of a level-0 pair is fused.
template <int OP, bool IN16, bool FMA>
__global__ void __launch_bounds__(COL_THREADS) reduce_cols_kernel(const ColParams p) {
  __shared__ float4 warp_total[COL_THREADS / 32][32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t col0 = (int64_t)blockIdx.x * COL_TILE + lane * 4;
  const int64_t row0 = (int64_t)blockIdx.y * ROWS_PER_CTA + warp * ROWS_PER_WARP;
  const int esz = IN16 ? 2 : 4;
  const bool vx = ((reinterpret_cast<uintptr_t>(p.x) | (uintptr_t)(p.ldx * esz)) & (uintptr_t)(4 * esz - 1)) == 0;
  const bool vy = OP == 1 && ((reinterpret_cast<uintptr_t>(p.y) | (uintptr_t)(p.ldy * esz)) & (uintptr_t)(4 * esz - 1)) == 0;
  float4 group_total[4];
#pragma unroll
  for (int g = 0; g < 4; ++g) {
    float4 xv[8], yv[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) xv[i] = load4<IN16>(p.x, p.ldx, row0 + g * 8 + i, p.R, col0, p.C, vx, -0.0f);
    if (OP == 1) {
#pragma unroll
      for (int i = 0; i < 8; ++i) yv[i] = load4<IN16>(p.y, p.ldy, row0 + g * 8 + i, p.R, col0, p.C, vy, 0.0f);
    }
    float4 pair[4];
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      if (OP == 0) {
        pair[t] = add4(xv[2 * t], xv[2 * t + 1]);
      } else if (FMA) {
        const float4 a = xv[2 * t], b = yv[2 * t], c = xv[2 * t + 1], d = yv[2 * t + 1];
        pair[t] = make_float4(f_fma(c.x, d.x, f_mul(a.x, b.x)), f_fma(c.y, d.y, f_mul(a.y, b.y)),
                              f_fma(c.z, d.z, f_mul(a.z, b.z)), f_fma(c.w, d.w, f_mul(a.w, b.w)));
      } else {
        const float4 a = xv[2 * t], b = yv[2 * t], c = xv[2 * t + 1], d = yv[2 * t + 1];
        pair[t] = make_float4(f_add(f_mul(a.x, b.x), f_mul(c.x, d.x)), f_add(f_mul(a.y, b.y), f_mul(c.y, d.y)),
                              f_add(f_mul(a.z, b.z), f_mul(c.z, d.z)), f_add(f_mul(a.w, b.w), f_mul(c.w, d.w)));
      }
    }
    group_total[g] = add4(add4(pair[0], pair[1]), add4(pair[2], pair[3]));
  }
  warp_total[warp][lane] = add4(add4(group_total[0], group_total[1]), add4(group_total[2], group_total[3]));
  __syncthreads();
  if (warp == 0 && col0 < p.C) {
    const float4 t = add4(add4(add4(warp_total[0][lane], warp_total[1][lane]), add4(warp_total[2][lane], warp_total[3][lane])),
                          add4(add4(warp_total[4][lane], warp_total[5][lane]), add4(warp_total[6][lane], warp_total[7][lane])));
    float* o = p.out + (int64_t)blockIdx.y * p.C + col0;
    if (col0 + 4 <= p.C && (reinterpret_cast<uintptr_t>(o) & 15) == 0) {
      *reinterpret_cast<float4*>(o) = t;
    } else {
      o[0] = t.x;
      if (col0 + 1 < p.C) o[1] = t.y;
      if (col0 + 2 < p.C) o[2] = t.z;
      if (col0 + 3 < p.C) o[3] = t.w;
    }
  }
}

// Left fold (RG_TREE_LEFT): one thread per column walks the rows in index order, ((l0 + l1) + l2) + ...;
// neighbouring threads read neighbouring columns, so every row is one coalesced run.  Eight rows are
// requested ahead of the chain.  With `fma` the dot product is the chain acc = fma(x, y, acc) from x0 * y0.
template <typename T, bool DOT>
__global__ void __launch_bounds__(128) reduce_cols_left_kernel(const void* xv, const void* yv, int64_t ldx, int64_t ldy, int64_t R, int64_t C,
                                                               int fma, float* out) {
  const int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= C) return;
  const T* x = static_cast<const T*>(xv) + c;
  const T* y = DOT ? static_cast<const T*>(yv) + c : nullptr;
  auto widen = [](T v) -> float { if constexpr (sizeof(T) == 2) return bf16_bits_to_f32(v); else return v; };
  float acc = 0.0f;
  for (int64_t r0 = 0; r0 < R; r0 += 8) {
    float a[8], b[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const bool ok = r0 + i < R;
      a[i] = ok ? widen(x[(r0 + i) * ldx]) : 0.0f;
      b[i] = (DOT && ok) ? widen(y[(r0 + i) * ldy]) : 0.0f;
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      if (r0 + i < R) {
        const bool first = r0 + i == 0;
        if (!DOT) acc = first ? a[i] : f_add(acc, a[i]);
        else acc = first ? f_mul(a[i], b[i]) : (fma ? f_fma(a[i], b[i], acc) : f_add(acc, f_mul(a[i], b[i])));
      }
    }
  }
  out[c] = acc;
}

template <int OP, bool IN16>
cudaError_t launch_stage(const ColParams& p, bool fma, dim3 grid, cudaStream_t st) {
  if (OP == 1 && fma) reduce_cols_kernel<OP, IN16, true><<<grid, COL_THREADS, 0, st>>>(p);
  else reduce_cols_kernel<OP, IN16, false><<<grid, COL_THREADS, 0, st>>>(p);
  return cudaGetLastError();
}

}  // namespace

size_t reduce_cols_workspace_bytes(int64_t R, int64_t C) {
  size_t rows = 0;
  for (int64_t r = (R + ROWS_PER_CTA - 1) / ROWS_PER_CTA; r > 1; r = (r + ROWS_PER_CTA - 1) / ROWS_PER_CTA) rows += (size_t)r;
  return rows * (size_t)C * sizeof(float);
}

// All arguments were validated by the caller.
rg_status_t launch_reduce_cols(int op, int tree, int fma, const rg_tensor_t* x, const rg_tensor_t* y, const rg_tensor_t* out,
                               void* ws, cudaStream_t st) {
  const int64_t C = x->cols;
  if (tree == RG_TREE_LEFT) {
    const unsigned grid = (unsigned)((C + 127) / 128);
    const bool in16 = x->dtype == RG_BF16;
    if (op == RG_COLOP_DOT) {
      if (in16) reduce_cols_left_kernel<uint16_t, true><<<grid, 128, 0, st>>>(x->ptr, y->ptr, x->ld, y->ld, x->rows, C, fma, static_cast<float*>(out->ptr));
      else reduce_cols_left_kernel<float, true><<<grid, 128, 0, st>>>(x->ptr, y->ptr, x->ld, y->ld, x->rows, C, fma, static_cast<float*>(out->ptr));
    } else {
      if (in16) reduce_cols_left_kernel<uint16_t, false><<<grid, 128, 0, st>>>(x->ptr, nullptr, x->ld, 0, x->rows, C, 0, static_cast<float*>(out->ptr));
      else reduce_cols_left_kernel<float, false><<<grid, 128, 0, st>>>(x->ptr, nullptr, x->ld, 0, x->rows, C, 0, static_cast<float*>(out->ptr));
    }
    return cudaGetLastError() == cudaSuccess ? RG_OK : RG_ERR_CUDA;
  }
  ColParams p;
  p.x = x->ptr; p.y = y ? y->ptr : nullptr; p.ldx = x->ld; p.ldy = y ? y->ld : 0;
  p.R = x->rows; p.C = C;
  bool in16 = x->dtype == RG_BF16;
  float* region = static_cast<float*>(ws);
  const unsigned gx = (unsigned)((C + COL_TILE - 1) / COL_TILE);
  for (int stage = 0;; ++stage) {
    const int64_t parts = (p.R + ROWS_PER_CTA - 1) / ROWS_PER_CTA;
    p.out = parts == 1 ? static_cast<float*>(out->ptr) : region;
    const dim3 grid(gx, (unsigned)parts, 1);
    cudaError_t err;
    if (stage == 0 && op == RG_COLOP_DOT) err = in16 ? launch_stage<1, true>(p, fma != 0, grid, st) : launch_stage<1, false>(p, fma != 0, grid, st);
    else err = in16 ? launch_stage<0, true>(p, false, grid, st) : launch_stage<0, false>(p, false, grid, st);
    if (err != cudaSuccess) return RG_ERR_CUDA;
    if (parts == 1) break;
    // the partial rows become the matrix the next stage folds
    p.x = region; p.y = nullptr; p.ldx = C; p.R = parts; in16 = false;
    region += parts * C;
  }
  return RG_OK;
}

}  // namespace rg
