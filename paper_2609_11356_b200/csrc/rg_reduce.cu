// Row reductions with a pinned balanced tree (Sec. 3.1 three-level tree; Sec. 5.1 count-up
// butterfly).  The tree is defined over the logical column index: level l combines aligned
// blocks of 2^l columns, an unpaired block moves up unchanged.  A pinned tree makes the data
// layout a free speed knob (Sec. 5.2), which is what the kernel spends:
//
//   thread : one 16-byte vector = an aligned block of V columns (V = 4 fp32 / 8 bf16), folded
//            in registers in index order                                  (levels 0 .. log2 V)
//   warp   : 32 lanes hold 32 neighbouring blocks; shuffle-xor offsets counted UP 1,2,4,8,16
//            so neighbours pair first                                     (next 5 levels)
//   unroll : a warp folds U consecutive warp-blocks (U independent loads in flight), then
//            combines the U values pairwise in registers                  (next log2 U levels)
//   CTA    : the remaining values go through shared memory and one last butterfly.
//
// Columns past the end of the row are the additive identity -0.0f: x + (-0) = x for every x,
// so padding is bit-identical to "moves up unchanged".  (+0.0 would not be: -0 + +0 = +0.)
// All adds are __fadd_rn; nothing here can be contracted or reassociated by the compiler.
#include "rg_common.cuh"

namespace rg {

namespace {

constexpr float NEG_ZERO = -0.0f;

enum : int { OP_SUM = 0, OP_RMS = 1, OP_SOFTMAX = 2 };

template <typename T> struct VecTraits;
template <> struct VecTraits<float> { static constexpr int V = 4; };
template <> struct VecTraits<uint16_t> { static constexpr int V = 8; };

__device__ __forceinline__ float elem_to_f32(float v) { return v; }
__device__ __forceinline__ float elem_to_f32(uint16_t v) { return bf16_bits_to_f32(v); }

// Load V consecutive elements starting at column `col` of a row; out-of-range columns are
// flagged invalid.  VEC: the row start is 16-byte aligned and ld is a multiple of V.
template <typename T, bool VEC>
__device__ __forceinline__ void load_block(const T* __restrict__ xr, int64_t col, int64_t C,
                                           float (&v)[VecTraits<T>::V], bool (&ok)[VecTraits<T>::V]) {
  constexpr int V = VecTraits<T>::V;
  if (VEC && col + V <= C) {
    const uint4 raw = __ldg(reinterpret_cast<const uint4*>(xr + col));
    if constexpr (sizeof(T) == 4) {
      v[0] = __uint_as_float(raw.x); v[1] = __uint_as_float(raw.y);
      v[2] = __uint_as_float(raw.z); v[3] = __uint_as_float(raw.w);
    } else {
      const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        v[2 * t] = bf16_bits_to_f32(w[t] & 0xffffu);
        v[2 * t + 1] = bf16_bits_to_f32(w[t] >> 16);
      }
    }
#pragma unroll
    for (int t = 0; t < V; ++t) ok[t] = true;
  } else {
#pragma unroll
    for (int t = 0; t < V; ++t) {
      ok[t] = (col + t) < C;
      v[t] = ok[t] ? elem_to_f32(xr[col + t]) : 0.0f;
    }
  }
}

// Fold one thread's V leaves in index order: (l0+l1), (l2+l3), ... then pairs of pairs.
template <int OP, int V>
__device__ __forceinline__ float fold_block(const float (&x)[V], const bool (&ok)[V], float shift, int fma) {
  float n[V / 2];
#pragma unroll
  for (int t = 0; t < V / 2; ++t) {
    const float x0 = x[2 * t], x1 = x[2 * t + 1];
    if (OP == OP_SUM) {
      n[t] = f_add(ok[2 * t] ? x0 : NEG_ZERO, ok[2 * t + 1] ? x1 : NEG_ZERO);
    } else if (OP == OP_RMS) {
      const float s0 = ok[2 * t] ? f_mul(x0, x0) : NEG_ZERO;
      if (fma) n[t] = ok[2 * t + 1] ? f_fma(x1, x1, s0) : s0;   // second square fused into the add
      else n[t] = f_add(s0, ok[2 * t + 1] ? f_mul(x1, x1) : NEG_ZERO);
    } else {
      const float e0 = ok[2 * t] ? rg_exp(f_add(x0, -shift)) : NEG_ZERO;
      const float e1 = ok[2 * t + 1] ? rg_exp(f_add(x1, -shift)) : NEG_ZERO;
      n[t] = f_add(e0, e1);
    }
  }
#pragma unroll
  for (int s = 1; s < V / 2; s <<= 1)
#pragma unroll
    for (int t = 0; t < V / 2; t += 2 * s) n[t] = f_add(n[t], n[t + s]);
  return n[0];
}

__device__ __forceinline__ float warp_tree(float v) {
  // count-up butterfly: neighbours pair first (Sec. 5.1, Fig. 3)
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) v = f_add(v, __shfl_xor_sync(0xffffffffu, v, off));
  return v;
}

// TREE over the row's leaves; every thread of the CTA returns the root.
// sb: shared scratch of 2 * cap floats (ping-pong), cap >= number of super-blocks.
template <typename T, int OP, bool VEC, int U>
__device__ float row_tree(const T* __restrict__ xr, int64_t C, float shift, int fma, float* sb, int cap) {
  constexpr int V = VecTraits<T>::V;
  constexpr int WB = 32 * V;           // columns per warp-block
  constexpr int SBW = WB * U;          // columns per super-block
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  const int nsb = (int)((C + SBW - 1) / SBW);
  for (int sbi = warp; sbi < nsb; sbi += nwarps) {
    const int64_t base = (int64_t)sbi * SBW + lane * V;
    float bv[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      float x[V]; bool ok[V];
      load_block<T, VEC>(xr, base + (int64_t)u * WB, C, x, ok);
      bv[u] = fold_block<OP, V>(x, ok, shift, fma);
    }
#pragma unroll
    for (int off = 1; off < 32; off <<= 1)
#pragma unroll
      for (int u = 0; u < U; ++u) bv[u] = f_add(bv[u], __shfl_xor_sync(0xffffffffu, bv[u], off));
#pragma unroll
    for (int s = 1; s < U; s <<= 1)
#pragma unroll
      for (int u = 0; u < U; u += 2 * s) bv[u] = f_add(bv[u], bv[u + s]);
    if (lane == 0) sb[sbi] = bv[0];
  }
  __syncthreads();
  // remaining levels over nsb values
  int n = nsb;
  float* cur = sb;
  float* nxt = sb + cap;
  while (n > 32) {
    const int half = (n + 1) >> 1;
    for (int t = threadIdx.x; t < half; t += blockDim.x)
      nxt[t] = (2 * t + 1 < n) ? f_add(cur[2 * t], cur[2 * t + 1]) : cur[2 * t];
    __syncthreads();
    float* tmp = cur; cur = nxt; nxt = tmp;
    n = half;
  }
  float v = (lane < n) ? cur[lane] : NEG_ZERO;
  v = warp_tree(v);
  __syncthreads();                      // scratch may be reused by the caller's next row
  return v;
}

struct ReduceParams {
  const void* x;
  void* out;
  const void* weight;
  float* aux;
  int64_t R, C, ldx, ldo;
  float eps;
  int32_t fma, out_dtype, w_dtype, cap;
};

template <typename T, int OP, bool VEC, int U>
__global__ void __launch_bounds__(256) reduce_rows_kernel(const ReduceParams p) {
  extern __shared__ float smem[];
  float* sb = smem;                     // 2 * cap floats
  float* red = smem + 2 * p.cap;        // 32 floats for the order-free max
  constexpr int V = VecTraits<T>::V;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  for (int64_t row = blockIdx.x; row < p.R; row += gridDim.x) {
    const T* xr = static_cast<const T*>(p.x) + row * p.ldx;
    float shift = 0.0f;
    if (OP == OP_SOFTMAX) {
      // The row maximum rounds nothing, so its order is free (App. F).
      float m = -INFINITY;
      for (int64_t c = (int64_t)threadIdx.x * V; c < p.C; c += (int64_t)blockDim.x * V) {
        float x[V]; bool ok[V];
        load_block<T, VEC>(xr, c, p.C, x, ok);
#pragma unroll
        for (int t = 0; t < V; ++t) if (ok[t]) m = fmaxf(m, x[t]);
      }
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
      if (lane == 0) red[warp] = m;
      __syncthreads();
      m = red[0];
      for (int w = 1; w < nwarps; ++w) m = fmaxf(m, red[w]);
      shift = m;
      __syncthreads();
    }
    const float root = row_tree<T, OP, VEC, U>(xr, p.C, shift, p.fma, sb, p.cap);
    if (OP == OP_SUM) {
      if (threadIdx.x == 0) static_cast<float*>(p.out)[row * p.ldo] = root;
    } else if (OP == OP_SOFTMAX) {
      if (threadIdx.x == 0) {
        static_cast<float*>(p.out)[row * p.ldo] = root;
        if (p.aux) p.aux[row] = shift;
      }
    } else {
      const float ms = __fdiv_rn(root, (float)p.C);
      const float rinv = __fdiv_rn(1.0f, __fsqrt_rn(f_add(ms, p.eps)));
      if (threadIdx.x == 0 && p.aux) p.aux[row] = rinv;
      const bool out_vec = VEC && ((reinterpret_cast<uintptr_t>(p.out) & 15) == 0) &&
                           (p.ldo % V == 0) && (p.out_dtype == (sizeof(T) == 2 ? RG_BF16 : RG_F32));
      for (int64_t c = (int64_t)threadIdx.x * V; c < p.C; c += (int64_t)blockDim.x * V) {
        float x[V]; bool ok[V];
        load_block<T, VEC>(xr, c, p.C, x, ok);
        float y[V];
#pragma unroll
        for (int t = 0; t < V; ++t) {
          const float w = (p.weight && ok[t]) ? load_scalar(p.weight, p.w_dtype, c + t) : 1.0f;
          y[t] = f_mul(f_mul(x[t], rinv), w);
        }
        if (out_vec && c + V <= p.C) {
          uint4 o;
          if constexpr (sizeof(T) == 4) {
            o = make_uint4(__float_as_uint(y[0]), __float_as_uint(y[1]), __float_as_uint(y[2]), __float_as_uint(y[3]));
            *reinterpret_cast<uint4*>(static_cast<float*>(p.out) + row * p.ldo + c) = o;
          } else {
            o = make_uint4(pack_bf16x2(y[0], y[1]), pack_bf16x2(y[2], y[3]), pack_bf16x2(y[4], y[5]), pack_bf16x2(y[6], y[7]));
            *reinterpret_cast<uint4*>(static_cast<uint16_t*>(p.out) + row * p.ldo + c) = o;
          }
        } else {
#pragma unroll
          for (int t = 0; t < V; ++t)
            if (ok[t]) {
              if (p.out_dtype == RG_BF16)
                static_cast<__nv_bfloat16*>(p.out)[row * p.ldo + c + t] = __float2bfloat16_rn(y[t]);
              else
                static_cast<float*>(p.out)[row * p.ldo + c + t] = y[t];
            }
        }
      }
    }
  }
}

template <typename T, int OP, bool VEC>
cudaError_t launch_u(const ReduceParams& p, int U, int threads, int grid, size_t smem, cudaStream_t st) {
  switch (U) {
    case 1: reduce_rows_kernel<T, OP, VEC, 1><<<grid, threads, smem, st>>>(p); break;
    case 2: reduce_rows_kernel<T, OP, VEC, 2><<<grid, threads, smem, st>>>(p); break;
    case 4: reduce_rows_kernel<T, OP, VEC, 4><<<grid, threads, smem, st>>>(p); break;
    default: reduce_rows_kernel<T, OP, VEC, 8><<<grid, threads, smem, st>>>(p); break;
  }
  return cudaGetLastError();
}

template <typename T, int OP>
cudaError_t launch_vec(const ReduceParams& p, bool vec, int U, int threads, int grid, size_t smem, cudaStream_t st) {
  return vec ? launch_u<T, OP, true>(p, U, threads, grid, smem, st)
             : launch_u<T, OP, false>(p, U, threads, grid, smem, st);
}

template <typename T>
cudaError_t launch_op(int op, const ReduceParams& p, bool vec, int U, int threads, int grid, size_t smem, cudaStream_t st) {
  switch (op) {
    case RG_OP_SUM: return launch_vec<T, OP_SUM>(p, vec, U, threads, grid, smem, st);
    case RG_OP_RMSNORM: return launch_vec<T, OP_RMS>(p, vec, U, threads, grid, smem, st);
    default: return launch_vec<T, OP_SOFTMAX>(p, vec, U, threads, grid, smem, st);
  }
}

}  // namespace

// Host launcher.  threads_hint / unroll_hint: 0 = choose; both are speed knobs only.
rg_status_t launch_reduce_rows(int op, int fma, const rg_tensor_t* x, const rg_tensor_t* out,
                               const rg_reduce_args_t* args, int threads_hint, int unroll_hint,
                               cudaStream_t st) {
  const int V = x->dtype == RG_BF16 ? 8 : 4;
  const int64_t C = x->cols;
  const int64_t nblocks = (C + 32 * V - 1) / (32 * V);          // warp-blocks in a row
  int U = unroll_hint;
  if (U != 1 && U != 2 && U != 4 && U != 8) {
    U = nblocks >= 64 ? 8 : nblocks >= 16 ? 4 : nblocks >= 4 ? 2 : 1;
  }
  const int64_t nsb = (nblocks + U - 1) / U;
  int threads = threads_hint;
  if (threads != 32 && threads != 64 && threads != 128 && threads != 256) {
    threads = nsb >= 8 ? 256 : nsb >= 4 ? 128 : nsb >= 2 ? 64 : 32;
  }
  if (nsb > 4096) return RG_ERR_UNSUPPORTED;                   // rows beyond ~4M fp32 columns
  const int cap = (int)((nsb + 31) / 32 * 32);
  const size_t smem = (size_t)(2 * cap + 32) * sizeof(float);
  const size_t esz = x->dtype == RG_BF16 ? 2 : 4;
  const bool vec = (reinterpret_cast<uintptr_t>(x->ptr) % 16 == 0) && ((x->ld * esz) % 16 == 0);
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int64_t max_grid = (int64_t)sms * (2048 / threads);
  const int grid = (int)(x->rows < max_grid ? x->rows : max_grid);
  ReduceParams p;
  p.x = x->ptr; p.out = out->ptr;
  p.weight = args ? args->weight : nullptr;
  p.aux = args ? static_cast<float*>(args->aux_out) : nullptr;
  p.R = x->rows; p.C = C; p.ldx = x->ld; p.ldo = out->ld;
  p.eps = args ? args->eps : 0.0f;
  p.fma = fma; p.out_dtype = out->dtype; p.w_dtype = args ? args->weight_dtype : RG_F32; p.cap = cap;
  cudaError_t e = x->dtype == RG_BF16 ? launch_op<uint16_t>(op, p, vec, U, threads, grid, smem, st)
                                      : launch_op<float>(op, p, vec, U, threads, grid, smem, st);
  return e == cudaSuccess ? RG_OK : RG_ERR_CUDA;
}

}  // namespace rg
