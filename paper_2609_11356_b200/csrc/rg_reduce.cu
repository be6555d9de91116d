// Row reductions with a pinned balanced tree (Sec. 3.1 three-level tree; Sec. 5.1 count-up
// butterfly).  The tree is defined over the logical column index: level l combines aligned
// blocks of 2^l columns, an unpaired block moves up unchanged.  A pinned tree makes the data
// layout a free speed knob (Sec. 5.2), which is what the kernels spend:
//
//   thread : one 16-byte vector = an aligned block of V columns (V = 4 fp32 / 8 bf16), folded
//            in registers in index order                                  (levels 0 .. log2 V)
//   warp   : 32 lanes hold 32 neighbouring blocks; shuffle-xor offsets counted UP 1,2,4,8,16
//            so neighbours pair first                                     (next 5 levels)
//   unroll : a warp folds U consecutive warp-blocks (U independent loads in flight), then
//            combines the U values pairwise in registers                  (next log2 U levels)
//   above  : "super-block" values are combined in index order with a binary-counter stack
//            (warp-per-row kernel) or through shared memory (CTA-per-row kernel); both visit
//            exactly the aligned pairs of the level-by-level definition.
//
// Columns past the end of the row are the additive identity -0.0f: x + (-0) = x for every x,
// so padding is bit-identical to "moves up unchanged".  (+0.0 would not be: -0 + +0 = +0.)
// All adds are __fadd_rn; nothing here can be contracted or reassociated by the compiler.
//
// Two kernels, same bits:
//   reduce_rows_warp_kernel  one warp owns a row: no barriers, all warps independent.  Used
//                            for sums and RMSNorm when there are enough rows to fill the GPU.
//   reduce_rows_cta_kernel   one CTA owns a row (32..1024 threads).  Used for few rows, and for
//                            the softmax normaliser, whose second pass re-reads the row (from L2).
#include "rg_common.cuh"
#include "rg_internal.h"
#include "rg_ptx.cuh"

namespace rg {

__device__ unsigned int g_reduce_status_word = 0;

namespace {

constexpr float NEG_ZERO = -0.0f;

// Every kernel here is launched with programmatic stream serialisation: its CTAs may be scheduled while the
// kernel ahead of it in the stream drains, and a kernel launched the same way behind it may be scheduled as
// soon as all of this kernel's CTAs have started.  Nothing is read before the kernels ahead have completed.
__device__ __forceinline__ void pdl_prologue() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
}
constexpr int MAX_LEVELS = 13;          // super-blocks per row < 2^13

enum : int { OP_SUM = 0, OP_RMS = 1, OP_SOFTMAX = 2 };

template <typename T> struct VecTraits;
template <> struct VecTraits<float> { static constexpr int V = 4; };
template <> struct VecTraits<uint16_t> { static constexpr int V = 8; };

__device__ __forceinline__ float elem_to_f32(float v) { return v; }
__device__ __forceinline__ float elem_to_f32(uint16_t v) { return bf16_bits_to_f32(v); }

template <typename T>
__device__ __forceinline__ void unpack(const uint4& raw, float (&v)[VecTraits<T>::V]) {
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
}

// exp(d) for d <= 0 (the softmax leaf x - max): the library's exponential with the branches
// that cannot trigger for d <= 0 removed and rint / the 2^n scaling done with bit-exact
// equivalents (round-to-integer by adding 1.5*2^23; one multiply by 2^n, n in [-126, 0]).
__device__ __forceinline__ float exp_nonpositive(float d) {
  const float y = f_mul(d, 0x1.715476p+0f);
  const float t = f_add(y, 12582912.0f);
  const float n = f_add(t, -12582912.0f);
  float r = f_fma(n, -0x1.62e400p-1f, d);
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
  const float s = __int_as_float((ni + 127) << 23);
  const float e = f_mul(p, s);
  return d < -87.33655f ? 0.0f : e;
}

// Fold one thread's V leaves in index order: (l0+l1), (l2+l3), ... then pairs of pairs.
// FULL: all V columns exist.  Otherwise `nvalid` leading ones do; the rest are -0.0f.
template <int OP, int V, bool FULL>
__device__ __forceinline__ float fold_block(const float (&x)[V], int nvalid, float shift, int fma) {
  if (OP == OP_SOFTMAX) {
    // exp(x - m) is exactly +0 below the library's underflow threshold.  When that holds for every
    // leaf this warp is folding, the block's sum is a sum of zeros and the polynomial is skipped
    // (a warp-uniform branch; called from warp-uniform control flow only).  Same bits, less work:
    // with wide-ranged logits most of a row lies that far below its maximum.
    bool live = false;
#pragma unroll
    for (int t = 0; t < V; ++t) live |= (FULL || t < nvalid) && !(f_add(x[t], -shift) < -87.33655f);
    if (!__any_sync(0xffffffffu, live)) return (FULL || nvalid > 0) ? 0.0f : NEG_ZERO;
  }
  float n[V / 2];
#pragma unroll
  for (int t = 0; t < V / 2; ++t) {
    const float x0 = x[2 * t], x1 = x[2 * t + 1];
    const bool ok0 = FULL || (2 * t < nvalid), ok1 = FULL || (2 * t + 1 < nvalid);
    if (OP == OP_SUM) {
      n[t] = f_add(ok0 ? x0 : NEG_ZERO, ok1 ? x1 : NEG_ZERO);
    } else if (OP == OP_RMS) {
      const float s0 = ok0 ? f_mul(x0, x0) : NEG_ZERO;
      if (fma) n[t] = ok1 ? f_fma(x1, x1, s0) : s0;      // second square fused into the add
      else n[t] = f_add(s0, ok1 ? f_mul(x1, x1) : NEG_ZERO);
    } else {
      // scalar on purpose: the packed f32x2 form measured slower here (the fp32 pipe, not issue, is the limit)
      const float e0 = ok0 ? exp_nonpositive(f_add(x0, -shift)) : NEG_ZERO;
      const float e1 = ok1 ? exp_nonpositive(f_add(x1, -shift)) : NEG_ZERO;
      n[t] = f_add(e0, e1);
    }
  }
#pragma unroll
  for (int s = 1; s < V / 2; s <<= 1)
#pragma unroll
    for (int t = 0; t < V / 2; t += 2 * s) n[t] = f_add(n[t], n[t + s]);
  return n[0];
}

// Load the V columns starting at `col` (VEC: 16-byte aligned rows) and fold them.
template <typename T, int OP, bool VEC>
__device__ __forceinline__ float load_fold(const T* __restrict__ xr, int64_t col, int64_t C, float shift, int fma) {
  constexpr int V = VecTraits<T>::V;
  float x[V];
  int nvalid = V;
  if (VEC && col + V <= C) {
    unpack<T>(__ldg(reinterpret_cast<const uint4*>(xr + col)), x);
  } else {
    nvalid = 0;
#pragma unroll
    for (int t = 0; t < V; ++t) {
      const bool ok = (col + t) < C;
      x[t] = ok ? elem_to_f32(xr[col + t]) : 0.0f;
      nvalid += ok ? 1 : 0;
    }
  }
  // The lanes of a warp may have taken different sides above (a ragged row end).  The fold votes
  // across the warp, so every lane must reach it through this one call, converged.
  __syncwarp();
  return fold_block<OP, V, false>(x, nvalid, shift, fma);
}

// One super-block (U warp-blocks of 32*V columns) folded by one warp; every lane returns it.
template <typename T, int OP, bool VEC, int U>
__device__ __forceinline__ float superblock(const T* __restrict__ xr, int64_t base, int64_t C, float shift, int fma, int lane) {
  constexpr int V = VecTraits<T>::V;
  constexpr int WB = 32 * V;
  float bv[U];
  if (VEC && base + (int64_t)U * WB <= C) {
    // whole super-block in range: issue all loads first
    uint4 raw[U];
#pragma unroll
    for (int u = 0; u < U; ++u) raw[u] = __ldg(reinterpret_cast<const uint4*>(xr + base + (int64_t)u * WB + lane * V));
#pragma unroll
    for (int u = 0; u < U; ++u) {
      float x[V];
      unpack<T>(raw[u], x);
      bv[u] = fold_block<OP, V, true>(x, V, shift, fma);
    }
  } else {
#pragma unroll
    for (int u = 0; u < U; ++u) bv[u] = load_fold<T, OP, VEC>(xr, base + (int64_t)u * WB + lane * V, C, shift, fma);
  }
#pragma unroll
  for (int off = 1; off < 32; off <<= 1)      // count-up butterfly: neighbours pair first
#pragma unroll
    for (int u = 0; u < U; ++u) bv[u] = f_add(bv[u], __shfl_xor_sync(0xffffffffu, bv[u], off));
#pragma unroll
  for (int s = 1; s < U; s <<= 1)
#pragma unroll
    for (int u = 0; u < U; u += 2 * s) bv[u] = f_add(bv[u], bv[u + s]);
  return bv[0];
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

// y = round((x * rinv) * w) for the V columns at `c` of one row.
template <typename T, bool VEC>
__device__ __forceinline__ void rms_scale_store(const ReduceParams& p, const T* __restrict__ xr, int64_t row, int64_t c,
                                                float rinv, bool out_vec) {
  constexpr int V = VecTraits<T>::V;
  float x[V], y[V];
  const bool full = c + V <= p.C;
  if (VEC && full) {
    unpack<T>(__ldg(reinterpret_cast<const uint4*>(xr + c)), x);
  } else {
#pragma unroll
    for (int t = 0; t < V; ++t) x[t] = (c + t) < p.C ? elem_to_f32(xr[c + t]) : 0.0f;
  }
  float w[V];
  const bool w_vec = full && p.weight && ((reinterpret_cast<uintptr_t>(p.weight) & 15) == 0) &&
                     p.w_dtype == (sizeof(T) == 2 ? RG_BF16 : RG_F32);
  if (w_vec) {
    unpack<T>(__ldg(reinterpret_cast<const uint4*>(static_cast<const T*>(p.weight) + c)), w);
  } else {
#pragma unroll
    for (int t = 0; t < V; ++t) w[t] = (p.weight && (c + t) < p.C) ? load_scalar(p.weight, p.w_dtype, c + t) : 1.0f;
  }
#pragma unroll
  for (int t = 0; t < V; ++t) y[t] = f_mul(f_mul(x[t], rinv), w[t]);
  if (out_vec && full) {
    if constexpr (sizeof(T) == 4) {
      *reinterpret_cast<uint4*>(static_cast<float*>(p.out) + row * p.ldo + c) =
          make_uint4(__float_as_uint(y[0]), __float_as_uint(y[1]), __float_as_uint(y[2]), __float_as_uint(y[3]));
    } else {
      *reinterpret_cast<uint4*>(static_cast<uint16_t*>(p.out) + row * p.ldo + c) =
          make_uint4(pack_bf16x2(y[0], y[1]), pack_bf16x2(y[2], y[3]), pack_bf16x2(y[4], y[5]), pack_bf16x2(y[6], y[7]));
    }
  } else {
#pragma unroll
    for (int t = 0; t < V; ++t)
      if ((c + t) < p.C) {
        if (p.out_dtype == RG_BF16) static_cast<__nv_bfloat16*>(p.out)[row * p.ldo + c + t] = __float2bfloat16_rn(y[t]);
        else static_cast<float*>(p.out)[row * p.ldo + c + t] = y[t];
      }
  }
}

template <typename T, bool VEC>
__device__ __forceinline__ bool rms_out_vec(const ReduceParams& p) {
  constexpr int V = VecTraits<T>::V;
  return VEC && ((reinterpret_cast<uintptr_t>(p.out) & 15) == 0) && (p.ldo % V == 0) &&
         (p.out_dtype == (sizeof(T) == 2 ? RG_BF16 : RG_F32));
}

__device__ __forceinline__ float rms_rinv(float ss, int64_t C, float eps) {
  const float ms = __fdiv_rn(ss, (float)C);
  return __fdiv_rn(1.0f, __fsqrt_rn(f_add(ms, eps)));
}

// ------------------------------------------------------------------ warp per row
template <typename T, int OP, bool VEC, int U>
__global__ void __launch_bounds__(256) reduce_rows_warp_kernel(const ReduceParams p) {
  static_assert(OP != OP_SOFTMAX, "the softmax normaliser re-reads its row: CTA kernel");
  constexpr int V = VecTraits<T>::V;
  constexpr int SBW = 32 * V * U;
  const int lane = threadIdx.x & 31;
  const int64_t warp0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  const int nsb = (int)((p.C + SBW - 1) / SBW);
  pdl_prologue();
  for (int64_t row = warp0; row < p.R; row += nwarps) {
    const T* xr = static_cast<const T*>(p.x) + row * p.ldx;
    float stk[MAX_LEVELS];
#pragma unroll
    for (int b = 0; b < MAX_LEVELS; ++b) stk[b] = NEG_ZERO;
    for (int sbi = 0; sbi < nsb; ++sbi) {
      float v = superblock<T, OP, VEC, U>(xr, (int64_t)sbi * SBW, p.C, 0.0f, p.fma, lane);
      // binary counter: a finished block of 2^b super-blocks meets its left sibling
      bool carry = true;
#pragma unroll
      for (int b = 0; b < MAX_LEVELS; ++b) {
        if (carry) {
          if ((sbi >> b) & 1) v = f_add(stk[b], v);
          else { stk[b] = v; carry = false; }
        }
      }
    }
    // leftovers: the lowest pending block moves up unchanged until it meets a sibling
    float root = NEG_ZERO;
    bool have = false;
#pragma unroll
    for (int b = 0; b < MAX_LEVELS; ++b) {
      if ((nsb >> b) & 1) {
        root = have ? f_add(stk[b], root) : stk[b];
        have = true;
      }
    }
    if (OP == OP_SUM) {
      if (lane == 0) static_cast<float*>(p.out)[row * p.ldo] = root;
    } else {
      const float rinv = rms_rinv(root, p.C, p.eps);
      if (lane == 0 && p.aux) p.aux[row] = rinv;
      const bool out_vec = rms_out_vec<T, VEC>(p);
      for (int64_t c = (int64_t)lane * V; c < p.C; c += 32 * V) rms_scale_store<T, VEC>(p, xr, row, c, rinv, out_vec);
    }
  }
}

// ------------------------------------------------------------------ CTA per row
template <typename T, int OP, bool VEC, int U>
__global__ void __launch_bounds__(1024) reduce_rows_cta_kernel(const ReduceParams p) {
  extern __shared__ float smem[];
  float* sb = smem;                     // 2 * cap floats (ping-pong)
  float* red = smem + 2 * p.cap;        // 32 floats for the order-free max
  constexpr int V = VecTraits<T>::V;
  constexpr int SBW = 32 * V * U;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  const int nsb = (int)((p.C + SBW - 1) / SBW);
  pdl_prologue();
  for (int64_t row = blockIdx.x; row < p.R; row += gridDim.x) {
    const T* xr = static_cast<const T*>(p.x) + row * p.ldx;
    float shift = 0.0f;
    if (OP == OP_SOFTMAX) {
      // The row maximum rounds nothing, so its order is free (App. F).
      float m = -INFINITY;
      const int64_t nvec = VEC ? p.C / V : 0;
      for (int64_t i = threadIdx.x; i < nvec; i += blockDim.x) {
        float x[V];
        unpack<T>(__ldg(reinterpret_cast<const uint4*>(xr) + i), x);
#pragma unroll
        for (int t = 0; t < V; ++t) m = fmaxf(m, x[t]);
      }
      for (int64_t c = nvec * V + threadIdx.x; c < p.C; c += blockDim.x) m = fmaxf(m, elem_to_f32(xr[c]));
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
      if (lane == 0) red[warp] = m;
      __syncthreads();
      m = red[0];
      for (int w = 1; w < nwarps; ++w) m = fmaxf(m, red[w]);
      shift = m;
    }
    for (int sbi = warp; sbi < nsb; sbi += nwarps) {
      const float v = superblock<T, OP, VEC, U>(xr, (int64_t)sbi * SBW, p.C, shift, p.fma, lane);
      if (lane == 0) sb[sbi] = v;
    }
    __syncthreads();
    // remaining levels over the nsb super-block values
    int n = nsb;
    float* cur = sb;
    float* nxt = sb + p.cap;
    while (n > 32) {
      const int half = (n + 1) >> 1;
      for (int t = threadIdx.x; t < half; t += blockDim.x)
        nxt[t] = (2 * t + 1 < n) ? f_add(cur[2 * t], cur[2 * t + 1]) : cur[2 * t];
      __syncthreads();
      float* tmp = cur; cur = nxt; nxt = tmp;
      n = half;
    }
    float root = (lane < n) ? cur[lane] : NEG_ZERO;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) root = f_add(root, __shfl_xor_sync(0xffffffffu, root, off));
    __syncthreads();                    // scratch is reused by the next row
    if (OP == OP_SUM) {
      if (threadIdx.x == 0) static_cast<float*>(p.out)[row * p.ldo] = root;
    } else if (OP == OP_SOFTMAX) {
      if (threadIdx.x == 0) {
        static_cast<float*>(p.out)[row * p.ldo] = root;
        if (p.aux) p.aux[row] = shift;
      }
    } else {
      const float rinv = rms_rinv(root, p.C, p.eps);
      if (threadIdx.x == 0 && p.aux) p.aux[row] = rinv;
      const bool out_vec = rms_out_vec<T, VEC>(p);
      for (int64_t c = (int64_t)threadIdx.x * V; c < p.C; c += (int64_t)blockDim.x * V)
        rms_scale_store<T, VEC>(p, xr, row, c, rinv, out_vec);
    }
  }
}

// ------------------------------------------------------------------ RMSNorm, row kept in registers
// One CTA per row; every warp owns at most one super-block of U vectors per lane.  A row is read from memory
// exactly once and unpacked once (the unpacked values serve the fold and the scaling), the registers of its
// raw vectors then receive the next row's, and the thread's weights are unpacked once per CTA.  Needs 16-byte
// aligned rows whose length is a multiple of V.
template <typename T, int U>
__global__ void __launch_bounds__(256) rmsnorm_keep_kernel(const ReduceParams p) {
  __shared__ float sb[2][8];
  constexpr int V = VecTraits<T>::V;
  constexpr int WB = 32 * V;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  const bool out_vec = rms_out_vec<T, true>(p);
  const int64_t base = (int64_t)warp * WB * U + lane * V;
  const bool w_vec = p.weight && ((reinterpret_cast<uintptr_t>(p.weight) & 15) == 0) &&
                     p.w_dtype == (sizeof(T) == 2 ? RG_BF16 : RG_F32);
  pdl_prologue();
  auto load_row = [&](int64_t row, uint4 (&raw)[U]) {
    const T* xr = static_cast<const T*>(p.x) + row * p.ldx;
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int64_t c = base + (int64_t)u * WB;
      raw[u] = c + V <= p.C ? __ldg(reinterpret_cast<const uint4*>(xr + c)) : make_uint4(0, 0, 0, 0);
    }
  };
  // this thread's weights, unpacked once: they are the same for every row
  float w[U][V];
#pragma unroll
  for (int u = 0; u < U; ++u) {
    const int64_t c = base + (int64_t)u * WB;
    if (w_vec && c + V <= p.C) unpack<T>(__ldg(reinterpret_cast<const uint4*>(static_cast<const T*>(p.weight) + c)), w[u]);
    else {
#pragma unroll
      for (int t = 0; t < V; ++t) w[u][t] = (p.weight && c + t < p.C) ? load_scalar(p.weight, p.w_dtype, c + t) : 1.0f;
    }
  }
  uint4 raw[U];
  if ((int64_t)blockIdx.x < p.R) load_row(blockIdx.x, raw);
  int par = 0;
  for (int64_t row = blockIdx.x; row < p.R; row += gridDim.x, par ^= 1) {
    // the row is unpacked once; its raw vectors' registers then take the next row's vectors, which travel
    // while this row is folded, scaled and stored
    float x[U][V];
#pragma unroll
    for (int u = 0; u < U; ++u) unpack<T>(raw[u], x[u]);
    if (row + gridDim.x < p.R) load_row(row + gridDim.x, raw);
    float bv[U];
#pragma unroll
    for (int u = 0; u < U; ++u)
      bv[u] = (base + (int64_t)u * WB + V <= p.C) ? fold_block<OP_RMS, V, true>(x[u], V, 0.0f, p.fma) : NEG_ZERO;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1)
#pragma unroll
      for (int u = 0; u < U; ++u) bv[u] = f_add(bv[u], __shfl_xor_sync(0xffffffffu, bv[u], off));
#pragma unroll
    for (int s2 = 1; s2 < U; s2 <<= 1)
#pragma unroll
      for (int u = 0; u < U; u += 2 * s2) bv[u] = f_add(bv[u], bv[u + s2]);
    if (lane == 0) sb[par][warp] = bv[0];
    __syncthreads();                                      // one barrier per row: the totals alternate between two buffers
    float root = (lane < nwarps) ? sb[par][lane] : NEG_ZERO;   // nwarps <= 8 super-blocks, padded with the identity
#pragma unroll
    for (int off = 1; off < 8; off <<= 1) root = f_add(root, __shfl_xor_sync(0xffffffffu, root, off));
    root = __shfl_sync(0xffffffffu, root, 0);
    const float rinv = rms_rinv(root, p.C, p.eps);
    if (threadIdx.x == 0 && p.aux) p.aux[row] = rinv;
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int64_t c = base + (int64_t)u * WB;
      if (c + V > p.C) continue;
      float y[V];
#pragma unroll
      for (int t = 0; t < V; t += 2) {
        const float2 q = __fmul2_rn(__fmul2_rn(make_float2(x[u][t], x[u][t + 1]), make_float2(rinv, rinv)), make_float2(w[u][t], w[u][t + 1]));
        y[t] = q.x; y[t + 1] = q.y;
      }
      if (out_vec) {
        if constexpr (sizeof(T) == 4)
          *reinterpret_cast<uint4*>(static_cast<float*>(p.out) + row * p.ldo + c) =
              make_uint4(__float_as_uint(y[0]), __float_as_uint(y[1]), __float_as_uint(y[2]), __float_as_uint(y[3]));
        else
          *reinterpret_cast<uint4*>(static_cast<uint16_t*>(p.out) + row * p.ldo + c) =
              make_uint4(pack_bf16x2(y[0], y[1]), pack_bf16x2(y[2], y[3]), pack_bf16x2(y[4], y[5]), pack_bf16x2(y[6], y[7]));
      } else {
#pragma unroll
        for (int t = 0; t < V; ++t) {
          if (p.out_dtype == RG_BF16) static_cast<__nv_bfloat16*>(p.out)[row * p.ldo + c + t] = __float2bfloat16_rn(y[t]);
          else static_cast<float*>(p.out)[row * p.ldo + c + t] = y[t];
        }
      }
    }
  }
}

// ------------------------------------------------------------------ left fold (RG_TREE_LEFT)
// The other end of the work/depth range (Sec. 3.1): ((l0 + l1) + l2) + ..., a chain of C - 1 dependent adds
// per row.  A lane owns a row and walks it in column order; the warp moves 32 rows x 32 columns at a time
// through shared memory so that global accesses stay coalesced (row-major input, one 128-byte run per row
// and tile).  With `fma` the sum of squares is the chain acc = fma(x, x, acc) from acc = x0 * x0.
template <typename T, int OP>
__global__ void __launch_bounds__(256) reduce_rows_left_kernel(const ReduceParams p) {
  __shared__ float tile[8][32][33];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  float (*tw)[33] = tile[warp];
  pdl_prologue();
  auto load_tile = [&](int64_t rb, int64_t c0) {
#pragma unroll 8
    for (int i = 0; i < 32; ++i) {
      const int64_t r = rb + i, c = c0 + lane;
      tw[i][lane] = (r < p.R && c < p.C) ? elem_to_f32(static_cast<const T*>(p.x)[r * p.ldx + c]) : 0.0f;
    }
    __syncwarp();
  };
  for (int64_t rb = ((int64_t)blockIdx.x * 8 + warp) * 32; rb < p.R; rb += (int64_t)gridDim.x * 8 * 32) {
    const int64_t row = rb + lane;
    float shift = 0.0f;
    if (OP == OP_SOFTMAX) {
      float m = -INFINITY;                                // the maximum rounds nothing: any order (App. F)
      for (int64_t c0 = 0; c0 < p.C; c0 += 32) {
        load_tile(rb, c0);
        const int n = (int)min((int64_t)32, p.C - c0);
        for (int j = 0; j < n; ++j) m = fmaxf(m, tw[lane][j]);
        __syncwarp();
      }
      shift = m;
    }
    float acc = 0.0f;
    for (int64_t c0 = 0; c0 < p.C; c0 += 32) {
      load_tile(rb, c0);
      const int n = (int)min((int64_t)32, p.C - c0);
      for (int j = 0; j < n; ++j) {
        const float v = tw[lane][j];
        const bool first = c0 == 0 && j == 0;
        if (OP == OP_SUM) acc = first ? v : f_add(acc, v);
        else if (OP == OP_RMS) acc = first ? f_mul(v, v) : (p.fma ? f_fma(v, v, acc) : f_add(acc, f_mul(v, v)));
        else { const float e = exp_nonpositive(f_add(v, -shift)); acc = first ? e : f_add(acc, e); }
      }
      __syncwarp();
    }
    if (OP == OP_SUM) {
      if (row < p.R) static_cast<float*>(p.out)[row * p.ldo] = acc;
    } else if (OP == OP_SOFTMAX) {
      if (row < p.R) { static_cast<float*>(p.out)[row * p.ldo] = acc; if (p.aux) p.aux[row] = shift; }
    } else {
      const float rinv = rms_rinv(acc, p.C, p.eps);
      if (row < p.R && p.aux) p.aux[row] = rinv;
      for (int64_t c0 = 0; c0 < p.C; c0 += 32) {
        load_tile(rb, c0);
        const int n = (int)min((int64_t)32, p.C - c0);
        for (int j = 0; j < n; ++j) {
          const float w = p.weight ? load_scalar(p.weight, p.w_dtype, c0 + j) : 1.0f;
          tw[lane][j] = f_mul(f_mul(tw[lane][j], rinv), w);
        }
        __syncwarp();
        for (int i = 0; i < 32; ++i) {
          const int64_t r = rb + i, c = c0 + lane;
          if (r < p.R && c < p.C) {
            if (p.out_dtype == RG_BF16) static_cast<__nv_bfloat16*>(p.out)[r * p.ldo + c] = __float2bfloat16_rn(tw[i][lane]);
            else static_cast<float*>(p.out)[r * p.ldo + c] = tw[i][lane];
          }
        }
        __syncwarp();
      }
    }
  }
}

// Launch with programmatic stream serialisation (see pdl_prologue).
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), int grid, int threads, size_t smem, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid, 1, 1);
  cfg.blockDim = dim3((unsigned)threads, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, args...);
}

template <typename T, int OP, bool VEC, int U>
cudaError_t launch_kernel(const ReduceParams& p, bool warp_rows, int threads, int grid, size_t smem, cudaStream_t st) {
  if constexpr (OP != OP_SOFTMAX) {
    if (warp_rows) return launch_pdl(reduce_rows_warp_kernel<T, OP, VEC, U>, grid, threads, 0, st, p);
  }
  return launch_pdl(reduce_rows_cta_kernel<T, OP, VEC, U>, grid, threads, smem, st, p);
}

template <typename T, int OP, bool VEC>
cudaError_t launch_u(const ReduceParams& p, bool wr, int U, int threads, int grid, size_t smem, cudaStream_t st) {
  switch (U) {
    case 1: return launch_kernel<T, OP, VEC, 1>(p, wr, threads, grid, smem, st);
    case 2: return launch_kernel<T, OP, VEC, 2>(p, wr, threads, grid, smem, st);
    case 4: return launch_kernel<T, OP, VEC, 4>(p, wr, threads, grid, smem, st);
    default: return launch_kernel<T, OP, VEC, 8>(p, wr, threads, grid, smem, st);
  }
}

template <typename T, int OP>
cudaError_t launch_vec(const ReduceParams& p, bool vec, bool wr, int U, int threads, int grid, size_t smem, cudaStream_t st) {
  return vec ? launch_u<T, OP, true>(p, wr, U, threads, grid, smem, st)
             : launch_u<T, OP, false>(p, wr, U, threads, grid, smem, st);
}

template <typename T>
cudaError_t launch_op(int op, const ReduceParams& p, bool vec, bool wr, int U, int threads, int grid, size_t smem, cudaStream_t st) {
  switch (op) {
    case RG_OP_SUM: return launch_vec<T, OP_SUM>(p, vec, wr, U, threads, grid, smem, st);
    case RG_OP_RMSNORM: return launch_vec<T, OP_RMS>(p, vec, wr, U, threads, grid, smem, st);
    default: return launch_vec<T, OP_SOFTMAX>(p, vec, wr, U, threads, grid, smem, st);
  }
}

// y[i] = one of the specified exponentials on x[i] (see rg_selftest_exp)
__global__ void __launch_bounds__(256) exp_selftest_kernel(int form, const float* __restrict__ x, float* __restrict__ y, int64_t n) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
    const float v = x[i];
    y[i] = form == 0 ? rg_exp(v) : form == 1 ? rg_exp2(v) : form == 2 ? rg_exp_inrange(v) : exp_nonpositive(v);
  }
}

}  // namespace

rg_status_t launch_exp_selftest(int form, const float* x, float* y, int64_t n, cudaStream_t st) {
  const int64_t need = (n + 255) / 256;
  exp_selftest_kernel<<<(unsigned)(need < 148 * 8 ? need : 148 * 8), 256, 0, st>>>(form, x, y, n);
  return cudaGetLastError() == cudaSuccess ? RG_OK : RG_ERR_CUDA;
}

// Host launcher.  Speed knobs only (0 = choose): threads_hint = threads per row, where 32 selects
// the warp-per-row kernel for sums and RMSNorm; unroll_hint = warp-blocks in flight per warp.
rg_status_t launch_reduce_rows(int op, int tree, int fma, const rg_tensor_t* x, const rg_tensor_t* out,
                               const rg_reduce_args_t* args, int threads_hint, int unroll_hint,
                               cudaStream_t st) {
  if (tree == RG_TREE_LEFT) {
    ReduceParams p;
    p.x = x->ptr; p.out = out->ptr;
    p.weight = args ? args->weight : nullptr;
    p.aux = args ? static_cast<float*>(args->aux_out) : nullptr;
    p.R = x->rows; p.C = x->cols; p.ldx = x->ld; p.ldo = out->ld;
    p.eps = args ? args->eps : 0.0f;
    p.fma = fma; p.out_dtype = out->dtype; p.w_dtype = args ? args->weight_dtype : RG_F32; p.cap = 0;
    const int64_t need = (x->rows + 255) / 256, max_grid = (int64_t)current_device().sms * 8;
    const int grid = (int)(need < max_grid ? need : max_grid);
    cudaError_t e;
    if (x->dtype == RG_BF16)
      e = op == RG_OP_SUM ? launch_pdl(reduce_rows_left_kernel<uint16_t, OP_SUM>, grid, 256, 0, st, p)
        : op == RG_OP_RMSNORM ? launch_pdl(reduce_rows_left_kernel<uint16_t, OP_RMS>, grid, 256, 0, st, p)
                              : launch_pdl(reduce_rows_left_kernel<uint16_t, OP_SOFTMAX>, grid, 256, 0, st, p);
    else
      e = op == RG_OP_SUM ? launch_pdl(reduce_rows_left_kernel<float, OP_SUM>, grid, 256, 0, st, p)
        : op == RG_OP_RMSNORM ? launch_pdl(reduce_rows_left_kernel<float, OP_RMS>, grid, 256, 0, st, p)
                              : launch_pdl(reduce_rows_left_kernel<float, OP_SOFTMAX>, grid, 256, 0, st, p);
    return e == cudaSuccess ? RG_OK : RG_ERR_CUDA;
  }
  const int V = x->dtype == RG_BF16 ? 8 : 4;
  const int64_t C = x->cols, R = x->rows;
  const size_t esz = x->dtype == RG_BF16 ? 2 : 4;
  const int64_t nblocks = (C + 32 * V - 1) / (32 * V);          // warp-blocks in a row
  int U = unroll_hint;
  if (U != 1 && U != 2 && U != 4 && U != 8) {
    // four vectors per lane and step keep enough bytes in flight without starving the CTA of warps
    U = op == RG_OP_SOFTMAX_DENOM ? (nblocks >= 8 ? 8 : nblocks >= 4 ? 4 : nblocks >= 2 ? 2 : 1)
                                  : (nblocks >= 4 ? 4 : nblocks >= 2 ? 2 : 1);
  }
  const int64_t nsb = (nblocks + U - 1) / U;
  if (nsb >= (1 << (MAX_LEVELS - 1))) return RG_ERR_UNSUPPORTED;   // rows beyond ~4M fp32 columns
  const int sms = current_device().sms;

  int threads = threads_hint;
  const bool valid_hint = threads == 32 || threads == 64 || threads == 128 || threads == 256 || threads == 512 || threads == 1024;
  bool warp_rows;
  if (valid_hint) {
    warp_rows = (threads == 32) && op != RG_OP_SOFTMAX_DENOM;
  } else if (op == RG_OP_SOFTMAX_DENOM) {
    // The second pass re-reads the row from L2.  CTAs of 256 threads measured best on 32768-column
    // rows (four are resident per SM at this kernel's register count): enough CTAs in different
    // phases to overlap the DRAM-bound maximum pass with the ALU-bound exp pass, few enough rows in
    // flight for the second pass to find its row in L2 (forcing more resident CTAs was slower).
    warp_rows = false;
    threads = 256;
    while (threads > 32 && nsb < threads / 32) threads /= 2;
  } else {
    // One CTA per row with (about) the whole row in flight at once: the CTAs resident at any moment
    // then read a few long contiguous runs instead of thousands of short ones 128 KB apart, which
    // DRAM serves with far fewer page misses (measured: 7.3 vs 6.7 TB/s on 32768-column rows,
    // 7.3 vs 6.3 TB/s on 4096-column rows).  Rows of one warp-block take the barrier-free kernel.
    threads = 32;
    while (threads < 1024 && threads / 32 < nsb) threads *= 2;
    warp_rows = threads == 32;
  }
  const bool vec = (reinterpret_cast<uintptr_t>(x->ptr) % 16 == 0) && ((x->ld * esz) % 16 == 0);
  ReduceParams p;
  p.x = x->ptr; p.out = out->ptr;
  p.weight = args ? args->weight : nullptr;
  p.aux = args ? static_cast<float*>(args->aux_out) : nullptr;
  p.R = R; p.C = C; p.ldx = x->ld; p.ldo = out->ld;
  p.eps = args ? args->eps : 0.0f;
  p.fma = fma; p.out_dtype = out->dtype; p.w_dtype = args ? args->weight_dtype : RG_F32; p.cap = 0;

  // RMSNorm of rows short enough to live in registers: each row is read once.
  if (op == RG_OP_RMSNORM && !valid_hint && vec && C % V == 0 && nblocks <= 32) {
    // vectors per lane: a thread keeps its part of the row, its weights and the next row's raw vectors in
    // registers (64 with two bf16 vectors, 113 with four), and the SM needs about 70 KB in flight to keep DRAM
    // busy: two vectors per lane wherever the row then fits eight warps (bf16 4096 columns: 5.7 TB/s against 5.4
    // with four; fp32 rows measured level, the shortest best with one)
    const int Uk = x->dtype == RG_BF16 ? (nblocks > 16 ? 4 : nblocks >= 2 ? 2 : 1) : (nblocks >= 16 ? 4 : nblocks > 8 ? 2 : 1);
    const int warps = (int)((nblocks + Uk - 1) / Uk);          // <= 8
    // every CTA takes the same number of rows (8192 rows on 2368 resident CTAs would leave a last round half
    // empty: four rows each on 2048 CTAs instead)
    void (*kern)(const ReduceParams);
    if (x->dtype == RG_BF16) kern = Uk == 4 ? rmsnorm_keep_kernel<uint16_t, 4> : Uk == 2 ? rmsnorm_keep_kernel<uint16_t, 2> : rmsnorm_keep_kernel<uint16_t, 1>;
    else kern = Uk == 4 ? rmsnorm_keep_kernel<float, 4> : Uk == 2 ? rmsnorm_keep_kernel<float, 2> : rmsnorm_keep_kernel<float, 1>;
    int per_sm = 0;                                        // CTAs of this kernel an SM holds (registers decide)
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, warps * 32, 0) != cudaSuccess || per_sm < 1) per_sm = 2048 / (warps * 32) / 2;
    const int64_t max_grid = (int64_t)sms * per_sm;
    const int64_t rows_per_cta = (R + max_grid - 1) / max_grid;
    const int grid = (int)((R + rows_per_cta - 1) / rows_per_cta);
    return launch_pdl(kern, grid, warps * 32, 0, st, p) == cudaSuccess ? RG_OK : RG_ERR_CUDA;
  }
  const int cap = (int)((nsb + 31) / 32 * 32);
  size_t smem = 0;
  int grid;
  if (warp_rows) {
    threads = 256;
    const int64_t need = (R + 7) / 8, max_grid = (int64_t)sms * 8;
    grid = (int)(need < max_grid ? need : max_grid);
  } else {
    smem = (size_t)(2 * cap + 32) * sizeof(float);
    const int64_t max_grid = (int64_t)sms * (2048 / threads);
    grid = (int)(R < max_grid ? R : max_grid);
  }
  p.cap = cap;
  cudaError_t e = x->dtype == RG_BF16 ? launch_op<uint16_t>(op, p, vec, warp_rows, U, threads, grid, smem, st)
                                      : launch_op<float>(op, p, vec, warp_rows, U, threads, grid, smem, st);
  return e == cudaSuccess ? RG_OK : RG_ERR_CUDA;
}

rg_status_t read_and_clear_reduce_status(uint32_t* code) {
  unsigned int v = 0, zero = 0;
  if (cudaMemcpyFromSymbol(&v, g_reduce_status_word, sizeof(v)) != cudaSuccess) return RG_ERR_CUDA;
  if (v != 0 && cudaMemcpyToSymbol(g_reduce_status_word, &zero, sizeof(zero)) != cudaSuccess) return RG_ERR_CUDA;
  if (code) *code = v;
  return v ? RG_ERR_TIMEOUT : RG_OK;
}

}  // namespace rg
