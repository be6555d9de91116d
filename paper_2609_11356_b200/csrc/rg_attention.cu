// Attention with a fixed reduction order (App. F): per query row the keys are walked in blocks
// of width w; each block contributes one rescale of the running output and denominator, so w,
// the row-sum tree, the type the probabilities are narrowed to and the place of the division
// are all part of the arithmetic and all come from the descriptor.
//
// One CTA owns 128 query rows of one head.  Per key block j:
//   warp 0 (TMA)      K_j [w x d] into one stage (refilled as soon as the scores that read it are done, a
//                     whole block before it is needed) and Vt_j [d x w] into a two-stage ring (Q once)
//   warp 1 (MMA)      the whole warp walks the loop, an elected lane issues.
//                     S = Q K_j^T   d/16 tcgen05.mma steps from a zero accumulator, ascending k; the
//                     scores of block j+1 are issued before the P V product of block j (two score
//                     accumulators in tensor memory), so the softmax threads never wait for scores
//                     PV = P Vt_j^T w/16 steps from a zero accumulator, ascending key, into one of two
//                     product accumulators (probabilities are double-buffered in shared memory too)
//   warps 2-17        four threads per query row (its TMEM lane), each with a quarter of the block's keys
//                     and a quarter of the output columns; partial maxima and partial row sums (subtrees
//                     of the same tree) meet in shared memory, one barrier per block:
//                     s_t = acc * scale; m_j = max(m_{j-1}, max_t s_t); alpha = exp(m_{j-1} - m_j);
//                     p_t = exp(s_t - m_j); l_j = alpha*l_{j-1} + TREE_t p_t (balanced tree over the
//                     block's keys in order); P = p narrowed to bf16, written to shared memory in the
//                     swizzled K-major layout the tensor core reads; O_j = alpha*O_{j-1} + PV, folded
//                     one block later so that the product has a whole block to finish
// and at the end O / l, one division, one rounding to the output type.  exp is one of the library's
// specified exponentials (rg_exp, or rg_exp2 with log2 e folded into the scale), not the hardware's.
// With causal masking the walk of a query tile stops at its own end, and the blocks from the tile's
// first row on add 0 (key <= query) or -1e6 (key > query) to every score before the maximum.  Keys past Nk are masked to
// -inf before the maximum, so their probabilities are exactly +0.
//
// Heads are stacked along the rows of Q [heads*Nq, d], K [heads*Nk, d], Vt [heads*d, Nk] and
// O [heads*Nq, d]; blockIdx.y is the head.  Rows of another head that a box may pick up at a head
// boundary are either masked (keys) or never stored (queries).
#include <cuda.h>

#include "rg_common.cuh"
#include "rg_internal.h"
#include "rg_ptx.cuh"

namespace rg {

__device__ unsigned int g_attn_status_word = 0;

namespace {

constexpr int QROWS = 128;          // query rows per CTA = TMEM lanes
constexpr int SPLIT = 4;            // threads per query row: each owns W / SPLIT keys and HD / SPLIT output columns
constexpr int SOFTMAX_THREADS = QROWS * SPLIT;
constexpr int ATT_THREADS = 64 + SOFTMAX_THREADS;    // warp 0 TMA, warp 1 MMA, then the softmax warps
constexpr int V_STAGES = 2;

// ---- PTX wrappers (tensor core side)
__device__ __forceinline__ void att_tma_load_2d(uint32_t dst, const CUtensorMap* map, int32_t x, int32_t y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void att_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void att_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void att_tmem_alloc(uint32_t dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
}
__device__ __forceinline__ void att_tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void att_tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void att_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void att_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void att_tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
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
__device__ __forceinline__ void att_tmem_ld32(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void att_tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// K-major tile with 128-byte rows and the 128-byte swizzle: 8-row groups 1024 bytes apart
__device__ __forceinline__ uint64_t att_kmajor_desc(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((smem_addr & 0x3ffffu) >> 4);
  d |= static_cast<uint64_t>(1) << 16;
  d |= static_cast<uint64_t>(1024 >> 4) << 32;
  d |= static_cast<uint64_t>(1) << 46;
  d |= static_cast<uint64_t>(2) << 61;
  return d;
}
// bf16 x bf16 -> fp32, both operands K-major, M = 128, N = n
__host__ __device__ constexpr uint32_t att_idesc(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(QROWS >> 4) << 24);
}

struct AttnParams {
  int32_t Nq, Nk;        // per head
  int32_t causal;        // query row i sees keys t <= i; the query tile is this CTA's 128 rows
  float scale;
  void* O;
  int64_t ldo;
  int32_t o_dtype;
};

// balanced "neighbours pair first" tree over 32 values in index order
// three-input maximum (one instruction on this architecture); NaN operands are ignored as in fmaxf
__device__ __forceinline__ float max3f(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}

// three-input minimum that returns NaN when any operand is NaN
__device__ __forceinline__ float min3f_nan(float a, float b, float c) {
  float r;
  asm("min.NaN.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}

// rg_exp2 for an argument in [-126, 0]: none of the range selects can fire and none is evaluated
// (same bits as rg_exp2 on that domain).
__device__ __forceinline__ float exp2_core(float x) {
  const float t = f_add(x, 12582912.0f);
  const float n = f_add(t, -12582912.0f);
  const float f = f_add(x, -n);
  float q = 0x1.ffcbfcp-17f;
  q = f_fma(q, f, 0x1.430912p-13f);
  q = f_fma(q, f, 0x1.5d87fep-10f);
  q = f_fma(q, f, 0x1.3b2ab6p-7f);
  q = f_fma(q, f, 0x1.c6b08ep-5f);
  q = f_fma(q, f, 0x1.ebfbe0p-3f);
  q = f_fma(q, f, 0x1.62e430p-1f);
  q = f_fma(q, f, 1.0f);
  return __int_as_float(__float_as_int(q) + (__float_as_int(t) << 23));      // t's low mantissa bits hold n
}

// rg_exp for an argument in [-87.33655, 0]: no range select can fire, n lies in [-126, 0], so 2^n is
// a normal number and the two-factor scaling of rg_exp equals one multiplication by it (scaling by
// a power of two is exact until the single final rounding).  Same bits as rg_exp on that domain.
__device__ __forceinline__ float exp_core(float x) {
  const float y = f_mul(x, 0x1.715476p+0f);
  const float t = f_add(y, 12582912.0f);
  const float n = f_add(t, -12582912.0f);
  float r = f_fma(n, -0x1.62e400p-1f, x);
  r = f_fma(n, -0x1.7f7d1cp-20f, r);
  float q = 0x1.a01a02p-13f;
  q = f_fma(q, r, 0x1.6c16c2p-10f);
  q = f_fma(q, r, 0x1.111112p-7f);
  q = f_fma(q, r, 0x1.555556p-5f);
  q = f_fma(q, r, 0x1.555556p-3f);
  q = f_fma(q, r, 0.5f);
  q = f_fma(q, r, 1.0f);
  q = f_fma(q, r, 1.0f);
  return f_mul(q, __int_as_float((__float_as_int(t) << 23) + 0x3f800000));   // t's low mantissa bits hold n
}

// exp_core on two arguments at once, with the packed fp32x2 instructions of this architecture
// (each half is one IEEE round-to-nearest operation, so every intermediate has the bits of the scalar form;
// x - n is written as fma(n, -1, x): the product is exact, so it is the same single rounding).  A thread then
// issues half as many floating-point instructions per key in the polynomial.  Only chains of fused multiply-adds
// are packed: a packed multiply feeding a packed add is contracted into one packed fma by the assembler even
// when both carry an explicit rounding mode (measured: 1 % of such pairs change their last bit), so the
// score scaling (multiply, then subtract the maximum) and the fold O = a * O + PV stay scalar, and so does the
// first multiply here: with y = x * log2(e) packed in front of the packed add that rounds it to an integer, 12 of
// the 1,118,743,633 arguments of this form's domain came out with another n and other bits (an exhaustive
// comparison with the scalar form; with the scalar multiply: none).  rg_selftest_exp exposes this function.
__device__ __forceinline__ float2 splat2(float v) { return make_float2(v, v); }
__device__ __forceinline__ float2 exp_core2(float2 x) {
  const float2 y = make_float2(f_mul(x.x, 0x1.715476p+0f), f_mul(x.y, 0x1.715476p+0f));
  const float2 t = __fadd2_rn(y, splat2(12582912.0f));
  const float2 n = __fadd2_rn(t, splat2(-12582912.0f));
  float2 r = __ffma2_rn(n, splat2(-0x1.62e400p-1f), x);
  r = __ffma2_rn(n, splat2(-0x1.7f7d1cp-20f), r);
  float2 q = splat2(0x1.a01a02p-13f);
  q = __ffma2_rn(q, r, splat2(0x1.6c16c2p-10f));
  q = __ffma2_rn(q, r, splat2(0x1.111112p-7f));
  q = __ffma2_rn(q, r, splat2(0x1.555556p-5f));
  q = __ffma2_rn(q, r, splat2(0x1.555556p-3f));
  q = __ffma2_rn(q, r, splat2(0.5f));
  q = __ffma2_rn(q, r, splat2(1.0f));
  q = __ffma2_rn(q, r, splat2(1.0f));
  return __fmul2_rn(q, make_float2(__int_as_float((__float_as_int(t.x) << 23) + 0x3f800000), __int_as_float((__float_as_int(t.y) << 23) + 0x3f800000)));
}

// rg_exp2 for an argument that is <= 0 or NaN: the overflow select can never fire and is left out
// (same bits as rg_exp2 on that domain).
__device__ __forceinline__ float exp2_nonpositive(float x) {
  const float t = f_add(x, 12582912.0f);
  const float n = f_add(t, -12582912.0f);
  const float f = f_add(x, -n);
  float q = 0x1.ffcbfcp-17f;
  q = f_fma(q, f, 0x1.430912p-13f);
  q = f_fma(q, f, 0x1.5d87fep-10f);
  q = f_fma(q, f, 0x1.3b2ab6p-7f);
  q = f_fma(q, f, 0x1.c6b08ep-5f);
  q = f_fma(q, f, 0x1.ebfbe0p-3f);
  q = f_fma(q, f, 0x1.62e430p-1f);
  q = f_fma(q, f, 1.0f);
  float e = __int_as_float(__float_as_int(q) + (__float_as_int(t) << 23));   // t's low mantissa bits hold n
  e = x < -126.0f ? 0.0f : e;
  return x != x ? x : e;
}

__device__ __forceinline__ float tree32(const float (&p)[16]) {
  float a[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) a[i] = f_add(p[2 * i], p[2 * i + 1]);
#pragma unroll
  for (int i = 0; i < 4; ++i) a[i] = f_add(a[2 * i], a[2 * i + 1]);
  return f_add(f_add(a[0], a[1]), f_add(a[2], a[3]));
}
__device__ __forceinline__ float tree32(const float (&p)[32]) {
  float a[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) a[i] = f_add(p[2 * i], p[2 * i + 1]);
#pragma unroll
  for (int i = 0; i < 8; ++i) a[i] = f_add(a[2 * i], a[2 * i + 1]);
#pragma unroll
  for (int i = 0; i < 4; ++i) a[i] = f_add(a[2 * i], a[2 * i + 1]);
  return f_add(f_add(a[0], a[1]), f_add(a[2], a[3]));
}

// W = key block width (64 or 128), HD = head dimension (64 or 128), BASE2 = base-two exponential
template <int W, int HD, bool BASE2>
__global__ void __launch_bounds__(ATT_THREADS, 1)
attention_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                 const __grid_constant__ CUtensorMap tmap_vt, const AttnParams p) {
  constexpr uint32_t Q_BOX = QROWS * 128;                 // bytes of one [128 rows x 64 columns] box
  constexpr uint32_t K_BOX = W * 128;                     // [W keys x 64 columns of d]
  constexpr uint32_t V_BOX = HD * 128;                    // [HD rows of Vt x 64 keys]
  constexpr uint32_t P_BOX = QROWS * 128;                 // [128 rows x 64 keys]
  constexpr int DB = HD / 64, WB = W / 64;                // boxes along d and along the keys
  constexpr uint32_t Q_BYTES = DB * Q_BOX, K_BYTES = DB * K_BOX, V_BYTES = WB * V_BOX, P_BYTES = WB * P_BOX;
  constexpr uint32_t TMEM_COLS = 512;                     // S of block j at columns [128*(j&1), ... + W), P V of block j at [256 + 128*(j&1), ... + HD)
  constexpr uint32_t IDESC_S = att_idesc(W), IDESC_PV = att_idesc(HD);

  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  // one K box set (the next block's keys are fetched as soon as the scores that read this one are
  // done, a whole block before they are needed), two V stages, two P buffers
  const uint32_t sQ = smem_base, sK = sQ + Q_BYTES, sV0 = sK + K_BYTES, sP = sV0 + V_STAGES * V_BYTES;
  uint8_t* sP_gen = smem_gen + Q_BYTES + K_BYTES + V_STAGES * V_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem_gen + Q_BYTES + K_BYTES + V_STAGES * V_BYTES + 2 * P_BYTES);
  // barriers: q_full, k_full, k_empty, pv_full[2], v_full[2], v_empty[2], s_full[2], p_full
  const uint32_t bar_q = smem_u32(bars);
  const uint32_t bar_k_full = bar_q + 8u, bar_k_empty = bar_k_full + 8u;
  const uint32_t bar_pv = bar_k_empty + 8u;
  const uint32_t bar_v_full = bar_pv + 16u, bar_v_empty = bar_v_full + 16u;
  const uint32_t bar_s = bar_v_empty + 16u, bar_p = bar_s + 16u;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 13);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  float* xm = reinterpret_cast<float*>(bars + 14);        // [2][SPLIT][128] partial maxima of the parts of a row, by block parity
  float* xs = xm + 2 * SPLIT * QROWS;                     // [2][SPLIT][128] partial row sums, by block parity

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int head = blockIdx.y;
  // causal walks grow with the tile index: the long ones are scheduled first
  const int q0 = (p.causal ? (int)(gridDim.x - 1 - blockIdx.x) : (int)blockIdx.x) * QROWS;   // first query row of this CTA within the head
  // causal: the walk stops at the end of the query tile; the blocks from q0 on straddle the diagonal
  const int kend = p.causal ? min(p.Nk, q0 + QROWS) : p.Nk;
  const int nblocks = (kend + W - 1) / W;

  if (threadIdx.x == 0) {
    mbar_init(bar_q, 1);
    mbar_init(bar_k_full, 1); mbar_init(bar_k_empty, 1);
    for (int s = 0; s < 2; ++s) {
      mbar_init(bar_v_full + 8u * s, 1); mbar_init(bar_v_empty + 8u * s, 1);
      mbar_init(bar_s + 8u * s, 1); mbar_init(bar_pv + 8u * s, 1);
    }
    mbar_init(bar_p, SOFTMAX_THREADS / 32);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    att_tmem_alloc(smem_u32(tmem_slot), TMEM_COLS);
    att_tmem_relinquish();
  }
  att_fence_before();
  __syncthreads();
  att_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      mbar_expect_tx(bar_q, Q_BYTES);
#pragma unroll
      for (int b = 0; b < DB; ++b) att_tma_load_2d(sQ + b * Q_BOX, &tmap_q, b * 64, head * p.Nq + q0, bar_q);
      for (int j = 0; j < nblocks; ++j) {
        const int stage = j & 1; const uint32_t phase = (j >> 1) & 1;
        if (!mbar_wait(bar_k_empty, (j & 1) ^ 1u, abort_flag, &g_attn_status_word, 0x1100u)) break;
        mbar_expect_tx(bar_k_full, K_BYTES);
#pragma unroll
        for (int b = 0; b < DB; ++b) att_tma_load_2d(sK + b * K_BOX, &tmap_k, b * 64, head * p.Nk + j * W, bar_k_full);
        if (!mbar_wait(bar_v_empty + 8u * stage, phase ^ 1u, abort_flag, &g_attn_status_word, 0x1180u | stage)) break;
        mbar_expect_tx(bar_v_full + 8u * stage, V_BYTES);
#pragma unroll
        for (int b = 0; b < WB; ++b) att_tma_load_2d(sV0 + stage * V_BYTES + b * V_BOX, &tmap_vt, j * W + b * 64, head * HD, bar_v_full + 8u * stage);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    // the whole warp walks the loop converged and an elected lane issues, so that the descriptor
    // arithmetic stays in the uniform datapath the tensor-core instruction reads its operands from
    {
      const bool leader = elect_one();
      bool alive = warp_mbar_wait(bar_q, 0, abort_flag, &g_attn_status_word, 0x1200u);
      // S_j = Q K_j^T into score accumulator j&1: ascending k over the head dimension, from zero
      auto issue_scores = [&](int j) -> bool {
        const int stage = j & 1;
        if (!warp_mbar_wait(bar_k_full, j & 1, abort_flag, &g_attn_status_word, 0x1300u)) return false;
        att_fence_after();
#pragma unroll
        for (int b = 0; b < DB; ++b) {
          const uint64_t adesc = att_kmajor_desc(sQ + b * Q_BOX), bdesc = att_kmajor_desc(sK + b * K_BOX);
#pragma unroll
          for (int a = 0; a < 4; ++a) if (leader) att_mma_bf16(tmem_base + 128u * stage, adesc + 2u * a, bdesc + 2u * a, IDESC_S, (b | a) ? 1u : 0u);
        }
        if (leader) att_commit(bar_s + 8u * stage);
        if (leader) att_commit(bar_k_empty);
        return true;
      };
      if (alive) alive = issue_scores(0);
      for (int j = 0; j < nblocks && alive; ++j) {
        // The next block's scores go first.  Their accumulator held block j-1's scores, which the
        // softmax threads had finished reading before they released P_{j-1} (waited for below, one
        // turn ago).
        if (j + 1 < nblocks && !issue_scores(j + 1)) break;
        // PV = P Vt^T: ascending key over the block, from zero, once the probabilities are in shared memory.
        // Probabilities and product alternate between two buffers: the softmax threads folded the
        // product of block j-2 and saw it complete before they wrote these probabilities.
        const int stage = j & 1; const uint32_t phase = (j >> 1) & 1;
        if (!warp_mbar_wait(bar_p, j & 1, abort_flag, &g_attn_status_word, 0x1400u)) break;
        if (!warp_mbar_wait(bar_v_full + 8u * stage, phase, abort_flag, &g_attn_status_word, 0x1480u | stage)) break;
        att_fence_after();
        const uint32_t sV = sV0 + stage * V_BYTES, sPj = sP + stage * P_BYTES;
#pragma unroll
        for (int b = 0; b < WB; ++b) {
          const uint64_t adesc = att_kmajor_desc(sPj + b * P_BOX), bdesc = att_kmajor_desc(sV + b * V_BOX);
#pragma unroll
          for (int a = 0; a < 4; ++a) if (leader) att_mma_bf16(tmem_base + 256u + 128u * stage, adesc + 2u * a, bdesc + 2u * a, IDESC_PV, (b | a) ? 1u : 0u);
        }
        if (leader) att_commit(bar_pv + 8u * stage);
        if (leader) att_commit(bar_v_empty + 8u * stage);               // the stage may be refilled once these steps have read it
      }
    }
  } else {
    // ------------------------------------------------------------ softmax and output rows
    const int quarter = warp & 3;                           // TMEM lanes [32*quarter, 32*quarter + 32)
    const int part = (warp - 2) >> 2;                       // which part of the keys and of the output columns
    const int r = quarter * 32 + lane;                      // row of the tile
    const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
    constexpr int KH = W / SPLIT, OH = HD / SPLIT;          // keys and output columns per thread
    constexpr int CK = KH < 32 ? KH : 32, CO = OH < 32 ? OH : 32;   // widths of one tensor-memory load
    const int kbase = part * KH, obase = part * OH;
    float m = -INFINITY, l = 0.0f;
    float O[OH];
#pragma unroll
    for (int c = 0; c < OH; ++c) O[c] = 0.0f;
    // O = a * O + PV on this thread's output columns
    auto fold_pv = [&](float a, int buf) {
      att_fence_after();
#pragma unroll
      for (int ci = 0; ci < OH / CO; ++ci) {
        uint32_t raw[CO];
        att_tmem_ld32(t_row + 256u + 128u * buf + obase + ci * CO, raw);
        att_tmem_ld_wait();
#pragma unroll
        for (int c = 0; c < CO; ++c) O[ci * CO + c] = f_add(f_mul(a, O[ci * CO + c]), __uint_as_float(raw[c]));
      }
      att_fence_before();
    };
    // the row's value from the SPLIT parts, paired as the balanced tree pairs them
    auto row_max = [&](const float* x) {
      float v = fmaxf(x[r], x[QROWS + r]);
#pragma unroll
      for (int q = 2; q < SPLIT; q += 2) v = fmaxf(v, fmaxf(x[q * QROWS + r], x[(q + 1) * QROWS + r]));
      return v;
    };
    auto row_sum = [&](const float* x) {
      if (SPLIT == 2) return f_add(x[r], x[QROWS + r]);
      return f_add(f_add(x[r], x[QROWS + r]), f_add(x[2 * QROWS + r], x[3 * QROWS + r]));
    };
    float alpha_prev = 0.0f;
    // A wait that gives up leaves this thread walking the loop without touching tensor memory, so
    // that the barriers of all softmax threads below are still met by everyone.
    bool alive = true;
    for (int j = 0; j < nblocks; ++j) {
      if (alive) alive = mbar_wait(bar_s + 8u * (j & 1), (j >> 1) & 1, abort_flag, &g_attn_status_word, 0x1500u);
      const uint32_t t_s = t_row + 128u * (j & 1);          // this block's score accumulator
      const int live = min(W, kend - j * W);                // keys of this block that exist
      const bool diagonal = p.causal && j * W >= q0;        // scores take the 0 / -1e6 offset (App. F)
      const int qi = q0 + r;                                // this row's query index within the head
      // pass 1: the maximum over this thread's keys, then over the row
      float mb = -INFINITY;
      if (alive) {
        att_fence_after();
#pragma unroll
        for (int c0 = 0; c0 < KH; c0 += CK) {
          uint32_t raw[CK];
          att_tmem_ld32(t_s + kbase + c0, raw);
          att_tmem_ld_wait();
          if (diagonal) {
#pragma unroll
            for (int c = 0; c < CK; ++c) {
              const int t = kbase + c0 + c;
              float sc = t < live ? f_mul(__uint_as_float(raw[c]), p.scale) : -INFINITY;
              sc = f_add(sc, j * W + t <= qi ? 0.0f : -1.0e6f);
              mb = fmaxf(mb, sc);
            }
          } else if (live == W) {                           // every key exists: no masking (all blocks but the last)
            if (p.scale > 0.0f) {
              // rounding a product by a positive scale is monotone, so the largest scaled score is the
              // scaled largest score: one multiply per load instead of one per key
              float rm = __uint_as_float(raw[0]);
#pragma unroll
              for (int c = 1; c + 1 < CK; c += 2) rm = max3f(rm, __uint_as_float(raw[c]), __uint_as_float(raw[c + 1]));
              rm = fmaxf(rm, __uint_as_float(raw[CK - 1]));
              mb = fmaxf(mb, f_mul(rm, p.scale));
            } else {
#pragma unroll
              for (int c = 0; c < CK; ++c) mb = fmaxf(mb, f_mul(__uint_as_float(raw[c]), p.scale));
            }
          } else {
#pragma unroll
            for (int c = 0; c < CK; ++c) {
              const float sc = kbase + c0 + c < live ? f_mul(__uint_as_float(raw[c]), p.scale) : -INFINITY;
              mb = fmaxf(mb, sc);
            }
          }
        }
      }
      float* xm_j = xm + (j & 1) * SPLIT * QROWS;
      xm_j[part * QROWS + r] = mb;
      // The only barrier of a block.  Behind it every thread of the row has also finished the block
      // before, so that block's partial row sums are complete; the exchange buffers alternate with
      // the block parity, and a thread can be at most one barrier ahead of another.
      asm volatile("bar.sync 1, %0;" ::"n"(SOFTMAX_THREADS) : "memory");
      const float m_new = fmaxf(m, row_max(xm_j));
      const float alpha = BASE2 ? rg_exp2(f_add(m, -m_new)) : rg_exp(f_add(m, -m_new));
      if (j > 0) l = f_add(f_mul(alpha_prev, l), row_sum(xs + ((j - 1) & 1) * SPLIT * QROWS));
      // pass 2: probabilities, the subtree of the row sum over this thread's keys, narrowed copies
      float psum = 0.0f;
      if (alive) {
        float chunk_sum[KH / CK];
#pragma unroll
        for (int ci = 0; ci < KH / CK; ++ci) {
          const int c0 = kbase + ci * CK;
          uint32_t raw[CK];
          att_tmem_ld32(t_s + c0, raw);
          att_tmem_ld_wait();
          float pr[CK];
          // the exponent x = s - m_new of every key: <= 0 (m_new bounds every score of the block), or NaN
          if (diagonal) {
#pragma unroll
            for (int c = 0; c < CK; ++c) {
              float sc = c0 + c < live ? f_mul(__uint_as_float(raw[c]), p.scale) : -INFINITY;
              sc = f_add(sc, j * W + c0 + c <= qi ? 0.0f : -1.0e6f);
              pr[c] = f_add(sc, -m_new);
            }
          } else if (live == W) {
#pragma unroll
            for (int c = 0; c < CK; ++c) pr[c] = f_add(f_mul(__uint_as_float(raw[c]), p.scale), -m_new);
          } else {
#pragma unroll
            for (int c = 0; c < CK; ++c) {
              const float sc = c0 + c < live ? f_mul(__uint_as_float(raw[c]), p.scale) : -INFINITY;
              pr[c] = f_add(sc, -m_new);
            }
          }
          {
            // the smallest exponent of the chunk, NaN if any is NaN: when it is above the underflow
            // threshold no element needs a range or NaN select of the specified exponential
            // (masked keys have x = -inf and take the selects)
            float xmin = pr[0];
#pragma unroll
            for (int c = 1; c + 1 < CK; c += 2) xmin = min3f_nan(xmin, pr[c], pr[c + 1]);
            xmin = min3f_nan(xmin, pr[CK - 1], pr[CK - 1]);
            if (xmin >= (BASE2 ? -126.0f : -87.33655f)) {
#pragma unroll
              if (BASE2) {
#pragma unroll
                for (int c = 0; c < CK; ++c) pr[c] = exp2_core(pr[c]);
              } else {
                // base e has three more floating-point operations per key than base two: packed, it gains 3 %
                // (452 against 437 TFLOP/s); base two does not (the threads wait on dependent results, not on issue slots)
#pragma unroll
                for (int c = 0; c < CK; c += 2) {
                  const float2 e2 = exp_core2(make_float2(pr[c], pr[c + 1]));
                  pr[c] = e2.x; pr[c + 1] = e2.y;
                }
              }
            } else {
#pragma unroll
              for (int c = 0; c < CK; ++c) pr[c] = BASE2 ? exp2_nonpositive(pr[c]) : rg_exp(pr[c]);
            }
          }
          chunk_sum[ci] = tree32(pr);
          // row r of the [128 x 64] box that holds keys c0..c0+CK-1: 16-byte pieces of 8 keys each
          uint8_t* box = sP_gen + (j & 1) * P_BYTES + (c0 >> 6) * P_BOX + (r >> 3) * 1024 + (r & 7) * 128;
#pragma unroll
          for (int q = 0; q < CK / 8; ++q) {
            const int piece = ((c0 & 63) >> 3) + q;         // 16-byte piece of the 128-byte row
            const uint4 v = make_uint4(pack_bf16x2(pr[8 * q], pr[8 * q + 1]), pack_bf16x2(pr[8 * q + 2], pr[8 * q + 3]),
                                       pack_bf16x2(pr[8 * q + 4], pr[8 * q + 5]), pack_bf16x2(pr[8 * q + 6], pr[8 * q + 7]));
            *reinterpret_cast<uint4*>(box + ((piece ^ (r & 7)) << 4)) = v;
          }
        }
        psum = KH / CK == 2 ? f_add(chunk_sum[0], chunk_sum[KH / CK - 1]) : chunk_sum[0];
      }
      xs[(j & 1) * SPLIT * QROWS + part * QROWS + r] = psum;
      // the tensor core reads shared memory through the async proxy; one arrival per warp once all
      // of its lanes have written and fenced their probabilities
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      att_fence_before();
      __syncwarp();
      if (lane == 0 && alive) mbar_arrive(bar_p);
      m = m_new;
      // The previous block's P V product has had this block's two passes to finish: fold it into O
      // (O_{j-1} = alpha_{j-1} O_{j-2} + P_{j-1} V_{j-1}).  Seeing it complete also licenses the
      // rewrite of its probability buffer two blocks after it was filled.
      if (j > 0) {
        if (alive) alive = mbar_wait(bar_pv + 8u * ((j - 1) & 1), ((j - 1) >> 1) & 1, abort_flag, &g_attn_status_word, 0x1600u);
        if (alive) fold_pv(alpha_prev, (j - 1) & 1);
      }
      alpha_prev = alpha;
    }
    asm volatile("bar.sync 1, %0;" ::"n"(SOFTMAX_THREADS) : "memory");
    l = f_add(f_mul(alpha_prev, l), row_sum(xs + ((nblocks - 1) & 1) * SPLIT * QROWS));
    if (alive) alive = mbar_wait(bar_pv + 8u * ((nblocks - 1) & 1), ((nblocks - 1) >> 1) & 1, abort_flag, &g_attn_status_word, 0x1700u);
    if (alive) fold_pv(alpha_prev, (nblocks - 1) & 1);
    // one division at the end, one rounding to the output type
    const int64_t row = (int64_t)q0 + r;
    if (alive && row < p.Nq) {
      const int64_t off = ((int64_t)head * p.Nq + row) * p.ldo + obase;
      float v[OH];
#pragma unroll
      for (int c = 0; c < OH; ++c) v[c] = __fdiv_rn(O[c], l);
      if (p.o_dtype == RG_F32) {
        float* dst = static_cast<float*>(p.O) + off;
#pragma unroll
        for (int c = 0; c < OH; ++c) dst[c] = v[c];
      } else {
        uint16_t* dst = static_cast<uint16_t*>(p.O) + off;
#pragma unroll
        for (int c = 0; c < OH; c += 2) *reinterpret_cast<uint32_t*>(dst + c) = pack_16x2(v[c], v[c + 1], p.o_dtype);
      }
    }
  }

  // ---------------------------------------------------------------- teardown
  __syncthreads();
  if (*abort_flag) {
    const uint64_t t0 = globaltimer_ns();
    while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 1) {
    att_fence_after();
    att_tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

template <int W, int HD>
size_t attn_smem_bytes() {
  return 1024 + (HD / 64) * QROWS * 128 + (HD / 64) * W * 128 + V_STAGES * (W / 64) * HD * 128 + 2 * (W / 64) * QROWS * 128 + 14 * 8 + 4 * SPLIT * QROWS * 4;
}

template <int W, int HD, bool BASE2>
cudaError_t launch_attention(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const AttnParams& p, dim3 grid,
                             cudaStream_t st) {
  const size_t smem = attn_smem_bytes<W, HD>();
  static DeviceOnce configured;                          // the attribute is per device
  const int dev = current_device().dev;
  if (!configured.has(dev)) {
    cudaError_t e = cudaFuncSetAttribute(attention_kernel<W, HD, BASE2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    configured.set(dev);
  }
  attention_kernel<W, HD, BASE2><<<grid, ATT_THREADS, smem, st>>>(tq, tk, tv, p);
  return cudaGetLastError();
}

// y[i] = one of this file's range-restricted exponentials on x[i] (see rg_selftest_exp)
__global__ void __launch_bounds__(256) exp_selftest_attention_kernel(int form, const float* __restrict__ x, float* __restrict__ y, int64_t n) {
  for (int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 2; i < n; i += (int64_t)gridDim.x * blockDim.x * 2) {
    const bool two = i + 1 < n;
    const float a = x[i], b = two ? x[i + 1] : x[i];
    float ra, rb;
    if (form == 3) { const float2 e = exp_core2(make_float2(a, b)); ra = e.x; rb = e.y; }
    else if (form == 4) { ra = exp2_core(a); rb = exp2_core(b); }
    else { ra = exp2_nonpositive(a); rb = exp2_nonpositive(b); }
    y[i] = ra;
    if (two) y[i + 1] = rb;
  }
}

}  // namespace

rg_status_t launch_exp_selftest_attention(int form, const float* x, float* y, int64_t n, cudaStream_t st) {
  const int64_t need = (n / 2 + 255) / 256 + 1;
  exp_selftest_attention_kernel<<<(unsigned)(need < 148 * 8 ? need : 148 * 8), 256, 0, st>>>(form, x, y, n);
  return cudaGetLastError() == cudaSuccess ? RG_OK : RG_ERR_CUDA;
}

// All arguments were validated by the caller: bf16 operands, d in {64, 128}, block_n in {64, 128},
// 16-byte aligned pointers, leading dimensions multiples of 8.
rg_status_t launch_attention_fixed(int block_n, int exp_base, int causal, float scale, int heads, const rg_tensor_t* Q, const rg_tensor_t* K,
                                   const rg_tensor_t* Vt, const rg_tensor_t* O, cudaStream_t st) {
  const int d = (int)Q->cols;
  const int64_t Nq = Q->rows / heads, Nk = K->rows / heads;
  CUtensorMap tq, tk, tv;
  if (!make_operand_tmap(&tq, Q->ptr, Q->dtype, Q->rows, Q->cols, Q->ld, QROWS) ||
      !make_operand_tmap(&tk, K->ptr, K->dtype, K->rows, K->cols, K->ld, block_n) ||
      !make_operand_tmap(&tv, Vt->ptr, Vt->dtype, Vt->rows, Vt->cols, Vt->ld, d))
    return RG_ERR_CUDA;
  AttnParams p;
  p.Nq = (int32_t)Nq; p.Nk = (int32_t)Nk; p.scale = scale; p.causal = causal;
  p.O = O->ptr; p.ldo = O->ld; p.o_dtype = O->dtype;
  const dim3 grid((unsigned)((Nq + QROWS - 1) / QROWS), (unsigned)heads, 1);
  cudaError_t err;
  const bool b2 = exp_base == 2;
  if (block_n == 128 && d == 128) err = b2 ? launch_attention<128, 128, true>(tq, tk, tv, p, grid, st) : launch_attention<128, 128, false>(tq, tk, tv, p, grid, st);
  else if (block_n == 64 && d == 128) err = b2 ? launch_attention<64, 128, true>(tq, tk, tv, p, grid, st) : launch_attention<64, 128, false>(tq, tk, tv, p, grid, st);
  else if (block_n == 128 && d == 64) err = b2 ? launch_attention<128, 64, true>(tq, tk, tv, p, grid, st) : launch_attention<128, 64, false>(tq, tk, tv, p, grid, st);
  else if (block_n == 64 && d == 64) err = b2 ? launch_attention<64, 64, true>(tq, tk, tv, p, grid, st) : launch_attention<64, 64, false>(tq, tk, tv, p, grid, st);
  else return RG_ERR_UNSUPPORTED;
  return err == cudaSuccess ? RG_OK : RG_ERR_CUDA;
}

rg_status_t read_and_clear_attn_status(uint32_t* code) {
  unsigned int v = 0, zero = 0;
  if (cudaMemcpyFromSymbol(&v, g_attn_status_word, sizeof(v)) != cudaSuccess) return RG_ERR_CUDA;
  if (v != 0 && cudaMemcpyToSymbol(g_attn_status_word, &zero, sizeof(zero)) != cudaSuccess) return RG_ERR_CUDA;
  if (code) *code = v;
  return v ? RG_ERR_TIMEOUT : RG_OK;
}

}  // namespace rg
