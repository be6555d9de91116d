// GEMV family (Sec. 3.2.2 "GEMV"): for a handful of rows the fold itself is spread over the lanes
// of a warp instead of an output tile over threads.  One warp owns one output column j (one row of
// B, read once, coalesced) and up to MR rows of A at a time:
//
//   lane   : owns tiles of 8 consecutive k (one 16-byte vector), streamed through shared memory by
//            asynchronous copies a few turns ahead of the arithmetic.  layout 0 (strided): tiles
//            lane, lane+32, lane+64, ...; layout 1 (contiguous): the lane-th run of
//            ceil(tiles/32) consecutive tiles.  Elements are folded in ascending k into one fp32
//            accumulator per (row, lane) with a scalar multiply-add: fused (one rounding) when the
//            descriptor's fma flag is set, multiply then add (two roundings) otherwise
//            (Sec. 3.2.1, scalar path).
//   warp   : the 32 lane totals are folded by a shuffle butterfly.  fold 0 counts the offsets up
//            (1,2,4,8,16): a balanced tree over the lanes in index order.  fold 1 counts them down
//            (16,...,1): a balanced tree over the lanes in bit-reversed order (a different sum).
//   then the same epilogue as the GEMM (bias, SiLU, residual, one rounding).
//
// This is a different bit class from the tensor-core path (atom = RG_ATOM_SCALAR); within the
// class every output element is independent of M, of the launch shape and of MR.
#include "rg_common.cuh"
#include "rg_internal.h"

namespace rg {

namespace {

struct GemvParams {
  const uint16_t* A;
  const uint16_t* B;
  void* C;
  int64_t lda, ldb, ldc;
  int32_t M, N, K;
  int32_t fma, layout, fold, c_dtype;
  int32_t b_static;       // 2: the caller's promise that neither operand is written by work in flight (loads do not wait for it)
  EpilogueArgs epi;
};

template <bool F16>
__device__ __forceinline__ float in_to_f32(uint32_t h) {
  return F16 ? f16_bits_to_f32(h) : bf16_bits_to_f32(h);
}

template <bool F16>
__device__ __forceinline__ void unpack8(const uint4& raw, float (&v)[8]) {
  const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
  for (int t = 0; t < 4; ++t) {
    v[2 * t] = in_to_f32<F16>(w[t] & 0xffffu);
    v[2 * t + 1] = in_to_f32<F16>(w[t] >> 16);
  }
}

template <bool FMA>
__device__ __forceinline__ float mul_add(float a, float b, float acc) {
  return FMA ? f_fma(a, b, acc) : f_add(acc, f_mul(a, b));
}

constexpr int GEMV_THREADS = 128;
// tiles of one lane per turn, and turns in the ring (one being folded, DEPTH-1 on their way):
// the same ring bytes for every MR, fewer tiles per turn where the rows need the registers
__host__ __device__ constexpr int gemv_unr(int mr) { return mr <= 2 ? 4 : mr <= 4 ? 2 : 1; }
__host__ __device__ constexpr int gemv_depth(int mr) { return mr <= 2 ? 3 : mr <= 4 ? 6 : 12; }

// 16 bytes global -> shared, asynchronously, past L1 (B is read once)
__device__ __forceinline__ void copy16_async(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void copy_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void copy_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Each lane streams its own tiles of the B row through its own slots of a shared-memory ring
// (slot (s, u) of lane l of warp w), so no lane reads what another lane copied and the only
// synchronisation is the lane's own wait on its copy groups.
template <int MR, bool F16, bool FMA>
__global__ void __launch_bounds__(GEMV_THREADS, 7) gemv_lane_tree_kernel(const GemvParams p) {
  constexpr int UNR = gemv_unr(MR), DEPTH = gemv_depth(MR);
  extern __shared__ __align__(16) uint4 gemv_ring[];
  const int lane = threadIdx.x & 31;
  uint4* const my = gemv_ring + (threadIdx.x >> 5) * (DEPTH * UNR * 32) + lane;
  const int64_t warp0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  const int tiles = (p.K + 7) >> 3;
  const int run = (tiles + 31) >> 5;
  // this lane's tiles: t_first, t_first + t_step, ... < t_end
  const int t_first = p.layout == 0 ? lane : lane * run;
  const int t_step = p.layout == 0 ? 32 : 1;
  const int t_end = p.layout == 0 ? tiles : min(tiles, (lane + 1) * run);
  // whole turns: UNR of this lane's tiles, all of them full (8 elements inside K)
  const int t_lim = min(t_end, p.K >> 3);
  const int n_full = t_lim > t_first ? (t_lim - t_first + t_step - 1) / t_step : 0;
  const int n_turns = n_full / UNR;
  // launched with programmatic stream serialisation: a kernel queued behind this one may start
  // its own set-up now, and this one reads nothing before the kernels ahead of it have finished
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  // (with the promise that neither operand is written by work in flight, b_static = 2, only the epilogue's reads and
  // the stores wait for the kernels ahead)
  bool deps_done = p.b_static < 2;
  if (deps_done) asm volatile("griddepcontrol.wait;" ::: "memory");
  for (int64_t j = warp0; j < p.N; j += nwarps) {
    const uint16_t* brow = p.B + j * p.ldb;
    for (int m0 = 0; m0 < p.M; m0 += MR) {
      float acc[MR];
#pragma unroll
      for (int r = 0; r < MR; ++r) acc[r] = 0.0f;
      // request turn i into ring slot s (an empty group when the lane has no such turn, so that
      // every lane counts groups alike)
      auto request = [&](int i, int s) {
        if (i < n_turns) {
#pragma unroll
          for (int u = 0; u < UNR; ++u)
            copy16_async(my + (s * UNR + u) * 32, brow + ((int64_t)(t_first + (i * UNR + u) * t_step) << 3));
        }
        copy_async_commit();
      };
#pragma unroll
      for (int i = 0; i < DEPTH - 1; ++i) request(i, i);
      int slot = 0, slot_req = DEPTH - 1;
      for (int i = 0; i < n_turns; ++i) {
        request(i + DEPTH - 1, slot_req);          // refills the slot folded one turn ago
        copy_async_wait<DEPTH - 1>();              // turn i has landed
        const int t = t_first + i * UNR * t_step;
        float w[UNR][8];
#pragma unroll
        for (int u = 0; u < UNR; ++u) unpack8<F16>(my[(slot * UNR + u) * 32], w[u]);
        // rows past M repeat the last row (their totals are not stored): no branch in the turn,
        // so all MR * UNR loads of A go out together
        uint4 araw[MR][UNR];
#pragma unroll
        for (int r = 0; r < MR; ++r) {
          const uint16_t* arow = p.A + (int64_t)min(m0 + r, p.M - 1) * p.lda;
#pragma unroll
          for (int u = 0; u < UNR; ++u) araw[r][u] = __ldg(reinterpret_cast<const uint4*>(arow + ((t + u * t_step) << 3)));
        }
#pragma unroll
        for (int u = 0; u < UNR; ++u) {
#pragma unroll
          for (int r = 0; r < MR; ++r) {
            float a[8];
            unpack8<F16>(araw[r][u], a);
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[r] = mul_add<FMA>(a[e], w[u][e], acc[r]);   // ascending k
          }
        }
        slot = slot + 1 == DEPTH ? 0 : slot + 1;
        slot_req = slot_req + 1 == DEPTH ? 0 : slot_req + 1;
      }
      copy_async_wait<0>();
      int t = t_first + n_turns * UNR * t_step;
      for (; t < t_end; t += t_step) {
        const int k = t << 3;
        if (k + 8 <= p.K) {
          float w[8];
          unpack8<F16>(__ldg(reinterpret_cast<const uint4*>(brow + k)), w);
#pragma unroll
          for (int r = 0; r < MR; ++r) {
            if (m0 + r < p.M) {
              float a[8];
              unpack8<F16>(__ldg(reinterpret_cast<const uint4*>(p.A + (int64_t)(m0 + r) * p.lda + k)), a);
#pragma unroll
              for (int e = 0; e < 8; ++e) acc[r] = mul_add<FMA>(a[e], w[e], acc[r]);   // ascending k
            }
          }
        } else {
          // the short last tile: missing products are absent
          for (int e = 0; k + e < p.K; ++e) {
            const float w = in_to_f32<F16>(brow[k + e]);
#pragma unroll
            for (int r = 0; r < MR; ++r)
              if (m0 + r < p.M) acc[r] = mul_add<FMA>(in_to_f32<F16>(p.A[(int64_t)(m0 + r) * p.lda + k + e]), w, acc[r]);
          }
        }
      }
      // lane fold: count-up pairs neighbours first; count-down pairs lanes 16 apart first
#pragma unroll
      for (int s = 0; s < 5; ++s) {
        const int off = p.fold == 0 ? (1 << s) : (16 >> s);
#pragma unroll
        for (int r = 0; r < MR; ++r) acc[r] = f_add(acc[r], __shfl_xor_sync(0xffffffffu, acc[r], off));
      }
      if (lane == 0) {
        if (!deps_done) { asm volatile("griddepcontrol.wait;" ::: "memory"); deps_done = true; }
#pragma unroll
        for (int r = 0; r < MR; ++r) {
          if (m0 + r < p.M) {
            const float v = apply_epilogue(acc[r], p.epi, m0 + r, j);
            store_scalar(p.C, p.c_dtype, (int64_t)(m0 + r) * p.ldc + j, v);
          }
        }
      }
    }
  }
}

template <int MR, bool F16>
cudaError_t launch_fma(const GemvParams& p, int grid, cudaStream_t st) {
  constexpr int smem = (GEMV_THREADS / 32) * gemv_depth(MR) * gemv_unr(MR) * 32 * 16;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid, 1, 1);
  cfg.blockDim = dim3(GEMV_THREADS, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (p.fma) return cudaLaunchKernelEx(&cfg, gemv_lane_tree_kernel<MR, F16, true>, p);
  return cudaLaunchKernelEx(&cfg, gemv_lane_tree_kernel<MR, F16, false>, p);
}

template <int MR>
cudaError_t launch_mr(const GemvParams& p, bool f16, int grid, cudaStream_t st) {
  return f16 ? launch_fma<MR, true>(p, grid, st) : launch_fma<MR, false>(p, grid, st);
}

}  // namespace

// All arguments were validated by the caller (operands 16-byte aligned, ld % 8 == 0).
rg_status_t launch_gemv(const rg_desc_t* d, const rg_tensor_t* A, const rg_tensor_t* B, const rg_tensor_t* C,
                        const rg_epilogue_t* epi, cudaStream_t st) {
  GemvParams p;
  p.A = static_cast<const uint16_t*>(A->ptr); p.B = static_cast<const uint16_t*>(B->ptr); p.C = C->ptr;
  p.lda = A->ld; p.ldb = B->ld; p.ldc = C->ld;
  p.M = (int32_t)A->rows; p.N = (int32_t)B->rows; p.K = (int32_t)A->cols;
  p.fma = d->fma; p.layout = d->gemv_layout; p.fold = d->gemv_fold; p.c_dtype = C->dtype; p.b_static = d->b_static;
  EpilogueArgs e{};
  if (epi) {
    e.bias = epi->bias; e.bias_dtype = epi->bias_dtype; e.act = epi->act;
    e.residual = epi->residual; e.residual_dtype = epi->residual_dtype; e.ldr = epi->ldr;
  }
  p.epi = e;
  const int sms = current_device().sms;                     // looked up once per device
  constexpr int WARPS = GEMV_THREADS / 32;
  const int64_t need = ((int64_t)p.N + WARPS - 1) / WARPS, cap = (int64_t)sms * (2048 / GEMV_THREADS);
  const int grid = (int)(need < cap ? need : cap);
  const bool f16 = A->dtype == RG_F16;
  cudaError_t err;
  if (p.M >= 8) err = launch_mr<8>(p, f16, grid, st);
  else if (p.M >= 4) err = launch_mr<4>(p, f16, grid, st);
  else if (p.M >= 2) err = launch_mr<2>(p, f16, grid, st);
  else err = launch_mr<1>(p, f16, grid, st);
  return err == cudaSuccess ? RG_OK : RG_ERR_CUDA;
}

}  // namespace rg
