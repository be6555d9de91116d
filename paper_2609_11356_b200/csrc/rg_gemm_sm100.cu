// Descriptor-fixed bf16 GEMM for sm_100a: TMA-fed tcgen05.mma with the fp32 accumulator in
// tensor memory, a fixed in-CTA K order, and a fused epilogue.
//
// What fixes the bits (Sec. 3.2.1, 3.2.2, App. E): for every output element and every
// split-K part, one accumulator starts at zero and receives one tcgen05.mma kind::f16 step per
// 16 consecutive k, in ascending k.  Everything else in this file is schedule and may change
// without moving a bit (Sec. 3.1): the tile shape, the shared-memory ring depth, which warp
// loads and which issues, the persistent tile walk, the double-buffered accumulator.
//
// CTA roles (320 threads):
//   warp 0           TMA producer: A[BM x 64] and B[BN x 64] boxes (128-byte swizzle), one lane per box
//   warp 1           MMA issuer: the warp walks the loop converged and an elected lane issues
//                    4 steps of K=16 per 64-wide box, ascending; tcgen05.commit frees the stage; a
//                    final commit publishes the accumulator.  The step is 128 rows, or 64 rows when
//                    the problem has at most 64 (half the A rows read from shared memory per step)
//   warps 2..9       epilogue: tcgen05.ld of their 32 TMEM lanes (warp % 4 picks the lane
//                    quarter; the two warps of a quarter take alternate 32-column chunks),
//                    epilogue math, global stores
// Two accumulators of BN columns each live in TMEM, so the epilogue of tile t overlaps the
// mainloop of tile t+1.
//
// Every wait is bounded: after ~2 s a waiter raises an abort flag, records a code in the
// device status word, and all roles drain and return; tensor memory is always released.
#include <cuda.h>

#include <atomic>
#include <mutex>

#include "rg_common.cuh"
#include "rg_internal.h"
#include "rg_ptx.cuh"

namespace rg {

__device__ unsigned int g_status_word = 0;

// Optional wall-clock stamps of the one-CTA kernel's roles (compiled in with -DRG_TIMELINE only; the
// library build has none of this): [launch % 8][CTA][what] in nanoseconds of the global timer.
#ifdef RG_TIMELINE
__device__ unsigned long long g_timeline[8][512][8];
// a call, not inline code: the stamps must not change the kernels' register counts (what fits beside what on an
// SM decides when the launch behind a kernel becomes resident, which is what the stamps are there to show)
static __device__ __noinline__ void rg_stamp(int seq, int slot) {
  if (blockIdx.x < 512) {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    g_timeline[seq & 7][blockIdx.x][slot] = t;
  }
}
#define RG_STAMP(slot) rg_stamp(p.launch_seq, slot)
#else
#define RG_STAMP(slot) do { } while (0)
#endif

namespace {

constexpr int BM = 128;           // rows per tile = TMEM lanes = UMMA M
constexpr int KBOX = 64;          // bf16 per 128-byte swizzle row
constexpr int UMMA_K = 16;        // instruction_k for 16-bit inputs
constexpr int NUM_THREADS = 320;
constexpr int NUM_EPI_WARPS = 8;

// ------------------------------------------------------------------ PTX wrappers (tensor core side)
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int32_t x, int32_t y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tcgen05_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tcgen05_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]^T, one K=16 step.  accumulate = 0 overwrites D.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// The same step on 8-bit e4m3 operands: 32 products per step (32 bytes of K per operand row).
__device__ __forceinline__ void umma_f8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_32x32b_x32(uint32_t taddr, uint32_t (&r)[32]) {
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
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// ---- two-SM (cta_group::2) forms: a pair of CTAs in a cluster works on one 256-row tile
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// shared::cluster address of the same variable in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// The box lands in this CTA's shared memory; its bytes are counted on `bar`, which may live in the peer.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int32_t x, int32_t y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// Arrive on the barrier at this offset in both CTAs of the pair once the steps issued so far are done.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  const uint16_t mask = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(mask) : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}

// Shared-memory matrix descriptor for a K-major bf16 tile whose rows are 128 bytes, stored
// with the 128-byte swizzle TMA produced: 8-row groups are 1024 bytes apart.
__device__ __forceinline__ uint64_t make_kmajor_sw128_desc(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((smem_addr & 0x3ffffu) >> 4);   // start address, 16-byte units
  d |= static_cast<uint64_t>(1) << 16;                         // leading byte offset: unused with swizzle
  d |= static_cast<uint64_t>(1024 >> 4) << 32;                 // stride byte offset between 8-row groups
  d |= static_cast<uint64_t>(1) << 46;                         // descriptor version for this architecture
  d |= static_cast<uint64_t>(2) << 61;                         // 128-byte swizzle
  return d;
}
// Instruction descriptor: 16-bit x 16-bit -> fp32, both operands K-major.
// operand format field: 0 = fp16, 1 = bf16
__device__ __forceinline__ void umma_f8_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// operand kinds of the kernels: what a 32-byte K step of an operand row holds
enum { KIND_BF16 = 0, KIND_F16 = 1, KIND_F8E4M3 = 2 };
// operand format field of the instruction descriptor: kind::f16 0 = fp16, 1 = bf16; kind::f8f6f4 0 = e4m3
__host__ __device__ constexpr uint32_t idesc_format(int kind) { return kind == KIND_BF16 ? 1u : 0u; }
template <int KIND>
__device__ __forceinline__ void umma_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  if (KIND == KIND_F8E4M3) umma_f8_pair(d_tmem, a_desc, b_desc, idesc, accumulate);
  else umma_bf16_pair(d_tmem, a_desc, b_desc, idesc, accumulate);
}

// The same step with the shared-memory descriptors given as (low word, high word): only the low word
// (the 16-byte-unit start address) changes from step to step, so the issuing thread does 32-bit adds.
// ACC: compile-time "accumulate onto D" (every step of a part but its first).
template <int KIND, bool ACC>
__device__ __forceinline__ void umma_pair_lo(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t hi, uint32_t idesc, uint32_t accumulate) {
  if (KIND == KIND_F8E4M3) {
    if (ACC) asm volatile("{\n\t.reg .b64 da, db;\n\t.reg .pred p;\n\tmov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\tsetp.eq.b32 p, %0, %0;\n\t"
                          "tcgen05.mma.cta_group::2.kind::f8f6f4 [%0], da, db, %4, p;\n\t}" ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc) : "memory");
    else asm volatile("{\n\t.reg .b64 da, db;\n\t.reg .pred p;\n\tmov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\tsetp.ne.b32 p, %5, 0;\n\t"
                      "tcgen05.mma.cta_group::2.kind::f8f6f4 [%0], da, db, %4, p;\n\t}" ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc), "r"(accumulate) : "memory");
  } else {
    if (ACC) asm volatile("{\n\t.reg .b64 da, db;\n\t.reg .pred p;\n\tmov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\tsetp.eq.b32 p, %0, %0;\n\t"
                          "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %4, p;\n\t}" ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc) : "memory");
    else asm volatile("{\n\t.reg .b64 da, db;\n\t.reg .pred p;\n\tmov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\tsetp.ne.b32 p, %5, 0;\n\t"
                      "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %4, p;\n\t}" ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc), "r"(accumulate) : "memory");
  }
}

// One-CTA form of the same: (low word, high word) descriptors, compile-time accumulate.
template <bool F8, bool ACC>
__device__ __forceinline__ void umma_one_lo(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t hi, uint32_t idesc, uint32_t accumulate) {
  if (F8) {
    if (ACC) asm volatile("{\n\t.reg .b64 da, db;\n\t.reg .pred p;\n\tmov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\tsetp.eq.b32 p, %0, %0;\n\t"
                          "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], da, db, %4, p;\n\t}" ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc) : "memory");
    else asm volatile("{\n\t.reg .b64 da, db;\n\t.reg .pred p;\n\tmov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\tsetp.ne.b32 p, %5, 0;\n\t"
                      "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], da, db, %4, p;\n\t}" ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc), "r"(accumulate) : "memory");
  } else {
    if (ACC) asm volatile("{\n\t.reg .b64 da, db;\n\t.reg .pred p;\n\tmov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\tsetp.eq.b32 p, %0, %0;\n\t"
                          "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t}" ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc) : "memory");
    else asm volatile("{\n\t.reg .b64 da, db;\n\t.reg .pred p;\n\tmov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\tsetp.ne.b32 p, %5, 0;\n\t"
                      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t}" ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc), "r"(accumulate) : "memory");
  }
}

__host__ __device__ constexpr uint32_t make_idesc(int bn, int m, uint32_t fmt) {
  return (1u << 4) | (fmt << 7) | (fmt << 10) | (static_cast<uint32_t>(bn >> 3) << 17) |
         (static_cast<uint32_t>(m >> 4) << 24);
}

__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* m) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(m)) : "memory");
}

struct GemmParams {
  int32_t M, N, K;
  int32_t tiles_m, tiles_n, n_parts;
  int32_t num_stages, raster, group_m;
  int32_t inner_span;     // second cut level: an accumulator is closed every inner_span k (0 = none; a multiple of the K step)
  int32_t bn;             // tile columns of the one-CTA kernel (any multiple of 16 up to 256)
  uint32_t idesc;         // instruction descriptor for N = bn
  int32_t mma_m;          // rows of the tensor-core step: 128, or 64 when the problem has at most 64 rows
  int32_t f8;             // operands are e4m3 bytes: M, N as given, every K quantity counted in byte pairs
  int32_t launch_seq;     // host-side launch counter (used by the optional timeline stamps only)
  int32_t b_static;       // the caller's promise that no work ahead in the stream writes B: its first boxes are fetched before the dependency wait
  uint32_t tmem_cols;     // tensor-memory columns allocated: two (or four) accumulators of equal width
  uint32_t a_box_bytes;   // bytes of one A box: 128 B per row actually loaded (rows past M are never fetched)
  uint32_t slack_bytes;   // readable bytes kept behind the ring for the tensor-core step's surplus A rows
  void* C;
  int64_t ldc;
  int32_t c_dtype;
  void* ws;             // split-K partials [part][M][ldw] at ws_dtype; null without cuts and with the in-cluster merge
  int64_t ldw;
  int32_t ws_dtype;
  unsigned int* tickets;  // TICKET kernels: one counter per output tile (zero on entry, zero again on exit), else null
  int32_t ticket_all;     // TICKET kernels: every work item has a CTA of its own (one round), so the CTAs of a tile may wait for each other
  // in-cluster merge (CLUSTER kernels): the n_parts CTAs of a cluster own the parts of one output tile
  int32_t tree, merge_dtype;   // how the parts are added (descriptor's tree, type of the running sum)
  int32_t part_rows;           // rows of a tile kept in a CTA's shared-memory partial buffer
  int32_t part_ld;             // floats between its rows (tile width + 4: spreads the rows over the banks)
  EpilogueArgs epi;
  int32_t part_begin[RG_MAX_CUTS + 1];
  int32_t part_end[RG_MAX_CUTS + 1];
};

__device__ __forceinline__ void decode_work(const GemmParams& p, int w, int& part, int& tm, int& tn) {
  const int tiles = p.tiles_m * p.tiles_n;
  part = w / tiles;
  const int t = w - part * tiles;
  if (p.raster == 1) {
    tm = t / p.tiles_n;
    tn = t - tm * p.tiles_n;
  } else {
    // grouped walk: group_m tile-rows share their B columns while they are hot in L2
    const int per_group = p.group_m * p.tiles_n;
    const int g = t / per_group;
    const int first_m = g * p.group_m;
    const int gsize = min(p.tiles_m - first_m, p.group_m);
    const int r = t - g * per_group;
    tm = first_m + r % gsize;
    tn = r / gsize;
  }
}

// bias -> SiLU -> residual on 32 consecutive columns of one row, stage by stage so that the 32
// independent chains of each stage overlap in the pipeline.
__device__ __forceinline__ void epilogue_row_segment(float (&v)[32], const EpilogueArgs& e, int64_t row, int col0, int ncols) {
  if (e.bias) {
    float b[32];
    load_row_segment(e.bias, e.bias_dtype, col0, ncols, b);
#pragma unroll
    for (int c = 0; c < 32; ++c) v[c] = f_add(v[c], b[c]);
  }
  if (e.act == 1) {
    float ex[32];
    // the largest |v| of the segment, NaN if any value is NaN: up to 87 no element needs a range
    // or NaN select of the specified exponential (same bits, about half the instructions)
    float amax = absmax3_nan(v[0], v[1], v[2]);
#pragma unroll
    for (int c = 3; c + 1 < 32; c += 2) amax = absmax3_nan(amax, v[c], v[c + 1]);
    amax = absmax3_nan(amax, v[31], v[31]);
    if (amax <= 87.0f) {
#pragma unroll
      for (int c = 0; c < 32; c += 2) {
        const float2 e2 = rg_exp_neg_inrange2(make_float2(v[c], v[c + 1]));
        ex[c] = f_add(1.0f, e2.x); ex[c + 1] = f_add(1.0f, e2.y);
      }
    } else {
#pragma unroll
      for (int c = 0; c < 32; ++c) ex[c] = f_add(1.0f, rg_exp(-v[c]));
    }
#pragma unroll
    for (int c = 0; c < 32; ++c) v[c] = __fdiv_rn(v[c], ex[c]);
  }
  if (e.residual) {
    float rr[32];
    load_row_segment(e.residual, e.residual_dtype, row * e.ldr + col0, ncols, rr);
#pragma unroll
    for (int c = 0; c < 32; ++c) v[c] = f_add(v[c], rr[c]);
  }
}

// Store up to 32 consecutive columns of one row of a row-major matrix, each value rounded once to
// `dtype`.  The type is tested once, outside the unrolled loops.
__device__ __forceinline__ void store_row_values(void* base, int dtype, int64_t off, int ncols, const float (&v)[32]) {
  if (dtype == RG_F32) {
    float* dst = static_cast<float*>(base) + off;
    if (ncols == 32 && (reinterpret_cast<uintptr_t>(dst) & 15) == 0) {
#pragma unroll
      for (int q = 0; q < 8; ++q)
        reinterpret_cast<float4*>(dst)[q] = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
    } else {
#pragma unroll
      for (int c = 0; c < 32; ++c) if (c < ncols) dst[c] = v[c];
    }
    return;
  }
  uint16_t* dst = static_cast<uint16_t*>(base) + off;
  const bool vec = ncols == 32 && (reinterpret_cast<uintptr_t>(dst) & 15) == 0;
  if (dtype == RG_BF16) {
    if (vec) {
#pragma unroll
      for (int q = 0; q < 4; ++q)
        reinterpret_cast<uint4*>(dst)[q] = make_uint4(pack_bf16x2(v[8 * q], v[8 * q + 1]), pack_bf16x2(v[8 * q + 2], v[8 * q + 3]),
                                                      pack_bf16x2(v[8 * q + 4], v[8 * q + 5]), pack_bf16x2(v[8 * q + 6], v[8 * q + 7]));
    } else {
#pragma unroll
      for (int c = 0; c < 32; ++c) if (c < ncols) dst[c] = __bfloat16_as_ushort(__float2bfloat16_rn(v[c]));
    }
  } else {
    if (vec) {
#pragma unroll
      for (int q = 0; q < 4; ++q)
        reinterpret_cast<uint4*>(dst)[q] = make_uint4(pack_f16x2(v[8 * q], v[8 * q + 1]), pack_f16x2(v[8 * q + 2], v[8 * q + 3]),
                                                      pack_f16x2(v[8 * q + 4], v[8 * q + 5]), pack_f16x2(v[8 * q + 6], v[8 * q + 7]));
    } else {
#pragma unroll
      for (int c = 0; c < 32; ++c) if (c < ncols) dst[c] = __half_as_ushort(__float2half_rn(v[c]));
    }
  }
}

// One 32-column chunk of one output row, held as fp32 bit patterns in r: a split-K part goes to the
// workspace rounded once to partial_dtype (untouched when that is fp32; Sec. 3.2.2); otherwise
// bias / SiLU / residual and one rounding to the output type.
__device__ __forceinline__ void epilogue_store_chunk(const GemmParams& p, int part, int64_t row, int col0, int ncols,
                                                     const uint32_t (&r)[32]) {
  float v[32];
#pragma unroll
  for (int c = 0; c < 32; ++c) v[c] = __uint_as_float(r[c]);
  if (p.ws) {
    store_row_values(p.ws, p.ws_dtype, ((int64_t)part * p.M + row) * p.ldw + col0, ncols, v);
  } else {
    epilogue_row_segment(v, p.epi, row, col0, ncols);
    store_row_values(p.C, p.c_dtype, row * p.ldc + col0, ncols, v);
  }
}

// Epilogue of one accumulator tile for one warp: the warp's 32 TMEM lanes (one output row per
// thread), 32-column chunks chunk0, chunk0+2, ...
__device__ __forceinline__ void epilogue_tile(const GemmParams& p, const int BN, int part, int64_t row, bool row_ok, int tn,
                                              uint32_t taddr, int chunk0, int chunk_step = 64) {
  const int col_end = min(p.N, (tn + 1) * BN);            // this tile's columns end here
#pragma unroll 1
  for (int c0 = chunk0 * 32; c0 < BN; c0 += chunk_step) {
    const int col0 = tn * BN + c0;
    if (col0 >= col_end) break;                           // uniform across the warp
    uint32_t r[32];
    tmem_ld_32x32b_x32(taddr + c0, r);
    tmem_ld_wait();
    if (row_ok) epilogue_store_chunk(p, part, row, col0, min(32, col_end - col0), r);
  }
}

// Second cut level (Sec. 3.2.2 "some kernels cut again inside a part"; App. E per-group accumulation):
// the MMA warp closes an accumulator every inner_span k; each epilogue warp adds every closed group,
// at fp32 and in ascending order, into a running sum held in registers, then finishes the tile from
// it.  A warp owns two 32-column chunks (tiles up to 128 columns, the running sum stays in registers) or four
// (tiles up to 256 columns: 128 running-sum registers, part of which the compiler keeps in local memory).
template <int NCH> struct GroupedAcc { uint32_t v[NCH][32]; };

// FIRST: the group that opens the running sum (a copy); the other groups are one add per element and nothing else.
template <int NCH, bool FIRST, int CSTEP>
__device__ __forceinline__ void grouped_add_t(const GemmParams& p, const int BN, int tn, uint32_t taddr, int chunk0, GroupedAcc<NCH>& acc) {
  const int col_end = min(p.N, (tn + 1) * BN);
#pragma unroll
  for (int j = 0; j < NCH; ++j) {
    const int c0 = (chunk0 + CSTEP * j) * 32;
    if (c0 < BN && tn * BN + c0 < col_end) {              // uniform across the warp
      if (FIRST) {
        tmem_ld_32x32b_x32(taddr + c0, acc.v[j]);
        tmem_ld_wait();
      } else {
        uint32_t r[32];
        tmem_ld_32x32b_x32(taddr + c0, r);
        tmem_ld_wait();
        // two adds per instruction (a packed add rounds each half like the scalar add; it feeds no multiply here)
#pragma unroll
        for (int c = 0; c < 32; c += 2) {
          const float2 q = __fadd2_rn(make_float2(__uint_as_float(acc.v[j][c]), __uint_as_float(acc.v[j][c + 1])),
                                      make_float2(__uint_as_float(r[c]), __uint_as_float(r[c + 1])));
          acc.v[j][c] = __float_as_uint(q.x); acc.v[j][c + 1] = __float_as_uint(q.y);
        }
      }
    }
  }
}
// CSTEP: the warp's chunks are chunk0, chunk0 + CSTEP, ... (CSTEP = epilogue warps per lane quarter)
template <int NCH, int CSTEP = 2>
__device__ __forceinline__ void grouped_add(const GemmParams& p, const int BN, int tn, uint32_t taddr, int chunk0, bool first,
                                            GroupedAcc<NCH>& acc) {
  if (first) grouped_add_t<NCH, true, CSTEP>(p, BN, tn, taddr, chunk0, acc);      // uniform across the warp
  else grouped_add_t<NCH, false, CSTEP>(p, BN, tn, taddr, chunk0, acc);
}

template <int NCH, int CSTEP = 2>
__device__ __forceinline__ void grouped_finish(const GemmParams& p, const int BN, int part, int64_t row, bool row_ok, int tn,
                                               int chunk0, const GroupedAcc<NCH>& acc) {
  const int col_end = min(p.N, (tn + 1) * BN);
#pragma unroll
  for (int j = 0; j < NCH; ++j) {
    const int c0 = (chunk0 + CSTEP * j) * 32;
    const int col0 = tn * BN + c0;
    if (c0 < BN && col0 < col_end && row_ok) epilogue_store_chunk(p, part, row, col0, min(32, col_end - col0), acc.v[j]);
  }
}

// ---- in-cluster split-K merge (App. E: "a single launch across the split-K slices"; Sec. 3.2.2 "Split-K")
__device__ __forceinline__ float4 ld_cluster_f4(uint32_t cluster_addr) {
  float4 v;
  asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(cluster_addr) : "memory");
  return v;
}

// Up to eight parts added in the descriptor's tree, the running sum kept at merge_dtype.  BALANCED is
// the level-by-level definition itself: neighbours pair, an unpaired last value moves up unchanged.
template <bool MERGE_16>
__device__ __forceinline__ float4 merge_upto8(float4 (&v)[8], int S, int tree, int merge_dtype) {
  auto add1 = [merge_dtype](float a, float b) -> float {
    const float r = f_add(a, b);
    return MERGE_16 ? round_through(r, merge_dtype) : r;
  };
  auto add4 = [&](const float4& a, const float4& b) -> float4 {
    return make_float4(add1(a.x, b.x), add1(a.y, b.y), add1(a.z, b.z), add1(a.w, b.w));
  };
  if (tree == RG_TREE_LEFT) {
    float4 acc = v[0];
#pragma unroll
    for (int i = 1; i < 8; ++i) if (i < S) acc = add4(acc, v[i]);
    return acc;
  }
  int n = S;
#pragma unroll
  for (int half = 4; half >= 1; half >>= 1) {
#pragma unroll
    for (int t = 0; t < half; ++t) {
      if (2 * t + 1 < n) v[t] = add4(v[2 * t], v[2 * t + 1]);
      else if (2 * t < n) v[t] = v[2 * t];
    }
    n = (n + 1) >> 1;
  }
  return v[0];
}

// bias -> SiLU -> residual -> one rounding for four consecutive columns of one row, then the store.
__device__ __forceinline__ void finish_and_store4(const EpilogueArgs& e, void* C, int64_t ldc, int c_dtype, int N, int64_t row, int col0, float4 acc) {
  float v[4] = {acc.x, acc.y, acc.z, acc.w};
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    if (col0 + c < N) {
      if (e.bias) v[c] = f_add(v[c], load_scalar(e.bias, e.bias_dtype, col0 + c));
      if (e.act == 1) v[c] = rg_silu(v[c]);
      if (e.residual) v[c] = f_add(v[c], load_scalar(e.residual, e.residual_dtype, row * e.ldr + col0 + c));
    }
  }
  uint16_t* const c16 = static_cast<uint16_t*>(C) + row * ldc + col0;
  if (col0 + 4 <= N && c_dtype != RG_F32 && (reinterpret_cast<uintptr_t>(c16) & 7) == 0) {
    uint2 o;
    o.x = pack_16x2(v[0], v[1], c_dtype);
    o.y = pack_16x2(v[2], v[3], c_dtype);
    *reinterpret_cast<uint2*>(c16) = o;
  } else {
#pragma unroll
    for (int c = 0; c < 4; ++c)
      if (col0 + c < N) store_scalar(C, c_dtype, row * ldc + col0 + c, v[c]);
  }
}

// KSUB: 64-wide boxes per pipeline stage (BK = 64 * KSUB); F8: e4m3 operands (kind::f8f6f4).
// CLUSTER: split-K in one launch.  The n_parts CTAs of a thread-block cluster own the parts of one output
// tile (CTA rank = part); each walks its part exactly as the plain kernel does, leaves its fp32 part (rounded
// once to partial_dtype) in its own shared memory, and after a cluster-wide hand-over every CTA merges one
// slice of the tile, reading the parts of all CTAs over distributed shared memory in the descriptor's
// tree, applies the epilogue and stores.  No workspace in global memory, no second launch, no atomics.  The tile width p.bn is a run-time value:
// any multiple of 16 up to 256 is a legal step width, which lets the host size tiles so that the
// work items fill whole waves.
// EPI_WARPS: 8 epilogue warps (320 threads, one CTA per SM), or 4 (192 threads, a warp takes every 32-column
// chunk of its lane quarter): that form is launched with at most half an SM's shared memory and tensor memory, so
// two CTAs share an SM, and the CTAs of the next launch in the stream can become resident, set themselves up and
// fetch their first weight boxes while this launch's last CTAs finish (used for the weight-streaming shapes).
// GROUPED: the second cut level (inner_span): accumulators closed inside a part and chained in the epilogue
// warps' registers; an instantiation of its own, so that its 128 running-sum registers per thread are not
// the plain kernel's problem.
// TICKET: split-K in one launch without clusters.  Work items are (part, tile) as in the plain kernel and the parts go to
// the workspace; the CTA that stores a tile's LAST part (an integer ticket per tile, taken after a device-wide fence)
// merges the tile from the workspace in the descriptor's tree, applies the epilogue and stores.  Nobody waits for
// anybody: which CTA merges depends on timing, what it computes does not (Sec. 3.1: the tree, not the schedule).
// When the work items fit one round (p.ticket_all) the tile's CTAs wait for each other instead (bounded) and each
// merges a slice of the tile.  Measured on the decode shape it does not pay: within 3 % of the two-kernel path at 1
// and 8 rows, 2 us slower at 32 rows (27.7 against 25.6 us): part store, device-wide fence, ticket, the spread of the
// tile's eight CTAs and one L2 round trip cost what the second launch costs.  Kept as an option.
template <int KSUB, bool F8, bool CLUSTER, int EPI_WARPS, bool GROUPED = false, int NCH = 2, bool TICKET = false>
__global__ void __launch_bounds__(64 + 32 * EPI_WARPS, EPI_WARPS == 4 ? 3 : 1)
gemm_tcgen05_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                    const GemmParams p) {
  // The A box holds only the rows that exist (a multiple of 8, so 1024-byte swizzle groups stay whole);
  // the tensor-core step still reads 128 rows, and whatever lies past the box only reaches
  // accumulator rows that are never stored.
  const uint32_t A_BOX_BYTES = p.a_box_bytes;
  const int BN = p.bn;
  const uint32_t B_BOX_BYTES = (uint32_t)BN * KBOX * 2;
  const uint32_t STAGE_BYTES = KSUB * (A_BOX_BYTES + B_BOX_BYTES);
  // Accumulators in tensor memory: two, or four for the second cut level on tiles up to 128 columns (its
  // groups are short, and more of them in flight hide the hand-over between the issuing warp and the epilogue)
  constexpr int NB = (GROUPED && NCH <= 2) ? 4 : 2;
  const uint32_t TMEM_COLS = p.tmem_cols;                // a power of two >= 32; accumulator b starts at column b * TMEM_COLS / NB
  const uint32_t ACC_STRIDE = TMEM_COLS / NB;
  const uint32_t IDESC = p.idesc;

  extern __shared__ uint8_t smem_raw[];
  // the swizzle pattern is a function of the absolute address: tiles sit on 1024-byte boundaries
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const int S = p.num_stages;
  // barriers sit behind the ring and behind the span a short A box leaves readable (see a_slack_bytes)
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem_gen + (size_t)S * STAGE_BYTES + p.slack_bytes);
  // layout: full[S], empty[S], tmem_full[NB], tmem_empty[NB], then tmem base slot and abort flag
  const uint32_t bar_full = smem_u32(bars);
  const uint32_t bar_empty = bar_full + 8u * S;
  const uint32_t bar_tfull = bar_empty + 8u * S;
  const uint32_t bar_tempty = bar_tfull + 8u * NB;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * S + 2 * NB);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  volatile int* ticket_flag = reinterpret_cast<volatile int*>(tmem_slot + 2);   // TICKET: "this CTA merges the tile"
  // CLUSTER: two more barriers (parts ready / parts read), then this CTA's partial tile
  const uint32_t bar_ready = bar_tempty + 8u * NB + 16u;
  const uint32_t bar_free = bar_ready + 8u;
  float* const part_buf = reinterpret_cast<float*>(bars + 2 * S + 2 * NB + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) RG_STAMP(0);                      // CTA entry
  // Work items: (part, tile) for the plain kernel, walked by CTA; tiles for the CLUSTER kernel, walked by
  // cluster, the CTA's rank in the cluster being its part.
  const int crank = CLUSTER ? (int)cluster_ctarank() : 0;
  const int total_work = CLUSTER ? p.tiles_m * p.tiles_n : p.tiles_m * p.tiles_n * p.n_parts;
  const int work_first = CLUSTER ? (int)blockIdx.x / p.n_parts : (int)blockIdx.x;
  const int work_step = CLUSTER ? (int)gridDim.x / p.n_parts : (int)gridDim.x;

  if (threadIdx.x == 0) {
    prefetch_tensormap(&tmap_a);
    prefetch_tensormap(&tmap_b);
    for (int s = 0; s < S; ++s) { mbar_init(bar_full + 8u * s, 1); mbar_init(bar_empty + 8u * s, 1); }
    for (int b = 0; b < NB; ++b) { mbar_init(bar_tfull + 8u * b, 1); mbar_init(bar_tempty + 8u * b, EPI_WARPS); }
    if (CLUSTER) { mbar_init(bar_ready, EPI_WARPS * p.n_parts); mbar_init(bar_free, EPI_WARPS * p.n_parts); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_slot), TMEM_COLS);
    tmem_relinquish();
  }
  tcgen05_fence_before();
  __syncthreads();
  if (CLUSTER) cluster_sync_all();                         // every CTA's barriers exist before any remote arrive
  tcgen05_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  if (threadIdx.x == 0) RG_STAMP(1);                      // set-up done
  // a split-K merge launched behind this kernel may be scheduled now; it still waits for this grid to finish
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  // This kernel is itself launched with programmatic stream serialisation, so it may be running
  // before the kernels ahead of it in the stream have finished.  Each role that touches global
  // memory waits for them (griddepcontrol.wait) immediately before its first access and not
  // earlier: the instructions leading up to that access are then already fetched (the weight
  // stream of the previous launch leaves no code in L2).  The MMA warp touches none.

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    // 2*KSUB lanes, one box each (lane < KSUB: A sub-box `lane`; otherwise B sub-box lane - KSUB):
    // the lanes run converged, so one instruction issue starts all of a stage's copies.
    if (lane < 2 * KSUB) {
      const bool is_b = lane >= KSUB;
      const int sub = is_b ? lane - KSUB : lane;
      const CUtensorMap* map = is_b ? &tmap_b : &tmap_a;
      const uint32_t box_off = is_b ? KSUB * A_BOX_BYTES + sub * B_BOX_BYTES : sub * A_BOX_BYTES;
      int stage = 0; uint32_t phase = 0;
      bool alive = true;
      bool deps_done = false;
      // Weights that nothing ahead in the stream writes (the caller's promise, `b_static`) need not wait for
      // the kernels ahead: the B boxes of the first work item's first stages (the ring is empty, so at most
      // S of them) go out at once, and only the A boxes of those stages wait for the dependency.
      int prefetched = 0;
      if (p.b_static && work_first < total_work) {
        int part, tm, tn;
        decode_work(p, work_first, part, tm, tn);
        if (CLUSTER) part = crank;
        const int k_begin = p.part_begin[part], k_end = p.part_end[part];
        for (int k0 = k_begin; k0 < k_end && prefetched < S; k0 += KBOX * KSUB, ++prefetched) {
          const uint32_t full = bar_full + 8u * prefetched;
          if (lane == 0) mbar_expect_tx(full, STAGE_BYTES);
          if (is_b) tma_load_2d(smem_base + prefetched * STAGE_BYTES + box_off, map, k0 + sub * KBOX, tn * BN, full);
        }
      }
      int issued = 0;                                      // stages handed to the ring so far
      for (int w = work_first; w < total_work && alive; w += work_step) {
        int part, tm, tn;
        decode_work(p, w, part, tm, tn);
        if (CLUSTER) part = crank;
        const int k_begin = p.part_begin[part], k_end = p.part_end[part];
        const int y = is_b ? tn * BN : tm * BM;
        for (int k0 = k_begin; k0 < k_end; k0 += KBOX * KSUB, ++issued) {
          const uint32_t full = bar_full + 8u * stage;
          const bool ahead = issued < prefetched;          // this stage's barrier is armed and its B boxes are on their way
          if (!ahead) {
            if (!mbar_wait(bar_empty + 8u * stage, phase ^ 1u, abort_flag, &g_status_word, 0x100u | stage)) { alive = false; break; }
            if (lane == 0) mbar_expect_tx(full, STAGE_BYTES);
          }
          // (b_static = 2: A is not written by work in flight either, so no load of this launch waits; its stores do)
          if (!deps_done && p.b_static < 2) { asm volatile("griddepcontrol.wait;" ::: "memory"); deps_done = true; if (lane == 0) RG_STAMP(2); }
          if (!ahead || !is_b) tma_load_2d(smem_base + stage * STAGE_BYTES + box_off, map, k0 + sub * KBOX, y, full);
          if (++stage == S) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    // The whole warp walks the loop with identical values and one elected lane issues: with every lane
    // converged the descriptor arithmetic stays in the uniform datapath, where the tensor-core
    // instruction takes its operands from (a single diverged thread pays a register-to-uniform move
    // for each of them, which dominates when the tile is narrow and a step is short).
    {
      const bool leader = elect_one();
      int stage = 0; uint32_t phase = 0;
      bool alive = true;
      int gc = 0;                                         // accumulators handed to the epilogue so far
      const uint64_t desc_a0 = make_kmajor_sw128_desc(smem_base);
      const uint64_t desc_b0 = make_kmajor_sw128_desc(smem_base + KSUB * A_BOX_BYTES);
      for (int w = work_first; w < total_work && alive; w += work_step) {
        int part, tm, tn;
        decode_work(p, w, part, tm, tn);
        if (CLUSTER) part = crank;
        const int k_begin = p.part_begin[part], k_end = p.part_end[part];
        // one accumulator per part, or one per group of inner_span k (a multiple of the K step)
        const int span = (GROUPED && p.inner_span > 0) ? p.inner_span : (k_end - k_begin);
        int group_end = k_begin;
        int buf = 0;
        uint32_t d_tmem = 0, accumulate = 0;
        // groups that end inside a pipeline stage (a span that is not a multiple of the stage width, down to one
        // instruction per accumulator: the two-rounding plan of Sec. 3.2.2 / App. E) take the step-by-step path below
        const bool step_groups = GROUPED && p.inner_span > 0 && (p.inner_span % (KBOX * KSUB)) != 0;
        for (int k0 = k_begin; k0 < k_end; k0 += KBOX * KSUB) {
          if (!step_groups && k0 >= group_end) {
            if (k0 > k_begin) { if (leader) umma_commit(bar_tfull + 8u * buf); ++gc; }   // the previous group is complete
            buf = gc % NB;
            if (!warp_mbar_wait(bar_tempty + 8u * buf, ((gc / NB) & 1) ^ 1u, abort_flag, &g_status_word, 0x200u | buf)) { alive = false; break; }
            tcgen05_fence_after();
            d_tmem = tmem_base + buf * ACC_STRIDE;
            accumulate = 0;                              // every part and every group starts from zero
            group_end = k0 + span;
          }
          if (!warp_mbar_wait(bar_full + 8u * stage, phase, abort_flag, &g_status_word, 0x300u | stage)) { alive = false; break; }
          if (step_groups) {
            tcgen05_fence_after();
            const uint64_t ad0 = desc_a0 + (uint64_t)((stage * STAGE_BYTES) >> 4);
            const uint64_t bd0 = desc_b0 + (uint64_t)((stage * STAGE_BYTES) >> 4);
#pragma unroll 1
            for (int sa = 0; sa < KSUB * (KBOX / UMMA_K) && alive; ++sa) {
              const int sub = sa / (KBOX / UMMA_K), a = sa % (KBOX / UMMA_K);
              const int kk = k0 + sub * KBOX + a * UMMA_K;
              if (kk >= k_end) break;                    // ascending k; nothing past the end of the part
              if (kk >= group_end) {                     // this step opens a new accumulator
                if (kk > k_begin) { if (leader) umma_commit(bar_tfull + 8u * buf); ++gc; }
                buf = gc % NB;
                if (!warp_mbar_wait(bar_tempty + 8u * buf, ((gc / NB) & 1) ^ 1u, abort_flag, &g_status_word, 0x200u | buf)) { alive = false; break; }
                tcgen05_fence_after();
                d_tmem = tmem_base + buf * ACC_STRIDE;
                accumulate = 0;
                group_end = kk + span;
              }
              const uint64_t ad = ad0 + (uint64_t)((sub * A_BOX_BYTES) >> 4) + 2u * a;
              const uint64_t bd = bd0 + (uint64_t)((sub * B_BOX_BYTES) >> 4) + 2u * a;
              if (leader) {
                if (F8) umma_f8(d_tmem, ad, bd, IDESC, accumulate);
                else umma_bf16(d_tmem, ad, bd, IDESC, accumulate);
              }
              accumulate = 1;
            }
            if (!alive) break;
            if (leader) umma_commit(bar_empty + 8u * stage);
            if (++stage == S) { stage = 0; phase ^= 1u; }
            continue;
          }
#ifdef RG_TIMELINE
          if (leader && w == work_first && k0 == k_begin) RG_STAMP(3);   // first stage landed
#endif
          tcgen05_fence_after();
          // descriptors differ from the stage-0 ones only in the 16-byte-unit start address (low word).
          // The operand kind is a template parameter: a run-time test in front of every step slowed
          // this thread enough to cost the weight-streaming shapes 5 us per call.
          const uint64_t adesc0 = desc_a0 + (uint64_t)((stage * STAGE_BYTES) >> 4);
          const uint64_t bdesc0 = desc_b0 + (uint64_t)((stage * STAGE_BYTES) >> 4);
          if (k0 + KBOX * KSUB <= k_end) {
            // whole stage inside the part: 4*KSUB steps, ascending k, no per-step tests; 32-bit arithmetic on
            // the descriptors' low words (the high words never change and nothing carries into them)
            const uint32_t a_lo = (uint32_t)adesc0, b_lo = (uint32_t)bdesc0, hi = (uint32_t)(desc_a0 >> 32);
#pragma unroll
            for (int sub = 0; sub < KSUB; ++sub) {
#pragma unroll
              for (int a = 0; a < KBOX / UMMA_K; ++a) {
                const uint32_t al = a_lo + ((sub * A_BOX_BYTES) >> 4) + 2u * a, bl = b_lo + ((sub * B_BOX_BYTES) >> 4) + 2u * a;
                if (leader) {
                  if (sub | a) umma_one_lo<F8, true>(d_tmem, al, bl, hi, IDESC, 1u);
                  else umma_one_lo<F8, false>(d_tmem, al, bl, hi, IDESC, accumulate);
                }
              }
            }
            accumulate = 1;
          } else {
#pragma unroll
            for (int sub = 0; sub < KSUB; ++sub) {
#pragma unroll
              for (int a = 0; a < KBOX / UMMA_K; ++a) {
                // ascending k; steps at or past the end of the part are not issued
                if (k0 + sub * KBOX + a * UMMA_K < k_end) {
                  const uint64_t ad = adesc0 + (uint64_t)((sub * A_BOX_BYTES) >> 4) + 2u * a;
                  const uint64_t bd = bdesc0 + (uint64_t)((sub * B_BOX_BYTES) >> 4) + 2u * a;
                  if (leader) {
                    if (F8) umma_f8(d_tmem, ad, bd, IDESC, accumulate);
                    else umma_bf16(d_tmem, ad, bd, IDESC, accumulate);
                  }
                  accumulate = 1;
                }
              }
            }
          }
          // stage reusable once these steps have read it (with the second cut level a group's last stage could be
          // released by the epilogue when it sees the group's accumulator complete, which saves this thread one of
          // its two commits per group: built and measured, 739 against 763 TFLOP/s at a group every 64 k; dropped)
          if (leader) umma_commit(bar_empty + 8u * stage);
          if (++stage == S) { stage = 0; phase ^= 1u; }
        }
        if (alive) { if (leader) umma_commit(bar_tfull + 8u * buf); ++gc; }   // last (or only) accumulator complete
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue warps
    const int quarter = warp & 3;                         // TMEM lanes [32*quarter, 32*quarter+32)
    const int chunk0 = (warp - 2) >> 2;                   // this warp takes chunks chunk0, chunk0 + EPI_WARPS / 4, ...
    constexpr int CHUNK_STEP = 32 * (EPI_WARPS / 4);
    bool alive = true;
    bool deps_done = false;
    int gc = 0;
    for (int w = work_first; w < total_work && (alive || TICKET); w += work_step) {
      int part, tm, tn;
      decode_work(p, w, part, tm, tn);
      if (CLUSTER) part = crank;
      // a 64-row step keeps rows 16q .. 16q+15 in the first 16 lanes of lane quarter q
      const int64_t row = p.mma_m == 64 ? (int64_t)(quarter * 16 + lane) : (int64_t)tm * BM + quarter * 32 + lane;
      const bool row_ok = row < p.M && (p.mma_m != 64 || lane < 16);
      const int klen = p.part_end[part] - p.part_begin[part];
      const int ngroups = (GROUPED && p.inner_span > 0) ? (klen + p.inner_span - 1) / p.inner_span : 1;
      if (CLUSTER) {
        // ---- this CTA's part of the tile: tensor memory -> its shared-memory partial buffer
        const int it = gc;                                  // tiles this cluster has finished
        const int buf = gc % NB;
        if (!mbar_wait(bar_tfull + 8u * buf, (gc / NB) & 1, abort_flag, &g_status_word, 0x400u | buf)) { alive = false; break; }
        tcgen05_fence_after();
        if (!deps_done) { asm volatile("griddepcontrol.wait;" ::: "memory"); deps_done = true; }
        // the buffer still holds the previous tile's part until every CTA of the cluster has read its slice
        if (it > 0 && !mbar_wait_cluster(bar_free, (uint32_t)(it - 1) & 1u, abort_flag, &g_status_word, 0x500u)) { alive = false; break; }
        const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + buf * ACC_STRIDE;
        const int row_in_tile = p.mma_m == 64 ? quarter * 16 + lane : quarter * 32 + lane;
        const int col_end = min(p.N, (tn + 1) * BN);
#pragma unroll 1
        for (int c0 = chunk0 * 32; c0 < BN; c0 += CHUNK_STEP) {
          if (tn * BN + c0 >= col_end) break;               // uniform across the warp
          uint32_t r[32];
          tmem_ld_32x32b_x32(taddr + c0, r);
          tmem_ld_wait();
          if (row_ok) {
            float4* dst = reinterpret_cast<float4*>(part_buf + (size_t)row_in_tile * p.part_ld + c0);
#pragma unroll
            for (int q = 0; q < 8; ++q) {
              if (c0 + 4 * q < BN)                          // the tile width is a multiple of 16, not of 32
                dst[q] = make_float4(round_through(__uint_as_float(r[4 * q]), p.ws_dtype), round_through(__uint_as_float(r[4 * q + 1]), p.ws_dtype),
                                     round_through(__uint_as_float(r[4 * q + 2]), p.ws_dtype), round_through(__uint_as_float(r[4 * q + 3]), p.ws_dtype));
            }
          }
        }
        tcgen05_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_tempty + 8u * buf);  // the accumulator may be overwritten
        ++gc;
        // ---- tell every CTA of the cluster that this warp's share of the part is in place, wait for all shares
        if (lane < p.n_parts) mbar_arrive_cluster(map_to_cta(bar_ready, (uint32_t)lane));
        if (!mbar_wait_cluster(bar_ready, (uint32_t)it & 1u, abort_flag, &g_status_word, 0x600u)) { alive = false; break; }
        // ---- merge this CTA's slice of the tile: groups of four columns, dealt to the CTAs in contiguous runs
        {
          const int tile_rows = min(p.part_rows, p.M - tm * BM);
          const int c4s = BN >> 2;
          const int units = tile_rows * c4s;
          const int per = (units + p.n_parts - 1) / p.n_parts;
          const int u_end = min(units, (crank + 1) * per);
          const uint32_t part_local = smem_u32(part_buf);
          for (int u = crank * per + (warp - 2) * 32 + lane; u < u_end; u += EPI_WARPS * 32) {
            const int r_t = u / c4s, c4 = u - r_t * c4s;
            const int col0 = tn * BN + 4 * c4;
            if (col0 >= p.N) continue;
            const uint32_t off = part_local + (uint32_t)(r_t * p.part_ld + 4 * c4) * 4u;
            float4 v[8];
#pragma unroll
            for (int s2 = 0; s2 < 8; ++s2) if (s2 < p.n_parts) v[s2] = ld_cluster_f4(map_to_cta(off, (uint32_t)s2));
            const float4 acc = p.merge_dtype == RG_F32 ? merge_upto8<false>(v, p.n_parts, p.tree, p.merge_dtype)
                                                        : merge_upto8<true>(v, p.n_parts, p.tree, p.merge_dtype);
            finish_and_store4(p.epi, p.C, p.ldc, p.c_dtype, p.N, (int64_t)tm * BM + r_t, col0, acc);
          }
        }
        __syncwarp();
        if (lane < p.n_parts) mbar_arrive_cluster(map_to_cta(bar_free, (uint32_t)lane));   // this warp no longer reads any CTA's part
      } else if (TICKET) {
        // A wait that gives up leaves this warp walking the loop without touching memory, so that the two
        // barriers of the epilogue warps below are still met by all of them.
        const int buf = gc % NB;
        if (alive) alive = mbar_wait(bar_tfull + 8u * buf, (gc / NB) & 1, abort_flag, &g_status_word, 0x400u | buf);
        if (alive) {
          tcgen05_fence_after();
          if (!deps_done) { asm volatile("griddepcontrol.wait;" ::: "memory"); deps_done = true; }
          const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + buf * ACC_STRIDE;
          epilogue_tile(p, BN, part, row, row_ok, tn, taddr, chunk0, CHUNK_STEP);      // this part of the tile -> workspace
          tcgen05_fence_before();
        }
        __syncwarp();
        if (lane == 0 && alive) mbar_arrive(bar_tempty + 8u * buf);
        ++gc;
        // ---- ticket: the part is in the workspace for every CTA to see before the tile's counter moves
        __threadfence();
        asm volatile("bar.sync 1, %0;" ::"n"(EPI_WARPS * 32) : "memory");
        const int tile = tm * p.tiles_n + tn;
        if (p.ticket_all) {
          // ---- one round of work items, each on a CTA of its own (all resident: one CTA per SM, no more items than
          // SMs): the tile's CTAs wait until all of its parts are in the workspace, and each merges one slice of
          // the tile, so that the merge after the last part is one L2 round trip of 256 threads per CTA, not the
          // whole tile on the last arriver.  The counter goes up once per CTA on arrival and once on leaving; the
          // CTA that brings it to twice the number of parts sets it back to zero (all have left their wait by then).
          if (warp == 2 && lane == 0) {
            volatile unsigned int* t = p.tickets + tile;
            atomicAdd(p.tickets + tile, 1u);
            bool ok = true;
            uint64_t t0 = 0;
            for (uint32_t it = 0; *t < (unsigned int)p.n_parts; ++it) {
              __nanosleep(40);
              if ((it & 63u) == 63u) {
                if (*abort_flag) { ok = false; break; }
                const uint64_t now = globaltimer_ns();
                if (t0 == 0) t0 = now;
                else if (now - t0 > WAIT_LIMIT_NS) { *abort_flag = 1; atomicCAS(&g_status_word, 0u, 0x700u); ok = false; break; }
              }
            }
            if (ok) {
              const unsigned int old = atomicAdd(p.tickets + tile, 1u);
              if (old == (unsigned int)(2 * p.n_parts - 1)) *t = 0u;
            }
            *ticket_flag = ok ? 1 : 0;
          }
          asm volatile("bar.sync 1, %0;" ::"n"(EPI_WARPS * 32) : "memory");
          if (*ticket_flag && alive) {
            __threadfence();
            const int tile_rows = min(BM, p.M - tm * BM);
            const int c4s = BN >> 2;
            const int units = tile_rows * c4s;
            const int per = (units + p.n_parts - 1) / p.n_parts;
            const int u_end = min(units, (part + 1) * per);
            const int64_t part_stride = (int64_t)p.M * p.ldw;
            for (int u = part * per + (warp - 2) * 32 + lane; u < u_end; u += EPI_WARPS * 32) {
              const int r_t = u / c4s, c4 = u - r_t * c4s;
              const int col0 = tn * BN + 4 * c4;
              if (col0 >= p.N) continue;
              const int64_t grow = (int64_t)tm * BM + r_t;
              const int64_t off = grow * p.ldw + col0;
              float4 v[8];
#pragma unroll
              for (int s2 = 0; s2 < 8; ++s2) {
                if (s2 < p.n_parts) {
                  if (p.ws_dtype == RG_F32) {
                    v[s2] = __ldcg(reinterpret_cast<const float4*>(static_cast<const float*>(p.ws) + s2 * part_stride + off));
                  } else {
                    const uint2 w = __ldcg(reinterpret_cast<const uint2*>(static_cast<const uint16_t*>(p.ws) + s2 * part_stride + off));
                    v[s2] = p.ws_dtype == RG_F16 ? make_float4(f16_bits_to_f32(w.x & 0xffffu), f16_bits_to_f32(w.x >> 16), f16_bits_to_f32(w.y & 0xffffu), f16_bits_to_f32(w.y >> 16))
                                                 : make_float4(bf16_bits_to_f32(w.x & 0xffffu), bf16_bits_to_f32(w.x >> 16), bf16_bits_to_f32(w.y & 0xffffu), bf16_bits_to_f32(w.y >> 16));
                  }
                }
              }
              const float4 acc = p.merge_dtype == RG_F32 ? merge_upto8<false>(v, p.n_parts, p.tree, p.merge_dtype)
                                                          : merge_upto8<true>(v, p.n_parts, p.tree, p.merge_dtype);
              finish_and_store4(p.epi, p.C, p.ldc, p.c_dtype, p.N, grow, col0, acc);
            }
          }
          continue;
        }
        if (warp == 2 && lane == 0) {
          const unsigned int old = atomicAdd(p.tickets + tile, 1u);
          const bool last = old == (unsigned int)(p.n_parts - 1);
          if (last) p.tickets[tile] = 0u;                  // nobody touches it again before the next call
          *ticket_flag = last ? 1 : 0;
        }
        asm volatile("bar.sync 1, %0;" ::"n"(EPI_WARPS * 32) : "memory");
        if (*ticket_flag && alive) {
          // ---- this CTA stored the tile's last part: merge all of them (read at L2: other SMs wrote them)
          __threadfence();
          const int tile_rows = min(BM, p.M - tm * BM);
          const int c4s = BN >> 2;
          const int units = tile_rows * c4s;
          const int64_t part_stride = (int64_t)p.M * p.ldw;
          for (int u = (warp - 2) * 32 + lane; u < units; u += EPI_WARPS * 32) {
            const int r_t = u / c4s, c4 = u - r_t * c4s;
            const int col0 = tn * BN + 4 * c4;
            if (col0 >= p.N) continue;
            const int64_t grow = (int64_t)tm * BM + r_t;
            const int64_t off = grow * p.ldw + col0;
            float4 v[8];
#pragma unroll
            for (int s2 = 0; s2 < 8; ++s2) {
              if (s2 < p.n_parts) {
                if (p.ws_dtype == RG_F32) {
                  v[s2] = __ldcg(reinterpret_cast<const float4*>(static_cast<const float*>(p.ws) + s2 * part_stride + off));
                } else {
                  const uint2 w = __ldcg(reinterpret_cast<const uint2*>(static_cast<const uint16_t*>(p.ws) + s2 * part_stride + off));
                  v[s2] = p.ws_dtype == RG_F16 ? make_float4(f16_bits_to_f32(w.x & 0xffffu), f16_bits_to_f32(w.x >> 16), f16_bits_to_f32(w.y & 0xffffu), f16_bits_to_f32(w.y >> 16))
                                               : make_float4(bf16_bits_to_f32(w.x & 0xffffu), bf16_bits_to_f32(w.x >> 16), bf16_bits_to_f32(w.y & 0xffffu), bf16_bits_to_f32(w.y >> 16));
                }
              }
            }
            const float4 acc = p.merge_dtype == RG_F32 ? merge_upto8<false>(v, p.n_parts, p.tree, p.merge_dtype)
                                                        : merge_upto8<true>(v, p.n_parts, p.tree, p.merge_dtype);
            finish_and_store4(p.epi, p.C, p.ldc, p.c_dtype, p.N, grow, col0, acc);
          }
        }
      } else if (!GROUPED) {
        const int buf = gc % NB;
        if (!mbar_wait(bar_tfull + 8u * buf, (gc / NB) & 1, abort_flag, &g_status_word, 0x400u | buf)) { alive = false; break; }
        tcgen05_fence_after();
        if (!deps_done) { asm volatile("griddepcontrol.wait;" ::: "memory"); deps_done = true; }
        const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + buf * ACC_STRIDE;
        epilogue_tile(p, BN, part, row, row_ok, tn, taddr, chunk0, CHUNK_STEP);
        tcgen05_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_tempty + 8u * buf);
        ++gc;
      } else if (EPI_WARPS >= 8) {                          // the second cut level runs with eight or sixteen epilogue warps
        GroupedAcc<NCH> acc;
        for (int g = 0; g < ngroups && alive; ++g, ++gc) {
          const int buf = gc % NB;
          if (!mbar_wait(bar_tfull + 8u * buf, (gc / NB) & 1, abort_flag, &g_status_word, 0x400u | buf)) { alive = false; break; }
          tcgen05_fence_after();
          if (!deps_done) { asm volatile("griddepcontrol.wait;" ::: "memory"); deps_done = true; }
          const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + buf * ACC_STRIDE;
          grouped_add<NCH, EPI_WARPS / 4>(p, BN, tn, taddr, chunk0, g == 0, acc);
          tcgen05_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_tempty + 8u * buf);
        }
        if (alive) grouped_finish<NCH, EPI_WARPS / 4>(p, BN, part, row, row_ok, tn, chunk0, acc);
      }
    }
  }

  // ---------------------------------------------------------------- teardown
  if (warp == 1 && lane == 0) RG_STAMP(4);                // last step issued
  __syncthreads();
  if (threadIdx.x == 0) RG_STAMP(5);                      // all roles done
  if (*abort_flag) {
    // let copies and steps already in flight land before shared and tensor memory go away
    const uint64_t t0 = globaltimer_ns();
    while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
    __syncthreads();
  }
  if (CLUSTER) cluster_sync_all();   // other CTAs may still be reading this CTA's part or arriving on its barriers
  if (warp == 1) {
    tcgen05_fence_after();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

// ------------------------------------------------------------------ two-SM kernel
// Same arithmetic, different schedule: two CTAs of a cluster share one 256 x BN output tile.
// CTA r loads rows [128r, 128r+128) of the A tile and rows [BN/2*r, ...) of the B tile into its own
// shared memory; the even CTA issues tcgen05.mma.cta_group::2 (M = 256), which reads both CTAs'
// shared memory and writes each CTA's 128 rows of the accumulator into that CTA's tensor memory.
// Each CTA moves half the B bytes, so a stage is 16 KiB + BN*64 B and the ring is deeper.
//   full[s]   lives in the even CTA; both CTAs' boxes count their bytes on it
//   empty[s]  in each CTA; tcgen05.commit arrives on both
//   tfull[b]  in each CTA; tcgen05.commit arrives on both
//   tempty[b] in the even CTA; the epilogue warps of both CTAs arrive on it
// GROUPED: the second cut level on the pair (see the one-CTA kernel): the issuing CTA closes an accumulator
// every inner_span k, the epilogue warps of both CTAs chain the closed groups in registers.
// BN_T = 0: the tile width is a launch parameter (any multiple of 16 from 32 to 256): a CTA then reads
// 128 + width/2 operand rows per step where the one-CTA kernel reads 128 + width, which is what a step's time is
// made of below 256 columns.  The widths that large problems use (256, 128) keep their compile-time forms.
template <int BN_T, int KSUB, int KIND, bool GROUPED = false>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_tcgen05_pair_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                         const GemmParams p) {
  constexpr bool RT = BN_T == 0;
  static_assert(!(RT && GROUPED), "the second cut level on the pair is built for 128 and 256 columns");
  const int BN = RT ? p.bn : BN_T;
  const int ACC = RT ? 256 : BN_T;                                          // tensor-memory columns between the two accumulators
  constexpr uint32_t A_BOX_BYTES = BM * KBOX * 2;
  const uint32_t B_BOX_BYTES = (uint32_t)(BN / 2) * KBOX * 2;
  const uint32_t STAGE_BYTES = KSUB * (A_BOX_BYTES + B_BOX_BYTES);          // per CTA
  constexpr uint32_t TMEM_COLS = RT ? 512u : 2u * BN_T;
  const uint32_t IDESC = RT ? p.idesc : make_idesc(BN_T, 2 * BM, idesc_format(KIND));

  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const int S = p.num_stages;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem_gen + (size_t)S * STAGE_BYTES);
  const uint32_t bar_full = smem_u32(bars);
  const uint32_t bar_empty = bar_full + 8u * S;
  const uint32_t bar_tfull = bar_empty + 8u * S;
  const uint32_t bar_tempty = bar_tfull + 16u;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * S + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();                 // 0 = the CTA that issues the steps
  const int pair_id = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
  const int total_work = p.tiles_m * p.tiles_n * p.n_parts;   // tiles_m counts 256-row tiles here

  if (threadIdx.x == 0) {
    prefetch_tensormap(&tmap_a);
    prefetch_tensormap(&tmap_b);
    for (int s = 0; s < S; ++s) { mbar_init(bar_full + 8u * s, 1); mbar_init(bar_empty + 8u * s, 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(bar_tfull + 8u * b, 1); mbar_init(bar_tempty + 8u * b, 2 * NUM_EPI_WARPS); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc_pair(smem_u32(tmem_slot), TMEM_COLS);
    tmem_relinquish_pair();
  }
  tcgen05_fence_before();
  __syncthreads();
  cluster_sync_all();                                      // both CTAs' barriers exist before any remote arrive
  tcgen05_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // a split-K merge launched behind this kernel may be scheduled now; it still waits for this grid to finish
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (both CTAs)
    // 2*KSUB lanes, one box each, converged: one instruction issue starts all of a stage's copies.
    if (lane < 2 * KSUB) {
      const bool is_b = lane >= KSUB;
      const int sub = is_b ? lane - KSUB : lane;
      const CUtensorMap* map = is_b ? &tmap_b : &tmap_a;
      const uint32_t box_off = is_b ? KSUB * A_BOX_BYTES + sub * B_BOX_BYTES : sub * A_BOX_BYTES;
      int stage = 0; uint32_t phase = 0;
      bool alive = true;
      // launched with programmatic stream serialisation like the one-CTA kernel: the kernels ahead in the stream
      // are waited for immediately before this role's first access to global memory (not at all when neither operand
      // is written by work in flight, b_static = 2: the epilogue still waits before its first store)
      if (p.b_static < 2) asm volatile("griddepcontrol.wait;" ::: "memory");
      for (int w = pair_id; w < total_work && alive; w += num_pairs) {
        int part, tm, tn;
        decode_work(p, w, part, tm, tn);
        const int k_begin = p.part_begin[part], k_end = p.part_end[part];
        const int y = is_b ? tn * BN + (int)rank * (BN / 2) : tm * 2 * BM + (int)rank * BM;
        for (int k0 = k_begin; k0 < k_end; k0 += KBOX * KSUB) {
          if (!mbar_wait(bar_empty + 8u * stage, phase ^ 1u, abort_flag, &g_status_word, 0x900u | stage)) { alive = false; break; }
          const uint32_t full_local = bar_full + 8u * stage;
          if (lane == 0 && rank == 0) mbar_expect_tx(full_local, 2u * STAGE_BYTES);      // bytes of both CTAs
          const uint32_t full = map_to_cta(full_local, 0);
          tma_load_2d_pair(smem_base + stage * STAGE_BYTES + box_off, map, k0 + sub * KBOX, y, full);
          if (++stage == S) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (even CTA only)
    // the whole warp walks the loop converged, an elected lane issues (see the one-CTA kernel)
    if (rank == 0) {
      const bool leader = elect_one();
      int stage = 0; uint32_t phase = 0;
      bool alive = true;
      int it = 0;
      const uint64_t desc_a0 = make_kmajor_sw128_desc(smem_base);
      const uint64_t desc_b0 = make_kmajor_sw128_desc(smem_base + KSUB * A_BOX_BYTES);
      // With a ring of exactly three stages (the default of the widest tile) whole turns of the ring are
      // issued from descriptor words computed once, with every barrier address a constant: this thread's
      // instruction stream is on the critical path whenever the epilogue warps compete for issue slots.
      constexpr int G = KSUB == 2 ? 3 : 7, STEPS = KSUB * (KBOX / UMMA_K);
      const uint32_t desc_hi = (uint32_t)(desc_a0 >> 32);
      uint32_t alo[G][STEPS], blo[G][STEPS];
#pragma unroll
      for (int g = 0; g < G; ++g)
#pragma unroll
        for (int i = 0; i < STEPS; ++i) {
          const uint32_t off = (uint32_t)((g * STAGE_BYTES) >> 4) + 2u * (i % (KBOX / UMMA_K));
          alo[g][i] = (uint32_t)desc_a0 + off + (((i / (KBOX / UMMA_K)) * A_BOX_BYTES) >> 4);
          blo[g][i] = (uint32_t)desc_b0 + off + (((i / (KBOX / UMMA_K)) * B_BOX_BYTES) >> 4);
        }
      if (GROUPED) {
        // step by step: a step that reaches the end of its group closes the accumulator and opens the other one
        int gc = 0;                                       // accumulators handed to the epilogue so far
        for (int w = pair_id; w < total_work && alive; w += num_pairs) {
          int part, tm, tn;
          decode_work(p, w, part, tm, tn);
          const int k_begin = p.part_begin[part], k_end = p.part_end[part];
          const int span = p.inner_span > 0 ? p.inner_span : (k_end - k_begin);
          int group_end = k_begin, buf = 0;
          uint32_t d_tmem = 0, accumulate = 0;
          for (int k0 = k_begin; k0 < k_end && alive; k0 += KBOX * KSUB) {
            if (!warp_mbar_wait(bar_full + 8u * stage, phase, abort_flag, &g_status_word, 0xb00u | stage)) { alive = false; break; }
            tcgen05_fence_after();
            const uint64_t adesc0 = desc_a0 + (uint64_t)((stage * STAGE_BYTES) >> 4);
            const uint64_t bdesc0 = desc_b0 + (uint64_t)((stage * STAGE_BYTES) >> 4);
#pragma unroll 1
            for (int sa = 0; sa < KSUB * (KBOX / UMMA_K); ++sa) {
              const int sub = sa / (KBOX / UMMA_K), a = sa % (KBOX / UMMA_K);
              const int kk = k0 + sub * KBOX + a * UMMA_K;
              if (kk >= k_end) break;
              if (kk >= group_end) {
                if (kk > k_begin) { if (leader) umma_commit_pair(bar_tfull + 8u * buf); ++gc; }
                buf = gc & 1;
                if (!warp_mbar_wait(bar_tempty + 8u * buf, ((gc >> 1) & 1) ^ 1u, abort_flag, &g_status_word, 0xa00u | buf)) { alive = false; break; }
                tcgen05_fence_after();
                d_tmem = tmem_base + buf * ACC;
                accumulate = 0;                            // every part and every group starts from zero
                group_end = kk + span;
              }
              if (leader) umma_pair<KIND>(d_tmem, adesc0 + (uint64_t)((sub * A_BOX_BYTES) >> 4) + 2u * a,
                                          bdesc0 + (uint64_t)((sub * B_BOX_BYTES) >> 4) + 2u * a, IDESC, accumulate);
              accumulate = 1;
            }
            if (!alive) break;
            if (leader) umma_commit_pair(bar_empty + 8u * stage);
            if (++stage == S) { stage = 0; phase ^= 1u; }
          }
          if (alive) { if (leader) umma_commit_pair(bar_tfull + 8u * buf); ++gc; }
        }
      }
      for (int w = pair_id; !GROUPED && w < total_work && alive; w += num_pairs, ++it) {
        int part, tm, tn;
        decode_work(p, w, part, tm, tn);
        const int k_begin = p.part_begin[part], k_end = p.part_end[part];
        const int buf = it & 1;
        const uint32_t acc_phase = (it >> 1) & 1;
        if (!warp_mbar_wait(bar_tempty + 8u * buf, acc_phase ^ 1u, abort_flag, &g_status_word, 0xa00u | buf)) { alive = false; break; }
        tcgen05_fence_after();
        const uint32_t d_tmem = tmem_base + buf * ACC;
        uint32_t accumulate = 0;                        // every part starts from a zero accumulator
        for (int k0 = k_begin; k0 < k_end; k0 += KBOX * KSUB) {
          if (S == G && stage == 0 && k0 + G * KBOX * KSUB <= k_end) {
            // one whole turn of the ring
#pragma unroll
            for (int g = 0; g < G; ++g) {
              if (alive && !warp_mbar_wait(bar_full + 8u * g, phase, abort_flag, &g_status_word, 0xb00u | g)) alive = false;
              if (alive) {
                tcgen05_fence_after();
#pragma unroll
                for (int i = 0; i < STEPS; ++i) {
                  if (leader) {
                    if (g | i) umma_pair_lo<KIND, true>(d_tmem, alo[g][i], blo[g][i], desc_hi, IDESC, 1u);
                    else umma_pair_lo<KIND, false>(d_tmem, alo[0][0], blo[0][0], desc_hi, IDESC, accumulate);
                  }
                }
                if (leader) umma_commit_pair(bar_empty + 8u * g);
              }
            }
            if (!alive) break;
            accumulate = 1;
            phase ^= 1u;
            k0 += (G - 1) * KBOX * KSUB;                  // the loop adds the last stage's width
            continue;
          }
          if (!warp_mbar_wait(bar_full + 8u * stage, phase, abort_flag, &g_status_word, 0xb00u | stage)) { alive = false; break; }
          tcgen05_fence_after();
          // descriptors differ from the stage-0 ones only in the 16-byte-unit start address (low word)
          const uint64_t adesc0 = desc_a0 + (uint64_t)((stage * STAGE_BYTES) >> 4);
          const uint64_t bdesc0 = desc_b0 + (uint64_t)((stage * STAGE_BYTES) >> 4);
          if (k0 + KBOX * KSUB <= k_end) {
            // whole stage inside the part: 4*KSUB steps, ascending k, no per-step tests; the descriptors'
            // high words are the same for every tile, and the low words never carry into them
            const uint32_t a_lo = (uint32_t)adesc0, b_lo = (uint32_t)bdesc0, hi = (uint32_t)(desc_a0 >> 32);
#pragma unroll
            for (int sub = 0; sub < KSUB; ++sub) {
#pragma unroll
              for (int a = 0; a < KBOX / UMMA_K; ++a) {
                const uint32_t al = a_lo + ((sub * A_BOX_BYTES) >> 4) + 2u * a, bl = b_lo + ((sub * B_BOX_BYTES) >> 4) + 2u * a;
                if (leader) {
                  if (sub | a) umma_pair_lo<KIND, true>(d_tmem, al, bl, hi, IDESC, 1u);
                  else umma_pair_lo<KIND, false>(d_tmem, al, bl, hi, IDESC, accumulate);
                }
              }
            }
            accumulate = 1;
          } else {
#pragma unroll
            for (int sub = 0; sub < KSUB; ++sub) {
#pragma unroll
              for (int a = 0; a < KBOX / UMMA_K; ++a) {
                if (k0 + sub * KBOX + a * UMMA_K < k_end) {   // ascending k; nothing past the end of the part
                  if (leader) umma_pair<KIND>(d_tmem, adesc0 + (uint64_t)((sub * A_BOX_BYTES) >> 4) + 2u * a,
                                 bdesc0 + (uint64_t)((sub * B_BOX_BYTES) >> 4) + 2u * a, IDESC, accumulate);
                  accumulate = 1;
                }
              }
            }
          }
          if (leader) umma_commit_pair(bar_empty + 8u * stage);   // frees the stage in both CTAs
          if (++stage == S) { stage = 0; phase ^= 1u; }
        }
        if (alive && leader) umma_commit_pair(bar_tfull + 8u * buf);   // accumulator complete, in both CTAs
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue warps (both CTAs)
    const int quarter = warp & 3;
    const int chunk0 = (warp - 2) >> 2;
    const uint32_t tempty_leader = map_to_cta(bar_tempty, 0);
    bool alive = true;
    int it = 0;
    bool deps_done = false;
    if (GROUPED) {
      int gc = 0;
      for (int w = pair_id; w < total_work && alive; w += num_pairs) {
        int part, tm, tn;
        decode_work(p, w, part, tm, tn);
        const int klen = p.part_end[part] - p.part_begin[part];
        const int ngroups = p.inner_span > 0 ? (klen + p.inner_span - 1) / p.inner_span : 1;
        const int64_t row = (int64_t)tm * 2 * BM + (int64_t)rank * BM + quarter * 32 + lane;
        GroupedAcc<(RT ? 64 : BN_T) / 64> acc;
        for (int g = 0; g < ngroups && alive; ++g, ++gc) {
          const int buf = gc & 1;
          if (!mbar_wait(bar_tfull + 8u * buf, (gc >> 1) & 1, abort_flag, &g_status_word, 0xc00u | buf)) { alive = false; break; }
          tcgen05_fence_after();
          if (!deps_done) { asm volatile("griddepcontrol.wait;" ::: "memory"); deps_done = true; }
          const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + buf * ACC;
          grouped_add(p, BN, tn, taddr, chunk0, g == 0, acc);
          tcgen05_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(tempty_leader + 8u * buf);
        }
        if (alive) grouped_finish(p, BN, part, row, row < p.M, tn, chunk0, acc);
      }
    }
    for (int w = pair_id; !GROUPED && w < total_work && alive; w += num_pairs, ++it) {
      int part, tm, tn;
      decode_work(p, w, part, tm, tn);
      const int buf = it & 1;
      const uint32_t acc_phase = (it >> 1) & 1;
      if (!mbar_wait(bar_tfull + 8u * buf, acc_phase, abort_flag, &g_status_word, 0xc00u | buf)) { alive = false; break; }
      tcgen05_fence_after();
      if (!deps_done) { asm volatile("griddepcontrol.wait;" ::: "memory"); deps_done = true; }
      const int64_t row = (int64_t)tm * 2 * BM + (int64_t)rank * BM + quarter * 32 + lane;
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + buf * ACC;
      epilogue_tile(p, BN, part, row, row < p.M, tn, taddr, chunk0);
      tcgen05_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(tempty_leader + 8u * buf);
    }
  }

  // ---------------------------------------------------------------- teardown
  __syncthreads();
  if (*abort_flag) {
    const uint64_t t0 = globaltimer_ns();
    while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
    __syncthreads();
  }
  cluster_sync_all();          // the peer may still be reading this CTA's shared memory or arriving on its barriers
  if (warp == 1) {
    tcgen05_fence_after();
    tmem_dealloc_pair(tmem_base, TMEM_COLS);
  }
}

// -------------------------------------------------------------- split-K merge
struct FixupParams {
  const void* ws;
  int64_t ldw;
  int32_t M, N, S, tree;
  int32_t partial_dtype, merge_dtype;
  int32_t launch_seq;     // the GEMM launch this merge belongs to (timeline stamps only)
  void* C;
  int64_t ldc;
  int32_t c_dtype;
  EpilogueArgs epi;
};

// One thread per (row, 4 consecutive columns).  The parts are combined in the descriptor's tree
// with fp32 adds, the running sum kept at merge_dtype (an add whose result is rounded to bf16 when
// the sum is kept at bf16); BALANCED is evaluated with a binary-counter stack, which visits
// exactly the aligned pairs of the level-by-level definition.
template <bool PART_16, bool MERGE_16>
__global__ void __launch_bounds__(256) splitk_fixup_kernel(const FixupParams p) {
  const int64_t ncol4 = (p.N + 3) / 4;
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  // launched with programmatic stream serialisation: the grid may start while the GEMM kernel is
  // still draining; nothing is read before that kernel has completed and flushed its stores.  A
  // kernel launched the same way behind this one may set itself up meanwhile.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
#ifdef RG_TIMELINE
  if (threadIdx.x == 0 && blockIdx.x < 512) g_timeline[p.launch_seq & 7][blockIdx.x][6] = globaltimer_ns();
#endif
  asm volatile("griddepcontrol.wait;" ::: "memory");
#ifdef RG_TIMELINE
  if (threadIdx.x == 0 && blockIdx.x < 512) g_timeline[p.launch_seq & 7][blockIdx.x][7] = globaltimer_ns();
#endif
  if (idx >= (int64_t)p.M * ncol4) return;
  const int64_t row = idx / ncol4;
  const int col0 = (int)(idx - row * ncol4) * 4;
  const int64_t part_stride = (int64_t)p.M * p.ldw;
  const int64_t off = row * p.ldw + col0;
  auto load = [&](int s) -> float4 {
    if (PART_16) {
      const uint2 w = *reinterpret_cast<const uint2*>(static_cast<const uint16_t*>(p.ws) + s * part_stride + off);
      if (p.partial_dtype == RG_F16)
        return make_float4(f16_bits_to_f32(w.x & 0xffffu), f16_bits_to_f32(w.x >> 16),
                           f16_bits_to_f32(w.y & 0xffffu), f16_bits_to_f32(w.y >> 16));
      return make_float4(bf16_bits_to_f32(w.x & 0xffffu), bf16_bits_to_f32(w.x >> 16),
                         bf16_bits_to_f32(w.y & 0xffffu), bf16_bits_to_f32(w.y >> 16));
    }
    return *reinterpret_cast<const float4*>(static_cast<const float*>(p.ws) + s * part_stride + off);
  };
  const int merge_dtype = p.merge_dtype;
  auto add1 = [merge_dtype](float a, float b) -> float {
    const float v = f_add(a, b);
    return MERGE_16 ? round_through(v, merge_dtype) : v;
  };
  auto add4 = [&](const float4& a, const float4& b) -> float4 {
    return make_float4(add1(a.x, b.x), add1(a.y, b.y), add1(a.z, b.z), add1(a.w, b.w));
  };
  // bias and residual are requested first so that their latency hides behind the parts'
  float bias4[4] = {0.0f, 0.0f, 0.0f, 0.0f}, res4[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    if (col0 + c < p.N) {
      if (p.epi.bias) bias4[c] = load_scalar(p.epi.bias, p.epi.bias_dtype, col0 + c);
      if (p.epi.residual) res4[c] = load_scalar(p.epi.residual, p.epi.residual_dtype, row * p.epi.ldr + col0 + c);
    }
  }
  // parts are fetched eight at a time (all eight loads in flight together), then folded in order
  float4 acc;
  if (p.tree == RG_TREE_LEFT) {
    for (int s0 = 0; s0 < p.S; s0 += 8) {
      float4 part[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) if (s0 + i < p.S) part[i] = load(s0 + i);
#pragma unroll
      for (int i = 0; i < 8; ++i) if (s0 + i < p.S) acc = (s0 + i == 0) ? part[i] : add4(acc, part[i]);
    }
  } else {
    // binary-counter stack with every index a compile-time constant, so it lives in registers
    float4 stack[7];
    for (int s0 = 0; s0 < p.S; s0 += 8) {
      float4 part[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) if (s0 + i < p.S) part[i] = load(s0 + i);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        if (s0 + i < p.S) {
          const int s = s0 + i;
          float4 v = part[i];
          bool placed = false;
#pragma unroll
          for (int b = 0; b < 7; ++b) {
            if (!placed) {
              if ((s >> b) & 1) v = add4(stack[b], v);
              else { stack[b] = v; placed = true; }
            }
          }
        }
      }
    }
    // leftovers: the lowest pending level moves up unchanged until it meets a sibling
    bool have = false;
#pragma unroll
    for (int b = 0; b < 7; ++b) {
      if (!((p.S >> b) & 1)) continue;
      if (!have) { acc = stack[b]; have = true; }
      else acc = add4(stack[b], acc);
    }
  }
  // bias -> SiLU -> residual -> one rounding, as in the GEMM kernels' epilogue
  float v[4] = {acc.x, acc.y, acc.z, acc.w};
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    if (p.epi.bias) v[c] = f_add(v[c], bias4[c]);
    if (p.epi.act == 1) v[c] = rg_silu(v[c]);
    if (p.epi.residual) v[c] = f_add(v[c], res4[c]);
  }
  uint16_t* const c16 = static_cast<uint16_t*>(p.C) + row * p.ldc + col0;
  if (col0 + 4 <= p.N && p.c_dtype != RG_F32 && (reinterpret_cast<uintptr_t>(c16) & 7) == 0) {
    // four 16-bit outputs as one 8-byte store
    uint2 o;
    o.x = pack_16x2(v[0], v[1], p.c_dtype);
    o.y = pack_16x2(v[2], v[3], p.c_dtype);
    *reinterpret_cast<uint2*>(c16) = o;
  } else {
#pragma unroll
    for (int c = 0; c < 4; ++c)
      if (col0 + c < p.N) store_scalar(p.C, p.c_dtype, row * p.ldc + col0 + c, v[c]);
  }
}

// The merge behind calls that do not depend on each other (b_static = 2), at most eight parts: 128-thread CTAs, two
// units of four columns per thread with the loads of both in flight together, at most 120 registers, so that four
// CTAs fit an SM.  The GEMM ahead of it leaves this kernel a few SMs of its own (GemmPlan::reserve_sms): its CTAs
// become resident there while that GEMM is still running, and they are not in the way when the next call's GEMM
// CTAs move in as this call's leave.  (The 256-thread CTAs of the general kernel cannot sit beside a GEMM CTA: the
// register file is four partitions of 16 K, a GEMM CTA's ten warps leave 4 K free on two of them, and two merge
// warps need more.  They take SMs as GEMM CTAs leave, two to an SM, and the next call's CTAs on those SMs start late.)
template <bool PART_16, bool MERGE_16>
__global__ void __maxnreg__(120) splitk_fixup_small_kernel(const FixupParams p) {
  const int64_t ncol4 = (p.N + 3) / 4, total = (int64_t)p.M * ncol4;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int64_t part_stride = (int64_t)p.M * p.ldw;
  int64_t row[2], off[2]; int col0[2]; bool on[2];
  float bias4[2][4], res4[2][4];
  float4 part[2][8];
#pragma unroll
  for (int u = 0; u < 2; ++u) {
    const int64_t idx = (int64_t)blockIdx.x * 256 + u * 128 + threadIdx.x;
    on[u] = idx < total;
    row[u] = on[u] ? idx / ncol4 : 0;
    col0[u] = on[u] ? (int)(idx - row[u] * ncol4) * 4 : 0;
    off[u] = row[u] * p.ldw + col0[u];
    // bias and residual are requested first so that their latency hides behind the parts'
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      bias4[u][c] = 0.0f; res4[u][c] = 0.0f;
      if (on[u] && col0[u] + c < p.N) {
        if (p.epi.bias) bias4[u][c] = load_scalar(p.epi.bias, p.epi.bias_dtype, col0[u] + c);
        if (p.epi.residual) res4[u][c] = load_scalar(p.epi.residual, p.epi.residual_dtype, row[u] * p.epi.ldr + col0[u] + c);
      }
    }
  }
#pragma unroll
  for (int u = 0; u < 2; ++u) {
#pragma unroll
    for (int s = 0; s < 8; ++s) {
      if (on[u] && s < p.S) {
        if (PART_16) {
          const uint2 w = *reinterpret_cast<const uint2*>(static_cast<const uint16_t*>(p.ws) + s * part_stride + off[u]);
          part[u][s] = p.partial_dtype == RG_F16
              ? make_float4(f16_bits_to_f32(w.x & 0xffffu), f16_bits_to_f32(w.x >> 16), f16_bits_to_f32(w.y & 0xffffu), f16_bits_to_f32(w.y >> 16))
              : make_float4(bf16_bits_to_f32(w.x & 0xffffu), bf16_bits_to_f32(w.x >> 16), bf16_bits_to_f32(w.y & 0xffffu), bf16_bits_to_f32(w.y >> 16));
        } else {
          part[u][s] = *reinterpret_cast<const float4*>(static_cast<const float*>(p.ws) + s * part_stride + off[u]);
        }
      }
    }
  }
#pragma unroll
  for (int u = 0; u < 2; ++u) {
    if (!on[u]) continue;
    const float4 acc = merge_upto8<MERGE_16>(part[u], p.S, p.tree, p.merge_dtype);
    // bias -> SiLU -> residual -> one rounding, as in the GEMM kernels' epilogue
    float v[4] = {acc.x, acc.y, acc.z, acc.w};
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      if (p.epi.bias) v[c] = f_add(v[c], bias4[u][c]);
      if (p.epi.act == 1) v[c] = rg_silu(v[c]);
      if (p.epi.residual) v[c] = f_add(v[c], res4[u][c]);
    }
    uint16_t* const c16 = static_cast<uint16_t*>(p.C) + row[u] * p.ldc + col0[u];
    if (col0[u] + 4 <= p.N && p.c_dtype != RG_F32 && (reinterpret_cast<uintptr_t>(c16) & 7) == 0) {
      uint2 o;
      o.x = pack_16x2(v[0], v[1], p.c_dtype);
      o.y = pack_16x2(v[2], v[3], p.c_dtype);
      *reinterpret_cast<uint2*>(c16) = o;
    } else {
#pragma unroll
      for (int c = 0; c < 4; ++c)
        if (col0[u] + c < p.N) store_scalar(p.C, p.c_dtype, row[u] * p.ldc + col0[u] + c, v[c]);
    }
  }
}

// -------------------------------------------------------------- self-test of the bounded wait
// One CTA, two warps, no copies and no tensor memory: a barrier that nothing ever arrives on.  Warp 0
// waits on it with the caller's (short) limit, gives up, raises the CTA's abort flag and records
// `code` in the status word; warp 1 waits on the same barrier with the library's long limit and must
// leave as soon as it sees the flag.  The kernel then returns normally: this is the path a real kernel
// takes when a copy or a tensor-core step it waits for never completes.
__global__ void __launch_bounds__(64) bounded_wait_selftest_kernel(uint64_t limit_ns, uint32_t code, unsigned int* left_early) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ int abort_flag_s;
  volatile int* abort_flag = &abort_flag_s;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag_s = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const int warp = threadIdx.x >> 5;
  bool ok;
  if (warp == 0) ok = mbar_wait(smem_u32(&bar), 0, abort_flag, &g_status_word, code, limit_ns);
  else ok = mbar_wait(smem_u32(&bar), 0, abort_flag, &g_status_word, code | 0x80u);      // 2 s limit: leaves through the flag
  if (!ok && (threadIdx.x & 31) == 0) atomicAdd(left_early, 1u);
}

// ------------------------------------------------------------ host: tensor maps
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

// 2-D tensor map (bf16 or fp16 elements) over a row-major [rows, cols] matrix: box = 64 columns x box_rows rows,
// 128-byte swizzle, zero fill outside the matrix (missing products are then exact zeros).  An e4m3
// matrix is described as byte pairs (cols and ld even, checked by the caller): the copy moves the
// same bytes, a box is 128 of its columns, and a zero pair is two zero operands.
bool make_tmap(CUtensorMap* map, const void* ptr, int dtype, int64_t rows, int64_t cols, int64_t ld, int box_rows) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  if (dtype == RG_F8E4M3) { cols /= 2; ld /= 2; }
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  const cuuint32_t box[2] = {(cuuint32_t)KBOX, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUtensorMapDataType tdt = dtype == RG_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : dtype == RG_F8E4M3 ? CU_TENSOR_MAP_DATA_TYPE_UINT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
  return fn(map, tdt, 2, const_cast<void*>(ptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Encoding a tensor map costs a driver call per operand, which shows on GEMMs of a few tens of
// microseconds (App. E, last paragraph: the descriptor path's host cost is visible under ~100 us).  A
// map depends only on (address, type, shape, pitch, box), never on the data, so the last few are kept:
// a decode loop that calls with the same weights and activations buffers encodes nothing.
struct TmapKey {
  const void* ptr; int64_t rows, cols, ld; int32_t dtype, box_rows;
  bool operator==(const TmapKey& o) const {
    return ptr == o.ptr && rows == o.rows && cols == o.cols && ld == o.ld && dtype == o.dtype && box_rows == o.box_rows;
  }
};
constexpr int TMAP_CACHE_ENTRIES = 64;
struct TmapCache {
  std::mutex mu;
  TmapKey key[TMAP_CACHE_ENTRIES];
  CUtensorMap map[TMAP_CACHE_ENTRIES];
  uint64_t stamp[TMAP_CACHE_ENTRIES] = {};   // 0 = empty; otherwise the tick of the last use
  uint64_t tick = 0;
};
TmapCache g_tmaps;

bool cached_tmap(CUtensorMap* out, const void* ptr, int dtype, int64_t rows, int64_t cols, int64_t ld, int box_rows) {
  const TmapKey k{ptr, rows, cols, ld, dtype, box_rows};
  std::lock_guard<std::mutex> lock(g_tmaps.mu);
  int victim = 0;
  for (int i = 0; i < TMAP_CACHE_ENTRIES; ++i) {
    if (g_tmaps.stamp[i] && g_tmaps.key[i] == k) {
      g_tmaps.stamp[i] = ++g_tmaps.tick;
      *out = g_tmaps.map[i];
      return true;
    }
    if (g_tmaps.stamp[i] < g_tmaps.stamp[victim]) victim = i;      // least recently used (or empty)
  }
  if (!make_tmap(out, ptr, dtype, rows, cols, ld, box_rows)) return false;
  g_tmaps.key[victim] = k; g_tmaps.map[victim] = *out; g_tmaps.stamp[victim] = ++g_tmaps.tick;
  return true;
}

constexpr size_t SMEM_LIMIT = 232448;   // 227 KiB of dynamic shared memory per CTA
constexpr size_t SMEM_LIMIT_HALF = 115712;   // 113 KiB: two CTAs (and their 1 KiB system shares) fit the 228 KiB of an SM

// The tensor-core step reads its full row count (128, or 64 for problems of at most 64 rows) from the start
// of an A box even when the box holds fewer rows.  Inside a stage the surplus falls on the boxes behind it;
// what the last A box of the last stage reads past the end of its stage must still lie inside the
// allocation (those rows feed accumulator rows nobody stores).
size_t a_slack_bytes(int bn, int ksub, int a_rows) {
  const int span_rows = a_rows <= 64 ? 64 : BM;
  const int64_t over = (int64_t)(span_rows - a_rows) * KBOX * 2 - (int64_t)ksub * bn * KBOX * 2;
  return over > 0 ? (size_t)over : 0;
}

size_t smem_bytes_for(int bn, int ksub, int stages, int a_rows) {
  const size_t stage = (size_t)ksub * ((size_t)a_rows * KBOX * 2 + (size_t)bn * KBOX * 2);
  return 1024 + stages * stage + a_slack_bytes(bn, ksub, a_rows) + (2 * stages + 8) * 8 + 16;   // room for four accumulator barrier pairs
}

// CLUSTER kernels: two more barriers and the CTA's partial tile behind the plain kernel's layout
size_t cluster_extra_bytes(int bn, int part_rows) { return 16 + (size_t)part_rows * (bn + 4) * 4; }

size_t smem_bytes_for_pair(int bn, int ksub, int stages) {
  const size_t stage = (size_t)ksub * (BM * KBOX * 2 + (size_t)(bn / 2) * KBOX * 2);
  return 1024 + stages * stage + (2 * stages + 4) * 8 + 16;
}

template <int BN, int KSUB, int KIND, bool GROUPED = false>
cudaError_t launch_pair_t(const CUtensorMap& ta, const CUtensorMap& tb, const GemmParams& p, int grid, cudaStream_t st) {
  const size_t smem = smem_bytes_for_pair(BN ? BN : p.bn, KSUB, p.num_stages);
  static DeviceOnce configured;
  const int dev = current_device().dev;
  if (!configured.has(dev)) {
    cudaError_t e = cudaFuncSetAttribute(gemm_tcgen05_pair_kernel<BN, KSUB, KIND, GROUPED>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_LIMIT);
    if (e != cudaSuccess) return e;
    configured.set(dev);
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid, 1, 1);
  cfg.blockDim = dim3(NUM_THREADS, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;     // set-up runs under the tail of the kernel ahead
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, gemm_tcgen05_pair_kernel<BN, KSUB, KIND, GROUPED>, ta, tb, p);
}

// the second cut level on the pair: 64-wide stages
template <int BN>
cudaError_t launch_pair_grouped(const CUtensorMap& ta, const CUtensorMap& tb, const GemmParams& p, int grid, int kind, cudaStream_t st) {
  if (kind == KIND_F16) return launch_pair_t<BN, 1, KIND_F16, true>(ta, tb, p, grid, st);
  if (kind == KIND_F8E4M3) return launch_pair_t<BN, 1, KIND_F8E4M3, true>(ta, tb, p, grid, st);
  return launch_pair_t<BN, 1, KIND_BF16, true>(ta, tb, p, grid, st);
}

template <int BN, int KSUB>
cudaError_t launch_pair(const CUtensorMap& ta, const CUtensorMap& tb, const GemmParams& p, int grid, int kind, cudaStream_t st) {
  if (kind == KIND_F16) return launch_pair_t<BN, KSUB, KIND_F16>(ta, tb, p, grid, st);
  if (kind == KIND_F8E4M3) return launch_pair_t<BN, KSUB, KIND_F8E4M3>(ta, tb, p, grid, st);
  return launch_pair_t<BN, KSUB, KIND_BF16>(ta, tb, p, grid, st);
}

template <int KSUB, bool F8>
cudaError_t configure_cluster_kernel() {
  static DeviceOnce configured;
  const int dev = current_device().dev;
  if (!configured.has(dev)) {
    cudaError_t e = cudaFuncSetAttribute(gemm_tcgen05_kernel<KSUB, F8, true, 8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_LIMIT);
    if (e != cudaSuccess) return e;
    configured.set(dev);
  }
  return cudaSuccess;
}

// The in-cluster split-K kernel: `clusters` clusters of p.n_parts CTAs, launched like the plain kernel
// (programmatic stream serialisation: set-up overlaps the previous kernel's tail).
template <int KSUB, bool F8>
cudaError_t launch_cluster_t(const CUtensorMap& ta, const CUtensorMap& tb, const GemmParams& p, int clusters, cudaStream_t st) {
  const size_t smem = smem_bytes_for(p.bn, KSUB, p.num_stages, (int)(p.a_box_bytes / (KBOX * 2))) + cluster_extra_bytes(p.bn, p.part_rows);
  cudaError_t e = configure_cluster_kernel<KSUB, F8>();
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(clusters * p.n_parts), 1, 1);
  cfg.blockDim = dim3(NUM_THREADS, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)p.n_parts; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, gemm_tcgen05_kernel<KSUB, F8, true, 8>, ta, tb, p);
}

// How many clusters of `csize` CTAs of the in-cluster kernel the device runs at once (each CTA takes a
// whole SM, and a cluster must fit one GPC).  0 if such a cluster cannot be scheduled at all.
template <int KSUB, bool F8>
int query_clusters_t(int csize) {
  if (configure_cluster_kernel<KSUB, F8>() != cudaSuccess) return 0;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(csize * 64), 1, 1);
  cfg.blockDim = dim3(NUM_THREADS, 1, 1);
  cfg.dynamicSmemBytes = SMEM_LIMIT;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)csize; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, gemm_tcgen05_kernel<KSUB, F8, true, 8>, &cfg) != cudaSuccess) { cudaGetLastError(); return 0; }
  return n;
}

template <int KSUB, bool F8, int EPI_WARPS = 8>
cudaError_t launch_one_t(const CUtensorMap& ta, const CUtensorMap& tb, const GemmParams& p, int grid, cudaStream_t st) {
  const size_t smem = smem_bytes_for(p.bn, KSUB, p.num_stages, (int)(p.a_box_bytes / (KBOX * 2)));
  static DeviceOnce configured;
  const int dev = current_device().dev;
  if (!configured.has(dev)) {
    cudaError_t e = cudaFuncSetAttribute(gemm_tcgen05_kernel<KSUB, F8, false, EPI_WARPS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)(EPI_WARPS == 4 ? SMEM_LIMIT_HALF : SMEM_LIMIT));
    if (e != cudaSuccess) return e;
    if (EPI_WARPS == 4) {
      // two CTAs per SM: ask for the largest shared-memory carve-out
      e = cudaFuncSetAttribute(gemm_tcgen05_kernel<KSUB, F8, false, EPI_WARPS>, cudaFuncAttributePreferredSharedMemoryCarveout, 100);
      if (e != cudaSuccess) return e;
    }
    configured.set(dev);
  }
  // programmatic stream serialisation: the CTAs may set themselves up (barriers, tensor memory,
  // descriptor prefetch) while the kernel before this one in the stream drains
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid, 1, 1);
  cfg.blockDim = dim3(64 + 32 * EPI_WARPS, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, gemm_tcgen05_kernel<KSUB, F8, false, EPI_WARPS>, ta, tb, p);
}

// split-K in one launch, the tile's last-arriving CTA merging (TICKET instantiations)
template <int KSUB, bool F8>
cudaError_t launch_ticket_t(const CUtensorMap& ta, const CUtensorMap& tb, const GemmParams& p, int grid, cudaStream_t st) {
  const size_t smem = smem_bytes_for(p.bn, KSUB, p.num_stages, (int)(p.a_box_bytes / (KBOX * 2)));
  static DeviceOnce configured;
  const int dev = current_device().dev;
  if (!configured.has(dev)) {
    cudaError_t e = cudaFuncSetAttribute(gemm_tcgen05_kernel<KSUB, F8, false, 8, false, 2, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_LIMIT);
    if (e != cudaSuccess) return e;
    configured.set(dev);
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid, 1, 1);
  cfg.blockDim = dim3(NUM_THREADS, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, gemm_tcgen05_kernel<KSUB, F8, false, 8, false, 2, true>, ta, tb, p);
}

// the second cut level: 64-wide stages; NCH = 32-column chunks a warp keeps a running sum of.  Eight epilogue warps:
// sixteen with one chunk each measured 8 % slower (702 against 763 TFLOP/s at a group every 64 k): the issuing
// thread paces this mode, and more polling warps take its issue slots.
template <bool F8, int NCH, int EPI = 8>
cudaError_t launch_grouped_t(const CUtensorMap& ta, const CUtensorMap& tb, const GemmParams& p, int grid, cudaStream_t st) {
  const size_t smem = smem_bytes_for(p.bn, 1, p.num_stages, (int)(p.a_box_bytes / (KBOX * 2)));
  static DeviceOnce configured;
  const int dev = current_device().dev;
  if (!configured.has(dev)) {
    cudaError_t e = cudaFuncSetAttribute(gemm_tcgen05_kernel<1, F8, false, EPI, true, NCH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_LIMIT);
    if (e != cudaSuccess) return e;
    configured.set(dev);
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid, 1, 1);
  cfg.blockDim = dim3(64 + 32 * EPI, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, gemm_tcgen05_kernel<1, F8, false, EPI, true, NCH>, ta, tb, p);
}

template <int KSUB>
cudaError_t launch_one(const CUtensorMap& ta, const CUtensorMap& tb, const GemmParams& p, int grid, cudaStream_t st) {
  return p.f8 ? launch_one_t<KSUB, true>(ta, tb, p, grid, st) : launch_one_t<KSUB, false>(ta, tb, p, grid, st);
}
// the form that shares an SM between two CTAs (four epilogue warps, half the shared and tensor memory)
template <int KSUB>
cudaError_t launch_one_half(const CUtensorMap& ta, const CUtensorMap& tb, const GemmParams& p, int grid, cudaStream_t st) {
  return p.f8 ? launch_one_t<KSUB, true, 4>(ta, tb, p, grid, st) : launch_one_t<KSUB, false, 4>(ta, tb, p, grid, st);
}

// The epilogue's SiLU as the kernels apply it: a thread takes 32 consecutive values (one accumulator chunk of one
// row) through epilogue_row_segment, which picks the range-free exponential when no magnitude of the segment
// exceeds 87 and the general one otherwise (see rg_selftest_exp, form 7).  n is a multiple of 32.
__global__ void __launch_bounds__(128) silu_selftest_kernel(const float* __restrict__ x, float* __restrict__ y, int64_t n) {
  EpilogueArgs e{};
  e.act = 1;
  for (int64_t s = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; s * 32 < n; s += (int64_t)gridDim.x * blockDim.x) {
    float v[32];
#pragma unroll
    for (int c = 0; c < 32; ++c) v[c] = x[s * 32 + c];
    epilogue_row_segment(v, e, 0, 0, 32);
#pragma unroll
    for (int c = 0; c < 32; ++c) y[s * 32 + c] = v[c];
  }
}

}  // namespace

rg_status_t launch_silu_selftest(const float* x, float* y, int64_t n, cudaStream_t st) {
  const int64_t need = (n / 32 + 127) / 128;
  silu_selftest_kernel<<<(unsigned)(need < 148 * 8 ? (need < 1 ? 1 : need) : 148 * 8), 128, 0, st>>>(x, y, n);
  return cudaGetLastError() == cudaSuccess ? RG_OK : RG_ERR_CUDA;
}

// The same tensor map for other kernels of the library (boxes of 64 columns x box_rows rows, 128-byte swizzle).
bool make_operand_tmap(CUtensorMap_st* map, const void* ptr, int dtype, int64_t rows, int64_t cols, int64_t ld, int box_rows) {
  return cached_tmap(map, ptr, dtype, rows, cols, ld, box_rows);
}

int a_box_rows_for(int64_t M) { return M >= BM ? BM : (int)((M + 7) / 8 * 8); }

int cluster_part_rows(int64_t M) { return M >= BM ? BM : (int)M; }

constexpr size_t TICKET_TILES_MAX = 16384;

// Bytes in front of the parts that hold the per-tile tickets of the TICKET kernels.  The size does not depend
// on the shape, so a workspace that serves calls of different shapes keeps its tickets where no call's parts
// ever land: 16384 tiles at most.
size_t ticket_bytes() { return TICKET_TILES_MAX * sizeof(unsigned int); }

// cluster_merge: the in-cluster split-K kernel, whose partial tile shares the shared memory with the ring
// (0 stages = it does not fit at all)
int max_stages_for(int bn, int bk, int cta_group, int64_t M, bool cluster_merge, bool half_sm) {
  const int ksub = bk / KBOX;
  int s = 1;
  if (cta_group == 2) { while (s < 8 && smem_bytes_for_pair(bn, ksub, s + 1) <= SMEM_LIMIT) ++s; }
  else {
    const size_t limit = half_sm ? SMEM_LIMIT_HALF : SMEM_LIMIT;
    const size_t extra = cluster_merge ? cluster_extra_bytes(bn, cluster_part_rows(M)) : 0;
    if (smem_bytes_for(bn, ksub, 1, a_box_rows_for(M)) + extra > limit) return 0;
    while (s < 32 && smem_bytes_for(bn, ksub, s + 1, a_box_rows_for(M)) + extra <= limit) ++s;
  }
  return s;
}

// Clusters of `csize` CTAs of the in-cluster split-K kernel that run at once on the current device
// (looked up once per device and cluster size).
int max_active_clusters(int csize, int bk, bool f8) {
  static std::mutex mu;
  static int cache[64][9][2][2];                            // [device][csize][bk == 128][f8], value + 1
  if (csize < 2 || csize > 8 || (bk != 64 && bk != 128)) return 0;
  const int dev = current_device().dev;
  std::lock_guard<std::mutex> lock(mu);
  int* slot = (dev >= 0 && dev < 64) ? &cache[dev][csize][bk == 128][f8 ? 1 : 0] : nullptr;
  if (slot && *slot) return *slot - 1;
  int n;
  if (bk == 128) n = f8 ? query_clusters_t<2, true>(csize) : query_clusters_t<2, false>(csize);
  else n = f8 ? query_clusters_t<1, true>(csize) : query_clusters_t<1, false>(csize);
  if (slot) *slot = n + 1;
  return n;
}

rg_status_t read_and_clear_status(uint32_t* code) {
  unsigned int v = 0, zero = 0;
  if (cudaDeviceSynchronize() != cudaSuccess) return RG_ERR_CUDA;
  if (cudaMemcpyFromSymbol(&v, g_status_word, sizeof(v)) != cudaSuccess) return RG_ERR_CUDA;
  if (v != 0 && cudaMemcpyToSymbol(g_status_word, &zero, sizeof(zero)) != cudaSuccess) return RG_ERR_CUDA;
  if (code) *code = v;
  return v ? RG_ERR_TIMEOUT : RG_OK;
}

rg_status_t launch_wait_selftest(uint64_t limit_ns, uint32_t code, unsigned int* left_early, cudaStream_t st) {
  bounded_wait_selftest_kernel<<<1, 64, 0, st>>>(limit_ns, code, left_early);
  return cudaGetLastError() == cudaSuccess ? RG_OK : RG_ERR_CUDA;
}

#ifdef RG_TIMELINE
extern "C" int rg_debug_read_timeline(unsigned long long* host_out) {     // [8][512][8]
  return cudaMemcpyFromSymbol(host_out, g_timeline, sizeof(g_timeline)) == cudaSuccess ? 0 : 1;
}
#endif

// Launch the GEMM (and the merge when there are cuts).  All arguments were validated by the caller.
rg_status_t launch_gemm(const GemmPlan& plan, const rg_tensor_t* A, const rg_tensor_t* B, const rg_tensor_t* C,
                        const rg_epilogue_t* epi, void* ws, cudaStream_t st) {
  // e4m3 operands: every K quantity below (K, part bounds, inner span) counts byte pairs, so the
  // kernels walk 32-byte steps of an operand row exactly as they do for 16-bit operands
  const int kdiv = A->dtype == RG_F8E4M3 ? 2 : 1;
  const int kind = A->dtype == RG_F16 ? KIND_F16 : A->dtype == RG_F8E4M3 ? KIND_F8E4M3 : KIND_BF16;
  const int64_t M = A->rows, K = A->cols / kdiv, N = B->rows;
  const bool pair = plan.cta_group == 2;
  const int tile_m = pair ? 2 * BM : BM;
  CUtensorMap ta, tb;
  const int a_rows = pair ? BM : a_box_rows_for(M);
  if (!cached_tmap(&ta, A->ptr, A->dtype, M, A->cols, A->ld, a_rows) ||
      !cached_tmap(&tb, B->ptr, B->dtype, N, B->cols, B->ld, pair ? plan.BN / 2 : plan.BN))
    return RG_ERR_CUDA;

  GemmParams p;
  p.M = (int32_t)M; p.N = (int32_t)N; p.K = (int32_t)K;
  p.tiles_m = (int32_t)((M + tile_m - 1) / tile_m);
  p.tiles_n = (int32_t)((N + plan.BN - 1) / plan.BN);
  p.n_parts = plan.n_parts;
  p.num_stages = plan.stages;
  p.raster = plan.raster;
  p.group_m = plan.group_m;
  p.a_box_bytes = (uint32_t)a_rows * KBOX * 2;
  p.slack_bytes = pair ? 0u : (uint32_t)a_slack_bytes(plan.BN, plan.BK / KBOX, a_rows);
  p.bn = plan.BN;
  p.inner_span = plan.inner_span / kdiv;
  p.f8 = kind == KIND_F8E4M3;
  p.b_static = plan.b_static;
  { static std::atomic<int> seq{0}; p.launch_seq = seq.fetch_add(1, std::memory_order_relaxed); }
  // At most 64 rows: the 64-row step reads half the A rows from shared memory, which is what a narrow tile's
  // step time is made of ((rows + width) x 32 bytes at 128 bytes per clock).  Same products, same order.
  p.mma_m = (!pair && M <= 64) ? 64 : BM;
  p.idesc = make_idesc(plan.BN, pair ? 2 * BM : p.mma_m, idesc_format(kind));
  {
    const uint32_t accumulators = (plan.inner_span && !pair && plan.BN <= 128) ? 4u : 2u;   // see NB in the one-CTA kernel
    uint32_t c = 32;
    while (c < accumulators * (uint32_t)((plan.BN + 31) / 32 * 32)) c <<= 1;
    p.tmem_cols = c;
  }
  for (int s = 0; s < plan.n_parts; ++s) { p.part_begin[s] = plan.part_begin[s] / kdiv; p.part_end[s] = plan.part_end[s] / kdiv; }
  EpilogueArgs e{};
  if (epi) {
    e.bias = epi->bias; e.bias_dtype = epi->bias_dtype; e.act = epi->act;
    e.residual = epi->residual; e.residual_dtype = epi->residual_dtype; e.ldr = epi->ldr;
  }
  const bool in_cluster = plan.cluster_merge != 0;            // parts merged inside the GEMM kernel, no workspace
  const bool ticket = plan.ticket_merge != 0;                 // parts through the workspace, merged by the tile's last CTA
  const bool split = plan.n_parts > 1 && !in_cluster;
  p.C = C->ptr; p.ldc = C->ld; p.c_dtype = C->dtype;
  // ticket mode: the tickets sit in front of the parts (see ticket_bytes)
  p.tickets = ticket ? static_cast<unsigned int*>(ws) : nullptr;
  p.ticket_all = 0;                                           // set below, once the number of work items is known
  p.ws = split ? (ticket ? static_cast<void*>(static_cast<uint8_t*>(ws) + ticket_bytes()) : ws) : nullptr;
  p.ws_dtype = plan.partial_dtype;
  p.ldw = (N + 3) / 4 * 4;
  p.epi = (split && !ticket) ? EpilogueArgs{} : e;
  p.tree = plan.tree; p.merge_dtype = plan.merge_dtype;
  p.part_rows = cluster_part_rows(M); p.part_ld = plan.BN + 4;

  const int64_t total = (int64_t)p.tiles_m * p.tiles_n * p.n_parts;
  const int sms = current_device().sms;
  cudaError_t err;
  const int ksub = plan.BK / KBOX;
  if (pair) {
    const int64_t pairs = sms / 2;
    const int grid = 2 * (int)(total < pairs ? total : pairs);
    if (plan.inner_span) {
      if (ksub != 1) return RG_ERR_UNSUPPORTED;
      if (plan.BN == 256) err = launch_pair_grouped<256>(ta, tb, p, grid, kind, st);
      else if (plan.BN == 128) err = launch_pair_grouped<128>(ta, tb, p, grid, kind, st);
      else return RG_ERR_UNSUPPORTED;
    }
    else if (plan.BN == 256 && ksub == 1) err = launch_pair<256, 1>(ta, tb, p, grid, kind, st);
    else if (plan.BN == 256 && ksub == 2) err = launch_pair<256, 2>(ta, tb, p, grid, kind, st);
    else if (plan.BN == 128 && ksub == 1) err = launch_pair<128, 1>(ta, tb, p, grid, kind, st);
    else if (plan.BN == 128 && ksub == 2) err = launch_pair<128, 2>(ta, tb, p, grid, kind, st);
    else if (plan.BN % 16 != 0 || plan.BN < 32 || plan.BN > 256) return RG_ERR_UNSUPPORTED;
    else if (ksub == 1) err = launch_pair<0, 1>(ta, tb, p, grid, kind, st);
    else if (ksub == 2) err = launch_pair<0, 2>(ta, tb, p, grid, kind, st);
    else return RG_ERR_UNSUPPORTED;
  } else if (in_cluster) {
    const int avail = max_active_clusters(plan.n_parts, plan.BK, kind == KIND_F8E4M3);
    if (avail < 1) return RG_ERR_UNSUPPORTED;
    const int64_t tiles = (int64_t)p.tiles_m * p.tiles_n;
    const int clusters = (int)(tiles < avail ? tiles : avail);
    if (ksub == 1) err = p.f8 ? launch_cluster_t<1, true>(ta, tb, p, clusters, st) : launch_cluster_t<1, false>(ta, tb, p, clusters, st);
    else if (ksub == 2) err = p.f8 ? launch_cluster_t<2, true>(ta, tb, p, clusters, st) : launch_cluster_t<2, false>(ta, tb, p, clusters, st);
    else return RG_ERR_UNSUPPORTED;
  } else if (plan.half_sm) {
    // one CTA per SM, each at half an SM's resources: the other half is where the next launch's CTAs set up
    const int grid = (int)(total < sms ? total : sms);
    if (ksub == 1) err = launch_one_half<1>(ta, tb, p, grid, st);
    else if (ksub == 2) err = launch_one_half<2>(ta, tb, p, grid, st);
    else return RG_ERR_UNSUPPORTED;
  } else if (ticket) {
    if ((size_t)p.tiles_m * (size_t)p.tiles_n > TICKET_TILES_MAX) return RG_ERR_UNSUPPORTED;   // more tiles than tickets
    const int grid = (int)(total < sms ? total : sms);
    p.ticket_all = total <= sms ? 1 : 0;                     // one round: every part of a tile has a resident CTA
    if (ksub == 1) err = p.f8 ? launch_ticket_t<1, true>(ta, tb, p, grid, st) : launch_ticket_t<1, false>(ta, tb, p, grid, st);
    else if (ksub == 2) err = p.f8 ? launch_ticket_t<2, true>(ta, tb, p, grid, st) : launch_ticket_t<2, false>(ta, tb, p, grid, st);
    else return RG_ERR_UNSUPPORTED;
  } else if (plan.inner_span) {
    if (ksub != 1) return RG_ERR_UNSUPPORTED;
    const int room = sms - plan.reserve_sms;                 // SMs left free for the merge's CTAs (see GemmPlan::reserve_sms)
    const int grid = (int)(total < room ? total : room);
    if (plan.BN <= 128) err = p.f8 ? launch_grouped_t<true, 2>(ta, tb, p, grid, st) : launch_grouped_t<false, 2>(ta, tb, p, grid, st);
    else err = p.f8 ? launch_grouped_t<true, 4>(ta, tb, p, grid, st) : launch_grouped_t<false, 4>(ta, tb, p, grid, st);
  } else {
    const int room = sms - plan.reserve_sms;                 // SMs left free for the merge's CTAs (see GemmPlan::reserve_sms)
    const int grid = (int)(total < room ? total : room);
    if (ksub == 1) err = launch_one<1>(ta, tb, p, grid, st);
    else if (ksub == 2) err = launch_one<2>(ta, tb, p, grid, st);
    else if (ksub == 4) err = launch_one<4>(ta, tb, p, grid, st);
    else return RG_ERR_UNSUPPORTED;
  }
  if (err != cudaSuccess) return RG_ERR_CUDA;

  if (split && !ticket) {
    FixupParams f;
    f.ws = ws; f.ldw = p.ldw; f.partial_dtype = plan.partial_dtype; f.merge_dtype = plan.merge_dtype;
    f.M = p.M; f.N = p.N; f.S = plan.n_parts; f.tree = plan.tree; f.launch_seq = p.launch_seq;
    f.C = C->ptr; f.ldc = C->ld; f.c_dtype = C->dtype; f.epi = e;
    const int64_t items = M * ((N + 3) / 4);
    cudaLaunchConfig_t cfg = {};
    const bool small = plan.merge_small != 0;                // the denser form of the merge that has SMs of its own (see splitk_fixup_small_kernel)
    cfg.gridDim = dim3((unsigned)((items + 255) / 256), 1, 1);
    cfg.blockDim = dim3(small ? 128 : 256, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t fe;
    if (small) {
      if (plan.partial_dtype == RG_F32) fe = cudaLaunchKernelEx(&cfg, splitk_fixup_small_kernel<false, false>, f);
      else if (plan.merge_dtype == RG_F32) fe = cudaLaunchKernelEx(&cfg, splitk_fixup_small_kernel<true, false>, f);
      else fe = cudaLaunchKernelEx(&cfg, splitk_fixup_small_kernel<true, true>, f);
    }
    else if (plan.partial_dtype == RG_F32) fe = cudaLaunchKernelEx(&cfg, splitk_fixup_kernel<false, false>, f);   // fp32 parts, fp32 sum
    else if (plan.merge_dtype == RG_F32) fe = cudaLaunchKernelEx(&cfg, splitk_fixup_kernel<true, false>, f);
    else fe = cudaLaunchKernelEx(&cfg, splitk_fixup_kernel<true, true>, f);
    if (fe != cudaSuccess) return RG_ERR_CUDA;
  }
  return RG_OK;
}

}  // namespace rg
