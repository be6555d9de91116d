// Internal host-side declarations shared by the translation units of the library.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "../../include/rg.h"

struct CUtensorMap_st;

namespace rg {

// Function attributes are per device: one bit per device ordinal and kernel instantiation.
struct DeviceOnce {
  std::atomic<uint64_t> mask{0};
  bool has(int dev) const { return dev >= 0 && dev < 64 && ((mask.load(std::memory_order_acquire) >> dev) & 1u); }
  void set(int dev) { if (dev >= 0 && dev < 64) mask.fetch_or(uint64_t(1) << dev, std::memory_order_release); }
};

struct DeviceInfo { int dev, sms; };
// The current device and its SM count (looked up once per device).
inline DeviceInfo current_device() {
  static std::atomic<int> sms_of[64];
  DeviceInfo d{0, 148};
  if (cudaGetDevice(&d.dev) != cudaSuccess) return d;
  if (d.dev >= 0 && d.dev < 64 && sms_of[d.dev].load(std::memory_order_relaxed) > 0) { d.sms = sms_of[d.dev].load(std::memory_order_relaxed); return d; }
  int sms = 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, d.dev) == cudaSuccess && sms > 0) {
    d.sms = sms;
    if (d.dev >= 0 && d.dev < 64) sms_of[d.dev].store(sms, std::memory_order_relaxed);
  }
  return d;
}

// A validated launch plan: speed knobs resolved, parts laid out.
struct GemmPlan {
  int BN, BK, stages, raster, group_m, cta_group;
  int b_static;             // caller's promise: nothing in flight on the stream writes B (its first boxes may be fetched early)
  int reserve_sms;          // SMs the GEMM leaves free for the CTAs of its split-K merge (calls that do not depend on each other, b_static = 2)
  int merge_small;          // that merge runs as 128-thread CTAs of two units per thread (four to an SM) instead of the general kernel
  int half_sm;              // the one-CTA kernel in its half-SM form: two CTAs share an SM (weight-streaming shapes)
  int ticket_merge;         // split-K parts through the workspace, merged inside the GEMM kernel by the CTA that stores a tile's last part
  int cluster_merge;        // split-K parts merged inside the GEMM kernel by a thread-block cluster (no workspace, one launch)
  int n_parts, tree;
  int partial_dtype, merge_dtype;
  int inner_span;
  int32_t part_begin[RG_MAX_CUTS + 1];
  int32_t part_end[RG_MAX_CUTS + 1];
};

int max_stages_for(int bn, int bk, int cta_group, int64_t M, bool cluster_merge = false, bool half_sm = false);
int max_active_clusters(int csize, int bk, bool f8);
size_t ticket_bytes();
rg_status_t launch_gemm(const GemmPlan& plan, const rg_tensor_t* A, const rg_tensor_t* B, const rg_tensor_t* C,
                        const rg_epilogue_t* epi, void* ws, cudaStream_t st);
rg_status_t launch_gemv(const rg_desc_t* d, const rg_tensor_t* A, const rg_tensor_t* B, const rg_tensor_t* C,
                        const rg_epilogue_t* epi, cudaStream_t st);
rg_status_t launch_reduce_rows(int op, int tree, int fma, const rg_tensor_t* x, const rg_tensor_t* out,
                               const rg_reduce_args_t* args, int threads_hint, int unroll_hint, cudaStream_t st);
size_t reduce_cols_workspace_bytes(int64_t R, int64_t C);
rg_status_t launch_reduce_cols(int op, int tree, int fma, const rg_tensor_t* x, const rg_tensor_t* y, const rg_tensor_t* out,
                               void* ws, cudaStream_t st);
bool make_operand_tmap(CUtensorMap_st* map, const void* ptr, int dtype, int64_t rows, int64_t cols, int64_t ld, int box_rows);
rg_status_t launch_attention_fixed(int block_n, int exp_base, int causal, float scale, int heads, const rg_tensor_t* Q, const rg_tensor_t* K,
                                   const rg_tensor_t* Vt, const rg_tensor_t* O, cudaStream_t st);
rg_status_t read_and_clear_attn_status(uint32_t* code);
rg_status_t read_and_clear_status(uint32_t* code);
rg_status_t launch_wait_selftest(uint64_t limit_ns, uint32_t code, unsigned int* left_early, cudaStream_t st);
// y[i] = FORM(x[i]) by the device functions the kernels use (forms 0-2 and 6; the attention kernel's forms 3-5)
rg_status_t launch_exp_selftest(int form, const float* x, float* y, int64_t n, cudaStream_t st);
rg_status_t launch_exp_selftest_attention(int form, const float* x, float* y, int64_t n, cudaStream_t st);
rg_status_t launch_silu_selftest(const float* x, float* y, int64_t n, cudaStream_t st);   // form 7: the epilogue's SiLU on segments of 32
rg_status_t read_and_clear_reduce_status(uint32_t* code);

}  // namespace rg
