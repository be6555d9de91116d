// rg_gemm_noalloc: split-K GEMM whose fp32 workspace lives inside the library image.
//
// Some callers may not allocate device memory at the moment they need a split-K GEMM: code that
// runs inside a serving loop whose memory pool is frozen after start-up, plugins whose host
// framework owns the allocator and hands out no scratch, and latency-critical decode paths
// where a cudaMalloc (which synchronises the device) is not acceptable.  For them the parts of
// the contracted axis are written to a fixed array that is part of this module, so the call
// needs nothing beyond its inputs and its output.
//
// The array is a file-scope device symbol.  In host code its name is only a stand-in for the
// symbol, not a device address, so the address is resolved once per device with
// cudaGetSymbolAddress (with that device current) and that pointer is what the kernels get.
#include <mutex>

#include "rg_internal.h"

namespace {

// Every GPU that loads the library holds this array until the process exits.
static __device__ __align__(256) unsigned char g_noalloc_ws[RG_NOALLOC_WS_BYTES];

constexpr int MAX_DEVICES = 64;
void* g_ws_addr[MAX_DEVICES] = {};
std::mutex g_ws_mutex;

// Resolve the array's address on the current device (first call per device only).
rg_status_t noalloc_ws_for_current_device(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return RG_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_ws_mutex);
  if (!g_ws_addr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_noalloc_ws) != cudaSuccess || !p) return RG_ERR_CUDA;
    g_ws_addr[dev] = p;
  }
  *out = g_ws_addr[dev];
  return RG_OK;
}

}  // namespace

extern "C" rg_status_t rg_gemm_noalloc(const rg_desc_t* d, const rg_tensor_t* A, const rg_tensor_t* B,
                                       const rg_tensor_t* C, const rg_epilogue_t* epi, void* cuda_stream) {
  if (!d || !A || !B || !C) return RG_ERR_NULL;
  if (d->n_cuts > RG_MAX_CUTS) return RG_ERR_INVALID_DESC;
  if (d->n_cuts == 0) return rg_gemm(d, A, B, C, epi, nullptr, 0, cuda_stream);   // no parts, no scratch
  // split_merge = 3 keeps tickets in the workspace that must be zero between calls; the shared array is also
  // written by calls that keep parts there, so that promise cannot be made for it
  if (d->split_merge == 3) return RG_ERR_UNSUPPORTED;
  // the size check comes first: a request beyond the fixed array is refused, never truncated
  const size_t need = rg_gemm_workspace_bytes(d, A->rows, B->rows);
  if (need > (size_t)RG_NOALLOC_WS_BYTES) return RG_ERR_WORKSPACE;
  void* ws = nullptr;
  rg_status_t s = noalloc_ws_for_current_device(&ws);
  if (s != RG_OK) return s;
  // Nothing in the array has to start at zero: the GEMM kernel writes every partial the merge
  // kernel reads for rows < M and columns < N, and the merge ignores the padding columns.
  return rg_gemm(d, A, B, C, epi, ws, RG_NOALLOC_WS_BYTES, cuda_stream);
}
