// mdn_chunk_fwd_static_scratch: the forward for callers that must not allocate device memory.
//
// Some users of this library cannot call cudaMalloc at the point where they need the forward:
// an inference server that handed every byte of device memory to its own arena at start-up, a
// plugin whose host application forbids allocator calls, or a latency-critical loop that cannot
// afford the device-wide synchronisation an allocation (and the matching free) implies.
// mdn_chunk_fwd asks such callers for a workspace they have nowhere to take from.  This variant
// keeps the scratch (chunk map, coefficient vectors, T and W matrices, status word) in a
// fixed-size array that is part of the library image itself, so nothing is allocated at any time.
//
// The price: the array has a fixed, modest size (problems that need more are refused), every GPU
// that loads the library carries it until the process exits, and all calls share it - two calls
// whose kernels overlap on the GPU (different streams, or different host threads) race on it.
#include <cuda_runtime.h>

#include <mutex>

#include "mdn.h"

namespace {

// The scratch itself.  In host code this name is only a stand-in for the symbol: its device
// address must be asked for with cudaGetSymbolAddress (once per device, below).
static __device__ __align__(256) unsigned char g_static_scratch[MDN_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
void* g_scratch_addr[kMaxDevices] = {};
bool g_scratch_ready[kMaxDevices] = {};

// Device address of the scratch array on the current device; looked up on the first call there.
mdn_status scratch_address(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MDN_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_scratch_ready[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return MDN_ERR_CUDA;
    g_scratch_addr[dev] = p;
    g_scratch_ready[dev] = true;
  }
  *out = g_scratch_addr[dev];
  return MDN_OK;
}

}  // namespace

extern "C" mdn_status mdn_chunk_fwd_static_scratch(const mdn_params* p, const void* q, const void* k, const void* v,
                                                   const float* beta, const float* log_alpha, const float* log_mu,
                                                   const float* eta, const float* initial_S, const float* initial_M,
                                                   const int32_t* cu_seqlens, void* o, float* final_S, float* final_M,
                                                   void* cuda_stream) {
  // Parameters the workspace entry point would refuse get the same status here; only a valid problem
  // that needs more scratch than the array holds is answered with MDN_ERR_STATIC_SCRATCH.
  mdn_ws_layout lay;
  const mdn_status ps = mdn_workspace_layout(p, &lay);
  if (ps != MDN_OK) return ps;
  if (p->num_seqs > 0 ? cu_seqlens == nullptr : cu_seqlens != nullptr) return MDN_ERR_INVALID_ARG;
  if (lay.total_bytes > (uint64_t)MDN_STATIC_SCRATCH_BYTES) return MDN_ERR_STATIC_SCRATCH;
  void* scratch = nullptr;
  const mdn_status st = scratch_address(&scratch);
  if (st != MDN_OK) return st;
  // The array keeps whatever the previous call left in it.  The only part that must start at zero
  // is the status word, which the forward clears on the stream before its first kernel; the chunk
  // map, coefficients and matrices are fully rewritten for every chunk this call touches.
  return mdn_chunk_fwd(p, q, k, v, beta, log_alpha, log_mu, eta, initial_S, initial_M, cu_seqlens, o, final_S,
                       final_M, scratch, (size_t)MDN_STATIC_SCRATCH_BYTES, cuda_stream);
}
