// rodimus_ddts_fwd_noalloc: chunked prefill for callers that may not allocate device memory.
//
// The ordinary entry point asks the caller for a small device workspace (a status word, and for
// packed sequences the order in which CTAs take them).  Some callers have no way to provide
// one: a plug-in running inside a host application that handed out all device memory at start-up
// and forbids further allocation, a latency-critical serving loop in which cudaMalloc's
// device-wide synchronisation is unacceptable, or code that is only given input and output
// buffers by its framework.  For them the workspace lives in a fixed array in the library's own
// device image, which every GPU that loads the library carries until the process exits.
#include <mutex>

#include "ddts_common.cuh"

namespace {

constexpr int kMaxSeqs = RODIMUS_NOALLOC_MAX_SEQS;
constexpr size_t kScratchBytes = sizeof(ddts::WorkspaceHeader) + (size_t)kMaxSeqs * sizeof(int32_t);

// File-scope scratch.  In HOST code this name is only a handle for the runtime, never a device
// address: the address each device gave it is looked up below and that is what kernels receive.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_addr[kMaxDevices] = {};   // per device, filled by that device's first call

// Address of the scratch array on the CURRENT device (looked up once per device).
cudaError_t scratch_address(void** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_addr[dev]) {
    void* ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
    if (e != cudaSuccess) return e;
    if (!ptr) return cudaErrorInvalidSymbol;
    g_scratch_addr[dev] = ptr;
  }
  *out = g_scratch_addr[dev];
  return cudaSuccess;
}

}  // namespace

extern "C" int rodimus_ddts_fwd_noalloc(const rodimus_ddts_fwd_params* p, const void** status_handle) {
  if (status_handle) *status_handle = nullptr;
  if (!p) return RODIMUS_ERR_NULL;
  if (p->struct_size != (int32_t)sizeof(rodimus_ddts_fwd_params)) return RODIMUS_ERR_DTYPE;
  // the only size the fixed array limits: the per-sequence order of a packed call
  if (p->cu_seqlens && p->N > kMaxSeqs) return RODIMUS_ERR_WORKSPACE;
  void* scratch = nullptr;
  if (scratch_address(&scratch) != cudaSuccess) return RODIMUS_ERR_CUDA;
  rodimus_ddts_fwd_params q = *p;        // same request, workspace replaced by the built-in one
  q.workspace = scratch;
  q.workspace_bytes = kScratchBytes;
  // Nothing in the array has to be zero on entry: the planning kernel (packed calls) or the
  // prefill kernel's first CTA (dense calls) rewrites the status word at the start of each call,
  // and the order list is rewritten in full before it is read.
  const int rc = rodimus_ddts_fwd(&q);
  if (rc == RODIMUS_OK && status_handle) *status_handle = scratch;
  return rc;
}
