// Internal declarations shared by the translation units of the DDTS library (not part of the ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "rodimus_ddts.h"

namespace ddts {

// Device-visible words at the start of the caller's workspace.
struct WorkspaceHeader {
  int32_t status;        // rodimus_status recorded by kernels (0 = ok); only ever raised
  int32_t pad[63];
};
static_assert(sizeof(WorkspaceHeader) == 256, "workspace header is 256 bytes");

constexpr int kMaxSortedSeqs = 4096;  // varlen: sequences beyond this keep their given order

// The current device and its SM count (the count is asked for once per device).
cudaError_t current_device(int* dev, int* sms);

// Opt-in to more than 48 KiB of dynamic shared memory, once per kernel and device: `done` is a
// per-kernel bit mask over device ordinals (devices beyond 63 simply ask every time).
template <typename Kernel>
inline cudaError_t opt_in_shared_memory(Kernel kernel, int bytes, int dev, std::atomic<unsigned long long>& done) {
  const unsigned long long bit = dev >= 0 && dev < 64 ? 1ull << dev : 0ull;
  if (bit && (done.load(std::memory_order_acquire) & bit)) return cudaSuccess;
  const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess && bit) done.fetch_or(bit, std::memory_order_release);
  return e;
}

// Limit, in clock cycles, that the tensor-core prefill kernels give each of their main-loop
// waits (see rodimus_ddts_test_set_wait_limit).
long long main_loop_wait_cycles();

// Launchers: all arguments validated by the caller; they return a cudaError_t.
cudaError_t launch_step(const rodimus_ddts_step_params& p, int* n_launches);
cudaError_t launch_plan(const rodimus_ddts_fwd_params& p, int* n_launches);
cudaError_t launch_fwd_simt(const rodimus_ddts_fwd_params& p, int* n_launches);
cudaError_t launch_fwd_tc(const rodimus_ddts_fwd_params& p, int* n_launches);
cudaError_t launch_fwd_pair(const rodimus_ddts_fwd_params& p, int* n_launches);
cudaError_t launch_bwd(const rodimus_ddts_bwd_params& p, size_t scratch_offset, int* n_launches);
bool bwd_supported(const rodimus_ddts_bwd_params& p);
size_t bwd_scratch_bytes(const rodimus_ddts_bwd_params& p);   // beyond the header and the order
cudaError_t launch_swska(const rodimus_swska_fwd_params& p, int* n_launches);
cudaError_t launch_swska_tc(const rodimus_swska_fwd_params& p, int* n_launches);   // bf16, tcgen05
bool swska_supported(const rodimus_swska_fwd_params& p);
bool fwd_tc_supported(const rodimus_ddts_fwd_params& p);
bool fwd_pair_supported(const rodimus_ddts_fwd_params& p);
// Workspace a dense call needs if its sequences are to be split along time (0: no split).
size_t fwd_pair_split_workspace_bytes(const rodimus_ddts_fwd_params& p);

// ---------------------------------------------------------------------------------------------
// Element access for the two token dtypes.
// ---------------------------------------------------------------------------------------------
template <typename T>
__device__ __forceinline__ float to_f32(T v);
template <>
__device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <>
__device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename T>
__device__ __forceinline__ T from_f32(float v);
template <>
__device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <>
__device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// ---------------------------------------------------------------------------------------------
// Gate math in full fp32 precision (Eq. "alpha_def"): natural-log decay and natural-log input
// weight for one key channel.  Used where accuracy matters more than issue slots (decode, fp32
// prefill).  log_alpha = -softplus(x) * sigmoid(y) <= 0;  log_ahat = sigmoid(y) * log(g) for
// the paper's form, sigmoid(y) * log(1 - exp(-g)) = -sigmoid(y) * softplus(-x) for the other.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float softplus_f32(float x) {
  return x > 0.f ? x + log1pf(expf(-x)) : log1pf(expf(x));
}

__device__ __forceinline__ void gate_logs_f32(float x, float y, int ingate, float& log_alpha,
                                              float& log_ahat) {
  const float g = softplus_f32(x);
  const float tau = y >= 0.f ? 1.f / (1.f + expf(-y)) : expf(y) / (1.f + expf(y));
  log_alpha = -g * tau;
  if (ingate == RODIMUS_INGATE_POW_G) {
    // g > 0 for every finite x >= -87; log(g) -> x as x -> -inf
    log_ahat = tau * logf(g);
  } else {
    log_ahat = -tau * softplus_f32(-x);
  }
}

}  // namespace ddts
