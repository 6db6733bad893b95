// Diagnostic: throughput of the special-function unit (the ex2 / lg2 / rcp approximations the
// gate math of the prefill kernels is made of).  The benchmark times this launch with CUDA
// events to put a measured "special-function bound" beside the HBM and tensor bounds of the
// roofline; nothing on the DDTS path calls it.
#include "ddts_common.cuh"

namespace {

constexpr int kProbeThreads = 256;
constexpr int kProbeChains = 8;   // independent dependency chains per thread

__global__ void __launch_bounds__(kProbeThreads)
ddts_sfu_probe_kernel(int iters, float* __restrict__ sink) {
  float v[kProbeChains];
#pragma unroll
  for (int c = 0; c < kProbeChains; ++c) v[c] = -1e-3f * (float)(threadIdx.x + 32 * c + 1);
  for (int i = 0; i < iters; ++i) {
#pragma unroll
    for (int c = 0; c < kProbeChains; ++c) {
      float y;
      asm volatile("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(v[c]));
      v[c] = -y;                       // stays in (-1, 0): the chain never saturates
    }
  }
  float s = 0.f;
#pragma unroll
  for (int c = 0; c < kProbeChains; ++c) s += v[c];
  if (s == 12345.678f) sink[0] = s;    // keeps the chains alive; practically never taken
}

}  // namespace

extern "C" int rodimus_ddts_sfu_probe(int iters, float* sink, void* stream, long long* ops) {
  if (!sink || !ops) return RODIMUS_ERR_NULL;
  if (iters <= 0 || iters > (1 << 24)) return RODIMUS_ERR_SHAPE;
  int dev = 0, sms = 0;
  if (ddts::current_device(&dev, &sms) != cudaSuccess) return RODIMUS_ERR_CUDA;
  const int ctas = sms * 8;            // 2048 threads per SM: every scheduler has work to hide latency
  ddts_sfu_probe_kernel<<<ctas, kProbeThreads, 0, reinterpret_cast<cudaStream_t>(stream)>>>(iters, sink);
  if (cudaGetLastError() != cudaSuccess) return RODIMUS_ERR_CUDA;
  *ops = (long long)ctas * kProbeThreads * kProbeChains * iters;
  return RODIMUS_OK;
}
