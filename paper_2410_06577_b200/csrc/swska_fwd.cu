// Sliding-window shared-key attention (SW-SKA, the attention half of the Rodimus+ block;
// Sec. "Shared-Key Attention for Lossless Head Compression"): softmax attention in which all
// heads share ONE key per token, queries and values are per head, and token t attends to the
// tokens i with t - W < i <= t:
//
//   s_ti = scale <q^h_t, k_i>     p_ti = softmax_i(s_ti)     o^h_t = sum_i p_ti v^h_i
//
// This file: the launcher and the fp32 validation kernel (one warp per query row, accurate expf,
// running maximum and sum).  bf16 tokens run the tcgen05 kernel of swska_fwd_tc.cu.
#include "ddts_common.cuh"

namespace ddts {
namespace {

constexpr int kD = 128;            // head size the kernels are built for (the paper's: 128)

struct SwArgs {
  const void *q, *k, *v;
  void* o;
  int B, H, T, window;
  float scale;
};

// fp32 validation kernel: one warp per query row, lane l owns channels 4l .. 4l+3.
__global__ void __launch_bounds__(128) swska_fwd_f32_kernel(const SwArgs a) {
  const int lane = threadIdx.x & 31;
  const long long row_id = (long long)blockIdx.x * 4 + (threadIdx.x >> 5);
  const long long rows = (long long)a.B * a.H * a.T;
  if (row_id >= rows) return;
  const int tq = (int)(row_id % a.T);
  const long long bh = row_id / a.T;
  const int b = (int)(bh / a.H);
  const float* q = (const float*)a.q + row_id * kD + lane * 4;
  const float* k = (const float*)a.k + (long long)b * a.T * kD + lane * 4;
  const float* v = (const float*)a.v + bh * a.T * kD + lane * 4;
  const float4 qv = *reinterpret_cast<const float4*>(q);
  float m = -INFINITY, l = 0.f;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int i = max(0, tq - a.window + 1); i <= tq; ++i) {
    const float4 kv = *reinterpret_cast<const float4*>(k + (long long)i * kD);
    float s = qv.x * kv.x + qv.y * kv.y + qv.z * kv.z + qv.w * kv.w;
#pragma unroll
    for (int off = 16; off; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
    s *= a.scale;
    const float m_new = fmaxf(m, s);
    const float al = expf(m - m_new), p = expf(s - m_new);
    const float4 vv = *reinterpret_cast<const float4*>(v + (long long)i * kD);
    l = l * al + p;
    acc.x = acc.x * al + p * vv.x; acc.y = acc.y * al + p * vv.y;
    acc.z = acc.z * al + p * vv.z; acc.w = acc.w * al + p * vv.w;
    m = m_new;
  }
  const float inv = 1.f / l;
  *reinterpret_cast<float4*>((float*)a.o + row_id * kD + lane * 4) =
      make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
}

}  // namespace

bool swska_supported(const rodimus_swska_fwd_params& p) { return p.d == kD; }

cudaError_t launch_swska(const rodimus_swska_fwd_params& p, int* n_launches) {
  *n_launches = 0;
  if ((long long)p.B * p.H * p.T == 0) return cudaSuccess;
  SwArgs a;
  a.q = p.q; a.k = p.k; a.v = p.v; a.o = p.o;
  a.B = p.B; a.H = p.H; a.T = p.T; a.window = p.window; a.scale = p.scale;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(p.stream);
  if (p.dtype == RODIMUS_BF16) return launch_swska_tc(p, n_launches);
  const long long rows = (long long)p.B * p.H * p.T;
  swska_fwd_f32_kernel<<<(unsigned)((rows + 3) / 4), 128, 0, st>>>(a);
  *n_launches = 1;
  return cudaGetLastError();
}

}  // namespace ddts
