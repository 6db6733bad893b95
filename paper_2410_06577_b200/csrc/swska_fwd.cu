// Sliding-window shared-key attention (SW-SKA, the attention half of the Rodimus+ block;
// Sec. "Shared-Key Attention for Lossless Head Compression"): softmax attention in which all
// heads share ONE key per token, queries and values are per head, and token t attends to the
// tokens i with t - W < i <= t:
//
//   s_ti = scale <q^h_t, k_i>     p_ti = softmax_i(s_ti)     o^h_t = sum_i p_ti v^h_i
//
// bf16 kernel: one CTA of 4 warps per (batch, head, 64 queries), 16 query rows per warp, key/value
// tiles of 64 tokens streamed through a two-deep cp.async ring, scores and outputs on the tensor
// cores (mma.sync m16n8k16, bf16 in, fp32 accumulate), softmax in the log2 domain with a running
// maximum and sum per row (nothing of size T x W is ever stored).  Only the key tiles that touch
// the window are visited: cost per query is O(W), the key tile is shared by the 16 heads' CTAs
// through L2.  Shared-memory tiles are rows of 256 bytes whose 16-byte pieces are XOR-swizzled
// with the row number, so the 8x8 matrix loads hit 32 banks.
// fp32 kernel (validation): one warp per query row, accurate expf, same running softmax.
#include "ddts_common.cuh"

namespace ddts {
namespace {

constexpr int kD = 128;            // head size the kernels are built for (the paper's: 128)
constexpr int kBM = 64, kBN = 64;  // queries per CTA, keys per tile
constexpr int kThreads = 128;
constexpr float kLog2e = 1.4426950408889634f;

struct SwArgs {
  const void *q, *k, *v;
  void* o;
  int B, H, T, window;
  float scale;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
// element offset of (row, 16-byte piece) inside a swizzled [rows][128] bf16 tile
__device__ __forceinline__ int swz(int row, int piece) { return row * kD + ((piece ^ (row & 7)) << 3); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
  const int n = valid ? 16 : 0;   // 0 bytes read: the 16 bytes are filled with zeros
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(n) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}

// rows [row0, row0 + 64) of a [T][128] bf16 matrix into a swizzled tile; rows outside [0, T) as zeros
__device__ __forceinline__ void load_tile(__nv_bfloat16* tile, const __nv_bfloat16* base, int row0, int T,
                                          int tid) {
#pragma unroll
  for (int i = 0; i < (kBN * kD / 8) / kThreads; ++i) {
    const int idx = tid + i * kThreads, r = idx >> 4, piece = idx & 15;
    const int row = row0 + r;
    const bool ok = row >= 0 && row < T;
    const __nv_bfloat16* src = base + (long long)(ok ? row : 0) * kD + piece * 8;
    cp_async16(smem_u32(tile + swz(r, piece)), src, ok);
  }
}

__global__ void __launch_bounds__(kThreads, 2) swska_fwd_bf16_kernel(const SwArgs a) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  __nv_bfloat16* sQ = reinterpret_cast<__nv_bfloat16*>(smem_raw);      // [64][128], later the output tile
  __nv_bfloat16* sK = sQ + kBM * kD;                                    // [2][64][128]
  __nv_bfloat16* sV = sK + 2 * kBN * kD;                                // [2][64][128]

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int m0 = blockIdx.x * kBM, h = blockIdx.y, b = blockIdx.z;
  const int T = a.T, W = a.window;
  const __nv_bfloat16* q = (const __nv_bfloat16*)a.q + ((long long)b * a.H + h) * T * kD;
  const __nv_bfloat16* k = (const __nv_bfloat16*)a.k + (long long)b * T * kD;           // one key per token
  const __nv_bfloat16* v = (const __nv_bfloat16*)a.v + ((long long)b * a.H + h) * T * kD;
  __nv_bfloat16* o = (__nv_bfloat16*)a.o + ((long long)b * a.H + h) * T * kD;

  // key tiles that intersect the windows of rows m0 .. m0+63
  const int first_key = max(0, m0 - W + 1);
  const int nt_lo = first_key / kBN, nt_hi = min(m0 + kBM - 1, T - 1) / kBN;

  load_tile(sQ, q, m0, T, tid);
  load_tile(sK, k, nt_lo * kBN, T, tid);
  load_tile(sV, v, nt_lo * kBN, T, tid);
  cp_async_commit();
  cp_async_wait<0>();
  __syncthreads();

  uint32_t qf[8][4];   // this warp's 16 query rows as A fragments, one per 16 channels
#pragma unroll
  for (int kk = 0; kk < 8; ++kk) {
    const int row = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, piece = 2 * kk + (lane >> 4);
    ldsm_x4(qf[kk], smem_u32(sQ + swz(row, piece)));
  }

  float oacc[16][4];
#pragma unroll
  for (int j = 0; j < 16; ++j) oacc[j][0] = oacc[j][1] = oacc[j][2] = oacc[j][3] = 0.f;
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
  const float sc = a.scale * kLog2e;
  const int row_lo = m0 + warp * 16 + g;   // this thread's rows: row_lo and row_lo + 8

  for (int nt = nt_lo; nt <= nt_hi; ++nt) {
    const int buf = (nt - nt_lo) & 1;
    if (nt > nt_lo) {
      cp_async_wait<0>();
      __syncthreads();        // tile nt has landed; everyone is done with the other buffer
    }
    if (nt < nt_hi) {
      load_tile(sK + (buf ^ 1) * kBN * kD, k, (nt + 1) * kBN, T, tid);
      load_tile(sV + (buf ^ 1) * kBN * kD, v, (nt + 1) * kBN, T, tid);
      cp_async_commit();
    }
    const __nv_bfloat16* tK = sK + buf * kBN * kD;
    const __nv_bfloat16* tV = sV + buf * kBN * kD;
    // a warp whose 16 rows see nothing of this tile skips it (tiles before its window, after its rows)
    const int n0 = nt * kBN;
    const int wrow0 = m0 + warp * 16;
    const bool touches = n0 <= wrow0 + 15 && n0 + kBN - 1 > wrow0 - W;
    if (touches) {
      float s[8][4];
#pragma unroll
      for (int j = 0; j < 8; ++j) s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f;
#pragma unroll
      for (int kk = 0; kk < 8; ++kk) {
#pragma unroll
        for (int j = 0; j < 8; j += 2) {
          uint32_t bk[4];
          const int row = 8 * j + (lane & 7) + ((lane >> 4) & 1) * 8, piece = 2 * kk + ((lane >> 3) & 1);
          ldsm_x4(bk, smem_u32(tK + swz(row, piece)));
          mma_bf16(s[j], qf[kk], bk[0], bk[1]);
          mma_bf16(s[j + 1], qf[kk], bk[2], bk[3]);
        }
      }
      // scale into the log2 domain; where the tile is not wholly inside the window of all 16
      // rows, mask what lies outside (row - W, row]
      float mx[2] = {-INFINITY, -INFINITY};
      const bool inside = n0 + kBN - 1 <= wrow0 && n0 > wrow0 + 15 - W;
      if (inside) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            s[j][e] *= sc;
            mx[e >> 1] = fmaxf(mx[e >> 1], s[j][e]);
          }
        }
      } else {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int key = n0 + 8 * j + 2 * t + (e & 1), row = row_lo + (e >> 1) * 8;
            const bool in = key <= row && key > row - W;
            const float x = in ? s[j][e] * sc : -INFINITY;
            s[j][e] = x;
            mx[e >> 1] = fmaxf(mx[e >> 1], x);
          }
        }
      }
      float alpha[2], m_use[2];
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
        mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
        const float m_new = fmaxf(m_run[r], mx[r]);
        m_use[r] = m_new == -INFINITY ? 0.f : m_new;     // a row that has seen no key yet
        alpha[r] = exp2f(m_run[r] - m_use[r]);
        m_run[r] = m_new;
      }
      float psum[2] = {0.f, 0.f};
#pragma unroll
      for (int j = 0; j < 8; ++j) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float p = exp2f(s[j][e] - m_use[e >> 1]);
          s[j][e] = p;
          psum[e >> 1] += p;
        }
      }
      l_run[0] = l_run[0] * alpha[0] + psum[0];
      l_run[1] = l_run[1] * alpha[1] + psum[1];
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        oacc[j][0] *= alpha[0]; oacc[j][1] *= alpha[0];
        oacc[j][2] *= alpha[1]; oacc[j][3] *= alpha[1];
      }
      // o += P V: the score fragments of two key groups of 8 are one A fragment of 16 keys
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) {
        const uint32_t pf[4] = {pack_bf16(s[2 * kk][0], s[2 * kk][1]), pack_bf16(s[2 * kk][2], s[2 * kk][3]),
                                pack_bf16(s[2 * kk + 1][0], s[2 * kk + 1][1]),
                                pack_bf16(s[2 * kk + 1][2], s[2 * kk + 1][3])};
#pragma unroll
        for (int jd = 0; jd < 16; jd += 2) {
          uint32_t bv[4];
          const int row = 16 * kk + (lane & 7) + ((lane >> 3) & 1) * 8, piece = jd + (lane >> 4);
          ldsm_x4_t(bv, smem_u32(tV + swz(row, piece)));
          mma_bf16(oacc[jd], pf, bv[0], bv[1]);
          mma_bf16(oacc[jd + 1], pf, bv[2], bv[3]);
        }
      }
    }
  }

  // normalise, stage the 64 x 128 output tile in shared memory (the query tile's space: the
  // query fragments are in registers), store whole rows
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 1);
    l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 2);
    l_run[r] = l_run[r] > 0.f ? 1.f / l_run[r] : 0.f;
  }
  __syncthreads();   // (all warps past their last use of sQ: it was read only before the loop)
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    const int r0 = warp * 16 + g;
    *reinterpret_cast<uint32_t*>(sQ + swz(r0, j) + 2 * t) = pack_bf16(oacc[j][0] * l_run[0], oacc[j][1] * l_run[0]);
    *reinterpret_cast<uint32_t*>(sQ + swz(r0 + 8, j) + 2 * t) = pack_bf16(oacc[j][2] * l_run[1], oacc[j][3] * l_run[1]);
  }
  __syncthreads();
#pragma unroll
  for (int i = 0; i < (kBM * kD / 8) / kThreads; ++i) {
    const int idx = tid + i * kThreads, r = idx >> 4, piece = idx & 15;
    if (m0 + r < T)
      *reinterpret_cast<uint4*>(o + (long long)(m0 + r) * kD + piece * 8) =
          *reinterpret_cast<const uint4*>(sQ + swz(r, piece));
  }
}

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

std::atomic<unsigned long long> g_sw_smem_done{0};

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
  if (p.dtype == RODIMUS_BF16) {
    int dev = 0, sms = 0;
    cudaError_t e = current_device(&dev, &sms);
    if (e != cudaSuccess) return e;
    constexpr int smem = (kBM + 4 * kBN) * kD * 2;   // 80 KiB
    e = opt_in_shared_memory(swska_fwd_bf16_kernel, smem, dev, g_sw_smem_done);
    if (e != cudaSuccess) return e;
    const dim3 grid((p.T + kBM - 1) / kBM, p.H, p.B);
    swska_fwd_bf16_kernel<<<grid, kThreads, smem, st>>>(a);
  } else {
    const long long rows = (long long)p.B * p.H * p.T;
    swska_fwd_f32_kernel<<<(unsigned)((rows + 3) / 4), 128, 0, st>>>(a);
  }
  *n_launches = 1;
  return cudaGetLastError();
}

}  // namespace ddts
