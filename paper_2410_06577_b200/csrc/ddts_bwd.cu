// Backward pass of the chunked prefill: gradients with respect to q, k, x, y, v and the initial
// state, given dL/do and dL/dS_T.  The paper trains the block through the chunkwise form
// (appendix "Chunkwise Parallel Representation of the Rodimus Block"); this is the adjoint of
// that form, chunk length 16, with the same notation:
//
//   b_r   = sum_{j<=r in chunk} log alpha_j                 (per key channel, b_C at the chunk end)
//   kt_i  = ahat_i . k_i        q'_r = scale . q_r
//   A_ri  = sum_d q'_rd kt_id exp(b_rd - b_id),  i <= r     (scores; difference formed BEFORE exp)
//   dA_ri = sum_j do_rj v_ij,                    i <= r
//   Qe_r  = q'_r . exp(b_r)     Ke_i = kt_i . exp(b_C - b_i)     D = exp(b_C)
//
//   forward sweep  (state S entering the chunk):
//     dq'_r = sum_{i<=r} dA_ri kt_i exp(b_r - b_i) + exp(b_r) . (S do_r)      S <- D . S + Ke^T V
//   reverse sweep  (G = dL/dS at the chunk end):
//     dkt_i = sum_{r>=i} dA_ri q'_r exp(b_r - b_i) + exp(b_C - b_i) . (G v_i)
//     dv_i  = sum_{r>=i} A_ri do_r + Ke_i G                                   G <- D . G + Qe^T dO
//   gates: with u_t = q_t . dq_t and w_t = kt_t . dkt_t (= dL/dlog ahat_t),
//     dL/dlog alpha_t = sum_{s>=t} (u_s - w_s) + sum_j dS_T[.,j] S_T[.,j]
//   (every pair (r,i) with i < t <= r appears once in the first sum and never in the second),
//   and dx, dy follow from Eq. "alpha_def" by the chain rule.
//
// One launch of 6 CTAs per (sequence, head): the forward sweep for each half of the key channels,
// the reverse sweep for each half of the key channels (dk), and the reverse sweep with the state
// transposed for each half of the value columns (dv).  Each CTA keeps its [64 x 256] (or
// [128 x 128]) slice of the state in REGISTERS as accumulator fragments of mma.sync.m16n8k8
// (tf32 inputs, fp32 accumulation); the same registers are the A operand of the contraction
// with dO or V (the k index of that instruction is a free permutation, applied to both
// operands).  The fp32 build splits every operand into two tf32 parts (three instructions per
// product), which keeps fp32 accuracy.  A second, small kernel forms the suffix sums and dx, dy.
#include "ddts_common.cuh"

namespace ddts {
namespace {

constexpr int kC = 16;            // chunk length
constexpr int DK = 128, DV = 256; // the widths this kernel is built for
constexpr int kThreads = 256;
constexpr int LDK = DK + 8;       // row strides = 8 mod 32 words: fragment loads hit 32 banks
constexpr int LDV = DV + 8;
constexpr int LDR = 17;

struct BwdArgs {
  const void *q, *k, *gx, *ty, *v, *dout;
  const float *s0, *dsT;
  void *dq, *dk, *dx, *dy, *dv;
  float* ds0;
  float *u, *w, *c;        // scratch: [rows, DK], [rows, DK], [n_seq * H, DK]
  float* seg_state;        // scratch: [n_seq * H * 6][64][256] state fragments handed from one time segment to the next
  int32_t* seg_flag;       // scratch: [n_seq * H * 6] number of segments of the sweep that have finished
  int nseg;                // time segments per sweep (1: a sweep is one CTA)
  long long limit;         // cycles a CTA waits for the segment before it
  const int32_t* cu;
  WorkspaceHeader* hdr;
  int H, T, n_seq;
  float scale;
  int ingate;
};

__device__ __forceinline__ int32_t ld_acquire_s32(const int32_t* p) {
  int32_t v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release_s32(int32_t* p, int32_t v) {
  asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

template <typename T>
__device__ __forceinline__ void load8(const T* p, float (&o)[8]);
template <>
__device__ __forceinline__ void load8<float>(const float* p, float (&o)[8]) {
  const float4 a = *reinterpret_cast<const float4*>(p), b = *reinterpret_cast<const float4*>(p + 4);
  o[0] = a.x; o[1] = a.y; o[2] = a.z; o[3] = a.w; o[4] = b.x; o[5] = b.y; o[6] = b.z; o[7] = b.w;
}
template <>
__device__ __forceinline__ void load8<__nv_bfloat16>(const __nv_bfloat16* p, float (&o)[8]) {
  const uint4 a = *reinterpret_cast<const uint4*>(p);
  const uint32_t w[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    o[2 * i] = __uint_as_float(w[i] << 16);
    o[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}
template <typename T>
__device__ __forceinline__ void store8(T* p, const float (&o)[8]);
template <>
__device__ __forceinline__ void store8<float>(float* p, const float (&o)[8]) {
  *reinterpret_cast<float4*>(p) = make_float4(o[0], o[1], o[2], o[3]);
  *reinterpret_cast<float4*>(p + 4) = make_float4(o[4], o[5], o[6], o[7]);
}
template <>
__device__ __forceinline__ void store8<__nv_bfloat16>(__nv_bfloat16* p, const float (&o)[8]) {
  uint32_t w[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(o[2 * i], o[2 * i + 1]);
    w[i] = *reinterpret_cast<const uint32_t*>(&h);
  }
  *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
}

__device__ __forceinline__ float tf32_round(float x) {
  uint32_t r;
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
  return __uint_as_float(r);
}

__device__ __forceinline__ void mma_tf32(float (&c)[4], const float (&a)[4], const float (&b)[2]) {
  asm volatile(
      "mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(__float_as_uint(a[0])), "r"(__float_as_uint(a[1])), "r"(__float_as_uint(a[2])),
        "r"(__float_as_uint(a[3])), "r"(__float_as_uint(b[0])), "r"(__float_as_uint(b[1])));
}

// c += a * b for one 16x8x8 tile.  EXACT (fp32 build): operands split as hi + lo (both tf32),
// the lo*lo term (2^-22 of the product) dropped.  Otherwise the operands go in as they are: what
// comes from shared memory is bf16 data or was rounded to tf32 when it was stored, and of the
// fp32 state fragments the instruction reads the tf32 part.
template <bool EXACT>
__device__ __forceinline__ void mma_tile(float (&c)[4], const float (&a)[4], const float (&b)[2]) {
  if (EXACT) {
    float ah[4], bh[2], al[4], bl[2];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      ah[i] = tf32_round(a[i]);
      al[i] = tf32_round(a[i] - ah[i]);
    }
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      bh[i] = tf32_round(b[i]);
      bl[i] = tf32_round(b[i] - bh[i]);
    }
    mma_tf32(c, al, bh);
    mma_tf32(c, ah, bl);
    mma_tf32(c, ah, bh);
  } else {
    mma_tf32(c, a, b);
  }
}

template <bool FAST>
__device__ __forceinline__ float exp_f(float x) { return FAST ? __expf(x) : expf(x); }

// log alpha and log ahat of one channel (Eq. "alpha_def").  FAST (bf16 build): hardware
// exponential / logarithm approximations (relative error about 2^-21, far inside the bf16 bar),
// with the two places where they would lose everything written out: log(1 + e) for small e, and
// log(softplus(x)) for very negative x, where softplus(x) = e^x (1 - e^x / 2 + ...).
template <bool FAST>
__device__ __forceinline__ void gate_logs(float x, float y, int ingate, float& la, float& lh) {
  if (!FAST) {
    gate_logs_f32(x, y, ingate, la, lh);
    return;
  }
  const float e = __expf(-fabsf(x));
  const float l1p = e < 0.0009765625f ? e * fmaf(-0.5f, e, 1.f) : __logf(1.f + e);
  const float g = fmaxf(x, 0.f) + l1p;
  const float tau = __fdividef(1.f, 1.f + __expf(-y));
  la = -g * tau;
  if (ingate == RODIMUS_INGATE_POW_G) {
    lh = tau * (x < -8.f ? fmaf(-0.5f, e, x) : __logf(g));
  } else {
    lh = -tau * (fmaxf(-x, 0.f) + l1p);
  }
}

template <typename T>
__device__ __forceinline__ void load4(const T* p, float (&o)[4]);
template <>
__device__ __forceinline__ void load4<float>(const float* p, float (&o)[4]) {
  const float4 a = *reinterpret_cast<const float4*>(p);
  o[0] = a.x; o[1] = a.y; o[2] = a.z; o[3] = a.w;
}
template <>
__device__ __forceinline__ void load4<__nv_bfloat16>(const __nv_bfloat16* p, float (&o)[4]) {
  const uint2 a = *reinterpret_cast<const uint2*>(p);
  o[0] = __uint_as_float(a.x << 16); o[1] = __uint_as_float(a.x & 0xffff0000u);
  o[2] = __uint_as_float(a.y << 16); o[3] = __uint_as_float(a.y & 0xffff0000u);
}

// MODE 0: forward sweep (dq, u, c); 1: reverse sweep, state [d][j] (dk, w, ds0);
// 2: reverse sweep, state [j][d] (dv).
// CTA index = ((segment * 6 + sweep slot) * items + item): all first segments, then all second ones ..
__device__ __forceinline__ int segment_of_this_cta(const BwdArgs& a) {
  return (int)(blockIdx.x / (gridDim.x / a.nseg));
}

template <typename T, int MODE>
__device__ void bwd_sweep(const BwdArgs& a, float* smem, const long long sh, const int half,
                          const long long row0, const int len, const int seg) {
  constexpr bool EXACT = sizeof(T) == 4, FAST = !EXACT;
  constexpr int NCH = MODE == 2 ? DK : DK / 2;      // key channels whose gates this CTA needs
  const int ch0 = MODE == 2 ? 0 : 64 * half;
  float* sQ = smem;                    // [kC][LDK] scale * q
  float* sKt = sQ + kC * LDK;          // ahat * k
  float* sLa = sKt + kC * LDK;         // log alpha
  float* sB = sLa + kC * LDK;          // b (inclusive cumulative log alpha)
  float* sQe = sB + kC * LDK;          // q' exp(b)
  float* sKe = sQe + kC * LDK;         // kt exp(b_C - b)      (MODE 1: ahat instead)
  float* sV = sKe + kC * LDK;          // [kC][LDV]
  float* sDO = sV + kC * LDV;          // [kC][LDV]
  float* sD = sDO + kC * LDV;          // [DK] exp(b_C)
  float* sP = sD + DK;                 // [kC][LDR] dA (MODE 0, 1) or A (MODE 2), masked
  float* sRedA = sP + kC * LDR;        // [8][kC][kC] partial dA of each warp
  float* sRed = sRedA + 8 * kC * kC;   // [8][16][LDR] partial contraction of each warp / dv tile

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const T* q = (const T*)a.q + row0 * DK;
  const T* k = (const T*)a.k + row0 * DK;
  const T* gx = (const T*)a.gx + row0 * DK;
  const T* ty = (const T*)a.ty + row0 * DK;
  const T* v = (const T*)a.v + row0 * DV;
  const T* dout = (const T*)a.dout + row0 * DV;
  const long long s_off = sh * (long long)DK * DV;

  // rows / columns of the state fragments this thread holds
  const int m0 = MODE == 2 ? 128 * half + 16 * warp : 64 * half + 16 * (warp >> 1);
  const int nbase = MODE == 2 ? 0 : 128 * (warp & 1);
  float st[16][4];
  // A sweep may be cut into time segments that run as CTAs of their own; a segment after the
  // first starts from the state the one before it left in the workspace, in the layout of s0.
  {
    const float* init = seg > 0 ? a.seg_state : (MODE == 0 ? a.s0 : a.dsT);
    const long long s_off = (seg > 0 ? sh * 3 + MODE : sh) * (long long)DK * DV;
#pragma unroll
    for (int n = 0; n < 16; ++n) {
      const int c0 = nbase + 8 * n + 2 * t;
      if (!init) {
        st[n][0] = st[n][1] = st[n][2] = st[n][3] = 0.f;
      } else if (MODE != 2) {
        const float2 lo = *reinterpret_cast<const float2*>(init + s_off + (long long)(m0 + g) * DV + c0);
        const float2 hi = *reinterpret_cast<const float2*>(init + s_off + (long long)(m0 + g + 8) * DV + c0);
        st[n][0] = lo.x; st[n][1] = lo.y; st[n][2] = hi.x; st[n][3] = hi.y;
      } else {   // transposed: fragment row = value column, fragment column = key channel
        st[n][0] = init[s_off + (long long)c0 * DV + m0 + g];
        st[n][1] = init[s_off + (long long)(c0 + 1) * DV + m0 + g];
        st[n][2] = init[s_off + (long long)c0 * DV + m0 + g + 8];
        st[n][3] = init[s_off + (long long)(c0 + 1) * DV + m0 + g + 8];
      }
    }
  }

  const int nchunks = (len + kC - 1) / kC;
  for (int ci = 0; ci < nchunks; ++ci) {
    const int t0 = (MODE == 0 ? ci : nchunks - 1 - ci) * kC;
    const int nr = min(kC, len - t0);
    // ---- (1) loads and gates: a thread per (row, 4 channels) of the channels this CTA needs
    // (its own half; all of them where the state is transposed); rows past the end read as zero.
    // All global loads of the chunk are issued before the first of them is used.
    {
      constexpr int kGroups = NCH / 4, kIter = kC * kGroups / kThreads;   // 1 or 2
      float fq[kIter][4], fk[kIter][4], fx[kIter][4], fy[kIter][4];
#pragma unroll
      for (int it = 0; it < kIter; ++it) {
        const int e = tid + it * kThreads, r = e / kGroups, d4 = ch0 + (e % kGroups) * 4;
        if (r < nr) {
          const long long i = (long long)(t0 + r) * DK + d4;
          load4<T>(q + i, fq[it]);
          load4<T>(k + i, fk[it]);
          load4<T>(gx + i, fx[it]);
          load4<T>(ty + i, fy[it]);
        }
      }
#pragma unroll
      for (int p = 0; p < 2; ++p) {
        const int e = tid + p * kThreads, rr = e >> 5, c8 = (e & 31) * 8;
        float fv[8], fd[8];
        if (rr < nr) {
          const long long i = (long long)(t0 + rr) * DV + c8;
          load8<T>(v + i, fv);
          load8<T>(dout + i, fd);
        } else {
#pragma unroll
          for (int x = 0; x < 8; ++x) fv[x] = fd[x] = 0.f;
        }
        store8<float>(sV + rr * LDV + c8, fv);
        store8<float>(sDO + rr * LDV + c8, fd);
      }
#pragma unroll
      for (int it = 0; it < kIter; ++it) {
        const int e = tid + it * kThreads, r = e / kGroups, d4 = ch0 + (e % kGroups) * 4;
        float fa[4], la[4];
        if (r < nr) {
#pragma unroll
          for (int x = 0; x < 4; ++x) {
            float lh;
            gate_logs<FAST>(fx[it][x], fy[it][x], a.ingate, la[x], lh);
            fa[x] = exp_f<FAST>(lh);
            fk[it][x] *= fa[x];
            fq[it][x] *= a.scale;
          }
        } else {
#pragma unroll
          for (int x = 0; x < 4; ++x) fq[it][x] = fk[it][x] = fa[x] = la[x] = 0.f;
        }
        *reinterpret_cast<float4*>(sQ + r * LDK + d4) = make_float4(fq[it][0], fq[it][1], fq[it][2], fq[it][3]);
        *reinterpret_cast<float4*>(sKt + r * LDK + d4) = make_float4(fk[it][0], fk[it][1], fk[it][2], fk[it][3]);
        *reinterpret_cast<float4*>(sLa + r * LDK + d4) = make_float4(la[0], la[1], la[2], la[3]);
        if (MODE == 1) *reinterpret_cast<float4*>(sKe + r * LDK + d4) = make_float4(fa[0], fa[1], fa[2], fa[3]);
      }
    }
    __syncthreads();
    // ---- (2) cumulative decay and scaled operands (rounded to tf32 where they only feed the
    // tensor cores); partial dA on the tensor cores.
    // Where no channel decays by more than e^-60 over the chunk, exp(b_r - b_i) is factored as
    // exp(b_r) exp(-b_i) (Ki = kt . exp(-b) stays below e^60 |kt|) and the sums over pairs become
    // plain contractions; otherwise the chunk takes the pair-by-pair form with the difference
    // formed before the exponential, which is exact for any decay.
    bool strong;
    {
      // job 0: b (and Qe), last job: D; Ke, Ki on the jobs between (all channels: two jobs only)
      constexpr int kJobs = kThreads / NCH;                 // 4 (own half) or 2 (all channels)
      const int d = ch0 + (tid % NCH), job = tid / NCH;
      float tot = 0.f;
#pragma unroll
      for (int r = 0; r < kC; ++r) tot += sLa[r * LDK + d];
      strong = __syncthreads_or(tot < -60.f) != 0;
      const bool do_qe = MODE != 0 && job == (kJobs == 4 ? 1 : 0);
      const bool do_ke = MODE != 1 && job == (kJobs == 4 ? 2 : 1);
      const bool do_ki = MODE == 0 && job == 1 && !strong;   // all channels: with Ke, below
      if (job == 0 || do_qe) {
        float acc = 0.f;
#pragma unroll 4
        for (int r = 0; r < kC; ++r) {
          acc += sLa[r * LDK + d];
          if (job == 0) sB[r * LDK + d] = acc;
          if (do_qe) {
            const float x = sQ[r * LDK + d] * exp_f<FAST>(acc);
            sQe[r * LDK + d] = FAST ? tf32_round(x) : x;
          }
        }
      }
      if (do_ke || do_ki) {
        float part = 0.f;
#pragma unroll 4
        for (int r = 0; r < kC; ++r) {
          part += sLa[r * LDK + d];      // same additions in the same order as above
          const float kt = sKt[r * LDK + d];
          if (do_ke) {
            const float x = kt * exp_f<FAST>(tot - part);
            sKe[r * LDK + d] = FAST ? tf32_round(x) : x;
          }
          if (do_ki) sQe[r * LDK + d] = kt * exp_f<FAST>(-part);
          if (MODE == 2 && !strong) {    // this thread is the array's only reader in this phase
            const float x = kt * exp_f<FAST>(-part);
            sKt[r * LDK + d] = FAST ? tf32_round(x) : x;
          }
        }
      }
      if (job == kJobs - 1) sD[d] = exp_f<FAST>(tot);
    }
    if (MODE != 2) {   // dA[r][i] = sum_j dO[r][j] V[i][j], this warp's 32 value columns
      float acc[2][4] = {};
#pragma unroll
      for (int ks = 0; ks < 4; ++ks) {
        const int j0 = 32 * warp + 8 * ks + 2 * t;
        const float2 x0 = *reinterpret_cast<const float2*>(sDO + g * LDV + j0);
        const float2 x1 = *reinterpret_cast<const float2*>(sDO + (g + 8) * LDV + j0);
        const float af[4] = {x0.x, x1.x, x0.y, x1.y};
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
          const float2 y = *reinterpret_cast<const float2*>(sV + (nt * 8 + g) * LDV + j0);
          const float bf[2] = {y.x, y.y};
          mma_tile<EXACT>(acc[nt], af, bf);
        }
      }
      float* red = sRedA + warp * kC * kC;
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
        red[g * kC + nt * 8 + 2 * t] = acc[nt][0];
        red[g * kC + nt * 8 + 2 * t + 1] = acc[nt][1];
        red[(g + 8) * kC + nt * 8 + 2 * t] = acc[nt][2];
        red[(g + 8) * kC + nt * 8 + 2 * t + 1] = acc[nt][3];
      }
    }
    __syncthreads();
    // ---- (3) masked dA (or scores A), the contraction with the state, the state update
    if (MODE != 2) {
      const int r = tid >> 4, i = tid & 15;
      float s = 0.f;
      if (i <= r) {
#pragma unroll
        for (int w = 0; w < 8; ++w) s += sRedA[w * kC * kC + tid];
      }
      sP[r * LDR + i] = s;
    } else if (strong) {   // A[r][i] pair by pair: lanes over key channels, pairs dealt round the warps
#pragma unroll 1
      for (int p = warp; p < kC * (kC + 1) / 2; p += 8) {
        int r = 0, rem = p;
        while (rem > r) { rem -= r + 1; ++r; }
        const int i = rem;
        float s = 0.f;
#pragma unroll
        for (int m = 0; m < DK / 32; ++m) {
          const int d = lane + 32 * m;
          s = fmaf(sQ[r * LDK + d] * sKt[i * LDK + d], exp_f<FAST>(sB[r * LDK + d] - sB[i * LDK + d]), s);
        }
#pragma unroll
        for (int o = 16; o; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (lane == 0) {
          sP[r * LDR + i] = s;
          if (i != r) sP[i * LDR + r] = 0.f;
        }
      }
    } else {               // A = Qe Ki^T on the tensor cores, this warp's 16 key channels
      float acc[2][4] = {};
#pragma unroll
      for (int ks = 0; ks < 2; ++ks) {
        const int d0 = 16 * warp + 8 * ks + 2 * t;
        const float2 x0 = *reinterpret_cast<const float2*>(sQe + g * LDK + d0);
        const float2 x1 = *reinterpret_cast<const float2*>(sQe + (g + 8) * LDK + d0);
        const float af[4] = {x0.x, x1.x, x0.y, x1.y};
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
          const float2 y = *reinterpret_cast<const float2*>(sKt + (nt * 8 + g) * LDK + d0);
          const float bf[2] = {y.x, y.y};
          mma_tile<EXACT>(acc[nt], af, bf);
        }
      }
      float* red = sRedA + warp * kC * kC;
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
        red[g * kC + nt * 8 + 2 * t] = acc[nt][0];
        red[g * kC + nt * 8 + 2 * t + 1] = acc[nt][1];
        red[(g + 8) * kC + nt * 8 + 2 * t] = acc[nt][2];
        red[(g + 8) * kC + nt * 8 + 2 * t + 1] = acc[nt][3];
      }
    }
    // contraction of the state with the chunk's dO (MODE 0), V (MODE 1) or Ke (MODE 2)
    float cacc[2][4] = {};
    {
      const float* opB = MODE == 0 ? sDO : (MODE == 1 ? sV : sKe);
      constexpr int ldb = MODE == 2 ? LDK : LDV;
#pragma unroll
      for (int n = 0; n < 16; ++n) {
        const int c0 = nbase + 8 * n + 2 * t;
        const float af[4] = {st[n][0], st[n][2], st[n][1], st[n][3]};
#pragma unroll
        for (int rt = 0; rt < 2; ++rt) {
          const float2 y = *reinterpret_cast<const float2*>(opB + (rt * 8 + g) * ldb + c0);
          const float bf[2] = {y.x, y.y};
          mma_tile<EXACT>(cacc[rt], af, bf);
        }
        if ((n & 3) == 3) asm volatile("" ::: "memory");   // keep the operand loads near their use
      }
      if (MODE != 2) {
        float* red = sRed + warp * 16 * LDR;
#pragma unroll
        for (int rt = 0; rt < 2; ++rt) {
          red[g * LDR + rt * 8 + 2 * t] = cacc[rt][0];
          red[g * LDR + rt * 8 + 2 * t + 1] = cacc[rt][1];
          red[(g + 8) * LDR + rt * 8 + 2 * t] = cacc[rt][2];
          red[(g + 8) * LDR + rt * 8 + 2 * t + 1] = cacc[rt][3];
        }
      }
      // state update: scale by D, add the chunk's outer products
      if (MODE != 2) {
        const float dl = sD[m0 + g], dh = sD[m0 + g + 8];
#pragma unroll
        for (int n = 0; n < 16; ++n) {
          st[n][0] *= dl; st[n][1] *= dl; st[n][2] *= dh; st[n][3] *= dh;
        }
        const float* opA = MODE == 0 ? sKe : sQe;
        const float* opV = MODE == 0 ? sV : sDO;
#pragma unroll
        for (int ks = 0; ks < 2; ++ks) {
          const int i0 = 8 * ks + t;
          const float af[4] = {opA[i0 * LDK + m0 + g], opA[i0 * LDK + m0 + g + 8],
                               opA[(i0 + 4) * LDK + m0 + g], opA[(i0 + 4) * LDK + m0 + g + 8]};
#pragma unroll
          for (int n = 0; n < 16; ++n) {
            const int j = nbase + 8 * n + g;
            const float bf[2] = {opV[i0 * LDV + j], opV[(i0 + 4) * LDV + j]};
            mma_tile<EXACT>(st[n], af, bf);
            if ((n & 3) == 3) asm volatile("" ::: "memory");
          }
        }
      } else {
#pragma unroll
        for (int n = 0; n < 16; ++n) {
          const float2 dd = *reinterpret_cast<const float2*>(sD + 8 * n + 2 * t);
          st[n][0] *= dd.x; st[n][1] *= dd.y; st[n][2] *= dd.x; st[n][3] *= dd.y;
        }
#pragma unroll
        for (int ks = 0; ks < 2; ++ks) {
          const int r0 = 8 * ks + t;
          const float af[4] = {sDO[r0 * LDV + m0 + g], sDO[r0 * LDV + m0 + g + 8],
                               sDO[(r0 + 4) * LDV + m0 + g], sDO[(r0 + 4) * LDV + m0 + g + 8]};
#pragma unroll
          for (int n = 0; n < 16; ++n) {
            const float bf[2] = {sQe[r0 * LDK + 8 * n + g], sQe[(r0 + 4) * LDK + 8 * n + g]};
            mma_tile<EXACT>(st[n], af, bf);
            if ((n & 3) == 3) asm volatile("" ::: "memory");
          }
        }
      }
    }
    __syncthreads();
    // ---- (4) finish the chunk's gradients
    if (MODE == 0) {
      const int dl = tid & 63, d = 64 * half + dl;
      const float* r0p = sRed + (2 * (dl >> 4)) * 16 * LDR + (dl & 15) * LDR;
      const float* r1p = r0p + 16 * LDR;
#pragma unroll 1
      for (int r = tid >> 6; r < nr; r += 4) {
        const float br = sB[r * LDK + d];
        float s = 0.f;
        if (strong) {
#pragma unroll 2
          for (int i = 0; i <= r; ++i)
            s = fmaf(sP[r * LDR + i] * sKt[i * LDK + d], exp_f<FAST>(br - sB[i * LDK + d]), s);
          s = fmaf(exp_f<FAST>(br), r0p[r] + r1p[r], s);
        } else {
          s = r0p[r] + r1p[r];
#pragma unroll 4
          for (int i = 0; i <= r; ++i) s = fmaf(sP[r * LDR + i], sQe[i * LDK + d], s);   // Ki
          s *= exp_f<FAST>(br);
        }
        const long long o = (row0 + t0 + r) * DK + d;   // s = dL/d(scale q)
        ((T*)a.dq)[o] = from_f32<T>(a.scale * s);
        a.u[o] = sQ[r * LDK + d] * s;                    // q . dq
      }
    } else if (MODE == 1) {
      const int dl = tid & 63, d = 64 * half + dl;
      const float* r0p = sRed + (2 * (dl >> 4)) * 16 * LDR + (dl & 15) * LDR;
      const float* r1p = r0p + 16 * LDR;
      const float bc = sB[(kC - 1) * LDK + d];
#pragma unroll 1
      for (int i = tid >> 6; i < nr; i += 4) {
        const float bi = sB[i * LDK + d];
        float s = 0.f;
        if (strong) {
#pragma unroll 2
          for (int r = i; r < nr; ++r)
            s = fmaf(sP[r * LDR + i] * sQ[r * LDK + d], exp_f<FAST>(sB[r * LDK + d] - bi), s);
          s = fmaf(exp_f<FAST>(bc - bi), r0p[i] + r1p[i], s);
        } else {
          s = sD[d] * (r0p[i] + r1p[i]);
#pragma unroll 4
          for (int r = i; r < nr; ++r) s = fmaf(sP[r * LDR + i], sQe[r * LDK + d], s);
          s *= exp_f<FAST>(-bi);
        }
        const long long o = (row0 + t0 + i) * DK + d;   // s = dL/d(ahat k)
        ((T*)a.dk)[o] = from_f32<T>(s * sKe[i * LDK + d]);
        a.w[o] = sKt[i * LDK + d] * s;
      }
    } else {
      constexpr int ldo = 128 + 4;
      if (!strong) {   // finish the scores: sum the warps' parts, keep i <= r
        const int r = tid >> 4, i = tid & 15;
        float s = 0.f;
        if (i <= r) {
#pragma unroll
          for (int w = 0; w < 8; ++w) s += sRedA[w * kC * kC + tid];
        }
        sP[r * LDR + i] = s;
      }
      __syncthreads();
      // dv^T[j][i] += sum_r dO[r][j] A[r][i] (A is zero above the diagonal and in rows past the end)
#pragma unroll
      for (int ks = 0; ks < 2; ++ks) {
        const int r0 = 8 * ks + t;
        const float af[4] = {sDO[r0 * LDV + m0 + g], sDO[r0 * LDV + m0 + g + 8],
                             sDO[(r0 + 4) * LDV + m0 + g], sDO[(r0 + 4) * LDV + m0 + g + 8]};
#pragma unroll
        for (int rt = 0; rt < 2; ++rt) {
          const float bf[2] = {sP[r0 * LDR + rt * 8 + g], sP[(r0 + 4) * LDR + rt * 8 + g]};
          mma_tile<true>(cacc[rt], af, bf);   // scores are fp32 values: keep both tf32 parts
        }
      }
      {
        const int jl = 16 * warp + g;
#pragma unroll
        for (int rt = 0; rt < 2; ++rt) {
          sRed[(rt * 8 + 2 * t) * ldo + jl] = cacc[rt][0];
          sRed[(rt * 8 + 2 * t + 1) * ldo + jl] = cacc[rt][1];
          sRed[(rt * 8 + 2 * t) * ldo + jl + 8] = cacc[rt][2];
          sRed[(rt * 8 + 2 * t + 1) * ldo + jl + 8] = cacc[rt][3];
        }
      }
      __syncthreads();
      const int i = tid >> 4, c8 = (tid & 15) * 8;
      if (i < nr) {
        float o8[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) o8[e] = sRed[i * ldo + c8 + e];
        store8<T>((T*)a.dv + (row0 + t0 + i) * DV + 128 * half + c8, o8);
      }
    }
    __syncthreads();
  }

  if (segment_of_this_cta(a) + 1 < a.nseg) {   // hand the state to the next segment
    float* hand = a.seg_state + (sh * 3 + MODE) * (long long)DK * DV;
#pragma unroll
    for (int n = 0; n < 16; ++n) {
      const int c0 = nbase + 8 * n + 2 * t;
      if (MODE != 2) {
        *reinterpret_cast<float2*>(hand + (long long)(m0 + g) * DV + c0) = make_float2(st[n][0], st[n][1]);
        *reinterpret_cast<float2*>(hand + (long long)(m0 + g + 8) * DV + c0) = make_float2(st[n][2], st[n][3]);
      } else {
        hand[(long long)c0 * DV + m0 + g] = st[n][0];
        hand[(long long)(c0 + 1) * DV + m0 + g] = st[n][1];
        hand[(long long)c0 * DV + m0 + g + 8] = st[n][2];
        hand[(long long)(c0 + 1) * DV + m0 + g + 8] = st[n][3];
      }
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) st_release_s32(a.seg_flag + sh * 6 + (MODE * 2 + half), segment_of_this_cta(a) + 1);
    return;
  }
  // ---- after the last chunk
  if (MODE == 0) {   // c[d] = sum_j dS_T[d][j] S_T[d][j]
    float p0 = 0.f, p1 = 0.f;
    if (a.dsT) {
#pragma unroll
      for (int n = 0; n < 16; ++n) {
        const int c0 = nbase + 8 * n + 2 * t;
        const float2 lo = *reinterpret_cast<const float2*>(a.dsT + s_off + (long long)(m0 + g) * DV + c0);
        const float2 hi = *reinterpret_cast<const float2*>(a.dsT + s_off + (long long)(m0 + g + 8) * DV + c0);
        p0 = fmaf(lo.x, st[n][0], fmaf(lo.y, st[n][1], p0));
        p1 = fmaf(hi.x, st[n][2], fmaf(hi.y, st[n][3], p1));
      }
    }
    p0 += __shfl_xor_sync(0xffffffffu, p0, 1);
    p0 += __shfl_xor_sync(0xffffffffu, p0, 2);
    p1 += __shfl_xor_sync(0xffffffffu, p1, 1);
    p1 += __shfl_xor_sync(0xffffffffu, p1, 2);
    if (t == 0) {
      sRed[warp * 16 + g] = p0;
      sRed[warp * 16 + g + 8] = p1;
    }
    __syncthreads();
    if (tid < 64)
      a.c[sh * DK + 64 * half + tid] = sRed[(2 * (tid >> 4)) * 16 + (tid & 15)] +
                                        sRed[(2 * (tid >> 4) + 1) * 16 + (tid & 15)];
  } else if (MODE == 1 && a.ds0) {
#pragma unroll
    for (int n = 0; n < 16; ++n) {
      const int c0 = nbase + 8 * n + 2 * t;
      *reinterpret_cast<float2*>(a.ds0 + s_off + (long long)(m0 + g) * DV + c0) = make_float2(st[n][0], st[n][1]);
      *reinterpret_cast<float2*>(a.ds0 + s_off + (long long)(m0 + g + 8) * DV + c0) = make_float2(st[n][2], st[n][3]);
    }
  }
}

constexpr size_t kSweepSmem =
    sizeof(float) * (6 * kC * LDK + 2 * kC * LDV + DK + kC * LDR + 8 * kC * kC + 8 * 16 * LDR);
static_assert(16 * (128 + 4) <= 8 * 16 * LDR, "the dv tile fits the space of the partials");

template <typename T>
__global__ void __launch_bounds__(kThreads, 2) ddts_bwd_sweep_kernel(const BwdArgs a) {
  extern __shared__ __align__(16) float smem[];
  // The three sweeps differ in length (on the layer shape: the transposed reverse sweep 1.14 ms,
  // the forward sweep 0.99, the reverse sweep 0.91) and the grid is about 1.3 times the resident
  // CTAs, so the index runs over the sweeps from the longest to the shortest and, within a sweep,
  // over all (sequence, head): what starts late is short.
  const unsigned n_items = gridDim.x / (6 * a.nseg);
  const long long sh = blockIdx.x % n_items;     // sequence * H + head
  const int seg = segment_of_this_cta(a);
  const int slot = (int)(blockIdx.x / n_items) % 6;
  const int part = slot < 2 ? 4 + slot : slot - 2, mode = part >> 1, half = part & 1;
  if (!a.cu && blockIdx.x == 0 && threadIdx.x == 0) a.hdr->status = RODIMUS_OK;
  const int h = (int)(sh % a.H);
  const long long n = sh / a.H;
  long long row0;
  int len;
  if (a.cu) {
    int lo = a.cu[n], hi = a.cu[n + 1];
    lo = lo < 0 ? 0 : (lo > a.T ? a.T : lo);
    hi = hi < lo ? lo : (hi > a.T ? a.T : hi);
    row0 = (long long)h * a.T + lo;
    len = hi - lo;
  } else {
    row0 = sh * a.T;
    len = a.T;
  }
  if (a.nseg > 1) {
    // this segment's rows: chunks c_lo .. c_hi-1 of the sweep, counted from the sequence's start
    // (forward sweep) or from its end (reverse sweeps); row0, len become those of the segment
    const int nchunks = (len + kC - 1) / kC;
    const int c_lo = (int)((long long)nchunks * seg / a.nseg), c_hi = (int)((long long)nchunks * (seg + 1) / a.nseg);
    const int r_lo = (mode == 0 ? c_lo : nchunks - c_hi) * kC;
    const int r_hi = min((mode == 0 ? c_hi : nchunks - c_lo) * kC, len);
    row0 += r_lo;
    len = r_hi > r_lo ? r_hi - r_lo : 0;
  }
  if (seg > 0) {
    // The segment before this one belongs to a CTA with a lower index, and CTAs start in the
    // order of their index: it is running or done.  The wait is bounded all the same.
    const int32_t* flag = a.seg_flag + sh * 6 + part;
    int late = 0;
    if (threadIdx.x == 0) {
      const long long t_start = clock64();
      while (ld_acquire_s32(flag) < seg) {
        if (clock64() - t_start > a.limit) { late = 1; break; }
        __nanosleep(256);
      }
    }
    if (__syncthreads_or(late)) {
      if (threadIdx.x == 0) atomicMax(&a.hdr->status, (int)RODIMUS_ERR_TIMEOUT);
      return;
    }
  }
  if (mode == 0) bwd_sweep<T, 0>(a, smem, sh, half, row0, len, seg);
  else if (mode == 1) bwd_sweep<T, 1>(a, smem, sh, half, row0, len, seg);
  else bwd_sweep<T, 2>(a, smem, sh, half, row0, len, seg);
}

// dL/dlog alpha by suffix sums over the sequence, then dx, dy (Eq. "alpha_def", chain rule):
//   log alpha = -g tau,  log ahat = tau ln u(g)   with u = g (paper) or 1 - e^-g = sigmoid(x)
//   dg   = -tau dla + w tau u'/u        dtau = -g dla + w ln u
//   dx   = dg sigmoid(x)                dy   = dtau tau (1 - tau)
// One CTA per (sequence, head, 32 channels): 32 channels x 16 time segments.
constexpr int kGateCh = 32, kGateSegs = 16;
template <typename T>
__global__ void __launch_bounds__(kGateCh * kGateSegs) ddts_bwd_gates_kernel(const BwdArgs a) {
  __shared__ double seg_sum[kGateSegs][kGateCh];
  const long long sh = blockIdx.x / (DK / kGateCh);
  const int dch = (blockIdx.x % (DK / kGateCh)) * kGateCh;
  const int h = (int)(sh % a.H);
  const long long n = sh / a.H;
  long long row0;
  int len;
  if (a.cu) {
    int lo = a.cu[n], hi = a.cu[n + 1];
    lo = lo < 0 ? 0 : (lo > a.T ? a.T : lo);
    hi = hi < lo ? lo : (hi > a.T ? a.T : hi);
    row0 = (long long)h * a.T + lo;
    len = hi - lo;
  } else {
    row0 = sh * a.T;
    len = a.T;
  }
  const int dl = threadIdx.x % kGateCh, d = dch + dl, seg = threadIdx.x / kGateCh;
  const int per = (len + kGateSegs - 1) / kGateSegs;
  const int lo = min(len, seg * per), hi = min(len, lo + per);
  double s = 0.0;
  for (int r = lo; r < hi; ++r) {
    const long long i = (row0 + r) * DK + d;
    s += (double)a.u[i] - (double)a.w[i];
  }
  seg_sum[seg][dl] = s;
  __syncthreads();
  double acc = (double)a.c[sh * DK + d];
  for (int s2 = seg + 1; s2 < kGateSegs; ++s2) acc += seg_sum[s2][dl];
  const T* gx = (const T*)a.gx;
  const T* ty = (const T*)a.ty;
  for (int r = hi - 1; r >= lo; --r) {
    const long long i = (row0 + r) * DK + d;
    const float w = a.w[i];
    acc += (double)a.u[i] - (double)w;
    const float dla = (float)acc;
    const float x = to_f32(gx[i]), y = to_f32(ty[i]);
    const float g = softplus_f32(x);
    const float tau = y >= 0.f ? 1.f / (1.f + expf(-y)) : expf(y) / (1.f + expf(y));
    const float sx = x >= 0.f ? 1.f / (1.f + expf(-x)) : expf(x) / (1.f + expf(x));
    float lnu, dgx;   // dgx = (u'/u) * sigmoid(x)
    if (a.ingate == RODIMUS_INGATE_POW_G) {
      lnu = logf(g);
      dgx = sx / g;
    } else {
      lnu = -softplus_f32(-x);
      dgx = x >= 0.f ? expf(-x) / (1.f + expf(-x)) : 1.f / (1.f + expf(x));   // 1 - sigmoid(x)
    }
    const float dxv = -tau * dla * sx + w * tau * dgx;
    const float dyv = (-g * dla + w * lnu) * tau * (1.f - tau);
    ((T*)a.dx)[i] = from_f32<T>(dxv);
    ((T*)a.dy)[i] = from_f32<T>(dyv);
  }
}

std::atomic<unsigned long long> g_smem_done_bf16{0}, g_smem_done_f32{0};

}  // namespace

bool bwd_supported(const rodimus_ddts_bwd_params& p) { return p.dk == DK && p.dv == DV; }

size_t bwd_scratch_bytes(const rodimus_ddts_bwd_params& p) {
  const size_t rows = (size_t)p.B * p.H * p.T;
  const size_t nseq = p.cu_seqlens ? (size_t)p.N : (size_t)p.B;
  size_t b = sizeof(float) * (2 * rows * DK + nseq * p.H * DK);
  b = (b + 255) & ~(size_t)255;
  b += nseq * p.H * 6 * (sizeof(float) * 64 * kThreads);        // state fragments between time segments
  b += (nseq * p.H * 6 * sizeof(int32_t) + 255) & ~(size_t)255; // and their flags
  return b;
}

cudaError_t launch_bwd(const rodimus_ddts_bwd_params& p, size_t scratch_offset, int* n_launches) {
  *n_launches = 0;
  BwdArgs a;
  a.q = p.q; a.k = p.k; a.gx = p.gate_x; a.ty = p.temp_y; a.v = p.v; a.dout = p.d_o;
  a.s0 = p.s0; a.dsT = p.d_sT;
  a.dq = p.d_q; a.dk = p.d_k; a.dx = p.d_gate_x; a.dy = p.d_temp_y; a.dv = p.d_v; a.ds0 = p.d_s0;
  const size_t rows = (size_t)p.B * p.H * p.T;
  a.u = reinterpret_cast<float*>(reinterpret_cast<char*>(p.workspace) + scratch_offset);
  a.w = a.u + rows * DK;
  a.c = a.w + rows * DK;
  {
    const size_t nseq = p.cu_seqlens ? (size_t)p.N : (size_t)p.B;
    const size_t first = (sizeof(float) * (2 * rows * DK + nseq * p.H * DK) + 255) & ~(size_t)255;
    a.seg_state = reinterpret_cast<float*>(reinterpret_cast<char*>(p.workspace) + scratch_offset + first);
    a.seg_flag = reinterpret_cast<int32_t*>(a.seg_state + nseq * p.H * 6 * (size_t)64 * kThreads);
  }
  a.cu = p.cu_seqlens;
  a.hdr = reinterpret_cast<WorkspaceHeader*>(p.workspace);
  a.H = p.H; a.T = p.T; a.n_seq = p.cu_seqlens ? p.N : p.B;
  a.scale = p.scale; a.ingate = p.ingate;
  const long long items = (long long)a.n_seq * p.H;
  if (items == 0) return cudaSuccess;
  if (items * 6 > 0x7fffffffLL) return cudaErrorInvalidValue;
  int dev = 0, sms = 0;
  cudaError_t e = current_device(&dev, &sms);
  if (e != cudaSuccess) return e;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(p.stream);
  // Time segments per sweep: a sweep is one serial scan, and 6 CTAs per (sequence, head) seldom
  // fill the resident CTA slots evenly (the layer shape: 384 CTAs of ~1 ms on 296 slots = two
  // rounds).  Cutting every sweep into n segments gives n times the CTAs at 1/n the length; n of
  // 1..8 minimises rounds(n) / n, with at least four chunks per segment.  Equal costs go to the
  // finer cut while the grid is only a few rounds (the three sweeps differ in length, and finer
  // pieces pack better: 1.87 ms for n = 3, 1.81 for 6 on the layer shape), else to the coarser.
  {
    const long long slots = 2LL * sms, per_seq = p.T / (p.cu_seqlens ? (a.n_seq > 0 ? a.n_seq : 1) : 1);
    const bool few_rounds = items * 6 < 4 * slots;
    int best = 1;
    double best_cost = 1e30;
    for (int n = 1; n <= 8; ++n) {
      if (n > 1 && per_seq < (long long)n * 4 * kC) break;
      const double cost = (double)((items * 6 * n + slots - 1) / slots) / n;
      if (cost < best_cost * 0.999 || (few_rounds && cost < best_cost * 1.001)) { best_cost = cost; best = n; }
    }
    a.nseg = best;
    a.limit = main_loop_wait_cycles();
    if (items * 6 * a.nseg > 0x7fffffffLL) return cudaErrorInvalidValue;
    if (a.nseg > 1) {
      e = cudaMemsetAsync(a.seg_flag, 0, sizeof(int32_t) * (size_t)items * 6, st);
      if (e != cudaSuccess) return e;
    }
  }
  if (p.dtype == RODIMUS_BF16) {
    e = opt_in_shared_memory(ddts_bwd_sweep_kernel<__nv_bfloat16>, (int)kSweepSmem, dev, g_smem_done_bf16);
    if (e != cudaSuccess) return e;
    ddts_bwd_sweep_kernel<__nv_bfloat16><<<(unsigned)(items * 6 * a.nseg), kThreads, kSweepSmem, st>>>(a);
    ddts_bwd_gates_kernel<__nv_bfloat16><<<(unsigned)(items * (DK / kGateCh)), kGateCh * kGateSegs, 0, st>>>(a);
  } else {
    e = opt_in_shared_memory(ddts_bwd_sweep_kernel<float>, (int)kSweepSmem, dev, g_smem_done_f32);
    if (e != cudaSuccess) return e;
    ddts_bwd_sweep_kernel<float><<<(unsigned)(items * 6 * a.nseg), kThreads, kSweepSmem, st>>>(a);
    ddts_bwd_gates_kernel<float><<<(unsigned)(items * (DK / kGateCh)), kGateCh * kGateSegs, 0, st>>>(a);
  }
  *n_launches = 2;
  return cudaGetLastError();
}

}  // namespace ddts
