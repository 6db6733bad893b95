// Chunked prefill on the CUDA cores, all arithmetic in fp32 (the validation build, and the
// kernel for every shape the tensor-core kernel does not cover).
//
// Same algebra as the appendix "Chunkwise Parallel Representation of the Rodimus Block", with
// the state entering the chunk in the inter-chunk readout:
//   b_r   = sum_{j<=r in chunk} log alpha_j                      (per key channel)
//   P_ri  = sum_d q_rd k_id ahat_id exp(b_rd - b_id),  i <= r    (difference formed BEFORE exp)
//   O_r   = sum_{i<=r} P_ri v_i + (q_r . exp(b_r)) S_in
//   S_out = diag(exp(b_C)) S_in + sum_i (k_i . ahat_i . exp(b_C - b_i))^T v_i
// Every exponent is <= 0 apart from log ahat, so no input in the documented domain overflows,
// whatever the decay.
//
// Optional value-side decay beta_t (general transition of Sec. 3.1.1, the arm the paper ablates
// and drops): with c_r = sum_{j<=r in chunk} log beta_j per value column,
//   O_r   = sum_{i<=r} P_ri (v_i . exp(c_r - c_i)) + exp(c_r) . ((q_r . exp(b_r)) S_in)
//   S_out = (exp(b_C)^T exp(c_C)) . S_in + sum_i (k_i . ahat_i . exp(b_C - b_i))^T (v_i . exp(c_C - c_i))
//
// Work item = (sequence, head, tile of kTileV state columns); one CTA per item keeps its
// [dk, kTileV] slice of the state in shared memory for the whole sequence.
#include "ddts_common.cuh"

namespace ddts {
namespace {

constexpr int kC = 16;          // chunk length
constexpr int kTileV = 64;      // state columns per CTA
constexpr int kThreads = 256;

struct SimtArgs {
  const void *q, *k, *gx, *ty, *v;
  const void *beta_hat, *feed_x;   // optional: value gate [.., dv], feed-through input [.., dv]
  const void *vdecay;              // optional: value-side decay beta_t [.., dv], numbers in (0,1]
  const float* feed_d;             // optional: feed-through weight [H, dv]
  void* o;
  const float* s0;
  float* sT;
  const int32_t* cu;  // device cu_seqlens or nullptr
  WorkspaceHeader* hdr;
  int H, T, dk, dv, n_seq, tiles;
  float scale;
  int ingate;
  int shared;   // 1: q,k,gx,ty are [B,1,T,dk], one set per token for all heads
};

template <typename T>
__global__ void __launch_bounds__(kThreads, 1) ddts_fwd_simt_kernel(const SimtArgs a) {
  extern __shared__ float smem[];
  const int dk = a.dk, dv = a.dv;
  const int ld = dk + 1;                       // padded row stride of the [kC, dk] arrays
  float* sS = smem;                            // [dk][kTileV]  state slice
  float* sQ = sS + dk * kTileV;                // [kC][ld]      q
  float* sW = sQ + kC * ld;                    // [kC][ld]      ahat * k
  float* sB = sW + kC * ld;                    // [kC][ld]      b (cumulative log decay)
  float* sV = sB + kC * ld;                    // [kC][kTileV]
  float* sP = sV + kC * kTileV;                // [kC][kC]
  float* sE = sP + kC * kC;                    // [dk]          b at the chunk end
  float* sC = sE + dk;                         // [kC][kTileV]  c (cumulative log beta), if given

  const int tid = threadIdx.x;
  const long long item = blockIdx.x;
  // dense calls have no planning kernel in front: the first CTA clears the device status
  if (!a.cu && item == 0 && tid == 0) a.hdr->status = RODIMUS_OK;
  const int tile = (int)(item % a.tiles);
  const long long sh = item / a.tiles;         // sequence * H + head
  const int h = (int)(sh % a.H);
  const long long n = sh / a.H;
  const int col0 = tile * kTileV;

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
  // rows of q,k,gx,ty: the head's own, or the sequence's single shared set
  const long long rq = a.shared ? row0 - ((long long)h + (a.cu ? 0 : n * (a.H - 1))) * a.T : row0;
  const T* q = (const T*)a.q + rq * dk;
  const T* k = (const T*)a.k + rq * dk;
  const T* gx = (const T*)a.gx + rq * dk;
  const T* ty = (const T*)a.ty + rq * dk;
  const T* v = (const T*)a.v + row0 * dv;
  T* o = (T*)a.o + row0 * dv;
  const T* bh = a.beta_hat ? (const T*)a.beta_hat + row0 * dv : nullptr;
  const T* fx = a.feed_d ? (const T*)a.feed_x + row0 * dv : nullptr;
  const float* fd = a.feed_d ? a.feed_d + (long long)h * dv : nullptr;
  const T* bd = a.vdecay ? (const T*)a.vdecay + row0 * dv : nullptr;
  const long long s_off = sh * (long long)dk * dv;

  for (int e = tid; e < dk * kTileV; e += kThreads) {
    const int d = e / kTileV, c = e % kTileV;
    sS[e] = (a.s0 && col0 + c < dv) ? a.s0[s_off + (long long)d * dv + col0 + c] : 0.f;
  }
  __syncthreads();

  for (int t0 = 0; t0 < len; t0 += kC) {
    const int nr = min(kC, len - t0);
    // (1) gates and in-chunk cumulative log decay: one thread per key channel
    for (int d = tid; d < dk; d += kThreads) {
      float b = 0.f;
      for (int r = 0; r < nr; ++r) {
        const long long i = (long long)(t0 + r) * dk + d;
        float la, lh;
        gate_logs_f32(to_f32(gx[i]), to_f32(ty[i]), a.ingate, la, lh);
        b += la;
        sB[r * ld + d] = b;
        sW[r * ld + d] = expf(lh) * to_f32(k[i]);
        sQ[r * ld + d] = to_f32(q[i]);
      }
      sE[d] = b;
    }
    for (int e = tid; e < kC * kTileV; e += kThreads) {
      const int r = e / kTileV, c = e % kTileV;
      float vv = 0.f;
      if (r < nr && col0 + c < dv) {
        const long long i = (long long)(t0 + r) * dv + col0 + c;
        vv = to_f32(v[i]);
        if (bh) vv *= to_f32(bh[i]);   // value gate (Eq. "beta_def")
      }
      sV[e] = vv;
    }
    if (bd) {   // cumulative log of the value-side decay: one thread per state column
      for (int c = tid; c < kTileV; c += kThreads) {
        float cum = 0.f;
        for (int r = 0; r < kC; ++r) {
          if (r < nr && col0 + c < dv)
            cum += logf(fmaxf(to_f32(bd[(long long)(t0 + r) * dv + col0 + c]), 1e-37f));
          sC[r * kTileV + c] = cum;
        }
      }
    }
    __syncthreads();
    // (2) intra-chunk scores, causal mask with the diagonal kept
    {
      const int r = tid / kC, i = tid % kC;
      float p = 0.f;
      if (i <= r && r < nr) {
        const float *qr = sQ + r * ld, *br = sB + r * ld, *wi = sW + i * ld, *bi = sB + i * ld;
        for (int d = 0; d < dk; ++d) p = fmaf(qr[d] * wi[d], expf(br[d] - bi[d]), p);
      }
      sP[tid] = p;
    }
    __syncthreads();
    // fold exp(b_r) into q for the inter-chunk readout (after the scores have used raw q)
    for (int e = tid; e < nr * dk; e += kThreads) {
      const int r = e / dk, d = e % dk;
      sQ[r * ld + d] *= expf(sB[r * ld + d]);
    }
    __syncthreads();
    // (3) output rows
    for (int e = tid; e < kC * kTileV; e += kThreads) {
      const int r = e / kTileV, c = e % kTileV;
      if (r < nr && col0 + c < dv) {
        float acc = 0.f;
        const float* qr = sQ + r * ld;
        if (bd) {
          const float cr = sC[r * kTileV + c];
          for (int d = 0; d < dk; ++d) acc = fmaf(qr[d], sS[d * kTileV + c], acc);
          acc *= expf(cr);
          for (int i = 0; i <= r; ++i)
            acc = fmaf(sP[r * kC + i], sV[i * kTileV + c] * expf(cr - sC[i * kTileV + c]), acc);
        } else {
          for (int i = 0; i <= r; ++i) acc = fmaf(sP[r * kC + i], sV[i * kTileV + c], acc);
          for (int d = 0; d < dk; ++d) acc = fmaf(qr[d], sS[d * kTileV + c], acc);
        }
        const long long i = (long long)(t0 + r) * dv + col0 + c;
        acc *= a.scale;
        if (fd) acc = fmaf(fd[col0 + c], to_f32(fx[i]), acc);   // feed-through d . x'
        o[i] = from_f32<T>(acc);
      }
    }
    __syncthreads();
    // (4) state update: fold exp(b_C - b_i) into ahat*k once, then contract over the chunk
    for (int e = tid; e < nr * dk; e += kThreads) {
      const int i = e / dk, d = e % dk;
      sW[i * ld + d] *= expf(sE[d] - sB[i * ld + d]);
    }
    if (bd) {   // v_i . exp(c_C - c_i), in place (the outputs are done with v)
      for (int e = tid; e < nr * kTileV; e += kThreads)
        sV[e] *= expf(sC[(kC - 1) * kTileV + e % kTileV] - sC[e]);
    }
    __syncthreads();
    for (int e = tid; e < dk * kTileV; e += kThreads) {
      const int d = e / kTileV, c = e % kTileV;
      float acc = expf(sE[d]) * sS[e];
      if (bd) acc *= expf(sC[(kC - 1) * kTileV + c]);
      for (int i = 0; i < nr; ++i) acc = fmaf(sW[i * ld + d], sV[i * kTileV + c], acc);
      sS[e] = acc;
    }
    __syncthreads();
  }

  if (a.sT) {
    for (int e = tid; e < dk * kTileV; e += kThreads) {
      const int d = e / kTileV, c = e % kTileV;
      if (col0 + c < dv) a.sT[s_off + (long long)d * dv + col0 + c] = sS[e];
    }
  }
}

size_t simt_smem_bytes(int dk) {
  const int ld = dk + 1;
  return sizeof(float) * ((size_t)dk * kTileV + 3 * (size_t)kC * ld + 2 * kC * kTileV + kC * kC + dk);
}

}  // namespace

cudaError_t launch_fwd_simt(const rodimus_ddts_fwd_params& p, int* n_launches) {
  *n_launches = 0;
  SimtArgs a;
  a.q = p.q; a.k = p.k; a.gx = p.gate_x; a.ty = p.temp_y; a.v = p.v; a.o = p.o;
  a.beta_hat = p.beta_hat; a.feed_x = p.feed_x; a.feed_d = p.feed_d; a.vdecay = p.value_decay;
  a.s0 = p.s0; a.sT = p.sT; a.cu = p.cu_seqlens;
  a.hdr = reinterpret_cast<WorkspaceHeader*>(p.workspace);
  a.H = p.H; a.T = p.T; a.dk = p.dk; a.dv = p.dv;
  a.n_seq = p.cu_seqlens ? p.N : p.B;
  a.tiles = (p.dv + kTileV - 1) / kTileV;
  a.scale = p.scale; a.ingate = p.ingate; a.shared = p.shared_gates;
  const long long items = (long long)a.n_seq * p.H * a.tiles;
  if (items == 0) return cudaSuccess;
  if (items > 0x7fffffffLL) return cudaErrorInvalidValue;
  const size_t smem = simt_smem_bytes(p.dk);
  cudaStream_t st = reinterpret_cast<cudaStream_t>(p.stream);
  cudaError_t e;
  if (p.dtype == RODIMUS_BF16) {
    e = cudaFuncSetAttribute(ddts_fwd_simt_kernel<__nv_bfloat16>,
                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    ddts_fwd_simt_kernel<__nv_bfloat16><<<(unsigned)items, kThreads, smem, st>>>(a);
  } else {
    e = cudaFuncSetAttribute(ddts_fwd_simt_kernel<float>,
                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    ddts_fwd_simt_kernel<float><<<(unsigned)items, kThreads, smem, st>>>(a);
  }
  *n_launches = 1;
  return cudaGetLastError();
}

}  // namespace ddts
