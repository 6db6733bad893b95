// Sliding-window shared-key attention on tcgen05 (bf16 tokens, head size 128):
//   s_ti = scale <q^h_t, k_i>,  t - W < i <= t      p_ti = softmax_i(s_ti)      o^h_t = sum_i p_ti v^h_i
// (Sec. "Shared-Key Attention for Lossless Head Compression": one key per token for all heads.)
//
// One CTA per (batch, head, 128 queries): 8 softmax warps, one warp that issues the contractions
// and one that issues the TMA loads.  Query row =
// tensor-memory lane; two softmax threads per row (32 of a tile's 64 key columns each; they
// exchange one maximum per tile and one sum at the end through shared memory).  Per key tile of
// 64 tokens:
//   S = Q K^T        tcgen05.mma, Q tile and K tile K-major in shared memory (TMA, 128-byte
//                    swizzle), accumulator [128 x 64] fp32 in tensor memory, TWO buffers: the
//                    scores of tile i+1 are computed while the softmax of tile i runs
//   softmax          each thread reads its part of a row of S (tcgen05.ld), keeps a reference
//                    exponent and a sum in the log2 domain, rescales its part of the row of O in
//                    tensor memory when the reference moved (lazily: only when a tile's maximum
//                    exceeds it by more than 2^8), and writes the probabilities back over S as
//                    packed bf16 (tcgen05.st)
//   O += P V         tcgen05.mma, A = P from tensor memory, B = the V tile (token-major, i.e.
//                    N-major) from shared memory
// Issuing a tcgen05.mma or a TMA load costs its thread about a hundred cycles here, which is why
// two threads of two warps share that work and the softmax warps do none of it.  Tensor memory: 256 columns
// (S twice 64, O 128); shared memory 96 KiB (Q 32, two K tiles, two V tiles; a tile is requested
// two tiles ahead, as soon as the contraction that read its slot is complete): two CTAs per SM.  Only key tiles that
// touch the 128 queries' windows are visited.  Every wait is bounded; a wait that runs out ends
// the kernel cleanly (copies and contractions in flight are waited for, tensor memory is freed)
// and raises RODIMUS_ERR_TIMEOUT in the status word.  No hardware barrier is used inside the
// loop (a role that gave up would leave the others at it).
#include "ddts_tc_ptx.cuh"

namespace ddts {
namespace {

constexpr int kD = 128, kBM = 128, kBN = 64, kHalf = kBN / 2;
constexpr int kSoftmaxWarps = 8, kIssuerWarp = 8, kProducerWarp = 9, kThreads = 32 * (kSoftmaxWarps + 2);
constexpr uint32_t kQSlabBytes = kBM * 128;           // [128 rows][64 columns] bf16
constexpr uint32_t kSlabBytes = kBN * 128;            // [64 rows][64 columns] bf16
constexpr uint32_t kTileBytes = 2 * kSlabBytes;       // 64 x 128 bf16
constexpr uint32_t kOffQ = 0, kOffK = 2 * kQSlabBytes, kOffV = kOffK + 2 * kTileBytes;
constexpr uint32_t kOffCtl = kOffV + 2 * kTileBytes;
constexpr uint32_t kOffMax = kOffCtl + 256;            // [2][2][128] floats: the halves' row maxima (by buffer) / sums
constexpr uint32_t kSmemBytes = kOffMax + 2048 + 1024; // + slack for 1024-byte alignment
constexpr uint32_t kTmemCols = 256, kColS = 0, kColO = 128;
constexpr float kLog2e = 1.4426950408889634f;

enum { BAR_Q = 0, BAR_K0, BAR_K1, BAR_V0, BAR_V1, BAR_S0, BAR_S1, BAR_P0, BAR_P1, BAR_O0, BAR_O1, BAR_PAIR0,
       BAR_DRAIN = BAR_PAIR0 + 4, kNumBars };

struct SwCtl {
  uint64_t bar[kNumBars];
  uint32_t tmem_base;
  int abort;
  long long limit;
  int k_sent, v_sent, k_seen, v_seen;   // loads asked for / seen complete (for the clean exit)
};

// Two fp32 operations in one instruction (packed pairs in 64-bit registers) and the three-input
// maximum: the softmax loop is bound by instruction issue and by the special-function unit, and
// these halve the count of everything around the exponentials.
__device__ __forceinline__ uint64_t pair_f32(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpair_f32(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

struct SwTcArgs {
  void* o;
  int32_t* status;   // may be nullptr
  int B, H, T, window, n_qtiles;
  float scale;
  long long limit;
};

__device__ __noinline__ bool sw_wait_slow(uint32_t bar, uint32_t parity, volatile SwCtl* c, int32_t* status) {
  const long long limit = c->limit, t0 = clock64();
  while (true) {
    if (limit > 0) {
#pragma unroll 1
      for (int i = 0; i < 16; ++i)
        if (mbar_try_park(bar, parity)) return true;
    }
    if (c->abort) return mbar_try(bar, parity);
    if (clock64() - t0 >= limit) {
      if (mbar_try(bar, parity)) return true;
      c->abort = 1;
      if (status) atomicMax(status, (int)RODIMUS_ERR_TIMEOUT);
      return false;
    }
  }
}
__device__ __forceinline__ bool sw_wait(uint32_t bar, uint32_t parity, volatile SwCtl* c, int32_t* status) {
  if (mbar_try(bar, parity)) return true;
  return sw_wait_slow(bar, parity, c, status);
}

__global__ void __launch_bounds__(kThreads, 2)
swska_fwd_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                    const __grid_constant__ CUtensorMap map_v, const SwTcArgs a) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* gen = smem_raw + (base - smem_u32(smem_raw));
  volatile SwCtl* ctl = reinterpret_cast<volatile SwCtl*>(gen + kOffCtl);
  auto bar = [&](int i) { return base + kOffCtl + 8u * (uint32_t)i; };
  float* sMax = reinterpret_cast<float*>(gen + kOffMax);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // Query tiles late in the sequence see the most keys.  CTAs are handed out in the order of
  // their index, so the index runs over the query tiles from the last one down and, within one
  // tile position, over all (batch, head): every long tile of the call starts before any short
  // one, and the short ones fill the tail.
  const int T = a.T, W = a.window;
  const int n_bh = a.B * a.H;
  const int m0 = (a.n_qtiles - 1 - (int)(blockIdx.x / (unsigned)n_bh)) * kBM;
  const long long bh = blockIdx.x % (unsigned)n_bh;
  const int b = (int)(bh / a.H);
  const long long qrow0 = bh * T + m0;           // row of the [B*H*T, 128] views of q, o
  const int krow0 = b * T;                       // row of the [B*T, 128] view of k
  const int vrow0 = (int)(bh * T);               // row of the [B*H*T, 128] view of v
  const int first_key = max(0, m0 - W + 1);
  const int nt_lo = first_key / kBN, nt_hi = min(m0 + kBM - 1, T - 1) / kBN;
  const int n_tiles = nt_hi - nt_lo + 1;

  if (tid == 0) {
    ctl->abort = 0;
    ctl->limit = a.limit;
    ctl->k_sent = ctl->v_sent = ctl->k_seen = ctl->v_seen = 0;
    for (int i = 0; i < kNumBars; ++i) {
      const bool per_warp = i == BAR_P0 || i == BAR_P1;
      const bool pair = i >= BAR_PAIR0 && i < BAR_PAIR0 + 4;
      mbar_init(bar(i), per_warp ? kSoftmaxWarps : (pair ? 2 : 1));
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kIssuerWarp) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(base + kOffCtl + (uint32_t)offsetof(SwCtl, tmem_base)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = ctl->tmem_base;

  if (warp == kProducerWarp) {
    // =========================== producer warp: every TMA load ================================
    if (lane == 0) {
      int k_sent = 0, v_sent = 0;
      auto load = [&](const CUtensorMap* map, uint32_t dst, uint32_t slab, int row, int which, uint32_t bytes) {
        mbar_expect_tx(bar(which), bytes);
        tma_load_2d(base + dst, map, 0, row, bar(which));
        tma_load_2d(base + dst + slab, map, 64, row, bar(which));
      };
      auto fill_k = [&](int j) {
        load(&map_k, kOffK + (j & 1) * kTileBytes, kSlabBytes, krow0 + (nt_lo + j) * kBN, BAR_K0 + (j & 1), kTileBytes);
        ++k_sent;
      };
      auto fill_v = [&](int j) {
        load(&map_v, kOffV + (j & 1) * kTileBytes, kSlabBytes, vrow0 + (nt_lo + j) * kBN, BAR_V0 + (j & 1), kTileBytes);
        ++v_sent;
      };
      load(&map_q, kOffQ, kQSlabBytes, (int)qrow0, BAR_Q, 2 * kQSlabBytes);
      fill_k(0);
      fill_v(0);
      if (n_tiles > 1) { fill_k(1); fill_v(1); }
      bool ok = true;
      // a slot is refilled as soon as the contraction that read it is complete: K two tiles ahead
      // of the scores that will read it, V two tiles ahead of its O += P V
      for (int it = 0; ok && it + 2 < n_tiles; ++it) {
        if (!(ok = sw_wait(bar(BAR_S0 + (it & 1)), (it >> 1) & 1, ctl, a.status))) break;
        fill_k(it + 2);
        if (!(ok = sw_wait(bar(BAR_O0 + (it & 1)), (it >> 1) & 1, ctl, a.status))) break;
        fill_v(it + 2);
      }
      ctl->k_sent = k_sent;
      ctl->v_sent = v_sent;
    }
    __syncwarp();
  } else if (warp == kIssuerWarp) {
    // =========================== issuing warp: every contraction ==============================
    if (lane == 0) {
      constexpr uint32_t kIdescS = make_idesc(kBM, kBN, 0, 0);   // S = Q K^T, both K-major
      constexpr uint32_t kIdescO = make_idesc(kBM, kD, 0, 1);    // O += P V: A in tensor memory, B N-major
      int k_seen = 0, v_seen = 0;
      auto issue_s = [&](int j) {   // scores of tile j into buffer j & 1
        const uint32_t dq0 = desc_lo_kmajor(base + kOffQ), dq1 = desc_lo_kmajor(base + kOffQ + kQSlabBytes);
        const uint32_t ks = base + kOffK + (j & 1) * kTileBytes;
        const uint32_t dk0 = desc_lo_kmajor(ks), dk1 = desc_lo_kmajor(ks + kSlabBytes);
        const uint32_t d = tmem + kColS + (j & 1) * kBN;
        umma_bf16_lo<false>(d, dq0, dk0, kIdescS);
#pragma unroll
        for (int kk = 1; kk < 4; ++kk) umma_bf16_lo<true>(d, dq0 + 2 * kk, dk0 + 2 * kk, kIdescS);
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) umma_bf16_lo<true>(d, dq1 + 2 * kk, dk1 + 2 * kk, kIdescS);
        umma_commit(bar(BAR_S0 + (j & 1)));
      };
      bool ok = sw_wait(bar(BAR_Q), 0, ctl, a.status);
      if (ok) { ok = sw_wait(bar(BAR_K0), 0, ctl, a.status); k_seen += ok; }
      if (ok) { tc_fence_after(); issue_s(0); }
      for (int it = 0; ok && it < n_tiles; ++it) {
        const int sb = it & 1;
        const uint32_t ph = (it >> 1) & 1;
        if (it + 1 < n_tiles) {            // the next tile's scores, while this tile's softmax runs
          ok = sw_wait(bar(BAR_K0 + (sb ^ 1)), ((it + 1) >> 1) & 1, ctl, a.status);
          k_seen += ok;
          if (!ok) break;
          tc_fence_after();
          issue_s(it + 1);
        }
        if (!(ok = sw_wait(bar(BAR_P0 + sb), ph, ctl, a.status))) break;   // probabilities in place
        ok = sw_wait(bar(BAR_V0 + sb), ph, ctl, a.status);
        v_seen += ok;
        if (!ok) break;
        tc_fence_after();
        const uint32_t dv = desc_lo_mnmajor(base + kOffV + sb * kTileBytes, kSlabBytes);
        const uint32_t pa = tmem + kColS + sb * kBN;
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
          if (kk == 0 && it == 0) umma_bf16_atmem<false>(tmem + kColO, pa, dv, kIdescO);
          else umma_bf16_atmem<true>(tmem + kColO, pa + 8 * kk, dv + 128 * kk, kIdescO);
        }
        umma_commit(bar(BAR_O0 + sb));   // (two barriers, by tile parity: a waiter is never two phases behind)
      }
      ctl->k_seen = k_seen;
      ctl->v_seen = v_seen;
    }
    __syncwarp();
  } else {
    // =========================== softmax warps =================================================
    // thread = (query row, half of a tile's 64 key columns): warps 0-3 the first half, warps 4-7
    // the second; a warp reaches the 32 tensor-memory lanes of its number mod 4
    const int rowl = tid & (kBM - 1), half = tid >> 7, col0 = half * kHalf;
    const int row = m0 + rowl;
    const uint32_t t_row = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    const uint32_t pair_bar = bar(BAR_PAIR0 + (warp & 3));   // this warp and the one with the other half
    const float sc = a.scale * kLog2e;        // > 0 (checked by the host)
    // Reference exponent of the row (log2 domain).  It follows the running maximum lazily: it
    // moves only when a tile's maximum exceeds it by more than 8, so probabilities stay below 2^8
    // and O, l are rescaled rarely; the final division by l makes the result independent of it.
    float m_ref = -INFINITY, l_run = 0.f;
    bool ok = true;
    int it = 0;
    // the two threads of a row exchange their maxima of a tile (both have then read S, which the
    // probabilities overwrite); the reference exponent follows; returns the factor for O and l
    auto exchange = [&](int sb, int it, float mx, float& alpha) -> bool {
      sMax[(sb * 2 + half) * kBM + rowl] = mx * sc;   // (-inf stays -inf: sc > 0)
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(pair_bar);
      bool good = sw_wait(pair_bar, it & 1, ctl, a.status);
      good = __all_sync(0xffffffffu, good);
      if (!good) return false;
      tc_fence_after();
      const float m_tile = fmaxf(sMax[(sb * 2) * kBM + rowl], sMax[(sb * 2 + 1) * kBM + rowl]);
      alpha = 1.f;
      if (m_tile > m_ref + 8.f) {               // also the first tile with a visible key
        alpha = ex2f(m_ref - m_tile);           // 0 when nothing had been seen
        m_ref = m_tile;
      }
      return true;
    };
    // rescaling O (rare) needs the previous O += P V complete; writing P does not
    auto rescale = [&](int it, float alpha) -> bool {
      if (it > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
        bool good = sw_wait(bar(BAR_O0 + ((it - 1) & 1)), ((it - 1) >> 1) & 1, ctl, a.status);
        good = __all_sync(0xffffffffu, good);
        if (!good) return false;
        tc_fence_after();
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          uint32_t r[32];
          tmem_ld32(t_row + kColO + 64 * half + 32 * c, r);
          tmem_ld_wait();
#pragma unroll
          for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * alpha);
          tmem_st32(t_row + kColO + 64 * half + 32 * c, r);
        }
      }
      return true;
    };
    auto publish = [&](int sb, const uint32_t (&pk)[kHalf / 2]) {
      tmem_st16(t_row + kColS + sb * kBN + 16 * half, pk);     // keys col0 .. col0+31, two per column
      tmem_st_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(BAR_P0 + sb));
    };
    for (; it < n_tiles; ++it) {
      const int sb = it & 1;
      const uint32_t ph = (it >> 1) & 1;
      const int n0 = (nt_lo + it) * kBN;
      ok = sw_wait(bar(BAR_S0 + sb), ph, ctl, a.status);
      ok = __all_sync(0xffffffffu, ok);     // the tensor-memory accesses below need the whole warp
      if (!ok) break;
      tc_fence_after();
      // the visible keys of this thread's 32 are e_lo .. e_hi (none when e_lo > e_hi)
      const int k0 = n0 + col0;
      const int e_lo = max(0, row - W + 1 - k0), e_hi = min(kHalf - 1, row - k0);
      if (__all_sync(0xffffffffu, e_lo > e_hi)) {
        // on the diagonal and at the window's far edge whole warps see no key of a tile: they
        // take part in the hand-offs and write zeros, without the arithmetic
        float alpha;
        if (!(ok = exchange(sb, it, -INFINITY, alpha))) break;
        l_run *= alpha;
        if (!(ok = rescale(it, alpha))) break;
        uint32_t pk[kHalf / 2];
#pragma unroll
        for (int e = 0; e < kHalf / 2; ++e) pk[e] = 0u;
        publish(sb, pk);
        continue;
      }
      // ---- this thread's 32 columns of its row of S: mask, maximum
      float sv[kHalf];
      float mx;
      {
        uint32_t r[32];
        tmem_ld32(t_row + kColS + sb * kBN + col0, r);
        tmem_ld_wait();
        if (e_lo == 0 && e_hi == kHalf - 1) {
#pragma unroll
          for (int e = 0; e < kHalf; ++e) sv[e] = __uint_as_float(r[e]);
        } else {
          const uint32_t bits = e_lo > e_hi ? 0u : ((0xffffffffu >> (kHalf - 1 - e_hi)) & (0xffffffffu << e_lo));
#pragma unroll
          for (int e = 0; e < kHalf; ++e) sv[e] = ((bits >> e) & 1u) ? __uint_as_float(r[e]) : -INFINITY;
        }
        // maximum as a tree: four independent chains of three-input steps over eight values each
        float m4[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const float* s8 = sv + 8 * c;
          m4[c] = fmaxf(max3(max3(max3(s8[0], s8[1], s8[2]), s8[3], s8[4]), s8[5], s8[6]), s8[7]);
        }
        mx = fmaxf(max3(m4[0], m4[1], m4[2]), m4[3]);
      }
      float alpha;
      if (!(ok = exchange(sb, it, mx, alpha))) break;
      const float m_use = m_ref == -INFINITY ? 0.f : m_ref;
      uint64_t ps[4] = {0ull, 0ull, 0ull, 0ull};     // four pairs of partial sums: short dependent chains
      uint32_t pk[kHalf / 2];
      const uint64_t sc2 = pair_f32(sc, sc), nm2 = pair_f32(-m_use, -m_use);
#pragma unroll
      for (int e = 0; e < kHalf; e += 2) {
        float x0, x1;
        unpair_f32(fma2(pair_f32(sv[e], sv[e + 1]), sc2, nm2), x0, x1);
        const float p0 = ex2f(x0), p1 = ex2f(x1);
        ps[(e >> 1) & 3] = add2(ps[(e >> 1) & 3], pair_f32(p0, p1));
        pk[e >> 1] = pack_bf16(p0, p1);
      }
      {
        float s0, s1;
        unpair_f32(add2(add2(ps[0], ps[1]), add2(ps[2], ps[3])), s0, s1);
        l_run = l_run * alpha + (s0 + s1);
      }
      if (!(ok = rescale(it, alpha))) break;
      publish(sb, pk);
    }
    // ---- the last O += P V, then normalise and store this thread's 64 columns of its row
    if (ok) ok = sw_wait(bar(BAR_O0 + ((n_tiles - 1) & 1)), ((n_tiles - 1) >> 1) & 1, ctl, a.status);
    ok = __all_sync(0xffffffffu, ok);
    if (ok) {
      tc_fence_after();
      sMax[half * kBM + rowl] = l_run;
      __syncwarp();
      if (lane == 0) mbar_arrive(pair_bar);
      ok = sw_wait(pair_bar, n_tiles & 1, ctl, a.status);
      ok = __all_sync(0xffffffffu, ok);
    }
    if (ok) {
      const float l = sMax[rowl] + sMax[kBM + rowl];
      const float inv = l > 0.f ? 1.f / l : 0.f;
      __nv_bfloat16* orow = (__nv_bfloat16*)a.o + (qrow0 + rowl) * kD + 64 * half;
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        uint32_t r[32];
        tmem_ld32(t_row + kColO + 64 * half + 32 * c, r);
        tmem_ld_wait();
        if (row < T) {
#pragma unroll
          for (int e = 0; e < 32; e += 8) {
            uint4 w;
            w.x = pack_bf16(__uint_as_float(r[e]) * inv, __uint_as_float(r[e + 1]) * inv);
            w.y = pack_bf16(__uint_as_float(r[e + 2]) * inv, __uint_as_float(r[e + 3]) * inv);
            w.z = pack_bf16(__uint_as_float(r[e + 4]) * inv, __uint_as_float(r[e + 5]) * inv);
            w.w = pack_bf16(__uint_as_float(r[e + 6]) * inv, __uint_as_float(r[e + 7]) * inv);
            *reinterpret_cast<uint4*>(orow + 32 * c + e) = w;
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (ctl->abort) {   // clean exit: nothing may still be writing this CTA's shared or tensor memory
    if (tid == 0) {
      mbar_drain(bar(BAR_Q), 0);
      for (int j = ctl->k_seen; j < ctl->k_sent; ++j) mbar_drain(bar(BAR_K0 + (j & 1)), (j >> 1) & 1);
      for (int j = ctl->v_seen; j < ctl->v_sent; ++j) mbar_drain(bar(BAR_V0 + (j & 1)), (j >> 1) & 1);
    }
    if (warp == kIssuerWarp && lane == 0) {   // (a commit follows the contractions of the thread that makes it)
      umma_commit(bar(BAR_DRAIN));            // completes when every contraction issued so far has
      mbar_drain(bar(BAR_DRAIN), 0);
    }
  }
  __syncthreads();
  if (warp == kIssuerWarp)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn sw_encode_fn() {
  static const EncodeTiledFn fn = []() -> EncodeTiledFn {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess) {
      cudaGetLastError();
      return nullptr;
    }
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

// [rows, 128] bf16 row-major; box = box_rows rows x 64 columns (128 bytes), 128-byte swizzle; rows
// past the end of the tensor read as zeros
bool sw_make_map(CUtensorMap* m, const void* ptr, uint64_t rows, uint32_t box_rows) {
  EncodeTiledFn fn = sw_encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)kD, rows};
  const cuuint64_t strides[1] = {(cuuint64_t)kD * 2};
  const cuuint32_t box[2] = {64u, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct SwMapCache {     // the three maps of the last call on this host thread
  const void *q = nullptr, *k = nullptr, *v = nullptr;
  uint64_t rows_q = 0, rows_k = 0;
  CUtensorMap mq, mk, mv;
};
thread_local SwMapCache t_sw_maps;
std::atomic<unsigned long long> g_sw_tc_smem_done{0};

}  // namespace

cudaError_t launch_swska_tc(const rodimus_swska_fwd_params& p, int* n_launches) {
  *n_launches = 0;
  const uint64_t rows_q = (uint64_t)p.B * p.H * p.T, rows_k = (uint64_t)p.B * p.T;
  SwMapCache& c = t_sw_maps;
  if (c.q != p.q || c.k != p.k || c.v != p.v || c.rows_q != rows_q || c.rows_k != rows_k) {
    if (!sw_make_map(&c.mq, p.q, rows_q, kBM) || !sw_make_map(&c.mk, p.k, rows_k, kBN) ||
        !sw_make_map(&c.mv, p.v, rows_q, kBN)) {
      c.q = nullptr;
      return cudaErrorInvalidValue;
    }
    c.q = p.q; c.k = p.k; c.v = p.v; c.rows_q = rows_q; c.rows_k = rows_k;
  }
  int dev = 0, sms = 0;
  cudaError_t e = current_device(&dev, &sms);
  if (e != cudaSuccess) return e;
  e = opt_in_shared_memory(swska_fwd_tc_kernel, (int)kSmemBytes, dev, g_sw_tc_smem_done);
  if (e != cudaSuccess) return e;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(p.stream);
  SwTcArgs a;
  a.o = p.o;
  a.status = reinterpret_cast<int32_t*>(p.workspace);
  a.B = p.B; a.H = p.H; a.T = p.T; a.window = p.window; a.scale = p.scale;
  a.n_qtiles = (p.T + kBM - 1) / kBM;
  const long long n_ctas = (long long)a.n_qtiles * p.B * p.H;
  if (n_ctas > 0x7fffffffLL) return cudaErrorInvalidValue;
  a.limit = main_loop_wait_cycles();
  if (a.status) {
    e = cudaMemsetAsync(a.status, 0, sizeof(int32_t), st);
    if (e != cudaSuccess) return e;
  }
  const dim3 grid((unsigned)n_ctas);
  swska_fwd_tc_kernel<<<grid, kThreads, kSmemBytes, st>>>(c.mq, c.mk, c.mv, a);
  *n_launches = 1;
  return cudaGetLastError();
}

}  // namespace ddts
