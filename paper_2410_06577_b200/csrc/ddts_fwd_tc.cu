// Chunked DDTS prefill on the 5th-generation tensor cores (tcgen05 + TMEM + TMA), bf16 inputs,
// dk = 128, 128 state columns per CTA.
//
// Chunkwise form (appendix "Chunkwise Parallel Representation of the Rodimus Block"), chunk
// length C = 64, all decays handled in the log2 domain and anchored at the chunk start:
//   b_r      = sum_{j<=r in chunk} log2 alpha_j                       (per key channel, <= 0)
//   Qt_r     = q_r . 2^{b_r}                                          bf16, K-major operand
//   Kt_i     = k_i . ahat_i . 2^{-b_i}                                bf16, K-major operand
//   Ke_i     = k_i . ahat_i . 2^{b_C - b_i}                           bf16, MN-major operand
//   P        = (Qt Kt^T) masked to i <= r                             [C,C]   fp32 in TMEM
//   O        = P V + Qt S_in            (S_in = state ENTERING the chunk) [C,128] fp32 in TMEM
//   S_out    = diag(2^{b_C}) S_in + Ke^T V                            [128,128] fp32 in TMEM
// The fp32 state never leaves TMEM between chunks; once per chunk it makes one trip through
// registers to be scaled by the chunk's total decay and copied, as bf16, to shared memory where
// the readout contraction can take it as an operand.
//
// One CTA = 20 warps with fixed roles, connected by mbarriers (every wait is bounded):
//   warp 0        TMA producer: q,k,x,y,v tiles of the next chunk into a 2-stage ring
//   warp 1        tcgen05.mma issuer (one elected lane), owns the TMEM allocation
//   warps 4-7     state group: TMEM <-> registers trip of S, initial/final state I/O
//   warps 8-11    score/output group: P -> masked bf16 operand, O -> global memory
//   warps 12-19   gate group: softplus/sigmoid/log/exp2 math, in-chunk scan, operand tiles
//                 written IN PLACE over the raw q,k,x tiles (same swizzled layout)
// Work item = (sequence, head, 128-column slice of dv), dealt round-robin to a persistent grid.
#include <cuda.h>

#include <cstring>

#include "ddts_common.cuh"
#include "ddts_tc_ptx.cuh"

namespace ddts {
namespace {

constexpr int kC = 64;                       // chunk rows
constexpr int kDK = 128;                     // key channels
constexpr int kDVS = 128;                    // value columns per CTA
constexpr int kStages = 2;
constexpr int kSlabBytes = kC * 128;         // [64 rows][64 bf16] = 8 KiB, 128-byte swizzled
constexpr int kTileBytes = 2 * kSlabBytes;   // [64][128] bf16 as two slabs
constexpr int kStageBytes = 5 * kTileBytes;  // q, k, x, y, v
constexpr int kOffQ = 0, kOffK = kTileBytes, kOffX = 2 * kTileBytes, kOffY = 3 * kTileBytes,
              kOffV = 4 * kTileBytes;
constexpr int kSsSlabBytes = kDK * 128;      // [128 rows][64 bf16]
constexpr int kOffSs = kStages * kStageBytes;            // bf16 copy of the state, 2 slabs
constexpr int kOffD = kOffSs + 2 * kSsSlabBytes;         // float [kStages][128]: 2^{b_C}
constexpr int kOffTot = kOffD + kStages * kDK * 4;       // float [2][8][64]: scan partials
constexpr int kOffBar = kOffTot + 2 * 8 * 64 * 4;        // mbarriers
constexpr int kNumBars = 16;
constexpr int kOffMisc = kOffBar + kNumBars * 8;         // control block
constexpr int kSmemUsed = kOffMisc + 256;
constexpr int kSmemBytes = kSmemUsed + 1024;             // slack for manual 1024-byte alignment

constexpr int kThreads = 640;
constexpr int kGateWarp0 = 12, kGateWarps = 8;

// TMEM columns (fp32 words): state, output, scores
constexpr uint32_t kColS = 0, kColO = 128, kColP = 256, kTmemCols = 512;

// mbarrier indices
enum { BAR_FULL0 = 0, BAR_FULL1, BAR_EMPTY0, BAR_EMPTY1, BAR_GATED0, BAR_GATED1, BAR_PFULL,
       BAR_PREADY, BAR_SREADY, BAR_SFULL, BAR_OFULL, BAR_OFREE, BAR_GSCAN,
       BAR_DRAIN };   // teardown after a timeout: issued contractions are done


struct TcArgs {
  void* o;
  const float* s0;
  float* sT;
  const int32_t* cu;
  const int32_t* order;
  WorkspaceHeader* hdr;
  int H, T, dv, n_seq, slices;
  long long n_items;
  float scale;
  long long wait_cycles;   // limit of one main-loop wait (clock cycles)
};

struct Item {
  long long row0;      // first global row (in the [rows, d] view) of this sequence and head
  long long state_off; // element offset of this (sequence, head) state slice start (column 0)
  int len;             // tokens
  int col0;            // first value column of the slice
};

__device__ __forceinline__ Item decode_item(const TcArgs& a, long long item) {
  Item it;
  const int slice = (int)(item % a.slices);
  const long long sh = item / a.slices;
  const int h = (int)(sh % a.H);
  long long n = sh / a.H;
  if (a.cu) {
    n = a.order[n];
    int lo = a.cu[n], hi = a.cu[n + 1];
    lo = lo < 0 ? 0 : (lo > a.T ? a.T : lo);
    hi = hi < lo ? lo : (hi > a.T ? a.T : hi);
    it.row0 = (long long)h * a.T + lo;
    it.len = hi - lo;
  } else {
    it.row0 = (n * a.H + h) * (long long)a.T;
    it.len = a.T;
  }
  it.col0 = slice * kDVS;
  it.state_off = (n * a.H + h) * (long long)kDK * a.dv + it.col0;
  return it;
}

// ---------------------------------------------------------------------------------------------
// kernel
// ---------------------------------------------------------------------------------------------
// A "fill" is one 64-row tile of q,k,x,y,v brought into a stage by the producer; a "pass" is a
// fill the gate group accepted and turned into operands.  The two differ because the chunk
// length adapts to the data: the anchored factorisation Qt = q 2^{b}, Kt = k ahat 2^{-b} needs
// the in-chunk decay range max_d(-b_C) to stay below kRange, so when a tile decays faster than
// that the gate group asks for the same position again with fewer live rows (halving, then
// doubling back), and the producer, which prefetches speculatively at a stride of 64 rows, is
// redirected.  Every fill carries the (item, position) it was issued for; fills that no longer
// match what the gate group expects are released unused.
struct PassDesc {
  int stage;      // which stage holds the operands
  int nr;         // live rows
  int flags;      // kPassFirst | kPassLast
  int pad;
  long long row;  // global row (in the [rows, d] view) of the pass's first token
};
constexpr int kPassFirst = 1, kPassLast = 2;

struct Control {            // lives in shared memory
  uint32_t tmem_base;
  int done;                 // gate group has finished every item of this CTA
  WaitCtl wait;             // abort flag and limit shared by every bounded wait of the CTA
  int redir_seq;            // bumped by the gate group after writing redir_j / redir_tpos
  int redir_j, redir_tpos;  // where the producer must continue (CTA-local item index, token)
  int pad[2];
  int tag[2][2];            // per stage: (item index, token position) of the fill it holds
  int pad2[4];
  PassDesc pd[4];
};
static_assert(sizeof(Control) <= 256, "control block");

template <int INGATE>
__global__ void __launch_bounds__(kThreads, 1)
ddts_fwd_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                   const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_y,
                   const __grid_constant__ CUtensorMap map_v, const TcArgs a) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gbase = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bars = base + kOffBar;
  auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
  volatile Control* ctl = reinterpret_cast<volatile Control*>(gbase + kOffMisc);
  volatile WaitCtl* abort_flag = &ctl->wait;
  float* sD = reinterpret_cast<float*>(gbase + kOffD);
  float* sTot = reinterpret_cast<float*>(gbase + kOffTot);

  const int tid = threadIdx.x;
  const int warp = tid >> 5, lane = tid & 31;

  if (!a.cu && blockIdx.x == 0 && tid == 0) a.hdr->status = RODIMUS_OK;

  if (tid == 0) {
    ctl->wait.abort_flag = 0;
    ctl->wait.limit = a.wait_cycles;
    ctl->done = 0;
    ctl->redir_seq = 0;
    mbar_init(bar(BAR_FULL0), 1);
    mbar_init(bar(BAR_FULL1), 1);
    mbar_init(bar(BAR_EMPTY0), 1);
    mbar_init(bar(BAR_EMPTY1), 1);
    mbar_init(bar(BAR_GATED0), kGateWarps);
    mbar_init(bar(BAR_GATED1), kGateWarps);
    mbar_init(bar(BAR_PFULL), 1);
    mbar_init(bar(BAR_PREADY), 128);
    mbar_init(bar(BAR_SREADY), 128);
    mbar_init(bar(BAR_SFULL), 1);
    mbar_init(bar(BAR_OFULL), 1);
    mbar_init(bar(BAR_OFREE), 128);
    mbar_init(bar(BAR_GSCAN), kGateWarps);
    mbar_init(bar(BAR_DRAIN), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(base + kOffMisc), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = ctl->tmem_base;
  auto item_of = [&](int j) { return (long long)blockIdx.x + (long long)j * gridDim.x; };

  if (warp == 0) {
    // ===================================== TMA producer =====================================
    if (lane == 0) {
      uint32_t f = 0;         // fills issued
      int j = 0, tpos = 0;    // speculative position: item index and token
      int seen = 0;           // last redirect taken
      bool ok = true;
      while (ok) {
        const uint32_t s = f & 1, ph = (f >> 1) & 1;
        if (!(ok = mbar_wait(bar(BAR_EMPTY0 + s), ph ^ 1, abort_flag, a.hdr))) break;
        Item it;
        bool have = false;
        const long long t0 = clock64();
        while (true) {
          const int sq = ctl->redir_seq;
          if (sq != seen) {
            __threadfence_block();
            j = ctl->redir_j;
            tpos = ctl->redir_tpos;
            seen = sq;
          }
          while (item_of(j) < a.n_items) {   // next position that has tokens left
            it = decode_item(a, item_of(j));
            if (tpos < it.len) { have = true; break; }
            ++j;
            tpos = 0;
          }
          if (have || ctl->done || abort_flag->abort_flag) break;
          if (clock64() - t0 >= abort_flag->limit) {
            abort_flag->abort_flag = 1;
            atomicMax(&a.hdr->status, (int)RODIMUS_ERR_TIMEOUT);
            break;
          }
          __nanosleep(100);
        }
        if (!have) break;
        ctl->tag[s][0] = j;
        ctl->tag[s][1] = tpos;
        const uint32_t st = base + s * kStageBytes;
        const uint32_t fb = bar(BAR_FULL0 + s);
        mbar_expect_tx(fb, kStageBytes);
        // rows beyond the tensor read as zeros; rows of the next sequence are masked later
        const int y = (int)(it.row0 + tpos);
        tma_load_2d(st + kOffQ, &map_q, 0, y, fb);
        tma_load_2d(st + kOffQ + kSlabBytes, &map_q, 64, y, fb);
        tma_load_2d(st + kOffK, &map_k, 0, y, fb);
        tma_load_2d(st + kOffK + kSlabBytes, &map_k, 64, y, fb);
        tma_load_2d(st + kOffX, &map_x, 0, y, fb);
        tma_load_2d(st + kOffX + kSlabBytes, &map_x, 64, y, fb);
        tma_load_2d(st + kOffY, &map_y, 0, y, fb);
        tma_load_2d(st + kOffY + kSlabBytes, &map_y, 64, y, fb);
        tma_load_2d(st + kOffV, &map_v, it.col0, y, fb);
        tma_load_2d(st + kOffV + kSlabBytes, &map_v, it.col0 + 64, y, fb);
        ++f;
        tpos += kC;
      }
      // Leave no bulk copy in flight when the CTA exits: the last two fills' barriers complete
      // by byte count, whoever consumed them.
      for (uint32_t back = 1; back <= 2 && back <= f; ++back) {
        const uint32_t ff = f - back;
        mbar_drain(bar(BAR_FULL0 + (ff & 1)), (ff >> 1) & 1);
      }
    }
  } else if (warp == 1) {
    // ====================================== MMA issuer ======================================
    if (lane == 0) {
      constexpr uint32_t kIdescP = make_idesc(64, 64, 0, 0);
      constexpr uint32_t kIdescO = make_idesc(64, kDVS, 0, 1);
      constexpr uint32_t kIdescS = make_idesc(128, kDVS, 1, 1);
      const uint32_t ss = base + kOffSs;
      uint32_t g = 0;
      bool ok = true;
      for (int j = 0; ok && item_of(j) < a.n_items; ++j) {
        const Item it = decode_item(a, item_of(j));
        if (it.len == 0) continue;
        bool last = false;
        while (!last) {
          const uint32_t ph1 = g & 1;
          if (!(ok = mbar_wait(bar(BAR_GATED0 + (g & 1)), (g >> 1) & 1, abort_flag, a.hdr))) break;
          const uint32_t s = (uint32_t)ctl->pd[g & 3].stage;
          last = (ctl->pd[g & 3].flags & kPassLast) != 0;
          const uint32_t st = base + s * kStageBytes;
          tc_fence_after();
          // P = Qt Kt^T : M = 64 (rows r), N = 64 (rows i), K = 128 channels
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) {
            const uint32_t off = (kk >> 2) * kSlabBytes + (kk & 3) * 32;
            umma_bf16(tmem + kColP, desc_kmajor(st + kOffQ + off), desc_kmajor(st + kOffK + off),
                      kIdescP, kk > 0);
          }
          umma_commit(bar(BAR_PFULL));
          if (!(ok = mbar_wait(bar(BAR_PREADY), ph1, abort_flag, a.hdr))) break;
          if (!(ok = mbar_wait(bar(BAR_SREADY), ph1, abort_flag, a.hdr))) break;
          if (!(ok = mbar_wait(bar(BAR_OFREE), ph1 ^ 1, abort_flag, a.hdr))) break;
          tc_fence_after();
          // O = P V : M = 64, N = 128, K = 64 rows i (P operand lives in the consumed y tile)
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {
            umma_bf16(tmem + kColO, desc_kmajor(st + kOffY + kk * 32),
                      desc_mnmajor(st + kOffV + kk * 2048, kSlabBytes), kIdescO, kk > 0);
          }
          // O += Qt S_in : K = 128 channels
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) {
            const uint32_t off = (kk >> 2) * kSlabBytes + (kk & 3) * 32;
            umma_bf16(tmem + kColO, desc_kmajor(st + kOffQ + off),
                      desc_mnmajor(ss + kk * 2048, kSsSlabBytes), kIdescO, 1);
          }
          umma_commit(bar(BAR_OFULL));
          // S = diag(D) S_in (already in TMEM) + Ke^T V : M = 128 channels, N = 128, K = 64 rows
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {
            umma_bf16(tmem + kColS, desc_mnmajor(st + kOffX + kk * 2048, kSlabBytes),
                      desc_mnmajor(st + kOffV + kk * 2048, kSlabBytes), kIdescS, 1);
          }
          umma_commit(bar(BAR_SFULL));
          umma_commit(bar(BAR_EMPTY0 + s));
          ++g;
        }
      }
    }
  } else if (warp >= 4 && warp < 8) {
    // ====================================== state group ======================================
    const int q4 = warp & 3;
    const int d = q4 * 32 + lane;                         // state row (key channel) of this thread
    const uint32_t t_lane = tmem + ((uint32_t)(q4 * 32) << 16);
    const uint32_t ss_row = base + kOffSs + d * 128;
    uint32_t g = 0;
    bool ok = true;
    for (int j = 0; ok && item_of(j) < a.n_items; ++j) {
      const Item it = decode_item(a, item_of(j));
      const long long srow = it.state_off + (long long)d * a.dv;
      if (it.len == 0) {  // empty sequence: final state = initial state
        if (a.sT) {
          for (int c4 = 0; c4 < kDVS / 4; ++c4) {
            float4 v4 = a.s0 ? *reinterpret_cast<const float4*>(a.s0 + srow + 4 * c4)
                             : make_float4(0.f, 0.f, 0.f, 0.f);
            *reinterpret_cast<float4*>(a.sT + srow + 4 * c4) = v4;
          }
        }
        continue;
      }
      bool last = false, first = true;
      while (!last) {
        const uint32_t ph1 = g & 1;
        if (!first) {
          if (!(ok = mbar_wait(bar(BAR_SFULL), ph1 ^ 1, abort_flag, a.hdr))) break;  // pass g-1
          tc_fence_after();
        }
        if (!(ok = mbar_wait(bar(BAR_GATED0 + (g & 1)), (g >> 1) & 1, abort_flag, a.hdr))) break;
        const int s = ctl->pd[g & 3].stage;
        last = (ctl->pd[g & 3].flags & kPassLast) != 0;
        const float D = sD[s * kDK + d];
#pragma unroll 1
        for (int piece = 0; piece < 4; ++piece) {
          uint32_t r[32];
          if (!first) {
            tmem_ld32(t_lane + kColS + piece * 32, r);
            tmem_ld_wait();
          } else if (a.s0) {
#pragma unroll
            for (int c4 = 0; c4 < 8; ++c4) {
              const float4 v4 = *reinterpret_cast<const float4*>(a.s0 + srow + piece * 32 + 4 * c4);
              r[4 * c4] = __float_as_uint(v4.x);
              r[4 * c4 + 1] = __float_as_uint(v4.y);
              r[4 * c4 + 2] = __float_as_uint(v4.z);
              r[4 * c4 + 3] = __float_as_uint(v4.w);
            }
          } else {
#pragma unroll
            for (int c4 = 0; c4 < 32; ++c4) r[c4] = 0u;
          }
          // bf16 copy of S_in for the readout: MN-major, row d, 64-column slab piece/2
          const uint32_t slab = ss_row + (piece >> 1) * kSsSlabBytes;
#pragma unroll
          for (int c8 = 0; c8 < 4; ++c8) {
            const int chunk = (piece & 1) * 4 + c8;
            sts128(slab + ((chunk ^ (d & 7)) << 4),
                   pack_bf16(__uint_as_float(r[8 * c8]), __uint_as_float(r[8 * c8 + 1])),
                   pack_bf16(__uint_as_float(r[8 * c8 + 2]), __uint_as_float(r[8 * c8 + 3])),
                   pack_bf16(__uint_as_float(r[8 * c8 + 4]), __uint_as_float(r[8 * c8 + 5])),
                   pack_bf16(__uint_as_float(r[8 * c8 + 6]), __uint_as_float(r[8 * c8 + 7])));
          }
#pragma unroll
          for (int c4 = 0; c4 < 32; ++c4) r[c4] = __float_as_uint(__uint_as_float(r[c4]) * D);
          tmem_st32(t_lane + kColS + piece * 32, r);
        }
        tmem_st_wait();
        fence_proxy_async();
        tc_fence_before();
        mbar_arrive(bar(BAR_SREADY));
        first = false;
        ++g;
      }
      if (!ok) break;
      // final state of this item (also keeps the next item's initial state from racing the MMAs)
      {
        const uint32_t lastg = g - 1;
        if (!(ok = mbar_wait(bar(BAR_SFULL), lastg & 1, abort_flag, a.hdr))) break;
        tc_fence_after();
        if (a.sT) {
#pragma unroll 1
          for (int piece = 0; piece < 4; ++piece) {
            uint32_t r[32];
            tmem_ld32(t_lane + kColS + piece * 32, r);
            tmem_ld_wait();
#pragma unroll
            for (int c4 = 0; c4 < 8; ++c4) {
              *reinterpret_cast<float4*>(a.sT + srow + piece * 32 + 4 * c4) =
                  make_float4(__uint_as_float(r[4 * c4]), __uint_as_float(r[4 * c4 + 1]),
                              __uint_as_float(r[4 * c4 + 2]), __uint_as_float(r[4 * c4 + 3]));
            }
          }
        }
        tc_fence_before();
      }
    }
  } else if (warp >= 8 && warp < 12) {
    // ================================== score / output group ==================================
    const int q4 = warp & 3;
    const int r_row = q4 * 16 + lane;                     // chunk row held by lanes 0..15 (M = 64)
    const bool has_row = lane < 16;
    const uint32_t t_lane = tmem + ((uint32_t)(q4 * 32) << 16);
    __nv_bfloat16* o = reinterpret_cast<__nv_bfloat16*>(a.o);
    uint32_t g = 0;
    bool ok = true;
    for (int j = 0; ok && item_of(j) < a.n_items; ++j) {
      const Item it = decode_item(a, item_of(j));
      if (it.len == 0) continue;
      bool last = false;
      while (!last) {
        const uint32_t ph1 = g & 1;
        if (!(ok = mbar_wait(bar(BAR_PFULL), ph1, abort_flag, a.hdr))) break;
        const int s = ctl->pd[g & 3].stage;
        const int nr = ctl->pd[g & 3].nr;
        const long long row = ctl->pd[g & 3].row;
        last = (ctl->pd[g & 3].flags & kPassLast) != 0;
        const uint32_t ps_row = base + s * kStageBytes + kOffY + r_row * 128;
        tc_fence_after();
#pragma unroll 1
        for (int half = 0; half < 2; ++half) {
          uint32_t r[32];
          tmem_ld32(t_lane + kColP + half * 32, r);
          tmem_ld_wait();
          if (has_row) {
#pragma unroll
            for (int c8 = 0; c8 < 4; ++c8) {
              uint32_t w[4];
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const int i0 = half * 32 + 8 * c8 + 2 * e;
                const float lo = (i0 <= r_row) ? __uint_as_float(r[8 * c8 + 2 * e]) : 0.f;
                const float hi = (i0 + 1 <= r_row) ? __uint_as_float(r[8 * c8 + 2 * e + 1]) : 0.f;
                w[e] = pack_bf16(lo, hi);
              }
              const int chunk = half * 4 + c8;
              sts128(ps_row + ((chunk ^ (r_row & 7)) << 4), w[0], w[1], w[2], w[3]);
            }
          }
        }
        fence_proxy_async();
        tc_fence_before();
        mbar_arrive(bar(BAR_PREADY));
        // output rows of this pass
        if (!(ok = mbar_wait(bar(BAR_OFULL), ph1, abort_flag, a.hdr))) break;
        tc_fence_after();
        __nv_bfloat16* orow = o + (row + r_row) * a.dv + it.col0;
#pragma unroll 1
        for (int piece = 0; piece < 4; ++piece) {
          uint32_t r[32];
          tmem_ld32(t_lane + kColO + piece * 32, r);
          tmem_ld_wait();
          if (has_row && r_row < nr) {
#pragma unroll
            for (int c8 = 0; c8 < 4; ++c8) {
              uint4 w;
              w.x = pack_bf16(a.scale * __uint_as_float(r[8 * c8]), a.scale * __uint_as_float(r[8 * c8 + 1]));
              w.y = pack_bf16(a.scale * __uint_as_float(r[8 * c8 + 2]), a.scale * __uint_as_float(r[8 * c8 + 3]));
              w.z = pack_bf16(a.scale * __uint_as_float(r[8 * c8 + 4]), a.scale * __uint_as_float(r[8 * c8 + 5]));
              w.w = pack_bf16(a.scale * __uint_as_float(r[8 * c8 + 6]), a.scale * __uint_as_float(r[8 * c8 + 7]));
              *reinterpret_cast<uint4*>(orow + piece * 32 + 8 * c8) = w;
            }
          }
        }
        tc_fence_before();
        mbar_arrive(bar(BAR_OFREE));
        ++g;
      }
    }
  } else if (warp >= kGateWarp0) {
    // ======================================= gate group =======================================
    const int gw = warp - kGateWarp0;                     // rows 8*gw .. 8*gw+7 of the tile
    constexpr float kLog2e = 1.4426950408889634f;
    constexpr float kLg2Ln2 = -0.5287663729448977f;       // log2(ln 2)
    constexpr float kRange = 60.f * kLog2e;               // largest in-chunk decay range, log2 units
    uint32_t f = 0, g = 0, sc = 0;                        // fills seen, passes published, scan syncs
    bool ok = true;
    auto group_sync = [&]() -> bool {                     // bounded barrier over the 8 gate warps
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(BAR_GSCAN));
      const bool r = mbar_wait(bar(BAR_GSCAN), sc & 1, abort_flag, a.hdr);
      ++sc;
      return r;
    };
    auto redirect = [&](int jj, int tt) {                 // one thread; before the stage is released
      ctl->redir_j = jj;
      ctl->redir_tpos = tt;
      __threadfence_block();
      ctl->redir_seq = ctl->redir_seq + 1;
    };
    for (int j = 0; ok && item_of(j) < a.n_items; ++j) {
      const Item it = decode_item(a, item_of(j));
      int tpos = 0, lcap = kC;
      bool first = true;
      while (ok && tpos < it.len) {
        const uint32_t s = f & 1, ph = (f >> 1) & 1;
        const uint32_t st = base + s * kStageBytes;
        if (!(ok = mbar_wait(bar(BAR_FULL0 + s), ph, abort_flag, a.hdr))) break;
        ++f;
        if (ctl->tag[s][0] != j || ctl->tag[s][1] != tpos) {
          // speculative fill for a position we are not at: hand the stage back unused
          if (!(ok = group_sync())) break;
          if (gw == 0 && lane == 0) mbar_arrive(bar(BAR_EMPTY0 + s));
          continue;
        }
        const int left = it.len - tpos;
        const int nr = min(min(kC, left), lcap);
        bool viol = false;
#pragma unroll 1
        for (int sl = 0; sl < 2; ++sl) {
          // element (row r, channels 64*sl + 2*lane, +1) sits at this swizzled byte offset
          const uint32_t slab = st + sl * kSlabBytes;
          float bq[8][2];   // inclusive in-chunk cumulative log2 decay (own rows only, so far)
          float eh[8][2];   // log2 ahat
          float run0 = 0.f, run1 = 0.f;
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const int r = gw * 8 + i;
            const uint32_t off = r * 128 + ((((uint32_t)lane >> 2) ^ (r & 7)) << 4) + ((lane & 3) << 2);
            const uint32_t xw = lds32(slab + kOffX + off), yw = lds32(slab + kOffY + off);
            const float xs[2] = {__uint_as_float(xw << 16), __uint_as_float(xw & 0xFFFF0000u)};
            const float ys[2] = {__uint_as_float(yw << 16), __uint_as_float(yw & 0xFFFF0000u)};
#pragma unroll
            for (int e = 0; e < 2; ++e) {
              const float u = ex2f(xs[e] * kLog2e);                       // e^x
              // g * log2(e) = log2(1 + e^x); series when 1 + u would round u away
              const float sp2 = u < 9.765625e-4f ? u * (kLog2e - 0.72134752f * u) : lg2f(1.f + u);
              const float tau = rcpf(1.f + ex2f(-ys[e] * kLog2e));
              float l2a = fmaxf(-sp2 * tau, -kRange);                     // per-step floor exp(-60)
              float l2h;
              if (INGATE == RODIMUS_INGATE_POW_G) {
                l2h = tau * (lg2f(sp2) + kLg2Ln2);                        // tau * log2(g)
              } else {
                l2h = tau * (xs[e] * kLog2e - sp2);                       // tau * log2(sigmoid(x))
              }
              if (r >= nr) l2a = 0.f;                                     // rows past the pass
              if (e == 0) { run0 += l2a; bq[i][0] = run0; } else { run1 += l2a; bq[i][1] = run1; }
              eh[i][e] = l2h;
            }
          }
          // exclusive prefix over the 8 row groups, and the chunk total
          float* tot = sTot + sl * (8 * 64);
          *reinterpret_cast<float2*>(tot + gw * 64 + 2 * lane) = make_float2(run0, run1);
          if (!(ok = group_sync())) break;
          float pre0 = 0.f, pre1 = 0.f, all0 = 0.f, all1 = 0.f;
#pragma unroll
          for (int w = 0; w < 8; ++w) {
            const float2 t = *reinterpret_cast<const float2*>(tot + w * 64 + 2 * lane);
            if (w < gw) { pre0 += t.x; pre1 += t.y; }
            all0 += t.x; all1 += t.y;
          }
          // every warp sees every channel's total, so all eight reach the same verdict
          viol = __any_sync(0xffffffffu, all0 < -kRange || all1 < -kRange) && nr > 1;
          if (viol) break;
          const float D0 = ex2f(all0), D1 = ex2f(all1);
          if (gw == 0) *reinterpret_cast<float2*>(sD + s * kDK + sl * 64 + 2 * lane) = make_float2(D0, D1);
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const int r = gw * 8 + i;
            const uint32_t off = r * 128 + ((((uint32_t)lane >> 2) ^ (r & 7)) << 4) + ((lane & 3) << 2);
            const uint32_t qw = lds32(slab + kOffQ + off), kw = lds32(slab + kOffK + off);
            const float b0 = bq[i][0] + pre0, b1 = bq[i][1] + pre1;
            const bool live = r < nr;
            const float q0 = live ? __uint_as_float(qw << 16) : 0.f;
            const float q1 = live ? __uint_as_float(qw & 0xFFFF0000u) : 0.f;
            const float k0 = live ? __uint_as_float(kw << 16) : 0.f;
            const float k1 = live ? __uint_as_float(kw & 0xFFFF0000u) : 0.f;
            const float kt0 = k0 * ex2f(eh[i][0] - b0), kt1 = k1 * ex2f(eh[i][1] - b1);
            sts32(slab + kOffQ + off, pack_bf16(q0 * ex2f(b0), q1 * ex2f(b1)));
            sts32(slab + kOffK + off, pack_bf16(kt0, kt1));
            sts32(slab + kOffX + off, pack_bf16(kt0 * D0, kt1 * D1));       // 2^{b_C - b_i} = 2^{-b_i} D
          }
        }
        if (!ok) break;
        if (viol) {
          // decays too fast for 'nr' rows at once: ask for this position again, fewer rows
          lcap = max(1, nr >> 1);
          fence_proxy_async();   // slab 0 may already be rewritten; the refill is a bulk copy
          if (!(ok = group_sync())) break;
          if (gw == 0 && lane == 0) {
            redirect(j, tpos);
            mbar_arrive(bar(BAR_EMPTY0 + s));
          }
          continue;
        }
        if (gw == 0 && lane == 0) {
          volatile PassDesc* pd = &ctl->pd[g & 3];
          pd->stage = (int)s;
          pd->nr = nr;
          pd->flags = (first ? kPassFirst : 0) | (nr == left ? kPassLast : 0);
          pd->row = it.row0 + tpos;
          if (nr < min(kC, left)) redirect(j, tpos + nr);   // the prefetcher assumed 64 rows
        }
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(BAR_GATED0 + (g & 1)));
        ++g;
        first = false;
        tpos += nr;
        if (lcap < kC) lcap = min(kC, lcap * 2);
      }
    }
    if (gw == 0 && lane == 0) ctl->done = 1;
  }

  // ------------------------------------------ teardown ------------------------------------------
  // After a wait that ran out the roles may have stopped anywhere: the contractions already
  // issued must finish before the tensor memory they write and the shared memory they read are
  // released.
  tc_fence_before();
  __syncthreads();
  if (ctl->wait.abort_flag && warp == 1) {
    if (lane == 0) {
      umma_commit(bar(BAR_DRAIN));
      mbar_drain(bar(BAR_DRAIN), 0);
    }
    __syncwarp();
  }
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols)
                 : "memory");
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  // looked up once (initialisation of a function-local static is thread-safe); a failed lookup
  // leaves nullptr and the callers report an error
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

// [rows, cols] bf16 row-major, box = 64 rows x 64 columns (128 bytes), 128-byte swizzle.
bool make_map(CUtensorMap* m, const void* ptr, uint64_t rows, uint64_t cols) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols * 2};
  const cuuint32_t box[2] = {64, (cuuint32_t)kC};
  const cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

cudaError_t launch_fwd_tc(const rodimus_ddts_fwd_params& p, int* n_launches) {
  *n_launches = 0;
  TcArgs a;
  a.o = p.o; a.s0 = p.s0; a.sT = p.sT; a.cu = p.cu_seqlens;
  a.hdr = reinterpret_cast<WorkspaceHeader*>(p.workspace);
  a.order = reinterpret_cast<const int32_t*>(reinterpret_cast<const char*>(p.workspace) +
                                             sizeof(WorkspaceHeader));
  a.H = p.H; a.T = p.T; a.dv = p.dv;
  a.n_seq = p.cu_seqlens ? p.N : p.B;
  a.slices = p.dv / kDVS;
  a.n_items = (long long)a.n_seq * p.H * a.slices;
  a.scale = p.scale;
  a.wait_cycles = main_loop_wait_cycles();
  if (a.n_items == 0) return cudaSuccess;
  const uint64_t rows = (uint64_t)p.B * p.H * p.T;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(p.stream);

  int dev = 0, sms = 0;
  cudaError_t e = current_device(&dev, &sms);
  if (e != cudaSuccess) return e;

  CUtensorMap mq, mk, mx, my, mv;
  if (rows > 0) {
    if (!make_map(&mq, p.q, rows, kDK) || !make_map(&mk, p.k, rows, kDK) ||
        !make_map(&mx, p.gate_x, rows, kDK) || !make_map(&my, p.temp_y, rows, kDK) ||
        !make_map(&mv, p.v, rows, (uint64_t)p.dv))
      return cudaErrorUnknown;
  } else {
    memset(&mq, 0, sizeof(mq)); mk = mq; mx = mq; my = mq; mv = mq;  // never dereferenced: no chunks
  }
  const int grid = (int)(a.n_items < sms ? a.n_items : sms);
  static std::atomic<unsigned long long> opted_g{0}, opted_s{0};
  if (p.ingate == RODIMUS_INGATE_POW_G) {
    e = opt_in_shared_memory(ddts_fwd_tc_kernel<RODIMUS_INGATE_POW_G>, kSmemBytes, dev, opted_g);
    if (e != cudaSuccess) return e;
    ddts_fwd_tc_kernel<RODIMUS_INGATE_POW_G><<<grid, kThreads, kSmemBytes, st>>>(mq, mk, mx, my, mv, a);
  } else {
    e = opt_in_shared_memory(ddts_fwd_tc_kernel<RODIMUS_INGATE_POW_SIGMOID>, kSmemBytes, dev, opted_s);
    if (e != cudaSuccess) return e;
    ddts_fwd_tc_kernel<RODIMUS_INGATE_POW_SIGMOID><<<grid, kThreads, kSmemBytes, st>>>(mq, mk, mx, my, mv, a);
  }
  *n_launches = 1;
  return cudaGetLastError();
}

}  // namespace ddts
