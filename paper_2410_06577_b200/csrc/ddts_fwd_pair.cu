// Chunked DDTS prefill on the 5th-generation tensor cores for dv a multiple of 256: two CTAs of
// a thread-block cluster work on one (sequence, head) and SHARE the gate math.
//
// Chunk algebra (appendix "Chunkwise Parallel Representation of the Rodimus Block"; chunk length
// 64, log2 domain, decays anchored at the chunk start, b_r = sum_{j<=r} log2 alpha_j <= 0):
//   Qt_r = q_r 2^{b_r}            Kt_i = k_i ahat_i 2^{-b_i}          D = 2^{b_C}
//   P = mask(Qt Kt^T)             O = P V + Qt S_in                   S_out = D . (S_in + Kt^T V)
// The state update is written with the chunk decay OUTSIDE the bracket, so the same Kt tile
// serves the scores and the state update, and the scaling by D happens when the state makes its
// once-per-chunk trip through registers.
//
// Everything that involves the value columns is computed TRANSPOSED, with the value column as
// the M extent of the tensor-core instruction (tensor-memory lane = value column):
//   S^T += V^T Kt            [128 value columns x 128 channels]   A = V^T (smem), B = Kt (smem)
//   O^T  = V^T P^T + Sb Qt^T [128 value columns x 64 rows]        A = V^T (smem) / Sb (TENSOR
//                                                                  MEMORY), B = P, Qt (smem)
// so every one of these instructions runs at M = 128 (an M = 64 instruction uses half of the
// datapath), and the bf16 copy Sb of the state that the readout contracts with is an A operand
// in tensor memory: it never goes through shared memory, which is the resource the roles of
// this kernel compete for.  With lane = value column, a warp's accesses to the initial and
// final states in global memory are 128 contiguous bytes per key channel.
//
// Every quantity that depends on the gates is per key channel and independent of the value
// column, so two CTAs that own the two 128-column halves of a 256-column slab of the state would
// otherwise repeat the whole softplus / sigmoid / log / exp2 pipeline.  Here CTA c of the pair
// loads q,k,x,y for key channels 64c..64c+63 only, turns them into Qt, Kt in place, and copies
// those two 8 KiB slabs (plus the 64 chunk decays) into the other CTA's shared memory with bulk
// shared-to-shared copies that complete on an mbarrier over there.  Each CTA then runs the three
// contractions on its own 128 value columns, taking half of the K (or M) extent from its own
// slab and half from the received one.
//
// The pair advances in lockstep: which rows form a pass is decided from the decay totals of all
// 128 channels, so each CTA sends its verdict along with its chunk decays and both take the OR.
//
// Roles in one CTA (28 warps), connected by mbarriers; every wait is bounded.  Warp w runs on
// scheduler w % 4, and a scheduler's first-level instruction cache holds about 8 KiB, less than
// the loops of all roles together: the single-warp roles, long straight-line code run once per
// pass, share scheduler 0, so that the loops of schedulers 1-3 (gate, state, score) stay cached.
//   warp 0          TMA producer (own channel slab of q,k,x,y and both slabs of the v slice)
//   warp 4          tcgen05.mma issuer, owns the TMEM allocation
//   warp 8          control: which fill is an attempt, scan of the row groups' sums, chunk decays,
//                   verdict exchange and slab copies to the partner, publishing, orders
//   warps 1-3, 12   state group (TMEM quarter = warp % 4): TMEM <-> registers trip of S^T, state I/O
//   warps 5-7, 16   score / output group
//   the other 16    gate workers (one on scheduler 0, five on each other): 4 rows x 2 channels
//                   per thread, packed fp32x2 arithmetic, on orders of the control warp
//
// The loop-carried chain is  state update of pass g -> rescaling of S -> state update of pass
// g+1 , so the issuer puts the state update of a pass BEFORE its output contractions, and the
// state lives in TWO TMEM buffers used alternately: the state group reads S_in + Kt^T V of the
// previous pass from one and writes D times it into the other, as fp32 for the next state update
// and as packed bf16 (also double-buffered) for the readout.
#include <cuda.h>

#include <cstring>
#include <mutex>

#include "ddts_common.cuh"
#include "ddts_tc_ptx.cuh"

namespace ddts {
namespace {

constexpr int kC = 64;                        // chunk rows
constexpr int kDK = 128;                      // key channels
constexpr int kCH = 64;                       // key channels whose gates one CTA computes
constexpr int kDVS = 128;                     // value columns per CTA
constexpr int kSlabBytes = kC * 128;          // [64 rows][64 bf16] = 8 KiB, 128-byte swizzled
// one stage of the TMA ring: own-channel slabs of q,k,x,y and the two slabs of v
constexpr int kStQ = 0, kStK = kSlabBytes, kStX = 2 * kSlabBytes, kStY = 3 * kSlabBytes,
              kStV = 4 * kSlabBytes;
constexpr int kStageBytes = 6 * kSlabBytes;   // 48 KiB
// one receive buffer: the partner's Qt, Kt slabs
constexpr int kRxQ = 0, kRxK = kSlabBytes;
constexpr int kRxBytes = 2 * kSlabBytes;      // 16 KiB
constexpr int kStages = 3, kRxBufs = 2;
constexpr int kOperandBytes = kStages * kStageBytes + kRxBufs * kRxBytes;  // 176 KiB
constexpr int kOtBytes = 2 * kSlabBytes;                  // output tile: two [64 rows][64 bf16] slabs
constexpr int kOffOt = kOperandBytes;                     // two output tiles (pass parity)
constexpr int kOffDp = kOffOt + 2 * kOtBytes;             // float [4][128]: chunk decays of all
                                                          // channels, per published pass (g & 3)
constexpr int kBlkFloats = 68;                            // 64 decays, verdict, stage, 2 pad
constexpr int kBlkBytes = kBlkFloats * 4;                 // 272 B, a multiple of 16
constexpr int kOffTx = kOffDp + 4 * kDK * 4;              // float [2][68]: block to send
constexpr int kOffRx = kOffTx + kRxBufs * kBlkBytes;      // float [2][68]: block received
constexpr int kGateWarp0 = 12, kGateWarps = 16;
constexpr int kGR = kC / kGateWarps;                       // rows per gate thread
constexpr int kOffTot = kOffRx + kRxBufs * kBlkBytes;     // float [2][8][64]: scan partials
constexpr int kOffBar = kOffTot + 2 * kGateWarps * kCH * 4;
constexpr int kNumBars = 40;
constexpr int kOffMisc = kOffBar + kNumBars * 8;          // control block
constexpr int kSmemUsed = kOffMisc + 320;
constexpr int kSmemBytes = kSmemUsed + 1024;              // slack for manual 1024-byte alignment
static_assert(kOffTx % 16 == 0 && kOffRx % 16 == 0 && kBlkBytes % 16 == 0, "bulk copy alignment");
static_assert(kSmemBytes <= 232448, "shared memory budget");

constexpr int kThreads = 32 * (kGateWarp0 + kGateWarps);   // 896: 28 warps (warp 24 has no role)

// TMEM columns (32-bit words): two state buffers S^T [lane = value column][128 channels], output
// O^T [lane = value column][64 rows], scores P [64 rows in 16-lane groups][64], and two buffers
// of the bf16 state copy Sb [lane = value column][64 columns = 128 channels, two per word]
constexpr uint32_t kColS = 0, kColO = 256, kColP = 320, kColSb = 384, kTmemCols = 512;

// mbarrier indices
enum { BAR_FULL0 = 0,                 // [3] TMA fill landed                      (1 + bytes)
       BAR_EMPTY0 = 3,                // [3] stage reusable: own release + partner's receipt (2)
       BAR_GATED0 = 6,                // [4] pass published by the control warp              (1)
       BAR_PEER0 = 10, BAR_PEER1,     // partner's two slabs landed                 (1 + bytes)
       BAR_VERD0, BAR_VERD1,          // own verdict written + partner's block landed (1 + bytes)
       BAR_RXFREE0, BAR_RXFREE1,      // partner is done with ITS receive buffer            (1)
       BAR_PFULL, BAR_PREADY,
       BAR_SREADY,                    // state entering the pass is in TMEM, fp32 and bf16 (128)
       BAR_SFULL, BAR_OFULL, BAR_OFREE, BAR_GSCAN,
       BAR_OTFULL0, BAR_OTFULL1,      // output tile written by the whole score group        (128)
       BAR_OTFREE0, BAR_OTFREE1,      // output tile's copies to global have read it            (1)
       BAR_GO0, BAR_GO1,              // an order for the gate warps is in its slot              (1)
       BAR_PRE,                       // the row groups' prefixes are in place                   (1)
       BAR_ROWS,                      // every gate warp has rewritten its rows of the pass
       BAR_DRAIN,                     // teardown after a timeout: issued contractions are done  (1)
       BAR_XFULL0, BAR_XFULL1 };      // feed-through tile x' landed in the output tile (1 + bytes)
static_assert(BAR_XFULL1 < kNumBars, "barrier count");

struct PairArgs {
  void* o;
  const float* s0;
  float* sT;
  const int32_t* cu;
  const int32_t* order;
  WorkspaceHeader* hdr;
  int H, T, dv, n_seq, pairs;
  long long n_items;     // (sequence, head, 256-column slab)
  float scale;
  long long wait_cycles; // limit of one main-loop wait (clock cycles)
  // optional terms of the full block (BLOCK instantiations only)
  const __nv_bfloat16* beta_hat;  // [rows, dv] value gate, or nullptr
  const float* feed_d;            // [H, dv] feed-through weight, or nullptr (then no x' either)
  int feed_H;                     // heads per sequence of the caller's layout (indexes feed_d)
  int gate_div;                   // 1, or for the shared-gate layout the caller's H: q,k,x,y hold
                                  // one set of rows per sequence, [B,1,T,dk]
  float* dtot;           // optional [n_seq, H, dk]: product of all chunk decays of each sequence
  int sT_only;           // >= 0: only this sequence's final state is stored, as if it were number 0
  int state_only;        // 1: launch the state-only instantiation of the kernel
};

struct Item {
  long long row0;      // first global row (in the [rows, d] view) of this sequence and head
  long long rowq;      // the same in q,k,x,y (differs from row0 in the shared-gate layout)
  long long state_off; // element offset of this CTA's state slice (row 0, first own column)
  long long seq_head;  // sequence * H + head
  int len;             // tokens
  int col0;            // first value column of this CTA
  int seq;             // sequence number (after the longest-first reordering)
};

__device__ __forceinline__ Item decode_item(const PairArgs& a, long long item, int rank) {
  Item it;
  const int pair = (int)(item % a.pairs);
  const long long sh = item / a.pairs;
  const int h = (int)(sh % a.H);
  long long n = sh / a.H;
  if (a.cu) {
    n = a.order[n];
    int lo = a.cu[n], hi = a.cu[n + 1];
    lo = lo < 0 ? 0 : (lo > a.T ? a.T : lo);
    hi = hi < lo ? lo : (hi > a.T ? a.T : hi);
    it.row0 = (long long)h * a.T + lo;
    it.rowq = (long long)(h / a.gate_div) * a.T + lo;
    it.len = hi - lo;
  } else {
    it.row0 = (n * a.H + h) * (long long)a.T;
    it.rowq = ((n * a.H + h) / a.gate_div) * (long long)a.T;
    it.len = a.T;
  }
  it.col0 = (pair * 2 + rank) * kDVS;
  it.seq_head = n * a.H + h;
  it.seq = (int)n;
  it.state_off = it.seq_head * (long long)kDK * a.dv + it.col0;
  return it;
}

// A "fill" is one 64-row tile brought into a stage by the producer; an "attempt" is a fill at
// the position the gate group expects (the producer prefetches speculatively, so some fills are
// not); a "pass" is an attempt both CTAs accepted.  Fill counters are private to a CTA; attempt
// and pass counters advance identically in both, which is what the receive buffers and their
// barriers are indexed by.
struct PassDesc {
  int stage;      // which stage holds the own-channel operands and v
  int nr;         // live rows
  int flags;      // kPassLast
  int rx;         // which receive buffer holds the partner's operands
  int rxph;       // parity of that buffer's barrier phase
  int pad;
  long long row;  // global row (in the [rows, d] view) of the pass's first token
};
constexpr int kPassLast = 2;

struct Control {            // lives in shared memory
  uint32_t tmem_base;
  int done;                 // gate group has finished every item of this CTA
  WaitCtl wait;             // abort flag and limit shared by every bounded wait of the CTA
  // teardown handshake of the pair: how many attempts' decay blocks / operand slabs this CTA
  // has copied to the partner and for how many it has armed its own receive barriers; and what
  // the partner says about itself (written by the partner before the first closing barrier)
  int sent_blk, sent_slab, armed_cnt;
  int peer_abort, peer_sent_blk, peer_sent_slab;
  int redir_seq;            // bumped by the gate group after writing redir_j / redir_tpos
  int redir_j, redir_tpos;  // where the producer must continue (CTA-local item index, token)
  int tag[kStages][2];      // per stage: (item index, token position) of the fill it holds
  int pad[2];
  PassDesc pd[4];
  // orders of the control warp to the gate warps (stage < 0: leave); row and col0 locate the
  // tile in global memory for the value gate
  struct { int stage, nr, col0, pad; long long row; } ord[2];
};
static_assert(sizeof(Control) <= 320, "control block");

// ---------------------------------------------------------------------------------------------
// gate math on pairs of adjacent key channels (packed fp32x2 adds / multiplies / fmas)
// ---------------------------------------------------------------------------------------------
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLg2Ln2 = -0.5287663729448977f;   // log2(ln 2)
constexpr float kRange = 60.f * kLog2e;           // largest in-chunk decay range, log2 units

__device__ __forceinline__ float2 bf16x2_to_f2(uint32_t w) {
  return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xFFFF0000u));
}
__device__ __forceinline__ float2 splat(float v) { return make_float2(v, v); }

// Phase 1 for this thread's kGR rows x 2 channels: log2 decay (cumulative over the thread's own
// rows, b) and log2 input weight (eh).  Returns the sum of those rows' log2 decays.
template <int INGATE>
__device__ __forceinline__ float2 gate_phase1(uint32_t xs, uint32_t ys, const uint32_t (&off)[kGR],
                                              int row0, int nr, float2 (&b)[kGR], float2 (&eh)[kGR]) {
  float2 run = splat(0.f);
#pragma unroll
  for (int i = 0; i < kGR; ++i) {
    const float2 x = bf16x2_to_f2(lds32(xs + off[i]));
    const float2 y = bf16x2_to_f2(lds32(ys + off[i]));
    const float2 xl = __fmul2_rn(x, splat(kLog2e));
    const float2 u = make_float2(ex2f(xl.x), ex2f(xl.y));               // e^x
    // log2(1 + e^x) = g log2(e); series where 1 + u would round u away
    const float2 w = __fadd2_rn(u, splat(1.f));
    const float2 ser = __fmul2_rn(u, __ffma2_rn(u, splat(-0.72134752f), splat(kLog2e)));
    const float2 sp2 = make_float2(u.x < 9.765625e-4f ? ser.x : lg2f(w.x),
                                   u.y < 9.765625e-4f ? ser.y : lg2f(w.y));
    // -tau = -sigmoid(y) = -1/2 - tanh(y/2)/2: one special-function operation instead of two
    // (the approximation's error, 2^-11 of tanh, is an absolute 2.5e-4 of tau)
    const float2 yh = __fmul2_rn(y, splat(0.5f));
    const float2 ntau = __ffma2_rn(make_float2(tanh_approx(yh.x), tanh_approx(yh.y)), splat(-0.5f), splat(-0.5f));
    float2 l2a = __fmul2_rn(sp2, ntau);                                 // log2 alpha <= 0
    l2a.x = fmaxf(l2a.x, -kRange);                                      // per-step floor exp(-60)
    l2a.y = fmaxf(l2a.y, -kRange);
    if (INGATE == RODIMUS_INGATE_POW_G) {                               // tau * log2(g)
      eh[i] = __fmul2_rn(ntau, __ffma2_rn(make_float2(lg2f(sp2.x), lg2f(sp2.y)), splat(-1.f),
                                          splat(-kLg2Ln2)));
    } else {                                                            // tau * log2(sigmoid(x))
      eh[i] = __fmul2_rn(ntau, __ffma2_rn(xl, splat(-1.f), sp2));
    }
    if (row0 + i >= nr) l2a = splat(0.f);                               // rows past the pass
    run = __fadd2_rn(run, l2a);
    b[i] = run;
  }
  return run;
}

// Phase 2: Qt = q 2^{b}, Kt = k 2^{eh - b}, written over q and k (same swizzled offsets).
// STATE_ONLY: the pass only updates the state, so Qt is not needed.
template <bool STATE_ONLY>
__device__ __forceinline__ void gate_phase2(uint32_t qs, uint32_t ks, const uint32_t (&off)[kGR],
                                            int row0, int nr, float2 pre, const float2 (&b)[kGR],
                                            const float2 (&eh)[kGR]) {
#pragma unroll
  for (int i = 0; i < kGR; ++i) {
    float2 k = bf16x2_to_f2(lds32(ks + off[i]));
    const float2 bb = __fadd2_rn(b[i], pre);
    const float2 hb = __ffma2_rn(bb, splat(-1.f), eh[i]);
    const float2 ek = make_float2(ex2f(hb.x), ex2f(hb.y));
    if (row0 + i >= nr) k = splat(0.f);
    const float2 kt = __fmul2_rn(k, ek);
    sts32(ks + off[i], pack_bf16(kt.x, kt.y));
    if (!STATE_ONLY) {
      float2 q = bf16x2_to_f2(lds32(qs + off[i]));
      const float2 eq = make_float2(ex2f(bb.x), ex2f(bb.y));
      if (row0 + i >= nr) q = splat(0.f);
      const float2 qt = __fmul2_rn(q, eq);
      sts32(qs + off[i], pack_bf16(qt.x, qt.y));
    }
  }
}

// STATE_ONLY: only final states and decay products are wanted (no q, scores, outputs); a
// compile-time switch so that the full kernel carries none of its branches.
// BLOCK: the optional terms of the full block are compiled in (value gate applied to the v tile
// in shared memory by the gate warps, feed-through added in the output path); the plain
// instantiations carry none of that code.
template <int INGATE, bool STATE_ONLY, bool BLOCK>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
ddts_fwd_pair_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                     const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_y,
                     const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_o,
                     const __grid_constant__ CUtensorMap map_o8, const __grid_constant__ CUtensorMap map_o1,
                     const __grid_constant__ CUtensorMap map_b, const __grid_constant__ CUtensorMap map_fx,
                     const PairArgs a) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gbase = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bars = base + kOffBar;
  auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
  volatile Control* ctl = reinterpret_cast<volatile Control*>(gbase + kOffMisc);
  volatile WaitCtl* abort_flag = &ctl->wait;
  float* sDp = reinterpret_cast<float*>(gbase + kOffDp);
  volatile float* sTx = reinterpret_cast<volatile float*>(gbase + kOffTx);
  volatile float* sRx = reinterpret_cast<volatile float*>(gbase + kOffRx);
  float* sTot = reinterpret_cast<float*>(gbase + kOffTot);

  const int tid = threadIdx.x;
  const int warp = tid >> 5, lane = tid & 31;
  // Warp w runs on scheduler w % 4.  The single-warp roles (long straight-line code once per pass)
  // all sit on scheduler 0 together with one gate worker; schedulers 1-3 run five gate workers,
  // a state warp and a score warp each, whose loops fit the scheduler's instruction cache.
  // role: 0 producer, 1 issuer, 2 control, 3 state, 4 score, 5 gate worker, 6 none
  int role, gw_of_warp = 0;
  if (warp == 0) role = 0;
  else if (warp == 4) role = 1;
  else if (warp == 8) role = 2;
  else if (warp == 24) role = 6;
  else if (warp == 12 || warp < 4) role = 3;
  else if (warp == 16 || warp < 8) role = 4;
  else {
    role = 5;
    // gate warps in increasing warp number: 9,10,11,13,14,15,17,18,19,20,21,22,23,25,26,27
    gw_of_warp = warp - 9 - (warp > 12) - (warp > 16) - (warp > 24);
  }
  const int rank = (int)cluster_ctarank();     // 0 or 1: which key-channel half and dv half
  const int peer = rank ^ 1;
  // The state update takes Kt for all 128 channels as ONE operand whose two 64-channel groups
  // must sit at increasing addresses: channels 0..63 first.  So the CTA that owns the low
  // channels keeps its stages below its receive buffers and the other CTA the opposite.
  const uint32_t stage_base = base + (rank == 0 ? 0u : (uint32_t)(kRxBufs * kRxBytes));
  const uint32_t rx_base = base + (rank == 0 ? (uint32_t)(kStages * kStageBytes) : 0u);
  const uint32_t peer_rx_base = base + (peer == 0 ? (uint32_t)(kStages * kStageBytes) : 0u);

  if (!a.cu && blockIdx.x == 0 && tid == 0) a.hdr->status = RODIMUS_OK;

  if (tid == 0) {
    ctl->wait.abort_flag = 0;
    ctl->wait.limit = a.wait_cycles;
    ctl->sent_blk = ctl->sent_slab = ctl->armed_cnt = 0;
    ctl->peer_abort = ctl->peer_sent_blk = ctl->peer_sent_slab = 0;
    ctl->done = 0;
    ctl->redir_seq = 0;
    for (int s = 0; s < kStages; ++s) {
      mbar_init(bar(BAR_FULL0 + s), 1);
      mbar_init(bar(BAR_EMPTY0 + s), 2);
    }
    for (int i = 0; i < 4; ++i) mbar_init(bar(BAR_GATED0 + i), 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar(BAR_PEER0 + i), 1);
      mbar_init(bar(BAR_VERD0 + i), 1);
      mbar_init(bar(BAR_RXFREE0 + i), 1);
    }
    mbar_init(bar(BAR_PFULL), 1);
    mbar_init(bar(BAR_PREADY), 128);
    mbar_init(bar(BAR_SREADY), 128);
    mbar_init(bar(BAR_SFULL), 1);
    mbar_init(bar(BAR_OFULL), 1);
    mbar_init(bar(BAR_OFREE), 128);
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar(BAR_OTFULL0 + i), 128);
      mbar_init(bar(BAR_OTFREE0 + i), 1);
    }
    mbar_init(bar(BAR_GSCAN), kGateWarps);
    mbar_init(bar(BAR_GO0), 1);
    mbar_init(bar(BAR_GO1), 1);
    mbar_init(bar(BAR_PRE), 1);
    mbar_init(bar(BAR_DRAIN), 1);
    mbar_init(bar(BAR_XFULL0), 1);
    mbar_init(bar(BAR_XFULL1), 1);
    mbar_init(bar(BAR_ROWS), kGateWarps);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // One 64-row tile of this CTA's operands into stage s (this thread is the producer).
  auto issue_fill = [&](uint32_t s, const Item& it, int j, int tpos) {
    ctl->tag[s][0] = j;
    ctl->tag[s][1] = tpos;
    const uint32_t st = stage_base + s * kStageBytes;
    const uint32_t fb = bar(BAR_FULL0 + s);
    mbar_expect_tx(fb, STATE_ONLY ? kStageBytes - kSlabBytes : kStageBytes);
    // rows beyond the tensor read as zeros; rows of the next sequence are masked later
    const int y = (int)(it.row0 + tpos);
    const int yq = (int)(it.rowq + tpos);
    const int xc = rank * kCH;
    tma_load_2d(st + kStX, &map_x, xc, yq, fb);
    tma_load_2d(st + kStY, &map_y, xc, yq, fb);
    if (!STATE_ONLY) tma_load_2d(st + kStQ, &map_q, xc, yq, fb);
    tma_load_2d(st + kStK, &map_k, xc, yq, fb);
    tma_load_2d(st + kStV, &map_v, it.col0, y, fb);
    tma_load_2d(st + kStV + kSlabBytes, &map_v, it.col0 + 64, y, fb);
    // The tile that will go into this stage NEXT time is asked into L2 now: a stage is refilled
    // only when its pass has been consumed, so the fill's latency is on the critical cycle of
    // the ring, and from L2 it is less than half of what it is from HBM.
    const int yp = y + kStages * kC, yqp = yq + kStages * kC;
    if (tpos + kStages * kC < it.len) {
      tma_prefetch_2d(&map_x, xc, yqp);
      tma_prefetch_2d(&map_y, xc, yqp);
      if (!STATE_ONLY) tma_prefetch_2d(&map_q, xc, yqp);
      tma_prefetch_2d(&map_k, xc, yqp);
      tma_prefetch_2d(&map_v, it.col0, yp);
      tma_prefetch_2d(&map_v, it.col0 + 64, yp);
      if (BLOCK && a.beta_hat) {
        tma_prefetch_2d(&map_b, it.col0, yp);
        tma_prefetch_2d(&map_b, it.col0 + 64, yp);
      }
      if (BLOCK && !STATE_ONLY && a.feed_d) {
        tma_prefetch_2d(&map_fx, it.col0, yp);
        tma_prefetch_2d(&map_fx, it.col0 + 64, yp);
      }
    }
  };
  // The first fill touches only this CTA's own barriers and shared memory, so it goes out
  // before the tensor-memory allocation and the cluster handshake instead of after them.
  uint32_t early_fills = 0;
  if (tid == 0) {
    const long long item0 = (long long)(blockIdx.x >> 1);
    if (item0 < a.n_items) {
      const Item it = decode_item(a, item0, rank);
      if (it.len > 0) {
        issue_fill(0, it, 0, 0);
        early_fills = 1;
      }
    }
  }
  if (role == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(base + kOffMisc), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  // both CTAs' barriers exist before either touches the other's shared memory
  cluster_arrive();
  cluster_wait();
  const uint32_t tmem = ctl->tmem_base;
  const long long n_pairs_grid = gridDim.x >> 1;
  const long long pair_id = blockIdx.x >> 1;
  auto item_of = [&](int j) { return pair_id + (long long)j * n_pairs_grid; };

  if (role == 0) {
    // ===================================== TMA producer =====================================
    if (lane == 0) {
      uint32_t f = early_fills;            // fills issued
      uint32_t s = early_fills, ph = 0;    // stage and phase of fill f
      int j = 0, tpos = early_fills * kC;  // speculative position: item index and token
      int seen = 0;           // last redirect taken
      bool ok = true;
      while (ok) {
        if (!(ok = mbar_wait_cluster(bar(BAR_EMPTY0 + s), ph ^ 1, abort_flag, a.hdr))) break;
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
            it = decode_item(a, item_of(j), rank);
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
        issue_fill(s, it, j, tpos);
        ++f;
        if (++s == kStages) { s = 0; ph ^= 1; }
        tpos += kC;
      }
      // Leave no bulk copy in flight when the CTA exits: the last fills' barriers complete by
      // byte count, whoever consumed them.
      for (uint32_t back = 1; back <= (uint32_t)kStages && back <= f; ++back) {
        const uint32_t ff = f - back;
        mbar_drain(bar(BAR_FULL0 + ff % kStages), (ff / kStages) & 1);
      }
    }
  } else if (role == 1) {
    // ====================================== MMA issuer ======================================
    // Every lane runs the loop (waits, descriptor arithmetic stay warp-uniform); lane 0 issues.
    {
      const bool issuer = lane == 0;
      constexpr uint32_t kIdescP = make_idesc(64, 64, 0, 0);       // P = Qt Kt^T
      constexpr uint32_t kIdescS = make_idesc(kDVS, kDK, 1, 1);    // S^T += V^T Kt
      constexpr uint32_t kIdescOv = make_idesc(kDVS, kC, 1, 0);    // O^T  = V^T P^T
      constexpr uint32_t kIdescOs = make_idesc(kDVS, kC, 0, 0);    // O^T += Sb Qt^T, A in TMEM
      uint32_t g = 0;
      bool ok = true;
      for (int j = 0; ok && item_of(j) < a.n_items; ++j) {
        const Item it = decode_item(a, item_of(j), rank);
        if (it.len == 0) continue;
        bool last = false;
        while (!last) {
          const uint32_t ph1 = g & 1;
          if (!(ok = mbar_wait(bar(BAR_GATED0 + (g & 3)), (g >> 2) & 1, abort_flag, a.hdr))) break;
          const uint32_t s = (uint32_t)ctl->pd[g & 3].stage;
          const uint32_t rxi = (uint32_t)ctl->pd[g & 3].rx;
          const uint32_t rxph = (uint32_t)ctl->pd[g & 3].rxph;
          last = (ctl->pd[g & 3].flags & kPassLast) != 0;
          if (!(ok = mbar_wait_cluster(bar(BAR_PEER0 + rxi), rxph, abort_flag, a.hdr))) break;
          const uint32_t st = stage_base + s * kStageBytes;
          const uint32_t rx = rx_base + rxi * kRxBytes;
          // Low descriptor halves of the pass's operands (channel slab 0 / 1 of Qt and Kt sit in
          // the stage or in the receive buffer depending on the rank); stepping K is one add.
          const uint32_t q_own = st + kStQ, q_rx = rx + kRxQ, k_own = st + kStK, k_rx = rx + kRxK;
          const uint32_t k_lo_addr = rank == 0 ? k_own : k_rx, k_hi_addr = rank == 0 ? k_rx : k_own;
          const uint32_t dq0 = desc_lo_kmajor(rank == 0 ? q_own : q_rx);
          const uint32_t dq1 = desc_lo_kmajor(rank == 0 ? q_rx : q_own);
          const uint32_t dk0 = desc_lo_kmajor(k_lo_addr), dk1 = desc_lo_kmajor(k_hi_addr);
          // Kt as [rows][128 channels], channels 0..63 and 64..127 in two slabs
          const uint32_t dkt = desc_lo_mnmajor(k_lo_addr, k_hi_addr - k_lo_addr);
          // V as [rows][128 value columns], two 64-column slabs
          const uint32_t dv = desc_lo_mnmajor(st + kStV, kSlabBytes);
          const uint32_t dp = desc_lo_kmajor(st + kStY);
          const uint32_t t_sb = tmem + kColSb + (g & 1) * 64;
          tc_fence_after();
          // P = Qt Kt^T : M = 64 (rows r), N = 64 (rows i), K = 128 channels
          if (issuer && !STATE_ONLY) {
            umma_bf16_lo<false>(tmem + kColP, dq0, dk0, kIdescP);
#pragma unroll
            for (int kk = 1; kk < 4; ++kk) umma_bf16_lo<true>(tmem + kColP, dq0 + 2 * kk, dk0 + 2 * kk, kIdescP);
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) umma_bf16_lo<true>(tmem + kColP, dq1 + 2 * kk, dk1 + 2 * kk, kIdescP);
            umma_commit(bar(BAR_PFULL));
          }
          if (!(ok = mbar_wait(bar(BAR_SREADY), ph1, abort_flag, a.hdr))) break;
          tc_fence_after();
          if (issuer) {
            // S_in^T + V^T Kt : M = 128 value columns, N = 128 channels, K = 64 rows (S_in^T sits
            // in buffer g & 1)
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
              umma_bf16_lo<true>(tmem + kColS + (g & 1) * 128, dv + 128 * kk, dkt + 128 * kk, kIdescS);
            umma_commit(bar(BAR_SFULL));
            if (STATE_ONLY) umma_commit(bar(BAR_EMPTY0 + s));
          }
          if (STATE_ONLY) { ++g; continue; }             // no scores, no outputs
          if (!(ok = mbar_wait(bar(BAR_PREADY), ph1, abort_flag, a.hdr))) break;
          if (!(ok = mbar_wait(bar(BAR_OFREE), ph1 ^ 1, abort_flag, a.hdr))) break;
          tc_fence_after();
          if (issuer) {
            // O^T = V^T P^T : M = 128 value columns, N = 64 rows r, K = 64 rows i (the masked
            // scores P[r][i] live in the consumed y slab)
            umma_bf16_lo<false>(tmem + kColO, dv, dp, kIdescOv);
#pragma unroll
            for (int kk = 1; kk < 4; ++kk) umma_bf16_lo<true>(tmem + kColO, dv + 128 * kk, dp + 2 * kk, kIdescOv);
            // O^T += Sb Qt^T : K = 128 channels; Sb (bf16 copy of S_in^T) is read from TMEM
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) umma_bf16_atmem<true>(tmem + kColO, t_sb + 8 * kk, dq0 + 2 * kk, kIdescOs);
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) umma_bf16_atmem<true>(tmem + kColO, t_sb + 8 * (kk + 4), dq1 + 2 * kk, kIdescOs);
            umma_commit(bar(BAR_OFULL));
            umma_commit(bar(BAR_EMPTY0 + s));   // every contraction of the pass has read its operands
          }
          ++g;
        }
      }
    }
  } else if (role == 3) {
    // ====================================== state group ======================================
    // Each thread owns one value column of the CTA's slice (= one TMEM lane of S^T); the 128
    // key channels are its TMEM columns.  Pass g accumulates its state update in buffer g & 1.
    // Once per pass the group reads S_in^T + V^T Kt of pass g-1 from the other buffer, scales
    // channel d by that pass's chunk decay D[d], and writes the result - the state entering
    // pass g - twice: as fp32 into buffer g & 1 (the state update of pass g accumulates onto
    // it) and as packed bf16 into Sb buffer g & 1 (the A operand of pass g's readout).  Both
    // targets are free: the tensor pipe runs in order, so the state update of pass g-1 having
    // completed means the readout of pass g-2, the last reader of either, has completed too.
    const int q4 = warp & 3;                              // TMEM lane quarter this warp may touch
    const int c = q4 * 32 + lane;                         // value column (TMEM lane) of this thread
    const uint32_t t_lane = tmem + ((uint32_t)(q4 * 32) << 16);
    const bool signaller = (warp & 3) == 0 && lane == 0;
    uint32_t g = 0;
    int prev_rx = 0;
    bool ok = true;
    for (int j = 0; ok && item_of(j) < a.n_items; ++j) {
      const Item it = decode_item(a, item_of(j), rank);
      // element (channel d, own column) of the state: soff + d * dv; a warp covers 32
      // consecutive columns, 128 contiguous bytes per channel
      const long long soff = it.state_off + c;
      if (it.len == 0) {  // empty sequence: final state = initial state
        if (a.sT) {
#pragma unroll 4
          for (int d = 0; d < kDK; ++d)
            a.sT[soff + (long long)d * a.dv] = a.s0 ? a.s0[soff + (long long)d * a.dv] : 0.f;
        }
        continue;
      }
      bool last = false, first = true;
      float Dall = 1.f;          // product of the chunk decays of channel c so far (for dtot)
      // 32 channels of the state entering the pass: D of the previous pass times the previous
      // buffer, or the caller's initial state for the first pass of a sequence
      auto load_piece = [&](uint32_t (&r)[32], uint32_t t_prev, const float* dprev, int piece) {
        if (!first) {
          tmem_ld32(t_prev + piece * 32, r);
          tmem_ld_wait();
#pragma unroll
          for (int c4 = 0; c4 < 8; ++c4) {
            const float4 dd = *reinterpret_cast<const float4*>(dprev + piece * 32 + 4 * c4);  // broadcast
            const float2 lo = __fmul2_rn(make_float2(__uint_as_float(r[4 * c4]), __uint_as_float(r[4 * c4 + 1])),
                                         make_float2(dd.x, dd.y));
            const float2 hi = __fmul2_rn(make_float2(__uint_as_float(r[4 * c4 + 2]), __uint_as_float(r[4 * c4 + 3])),
                                         make_float2(dd.z, dd.w));
            r[4 * c4] = __float_as_uint(lo.x);
            r[4 * c4 + 1] = __float_as_uint(lo.y);
            r[4 * c4 + 2] = __float_as_uint(hi.x);
            r[4 * c4 + 3] = __float_as_uint(hi.y);
          }
        } else if (a.s0) {
#pragma unroll
          for (int i = 0; i < 32; ++i)
            r[i] = __float_as_uint(a.s0[soff + (long long)(piece * 32 + i) * a.dv]);
        } else {
#pragma unroll
          for (int i = 0; i < 32; ++i) r[i] = 0u;
        }
      };
      while (!last) {
        const uint32_t ph1 = g & 1;
        const uint32_t t_cur = t_lane + kColS + (g & 1) * 128, t_prev = t_lane + kColS + ((g & 1) ^ 1) * 128;
        const uint32_t t_sb = t_lane + kColSb + (g & 1) * 64;
        const float* dprev = sDp + ((g - 1) & 3) * kDK;
        if (!first) {
          if (!(ok = mbar_wait(bar(BAR_SFULL), ph1 ^ 1, abort_flag, a.hdr))) break;  // pass g-1
          tc_fence_after();
        }
#pragma unroll 1
        for (int piece = 0; piece < 4; ++piece) {
          uint32_t r[32];
          load_piece(r, t_prev, dprev, piece);
          tmem_st32(t_cur + piece * 32, r);
          if (!STATE_ONLY) {
            uint32_t w[16];
#pragma unroll
            for (int i = 0; i < 16; ++i)
              w[i] = pack_bf16(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1]));
            tmem_st16(t_sb + piece * 16, w);
          }
        }
        tmem_st_wait();
        tc_fence_before();
        mbar_arrive(bar(BAR_SREADY));
        if (!first) {
          // the previous pass's contractions have all read their operands: the partner may reuse
          // the receive buffer.  Signalled before waiting for pass g: publishing pass g may
          // itself need that buffer.
          if (!STATE_ONLY && !(ok = mbar_wait(bar(BAR_OFULL), ph1 ^ 1, abort_flag, a.hdr))) break;
          if (signaller) mbar_arrive_remote(map_to_cta(bar(BAR_RXFREE0 + prev_rx), peer));
        }
        if (!(ok = mbar_wait(bar(BAR_GATED0 + (g & 3)), (g >> 2) & 1, abort_flag, a.hdr))) break;
        prev_rx = ctl->pd[g & 3].rx;
        last = (ctl->pd[g & 3].flags & kPassLast) != 0;
        Dall *= sDp[(g & 3) * kDK + c];                   // thread c follows channel c
        first = false;
        ++g;
      }
      if (!ok) break;
      if (a.dtot && it.col0 == 0) a.dtot[it.seq_head * kDK + c] = Dall;
      // final state of this item (also keeps the next item's initial state from racing the MMAs)
      {
        const uint32_t lastg = g - 1;
        if (!(ok = mbar_wait(bar(BAR_SFULL), lastg & 1, abort_flag, a.hdr))) break;
        if (!STATE_ONLY && !(ok = mbar_wait(bar(BAR_OFULL), lastg & 1, abort_flag, a.hdr))) break;
        tc_fence_after();
        if (signaller) mbar_arrive_remote(map_to_cta(bar(BAR_RXFREE0 + prev_rx), peer));
        if (a.sT && (a.sT_only < 0 || it.seq == a.sT_only)) {
          const long long foff = a.sT_only < 0 ? soff : soff - (long long)a.sT_only * a.H * kDK * a.dv;
          const uint32_t t_fin = t_lane + kColS + (lastg & 1) * 128;
          const float* dlast = sDp + (lastg & 3) * kDK;
#pragma unroll 1
          for (int piece = 0; piece < 4; ++piece) {
            uint32_t r[32];
            tmem_ld32(t_fin + piece * 32, r);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i)
              a.sT[foff + (long long)(piece * 32 + i) * a.dv] = dlast[piece * 32 + i] * __uint_as_float(r[i]);
          }
        }
        tc_fence_before();
      }
    }
  } else if (role == 4) {
    // ================================== score / output group ==================================
    const int q4 = warp & 3;
    // stmatrix roles of this thread: it addresses row mat_k of matrix lane/8 of each x4 group;
    // matrices 0,1 are the low / high 8 rows of one 8-column block, 2,3 those of the next block
    const int mat_k = lane & 7, mat_h = (lane >> 3) & 1, mat_j = lane >> 4;
    // diagonal block: element (row t/4, columns 2(t%4) + e) is kept iff the column does not
    // exceed the row
    const uint32_t mask_diag = (2 * (lane & 3) <= (lane >> 2) ? 0x0000FFFFu : 0u) |
                               (2 * (lane & 3) + 1 <= (lane >> 2) ? 0xFFFF0000u : 0u);
    const uint32_t t_lane = tmem + ((uint32_t)(q4 * 32) << 16);
    const bool unit_scale = a.scale == 1.0f;
    uint32_t g = 0;
    bool ok = true;
    for (int j = 0; ok && item_of(j) < a.n_items; ++j) {
      const Item it = decode_item(a, item_of(j), rank);
      if (it.len == 0) continue;
      bool last = false;
      while (!last) {
        const uint32_t ph1 = g & 1;
        if (STATE_ONLY) {
          // nothing to mask or store: only the partner's stage is handed back, once its slab has
          // landed here
          if (!(ok = mbar_wait(bar(BAR_GATED0 + (g & 3)), (g >> 2) & 1, abort_flag, a.hdr))) break;
          const int rxi = ctl->pd[g & 3].rx;
          last = (ctl->pd[g & 3].flags & kPassLast) != 0;
          if (!(ok = mbar_wait_cluster(bar(BAR_PEER0 + rxi), (uint32_t)ctl->pd[g & 3].rxph, abort_flag, a.hdr))) break;
          if (q4 == 0 && lane == 0) {
            const int peer_stage = __float_as_int(sRx[rxi * kBlkFloats + 65]);
            mbar_arrive_remote(map_to_cta(bar(BAR_EMPTY0 + peer_stage), peer));
          }
          ++g;
          continue;
        }
        if (!(ok = mbar_wait(bar(BAR_PFULL), ph1, abort_flag, a.hdr))) break;
        const int s = ctl->pd[g & 3].stage;
        const int nr = ctl->pd[g & 3].nr;
        const long long row = ctl->pd[g & 3].row;
        last = (ctl->pd[g & 3].flags & kPassLast) != 0;
        // row of the P tile ([r][i], 128-byte rows, 16-byte chunks swizzled by r & 7) whose
        // address this thread supplies to stmatrix: row block mat_h, row mat_k within it
        const uint32_t ps_mat = stage_base + s * kStageBytes + kStY + (q4 * 16 + mat_h * 8 + mat_k) * 128;
        tc_fence_after();
        const bool feed = BLOCK && a.feed_d != nullptr;
        if (feed && q4 == 0) {
          // Feed-through: the x' tile of this pass is fetched INTO the output tile (same two-slab
          // swizzled layout), to be combined with the accumulators in place further down.  The
          // tile must be free first: the copies that read it two passes ago are done.
          if (!(ok = mbar_wait(bar(BAR_OTFREE0 + ph1), ((g >> 1) & 1) ^ 1, abort_flag, a.hdr))) break;
          if (lane == 0) {
            const uint32_t xb = bar(BAR_XFULL0 + ph1);
            const uint32_t xt = base + kOffOt + ph1 * kOtBytes;
            mbar_expect_tx(xb, kOtBytes);
            tma_load_2d(xt, &map_fx, it.col0, (int)row, xb);
            tma_load_2d(xt + kSlabBytes, &map_fx, it.col0 + 64, (int)row, xb);
          }
        }
        if (q4 == 0 && lane == 0) {
          // P exists, so the partner's copies out of ITS stage have all landed here (the issuer
          // waited for them): let the partner reuse that stage
          const int rxi = ctl->pd[g & 3].rx;
          const int peer_stage = __float_as_int(sRx[rxi * kBlkFloats + 65]);
          mbar_arrive_remote(map_to_cta(bar(BAR_EMPTY0 + peer_stage), peer));
        }
        // Causal mask (i <= r kept) and conversion to bf16.  The M = 64 accumulator keeps this
        // warp's rows 16*q4 .. 16*q4+15 in the first 16 lanes of its TMEM quarter; the 16x256b
        // load hands them out in 8x8-matrix fragments (all 32 threads busy: thread t holds rows
        // t/4 and t/4 + 8 of the warp's 16, two adjacent columns per 8-column block), so a pair
        // of columns packs into one word and four blocks go to shared memory per stmatrix.  Of
        // the four 16-column groups, those left of the diagonal are kept whole, the one on the
        // diagonal is masked with a per-thread constant, those right of it are zeros that are
        // not even read.
#pragma unroll
        for (int jp = 0; jp < 4; ++jp) {
          uint32_t m0 = 0u, m1 = 0u, m2 = 0u, m3 = 0u;   // (rows lo, cols j0) (hi, j0) (lo, j1) (hi, j1)
          if (jp <= q4) {
            uint32_t r[8];
            tmem_ld_16x256b_x2(t_lane + kColP + 16 * jp, r);
            tmem_ld_wait();
            m0 = pack_bf16(__uint_as_float(r[0]), __uint_as_float(r[1]));
            m1 = pack_bf16(__uint_as_float(r[2]), __uint_as_float(r[3]));
            m2 = pack_bf16(__uint_as_float(r[4]), __uint_as_float(r[5]));
            m3 = pack_bf16(__uint_as_float(r[6]), __uint_as_float(r[7]));
            if (jp == q4) {   // columns 16*q4 .. 16*q4+15 against rows 16*q4 + t/4 (+ 8)
              m0 &= mask_diag;
              m2 = 0u;
              m3 &= mask_diag;
            }
          }
          stmatrix_x4(ps_mat + (((uint32_t)(2 * jp + mat_j) ^ (uint32_t)mat_k) << 4), m0, m1, m2, m3);
        }
        fence_proxy_async();
        tc_fence_before();
        mbar_arrive(bar(BAR_PREADY));
        // Outputs of this pass.  O^T has the CTA's value columns in the TMEM lanes and the pass's
        // rows in its columns.  The 16x256b load hands out 8x8 fragments [value column][row];
        // stmatrix.trans writes each transposed, 16 bytes (8 value columns) of one output row at
        // a time, into a tile of two 64-column slabs laid out like the operand tiles (128-byte
        // rows, 16-byte chunks swizzled by row & 7: conflict-free), and the tile leaves through
        // tensor copies that undo the swizzle.  Two tiles alternate, so the copies of a pass are
        // still reading while the next pass is written.
        if (!(ok = mbar_wait(bar(BAR_OFULL), ph1, abort_flag, a.hdr))) break;
        tc_fence_after();
        // the copies that read this tile two passes ago have finished reading (with the
        // feed-through, the x' tile that was fetched into it afterwards has landed)
        if (feed) {
          if (!(ok = mbar_wait(bar(BAR_XFULL0 + ph1), (g >> 1) & 1, abort_flag, a.hdr))) break;
        } else {
          if (!(ok = mbar_wait(bar(BAR_OTFREE0 + ph1), ((g >> 1) & 1) ^ 1, abort_flag, a.hdr))) break;
        }
        const uint32_t ot = base + kOffOt + ph1 * kOtBytes;
        // this thread addresses output row 8 * (2 jp + mat_j) + mat_k of column block mat_h
        const uint32_t ot_mat = ot + (q4 >> 1) * kSlabBytes + (mat_j * 8 + mat_k) * 128;
#pragma unroll 1
        for (int hv = 0; hv < 2; ++hv) {                  // lanes 0..15 / 16..31 of the TMEM quarter
          uint32_t r[32];
          tmem_ld_16x256b_x8(t_lane + ((uint32_t)(16 * hv) << 16) + kColO, r);
          tmem_ld_wait();
          if (hv == 1) {                                  // the accumulator is free again
            tc_fence_before();
            mbar_arrive(bar(BAR_OFREE));
          }
          if (!unit_scale) {
#pragma unroll
            for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * a.scale);
          }
          // 16-byte chunk (8 value columns) of this thread's matrices within the slab
          const uint32_t chunk = (uint32_t)(4 * (q4 & 1) + 2 * hv + mat_h);
          const uint32_t dst = ot_mat + ((chunk ^ (uint32_t)mat_k) << 4);
          if (feed) {
            // o = scale q S + d . x': the x' fragments come out of the tile with the transposing
            // matrix load, which hands thread t exactly the elements (value column, row pair) its
            // accumulator registers hold; d belongs to the value column, two per thread
            const float* dh = a.feed_d + (it.seq_head % a.feed_H) * (long long)a.dv + it.col0 + q4 * 32 + 16 * hv + (lane >> 2);
            const float d_lo = __ldg(dh), d_hi = __ldg(dh + 8);
#pragma unroll
            for (int jp = 0; jp < 4; ++jp) {
              uint32_t xf[4];
              ldmatrix_x4_trans(dst + jp * 16 * 128, xf);
#pragma unroll
              for (int mi = 0; mi < 4; ++mi) {            // (lo, j0) (hi, j0) (lo, j1) (hi, j1)
                const int ri = 4 * (2 * jp + (mi >> 1)) + 2 * (mi & 1);
                const float dd = (mi & 1) ? d_hi : d_lo;
                const float2 xv = bf16x2_to_f2(xf[mi]);
                r[ri] = __float_as_uint(fmaf(dd, xv.x, __uint_as_float(r[ri])));
                r[ri + 1] = __float_as_uint(fmaf(dd, xv.y, __uint_as_float(r[ri + 1])));
              }
            }
          }
#pragma unroll
          for (int jp = 0; jp < 4; ++jp) {                // output rows 16 jp .. 16 jp + 15
            const int j0 = 2 * jp, j1 = 2 * jp + 1;
            stmatrix_x4_trans(dst + jp * 16 * 128,
                              pack_bf16(__uint_as_float(r[4 * j0]), __uint_as_float(r[4 * j0 + 1])),
                              pack_bf16(__uint_as_float(r[4 * j0 + 2]), __uint_as_float(r[4 * j0 + 3])),
                              pack_bf16(__uint_as_float(r[4 * j1]), __uint_as_float(r[4 * j1 + 1])),
                              pack_bf16(__uint_as_float(r[4 * j1 + 2]), __uint_as_float(r[4 * j1 + 3])));
          }
        }
        fence_proxy_async();
        mbar_arrive(bar(BAR_OTFULL0 + ph1));
        if (q4 == 0) {
          // One warp sends the tile.  A full tile is two tensor copies (one per slab; the copy
          // engine takes its requests one after another, so few large ones).  A ragged last tile
          // of a sequence goes in boxes of 8 rows and of 1 row, one per lane, so that nothing is
          // written into the rows of the next sequence.
          if (!(ok = mbar_wait(bar(BAR_OTFULL0 + ph1), (g >> 1) & 1, abort_flag, a.hdr))) break;
          if (nr == kC) {
            if (lane < 2) tma_store_2d(&map_o, it.col0 + 64 * lane, (int)row, ot + lane * kSlabBytes);
          } else {
            const int n8 = nr >> 3, n1 = nr & 7;          // at most 7 + 7 boxes per slab
            const int slab = lane & 1, v = lane >> 1;
            if (v < n8)
              tma_store_2d(&map_o8, it.col0 + 64 * slab, (int)row + 8 * v, ot + slab * kSlabBytes + 8 * v * 128);
            else if (v < n8 + n1)
              tma_store_2d(&map_o1, it.col0 + 64 * slab, (int)row + 8 * n8 + (v - n8),
                           ot + slab * kSlabBytes + (8 * n8 + (v - n8)) * 128);
          }
          bulk_commit();
          // the previous pass's copies (the other tile) have finished reading
          bulk_wait_read<1>();
          __syncwarp();
          if (g > 0 && lane == 0) mbar_arrive(bar(BAR_OTFREE0 + (ph1 ^ 1)));
        }
        ++g;
      }
    }
    bulk_wait_read<0>();   // this thread's output copies have read their tile before the CTA may exit
                           // (their writes complete with the kernel)
  } else if (role == 5 || role == 2) {
    // ============================== gate group and its control warp ==============================
    // The gate warps are workers: for every order of the control warp (a stage and a row count)
    // they run phase 1 on their rows, hand in the column sums, wait for their prefix, run phase
    // 2 and report.  Everything serial or rare lives in the control warp: which fill is an
    // attempt, the scan over the 16 row groups, decays, verdict exchange, the copies to the
    // partner, refusals and redirects, publishing the pass.
    const int gw = gw_of_warp;                            // rows kGR*gw .. kGR*gw+kGR-1 of the tile
    const bool is_ctl = role == 2;
    bool ok = true;
    if (!is_ctl) {
      uint32_t off[kGR]; // swizzled byte offsets of the thread's element pairs inside a slab
#pragma unroll
      for (int i = 0; i < kGR; ++i) {
        const int r = gw * kGR + i;
        off[i] = r * 128 + ((((uint32_t)lane >> 2) ^ (r & 7)) << 4) + ((lane & 3) << 2);
      }
      for (uint32_t oc = 0;; ++oc) {                      // order counter
        if (!mbar_wait(bar(BAR_GO0 + (oc & 1)), (oc >> 1) & 1, abort_flag, a.hdr)) break;
        const int s = ctl->ord[oc & 1].stage;
        const int nr = ctl->ord[oc & 1].nr;
        if (s < 0) break;                                 // no more work
        const uint32_t st = stage_base + (uint32_t)s * kStageBytes;
        float* tot = sTot + (oc & 1) * (kGateWarps * kCH) + gw * kCH + 2 * lane;
        float2 b[kGR], eh[kGR];
        const float2 run = gate_phase1<INGATE>(st + kStX, st + kStY, off, gw * kGR, nr, b, eh);
        *reinterpret_cast<float2*>(tot) = run;
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(BAR_GSCAN));
        if (BLOCK && a.beta_hat) {
          // Value gate (Eq. "beta_def"): the v tile becomes beta_hat . v in place, while the
          // control warp scans.  Every gate thread takes its share of 16-byte chunks (8 value columns); the
          // gate comes straight from global memory (asked into L2 when the stage was filled).
          const long long row = ctl->ord[oc & 1].row;
          const int col0 = ctl->ord[oc & 1].col0;
#pragma unroll
          for (int u = 0; u < kC * 16 / (kGateWarps * 32); ++u) {
            const int ci = gw * 32 + lane + kGateWarps * 32 * u;   // chunk of the [64 rows][16 chunks] tile
            const int r = ci >> 4, c16 = ci & 15;
            if (r < nr) {
              const uint4 g4 = __ldg(reinterpret_cast<const uint4*>(
                  a.beta_hat + (row + r) * a.dv + col0 + c16 * 8));
              const uint32_t va = st + kStV + (c16 >> 3) * kSlabBytes + r * 128 +
                                  ((((uint32_t)c16 & 7u) ^ ((uint32_t)r & 7u)) << 4);
              uint4 v4 = lds128(va);
              v4.x = hmul2_bf16(v4.x, g4.x);
              v4.y = hmul2_bf16(v4.y, g4.y);
              v4.z = hmul2_bf16(v4.z, g4.z);
              v4.w = hmul2_bf16(v4.w, g4.w);
              sts128(va, v4.x, v4.y, v4.z, v4.w);
            }
          }
        }
        // the control warp replaces each row group's sum by the sum of the groups before it
        if (!mbar_wait(bar(BAR_PRE), oc & 1, abort_flag, a.hdr)) break;
        const float2 pre = *reinterpret_cast<const float2*>(tot);
        gate_phase2<STATE_ONLY>(st + kStQ, st + kStK, off, gw * kGR, nr, pre, b, eh);
        // the rewritten rows are visible to the bulk-copy engine and to the tensor core; the
        // control warp sends the whole slabs to the partner once every gate warp has said so
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(BAR_ROWS));
      }
    } else {
      const bool leader = lane == 0;
      uint32_t fs = 0, fph = 0;                           // stage and phase of the next fill
      uint32_t g = 0, m = 0, oc = 0;                      // passes, exchanged attempts, orders given
      bool armed = false;                                 // attempt m's receive barriers expect bytes
      uint32_t sent_blk = 0, sent_slab = 0;               // leader: copies issued to the partner
      auto redirect = [&](int jj, int tt) {               // one thread; before the stage is released
        ctl->redir_j = jj;
        ctl->redir_tpos = tt;
        __threadfence_block();
        ctl->redir_seq = ctl->redir_seq + 1;
      };
      // Order number oc goes into slot oc & 1.  The workers read order oc-2 before they reported
      // on it, and at most two orders are outstanding.
      auto give_order = [&](int stage, int nr, long long row = 0, int col0 = 0) {
        if (leader) {
          ctl->ord[oc & 1].stage = stage;
          ctl->ord[oc & 1].nr = nr;
          if (BLOCK) {
            ctl->ord[oc & 1].row = row;
            ctl->ord[oc & 1].col0 = col0;
          }
          mbar_arrive(bar(BAR_GO0 + (oc & 1)));
        }
        ++oc;
      };
      // position of the attempt at hand: CTA-local item index, the item, token, row cap
      int j = 0, tpos = 0, lcap = kC;
      Item it;
      auto seek = [&](int& jj, Item& ii, int& tt) {       // first position at or after (jj, tt) with tokens
        while (item_of(jj) < a.n_items) {
          ii = decode_item(a, item_of(jj), rank);
          if (tt < ii.len) return true;
          ++jj;
          tt = 0;
        }
        return false;
      };
      bool have = seek(j, it, tpos);
      // An order given ahead of time: while the workers are in phase 2 of an attempt, the next
      // fill - if it has landed and is the tile that follows when the attempt is accepted - is
      // ordered at once, so that the workers never wait for the control warp's serial tail
      // (copies to the partner, verdict, publishing).  If the attempt is then refused, the
      // order ahead is carried through (the workers are on it) and its stage handed back unused.
      bool ahead = false;
      uint32_t ahead_s = 0;
      int ahead_nr = 0;
      while (ok && have) {
        uint32_t s;
        int nr;
        const int left = it.len - tpos;
        if (ahead) {
          s = ahead_s;
          nr = ahead_nr;
          ahead = false;
        } else {
          s = fs;
          if (!(ok = mbar_wait(bar(BAR_FULL0 + s), fph, abort_flag, a.hdr))) break;
          if (++fs == kStages) { fs = 0; fph ^= 1; }
          if (ctl->tag[s][0] != j || ctl->tag[s][1] != tpos) {
            // speculative fill for a position we are not at: hand the stage back unused
            if (leader) mbar_arrive_cnt(bar(BAR_EMPTY0 + s), 2);   // nothing was sent from it
            continue;
          }
          nr = min(min(kC, left), lcap);
          give_order((int)s, nr, it.row0 + tpos, it.col0);
        }
        const uint32_t st = stage_base + s * kStageBytes;
        const uint32_t ocur = oc - 1;                     // the order of this attempt
        // ---- the position that follows if this attempt is accepted, and the order ahead
        int nj = j, ntpos = tpos + nr, nlcap = lcap < kC ? min(kC, lcap * 2) : kC;
        Item nit = it;
        const bool nhave = ntpos < it.len ? true : seek(nj, nit, ntpos);
        auto try_ahead = [&]() {
          if (ahead || !nhave || !mbar_test(bar(BAR_FULL0 + fs), fph)) return;
          if (ctl->tag[fs][0] != nj || ctl->tag[fs][1] != ntpos) return;
          ahead = true;
          ahead_s = fs;
          ahead_nr = min(min(kC, nit.len - ntpos), nlcap);
          if (++fs == kStages) { fs = 0; fph ^= 1; }
          give_order((int)ahead_s, ahead_nr, nit.row0 + ntpos, nit.col0);
        };
        // ---- attempt m
        const uint32_t rxi = m & 1, rxph = (m >> 1) & 1;
        float* tot = sTot + (ocur & 1) * (kGateWarps * kCH) + 2 * lane;
        if (!(ok = mbar_wait(bar(BAR_GSCAN), ocur & 1, abort_flag, a.hdr))) break;
        // scan over the row groups (this lane: two channels): each group's sum becomes the sum
        // of the groups before it; the total gives the chunk decays and the verdict
        float2 all = splat(0.f);
        {
          float2 t[kGateWarps];
#pragma unroll
          for (int w = 0; w < kGateWarps; ++w) t[w] = *reinterpret_cast<const float2*>(tot + w * kCH);
#pragma unroll
          for (int w = 0; w < kGateWarps; ++w) {
            *reinterpret_cast<float2*>(tot + w * kCH) = all;
            all = __fadd2_rn(all, t[w]);
          }
        }
        __syncwarp();
        if (leader) mbar_arrive(bar(BAR_PRE));
        try_ahead();                                      // if the next fill had not landed before
        const bool viol_own = __any_sync(0xffffffffu, all.x < -kRange || all.y < -kRange) && nr > 1;
        const float2 D = make_float2(ex2f(all.x), ex2f(all.y));
        // the send block m&1 (like the partner's receive buffer m&1) must be free again
        if (!(ok = mbar_wait_cluster(bar(BAR_RXFREE0 + rxi), rxph ^ 1, abort_flag, a.hdr))) break;
        volatile float* blk = sTx + rxi * kBlkFloats;
        blk[2 * lane] = D.x;
        blk[2 * lane + 1] = D.y;
        if (leader) {
          blk[64] = __int_as_float(viol_own ? 1 : 0);
          blk[65] = __int_as_float((int)s);
        }
        fence_proxy_async();
        __syncwarp();
        if (leader) {
          // the partner's block and slabs complete the two barriers by byte count
          mbar_expect_tx(bar(BAR_VERD0 + rxi), kBlkBytes);
          mbar_expect_tx(bar(BAR_PEER0 + rxi), STATE_ONLY ? kRxBytes - kSlabBytes : kRxBytes);
          armed = true;
          dsmem_bulk_copy(map_to_cta(base + kOffRx + rxi * kBlkBytes, peer),
                          base + kOffTx + rxi * kBlkBytes, kBlkBytes,
                          map_to_cta(bar(BAR_VERD0 + rxi), peer));
          ++sent_blk;
          // the descriptor of the pass this attempt becomes if both CTAs accept it (slot g & 3
          // is not read before its barrier completes; a refused attempt's entry is overwritten)
          volatile PassDesc* pd = &ctl->pd[g & 3];
          pd->stage = (int)s;
          pd->nr = nr;
          pd->flags = (nr == left ? kPassLast : 0);
          pd->rx = (int)rxi;
          pd->rxph = (int)rxph;
          pd->row = it.row0 + tpos;
        }
        // both operand slabs of the attempt go to the partner in one copy each (also when the
        // attempt turns out to be abandoned: the byte count the partner's barrier expects is
        // fixed); the partner's receive buffer m&1 is free, see above
        try_ahead();                                      // second chance: the fill may have landed by now
        if (!(ok = mbar_wait(bar(BAR_ROWS), ocur & 1, abort_flag, a.hdr))) break;
        if (leader) {
          const uint32_t dst = peer_rx_base + rxi * kRxBytes;
          const uint32_t pb = map_to_cta(bar(BAR_PEER0 + rxi), peer);
          if (!STATE_ONLY) dsmem_bulk_copy(map_to_cta(dst + kRxQ, peer), st + kStQ, kSlabBytes, pb);
          dsmem_bulk_copy(map_to_cta(dst + kRxK, peer), st + kStK, kSlabBytes, pb);
          ++sent_slab;
        }
        // both verdicts: the own one and the partner's (came with its decay block)
        if (!(ok = mbar_wait_cluster(bar(BAR_VERD0 + rxi), rxph, abort_flag, a.hdr))) break;
        const bool viol = viol_own || __float_as_int(sRx[rxi * kBlkFloats + 64]) != 0;
        ++m;
        armed = false;
        if (viol) {
          // decays too fast for 'nr' rows at once: ask for this position again, fewer rows
          lcap = max(1, nr >> 1);
          if (ahead) {
            // carry the order ahead through with the workers, then drop it
            const uint32_t oa = oc - 1;
            if (!(ok = mbar_wait(bar(BAR_GSCAN), oa & 1, abort_flag, a.hdr))) break;
            if (leader) mbar_arrive(bar(BAR_PRE));
            if (!(ok = mbar_wait(bar(BAR_ROWS), oa & 1, abort_flag, a.hdr))) break;
            if (leader) mbar_arrive_cnt(bar(BAR_EMPTY0 + ahead_s), 2);
            ahead = false;
          }
          // whatever the partner sent for this attempt must have landed before its buffer
          // and its stage are declared reusable
          if (!(ok = mbar_wait_cluster(bar(BAR_PEER0 + rxi), rxph, abort_flag, a.hdr))) break;
          if (leader) {
            const int peer_stage = __float_as_int(sRx[rxi * kBlkFloats + 65]);
            mbar_arrive_remote(map_to_cta(bar(BAR_EMPTY0 + peer_stage), peer));
            mbar_arrive_remote(map_to_cta(bar(BAR_RXFREE0 + rxi), peer));
            redirect(j, tpos);
            mbar_arrive(bar(BAR_EMPTY0 + s));
          }
          continue;
        }
        // Publish the pass (its descriptor is already written; every gate warp's rows were seen
        // through BAR_ROWS).  With it go the chunk decays of all 128 channels (own half from
        // registers, the partner's from its block) for the state group, in a slot of their
        // own: the stage and the block are recycled sooner.
        {
          float* dp = sDp + (g & 3) * kDK;
          *reinterpret_cast<float2*>(dp + rank * kCH + 2 * lane) = D;
          *reinterpret_cast<float2*>(dp + peer * kCH + 2 * lane) =
              make_float2(sRx[rxi * kBlkFloats + 2 * lane], sRx[rxi * kBlkFloats + 2 * lane + 1]);
          __syncwarp();
        }
        if (leader) {
          if (nr < min(kC, left)) redirect(j, tpos + nr);   // the prefetcher assumed 64 rows
          mbar_arrive(bar(BAR_GATED0 + (g & 3)));
        }
        ++g;
        j = nj;
        it = nit;
        tpos = ntpos;
        lcap = nlcap;
        have = nhave;
      }
      give_order(-1, 0);                                  // the workers leave (also after a failed wait)
      if (leader) {
        ctl->done = 1;
        ctl->sent_blk = (int)sent_blk;                    // for the closing handshake
        ctl->sent_slab = (int)sent_slab;
        ctl->armed_cnt = (int)(m + (armed ? 1u : 0u));
      }
    }
  }

  // ------------------------------------------ teardown ------------------------------------------
  // Normal end: every copy the pair exchanged has been consumed, nothing is in flight.  After a
  // wait that ran out the two CTAs may have stopped anywhere, so they tell each other how far
  // they got and each waits (bounded) for exactly what the other has sent before either leaves;
  // the issuer first lets the contractions it has issued finish, since they read shared memory
  // and write tensor memory that is about to be released.
  tc_fence_before();
  __syncthreads();
  const bool my_abort = ctl->wait.abort_flag != 0;
  if (tid == 0) {
    const uint32_t pc = map_to_cta(smem_u32(const_cast<int*>(&ctl->peer_abort)), peer);
    st_cluster_u32(pc, my_abort ? 1u : 0u);
    st_cluster_u32(pc + 4, (uint32_t)ctl->sent_blk);
    st_cluster_u32(pc + 8, (uint32_t)ctl->sent_slab);
  }
  if (my_abort && role == 1) {
    if (lane == 0) {
      umma_commit(bar(BAR_DRAIN));
      mbar_drain(bar(BAR_DRAIN), 0);
    }
    __syncwarp();
  }
  cluster_arrive();     // release: the stores above; acquire: the partner's
  cluster_wait();
  if (my_abort || ctl->peer_abort) {
    if (tid == 0) {
      const uint32_t nb = (uint32_t)ctl->peer_sent_blk, ns = (uint32_t)ctl->peer_sent_slab;
      const uint32_t top = nb > ns ? nb : ns;
      // receive barriers this CTA never armed, for attempts the partner did send
      for (uint32_t at = (uint32_t)ctl->armed_cnt; at < top; ++at) {
        mbar_expect_tx(bar(BAR_VERD0 + (at & 1)), kBlkBytes);
        mbar_expect_tx(bar(BAR_PEER0 + (at & 1)), STATE_ONLY ? kRxBytes - kSlabBytes : kRxBytes);
      }
      // the last attempt of each parity that was sent: its bytes have landed
      for (uint32_t back = 1; back <= 2; ++back) {
        if (nb >= back) mbar_drain(bar(BAR_VERD0 + ((nb - back) & 1)), ((nb - back) >> 1) & 1);
        if (ns >= back) mbar_drain(bar(BAR_PEER0 + ((ns - back) & 1)), ((ns - back) >> 1) & 1);
      }
    }
    __syncthreads();
    // neither CTA leaves while a copy of the other may still be reading its shared memory
    cluster_arrive();
    cluster_wait();
  }
  if (role == 1) {
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

// [rows, cols] bf16 row-major; box = box_rows rows x 64 columns (128 bytes), 128-byte swizzle.
// Operands and full output tiles use 64-row boxes; ragged output tiles 8-row and 1-row boxes.
bool make_map(CUtensorMap* m, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows = kC) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols * 2};
  const cuuint32_t box[2] = {64u, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct PairMaps {
  CUtensorMap q, k, x, y, v, o, o8, o1;
  CUtensorMap b, fx;   // value gate (only ever prefetched through it) and feed-through input
};

// A tensor map depends only on (address, rows, columns, box rows): each host thread keeps the
// last few it encoded, so that repeated calls on the same buffers (a decode loop's prefill, a
// benchmark) skip the eight driver calls.
struct MapKey {
  const void* ptr;
  uint64_t rows, cols;
  uint32_t box_rows;
};
constexpr int kMapCacheSize = 32;
struct MapCache {
  MapKey key[kMapCacheSize];
  CUtensorMap map[kMapCacheSize];
  int used = 0, next = 0;
};
thread_local MapCache t_maps;

bool cached_map(CUtensorMap* m, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows = kC) {
  MapCache& c = t_maps;
  for (int i = 0; i < c.used; ++i) {
    const MapKey& k = c.key[i];
    if (k.ptr == ptr && k.rows == rows && k.cols == cols && k.box_rows == box_rows) {
      *m = c.map[i];
      return true;
    }
  }
  if (!make_map(m, ptr, rows, cols, box_rows)) return false;
  const int slot = c.next;
  c.key[slot] = MapKey{ptr, rows, cols, box_rows};
  c.map[slot] = *m;
  c.next = (slot + 1) % kMapCacheSize;
  if (c.used < kMapCacheSize) ++c.used;
  return true;
}

template <int INGATE, bool STATE_ONLY, bool BLOCK>
cudaError_t launch_pair(const PairMaps& m, const PairArgs& a, int max_pairs, int dev, cudaStream_t st) {
  static std::atomic<unsigned long long> opted{0};   // one per instantiation
  cudaError_t e = opt_in_shared_memory(ddts_fwd_pair_kernel<INGATE, STATE_ONLY, BLOCK>, kSmemBytes, dev, opted);
  if (e != cudaSuccess) return e;
  const long long pairs = a.n_items < max_pairs ? a.n_items : max_pairs;
  ddts_fwd_pair_kernel<INGATE, STATE_ONLY, BLOCK><<<(unsigned)(2 * pairs), kThreads, kSmemBytes, st>>>(
      m.q, m.k, m.x, m.y, m.v, m.o, m.o8, m.o1, m.b, m.fx, a);
  return cudaGetLastError();
}

}  // namespace

bool fwd_pair_supported(const rodimus_ddts_fwd_params& p) {
  return p.dtype == RODIMUS_BF16 && p.dk == kDK && p.dv % (2 * kDVS) == 0;
}

namespace {

// ---------------------------------------------------------------------------------------------
// Long sequences, few heads: split along time
// ---------------------------------------------------------------------------------------------
// The state recurrence is linear, S_end = D_seg . S_start + dS_seg, where dS_seg is the segment's
// final state from a zero start and D_seg the product of its decays.  When a dense call has fewer
// (sequence, head, 256-column) items than the device has CTA pairs, the sequence is cut into a
// short head segment 0 and G equal segments 1..G that run as separate packed "sequences":
//   launch A   segments 1..G-1 from a zero state, state only: dS_seg and D_seg      } side by side,
//   launch C0  segment 0 from the caller's initial state: outputs, S_start(1)       } two streams
//   combine    S_start(k+1) = D(k) . S_start(k) + dS(k), k = 1..G-1 (elementwise, tiny)
//   launch C   segments 1..G from their true initial states: outputs, final state
// Segment 0 is shorter by the ratio of a state-only pass to a full pass, so that A and C0 end
// together; the whole trades about (2G - 0.35)/(G + 0.65) of the work for G times the parallelism.
struct SplitPlan {
  int G = 0;            // segments after the head segment (0: do not split)
  int L0 = 0;           // rows of the head segment (any number: T - G * L)
  int L = 0;            // rows of each later segment (multiple of the chunk length)
  size_t off_order = 0, off_cu = 0, off_dtot = 0, off_ds = 0, off_start = 0, bytes = 0;
};

constexpr int kMinSegmentRows = 2048;
constexpr int kMaxSegments = 16;
constexpr double kStateOnlyCost = 0.65;  // head segment length relative to the others (state-only pass / full pass; best of a sweep)

SplitPlan make_split_plan(const rodimus_ddts_fwd_params& p) {
  SplitPlan sp;
  if (p.cu_seqlens || p.cu_seqlens_host || !fwd_pair_supported(p)) return sp;
  int dev = 0, sms = 0;
  if (current_device(&dev, &sms) != cudaSuccess) {
    cudaGetLastError();
    return sp;
  }
  const long long items = (long long)p.B * p.H * (p.dv / (2 * kDVS));
  if (items <= 0 || p.T < 2 * kMinSegmentRows) return sp;
  long long g = (sms / 2) / items;
  if (g > p.T / kMinSegmentRows) g = p.T / kMinSegmentRows;
  if (g > kMaxSegments) g = kMaxSegments;
  if (g < 2) return sp;
  int L = (int)((long long)(p.T / (g + kStateOnlyCost)) + kC - 1) / kC * kC;
  if ((long long)g * L >= p.T) L = (int)((p.T / (g + 1)) / kC * kC);   // keep a head segment
  const int L0 = p.T - (int)g * L;
  if (L <= 0 || L0 <= 0) return sp;
  auto up = [](size_t v) { return (v + 255) & ~(size_t)255; };
  const size_t state = (size_t)p.B * p.H * kDK * p.dv * sizeof(float);
  sp.G = (int)g; sp.L0 = L0; sp.L = L;
  sp.off_order = sizeof(WorkspaceHeader);
  sp.off_cu = sp.off_order + up((size_t)(g + 1) * 4);
  sp.off_dtot = sp.off_cu + up((size_t)(g + 2) * 4);
  sp.off_ds = sp.off_dtot + up((size_t)(g - 1) * p.B * p.H * kDK * 4);
  sp.off_start = sp.off_ds + (size_t)(g - 1) * state;
  sp.bytes = sp.off_start + (size_t)g * state;
  return sp;
}

// cu_seqlens of the head segment and the G later ones, and an identity order; clears the status word.
__global__ void ddts_segments_kernel(WorkspaceHeader* hdr, int32_t* order, int32_t* cu, int G, int L0,
                                     int L, int T) {
  const int i = threadIdx.x;
  if (i == 0) hdr->status = RODIMUS_OK;
  if (i <= G) order[i] = i;
  if (i <= G + 1) cu[i] = i == 0 ? 0 : min(L0 + (i - 1) * L, T);
}

// start[0] = S_start(1) is given (final state of the head segment); start[k] = D(k) . start[k-1]
// + dS(k) for k = 1..n, with ds / dtot entry k-1 belonging to segment k.  One thread per four
// state columns of one (batch, head, channel) row; BHD = B*H*dk rows of dv columns.
__global__ void ddts_combine_kernel(const float* __restrict__ ds, const float* __restrict__ dtot,
                                    float* __restrict__ start, int n, long long BHD, int dv) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const int v4 = dv / 4;
  if (idx >= BHD * v4) return;
  const long long row = idx / v4;
  const long long e = row * dv + (idx % v4) * 4;
  const long long seg = BHD * dv;
  float4 s = *reinterpret_cast<const float4*>(start + e);
  for (int k = 1; k <= n; ++k) {
    const float d = dtot[(long long)(k - 1) * BHD + row];
    const float4 t = *reinterpret_cast<const float4*>(ds + (long long)(k - 1) * seg + e);
    s = make_float4(fmaf(d, s.x, t.x), fmaf(d, s.y, t.y), fmaf(d, s.z, t.z), fmaf(d, s.w, t.w));
    *reinterpret_cast<float4*>(start + (long long)k * seg + e) = s;
  }
}

// A second stream and two events per device, so that the two independent launches of the time
// split can run side by side.  Created on first use; if that fails the launches simply follow
// each other on the caller's stream.
struct SideStream {
  bool tried = false, ok = false;
  cudaStream_t stream = nullptr;
  cudaEvent_t fork = nullptr, join = nullptr;
};
constexpr int kMaxDevices = 64;
SideStream g_side[kMaxDevices];
std::mutex g_side_mutex;        // creation of the entries
std::mutex g_side_use_mutex;    // the fork ... join sequence: an event holds the LAST record only, so
                                // two host threads must not interleave their records and waits

SideStream* side_stream(int dev) {
  if (dev < 0 || dev >= kMaxDevices) return nullptr;
  std::lock_guard<std::mutex> lock(g_side_mutex);
  SideStream& s = g_side[dev];
  if (!s.tried) {
    s.tried = true;
    s.ok = cudaStreamCreateWithFlags(&s.stream, cudaStreamNonBlocking) == cudaSuccess &&
           cudaEventCreateWithFlags(&s.fork, cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&s.join, cudaEventDisableTiming) == cudaSuccess;
    if (!s.ok) cudaGetLastError();
  }
  return s.ok ? &s : nullptr;
}

}  // namespace

size_t fwd_pair_split_workspace_bytes(const rodimus_ddts_fwd_params& p) { return make_split_plan(p).bytes; }

cudaError_t launch_fwd_pair(const rodimus_ddts_fwd_params& p, int* n_launches) {
  *n_launches = 0;
  const long long n_seq0 = p.cu_seqlens ? p.N : p.B;
  if (n_seq0 * p.H == 0) return cudaSuccess;
  const uint64_t rows = (uint64_t)p.B * p.H * p.T;
  const uint64_t rows_q = p.shared_gates ? (uint64_t)p.B * p.T : rows;   // rows of q,k,x,y
  cudaStream_t st = reinterpret_cast<cudaStream_t>(p.stream);

  int dev = 0, sms = 0;
  cudaError_t e = current_device(&dev, &sms);
  if (e != cudaSuccess) return e;

  PairMaps m;
  if (rows > 0) {
    const uint64_t dv = (uint64_t)p.dv;
    if (!cached_map(&m.q, p.q, rows_q, kDK) || !cached_map(&m.k, p.k, rows_q, kDK) ||
        !cached_map(&m.x, p.gate_x, rows_q, kDK) || !cached_map(&m.y, p.temp_y, rows_q, kDK) ||
        !cached_map(&m.v, p.v, rows, dv) || !cached_map(&m.o, p.o, rows, dv) ||
        !cached_map(&m.o8, p.o, rows, dv, 8) || !cached_map(&m.o1, p.o, rows, dv, 1))
      return cudaErrorUnknown;
    m.b = m.v;      // placeholders where a term is absent (never used then)
    m.fx = m.v;
    if (p.beta_hat && !cached_map(&m.b, p.beta_hat, rows, dv)) return cudaErrorUnknown;
    if (p.feed_x && !cached_map(&m.fx, p.feed_x, rows, dv)) return cudaErrorUnknown;
  } else {
    memset(&m, 0, sizeof(m));   // never dereferenced: no chunks
  }
  const int max_pairs = sms / 2 > 0 ? sms / 2 : 1;   // one CTA per SM; a pair shares a TPC
  const bool block = p.beta_hat || p.feed_d;
  auto run = [&](const PairArgs& a, cudaStream_t st) {
    const bool g = p.ingate == RODIMUS_INGATE_POW_G;
    if (block) {
      if (a.state_only)
        return g ? launch_pair<RODIMUS_INGATE_POW_G, true, true>(m, a, max_pairs, dev, st)
                 : launch_pair<RODIMUS_INGATE_POW_SIGMOID, true, true>(m, a, max_pairs, dev, st);
      return g ? launch_pair<RODIMUS_INGATE_POW_G, false, true>(m, a, max_pairs, dev, st)
               : launch_pair<RODIMUS_INGATE_POW_SIGMOID, false, true>(m, a, max_pairs, dev, st);
    }
    if (a.state_only)
      return g ? launch_pair<RODIMUS_INGATE_POW_G, true, false>(m, a, max_pairs, dev, st)
               : launch_pair<RODIMUS_INGATE_POW_SIGMOID, true, false>(m, a, max_pairs, dev, st);
    return g ? launch_pair<RODIMUS_INGATE_POW_G, false, false>(m, a, max_pairs, dev, st)
             : launch_pair<RODIMUS_INGATE_POW_SIGMOID, false, false>(m, a, max_pairs, dev, st);
  };
  char* ws = reinterpret_cast<char*>(p.workspace);
  PairArgs a;
  a.o = p.o; a.s0 = p.s0; a.sT = p.sT; a.cu = p.cu_seqlens;
  a.hdr = reinterpret_cast<WorkspaceHeader*>(ws);
  a.order = reinterpret_cast<const int32_t*>(ws + sizeof(WorkspaceHeader));
  a.H = p.H; a.T = p.T; a.dv = p.dv;
  a.n_seq = (int)n_seq0;
  a.pairs = p.dv / (2 * kDVS);
  a.n_items = n_seq0 * p.H * a.pairs;
  a.scale = p.scale;
  a.wait_cycles = main_loop_wait_cycles();
  a.beta_hat = reinterpret_cast<const __nv_bfloat16*>(p.beta_hat);
  a.feed_d = p.feed_d;
  a.feed_H = p.H;
  a.gate_div = p.shared_gates ? p.H : 1;
  a.dtot = nullptr;
  a.sT_only = -1;
  a.state_only = 0;

  const SplitPlan sp = make_split_plan(p);
  if (sp.G < 2 || p.workspace_bytes < sp.bytes) {   // one launch over whole sequences
    e = run(a, st);
    if (e == cudaSuccess) *n_launches = 1;
    return e;
  }
  // ---- split along time: the (batch, head) pairs act as heads of packed sequences
  int32_t* order = reinterpret_cast<int32_t*>(ws + sp.off_order);
  int32_t* cu = reinterpret_cast<int32_t*>(ws + sp.off_cu);
  float* dtot = reinterpret_cast<float*>(ws + sp.off_dtot);
  float* ds = reinterpret_cast<float*>(ws + sp.off_ds);
  float* start = reinterpret_cast<float*>(ws + sp.off_start);
  const int BH = p.B * p.H;
  ddts_segments_kernel<<<1, 32, 0, st>>>(a.hdr, order, cu, sp.G, sp.L0, sp.L, p.T);
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  SideStream* side = side_stream(dev);
  cudaStream_t st0 = st;                             // stream of launch C0
  std::unique_lock<std::mutex> side_use(g_side_use_mutex, std::defer_lock);
  if (side) side_use.lock();
  if (side) {
    if (cudaEventRecord(side->fork, st) == cudaSuccess &&
        cudaStreamWaitEvent(side->stream, side->fork, 0) == cudaSuccess) {
      st0 = side->stream;
    } else {
      cudaGetLastError();
      side = nullptr;
    }
  }
  a.order = order; a.H = BH;
  // Whatever happens after the fork, the side stream is joined back into the caller's stream
  // before this call returns, so that no work of the call is left outside `stream` (and an
  // enclosing stream capture is not left with an unjoined branch).
  auto join = [&]() -> cudaError_t {
    if (!side) return cudaSuccess;
    cudaError_t je = cudaEventRecord(side->join, st0);
    if (je == cudaSuccess) je = cudaStreamWaitEvent(st, side->join, 0);
    side_use.unlock();
    side = nullptr;
    return je;
  };
  // A: local final states and decay products of segments 1..G-1
  a.cu = cu + 1;
  a.n_seq = sp.G - 1;
  a.n_items = (long long)a.n_seq * BH * a.pairs;
  a.s0 = nullptr; a.sT = ds; a.dtot = dtot; a.state_only = 1;
  if ((e = run(a, st)) != cudaSuccess) { join(); return e; }
  // C0: the head segment from the caller's initial state; its final state starts segment 1
  a.cu = cu;
  a.n_seq = 1;
  a.n_items = (long long)BH * a.pairs;
  a.s0 = p.s0; a.sT = start; a.dtot = nullptr; a.state_only = 0;
  e = run(a, st0);
  const cudaError_t je = join();
  if (e != cudaSuccess) return e;
  if (je != cudaSuccess) return je;
  // combine
  {
    const long long BHD = (long long)BH * kDK;
    const long long threads = BHD * (p.dv / 4);
    ddts_combine_kernel<<<(unsigned)((threads + 255) / 256), 256, 0, st>>>(ds, dtot, start, sp.G - 1, BHD, p.dv);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
  }
  // C: segments 1..G from their true initial states
  a.cu = cu + 1;
  a.n_seq = sp.G;
  a.n_items = (long long)a.n_seq * BH * a.pairs;
  a.s0 = start; a.sT = p.sT; a.dtot = nullptr; a.sT_only = sp.G - 1; a.state_only = 0;
  if ((e = run(a, st)) != cudaSuccess) return e;
  *n_launches = 5;
  return cudaSuccess;
}

}  // namespace ddts
