/*
 * rodimus_ddts.h -- C ABI of the B200 (sm_100a) DDTS linear-attention library.
 *
 * The library computes the data-dependent tempered selection (DDTS) recurrence of the
 * Rodimus block (Rodimus paper, Sec. 3.1.2 Eq. "alpha_def" and Sec. 3.1.3
 * Eq. "rodimus_recurrent_form", with the value-side decay beta_t = 1 of Sec. 3.1.1):
 *
 *   g_t = softplus(x_t)      tau_t = sigmoid(y_t)              per key channel
 *   alpha_t = exp(-g_t * tau_t)                                 decay
 *   ahat_t  = g_t ^ tau_t            (RODIMUS_INGATE_POW_G, the paper's Eq. "alpha_def")
 *           = (1 - exp(-g_t)) ^ tau_t   (RODIMUS_INGATE_POW_SIGMOID, alternate reading)
 *   S_t = diag(alpha_t) S_{t-1} + (ahat_t . k_t)^T v_t          S_t is [dk, dv], fp32
 *   o_t = scale * q_t S_t                                       state AFTER the update
 *
 * The projections that produce q, k, v, x, y and the value gate are the caller's.  The value
 * gate beta_hat_t (Eq. "beta_def") and the feed-through d . x'_t of Eq. "rodimus_recurrent_form"
 * can be handed in as optional tensors and are then applied inside the same pass: v_t is
 * multiplied by beta_hat_t where it is loaded, d . x'_t is added to o_t where it is stored.
 *
 * Conventions shared by every entry point
 *   - All data pointers are DEVICE pointers unless a name ends in "_host".
 *   - The caller owns every buffer, the workspace and the stream.  The library allocates no
 *     device memory and never synchronises the device, except rodimus_ddts_device_status,
 *     which waits for the stream it is given.  The only state it keeps between calls is, per
 *     device, one extra stream and two events, created the first time a call is split along
 *     time (see rodimus_ddts_fwd_workspace_bytes); if they cannot be created the split runs
 *     on the caller's stream alone.  Calls from several host threads are allowed (each with
 *     its own buffers, workspace and stream); the enqueueing of split calls is serialised
 *     inside the library.
 *   - Calls enqueue work on `stream` and return; outputs are valid once the stream has
 *     reached that point.
 *   - Every function returns a rodimus_status.  Argument errors are found on the host before
 *     anything is launched.  Nothing aborts, throws or traps.
 *   - Tensors are contiguous, row-major, last index fastest; pointers are 16-byte aligned.
 *   - Inputs must be finite, with |x|, |y| <= 80.  Per-step decay factors below exp(-60) are
 *     applied as exp(-60) by the bf16 prefill kernel (difference below 2^-86 of the state).
 */
#ifndef RODIMUS_DDTS_H_
#define RODIMUS_DDTS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  RODIMUS_OK = 0,
  RODIMUS_ERR_NULL = 1,        /* a required pointer is NULL                                  */
  RODIMUS_ERR_SHAPE = 2,       /* a size is negative, zero where it may not be, or overflows  */
  RODIMUS_ERR_DTYPE = 3,       /* dtype / ingate / struct_size not understood                 */
  RODIMUS_ERR_ALIGN = 4,       /* a pointer is not 16-byte aligned                            */
  RODIMUS_ERR_SEQLENS = 5,     /* cu_seqlens does not start at 0, decreases, or ends != T     */
  RODIMUS_ERR_WORKSPACE = 6,   /* workspace missing or smaller than ..._workspace_bytes       */
  RODIMUS_ERR_UNSUPPORTED = 7, /* dk or dv not a multiple of 16, dk > 256 or dv > 1024        */
  RODIMUS_ERR_CUDA = 8,        /* a CUDA runtime or driver call failed                        */
  RODIMUS_ERR_TIMEOUT = 9      /* a bounded wait inside a kernel ran out (device status only) */
} rodimus_status;

typedef enum { RODIMUS_BF16 = 0, RODIMUS_F32 = 1 } rodimus_dtype; /* of q,k,x,y,v,o alike */

typedef enum {
  RODIMUS_INGATE_POW_G = 0,      /* ahat = g^tau              (Eq. "alpha_def")            */
  RODIMUS_INGATE_POW_SIGMOID = 1 /* ahat = (1-exp(-g))^tau    (alternate reading)          */
} rodimus_ingate;

/*
 * Chunked prefill over whole sequences (appendix "Chunkwise Parallel Representation of the
 * Rodimus Block": intra-chunk masked parallel form plus inter-chunk state recurrence; the
 * chunk length is internal and does not change the result beyond rounding).
 *
 * Dense:  q,k,gate_x,temp_y are [B,H,T,dk]; v,o are [B,H,T,dv]; s0,sT are [B,H,dk,dv].
 * Varlen: cu_seqlens != NULL, B must be 1, the N sequences are packed along T
 *         (sequence n owns rows cu_seqlens[n] .. cu_seqlens[n+1]-1 of every head),
 *         s0,sT are [N,H,dk,dv].  Sequences of length 0 are legal (sT = s0, or zeros).
 * s0 == NULL means a zero initial state; sT == NULL means the final state is not wanted;
 * s0 and sT may be the same buffer.  o must not overlap any input.
 *
 * Kernels: dtype BF16 with dk == 128 and dv a multiple of 128 runs on the tcgen05 tensor
 * cores; every other supported shape (dk, dv multiples of 16, dk <= 256, dv <= 1024) and
 * dtype F32 run the fp32 CUDA-core kernel, which keeps all arithmetic in fp32.
 */
typedef struct {
  int32_t struct_size;       /* sizeof(rodimus_ddts_fwd_params), checked                        */
  int32_t dtype;             /* rodimus_dtype                                                   */
  int32_t ingate;            /* rodimus_ingate                                                  */
  int32_t B, H, T, dk, dv;   /* varlen: B = 1 and T = cu_seqlens[N]; B*H*T < 2^31               */
  float scale;               /* multiplies o; 1.0f when q is already divided by sqrt(dk)        */
  int32_t N;                 /* number of sequences when cu_seqlens != NULL, else ignored       */
  const void *q, *k;         /* device [B,H,T,dk]                                               */
  const void *gate_x;        /* device [B,H,T,dk]: pre-activation of the selection gate g       */
  const void *temp_y;        /* device [B,H,T,dk]: pre-activation of the temperature gate tau   */
  const void *v;             /* device [B,H,T,dv]                                               */
  void *o;                   /* device [B,H,T,dv], written                                      */
  const float *s0;           /* device fp32 [B|N,H,dk,dv] or NULL                               */
  float *sT;                 /* device fp32 [B|N,H,dk,dv] or NULL, written                      */
  const int32_t *cu_seqlens; /* device int32 [N+1] or NULL                                      */
  const int32_t *cu_seqlens_host; /* optional host copy of cu_seqlens: checked before launch.   */
                             /* Without it the device checks the values and reports through     */
                             /* rodimus_ddts_device_status; bad entries are clamped, never read */
                             /* out of bounds.                                                  */
  void *workspace;           /* device, >= rodimus_ddts_fwd_workspace_bytes(), 256-byte aligned */
  size_t workspace_bytes;
  void *stream;              /* cudaStream_t of the caller (NULL = default stream)              */
  /* Optional terms of the full block, fused into the same pass (all NULL = the recurrence alone): */
  const void *beta_hat;      /* device [B,H,T,dv], dtype of v: value gate of Eq. "beta_def", already */
                             /* passed through its sigmoid; v_t enters the state as beta_hat_t * v_t */
  const float *feed_d;       /* device fp32 [H,dv]: feed-through weight d of Eq.                     */
                             /* "rodimus_recurrent_form"; given together with feed_x or not at all   */
  const void *feed_x;        /* device [B,H,T,dv], dtype of v: x'_t; o_t = scale q_t S_t + d . x'_t  */
  int32_t shared_gates;      /* 0: q,k,gate_x,temp_y are [B,H,T,dk], a set per head (above).          */
                             /* 1: the layout Eq. "rodimus_recurrent_form" is written in - decay and   */
                             /* input weight are the same for all value columns (state "n x 2d"):     */
                             /* q,k,gate_x,temp_y are [B,1,T,dk], one set per token shared by the H    */
                             /* groups of dv value columns; v, o, s0, sT keep their H.                 */
  int32_t reserved;          /* 0                                                                    */
  const void *value_decay;   /* optional, device [B,H,T,dv], dtype of v: the value-side decay beta_t of */
                             /* the general transition (Sec. 3.1.1, Eq. "general_state_transition"),    */
                             /* numbers in (0,1]: state element (d,j) decays by alpha_t[d]*beta_t[j].   */
                             /* The paper's model sets beta_t = 1 (NULL) after the ablation of its      */
                             /* table "beta_type"; requests that give it run the fp32 CUDA-core kernel. */
} rodimus_ddts_fwd_params;

/*
 * One decode step for Nseq independent sequences (Eq. "rodimus_recurrent_form" applied once;
 * Sec. 3.1.3, last paragraph: O(1) time and memory per token at inference).
 * q,k,gate_x,temp_y are [Nseq,H,dk]; v,o are [Nseq,H,dv]; state is fp32 [Nseq,H,dk,dv],
 * read and written in place; o reads the updated state.  dk and dv are multiples of 16 with
 * dk <= 256 and dv <= 1024.  All arithmetic is fp32.
 */
typedef struct {
  int32_t struct_size; /* sizeof(rodimus_ddts_step_params) */
  int32_t dtype;       /* rodimus_dtype of q,k,gate_x,temp_y,v,o */
  int32_t ingate;      /* rodimus_ingate */
  int32_t Nseq, H, dk, dv;
  float scale;
  const void *q, *k, *gate_x, *temp_y; /* device [Nseq,H,dk] */
  const void *v;                       /* device [Nseq,H,dv] */
  void *o;                             /* device [Nseq,H,dv], written */
  float *state;                        /* device fp32 [Nseq,H,dk,dv], updated in place */
  void *stream;
  const void *beta_hat;                /* optional, device [Nseq,H,dv]: value gate (see the prefill) */
  const float *feed_d;                 /* optional, device fp32 [H,dv]: feed-through weight          */
  const void *feed_x;                  /* optional with feed_d, device [Nseq,H,dv]: x'_t             */
  int32_t shared_gates;                /* 1: q,k,gate_x,temp_y are [Nseq,1,dk] (see the prefill)     */
  int32_t reserved;                    /* 0                                                          */
  const void *value_decay;             /* optional, device [Nseq,H,dv]: value-side decay beta_t      */
                                       /* (see the prefill); NULL = 1                                */
} rodimus_ddts_step_params;

/* Bytes of device workspace rodimus_ddts_fwd needs for these sizes (pointers are not read).
 * Returns 0 if the sizes are not valid.
 * For a dense bf16 call with long sequences and fewer (sequence, head) units than the device
 * has SM pairs, the size includes room for per-segment states: given that much, the call cuts
 * the sequences into time segments that run side by side (the state recurrence is linear in
 * the state, so segments are joined exactly up to rounding) and part of the work is enqueued
 * on the library's own second stream, forked from and joined back into `stream` with events, so
 * the call still behaves as one piece of work on `stream`.  A caller that passes less (never
 * less than 256 bytes plus 4 bytes per packed sequence, rounded up to 256) gets the same
 * result from a single launch. */
size_t rodimus_ddts_fwd_workspace_bytes(const rodimus_ddts_fwd_params *p);

/* Chunked prefill; see rodimus_ddts_fwd_params. */
int rodimus_ddts_fwd(const rodimus_ddts_fwd_params *p);

/* One-token decode; see rodimus_ddts_step_params. */
int rodimus_ddts_step(const rodimus_ddts_step_params *p);

/*
 * Backward pass of the prefill: the gradient of a scalar loss L with respect to every input of
 * rodimus_ddts_fwd, given d_o = dL/do and d_sT = dL/dS_T.  The paper trains the block through
 * the chunkwise form (appendix "Chunkwise Parallel Representation of the Rodimus Block") and
 * prints no backward formulas; the result is defined by Eq. "alpha_def" and
 * Eq. "rodimus_recurrent_form" and computed as the adjoint of the chunkwise form (chunk length
 * internal): a forward sweep over the chunks carries S and yields dq, a reverse sweep carries
 * dL/dS and yields dk and dv, and the gradients of the two gates follow from suffix sums of
 * q . dq - (ahat k) . d(ahat k) over the sequence.
 *
 * Layouts as rodimus_ddts_fwd_params (dense, or packed with cu_seqlens and B = 1).  Inputs:
 * q,k,gate_x,temp_y [B,H,T,dk], v and d_o [B,H,T,dv] in `dtype`; s0 and d_sT fp32 [B|N,H,dk,dv]
 * or NULL (zero).  Outputs, written: d_q,d_k,d_gate_x,d_temp_y [B,H,T,dk] and d_v [B,H,T,dv] in
 * `dtype`; d_s0 fp32 [B|N,H,dk,dv] or NULL (not wanted).  No output may overlap an input.
 * Supported widths: dk = 128 and dv = 256 (others: RODIMUS_ERR_UNSUPPORTED); the value gate,
 * the feed-through and the shared-gate layout of the forward call have no backward here.
 * dtype BF16 contracts tf32 operands on the tensor cores with fp32 accumulation; dtype F32
 * splits each operand in two tf32 parts and keeps fp32 accuracy.  The workspace holds the
 * status word, 8 * dk bytes per token and head of scratch, and 6 * dk/2 * dv * 4 bytes per
 * (sequence, head): each sweep may be cut into time segments that run as thread blocks of their
 * own and hand their slice of the state to the next one through that area.  A segment waits
 * for the one before it under the same limit as every other wait (rodimus_ddts_test_set_wait_limit);
 * if that ran out the status word holds RODIMUS_ERR_TIMEOUT and the outputs are unspecified.
 */
typedef struct {
  int32_t struct_size;       /* sizeof(rodimus_ddts_bwd_params), checked                        */
  int32_t dtype;             /* rodimus_dtype of q,k,gate_x,temp_y,v,d_o and of the d_ outputs  */
  int32_t ingate;            /* rodimus_ingate                                                  */
  int32_t B, H, T, dk, dv;
  float scale;
  int32_t N;                 /* number of sequences when cu_seqlens != NULL                     */
  const void *q, *k, *gate_x, *temp_y; /* device [B,H,T,dk]: the forward call's inputs          */
  const void *v;             /* device [B,H,T,dv]                                               */
  const float *s0;           /* device fp32 [B|N,H,dk,dv] or NULL: the forward's initial state  */
  const void *d_o;           /* device [B,H,T,dv]: dL/do                                        */
  const float *d_sT;         /* device fp32 [B|N,H,dk,dv] or NULL: dL/dS_T                      */
  void *d_q, *d_k, *d_gate_x, *d_temp_y; /* device [B,H,T,dk], written                          */
  void *d_v;                 /* device [B,H,T,dv], written                                      */
  float *d_s0;               /* device fp32 [B|N,H,dk,dv] or NULL, written                      */
  const int32_t *cu_seqlens; /* device int32 [N+1] or NULL                                      */
  const int32_t *cu_seqlens_host; /* optional host copy, checked before launch (see the prefill) */
  void *workspace;           /* device, >= rodimus_ddts_bwd_workspace_bytes(), 256-byte aligned */
  size_t workspace_bytes;
  void *stream;
} rodimus_ddts_bwd_params;

/* Bytes of device workspace rodimus_ddts_bwd needs (pointers are not read, except that a
 * non-NULL cu_seqlens or cu_seqlens_host marks the call as packed); 0 if the sizes are not valid
 * or not supported. */
size_t rodimus_ddts_bwd_workspace_bytes(const rodimus_ddts_bwd_params *p);

/* Backward pass; see rodimus_ddts_bwd_params.  The device-side status (cu_seqlens check) is read
 * with rodimus_ddts_device_status as for the prefill. */
int rodimus_ddts_bwd(const rodimus_ddts_bwd_params *p);

/*
 * Sliding-window shared-key attention (SW-SKA), the attention half of the Rodimus+ block
 * (Sec. "Shared-Key Attention for Lossless Head Compression": softmax attention,
 * Eq. "attention_parallel", with one key per token shared by all heads, queries and values per
 * head; combined with a sliding window):
 *
 *   s_ti = scale * <q^h_t, k_i>,  t - window < i <= t      p_ti = softmax over those i
 *   o^h_t = sum_i p_ti v^h_i
 *
 * q, v, o are [B,H,T,d]; k is [B,T,d] (no head index).  d = 128 (the paper's head size; other
 * sizes: RODIMUS_ERR_UNSUPPORTED); window >= 1 (the paper uses half the training context); dense
 * batches only.  dtype BF16 runs on the tcgen05 tensor cores with a running softmax (cost
 * O(T * window), nothing of size T x window is stored); dtype F32 is a plain fp32 validation
 * kernel.  Inputs must be finite (a tile may span the rows of two heads; what lies outside a
 * query's window is weighted by zero, which a NaN or infinity would not survive).  o must not
 * overlap an input.  `workspace` is optional: given (>= 256 bytes, 256-byte
 * aligned), its first word is the status rodimus_ddts_device_status reads (RODIMUS_ERR_TIMEOUT
 * if a bounded wait inside the kernel ran out; outputs are then unspecified).
 */
typedef struct {
  int32_t struct_size; /* sizeof(rodimus_swska_fwd_params), checked */
  int32_t dtype;       /* rodimus_dtype of q, k, v, o */
  int32_t B, H, T, d;
  int32_t window;      /* tokens a query sees, itself included */
  float scale;         /* multiplies the scores, > 0; 1/sqrt(d) for the usual attention */
  const void *q;       /* device [B,H,T,d] */
  const void *k;       /* device [B,T,d] */
  const void *v;       /* device [B,H,T,d] */
  void *o;             /* device [B,H,T,d], written */
  void *stream;
  void *workspace;     /* optional device status area, see above */
  size_t workspace_bytes;
} rodimus_swska_fwd_params;

int rodimus_swska_fwd(const rodimus_swska_fwd_params *p);

/*
 * rodimus_ddts_fwd for callers that cannot allocate device memory.  (A convenience of this
 * library: the paper has no counterpart.)
 *
 * Who needs it: code that receives only input and output buffers and has no allocator to turn
 * to -- a plug-in inside an application that distributed all device memory at start-up, a
 * serving loop that must never hit cudaMalloc's device-wide synchronisation, a runtime that
 * forbids allocation after initialisation.  rodimus_ddts_fwd needs a small workspace from its
 * caller; this variant uses a fixed array inside the library's device image instead
 * (256 + 4 * RODIMUS_NOALLOC_MAX_SEQS bytes, present on every GPU that loads the library, for
 * the life of the process).  It allocates and frees nothing, on the device or through any
 * library.
 *
 * p is read exactly as by rodimus_ddts_fwd, except that p->workspace and p->workspace_bytes are
 * ignored.  Limit: a packed (cu_seqlens) call may hold at most RODIMUS_NOALLOC_MAX_SEQS
 * sequences; more returns RODIMUS_ERR_WORKSPACE before anything is launched.  Every other
 * status is that of rodimus_ddts_fwd; RODIMUS_ERR_CUDA also covers a failed look-up of the
 * array's address.
 *
 * The first call on each device looks up that device's address of the array (with the device
 * current, once, under a lock); make that first call outside any stream capture.
 *
 * All calls on a device share the one array, and it keeps the previous call's contents.  Nothing
 * in it needs clearing by the caller: each call rewrites what it later reads.  But two calls
 * whose kernels may overlap on the GPU (different streams, no dependency) race on it; order
 * them.
 *
 * status_handle, if not NULL, receives a device pointer to pass as `workspace` to
 * rodimus_ddts_device_status (NULL if the call failed); it stays valid until the next call on
 * the same device overwrites what it points at.
 */
#define RODIMUS_NOALLOC_MAX_SEQS 4096
int rodimus_ddts_fwd_noalloc(const rodimus_ddts_fwd_params *p, const void **status_handle);

/*
 * Waits for `stream`, then returns what the kernels of the last rodimus_ddts_fwd call that
 * used `workspace` recorded: RODIMUS_OK, RODIMUS_ERR_SEQLENS (device-side cu_seqlens check)
 * or RODIMUS_ERR_TIMEOUT (a bounded wait ran out; outputs are then unspecified).
 */
int rodimus_ddts_device_status(const void *workspace, void *stream);

/* How many kernels the last successful rodimus_ddts_fwd / _bwd / _step call on this host
 * thread launched (for benchmarks that report launch counts). */
int rodimus_ddts_last_launch_count(void);

/* Name of the kernel family the given prefill request would run: "tcgen05", "simt" or
 * "invalid".  Pointers are not read. */
const char *rodimus_ddts_fwd_kernel_name(const rodimus_ddts_fwd_params *p);

/* Diagnostic for benchmarks (the paper has no counterpart): enqueues on `stream` one launch that
 * does nothing but special-function-unit approximations (ex2), `iters` rounds of 8 per thread
 * on a grid that fills the device, and stores in *ops (host) how many it will execute.  The
 * caller times the launch with events: ops / time is the rate that bounds the gate math
 * (softplus, sigmoid, logarithms and exponentials of Eq. "alpha_def") of the prefill kernels.
 * `sink` is one device float (written only in a case that does not occur).  iters in 1 .. 2^24. */
int rodimus_ddts_sfu_probe(int iters, float *sink, void *stream, long long *ops);

/* Test hook (the paper has no counterpart).  Every wait inside the tensor-core prefill kernels,
 * the attention kernel and between the time segments of the backward sweeps is bounded: when one runs out, the kernel stops early, frees what it holds and records
 * RODIMUS_ERR_TIMEOUT in the workspace status word (outputs are then unspecified, the device
 * stays usable).  The bound is a launch argument of about two seconds' worth of clock cycles;
 * this call replaces it, process-wide, for the launches that follow: 0 makes the first wait that
 * is not satisfied at once run out, which is how the tests reach that path without hanging
 * anything; a negative value restores the default.  Not for production use. */
int rodimus_ddts_test_set_wait_limit(long long cycles);

const char *rodimus_status_str(int status);
int rodimus_version(void);

#ifdef __cplusplus
}
#endif
#endif /* RODIMUS_DDTS_H_ */
