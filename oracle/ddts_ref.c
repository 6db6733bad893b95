/*
 * ddts_ref.c -- fp64 CPU oracle for the DDTS linear-attention recurrence.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
 * CUDA library is checked against.  It shares no code with the CUDA path and
 * must never be called from it; only the tests, the smoke check and the
 * benchmark's CPU-baseline leg load it.
 *
 * What it computes (Rodimus paper, Eq. "alpha_def" of Sec. 3.1.2 and
 * Eq. "rodimus_recurrent_form" of Sec. 3.1.3, with the value-side decay
 * beta_t = 1 as Sec. 3.1.1 chooses; the value gate beta_hat of Eq. "beta_def" and
 * the feed-through term d . x' of Eq. "rodimus_recurrent_form" are optional inputs
 * of the ..._block entry points: v_t is replaced by beta_hat_t . v_t and d . x'_t is
 * added to o_t; their projections stay with the caller; the ..._vdecay entry points also take the
 * value-side decay beta_t of the general transition, Eq. "general_state_transition", as numbers):
 *
 *   g_t     = softplus(x_t)                    selection gate,   per key channel
 *   tau_t   = sigmoid(y_t)                     temperature gate, per key channel
 *   alpha_t = exp(-g_t * tau_t)                decay
 *   ahat_t  = g_t ^ tau_t                      input weight (paper, mode 0)
 *           = (1 - exp(-g_t)) ^ tau_t          input weight (alternate, mode 1)
 *   S_t[d,:] = alpha_t[d] * S_{t-1}[d,:] + (ahat_t[d] * k_t[d]) * v_t[:]
 *   o_t[:]   = scale * sum_d q_t[d] * S_t[d,:]          (state AFTER the update)
 *
 * Strictly sequential in t, no chunking, no reordering: one loop per symbol of
 * the equations.  Inputs arrive as float (the caller has already rounded them to
 * the dtype the GPU sees, so input rounding is not counted as error) and are
 * promoted to double before any arithmetic.  Outputs and states are double.
 *
 * Parity pins (tests, CPU only): equality with the O(T^2) masked parallel form
 * (App. "Chunkwise Parallel Representation", Eq. "rodimus_parallel_form") and with
 * the unrolled double sum of Sec. 3.1.1, reduction to unnormalised causal linear
 * attention when alpha = ahat = 1, a geometric-series closed form, T = 1 by hand,
 * the gate identities of Sec. 3.1.2 and the derivative product of the
 * selection-mechanism proof, linearity, prefill == repeated steps == split runs.
 * The choice between the two input-weight modes cannot be pinned by a printed
 * value (the paper prints no worked example): for that choice alone, "parity
 * unpinned"; both modes are implemented and each is pinned by every other test.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { DDTS_REF_POW_G = 0, DDTS_REF_POW_SIGMOID = 1 };

/* softplus(x) = log(1 + e^x), written so that neither branch overflows. */
static double ref_softplus(double x) {
  return x > 0.0 ? x + log1p(exp(-x)) : log1p(exp(x));
}

/* sigmoid(y) = 1 / (1 + e^-y). */
static double ref_sigmoid(double y) {
  if (y >= 0.0) return 1.0 / (1.0 + exp(-y));
  double e = exp(y);
  return e / (1.0 + e);
}

/* Eq. "alpha_def": one key channel of one token. */
static void ref_gate(int ingate, double x, double y, double *alpha, double *ahat) {
  double g = ref_softplus(x);
  double tau = ref_sigmoid(y);
  *alpha = exp(-g * tau);
  if (ingate == DDTS_REF_POW_G) {
    *ahat = pow(g, tau);
  } else {
    *ahat = pow(-expm1(-g), tau); /* 1 - exp(-g) */
  }
}

/* Gates of n (token, channel) pairs; exported so that tests can pin them alone. */
int ddts_ref_gates(int ingate, int64_t n, const float *x, const float *y, double *alpha,
                   double *ahat) {
  if (ingate != DDTS_REF_POW_G && ingate != DDTS_REF_POW_SIGMOID) return 3;
  for (int64_t i = 0; i < n; ++i) ref_gate(ingate, (double)x[i], (double)y[i], &alpha[i], &ahat[i]);
  return 0;
}

/* One sequence, one head: rows [0,len) of q,k,x,y (row stride dk) and v,o (row stride dv). */
/* Optional terms of the full block (Eq. "beta_def", Eq. "rodimus_recurrent_form"): bh, rows of
 * the value gate beta_hat (multiplies v_t element by element), and the feed-through d . x'_t
 * added to o_t after the scaling (d: one weight per value column, fx: rows of x').  NULL = absent,
 * and then the arithmetic is exactly that of the plain recurrence. */
static void ref_one_sequence(int ingate, int64_t len, int dk, int dv, double scale, const float *q,
                             const float *k, const float *x, const float *y, const float *v,
                             const double *s0, double *o, double *sT, double *S, const float *bh,
                             const float *d_feed, const float *fx, const float *bd) {
  if (s0)
    memcpy(S, s0, sizeof(double) * (size_t)dk * dv);
  else
    memset(S, 0, sizeof(double) * (size_t)dk * dv);
  for (int64_t t = 0; t < len; ++t) {
    const float *qt = q + t * dk, *kt = k + t * dk, *xt = x + t * dk, *yt = y + t * dk;
    const float *vt = v + t * dv;
    double *ot = o ? o + t * dv : NULL;
    if (ot)
      for (int j = 0; j < dv; ++j) ot[j] = 0.0;
    for (int d = 0; d < dk; ++d) {
      double alpha, ahat;
      ref_gate(ingate, (double)xt[d], (double)yt[d], &alpha, &ahat);
      double w = ahat * (double)kt[d];
      double *Sd = S + (size_t)d * dv;
      if (bd) {
        /* value-side decay beta_t of Eq. "general_state_transition": the state element (d, j)
         * decays by alpha_t[d] * beta_t[j]; the input term is as below */
        const float *dt = bd + t * dv;
        for (int j = 0; j < dv; ++j) {
          double vj = bh ? (double)bh[t * dv + j] * (double)vt[j] : (double)vt[j];
          Sd[j] = (alpha * (double)dt[j]) * Sd[j] + w * vj;
        }
      } else if (bh) {
        const float *bt = bh + t * dv;
        for (int j = 0; j < dv; ++j) Sd[j] = alpha * Sd[j] + w * ((double)bt[j] * (double)vt[j]);
      } else {
        for (int j = 0; j < dv; ++j) Sd[j] = alpha * Sd[j] + w * (double)vt[j];
      }
      if (ot) {
        double qd = (double)qt[d];
        for (int j = 0; j < dv; ++j) ot[j] += qd * Sd[j];
      }
    }
    if (ot) {
      for (int j = 0; j < dv; ++j) ot[j] *= scale;
      if (d_feed && fx) {
        const float *ft = fx + t * dv;
        for (int j = 0; j < dv; ++j) ot[j] += (double)d_feed[j] * (double)ft[j];
      }
    }
  }
  if (sT) memcpy(sT, S, sizeof(double) * (size_t)dk * dv);
}

/*
 * Prefill.  Dense: q,k,x,y are [B,H,T,dk], v,o are [B,H,T,dv], s0/sT are
 * [B,H,dk,dv] (either may be NULL: zero initial state / final state not wanted).
 * Varlen (cu_seqlens != NULL): B must be 1, the N sequences are packed along T,
 * sequence n owns rows cu_seqlens[n] .. cu_seqlens[n+1]-1 of every head, and
 * s0/sT are [N,H,dk,dv].  o may be NULL (state only).  Returns 0, or a nonzero
 * code for arguments that make no sense.
 */
/* shared != 0: the layout the paper writes the block in (Eq. "rodimus_recurrent_form": the decay
 * exp(-g.tau)^T 1_m and the input weight multiply ALL m value columns, Table of A_t/B_t: state
 * "n x 2d"): one q, k, x, y of width dk per token, [B,1,T,dk], shared by the H groups of dv value
 * columns; v, o and the states keep their H.  Each group then runs the same recurrence. */
static int ref_fwd_impl(int ingate, int B, int H, int64_t T, int dk, int dv, double scale,
                        const float *q, const float *k, const float *x, const float *y,
                        const float *v, const double *s0, double *o, double *sT,
                        const int32_t *cu_seqlens, int N, const float *beta_hat,
                        const float *feed_d, const float *feed_x, int shared,
                        const float *value_decay) {
  if (ingate != DDTS_REF_POW_G && ingate != DDTS_REF_POW_SIGMOID) return 3;
  if (B < 0 || H < 0 || T < 0 || dk <= 0 || dv <= 0) return 2;
  int nseq = B;
  if (cu_seqlens) {
    if (B != 1 || N < 0) return 2;
    if (cu_seqlens[0] != 0 || cu_seqlens[N] != T) return 5;
    for (int n = 0; n < N; ++n)
      if (cu_seqlens[n + 1] < cu_seqlens[n]) return 5;
    nseq = N;
  }
  int64_t items = (int64_t)nseq * H;
  int failed = 0;
#pragma omp parallel
  {
    double *S = (double *)malloc(sizeof(double) * (size_t)dk * dv);
    if (!S) {
#pragma omp atomic write
      failed = 1;
    }
#pragma omp for schedule(dynamic, 1)
    for (int64_t it = 0; it < items; ++it) {
      if (!S) continue;
      int64_t n = it / H, h = it % H;
      int64_t row0, len;
      if (cu_seqlens) {
        row0 = h * T + cu_seqlens[n];
        len = cu_seqlens[n + 1] - cu_seqlens[n];
      } else {
        row0 = (n * H + h) * T;
        len = T;
      }
      size_t so = (size_t)it * dk * dv;
      /* rows of q, k, x, y: the head's own, or the single shared set of the sequence */
      int64_t rq = row0;
      if (shared) rq = cu_seqlens ? (int64_t)cu_seqlens[n] : n * T;
      ref_one_sequence(ingate, len, dk, dv, scale, q + rq * dk, k + rq * dk, x + rq * dk,
                       y + rq * dk, v + row0 * dv, s0 ? s0 + so : NULL, o ? o + row0 * dv : NULL,
                       sT ? sT + so : NULL, S, beta_hat ? beta_hat + row0 * dv : NULL,
                       feed_d ? feed_d + (size_t)h * dv : NULL, feed_x ? feed_x + row0 * dv : NULL,
                       value_decay ? value_decay + row0 * dv : NULL);
    }
    free(S);
  }
  return failed ? 8 : 0;
}

int ddts_ref_fwd_block(int ingate, int B, int H, int64_t T, int dk, int dv, double scale,
                       const float *q, const float *k, const float *x, const float *y,
                       const float *v, const double *s0, double *o, double *sT,
                       const int32_t *cu_seqlens, int N, const float *beta_hat,
                       const float *feed_d, const float *feed_x) {
  return ref_fwd_impl(ingate, B, H, T, dk, dv, scale, q, k, x, y, v, s0, o, sT, cu_seqlens, N,
                      beta_hat, feed_d, feed_x, 0, NULL);
}

/* The general transition of Sec. 3.1.1 (Eq. "general_state_transition") with a value-side decay
 * beta_t in (0,1]^dv, [B,H,T,dv], handed in as numbers: S_t = (alpha_t^T beta_t) . S_{t-1} +
 * (ahat_t . k_t)^T (beta_hat_t . v_t).  The paper sets beta_t = 1 after its ablation (table
 * "beta_type"); this entry point exists for that ablation arm.  shared: as ddts_ref_fwd_shared. */
int ddts_ref_fwd_vdecay(int ingate, int B, int H, int64_t T, int dk, int dv, double scale,
                        const float *q, const float *k, const float *x, const float *y,
                        const float *v, const double *s0, double *o, double *sT,
                        const int32_t *cu_seqlens, int N, const float *beta_hat,
                        const float *feed_d, const float *feed_x, const float *value_decay,
                        int shared) {
  return ref_fwd_impl(ingate, B, H, T, dk, dv, scale, q, k, x, y, v, s0, o, sT, cu_seqlens, N,
                      beta_hat, feed_d, feed_x, shared, value_decay);
}

/* Shared-gate layout: q, k, x, y are [B,1,T,dk]; everything else as ddts_ref_fwd_block. */
int ddts_ref_fwd_shared(int ingate, int B, int H, int64_t T, int dk, int dv, double scale,
                        const float *q, const float *k, const float *x, const float *y,
                        const float *v, const double *s0, double *o, double *sT,
                        const int32_t *cu_seqlens, int N, const float *beta_hat,
                        const float *feed_d, const float *feed_x) {
  return ref_fwd_impl(ingate, B, H, T, dk, dv, scale, q, k, x, y, v, s0, o, sT, cu_seqlens, N,
                      beta_hat, feed_d, feed_x, 1, NULL);
}

/* The recurrence alone (no value gate, no feed-through). */
int ddts_ref_fwd(int ingate, int B, int H, int64_t T, int dk, int dv, double scale, const float *q,
                 const float *k, const float *x, const float *y, const float *v, const double *s0,
                 double *o, double *sT, const int32_t *cu_seqlens, int N) {
  return ddts_ref_fwd_block(ingate, B, H, T, dk, dv, scale, q, k, x, y, v, s0, o, sT, cu_seqlens,
                            N, NULL, NULL, NULL);
}

/*
 * One decode step for Nseq independent sequences: q,k,x,y are [Nseq,H,dk], v,o are
 * [Nseq,H,dv], state is [Nseq,H,dk,dv] and is updated in place; o reads the state
 * after the update (Eq. "rodimus_recurrent_form": o_t = q_t S_t).
 */
static int ref_step_impl(int ingate, int Nseq, int H, int dk, int dv, double scale, const float *q,
                         const float *k, const float *x, const float *y, const float *v, double *o,
                         double *state, const float *beta_hat, const float *feed_d,
                         const float *feed_x, int shared, const float *value_decay) {
  if (ingate != DDTS_REF_POW_G && ingate != DDTS_REF_POW_SIGMOID) return 3;
  if (Nseq < 0 || H < 0 || dk <= 0 || dv <= 0) return 2;
  int64_t items = (int64_t)Nseq * H;
#pragma omp parallel for schedule(static)
  for (int64_t it = 0; it < items; ++it) {
    const int64_t iq = shared ? it / H : it; /* shared: one q, k, x, y per sequence, [Nseq,1,dk] */
    const float *qt = q + iq * dk, *kt = k + iq * dk, *xt = x + iq * dk, *yt = y + iq * dk;
    const float *vt = v + it * dv;
    double *ot = o + it * dv;
    double *S = state + (size_t)it * dk * dv;
    for (int j = 0; j < dv; ++j) ot[j] = 0.0;
    for (int d = 0; d < dk; ++d) {
      double alpha, ahat;
      ref_gate(ingate, (double)xt[d], (double)yt[d], &alpha, &ahat);
      double w = ahat * (double)kt[d];
      double qd = (double)qt[d];
      double *Sd = S + (size_t)d * dv;
      if (value_decay) {
        const float *dt = value_decay + it * dv;
        for (int j = 0; j < dv; ++j) {
          double vj = beta_hat ? (double)beta_hat[it * dv + j] * (double)vt[j] : (double)vt[j];
          Sd[j] = (alpha * (double)dt[j]) * Sd[j] + w * vj;
          ot[j] += qd * Sd[j];
        }
      } else if (beta_hat) {
        const float *bt = beta_hat + it * dv;
        for (int j = 0; j < dv; ++j) {
          Sd[j] = alpha * Sd[j] + w * ((double)bt[j] * (double)vt[j]);
          ot[j] += qd * Sd[j];
        }
      } else {
        for (int j = 0; j < dv; ++j) {
          Sd[j] = alpha * Sd[j] + w * (double)vt[j];
          ot[j] += qd * Sd[j];
        }
      }
    }
    for (int j = 0; j < dv; ++j) ot[j] *= scale;
    if (feed_d && feed_x) {
      const float *dh = feed_d + (size_t)(it % H) * dv, *ft = feed_x + it * dv;
      for (int j = 0; j < dv; ++j) ot[j] += (double)dh[j] * (double)ft[j];
    }
  }
  return 0;
}

int ddts_ref_step_block(int ingate, int Nseq, int H, int dk, int dv, double scale, const float *q,
                        const float *k, const float *x, const float *y, const float *v, double *o,
                        double *state, const float *beta_hat, const float *feed_d,
                        const float *feed_x) {
  return ref_step_impl(ingate, Nseq, H, dk, dv, scale, q, k, x, y, v, o, state, beta_hat, feed_d,
                       feed_x, 0, NULL);
}

/* Decode step with the value-side decay beta_t [Nseq,H,dv] (see ddts_ref_fwd_vdecay). */
int ddts_ref_step_vdecay(int ingate, int Nseq, int H, int dk, int dv, double scale, const float *q,
                         const float *k, const float *x, const float *y, const float *v, double *o,
                         double *state, const float *beta_hat, const float *feed_d,
                         const float *feed_x, const float *value_decay, int shared) {
  return ref_step_impl(ingate, Nseq, H, dk, dv, scale, q, k, x, y, v, o, state, beta_hat, feed_d,
                       feed_x, shared, value_decay);
}

/* Shared-gate layout for decode: q, k, x, y are [Nseq,1,dk]. */
int ddts_ref_step_shared(int ingate, int Nseq, int H, int dk, int dv, double scale, const float *q,
                         const float *k, const float *x, const float *y, const float *v, double *o,
                         double *state, const float *beta_hat, const float *feed_d,
                         const float *feed_x) {
  return ref_step_impl(ingate, Nseq, H, dk, dv, scale, q, k, x, y, v, o, state, beta_hat, feed_d,
                       feed_x, 1, NULL);
}

int ddts_ref_step(int ingate, int Nseq, int H, int dk, int dv, double scale, const float *q,
                  const float *k, const float *x, const float *y, const float *v, double *o,
                  double *state) {
  return ddts_ref_step_block(ingate, Nseq, H, dk, dv, scale, q, k, x, y, v, o, state, NULL, NULL,
                             NULL);
}

/*
 * Backward pass: the gradient of a scalar loss L with respect to every input of the prefill,
 * given dL/do (rows of do) and dL/dS_T (dsT).  The paper trains the block through the
 * chunkwise form (App. "Chunkwise Parallel Representation of the Rodimus Block") and prints no
 * backward formulas: the quantity is defined by the forward equations above, and this is their
 * adjoint written step by step, in reverse order of t, one statement per forward statement:
 *
 *   forward, step t, channel d:   w = ahat * k ;  S_t[d,:] = alpha * S_{t-1}[d,:] + w * v_t[:]
 *                                 o_t[:] = scale * sum_d q_t[d] * S_t[d,:]
 *   adjoint (G = dL/dS_t, starts at dsT and ends as dL/dS_0):
 *     G[d,:]   += scale * q_t[d] * do_t[:]             dq_t[d] = scale * sum_j S_t[d,j] do_t[j]
 *     dalpha    = sum_j G[d,j] * S_{t-1}[d,j]          dw      = sum_j G[d,j] * v_t[j]
 *     dv_t[:]  += w * G[d,:]                           G[d,:] *= alpha         (now dL/dS_{t-1})
 *     dk_t[d]   = dw * ahat ;  dahat = dw * k_t[d]
 *     alpha = exp(-g tau):   dg  = -tau * alpha * dalpha ;  dtau  = -g * alpha * dalpha
 *     ahat  = u^tau      :   dg += tau * u^(tau-1) * u'(g) * dahat ;  dtau += ahat * ln(u) * dahat
 *                            (u = g, u' = 1 in mode 0;  u = 1 - e^-g, u' = e^-g in mode 1)
 *     dx_t[d] = dg * sigmoid(x) ;  dy_t[d] = dtau * tau * (1 - tau)
 *
 * The states S_{t-1}, S_t that the adjoint needs are the forward's own: they are recomputed with
 * the same statements from stored copies taken every kBwdBlock steps (storage only; no step is
 * reordered or merged).  Pins (tests, CPU only): central finite differences of ddts_ref_fwd,
 * reverse-mode differentiation of a separately written forward by an autograd library, linearity
 * in (do, dsT), the chain of two half-length calls through ds0 -> dsT, T = 1 by hand.
 */
enum { kBwdBlock = 32 };

/* One forward step of one sequence, the statements of ref_one_sequence without the outputs. */
static void ref_state_step(int ingate, int dk, int dv, const float *kt, const float *xt,
                           const float *yt, const float *vt, const double *Sin, double *Sout) {
  for (int d = 0; d < dk; ++d) {
    double alpha, ahat;
    ref_gate(ingate, (double)xt[d], (double)yt[d], &alpha, &ahat);
    double w = ahat * (double)kt[d];
    const double *a = Sin + (size_t)d * dv;
    double *b = Sout + (size_t)d * dv;
    for (int j = 0; j < dv; ++j) b[j] = alpha * a[j] + w * (double)vt[j];
  }
}

static int ref_bwd_one_sequence(int ingate, int64_t len, int dk, int dv, double scale,
                                const float *q, const float *k, const float *x, const float *y,
                                const float *v, const double *s0, const float *dout,
                                const double *dsT, double *dq, double *dkk, double *dx, double *dy,
                                double *dvv, double *ds0) {
  const size_t sz = (size_t)dk * dv;
  const int64_t nblk = (len + kBwdBlock - 1) / kBwdBlock;
  double *ck = (double *)malloc(sizeof(double) * sz * (size_t)(nblk + 1));
  double *Sb = (double *)malloc(sizeof(double) * sz * (kBwdBlock + 1));
  double *G = (double *)malloc(sizeof(double) * sz);
  if (!ck || !Sb || !G) {
    free(ck); free(Sb); free(G);
    return 8;
  }
  /* forward: the state at the start of every block */
  if (s0) memcpy(ck, s0, sizeof(double) * sz); else memset(ck, 0, sizeof(double) * sz);
  memcpy(Sb, ck, sizeof(double) * sz);
  for (int64_t t = 0; t < len; ++t) {
    double *cur = Sb + (size_t)(t & 1) * sz, *nxt = Sb + (size_t)((t + 1) & 1) * sz;
    ref_state_step(ingate, dk, dv, k + t * dk, x + t * dk, y + t * dk, v + t * dv, cur, nxt);
    if ((t + 1) % kBwdBlock == 0) memcpy(ck + sz * (size_t)((t + 1) / kBwdBlock), nxt, sizeof(double) * sz);
  }
  if (dsT) memcpy(G, dsT, sizeof(double) * sz); else memset(G, 0, sizeof(double) * sz);

  for (int64_t blk = nblk - 1; blk >= 0; --blk) {
    const int64_t t0 = blk * kBwdBlock;
    const int n = (int)((len - t0) < kBwdBlock ? (len - t0) : kBwdBlock);
    memcpy(Sb, ck + sz * (size_t)blk, sizeof(double) * sz);
    for (int i = 0; i < n; ++i) {
      const int64_t t = t0 + i;
      ref_state_step(ingate, dk, dv, k + t * dk, x + t * dk, y + t * dk, v + t * dv,
                     Sb + sz * (size_t)i, Sb + sz * (size_t)(i + 1));
    }
    for (int i = n - 1; i >= 0; --i) {
      const int64_t t = t0 + i;
      const double *Sprev = Sb + sz * (size_t)i, *Scur = Sb + sz * (size_t)(i + 1);
      const float *qt = q + t * dk, *kt = k + t * dk, *xt = x + t * dk, *yt = y + t * dk;
      const float *vt = v + t * dv, *dot = dout + t * dv;
      double *dvt = dvv + t * dv;
      for (int j = 0; j < dv; ++j) dvt[j] = 0.0;
      for (int d = 0; d < dk; ++d) {
        const double g = ref_softplus((double)xt[d]), tau = ref_sigmoid((double)yt[d]);
        double alpha, ahat;
        ref_gate(ingate, (double)xt[d], (double)yt[d], &alpha, &ahat);
        const double w = ahat * (double)kt[d];
        double *Gd = G + (size_t)d * dv;
        const double *Sp = Sprev + (size_t)d * dv, *Sc = Scur + (size_t)d * dv;
        double dqd = 0.0, dalpha = 0.0, dw = 0.0;
        for (int j = 0; j < dv; ++j) {
          Gd[j] += scale * (double)qt[d] * (double)dot[j];
          dqd += Sc[j] * (double)dot[j];
        }
        for (int j = 0; j < dv; ++j) {
          dalpha += Gd[j] * Sp[j];
          dw += Gd[j] * (double)vt[j];
          dvt[j] += w * Gd[j];
          Gd[j] *= alpha;
        }
        dq[t * dk + d] = scale * dqd;
        dkk[t * dk + d] = dw * ahat;
        const double dahat = dw * (double)kt[d];
        double dg = -tau * alpha * dalpha, dtau = -g * alpha * dalpha;
        double u, du;
        if (ingate == DDTS_REF_POW_G) {
          u = g; du = 1.0;
        } else {
          u = -expm1(-g); du = exp(-g);
        }
        dg += tau * pow(u, tau - 1.0) * du * dahat;
        dtau += ahat * log(u) * dahat;
        dx[t * dk + d] = dg * ref_sigmoid((double)xt[d]);
        dy[t * dk + d] = dtau * tau * (1.0 - tau);
      }
    }
  }
  if (ds0) memcpy(ds0, G, sizeof(double) * sz);
  free(ck); free(Sb); free(G);
  return 0;
}

/*
 * Layouts as ddts_ref_fwd (dense, or packed with cu_seqlens and B = 1).  dout is [B,H,T,dv]
 * (float, already rounded to the GPU's input type), dsT [B|N,H,dk,dv] or NULL (zero).  Outputs,
 * all double: dq, dk, dx, dy [B,H,T,dk], dv [B,H,T,dv], ds0 [B|N,H,dk,dv] or NULL (not wanted).
 */
int ddts_ref_bwd(int ingate, int B, int H, int64_t T, int dk, int dv, double scale, const float *q,
                 const float *k, const float *x, const float *y, const float *v, const double *s0,
                 const float *dout, const double *dsT, double *dq, double *dkk, double *dx,
                 double *dy, double *dvv, double *ds0, const int32_t *cu_seqlens, int N) {
  if (ingate != DDTS_REF_POW_G && ingate != DDTS_REF_POW_SIGMOID) return 3;
  if (B < 0 || H < 0 || T < 0 || dk <= 0 || dv <= 0) return 2;
  int nseq = B;
  if (cu_seqlens) {
    if (B != 1 || N < 0) return 2;
    if (cu_seqlens[0] != 0 || cu_seqlens[N] != T) return 5;
    for (int n = 0; n < N; ++n)
      if (cu_seqlens[n + 1] < cu_seqlens[n]) return 5;
    nseq = N;
  }
  int64_t items = (int64_t)nseq * H;
  int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t it = 0; it < items; ++it) {
    int64_t n = it / H, h = it % H;
    int64_t row0, len;
    if (cu_seqlens) {
      row0 = h * T + cu_seqlens[n];
      len = cu_seqlens[n + 1] - cu_seqlens[n];
    } else {
      row0 = (n * H + h) * T;
      len = T;
    }
    size_t so = (size_t)it * dk * dv;
    int rc = ref_bwd_one_sequence(ingate, len, dk, dv, scale, q + row0 * dk, k + row0 * dk,
                                  x + row0 * dk, y + row0 * dk, v + row0 * dv, s0 ? s0 + so : NULL,
                                  dout + row0 * dv, dsT ? dsT + so : NULL, dq + row0 * dk,
                                  dkk + row0 * dk, dx + row0 * dk, dy + row0 * dk, dvv + row0 * dv,
                                  ds0 ? ds0 + so : NULL);
    if (rc) {
#pragma omp atomic write
      failed = 1;
    }
  }
  return failed ? 8 : 0;
}

/* Threads the parallel regions above will use (1 without OpenMP). */
int ddts_ref_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}
