"""ctypes front end of the fp64 CPU oracle (``ddts_ref.c``) plus two slow numpy
restatements of other forms the paper gives for the same quantity.

TEST INFRASTRUCTURE ONLY: tests, the smoke check and the benchmark's CPU-baseline
leg may import this module; the CUDA library and its Python binding never do.

* ``ref_fwd`` / ``ref_step`` / ``ref_gates`` call the sequential recurrence
  (Eq. "alpha_def", Eq. "rodimus_recurrent_form").
* ``ref_bwd`` calls the adjoint of that recurrence, statement by statement in reverse order
  (the gradient of a scalar loss with respect to q, k, x, y, v and the initial state).
* ``parallel_form`` is the O(T^2) masked form of the appendix on the chunkwise
  representation (Eq. "rodimus_parallel_form"), for one sequence and one head.
* ``unrolled_sum`` is the double sum obtained by unfolding the general gated
  transition (Sec. 3.1.1, the equation after "general_state_transition").

The last two exist to pin the first: they are written from different equations and
share no code with it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ddts_ref.c")
_LIB = os.path.join(_HERE, "libddts_ref.so")
_lock = threading.Lock()
_lib = None

POW_G = 0        # ahat = g ** tau                (paper, Eq. "alpha_def")
POW_SIGMOID = 1  # ahat = (1 - exp(-g)) ** tau    (alternate reading)


def build(force: bool = False) -> str:
    """Compile ``ddts_ref.c`` into ``libddts_ref.so`` beside it (gcc, OpenMP)."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + f".tmp{os.getpid()}"
            cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        f32p = ctypes.POINTER(ctypes.c_float)
        f64p = ctypes.POINTER(ctypes.c_double)
        i32p = ctypes.POINTER(ctypes.c_int32)
        lib.ddts_ref_gates.argtypes = [ctypes.c_int, ctypes.c_int64, f32p, f32p, f64p, f64p]
        lib.ddts_ref_gates.restype = ctypes.c_int
        lib.ddts_ref_fwd.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int64,
                                     ctypes.c_int, ctypes.c_int, ctypes.c_double,
                                     f32p, f32p, f32p, f32p, f32p, f64p, f64p, f64p, i32p,
                                     ctypes.c_int]
        lib.ddts_ref_fwd.restype = ctypes.c_int
        lib.ddts_ref_fwd_block.argtypes = lib.ddts_ref_fwd.argtypes + [f32p, f32p, f32p]
        lib.ddts_ref_fwd_block.restype = ctypes.c_int
        lib.ddts_ref_fwd_shared.argtypes = lib.ddts_ref_fwd_block.argtypes
        lib.ddts_ref_fwd_shared.restype = ctypes.c_int
        lib.ddts_ref_fwd_vdecay.argtypes = lib.ddts_ref_fwd_block.argtypes + [f32p, ctypes.c_int]
        lib.ddts_ref_fwd_vdecay.restype = ctypes.c_int
        lib.ddts_ref_step.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                      ctypes.c_int, ctypes.c_double,
                                      f32p, f32p, f32p, f32p, f32p, f64p, f64p]
        lib.ddts_ref_step.restype = ctypes.c_int
        lib.ddts_ref_step_block.argtypes = lib.ddts_ref_step.argtypes + [f32p, f32p, f32p]
        lib.ddts_ref_step_block.restype = ctypes.c_int
        lib.ddts_ref_step_shared.argtypes = lib.ddts_ref_step_block.argtypes
        lib.ddts_ref_step_shared.restype = ctypes.c_int
        lib.ddts_ref_step_vdecay.argtypes = lib.ddts_ref_step_block.argtypes + [f32p, ctypes.c_int]
        lib.ddts_ref_step_vdecay.restype = ctypes.c_int
        lib.ddts_ref_bwd.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int64,
                                     ctypes.c_int, ctypes.c_int, ctypes.c_double,
                                     f32p, f32p, f32p, f32p, f32p, f64p, f32p, f64p,
                                     f64p, f64p, f64p, f64p, f64p, f64p, i32p, ctypes.c_int]
        lib.ddts_ref_bwd.restype = ctypes.c_int
        lib.ddts_ref_num_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a, a.ctypes.data_as(ctypes.POINTER(ctypes.c_float))


def _f64p(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double)) if a is not None else None


def num_threads() -> int:
    return int(_load().ddts_ref_num_threads())


def ref_gates(x, y, ingate: int = POW_G):
    """alpha = exp(-softplus(x) * sigmoid(y)) and ahat, element by element (fp64)."""
    lib = _load()
    xa, xp = _f32(x)
    ya, yp = _f32(y)
    alpha = np.empty(xa.shape, dtype=np.float64)
    ahat = np.empty(xa.shape, dtype=np.float64)
    rc = lib.ddts_ref_gates(ingate, xa.size, xp, yp, _f64p(alpha), _f64p(ahat))
    if rc:
        raise ValueError(f"ddts_ref_gates returned {rc}")
    return alpha, ahat


def ref_fwd(q, k, x, y, v, s0=None, cu_seqlens=None, scale: float = 1.0, ingate: int = POW_G,
            want_o: bool = True, want_sT: bool = True, beta_hat=None, feed_d=None, feed_x=None,
            shared_gates: bool = False, value_decay=None):
    """Sequential prefill.  q,k,x,y: [B,H,T,dk]; v: [B,H,T,dv]; s0: [B|N,H,dk,dv] or None.

    Optional terms of the full block: beta_hat [B,H,T,dv] (value gate, Eq. "beta_def": v_t is
    replaced by beta_hat_t * v_t) and the feed-through feed_d [H,dv], feed_x [B,H,T,dv]
    (Eq. "rodimus_recurrent_form": o_t = scale * q_t S_t + d * x'_t).

    shared_gates: the layout the paper writes the block in - q,k,x,y are [B,1,T,dk], one set per
    token shared by all H groups of dv value columns (v, o, states keep their H).

    value_decay: beta_t in (0,1], [B,H,T,dv]: the value-side decay of the general transition
    (Eq. "general_state_transition"): state element (d, j) decays by alpha_t[d] * beta_t[j].  The
    paper's model sets it to 1; this is its ablation arm.

    Returns (o [B,H,T,dv] float64 or None, sT [B|N,H,dk,dv] float64 or None).
    """
    lib = _load()
    qa, qp = _f32(q)
    ka, kp = _f32(k)
    xa, xp = _f32(x)
    ya, yp = _f32(y)
    va, vp = _f32(v)
    B, Hq, T, dk = qa.shape
    H = va.shape[1]
    dv = va.shape[-1]
    assert ka.shape == qa.shape == xa.shape == ya.shape and va.shape[:3] == (B, H, T)
    assert Hq == (1 if shared_gates else H)
    cu = None
    cup = None
    nseq = B
    N = 0
    if cu_seqlens is not None:
        cu = np.ascontiguousarray(cu_seqlens, dtype=np.int32)
        N = cu.size - 1
        nseq = N
        cup = cu.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))
    s0a = None
    if s0 is not None:
        s0a = np.ascontiguousarray(s0, dtype=np.float64)
        assert s0a.shape == (nseq, H, dk, dv)
    o = np.empty((B, H, T, dv), dtype=np.float64) if want_o else None
    sT = np.empty((nseq, H, dk, dv), dtype=np.float64) if want_sT else None
    if beta_hat is None and feed_d is None and feed_x is None and not shared_gates \
            and value_decay is None:
        rc = lib.ddts_ref_fwd(ingate, B, H, T, dk, dv, float(scale), qp, kp, xp, yp, vp,
                              _f64p(s0a), _f64p(o), _f64p(sT), cup, N)
    elif value_decay is not None:
        assert (feed_d is None) == (feed_x is None)
        ba, bp = (None, None) if beta_hat is None else _f32(beta_hat)
        da, dp = (None, None) if feed_d is None else _f32(feed_d)
        fa, fp = (None, None) if feed_x is None else _f32(feed_x)
        ga, gp = _f32(value_decay)
        assert ga.shape == va.shape and (ba is None or ba.shape == va.shape)
        rc = lib.ddts_ref_fwd_vdecay(ingate, B, H, T, dk, dv, float(scale), qp, kp, xp, yp, vp,
                                     _f64p(s0a), _f64p(o), _f64p(sT), cup, N, bp, dp, fp, gp,
                                     1 if shared_gates else 0)
    else:
        assert (feed_d is None) == (feed_x is None)
        ba, bp = (None, None) if beta_hat is None else _f32(beta_hat)
        da, dp = (None, None) if feed_d is None else _f32(feed_d)
        fa, fp = (None, None) if feed_x is None else _f32(feed_x)
        assert ba is None or ba.shape == va.shape
        assert da is None or (da.shape == (H, dv) and fa.shape == va.shape)
        fn = lib.ddts_ref_fwd_shared if shared_gates else lib.ddts_ref_fwd_block
        rc = fn(ingate, B, H, T, dk, dv, float(scale), qp, kp, xp, yp, vp,
                _f64p(s0a), _f64p(o), _f64p(sT), cup, N, bp, dp, fp)
    if rc:
        raise ValueError(f"ddts_ref_fwd returned {rc}")
    return o, sT


def ref_step(q, k, x, y, v, state, scale: float = 1.0, ingate: int = POW_G, beta_hat=None,
             feed_d=None, feed_x=None, shared_gates: bool = False, value_decay=None):
    """One decode step; ``state`` ([Nseq,H,dk,dv] float64, C-contiguous) is updated in place.
    beta_hat, feed_x: [Nseq,H,dv]; feed_d: [H,dv] (optional, as in ``ref_fwd``)."""
    lib = _load()
    qa, qp = _f32(q)
    ka, kp = _f32(k)
    xa, xp = _f32(x)
    ya, yp = _f32(y)
    va, vp = _f32(v)
    Nseq, Hq, dk = qa.shape
    H = va.shape[1]
    dv = va.shape[-1]
    assert Hq == (1 if shared_gates else H)     # shared: q,k,x,y are [Nseq,1,dk]
    assert state.dtype == np.float64 and state.flags["C_CONTIGUOUS"]
    assert state.shape == (Nseq, H, dk, dv)
    o = np.empty((Nseq, H, dv), dtype=np.float64)
    if beta_hat is None and feed_d is None and feed_x is None and not shared_gates \
            and value_decay is None:
        rc = lib.ddts_ref_step(ingate, Nseq, H, dk, dv, float(scale), qp, kp, xp, yp, vp,
                               _f64p(o), _f64p(state))
    elif value_decay is not None:
        ba, bp = (None, None) if beta_hat is None else _f32(beta_hat)
        da, dp = (None, None) if feed_d is None else _f32(feed_d)
        fa, fp = (None, None) if feed_x is None else _f32(feed_x)
        ga, gp = _f32(value_decay)
        rc = lib.ddts_ref_step_vdecay(ingate, Nseq, H, dk, dv, float(scale), qp, kp, xp, yp, vp,
                                      _f64p(o), _f64p(state), bp, dp, fp, gp,
                                      1 if shared_gates else 0)
    else:
        assert (feed_d is None) == (feed_x is None)
        ba, bp = (None, None) if beta_hat is None else _f32(beta_hat)
        da, dp = (None, None) if feed_d is None else _f32(feed_d)
        fa, fp = (None, None) if feed_x is None else _f32(feed_x)
        fn = lib.ddts_ref_step_shared if shared_gates else lib.ddts_ref_step_block
        rc = fn(ingate, Nseq, H, dk, dv, float(scale), qp, kp, xp, yp, vp,
                _f64p(o), _f64p(state), bp, dp, fp)
    if rc:
        raise ValueError(f"ddts_ref_step returned {rc}")
    return o


def ref_bwd(q, k, x, y, v, do, s0=None, dsT=None, cu_seqlens=None, scale: float = 1.0,
            ingate: int = POW_G, want_ds0: bool = True):
    """Gradients of L for given do = dL/do [B,H,T,dv] and dsT = dL/dS_T [B|N,H,dk,dv] (or None).

    Layouts as ``ref_fwd``.  Returns a dict of float64 arrays: dq, dk, dx, dy [B,H,T,dk],
    dv [B,H,T,dv], ds0 [B|N,H,dk,dv] (None unless wanted).
    """
    lib = _load()
    qa, qp = _f32(q)
    ka, kp = _f32(k)
    xa, xp = _f32(x)
    ya, yp = _f32(y)
    va, vp = _f32(v)
    da, dp = _f32(do)
    B, H, T, dk = qa.shape
    dv = va.shape[-1]
    assert ka.shape == qa.shape == xa.shape == ya.shape and va.shape == da.shape == (B, H, T, dv)
    cup = None
    nseq = B
    N = 0
    if cu_seqlens is not None:
        cu = np.ascontiguousarray(cu_seqlens, dtype=np.int32)
        N = cu.size - 1
        nseq = N
        cup = cu.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))
    s0a = None if s0 is None else np.ascontiguousarray(s0, dtype=np.float64)
    dsa = None if dsT is None else np.ascontiguousarray(dsT, dtype=np.float64)
    assert s0a is None or s0a.shape == (nseq, H, dk, dv)
    assert dsa is None or dsa.shape == (nseq, H, dk, dv)
    out = {n: np.zeros((B, H, T, dk), dtype=np.float64) for n in ("dq", "dk", "dx", "dy")}
    out["dv"] = np.zeros((B, H, T, dv), dtype=np.float64)
    out["ds0"] = np.zeros((nseq, H, dk, dv), dtype=np.float64) if want_ds0 else None
    rc = lib.ddts_ref_bwd(ingate, B, H, T, dk, dv, float(scale), qp, kp, xp, yp, vp, _f64p(s0a),
                          dp, _f64p(dsa), _f64p(out["dq"]), _f64p(out["dk"]), _f64p(out["dx"]),
                          _f64p(out["dy"]), _f64p(out["dv"]), _f64p(out["ds0"]), cup, N)
    if rc:
        raise ValueError(f"ddts_ref_bwd returned {rc}")
    return out


# ----------------------------------------------------------------------------------------------
# Other forms of the same quantity, written from other equations (pins for the recurrence above).
# ----------------------------------------------------------------------------------------------

def _gates_np(x, y, ingate):
    x = np.asarray(x, dtype=np.float64)
    y = np.asarray(y, dtype=np.float64)
    g = np.logaddexp(0.0, x)
    tau = 1.0 / (1.0 + np.exp(-y))
    log_alpha = -g * tau
    if ingate == POW_G:
        ahat = np.power(g, tau)
    else:
        ahat = np.power(-np.expm1(-g), tau)
    return log_alpha, ahat


def parallel_form(q, k, x, y, v, scale: float = 1.0, ingate: int = POW_G):
    """O = ((Q . A)(K / A . ahat)^T . M) V for ONE sequence and head, zero initial state.

    Eq. "rodimus_parallel_form": A_t is the cumulative product of alpha up to t and M the
    causal mask with the diagonal kept.  The quotient A_t / A_i is formed per pair as the
    exponential of a difference of prefix sums of log(alpha), never as a division.
    q,k,x,y: [T,dk]; v: [T,dv]; returns [T,dv] float64.
    """
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    log_alpha, ahat = _gates_np(x, y, ingate)
    cum = np.cumsum(log_alpha, axis=0)                      # log A_t, [T,dk]
    T = q.shape[0]
    # scores[t,i] = sum_d q[t,d] * k[i,d] * ahat[i,d] * exp(cum[t,d] - cum[i,d])
    diff = cum[:, None, :] - cum[None, :, :]                 # [T,T,dk]
    mask = np.tril(np.ones((T, T), dtype=bool))
    w = np.where(mask[:, :, None], np.exp(np.where(mask[:, :, None], diff, 0.0)), 0.0)
    scores = np.einsum("td,id,tid->ti", q, k * ahat, w)
    return scale * (scores @ v)


def unrolled_sum(q, k, x, y, v, scale: float = 1.0, ingate: int = POW_G, value_decay=None,
                 beta_hat=None):
    """o_t = sum_{i<=t} [q_t (prod_{j=i+1..t} alpha_j . ahat_i . k_i)^T]
                        (prod_{j=i+1..t} beta_j . beta_hat_i . v_i), by explicit loops.

    Sec. 3.1.1, the equation obtained by unfolding the general transition; beta (value_decay,
    [T,dv]) and beta_hat ([T,dv]) default to 1.  Pure Python loops: tiny inputs only.
    """
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    log_alpha, ahat = _gates_np(x, y, ingate)
    alpha = np.exp(log_alpha)
    T, dk = q.shape
    beta = None if value_decay is None else np.asarray(value_decay, dtype=np.float64)
    bhat = None if beta_hat is None else np.asarray(beta_hat, dtype=np.float64)
    o = np.zeros((T, v.shape[1]), dtype=np.float64)
    for t in range(T):
        for i in range(t + 1):
            prod = np.ones(dk)
            vprod = np.ones(v.shape[1])
            for j in range(i + 1, t + 1):
                prod = prod * alpha[j]
                if beta is not None:
                    vprod = vprod * beta[j]
            vi = v[i] if bhat is None else bhat[i] * v[i]
            o[t] += float(np.dot(q[t], prod * ahat[i] * k[i])) * (vprod * vi)
    return scale * o
