"""Python binding of the DDTS CUDA library: argument marshalling only.

Every step of the path runs in the kernels behind the C ABI of ``include/rodimus_ddts.h``;
PyTorch is used for device memory and streams.  There is no CPU fallback: if the shared
library has not been built, or no CUDA device is present, calls raise.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "librodimus_ddts.so")

# status codes / enums of the header
OK, ERR_NULL, ERR_SHAPE, ERR_DTYPE, ERR_ALIGN, ERR_SEQLENS, ERR_WORKSPACE, ERR_UNSUPPORTED, \
    ERR_CUDA, ERR_TIMEOUT = range(10)
BF16, F32 = 0, 1
INGATE_POW_G, INGATE_POW_SIGMOID = 0, 1

EXPORTED_SYMBOLS = (
    "rodimus_ddts_fwd_workspace_bytes", "rodimus_ddts_fwd", "rodimus_ddts_step",
    "rodimus_ddts_device_status", "rodimus_ddts_last_launch_count",
    "rodimus_ddts_fwd_kernel_name", "rodimus_status_str", "rodimus_version",
    "rodimus_ddts_fwd_noalloc", "rodimus_ddts_sfu_probe", "rodimus_ddts_test_set_wait_limit",
    "rodimus_ddts_bwd_workspace_bytes", "rodimus_ddts_bwd", "rodimus_swska_fwd",
)
NOALLOC_MAX_SEQS = 4096


class RodimusError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: status {status} ({status_str(status)})")


class FwdParams(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_int32), ("dtype", ctypes.c_int32), ("ingate", ctypes.c_int32),
        ("B", ctypes.c_int32), ("H", ctypes.c_int32), ("T", ctypes.c_int32),
        ("dk", ctypes.c_int32), ("dv", ctypes.c_int32),
        ("scale", ctypes.c_float), ("N", ctypes.c_int32),
        ("q", ctypes.c_void_p), ("k", ctypes.c_void_p),
        ("gate_x", ctypes.c_void_p), ("temp_y", ctypes.c_void_p),
        ("v", ctypes.c_void_p), ("o", ctypes.c_void_p),
        ("s0", ctypes.c_void_p), ("sT", ctypes.c_void_p),
        ("cu_seqlens", ctypes.c_void_p), ("cu_seqlens_host", ctypes.c_void_p),
        ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t),
        ("stream", ctypes.c_void_p),
        ("beta_hat", ctypes.c_void_p), ("feed_d", ctypes.c_void_p), ("feed_x", ctypes.c_void_p),
        ("shared_gates", ctypes.c_int32), ("reserved", ctypes.c_int32),
        ("value_decay", ctypes.c_void_p),
    ]


class StepParams(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_int32), ("dtype", ctypes.c_int32), ("ingate", ctypes.c_int32),
        ("Nseq", ctypes.c_int32), ("H", ctypes.c_int32), ("dk", ctypes.c_int32),
        ("dv", ctypes.c_int32), ("scale", ctypes.c_float),
        ("q", ctypes.c_void_p), ("k", ctypes.c_void_p),
        ("gate_x", ctypes.c_void_p), ("temp_y", ctypes.c_void_p),
        ("v", ctypes.c_void_p), ("o", ctypes.c_void_p),
        ("state", ctypes.c_void_p), ("stream", ctypes.c_void_p),
        ("beta_hat", ctypes.c_void_p), ("feed_d", ctypes.c_void_p), ("feed_x", ctypes.c_void_p),
        ("shared_gates", ctypes.c_int32), ("reserved", ctypes.c_int32),
        ("value_decay", ctypes.c_void_p),
    ]


class BwdParams(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_int32), ("dtype", ctypes.c_int32), ("ingate", ctypes.c_int32),
        ("B", ctypes.c_int32), ("H", ctypes.c_int32), ("T", ctypes.c_int32),
        ("dk", ctypes.c_int32), ("dv", ctypes.c_int32),
        ("scale", ctypes.c_float), ("N", ctypes.c_int32),
        ("q", ctypes.c_void_p), ("k", ctypes.c_void_p),
        ("gate_x", ctypes.c_void_p), ("temp_y", ctypes.c_void_p),
        ("v", ctypes.c_void_p), ("s0", ctypes.c_void_p),
        ("d_o", ctypes.c_void_p), ("d_sT", ctypes.c_void_p),
        ("d_q", ctypes.c_void_p), ("d_k", ctypes.c_void_p),
        ("d_gate_x", ctypes.c_void_p), ("d_temp_y", ctypes.c_void_p),
        ("d_v", ctypes.c_void_p), ("d_s0", ctypes.c_void_p),
        ("cu_seqlens", ctypes.c_void_p), ("cu_seqlens_host", ctypes.c_void_p),
        ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t),
        ("stream", ctypes.c_void_p),
    ]


class SwskaParams(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_int32), ("dtype", ctypes.c_int32),
        ("B", ctypes.c_int32), ("H", ctypes.c_int32), ("T", ctypes.c_int32), ("d", ctypes.c_int32),
        ("window", ctypes.c_int32), ("scale", ctypes.c_float),
        ("q", ctypes.c_void_p), ("k", ctypes.c_void_p), ("v", ctypes.c_void_p),
        ("o", ctypes.c_void_p), ("stream", ctypes.c_void_p),
        ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t),
    ]


_lib = None


def load_library() -> ctypes.CDLL:
    """Loads ``librodimus_ddts.so`` (built by ``paper_2410_06577_b200.build``); raises if absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: run `python -m paper_2410_06577_b200.build` "
                "(there is no fallback path)")
        lib = ctypes.CDLL(LIB_PATH)
        lib.rodimus_ddts_fwd_workspace_bytes.argtypes = [ctypes.POINTER(FwdParams)]
        lib.rodimus_ddts_fwd_workspace_bytes.restype = ctypes.c_size_t
        lib.rodimus_ddts_fwd.argtypes = [ctypes.POINTER(FwdParams)]
        lib.rodimus_ddts_fwd.restype = ctypes.c_int
        lib.rodimus_ddts_fwd_noalloc.argtypes = [ctypes.POINTER(FwdParams),
                                                 ctypes.POINTER(ctypes.c_void_p)]
        lib.rodimus_ddts_fwd_noalloc.restype = ctypes.c_int
        lib.rodimus_ddts_step.argtypes = [ctypes.POINTER(StepParams)]
        lib.rodimus_ddts_step.restype = ctypes.c_int
        lib.rodimus_ddts_device_status.argtypes = [ctypes.c_void_p, ctypes.c_void_p]
        lib.rodimus_ddts_device_status.restype = ctypes.c_int
        lib.rodimus_ddts_last_launch_count.restype = ctypes.c_int
        lib.rodimus_ddts_fwd_kernel_name.argtypes = [ctypes.POINTER(FwdParams)]
        lib.rodimus_ddts_fwd_kernel_name.restype = ctypes.c_char_p
        lib.rodimus_ddts_sfu_probe.argtypes = [ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p,
                                               ctypes.POINTER(ctypes.c_longlong)]
        lib.rodimus_ddts_sfu_probe.restype = ctypes.c_int
        lib.rodimus_ddts_test_set_wait_limit.argtypes = [ctypes.c_longlong]
        lib.rodimus_ddts_test_set_wait_limit.restype = ctypes.c_int
        lib.rodimus_ddts_bwd_workspace_bytes.argtypes = [ctypes.POINTER(BwdParams)]
        lib.rodimus_ddts_bwd_workspace_bytes.restype = ctypes.c_size_t
        lib.rodimus_ddts_bwd.argtypes = [ctypes.POINTER(BwdParams)]
        lib.rodimus_ddts_bwd.restype = ctypes.c_int
        lib.rodimus_swska_fwd.argtypes = [ctypes.POINTER(SwskaParams)]
        lib.rodimus_swska_fwd.restype = ctypes.c_int
        lib.rodimus_status_str.argtypes = [ctypes.c_int]
        lib.rodimus_status_str.restype = ctypes.c_char_p
        lib.rodimus_version.restype = ctypes.c_int
        _lib = lib
    return _lib


def status_str(status: int) -> str:
    return load_library().rodimus_status_str(int(status)).decode()


def version() -> int:
    return int(load_library().rodimus_version())


def last_launch_count() -> int:
    return int(load_library().rodimus_ddts_last_launch_count())


def _dtype_code(t) -> int:
    import torch
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.float32:
        return F32
    raise RodimusError(ERR_DTYPE, f"unsupported tensor dtype {t.dtype}")


def _ptr(t) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _check_cuda(*tensors):
    for t in tensors:
        if t is not None and not (t.is_cuda and t.is_contiguous()):
            raise ValueError("tensors must be contiguous CUDA tensors")


def fwd_params(q, k, gate_x, temp_y, v, o, s0=None, sT=None, cu_seqlens=None,
               cu_seqlens_host=None, workspace=None, scale: float = 1.0,
               ingate: int = INGATE_POW_G, stream: Optional[int] = None, beta_hat=None,
               feed_d=None, feed_x=None, value_decay=None) -> FwdParams:
    """Fills a ``rodimus_ddts_fwd_params`` from torch tensors (no checks beyond layout)."""
    import torch
    B, Hq, T, dk = q.shape
    H = v.shape[1]
    p = FwdParams()
    p.shared_gates = 1 if (Hq == 1 and H > 1) else 0     # q,k,x,y [B,1,T,dk]: one set for all heads
    p.struct_size = ctypes.sizeof(FwdParams)
    p.dtype = _dtype_code(q)
    p.ingate = ingate
    p.B, p.H, p.T, p.dk, p.dv = B, H, T, dk, v.shape[-1]
    p.scale = scale
    p.N = 0 if cu_seqlens is None else cu_seqlens.numel() - 1
    p.q, p.k, p.gate_x, p.temp_y, p.v, p.o = (_ptr(t) for t in (q, k, gate_x, temp_y, v, o))
    p.s0, p.sT = _ptr(s0), _ptr(sT)
    p.cu_seqlens = _ptr(cu_seqlens)
    p.cu_seqlens_host = _ptr(cu_seqlens_host)
    p.workspace = _ptr(workspace)
    p.workspace_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    p.stream = torch.cuda.current_stream().cuda_stream if stream is None else stream
    p.beta_hat, p.feed_d, p.feed_x = _ptr(beta_hat), _ptr(feed_d), _ptr(feed_x)
    p.value_decay = _ptr(value_decay)
    return p


def fwd_workspace_bytes(p: FwdParams) -> int:
    return int(load_library().rodimus_ddts_fwd_workspace_bytes(ctypes.byref(p)))


def fwd_kernel_name(p: FwdParams) -> str:
    return load_library().rodimus_ddts_fwd_kernel_name(ctypes.byref(p)).decode()


def fwd_raw(p: FwdParams) -> int:
    """Calls ``rodimus_ddts_fwd`` and returns its status without raising."""
    return int(load_library().rodimus_ddts_fwd(ctypes.byref(p)))


def fwd_noalloc_raw(p: FwdParams):
    """Calls ``rodimus_ddts_fwd_noalloc`` (the prefill that uses the library's built-in scratch
    array instead of a caller workspace).  Returns (status, handle); the handle is an integer
    device address accepted by ``device_status_ptr``, or None if the call failed."""
    h = ctypes.c_void_p()
    rc = int(load_library().rodimus_ddts_fwd_noalloc(ctypes.byref(p), ctypes.byref(h)))
    return rc, h.value


def device_status_ptr(ptr: int, stream: Optional[int] = None) -> int:
    """``rodimus_ddts_device_status`` for a raw device address (see ``fwd_noalloc_raw``)."""
    import torch
    st = torch.cuda.current_stream().cuda_stream if stream is None else stream
    return int(load_library().rodimus_ddts_device_status(ptr, st))


def sfu_probe(iters: int, sink, stream: Optional[int] = None) -> int:
    """Enqueues the special-function-unit probe (``rodimus_ddts_sfu_probe``) on the current
    stream and returns the number of approximations it executes; the caller times it."""
    import torch
    st = torch.cuda.current_stream().cuda_stream if stream is None else stream
    ops = ctypes.c_longlong(0)
    rc = int(load_library().rodimus_ddts_sfu_probe(int(iters), sink.data_ptr(), st, ctypes.byref(ops)))
    if rc != OK:
        raise RodimusError(rc, "rodimus_ddts_sfu_probe")
    return int(ops.value)


def test_set_wait_limit(cycles: int) -> None:
    """Test hook (``rodimus_ddts_test_set_wait_limit``): bound of the kernels' main-loop waits in
    clock cycles for the launches that follow; 0 = the first unsatisfied wait times out, negative =
    back to the default."""
    load_library().rodimus_ddts_test_set_wait_limit(int(cycles))


test_set_wait_limit.__test__ = False   # not a pytest test


def step_raw(p: StepParams) -> int:
    return int(load_library().rodimus_ddts_step(ctypes.byref(p)))


def device_status(workspace, stream: Optional[int] = None) -> int:
    import torch
    st = torch.cuda.current_stream().cuda_stream if stream is None else stream
    return int(load_library().rodimus_ddts_device_status(workspace.data_ptr(), st))


def new_workspace(p: FwdParams, device):
    import torch
    n = max(fwd_workspace_bytes(p), 256)
    return torch.empty(n, dtype=torch.uint8, device=device)


def bwd_params(q, k, gate_x, temp_y, v, d_o, d_q, d_k, d_gate_x, d_temp_y, d_v, s0=None,
               d_sT=None, d_s0=None, cu_seqlens=None, cu_seqlens_host=None, workspace=None,
               scale: float = 1.0, ingate: int = INGATE_POW_G,
               stream: Optional[int] = None) -> BwdParams:
    """Fills a ``rodimus_ddts_bwd_params`` from torch tensors (no checks beyond layout)."""
    import torch
    B, H, T, dk = q.shape
    p = BwdParams()
    p.struct_size = ctypes.sizeof(BwdParams)
    p.dtype = _dtype_code(q)
    p.ingate = ingate
    p.B, p.H, p.T, p.dk, p.dv = B, H, T, dk, v.shape[-1]
    p.scale = scale
    p.N = 0 if cu_seqlens is None else cu_seqlens.numel() - 1
    p.q, p.k, p.gate_x, p.temp_y, p.v = (_ptr(t) for t in (q, k, gate_x, temp_y, v))
    p.s0, p.d_o, p.d_sT = _ptr(s0), _ptr(d_o), _ptr(d_sT)
    p.d_q, p.d_k, p.d_gate_x, p.d_temp_y = (_ptr(t) for t in (d_q, d_k, d_gate_x, d_temp_y))
    p.d_v, p.d_s0 = _ptr(d_v), _ptr(d_s0)
    p.cu_seqlens = _ptr(cu_seqlens)
    p.cu_seqlens_host = _ptr(cu_seqlens_host)
    p.workspace = _ptr(workspace)
    p.workspace_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    p.stream = torch.cuda.current_stream().cuda_stream if stream is None else stream
    return p


def bwd_workspace_bytes(p: BwdParams) -> int:
    return int(load_library().rodimus_ddts_bwd_workspace_bytes(ctypes.byref(p)))


def bwd_raw(p: BwdParams) -> int:
    """Calls ``rodimus_ddts_bwd`` and returns its status without raising."""
    return int(load_library().rodimus_ddts_bwd(ctypes.byref(p)))


def ddts_bwd(q, k, gate_x, temp_y, v, d_o, s0=None, d_sT=None, cu_seqlens=None,
             cu_seqlens_host=None, scale: float = 1.0, ingate: int = INGATE_POW_G,
             want_d_s0: bool = True, workspace=None):
    """Backward pass of the prefill (``rodimus_ddts_bwd``).

    Inputs as ``ddts_fwd`` plus d_o = dL/do [B,H,T,dv] and d_sT = dL/dS_T (fp32 [B|N,H,dk,dv] or
    None).  Returns a dict with d_q, d_k, d_gate_x, d_temp_y [B,H,T,dk], d_v [B,H,T,dv] (dtype of
    the inputs) and d_s0 (fp32, None unless wanted).  Asynchronous on the current stream.
    """
    import torch
    _check_cuda(q, k, gate_x, temp_y, v, d_o, s0, d_sT, cu_seqlens)
    B, H, T, dk = q.shape
    dv = v.shape[-1]
    nseq = B if cu_seqlens is None else cu_seqlens.numel() - 1
    out = {n: torch.empty_like(q) for n in ("d_q", "d_k", "d_gate_x", "d_temp_y")}
    out["d_v"] = torch.empty_like(v)
    out["d_s0"] = (torch.empty((nseq, H, dk, dv), dtype=torch.float32, device=q.device)
                   if want_d_s0 else None)
    p = bwd_params(q, k, gate_x, temp_y, v, d_o, out["d_q"], out["d_k"], out["d_gate_x"],
                   out["d_temp_y"], out["d_v"], s0, d_sT, out["d_s0"], cu_seqlens,
                   cu_seqlens_host, None, scale, ingate)
    ws = workspace
    if ws is None:
        ws = torch.empty(max(bwd_workspace_bytes(p), 256), dtype=torch.uint8, device=q.device)
    p.workspace = ws.data_ptr()
    p.workspace_bytes = ws.numel() * ws.element_size()
    rc = bwd_raw(p)
    if rc != OK:
        raise RodimusError(rc, "rodimus_ddts_bwd")
    return out


def swska_params(q, k, v, o, window: int, scale: float, stream: Optional[int] = None,
                 workspace=None) -> SwskaParams:
    """Fills a ``rodimus_swska_fwd_params`` from torch tensors (no checks beyond layout)."""
    import torch
    B, H, T, d = q.shape
    p = SwskaParams()
    p.struct_size = ctypes.sizeof(SwskaParams)
    p.dtype = _dtype_code(q)
    p.B, p.H, p.T, p.d = B, H, T, d
    p.window, p.scale = int(window), float(scale)
    p.q, p.k, p.v, p.o = (_ptr(t) for t in (q, k, v, o))
    p.stream = torch.cuda.current_stream().cuda_stream if stream is None else stream
    p.workspace = _ptr(workspace)
    p.workspace_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    return p


def swska_raw(p: SwskaParams) -> int:
    """Calls ``rodimus_swska_fwd`` and returns its status without raising."""
    return int(load_library().rodimus_swska_fwd(ctypes.byref(p)))


def swska_fwd(q, k, v, window: int, scale: Optional[float] = None, out=None):
    """Sliding-window shared-key attention (``rodimus_swska_fwd``): q, v [B,H,T,d], k [B,T,d]
    (one key per token for all heads); token t attends to tokens t-window+1 .. t.  ``scale``
    defaults to 1/sqrt(d).  Returns o [B,H,T,d].  Asynchronous on the current stream."""
    import torch
    _check_cuda(q, k, v)
    if k.shape != (q.shape[0], q.shape[2], q.shape[3]) or v.shape != q.shape:
        raise ValueError("q, v must be [B,H,T,d] and k [B,T,d]")
    o = out if out is not None else torch.empty_like(q)
    p = swska_params(q, k, v, o, window, q.shape[-1] ** -0.5 if scale is None else scale)
    rc = swska_raw(p)
    if rc != OK:
        raise RodimusError(rc, "rodimus_swska_fwd")
    return o


def ddts_fwd(q, k, gate_x, temp_y, v, s0=None, cu_seqlens=None, cu_seqlens_host=None,
             scale: float = 1.0, ingate: int = INGATE_POW_G, want_final_state: bool = True,
             out=None, final_state=None, workspace=None, beta_hat=None, feed_d=None,
             feed_x=None, value_decay=None) -> Tuple["torch.Tensor", Optional["torch.Tensor"]]:
    """Chunked DDTS prefill (``rodimus_ddts_fwd``).

    q,k,gate_x,temp_y: [B,H,T,dk]; v: [B,H,T,dv] (bf16 or fp32, all alike); s0: fp32
    [B|N,H,dk,dv] or None; cu_seqlens: int32 CUDA tensor [N+1] for packed sequences (B = 1).
    Optional, fused into the same pass: beta_hat [B,H,T,dv] (value gate, multiplies v), and the
    feed-through feed_d fp32 [H,dv] with feed_x [B,H,T,dv] (o += feed_d * feed_x).
    value_decay [B,H,T,dv] in (0,1]: the value-side decay of the general transition (the arm the
    paper ablates and drops; fp32 CUDA-core kernel).
    Returns (o, sT) with sT None unless ``want_final_state``.  Asynchronous on the current stream.
    """
    import torch
    _check_cuda(q, k, gate_x, temp_y, v, s0, cu_seqlens, beta_hat, feed_d, feed_x, value_decay)
    B, _, T, dk = q.shape
    H = v.shape[1]            # q,k,gate_x,temp_y may have a single head shared by all H of v
    dv = v.shape[-1]
    nseq = B if cu_seqlens is None else cu_seqlens.numel() - 1
    o = out if out is not None else torch.empty((B, H, T, dv), dtype=q.dtype, device=q.device)
    sT = final_state
    if sT is None and want_final_state:
        sT = torch.empty((nseq, H, dk, dv), dtype=torch.float32, device=q.device)
    p = fwd_params(q, k, gate_x, temp_y, v, o, s0, sT, cu_seqlens, cu_seqlens_host, None, scale,
                   ingate, beta_hat=beta_hat, feed_d=feed_d, feed_x=feed_x, value_decay=value_decay)
    ws = workspace if workspace is not None else new_workspace(p, q.device)
    p.workspace = ws.data_ptr()
    p.workspace_bytes = ws.numel() * ws.element_size()
    rc = fwd_raw(p)
    if rc != OK:
        raise RodimusError(rc, "rodimus_ddts_fwd")
    return o, sT


def ddts_step(q, k, gate_x, temp_y, v, state, scale: float = 1.0, ingate: int = INGATE_POW_G,
              out=None, beta_hat=None, feed_d=None, feed_x=None, value_decay=None):
    """One decode step (``rodimus_ddts_step``): ``state`` fp32 [Nseq,H,dk,dv] is updated in place.

    q,k,gate_x,temp_y: [Nseq,H,dk]; v: [Nseq,H,dv].  Returns o [Nseq,H,dv].
    """
    import torch
    _check_cuda(q, k, gate_x, temp_y, v, state, beta_hat, feed_d, feed_x, value_decay)
    Nseq, Hq, dk = q.shape
    H = v.shape[1]
    dv = v.shape[-1]
    o = out if out is not None else torch.empty((Nseq, H, dv), dtype=q.dtype, device=q.device)
    p = StepParams()
    p.struct_size = ctypes.sizeof(StepParams)
    p.dtype = _dtype_code(q)
    p.ingate = ingate
    p.Nseq, p.H, p.dk, p.dv = Nseq, H, dk, dv
    p.scale = scale
    p.q, p.k, p.gate_x, p.temp_y, p.v, p.o = (_ptr(t) for t in (q, k, gate_x, temp_y, v, o))
    p.state = _ptr(state)
    p.stream = torch.cuda.current_stream().cuda_stream
    p.beta_hat, p.feed_d, p.feed_x = _ptr(beta_hat), _ptr(feed_d), _ptr(feed_x)
    p.shared_gates = 1 if (Hq == 1 and H > 1) else 0
    p.value_decay = _ptr(value_decay)
    rc = step_raw(p)
    if rc != OK:
        raise RodimusError(rc, "rodimus_ddts_step")
    return o


def ddts_fwd_host(q, k, gate_x, temp_y, v, s0=None, cu_seqlens=None, scale: float = 1.0,
                  ingate: int = INGATE_POW_G, want_final_state: bool = True, device="cuda:0"):
    """``ddts_fwd`` for HOST tensors (pinned for full copy speed): copies the inputs to the
    device, runs the prefill through the C ABI, copies o (and sT) back, and waits for them.
    """
    import torch
    dev = torch.device(device)
    up = lambda t: None if t is None else t.to(dev, non_blocking=True)
    cu_d = up(cu_seqlens)
    o, sT = ddts_fwd(up(q), up(k), up(gate_x), up(temp_y), up(v), up(s0), cu_d,
                     cu_seqlens.contiguous() if cu_seqlens is not None else None, scale, ingate,
                     want_final_state)
    o_h = torch.empty(o.shape, dtype=o.dtype, pin_memory=True)
    o_h.copy_(o, non_blocking=True)
    sT_h = None
    if sT is not None:
        sT_h = torch.empty(sT.shape, dtype=sT.dtype, pin_memory=True)
        sT_h.copy_(sT, non_blocking=True)
    torch.cuda.current_stream().synchronize()
    return o_h, sT_h
