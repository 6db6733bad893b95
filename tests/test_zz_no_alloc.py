"""The allocation-free prefill entry point (``rodimus_ddts_fwd_noalloc``) against the ordinary one.

Some users of this library are handed input and output buffers and nothing else: they run inside
an application that gave away all device memory at start-up, or in a serving loop where a
``cudaMalloc`` (and the device-wide synchronisation it implies) is not acceptable.  They cannot
supply the small workspace ``rodimus_ddts_fwd`` asks for, so the library carries one of fixed
size in its own device image.  These tests call that variant through the C ABI, twice in a row
(the built-in array keeps whatever the previous call left in it), and require the same outputs
as the ordinary entry point and, like it, agreement with the CPU oracle.

This file sorts last on purpose: a run that stops at the first failure has then already been
through every other test.
"""
import ctypes

import numpy as np
import pytest

import paper_2410_06577_b200 as rd
from paper_2410_06577_b200 import workloads as wl
from oracle import ddts_oracle as orc
from tests._util import TOL_BF16, TOL_F32, host, prefill_to_device, rel_err


def _params(d, o, sT, ws=None):
    p = rd.fwd_params(d["q"], d["k"], d["x"], d["y"], d["v"], o, d["s0"], sT, d["cu"], d["cu_host"],
                      ws, 0.5)
    return p


def _both_ways(p_in, tol):
    import torch
    d = prefill_to_device(p_in)
    B, H, T, dk = d["q"].shape
    dv = d["v"].shape[-1]
    nseq = B if d["cu"] is None else d["cu"].numel() - 1
    new_o = lambda: torch.full((B, H, T, dv), float("nan"), dtype=d["q"].dtype, device="cuda")
    new_s = lambda: torch.full((nseq, H, dk, dv), float("nan"), dtype=torch.float32, device="cuda")
    # ordinary entry point, caller-provided workspace
    o_ref, s_ref = new_o(), new_s()
    p = _params(d, o_ref, s_ref)
    ws = rd.new_workspace(p, "cuda")
    p.workspace, p.workspace_bytes = ws.data_ptr(), ws.numel()
    assert rd.fwd_raw(p) == rd.OK
    assert rd.device_status(ws) == rd.OK
    ro, rs = orc.ref_fwd(p_in.q, p_in.k, p_in.x, p_in.y, p_in.v, s0=p_in.s0,
                         cu_seqlens=p_in.cu_seqlens, scale=0.5)
    # the variant without a workspace, two calls in a row
    for _ in range(2):
        o, s = new_o(), new_s()
        q = _params(d, o, s)          # workspace fields left empty: they must be ignored
        rc, handle = rd.fwd_noalloc_raw(q)
        assert rc == rd.OK and handle
        assert rd.device_status_ptr(handle) == rd.OK
        torch.cuda.synchronize()
        assert rel_err(host(o), host(o_ref)) <= tol
        assert rel_err(host(s), host(s_ref)) <= tol
        # and directly against the oracle, sequence by sequence for packed inputs
        cu = p_in.cu_seqlens if p_in.cu_seqlens is not None else [0, T]
        for n in range(len(cu) - 1):
            lo, hi = int(cu[n]), int(cu[n + 1])
            so = np.s_[:, :, lo:hi] if p_in.cu_seqlens is not None else np.s_[...]
            ss = np.s_[n] if p_in.cu_seqlens is not None else np.s_[...]
            if hi > lo:
                assert rel_err(host(o)[so], ro[so]) <= tol, n
            assert rel_err(host(s)[ss], rs[ss]) <= tol, n


@pytest.mark.gpu
def test_noalloc_dense_bf16_matches_workspace_entry_point():
    _both_ways(wl.make_prefill(41, 2, 2, 200, 128, 256, "bf16", s0_std=0.1), TOL_BF16)


@pytest.mark.gpu
def test_noalloc_varlen_bf16_matches_workspace_entry_point():
    cu = np.concatenate([[0], np.cumsum([70, 0, 129, 64, 5])]).astype(np.int32)
    p = wl.make_prefill(42, 1, 2, int(cu[-1]), 128, 256, "bf16", s0_std=0.2, cu_seqlens=cu)
    _both_ways(p, TOL_BF16)


@pytest.mark.gpu
def test_noalloc_fp32_kernel_matches_workspace_entry_point():
    _both_ways(wl.make_prefill(43, 1, 2, 90, 64, 64, "f32", s0_std=0.3), TOL_F32)


@pytest.mark.gpu
def test_noalloc_rejects_more_sequences_than_the_built_in_array_holds():
    import torch
    n = rd.NOALLOC_MAX_SEQS + 1
    cu = torch.zeros(n + 1, dtype=torch.int32, device="cuda")      # all sequences empty, T = 0
    z = torch.zeros((1, 1, 0, 128), dtype=torch.bfloat16, device="cuda")
    v = torch.zeros((1, 1, 0, 256), dtype=torch.bfloat16, device="cuda")
    sT = torch.zeros((n, 1, 128, 256), dtype=torch.float32, device="cuda")
    p = rd.fwd_params(z, z, z, z, v, v.clone(), None, sT, cu)
    rc, handle = rd.fwd_noalloc_raw(p)
    assert rc == rd.ERR_WORKSPACE and handle is None
