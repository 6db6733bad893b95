"""GPU parity of the backward pass: ``rodimus_ddts_bwd`` through the C ABI against the fp64 adjoint
recurrence of the oracle on the same seeded inputs.  Bar, per gradient tensor:
max|err|/max|ref| <= 2e-2 (bf16 tokens: tf32 contractions, fp32 accumulation, bf16 outputs) and
<= 1e-4 (fp32 build: split-tf32 contractions at fp32 accuracy)."""
import numpy as np
import pytest

import paper_2410_06577_b200 as rd
from paper_2410_06577_b200 import workloads as wl
from oracle import ddts_oracle as orc
from tests._util import TOL_BF16, TOL_F32, dev, host, prefill_to_device, rel_err

pytestmark = pytest.mark.gpu

PAIRS = (("d_q", "dq"), ("d_k", "dk"), ("d_gate_x", "dx"), ("d_temp_y", "dy"), ("d_v", "dv"))


def _run_bwd(p, d_o, d_sT, ingate, scale, host_cu=True, want_d_s0=True):
    """Calls the library with NaN-filled outputs (an element the kernels never store stays NaN)."""
    import torch
    d = prefill_to_device(p)
    B, H, T, dk = d["q"].shape
    dv = d["v"].shape[-1]
    nseq = B if d["cu"] is None else d["cu"].numel() - 1
    g_o = dev(d_o, p.dtype)
    g_s = None if d_sT is None else torch.from_numpy(d_sT).cuda()
    out = {n: torch.full_like(d["q"], float("nan")) for n in ("d_q", "d_k", "d_gate_x", "d_temp_y")}
    out["d_v"] = torch.full_like(d["v"], float("nan"))
    out["d_s0"] = (torch.full((nseq, H, dk, dv), float("nan"), dtype=torch.float32, device="cuda")
                   if want_d_s0 else None)
    prm = rd.bwd_params(d["q"], d["k"], d["x"], d["y"], d["v"], g_o, out["d_q"], out["d_k"],
                        out["d_gate_x"], out["d_temp_y"], out["d_v"], d["s0"], g_s, out["d_s0"],
                        d["cu"], d["cu_host"] if host_cu else None, None, scale, ingate)
    ws = torch.empty(max(rd.bwd_workspace_bytes(prm), 256), dtype=torch.uint8, device="cuda")
    prm.workspace, prm.workspace_bytes = ws.data_ptr(), ws.numel()
    rc = rd.bwd_raw(prm)
    assert rc == rd.OK, rd.status_str(rc)
    assert rd.device_status(ws) == rd.OK
    torch.cuda.synchronize()
    return {n: (None if t is None else host(t)) for n, t in out.items()}


def _check(p, seed, with_state, ingate=rd.INGATE_POW_G, scale=1.0, **kw):
    d_o, d_sT = wl.make_grads(seed, p, with_state)
    got = _run_bwd(p, d_o, d_sT, ingate, scale, **kw)
    ref = orc.ref_bwd(p.q, p.k, p.x, p.y, p.v, d_o, s0=p.s0, dsT=d_sT, cu_seqlens=p.cu_seqlens,
                      scale=scale, ingate=ingate)
    tol = TOL_BF16 if p.dtype == "bf16" else TOL_F32
    errs = {}
    if p.cu_seqlens is None:
        for a, b in PAIRS:
            errs[a] = rel_err(got[a], ref[b])
    else:   # packed: every sequence against its own scale, empty ones have nothing to compare
        cu = p.cu_seqlens
        for a, b in PAIRS:
            errs[a] = max([rel_err(got[a][:, :, cu[n]:cu[n + 1]], ref[b][:, :, cu[n]:cu[n + 1]])
                           for n in range(len(cu) - 1) if cu[n + 1] > cu[n]] or [0.0])
    if got["d_s0"] is not None:
        errs["d_s0"] = rel_err(got["d_s0"], ref["ds0"])
    assert all(e <= tol for e in errs.values()), (p.name, errs)
    return errs


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("B,H,T,with_state", [
    (1, 1, 1, True),        # a single step
    (2, 2, 16, False),      # exactly one chunk, zero initial state, no state gradient
    (1, 2, 37, True),       # ragged tail
    (2, 3, 150, True),      # several chunks and a ragged tail
])
def test_bwd_matches_oracle(dtype, B, H, T, with_state):
    p = wl.make_prefill(100 + T, B, H, T, 128, 256, dtype, gate_mean=-3.0,
                        s0_std=0.1 if with_state else None, name=f"bwd_{dtype}_{T}")
    _check(p, 200 + T, with_state, scale=0.5)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_bwd_alternate_input_gate_and_strong_decay(dtype):
    # gate pre-activations around +2: decays of e^-1 per step and more, cumulative exponents far
    # below the range of a factored form; every exponential here has a non-positive argument
    p = wl.make_prefill(301, 1, 2, 90, 128, 256, dtype, gate_mean=2.0, s0_std=0.1, name="bwd_strong")
    _check(p, 302, True, ingate=rd.INGATE_POW_SIGMOID)
    _check(p, 303, True, ingate=rd.INGATE_POW_G)
    # pre-activations around +12: a chunk of 16 steps decays by far more than e^-60, which the
    # kernel answers with its pair-by-pair form; milder chunks of the same call take the factored one
    p = wl.make_prefill(304, 1, 2, 70, 128, 256, dtype, gate_mean=12.0, s0_std=0.1, name="bwd_very_strong")
    p.x[:, :, 32:48] = wl.make_prefill(305, 1, 2, 16, 128, 256, dtype, gate_mean=-3.0).x
    _check(p, 306, True, ingate=rd.INGATE_POW_G)
    _check(p, 307, True, ingate=rd.INGATE_POW_SIGMOID)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_bwd_packed_sequences(dtype):
    lens = [40, 0, 1, 16, 77, 3]
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    p = wl.make_prefill(401, 1, 2, int(cu[-1]), 128, 256, dtype, s0_std=0.1, cu_seqlens=cu,
                        name="bwd_packed")
    errs = _check(p, 402, True)
    assert "d_s0" in errs
    _check(p, 403, True, host_cu=False, want_d_s0=False)


def test_bwd_bad_cu_seqlens_reported_by_the_device():
    import torch
    cu = np.array([0, 30, 20, 64], dtype=np.int32)          # decreasing
    p = wl.make_prefill(501, 1, 1, 64, 128, 256, "bf16", name="bwd_badcu")
    d = prefill_to_device(p)
    d_o, _ = wl.make_grads(502, p, False)
    outs = [torch.zeros_like(d["q"]) for _ in range(4)] + [torch.zeros_like(d["v"])]
    prm = rd.bwd_params(d["q"], d["k"], d["x"], d["y"], d["v"], dev(d_o, "bf16"), *outs,
                        cu_seqlens=torch.from_numpy(cu).cuda())
    ws = torch.empty(rd.bwd_workspace_bytes(prm), dtype=torch.uint8, device="cuda")
    prm.workspace, prm.workspace_bytes = ws.data_ptr(), ws.numel()
    assert rd.bwd_raw(prm) == rd.OK                          # no host copy: found on the device
    assert rd.device_status(ws) == rd.ERR_SEQLENS
    torch.cuda.synchronize()


def test_bwd_config1_shape_sampled_heads():
    """The layer-prefill shape (B=4, H=16, T=2048) in one call; the oracle checks two heads."""
    import torch
    p = wl.config(1)
    d_o, d_sT = wl.make_grads(601, p, True)
    got = _run_bwd(p, d_o, d_sT, rd.INGATE_POW_G, 1.0)
    for name in got:
        assert np.all(np.isfinite(got[name])), name
    for b, h in ((0, 3), (3, 15)):
        sl = (slice(b, b + 1), slice(h, h + 1))
        ref = orc.ref_bwd(p.q[sl], p.k[sl], p.x[sl], p.y[sl], p.v[sl], d_o[sl], dsT=d_sT[sl])
        for a, r in PAIRS:
            assert rel_err(got[a][sl], ref[r]) <= TOL_BF16, (a, b, h)
        assert rel_err(got["d_s0"][sl], ref["ds0"]) <= TOL_BF16


def test_bwd_long_sequence_and_many_packed_sequences():
    # 1000 steps (63 chunks): the suffix sums run over the whole sequence in 16 time segments
    p = wl.make_prefill(701, 1, 2, 1000, 128, 256, "bf16", s0_std=0.1, name="bwd_long")
    _check(p, 702, True)
    # 40 packed sequences of mixed lengths, several of them shorter than a chunk
    lens = list(np.random.default_rng(703).integers(0, 90, 40))
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    p = wl.make_prefill(704, 1, 2, int(cu[-1]), 128, 256, "bf16", s0_std=0.1, cu_seqlens=cu, name="bwd_many")
    _check(p, 705, True)


def test_bwd_segment_wait_that_runs_out_reports_timeout():
    """A long sweep is cut into time segments that run as thread blocks of their own; each waits,
    with a limit, for the one before it.  With the limit at zero the later segments find their
    predecessors unfinished, give up and return: the call reports TIMEOUT, nothing hangs, and the
    next call is clean."""
    import torch
    p = wl.make_prefill(801, 1, 2, 1000, 128, 256, "bf16", s0_std=0.1, name="bwd_wait")
    d = prefill_to_device(p)
    d_o, d_sT = wl.make_grads(802, p, True)
    outs = [torch.zeros_like(d["q"]) for _ in range(4)] + [torch.zeros_like(d["v"])]
    prm = rd.bwd_params(d["q"], d["k"], d["x"], d["y"], d["v"], dev(d_o, "bf16"), *outs,
                        s0=d["s0"], d_sT=torch.from_numpy(d_sT).cuda())
    ws = torch.empty(rd.bwd_workspace_bytes(prm), dtype=torch.uint8, device="cuda")
    prm.workspace, prm.workspace_bytes = ws.data_ptr(), ws.numel()
    rd.test_set_wait_limit(0)
    try:
        assert rd.bwd_raw(prm) == rd.OK
        assert rd.device_status(ws) == rd.ERR_TIMEOUT
    finally:
        rd.test_set_wait_limit(-1)
    torch.cuda.synchronize()
    _check(p, 802, True)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_bwd_packed_sequences_cut_into_time_segments(dtype):
    # long enough on average for the sweeps to be cut into time segments, with an empty sequence,
    # one of two chunks (one row in the second) and ragged tails among them
    lens = [300, 0, 200, 17, 129]
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    p = wl.make_prefill(901, 1, 2, int(cu[-1]), 128, 256, dtype, s0_std=0.1, cu_seqlens=cu,
                        name="bwd_packed_segments")
    _check(p, 902, True)
    _check(p, 903, False, host_cu=False, want_d_s0=False)
