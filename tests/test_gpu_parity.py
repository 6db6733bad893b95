"""GPU parity: the CUDA library, called through its C ABI, against the fp64 CPU oracle on the
same seeded inputs.  Bar: max|err|/max|ref| <= 2e-2 (bf16 in, fp32 accumulate) and <= 1e-4
(fp32 build), per output tensor (o and the final state separately)."""
import os

import numpy as np
import pytest

import paper_2410_06577_b200 as rd
from paper_2410_06577_b200 import workloads as wl
from oracle import ddts_oracle as orc
from tests._util import TOL_BF16, TOL_F32, dev, host, prefill_to_device, rel_err

pytestmark = pytest.mark.gpu


def _tol(dtype):
    return TOL_BF16 if dtype == "bf16" else TOL_F32


def _nan_outputs(d, want_final_state=True):
    """Fresh outputs filled with NaN: a row or a state the kernels never store shows up as a
    non-finite value (rel_err rejects those) instead of passing on recycled memory."""
    import torch
    B, H, T, dk = d["q"].shape
    dv = d["v"].shape[-1]
    nseq = B if d["cu"] is None else d["cu"].numel() - 1
    o = torch.full((B, H, T, dv), float("nan"), dtype=d["q"].dtype, device="cuda")
    sT = None
    if want_final_state:
        sT = torch.full((nseq, H, dk, dv), float("nan"), dtype=torch.float32, device="cuda")
    return o, sT


def _run_prefill(p, ingate=rd.INGATE_POW_G, scale=1.0, host_cu=True, want_final_state=True):
    import torch
    d = prefill_to_device(p)
    o, sT = _nan_outputs(d, want_final_state)
    o, sT = rd.ddts_fwd(d["q"], d["k"], d["x"], d["y"], d["v"], d["s0"], d["cu"],
                        d["cu_host"] if host_cu else None, scale, ingate, want_final_state,
                        out=o, final_state=sT)
    torch.cuda.synchronize()
    return host(o), (None if sT is None else host(sT))


def _worst_err(o, sT, ro, rs, cu, p=None, ingate=rd.INGATE_POW_G, scale=1.0):
    """The parity measure, max|err|/max|ref|, of o and of the final state.  Packed inputs are
    judged sequence by sequence (each against its own maximum, empty ones skipped), so that a
    short sequence is not measured against the scale of a long neighbour.

    One kind of sequence has no meaningful relative measure: a single token starting from a zero
    state.  Its whole output is ONE score, a sum of dk products of bf16-rounded operands, times
    v; where those products happen to cancel, max|ref| is arbitrarily small while the rounding
    error is not.  Such sequences (when `p` is given) are held to the a-priori bound of that
    sum instead: |err| <= 4 * 2^-9 * sum_d |q_d k_d ahat_d| * max|v| (two operand roundings, the
    score's and the output's own)."""
    if cu is None:
        return rel_err(o, ro), rel_err(sT, rs)
    eo = es = 0.0
    for n in range(len(cu) - 1):
        lo, hi = int(cu[n]), int(cu[n + 1])
        if hi - lo == 1 and p is not None and p.dtype == "bf16" and p.s0 is None:
            _, ahat = orc.ref_gates(p.x[0, :, lo], p.y[0, :, lo], ingate)          # [H, dk]
            terms = np.sum(np.abs(p.q[0, :, lo].astype(np.float64) * p.k[0, :, lo] * ahat), axis=-1)
            bound = 4.0 * 2.0 ** -9 * terms * np.max(np.abs(p.v[0, :, lo]), axis=-1) * abs(scale)
            err = np.max(np.abs(o[0, :, lo] - ro[0, :, lo]), axis=-1)               # [H]
            assert np.all(np.isfinite(o[0, :, lo])) and np.all(err <= bound), (n, err, bound)
        elif hi > lo:
            eo = max(eo, rel_err(o[:, :, lo:hi], ro[:, :, lo:hi]))
        es = max(es, rel_err(sT[n], rs[n]))
    return eo, es


def _check_prefill(p, ingate=rd.INGATE_POW_G, scale=1.0, tol=None, **kw):
    o, sT = _run_prefill(p, ingate, scale, **kw)
    ro, rs = orc.ref_fwd(p.q, p.k, p.x, p.y, p.v, s0=p.s0, cu_seqlens=p.cu_seqlens, scale=scale,
                         ingate=ingate)
    tol = tol or _tol(p.dtype)
    eo, es = _worst_err(o, sT, ro, rs, p.cu_seqlens, p, ingate, scale)
    assert eo <= tol and es <= tol, (p.name, eo, es)
    return eo, es


# ------------------------------------------------------------------------------------------
# decode
# ------------------------------------------------------------------------------------------

@pytest.mark.parametrize("dtype,Nseq,H,dk,dv", [
    ("bf16", 16, 4, 128, 256),     # config 3 shrunk
    ("f32", 3, 2, 64, 64),
    ("bf16", 5, 3, 48, 80),        # ragged column tile, short rows
    ("f32", 2, 1, 256, 1024),      # maximum sizes
])
@pytest.mark.parametrize("ingate", [rd.INGATE_POW_G, rd.INGATE_POW_SIGMOID])
def test_decode_steps_match_oracle(dtype, Nseq, H, dk, dv, ingate):
    import torch
    w = wl.make_decode(3, Nseq, H, dk, dv, ring=16, dtype=dtype)
    state = torch.from_numpy(w.state).cuda()
    ref_state = w.state.astype(np.float64)
    tol = _tol(dtype)
    for s in range(16):
        o = rd.ddts_step(dev(w.q[s], dtype), dev(w.k[s], dtype), dev(w.x[s], dtype),
                         dev(w.y[s], dtype), dev(w.v[s], dtype), state, scale=0.5, ingate=ingate)
        ro = orc.ref_step(w.q[s], w.k[s], w.x[s], w.y[s], w.v[s], ref_state, scale=0.5,
                          ingate=ingate)
        assert rel_err(host(o), ro) <= tol
    # the fp32 state itself is held to the fp32 bar whatever the token dtype
    assert rel_err(host(state), ref_state) <= TOL_F32


def test_decode_full_width_sixteen_steps_every_state():
    """Config 3 at full width (256 sequences x 16 heads): after 16 in-place steps the whole
    fp32 state and the last outputs are compared with the oracle."""
    import torch
    w = wl.config(3)
    assert w.state.shape == (256, 16, 128, 256)
    state = torch.from_numpy(w.state).cuda()
    ref_state = w.state.astype(np.float64)
    o = torch.full((256, 16, 256), float("nan"), dtype=torch.bfloat16, device="cuda")
    for s in range(16):
        rd.ddts_step(*(dev(a[s], "bf16") for a in (w.q, w.k, w.x, w.y, w.v)), state, out=o)
        ro = orc.ref_step(w.q[s], w.k[s], w.x[s], w.y[s], w.v[s], ref_state)
    torch.cuda.synchronize()
    assert rel_err(host(o), ro) <= TOL_BF16
    got = host(state)
    for n in range(0, 256, 32):   # per block of sequences, each against its own maximum
        assert rel_err(got[n:n + 32], ref_state[n:n + 32]) <= TOL_F32, n


def test_decode_full_width_many_steps():
    """Config 3 at full width (256 sequences x 16 heads), 1000 in-place steps; the oracle follows
    8 of the sequences."""
    import torch
    w = wl.config(3)
    Nseq = w.state.shape[0]
    pick = np.array([0, 1, 37, 100, 128, 200, 254, 255])
    state = torch.from_numpy(w.state).cuda()
    ref_state = np.ascontiguousarray(w.state[pick]).astype(np.float64)
    ring = [tuple(dev(a[s], "bf16") for a in (w.q, w.k, w.x, w.y, w.v)) for s in range(16)]
    o = torch.full((Nseq, 16, 256), float("nan"), dtype=torch.bfloat16, device="cuda")
    for step in range(1000):
        q, k, x, y, v = ring[step % 16]
        rd.ddts_step(q, k, x, y, v, state, out=o)
        if step in (0, 15, 999):
            torch.cuda.synchronize()
        s = step % 16
        ro = orc.ref_step(w.q[s][pick], w.k[s][pick], w.x[s][pick], w.y[s][pick], w.v[s][pick],
                          ref_state)
        if step in (0, 15, 999):
            assert rel_err(host(o)[pick], ro) <= TOL_BF16, step
    assert rel_err(host(state)[pick], ref_state) <= TOL_F32


# ------------------------------------------------------------------------------------------
# prefill: fp32 validation build
# ------------------------------------------------------------------------------------------

@pytest.mark.parametrize("ingate", [rd.INGATE_POW_G, rd.INGATE_POW_SIGMOID])
def test_config0_fp32(ingate):
    p = wl.config(0)
    _check_prefill(p, ingate)
    # and the O(T^2) masked parallel form agrees too (zero initial state)
    o, _ = _run_prefill(p, ingate)
    ref = orc.parallel_form(p.q[0, 0], p.k[0, 0], p.x[0, 0], p.y[0, 0], p.v[0, 0], ingate=ingate)
    assert rel_err(o[0, 0], ref) <= TOL_F32


@pytest.mark.parametrize("B,H,T,dk,dv", [
    (2, 2, 1, 64, 64),       # single token
    (1, 3, 37, 48, 80),      # ragged everything
    (1, 1, 131, 256, 256),   # widest keys
    (2, 1, 16, 16, 16),      # smallest legal sizes, exactly one chunk
    (1, 2, 40, 64, 320),     # more value columns than one 256-column tile
])
def test_fp32_shapes_state_and_scale(B, H, T, dk, dv):
    p = wl.make_prefill(100 + T, B, H, T, dk, dv, "f32", gate_mean=-1.0, s0_std=0.5)
    _check_prefill(p, scale=0.25)
    _check_prefill(p, rd.INGATE_POW_SIGMOID, scale=3.0)


def test_fp32_empty_sequence_returns_initial_state():
    import torch
    p = wl.make_prefill(7, 2, 2, 0, 64, 64, "f32", s0_std=1.0)
    o, sT = _run_prefill(p)
    assert o.shape == (2, 2, 0, 64)
    assert np.array_equal(sT, p.s0.astype(np.float64))


# ------------------------------------------------------------------------------------------
# prefill: bf16 path (tensor-core kernel for dk = 128, dv % 128 == 0)
# ------------------------------------------------------------------------------------------

@pytest.mark.parametrize("B,H,T,dv", [
    (2, 2, 200, 256),    # several chunks and a ragged tail
    (1, 2, 64, 128),     # exactly one chunk
    (1, 1, 1, 256),      # one token
    (1, 2, 65, 256),     # tail of one row
    (3, 1, 333, 128),
])
@pytest.mark.parametrize("ingate", [rd.INGATE_POW_G, rd.INGATE_POW_SIGMOID])
def test_bf16_prefill_small(B, H, T, dv, ingate):
    p = wl.make_prefill(200 + T, B, H, T, 128, dv, "bf16", s0_std=0.1)
    _check_prefill(p, ingate, scale=0.5)
    p0 = wl.make_prefill(300 + T, B, H, T, 128, dv, "bf16")       # zero initial state
    _check_prefill(p0, ingate)


def test_bf16_other_shapes_use_cuda_core_kernel():
    p = wl.make_prefill(11, 1, 2, 90, 64, 96, "bf16", s0_std=0.1)
    _check_prefill(p)


def test_bf16_output_only_and_state_aliasing():
    import torch
    p = wl.make_prefill(12, 1, 2, 150, 128, 256, "bf16", s0_std=0.1)
    d = prefill_to_device(p)
    o1, none = rd.ddts_fwd(d["q"], d["k"], d["x"], d["y"], d["v"], d["s0"], want_final_state=False)
    assert none is None
    s_inout = d["s0"].clone()
    o2, sT = rd.ddts_fwd(d["q"], d["k"], d["x"], d["y"], d["v"], s_inout, final_state=s_inout)
    torch.cuda.synchronize()
    assert torch.equal(o1, o2)
    ro, rs = orc.ref_fwd(p.q, p.k, p.x, p.y, p.v, s0=p.s0)
    assert rel_err(host(o1), ro) <= TOL_BF16 and rel_err(host(s_inout), rs) <= TOL_BF16


def test_bf16_prefill_equals_split_runs_and_decode_steps():
    import torch
    p = wl.make_prefill(13, 1, 2, 192, 128, 256, "bf16", s0_std=0.1)
    d = prefill_to_device(p)
    o, sT = rd.ddts_fwd(d["q"], d["k"], d["x"], d["y"], d["v"], d["s0"])
    cut = 100
    sl = lambda t, lo, hi: t[:, :, lo:hi].contiguous()
    o1, s1 = rd.ddts_fwd(*(sl(d[n], 0, cut) for n in "qkxyv"), d["s0"])
    o2, s2 = rd.ddts_fwd(*(sl(d[n], cut, 192) for n in "qkxyv"), s1)
    torch.cuda.synchronize()
    ro, rs = orc.ref_fwd(p.q, p.k, p.x, p.y, p.v, s0=p.s0)
    assert rel_err(host(torch.cat([o1, o2], dim=2)), ro) <= TOL_BF16
    assert rel_err(host(s2), rs) <= TOL_BF16 and rel_err(host(sT), rs) <= TOL_BF16
    # repeated decode steps from the same initial state
    state = d["s0"].clone()
    outs = []
    for t in range(192):
        outs.append(rd.ddts_step(*(d[n][:, :, t].contiguous() for n in "qkxyv"), state))
    torch.cuda.synchronize()
    assert rel_err(host(torch.stack(outs, dim=2)), ro) <= TOL_BF16
    assert rel_err(host(state), rs) <= TOL_F32


@pytest.mark.parametrize("xv,yv", [(8.0, 8.0), (-12.0, 0.0), (3.0, -2.0)])
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_strong_decay_and_long_memory(xv, yv, dtype):
    """Adversarial gates: about 8 nats of decay per step, and almost none."""
    p = wl.make_prefill(14, 1, 2, 150, 128, 128, dtype, s0_std=0.1)
    p.x[...] = xv
    p.y[...] = yv
    _check_prefill(p)


def test_bf16_mixed_decay_channels():
    """Fast- and slow-decaying channels side by side inside one chunk."""
    p = wl.make_prefill(15, 1, 2, 200, 128, 256, "bf16", s0_std=0.1)
    p.x[..., ::2] = wl.round_to_bf16(p.x[..., ::2] + 5.0)
    p.y[..., ::4] = 4.0
    _check_prefill(p)


def test_results_are_deterministic():
    import torch
    p = wl.make_prefill(16, 2, 2, 300, 128, 256, "bf16", s0_std=0.1)
    d = prefill_to_device(p)
    a = rd.ddts_fwd(d["q"], d["k"], d["x"], d["y"], d["v"], d["s0"])
    b = rd.ddts_fwd(d["q"], d["k"], d["x"], d["y"], d["v"], d["s0"])
    torch.cuda.synchronize()
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])


# ------------------------------------------------------------------------------------------
# varlen
# ------------------------------------------------------------------------------------------

def _varlen(seed, lens, H, dk, dv, dtype, s0_std=0.2):
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    return wl.make_prefill(seed, 1, H, int(cu[-1]), dk, dv, dtype, s0_std=s0_std, cu_seqlens=cu)


@pytest.mark.parametrize("dtype,dk,dv", [("bf16", 128, 256), ("f32", 64, 64), ("bf16", 128, 128)])
@pytest.mark.parametrize("host_cu", [True, False])
def test_varlen_matches_oracle(dtype, dk, dv, host_cu):
    lens = [5, 0, 130, 64, 1, 77, 0, 128, 63]
    p = _varlen(20, lens, 2, dk, dv, dtype)
    _check_prefill(p, host_cu=host_cu)


def _mixed_lengths(seed, n, longest=210):
    """Short sequences of every awkward length (0, 1, around one and two chunks, ...) in a
    seeded shuffle, so that empty ones sit between the others."""
    rng = np.random.default_rng(seed)
    base = [0, 1, 2, 63, 64, 65, 127, 128, 129, 130, 17, 200, 5, 96]
    lens = [base[i % len(base)] for i in range(n)]
    lens = [l if l else int(rng.integers(0, 2)) * int(rng.integers(1, longest)) for l in lens]
    rng.shuffle(lens)
    return [int(l) for l in lens]


@pytest.mark.parametrize("dv", [128, 256, 384])
@pytest.mark.parametrize("ingate", [rd.INGATE_POW_G, rd.INGATE_POW_SIGMOID])
@pytest.mark.parametrize("with_s0", [True, False])
def test_bf16_many_items_per_cta(dv, ingate, with_s0):
    """More (sequence, head, column slab) items than the persistent grids have CTAs, so every
    CTA (pair) walks a list of several items: state re-initialisation between items, reuse of
    tensor memory and of the operand ring across items, empty items inside the list."""
    H, n_seq = 4, 120
    lens = _mixed_lengths(50 + dv, n_seq)
    assert lens.count(0) >= 4 and n_seq * H * max(1, dv // 256) >= 3 * 148
    p = _varlen(60 + dv + ingate, lens, H, 128, dv, "bf16", s0_std=0.2 if with_s0 else None)
    d = prefill_to_device(p)
    prm = rd.fwd_params(d["q"], d["k"], d["x"], d["y"], d["v"], d["q"])
    assert rd.fwd_kernel_name(prm) == "tcgen05"
    _check_prefill(p, ingate, scale=0.5)


def test_bf16_more_sequences_than_the_planner_sorts():
    """Beyond 4096 packed sequences the planner keeps the given order for the rest, so empty
    sequences stay where the caller put them: in the middle of a CTA's list of items."""
    n_seq = 4096 + 160
    rng = np.random.default_rng(77)
    lens = rng.integers(1, 40, n_seq)
    lens[rng.random(n_seq) < 0.2] = 0
    lens[4096:] = [0, 33, 0, 0, 64, 1, 0, 65] * 20
    p = _varlen(78, [int(l) for l in lens], 1, 128, 256, "bf16", s0_std=0.2)
    _check_prefill(p, host_cu=False)
    p = _varlen(79, [int(l) for l in lens], 1, 128, 128, "bf16", s0_std=None)
    _check_prefill(p)


def test_varlen_no_leak_between_sequences():
    """Huge values in the neighbours must not reach a sequence's outputs or state."""
    import torch
    lens = [70, 33, 90]
    p = _varlen(21, lens, 2, 128, 256, "bf16")
    cu = p.cu_seqlens
    lo, hi = int(cu[1]), int(cu[2])
    clean_o, clean_s = _run_prefill(p)
    for name in ("q", "k", "v"):
        a = getattr(p, name)
        a[:, :, :lo] = wl.round_to_bf16(a[:, :, :lo] * 64.0 + 9.0)
        a[:, :, hi:] = wl.round_to_bf16(a[:, :, hi:] * 64.0 - 9.0)
    p.x[:, :, :lo] = 2.0
    p.x[:, :, hi:] = 2.0
    o, s = _run_prefill(p)
    assert np.array_equal(o[:, :, lo:hi], clean_o[:, :, lo:hi])
    assert np.array_equal(s[1], clean_s[1])
    assert not np.array_equal(s[0], clean_s[0])


def test_varlen_bad_seqlens_reported_by_device_without_fault():
    import torch
    p = _varlen(22, [40, 50, 30], 2, 128, 256, "bf16")
    d = prefill_to_device(p)
    bad = d["cu"].clone()
    bad[1] = 100            # decreases afterwards: 0,100,90,120
    B, H, T, dk = d["q"].shape
    o = torch.zeros((B, H, T, 256), dtype=torch.bfloat16, device="cuda")
    sT = torch.zeros((3, H, dk, 256), dtype=torch.float32, device="cuda")
    prm = rd.fwd_params(d["q"], d["k"], d["x"], d["y"], d["v"], o, d["s0"], sT, bad)
    ws = rd.new_workspace(prm, "cuda")
    prm.workspace, prm.workspace_bytes = ws.data_ptr(), ws.numel()
    assert rd.fwd_raw(prm) == rd.OK            # host had nothing to check
    assert rd.device_status(ws) == rd.ERR_SEQLENS
    assert torch.isfinite(o.float()).all()
    # with the host copy the same request is refused before any launch
    bad_host = bad.cpu()
    prm.cu_seqlens_host = bad_host.data_ptr()
    assert rd.fwd_raw(prm) == rd.ERR_SEQLENS
    # and a good request on the same workspace clears the device status
    prm.cu_seqlens, prm.cu_seqlens_host = d["cu"].data_ptr(), None
    assert rd.fwd_raw(prm) == rd.OK and rd.device_status(ws) == rd.OK


# ------------------------------------------------------------------------------------------
# the named configurations at full size, in the launch configuration the benchmark times
# ------------------------------------------------------------------------------------------

def test_config1_full_size():
    p = wl.config(1)
    assert p.shape == (4, 16, 2048, 128, 256)
    _check_prefill(p)
    _check_prefill(p, rd.INGATE_POW_SIGMOID)


def test_config2_full_size_and_split_halves():
    """T = 32768 with a nonzero initial state: every head against the oracle, and the GPU result
    must also equal two T = 16384 runs that pass the state across the split."""
    import torch
    p = wl.config(2)
    assert p.shape == (1, 16, 32768, 128, 256)
    d = prefill_to_device(p)
    o, sT = _nan_outputs(d)
    rd.ddts_fwd(d["q"], d["k"], d["x"], d["y"], d["v"], d["s0"], out=o, final_state=sT)
    half = 16384
    sl = lambda t, lo, hi: t[:, :, lo:hi].contiguous()
    o1, s1 = rd.ddts_fwd(*(sl(d[n], 0, half) for n in "qkxyv"), d["s0"])
    o2, s2 = rd.ddts_fwd(*(sl(d[n], half, 2 * half) for n in "qkxyv"), s1)
    torch.cuda.synchronize()
    ro, rs = orc.ref_fwd(p.q, p.k, p.x, p.y, p.v, s0=p.s0)
    for h in range(16):       # head by head: each against its own maximum
        assert rel_err(host(o[:, h]), ro[:, h]) <= TOL_BF16, h
        assert rel_err(host(sT[:, h]), rs[:, h]) <= TOL_BF16, h
        assert rel_err(host(torch.cat([o1[:, h], o2[:, h]], dim=1)), ro[:, h]) <= TOL_BF16, h
        assert rel_err(host(s2[:, h]), rs[:, h]) <= TOL_BF16, h
    # the halves and the single run follow the same chunk grid, so they agree far tighter
    assert rel_err(host(torch.cat([o1, o2], dim=2)), host(o)) <= 1e-2


@pytest.mark.gpu
def test_time_split_with_the_alternate_input_gate_and_fast_decay():
    """The split's state-only instantiation exists per input-gate mode, and a segment's decay
    product can underflow to zero (strong decay): both must still give the sequential result."""
    import torch
    B, H, T, dv = 1, 3, 4500, 256
    for ingate, gate_mean in ((rd.INGATE_POW_SIGMOID, -3.0), (rd.INGATE_POW_G, 1.5)):
        p = wl.make_prefill(900 + ingate, B, H, T, 128, dv, "bf16", gate_mean=gate_mean, s0_std=0.3)
        d = prefill_to_device(p)
        o = torch.full((B, H, T, dv), float("nan"), dtype=torch.bfloat16, device="cuda")
        sT = torch.full((B, H, 128, dv), float("nan"), dtype=torch.float32, device="cuda")
        prm = rd.fwd_params(d["q"], d["k"], d["x"], d["y"], d["v"], o, d["s0"], sT, ingate=ingate)
        need = rd.fwd_workspace_bytes(prm)
        ws = torch.empty(need, dtype=torch.uint8, device="cuda")
        prm.workspace, prm.workspace_bytes = ws.data_ptr(), need
        assert rd.fwd_raw(prm) == rd.OK and rd.last_launch_count() == 5
        assert rd.device_status(ws) == rd.OK
        ro, rs = orc.ref_fwd(p.q, p.k, p.x, p.y, p.v, s0=p.s0, ingate=ingate)
        assert rel_err(host(o), ro) <= TOL_BF16 and rel_err(host(sT), rs) <= TOL_BF16


@pytest.mark.gpu
def test_time_split_from_two_host_threads():
    """Two host threads, each on its own stream, issue split calls at the same time (the C call
    runs without the interpreter lock): the library's one extra stream per device is shared, so
    the fork and join of one call must not pick up the other call's events."""
    import threading
    import torch
    B, H, T, dv = 1, 2, 4300, 256
    results = {}

    def worker(tag):
        torch.cuda.set_device(0)
        stream = torch.cuda.Stream()
        outs = []
        with torch.cuda.stream(stream):
            for i in range(4):
                p = wl.make_prefill(1200 + 10 * tag + i, B, H, T, 128, dv, "bf16", s0_std=0.1)
                d = prefill_to_device(p)
                o = torch.full((B, H, T, dv), float("nan"), dtype=torch.bfloat16, device="cuda")
                sT = torch.full((B, H, 128, dv), float("nan"), dtype=torch.float32, device="cuda")
                prm = rd.fwd_params(d["q"], d["k"], d["x"], d["y"], d["v"], o, d["s0"], sT)
                need = rd.fwd_workspace_bytes(prm)
                ws = torch.empty(need, dtype=torch.uint8, device="cuda")
                prm.workspace, prm.workspace_bytes = ws.data_ptr(), need
                rc = rd.fwd_raw(prm)
                outs.append((rc, p, o, sT, ws, d))
            stream.synchronize()
        results[tag] = outs

    threads = [threading.Thread(target=worker, args=(t,)) for t in (0, 1)]
    for t in threads: t.start()
    for t in threads: t.join()
    for tag in (0, 1):
        for rc, p, o, sT, ws, _ in results[tag]:
            assert rc == rd.OK and rd.device_status(ws) == rd.OK
            ro, rs = orc.ref_fwd(p.q, p.k, p.x, p.y, p.v, s0=p.s0)
            assert rel_err(host(o), ro) <= TOL_BF16 and rel_err(host(sT), rs) <= TOL_BF16


@pytest.mark.gpu
def test_time_split_on_a_user_stream_back_to_back():
    """The time split forks to a second stream and joins again: on a non-default user stream,
    with calls issued back to back into the same buffers' successors and read on that stream
    without any device-wide synchronisation, every call must see its own complete result."""
    import torch
    B, H, T, dv = 1, 2, 5000, 256
    ps = [wl.make_prefill(700 + i, B, H, T, 128, dv, "bf16", s0_std=0.1) for i in range(3)]
    side = torch.cuda.Stream()
    outs = []
    with torch.cuda.stream(side):
        ds = [prefill_to_device(p) for p in ps]
        for d in ds:
            o = torch.full((B, H, T, dv), float("nan"), dtype=torch.bfloat16, device="cuda")
            sT = torch.full((B, H, 128, dv), float("nan"), dtype=torch.float32, device="cuda")
            prm = rd.fwd_params(d["q"], d["k"], d["x"], d["y"], d["v"], o, d["s0"], sT)
            need = rd.fwd_workspace_bytes(prm)
            ws = torch.empty(need, dtype=torch.uint8, device="cuda")
            prm.workspace, prm.workspace_bytes = ws.data_ptr(), need
            assert rd.fwd_raw(prm) == rd.OK and rd.last_launch_count() == 5
            # consumers on the same stream, queued right behind the call
            outs.append((o.float().sum(dim=-1), sT.clone(), o, ws))
        side.synchronize()
    for p, (osum, sT, o, ws) in zip(ps, outs):
        assert rd.device_status(ws) == rd.OK
        ro, rs = orc.ref_fwd(p.q, p.k, p.x, p.y, p.v, s0=p.s0)
        assert rel_err(host(o), ro) <= TOL_BF16 and rel_err(host(sT), rs) <= TOL_BF16
        assert rel_err(host(osum), np.asarray(host(o), dtype=np.float64).sum(axis=-1)) <= 1e-2


@pytest.mark.parametrize("B,H,T,dv,with_s0", [
    (1, 2, 4096 + 100, 256, True),     # head segment + two segments, ragged last segment
    (2, 3, 6500, 256, False),          # six (batch, head) pairs, head segment + three segments
    (1, 1, 9000, 512, True),           # two 256-column slabs per head, head segment + four segments
])
def test_long_sequences_split_along_time(B, H, T, dv, with_s0):
    """Dense calls with fewer heads than CTA pairs are cut into time segments joined through the
    linear state recurrence (five launches: segment table, state-only pass and head segment side
    by side, combine, full pass); outputs and final state must still match the sequential oracle,
    and must agree with the unsplit kernel (base-size workspace) far more tightly."""
    import torch
    p = wl.make_prefill(31 + T, B, H, T, 128, dv, "bf16", s0_std=0.2 if with_s0 else None)
    d = prefill_to_device(p)
    o = torch.full((B, H, T, dv), float("nan"), dtype=torch.bfloat16, device="cuda")
    sT = torch.full((B, H, 128, dv), float("nan"), dtype=torch.float32, device="cuda")
    prm = rd.fwd_params(d["q"], d["k"], d["x"], d["y"], d["v"], o, d["s0"], sT, scale=0.5)
    need = rd.fwd_workspace_bytes(prm)
    assert need > 4096, "this shape should ask for the segments' state workspace"
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    prm.workspace, prm.workspace_bytes = ws.data_ptr(), need
    assert rd.fwd_raw(prm) == rd.OK and rd.last_launch_count() == 5
    assert rd.device_status(ws) == rd.OK
    ro, rs = orc.ref_fwd(p.q, p.k, p.x, p.y, p.v, s0=p.s0, scale=0.5)
    assert rel_err(host(o), ro) <= TOL_BF16 and rel_err(host(sT), rs) <= TOL_BF16
    # same request with only the base workspace: one launch, no split
    o1, s1 = torch.full_like(o, float("nan")), torch.full_like(sT, float("nan"))
    prm1 = rd.fwd_params(d["q"], d["k"], d["x"], d["y"], d["v"], o1, d["s0"], s1, scale=0.5)
    ws1 = torch.empty(256, dtype=torch.uint8, device="cuda")
    prm1.workspace, prm1.workspace_bytes = ws1.data_ptr(), 256
    assert rd.fwd_raw(prm1) == rd.OK and rd.last_launch_count() == 1
    torch.cuda.synchronize()
    assert rel_err(host(o), host(o1)) <= 1e-2 and rel_err(host(sT), host(s1)) <= 1e-2
    # output only (no final state wanted), into a fresh buffer
    o2 = torch.full_like(o, float("nan"))
    prm.o, prm.sT = o2.data_ptr(), None
    assert rd.fwd_raw(prm) == rd.OK
    torch.cuda.synchronize()
    assert rel_err(host(o2), ro) <= TOL_BF16


def test_config4_full_size_every_sequence():
    """All 64 packed sequences x 16 heads against the oracle, outputs and final states judged
    sequence by sequence (the oracle runs four heads at a time to bound host memory)."""
    import torch
    p = wl.config(4)
    cu = p.cu_seqlens
    assert len(cu) == 65 and p.shape[1] == 16
    d = prefill_to_device(p)
    o, sT = _nan_outputs(d)
    rd.ddts_fwd(d["q"], d["k"], d["x"], d["y"], d["v"], None, d["cu"], d["cu_host"], out=o,
                final_state=sT)
    torch.cuda.synchronize()
    for h0 in range(0, 16, 4):
        hs = slice(h0, h0 + 4)
        sl = lambda a: np.ascontiguousarray(a[:, hs])
        ro, rs = orc.ref_fwd(sl(p.q), sl(p.k), sl(p.x), sl(p.y), sl(p.v), cu_seqlens=cu)
        eo, es = _worst_err(host(o[:, hs]), host(sT[:, hs]), ro, rs, cu)
        assert eo <= TOL_BF16 and es <= TOL_BF16, (h0, eo, es)


# ------------------------------------------------------------------------------------------
# bounded waits: a wait that runs out is reported, nothing hangs, the device stays usable
# ------------------------------------------------------------------------------------------

@pytest.mark.parametrize("dv", [256, 128])      # cluster-pair kernel / single-CTA kernel
def test_wait_that_runs_out_is_reported_and_the_next_call_is_clean(dv):
    """The main-loop waits of the tensor-core kernels take their bound from the launch.  With a
    bound of zero the first wait that is not satisfied at once gives up (at kernel start the
    issuer always finds no pass published yet): the call itself returns OK, the kernel ends by
    its teardown path, the status word says TIMEOUT; a normal call on the same workspace then
    reports OK and matches the oracle."""
    import torch
    p = wl.make_prefill(40 + dv, 1, 1, 64, 128, dv, "bf16", s0_std=0.1)
    d = prefill_to_device(p)
    o, sT = _nan_outputs(d)
    prm = rd.fwd_params(d["q"], d["k"], d["x"], d["y"], d["v"], o, d["s0"], sT)
    ws = rd.new_workspace(prm, "cuda")
    prm.workspace, prm.workspace_bytes = ws.data_ptr(), ws.numel()
    try:
        rd.test_set_wait_limit(0)
        assert rd.fwd_raw(prm) == rd.OK
        assert rd.device_status(ws) == rd.ERR_TIMEOUT
    finally:
        rd.test_set_wait_limit(-1)
    o, sT = _nan_outputs(d)
    prm.o, prm.sT = o.data_ptr(), sT.data_ptr()
    assert rd.fwd_raw(prm) == rd.OK
    assert rd.device_status(ws) == rd.OK
    ro, rs = orc.ref_fwd(p.q, p.k, p.x, p.y, p.v, s0=p.s0)
    assert rel_err(host(o), ro) <= TOL_BF16 and rel_err(host(sT), rs) <= TOL_BF16


# ------------------------------------------------------------------------------------------
# optional terms of the full block: value gate beta_hat (multiplies v) and feed-through d . x'
# ------------------------------------------------------------------------------------------

def _block_terms(p, seed, H):
    """Seeded beta_hat in (0, 1) (a sigmoid's range), d ~ N(0, 1), x' ~ N(0, 1), rounded to the
    workload's dtype where the GPU reads them in it."""
    rng = np.random.default_rng(seed)
    dv = p.v.shape[-1]
    rnd = wl.round_to_bf16 if p.dtype == "bf16" else (lambda a: a.astype(np.float32))
    beta = rnd(rng.random(p.v.shape, dtype=np.float32))
    fx = rnd(rng.standard_normal(p.v.shape, dtype=np.float32))
    d = rng.standard_normal((H, dv), dtype=np.float32)
    return beta, d, fx


def _check_block(p, which="both", ingate=rd.INGATE_POW_G, scale=0.5, expect_kernel=None, ws_bytes=None):
    import torch
    B, H, T, dk, dv = p.shape
    beta, d, fx = _block_terms(p, 5, H)
    use_b, use_f = which in ("both", "gate"), which in ("both", "feed")
    dd = prefill_to_device(p)
    o, sT = _nan_outputs(dd)
    kw = dict(beta_hat=dev(beta, p.dtype) if use_b else None,
              feed_d=torch.from_numpy(d).cuda() if use_f else None,
              feed_x=dev(fx, p.dtype) if use_f else None)
    prm = rd.fwd_params(dd["q"], dd["k"], dd["x"], dd["y"], dd["v"], o, dd["s0"], sT, dd["cu"],
                        dd["cu_host"], None, scale, ingate, **kw)
    if expect_kernel:
        assert rd.fwd_kernel_name(prm) == expect_kernel
    need = rd.fwd_workspace_bytes(prm) if ws_bytes is None else ws_bytes
    ws = torch.empty(max(need, 256), dtype=torch.uint8, device="cuda")
    prm.workspace, prm.workspace_bytes = ws.data_ptr(), ws.numel()
    assert rd.fwd_raw(prm) == rd.OK and rd.device_status(ws) == rd.OK
    ro, rs = orc.ref_fwd(p.q, p.k, p.x, p.y, p.v, s0=p.s0, cu_seqlens=p.cu_seqlens, scale=scale,
                         ingate=ingate, beta_hat=beta if use_b else None,
                         feed_d=d if use_f else None, feed_x=fx if use_f else None)
    tol = _tol(p.dtype)
    eo, es = _worst_err(host(o), host(sT), ro, rs, p.cu_seqlens)
    assert eo <= tol and es <= tol, (which, eo, es)
    return rd.last_launch_count()


@pytest.mark.parametrize("which", ["both", "gate", "feed"])
@pytest.mark.parametrize("ingate", [rd.INGATE_POW_G, rd.INGATE_POW_SIGMOID])
def test_block_terms_bf16_tensor_core_kernel(which, ingate):
    p = wl.make_prefill(501, 2, 2, 200, 128, 256, "bf16", s0_std=0.1)       # ragged last tile
    _check_block(p, which, ingate, expect_kernel="tcgen05")
    p = wl.make_prefill(502, 1, 3, 64, 128, 512, "bf16")                    # two slabs per head
    _check_block(p, which, ingate, expect_kernel="tcgen05")


def test_block_terms_bf16_packed_sequences_many_items():
    lens = _mixed_lengths(503, 100)
    p = _varlen(504, lens, 4, 128, 256, "bf16", s0_std=0.2)
    _check_block(p, "both")


def test_block_terms_with_the_time_split():
    p = wl.make_prefill(505, 1, 2, 4500, 128, 256, "bf16", s0_std=0.2)
    assert _check_block(p, "both") == 5                                     # split: five launches
    assert _check_block(p, "both", ws_bytes=256) == 1                       # same request, unsplit


@pytest.mark.parametrize("dtype,dk,dv", [("f32", 64, 64), ("bf16", 128, 128), ("bf16", 48, 80)])
def test_block_terms_cuda_core_kernel(dtype, dk, dv):
    p = wl.make_prefill(506, 1, 2, 90, dk, dv, dtype, s0_std=0.2)
    _check_block(p, "both", expect_kernel="simt")
    _check_block(p, "gate", rd.INGATE_POW_SIGMOID)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_block_terms_decode_steps(dtype):
    import torch
    Nseq, H, dk, dv = 5, 3, 128, 256
    w = wl.make_decode(507, Nseq, H, dk, dv, ring=4, dtype=dtype)
    rng = np.random.default_rng(6)
    rnd = wl.round_to_bf16 if dtype == "bf16" else (lambda a: a.astype(np.float32))
    beta = rnd(rng.random((4, Nseq, H, dv), dtype=np.float32))
    fx = rnd(rng.standard_normal((4, Nseq, H, dv), dtype=np.float32))
    d = rng.standard_normal((H, dv), dtype=np.float32)
    state = torch.from_numpy(w.state).cuda()
    ref_state = w.state.astype(np.float64)
    for s in range(4):
        o = rd.ddts_step(*(dev(a[s], dtype) for a in (w.q, w.k, w.x, w.y, w.v)), state, scale=0.5,
                         beta_hat=dev(beta[s], dtype), feed_d=torch.from_numpy(d).cuda(),
                         feed_x=dev(fx[s], dtype))
        ro = orc.ref_step(w.q[s], w.k[s], w.x[s], w.y[s], w.v[s], ref_state, scale=0.5,
                          beta_hat=beta[s], feed_d=d, feed_x=fx[s])
        assert rel_err(host(o), ro) <= _tol(dtype)
    assert rel_err(host(state), ref_state) <= TOL_F32


# ------------------------------------------------------------------------------------------
# value-side decay beta_t of the general transition (the arm the paper ablates and drops)
# ------------------------------------------------------------------------------------------

@pytest.mark.parametrize("dtype,dk,dv", [("f32", 64, 64), ("bf16", 128, 256), ("f32", 48, 80)])
@pytest.mark.parametrize("with_gate", [False, True])
def test_value_decay_prefill(dtype, dk, dv, with_gate):
    import torch
    p = wl.make_prefill(801, 2, 2, 90, dk, dv, dtype, s0_std=0.2)            # chunks and a ragged tail
    beta = wl.make_value_decay(802, p.v.shape, dtype)
    bhat, d, fx = _block_terms(p, 803, 2)
    dd = prefill_to_device(p)
    o, sT = _nan_outputs(dd)
    kw = dict(value_decay=dev(beta, dtype))
    ref_kw = dict(value_decay=beta)
    if with_gate:
        kw.update(beta_hat=dev(bhat, dtype), feed_d=torch.from_numpy(d).cuda(), feed_x=dev(fx, dtype))
        ref_kw.update(beta_hat=bhat, feed_d=d, feed_x=fx)
    prm = rd.fwd_params(dd["q"], dd["k"], dd["x"], dd["y"], dd["v"], o, dd["s0"], sT, scale=0.5, **kw)
    assert rd.fwd_kernel_name(prm) == "simt"                  # also for the tensor-core shape
    ws = rd.new_workspace(prm, "cuda")
    prm.workspace, prm.workspace_bytes = ws.data_ptr(), ws.numel()
    assert rd.fwd_raw(prm) == rd.OK and rd.device_status(ws) == rd.OK
    ro, rs = orc.ref_fwd(p.q, p.k, p.x, p.y, p.v, s0=p.s0, scale=0.5, **ref_kw)
    # the fp32 kernel computes in fp32 whatever the token dtype; bf16 only rounds o
    assert rel_err(host(o), ro) <= _tol(dtype) and rel_err(host(sT), rs) <= TOL_F32


def test_value_decay_with_shared_gates():
    """The value-side decay together with the one-set-per-token layout (both go to the fp32 kernel)."""
    pq, pv = _shared_inputs(821, 2, 3, 75, 64, 64, "f32")
    beta = wl.make_value_decay(822, pv.v.shape, "f32")
    dq_ = {n: dev(getattr(pq, n), "f32") for n in ("q", "k", "x", "y")}
    import torch
    o, sT = rd.ddts_fwd(dq_["q"], dq_["k"], dq_["x"], dq_["y"], dev(pv.v, "f32"),
                        torch.from_numpy(pv.s0).cuda(), value_decay=dev(beta, "f32"))
    ro, rs = orc.ref_fwd(pq.q, pq.k, pq.x, pq.y, pv.v, s0=pv.s0, shared_gates=True, value_decay=beta)
    assert rel_err(host(o), ro) <= TOL_F32 and rel_err(host(sT), rs) <= TOL_F32


def test_value_decay_packed_sequences_and_decode_steps():
    import torch
    lens = [33, 0, 1, 70]
    p = _varlen(811, lens, 2, 128, 256, "bf16", s0_std=0.2)
    beta = wl.make_value_decay(812, p.v.shape, "bf16")
    dd = prefill_to_device(p)
    o, sT = rd.ddts_fwd(dd["q"], dd["k"], dd["x"], dd["y"], dd["v"], dd["s0"], dd["cu"], dd["cu_host"],
                        value_decay=dev(beta, "bf16"))
    ro, rs = orc.ref_fwd(p.q, p.k, p.x, p.y, p.v, s0=p.s0, cu_seqlens=p.cu_seqlens, value_decay=beta)
    eo, es = _worst_err(host(o), host(sT), ro, rs, p.cu_seqlens)
    assert eo <= TOL_BF16 and es <= TOL_F32
    # decode: four steps with a decay per step, bf16 and fp32 tokens
    for dtype in ("bf16", "f32"):
        Nseq, H, dk, dv = 5, 3, 128, 256
        w = wl.make_decode(813, Nseq, H, dk, dv, ring=4, dtype=dtype)
        bd = wl.make_value_decay(814, (4, Nseq, H, dv), dtype)
        state = torch.from_numpy(w.state).cuda()
        ref_state = w.state.astype(np.float64)
        for s in range(4):
            og = rd.ddts_step(*(dev(a[s], dtype) for a in (w.q, w.k, w.x, w.y, w.v)), state, scale=0.5,
                              value_decay=dev(bd[s], dtype))
            rg = orc.ref_step(w.q[s], w.k[s], w.x[s], w.y[s], w.v[s], ref_state, scale=0.5,
                              value_decay=bd[s])
            assert rel_err(host(og), rg) <= _tol(dtype)
        assert rel_err(host(state), ref_state) <= TOL_F32


# ------------------------------------------------------------------------------------------
# shared-gate layout: q,k,x,y [B,1,T,dk], one set per token for all H groups of value columns
# ------------------------------------------------------------------------------------------

def _shared_inputs(seed, B, H, T, dk, dv, dtype, s0_std=0.1, cu=None, gate_mean=-3.0):
    """A workload whose q,k,x,y have a single head; v and the states keep H heads."""
    pq = wl.make_prefill(seed, B, 1, T, dk, dv, dtype, gate_mean=gate_mean)
    pv = wl.make_prefill(seed + 1, B, H, T, dk, dv, dtype, s0_std=s0_std, cu_seqlens=cu)
    return pq, pv


def _check_shared(seed, B, H, T, dk, dv, dtype, cu=None, block=False, expect_kernel=None, ingate=rd.INGATE_POW_G):
    import torch
    pq, pv = _shared_inputs(seed, B, H, T, dk, dv, dtype, cu=cu)
    beta, d, fx = _block_terms(pv, 7, H)
    up = lambda a: dev(a, dtype)
    q, k, x, y, v = up(pq.q), up(pq.k), up(pq.x), up(pq.y), up(pv.v)
    s0 = torch.from_numpy(pv.s0).cuda()
    cu_d = None if cu is None else torch.from_numpy(cu).cuda()
    cu_h = None if cu is None else torch.from_numpy(cu)
    nseq = B if cu is None else len(cu) - 1
    o = torch.full((B, H, T, dv), float("nan"), dtype=q.dtype, device="cuda")
    sT = torch.full((nseq, H, dk, dv), float("nan"), dtype=torch.float32, device="cuda")
    kw = dict(beta_hat=up(beta), feed_d=torch.from_numpy(d).cuda(), feed_x=up(fx)) if block else {}
    prm = rd.fwd_params(q, k, x, y, v, o, s0, sT, cu_d, cu_h, None, 0.5, ingate, **kw)
    assert prm.shared_gates == 1 and prm.H == H
    if expect_kernel:
        assert rd.fwd_kernel_name(prm) == expect_kernel
    ws = torch.empty(max(rd.fwd_workspace_bytes(prm), 256), dtype=torch.uint8, device="cuda")
    prm.workspace, prm.workspace_bytes = ws.data_ptr(), ws.numel()
    assert rd.fwd_raw(prm) == rd.OK and rd.device_status(ws) == rd.OK
    okw = dict(beta_hat=beta, feed_d=d, feed_x=fx) if block else {}
    ro, rs = orc.ref_fwd(pq.q, pq.k, pq.x, pq.y, pv.v, s0=pv.s0, cu_seqlens=cu, scale=0.5,
                         ingate=ingate, shared_gates=True, **okw)
    eo, es = _worst_err(host(o), host(sT), ro, rs, cu)
    tol = _tol(dtype)
    assert eo <= tol and es <= tol, (eo, es)
    return rd.last_launch_count()


@pytest.mark.parametrize("ingate", [rd.INGATE_POW_G, rd.INGATE_POW_SIGMOID])
def test_shared_gates_tensor_core_kernel(ingate):
    _check_shared(601, 2, 4, 200, 128, 256, "bf16", expect_kernel="tcgen05", ingate=ingate)
    _check_shared(603, 1, 3, 130, 128, 512, "bf16", block=True, ingate=ingate)


def test_shared_gates_packed_and_time_split():
    lens = _mixed_lengths(605, 40)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    _check_shared(606, 1, 4, int(cu[-1]), 128, 256, "bf16", cu=cu)
    assert _check_shared(608, 2, 2, 4500, 128, 256, "bf16") == 5     # (batch, head) units split along time


@pytest.mark.parametrize("dtype,dk,dv,H", [("f32", 64, 64, 4), ("bf16", 64, 256, 16), ("bf16", 128, 128, 3)])
def test_shared_gates_cuda_core_kernel(dtype, dk, dv, H):
    """dk = 64 with 16 groups of 256 value columns is the paper's own state shape (64 x 2d)."""
    _check_shared(610, 1, H, 70, dk, dv, dtype, expect_kernel="simt")
    lens = [5, 0, 33, 17]
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    _check_shared(612, 1, H, int(cu[-1]), dk, dv, dtype, cu=cu, block=True)


def test_shared_gates_decode_steps():
    import torch
    Nseq, H, dk, dv = 6, 4, 64, 256
    wq = wl.make_decode(620, Nseq, 1, dk, dv, ring=3)
    wv = wl.make_decode(621, Nseq, H, dk, dv, ring=3)
    state = torch.from_numpy(wv.state).cuda()
    ref_state = wv.state.astype(np.float64)
    for s in range(3):
        o = rd.ddts_step(*(dev(a[s], "bf16") for a in (wq.q, wq.k, wq.x, wq.y, wv.v)), state)
        ro = orc.ref_step(wq.q[s], wq.k[s], wq.x[s], wq.y[s], wv.v[s], ref_state, shared_gates=True)
        assert o.shape == (Nseq, H, dv) and rel_err(host(o), ro) <= TOL_BF16
    assert rel_err(host(state), ref_state) <= TOL_F32
