"""GPU parity of the sliding-window shared-key attention (``rodimus_swska_fwd``) against its fp64
oracle on the same seeded inputs: max|err|/max|ref| <= 2e-2 for bf16 (bf16 probabilities and
operands, fp32 accumulation) and <= 1e-4 for the fp32 validation kernel."""
import numpy as np
import pytest

import paper_2410_06577_b200 as rd
from paper_2410_06577_b200 import workloads as wl
from oracle import swska_oracle as sw
from tests._util import TOL_BF16, TOL_F32, dev, host, rel_err

pytestmark = pytest.mark.gpu


def _run(q, k, v, window, scale, dtype):
    import torch
    dq, dk, dv_ = dev(q, dtype), dev(k, dtype), dev(v, dtype)
    o = torch.full_like(dq, float("nan"))          # a row the kernel never stores stays NaN
    rd.swska_fwd(dq, dk, dv_, window, scale, out=o)
    torch.cuda.synchronize()
    return host(o)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("B,H,T,window", [
    (1, 1, 1, 1),          # one token
    (2, 3, 64, 64),        # one tile, window = everything
    (1, 2, 150, 40),       # ragged last tile, window inside a tile and across two
    (2, 2, 333, 128),      # several tiles, window of two tiles
    (1, 2, 200, 1),        # every token sees only itself
    (1, 2, 260, 1000),     # window longer than the sequence: plain causal attention
    (1, 1, 300, 65),       # window one past a tile: three tiles touch a query tile
    (3, 5, 129, 129),      # one row past a query tile, odd batch and head counts
    (1, 2, 513, 200),      # five query tiles, window of three key tiles and a bit
])
def test_swska_matches_oracle(dtype, B, H, T, window):
    q, k, v = wl.make_swska(900 + T, B, H, T, 128, dtype)
    scale = 128 ** -0.5
    got = _run(q, k, v, window, scale, dtype)
    ref = sw.swska_ref(q, k, v, window, scale)
    assert rel_err(got, ref) <= (TOL_BF16 if dtype == "bf16" else TOL_F32)


def test_swska_peaked_scores_and_large_scale():
    # scale 1 with N(0,1) inputs of width 128: scores of +-30, softmax close to one-hot; the
    # running maximum must keep exp2 in range and the normalisation exact
    q, k, v = wl.make_swska(950, 1, 2, 256, 128, "bf16")
    got = _run(q, k, v, 100, 1.0, "bf16")
    assert rel_err(got, sw.swska_ref(q, k, v, 100, 1.0)) <= TOL_BF16


def test_swska_layer_shape_sampled_heads():
    """B=4, H=16, T=2048, window 1024 (half the context) in one call; the oracle checks two heads."""
    q, k, v = wl.make_swska(960, 4, 16, 2048, 128, "bf16")
    got = _run(q, k, v, 1024, 128 ** -0.5, "bf16")
    assert np.all(np.isfinite(got))
    for b, h in ((0, 0), (3, 11)):
        ref = sw.swska_ref(q[b:b + 1, h:h + 1], k[b:b + 1], v[b:b + 1, h:h + 1], 1024, 128 ** -0.5)
        assert rel_err(got[b:b + 1, h:h + 1], ref) <= TOL_BF16


def test_swska_wait_that_runs_out_is_reported_and_leaves_the_device_usable():
    """With the wait limit set to zero the tensor-core kernel's first unsatisfied wait runs out: the
    kernel must end by itself, report RODIMUS_ERR_TIMEOUT in the status word and leave the device
    usable; the next call, with the default limit, is correct."""
    import torch
    q, k, v = wl.make_swska(970, 1, 2, 300, 128, "bf16")
    dq, dk, dv_ = dev(q, "bf16"), dev(k, "bf16"), dev(v, "bf16")
    o = torch.zeros_like(dq)
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    prm = rd.swska_params(dq, dk, dv_, o, 100, 128 ** -0.5, workspace=ws)
    rd.test_set_wait_limit(0)
    try:
        assert rd.swska_raw(prm) == rd.OK
        assert rd.device_status(ws) == rd.ERR_TIMEOUT
    finally:
        rd.test_set_wait_limit(-1)
    o = torch.full_like(dq, float("nan"))
    prm = rd.swska_params(dq, dk, dv_, o, 100, 128 ** -0.5, workspace=ws)
    assert rd.swska_raw(prm) == rd.OK
    assert rd.device_status(ws) == rd.OK
    assert rel_err(host(o), sw.swska_ref(q, k, v, 100, 128 ** -0.5)) <= TOL_BF16
