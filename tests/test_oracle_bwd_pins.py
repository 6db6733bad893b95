"""Pins for the backward oracle (``ref_bwd``): each check compares the adjoint recurrence with
something fixed outside it - finite differences of the forward oracle, reverse-mode differentiation
of a separately written forward by an autograd library, a single step worked out by hand, and
structural properties (linearity in the incoming gradients, chaining of two calls).  CPU only.
"""
import numpy as np
import pytest

from oracle import ddts_oracle as orc

MODES = [orc.POW_G, orc.POW_SIGMOID]
NAMES = ("dq", "dk", "dx", "dy", "dv")


def _grid(a, step=2.0 ** -6):
    """Round to a coarse binary grid so that +-2^-10 perturbations stay exact in float32."""
    return (np.round(np.asarray(a, dtype=np.float64) / step) * step).astype(np.float32)


def _draw(seed, B, H, T, dk, dv, gate_mean=-1.0):
    rng = np.random.default_rng(seed)
    q = _grid(rng.standard_normal((B, H, T, dk)))
    k = _grid(rng.standard_normal((B, H, T, dk)))
    v = _grid(rng.standard_normal((B, H, T, dv)))
    x = _grid(rng.standard_normal((B, H, T, dk)) + gate_mean)
    y = _grid(rng.standard_normal((B, H, T, dk)))
    do = _grid(rng.standard_normal((B, H, T, dv)))
    return q, k, x, y, v, do


def _rel(a, b):
    return np.max(np.abs(a - b)) / max(np.max(np.abs(b)), 1e-300)


def _loss(q, k, x, y, v, do, s0, dsT, **kw):
    o, sT = orc.ref_fwd(q, k, x, y, v, s0=s0, **kw)
    L = float(np.sum(o * do.astype(np.float64)))
    if dsT is not None:
        L += float(np.sum(sT * dsT))
    return L


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("with_state", [False, True])
def test_matches_central_finite_differences_of_the_forward(mode, with_state):
    B, H, T, dk, dv = 1, 2, 40, 5, 3          # 40 steps: crosses a storage block of the oracle
    q, k, x, y, v, do = _draw(3, B, H, T, dk, dv)
    rng = np.random.default_rng(4)
    s0 = rng.standard_normal((B, H, dk, dv)) if with_state else None
    dsT = rng.standard_normal((B, H, dk, dv)) if with_state else None
    kw = dict(scale=0.7, ingate=mode)
    g = orc.ref_bwd(q, k, x, y, v, do, s0=s0, dsT=dsT, **kw)
    eps = 2.0 ** -10
    ins = {"dq": q, "dk": k, "dx": x, "dy": y, "dv": v}
    pick = np.random.default_rng(5)
    for name, arr in ins.items():
        worst = 0.0
        scale_ref = np.max(np.abs(g[name]))
        for _ in range(24):
            idx = tuple(int(pick.integers(0, n)) for n in arr.shape)
            args = {n: a for n, a in ins.items()}
            up, dn = arr.copy(), arr.copy()
            up[idx] += eps
            dn[idx] -= eps
            assert float(up[idx]) - float(dn[idx]) == 2 * eps      # exact in float32
            Lp = _loss(**{n[1:]: (up if n == name else a) for n, a in args.items()},
                       do=do, s0=s0, dsT=dsT, **kw)
            Lm = _loss(**{n[1:]: (dn if n == name else a) for n, a in args.items()},
                       do=do, s0=s0, dsT=dsT, **kw)
            fd = (Lp - Lm) / (2 * eps)
            worst = max(worst, abs(fd - g[name][idx]) / scale_ref)
        assert worst < 2e-5, (name, worst)        # O(eps^2) truncation of the difference quotient
    if with_state:
        # the initial state is a float64 input of the forward: a small step is exact enough
        for _ in range(12):
            idx = tuple(int(pick.integers(0, n)) for n in s0.shape)
            up, dn = s0.copy(), s0.copy()
            up[idx] += 1e-4
            dn[idx] -= 1e-4
            fd = (_loss(q, k, x, y, v, do, up, dsT, **kw) - _loss(q, k, x, y, v, do, dn, dsT, **kw)) / 2e-4
            assert abs(fd - g["ds0"][idx]) < 1e-8 * max(1.0, np.max(np.abs(g["ds0"])))


@pytest.mark.parametrize("mode", MODES)
def test_matches_autograd_of_a_separately_written_forward(mode):
    torch = pytest.importorskip("torch")
    B, H, T, dk, dv = 2, 2, 70, 6, 5
    q, k, x, y, v, do = _draw(11, B, H, T, dk, dv)
    rng = np.random.default_rng(12)
    s0 = rng.standard_normal((B, H, dk, dv))
    dsT = rng.standard_normal((B, H, dk, dv))
    t = {n: torch.tensor(a.astype(np.float64), requires_grad=True)
         for n, a in dict(q=q, k=k, x=x, y=y, v=v).items()}
    S = torch.tensor(s0, requires_grad=True)
    S0 = S
    g = torch.nn.functional.softplus(t["x"])
    tau = torch.sigmoid(t["y"])
    alpha = torch.exp(-g * tau)
    ahat = g ** tau if mode == orc.POW_G else (1 - torch.exp(-g)) ** tau
    L = 0.0
    for i in range(T):   # Eq. "rodimus_recurrent_form", written with whole-tensor operations
        S = alpha[:, :, i, :, None] * S + (ahat[:, :, i] * t["k"][:, :, i])[..., None] * t["v"][:, :, i, None, :]
        o = 0.7 * torch.einsum("bhd,bhdj->bhj", t["q"][:, :, i], S)
        L = L + (o * torch.tensor(do[:, :, i].astype(np.float64))).sum()
    L = L + (S * torch.tensor(dsT)).sum()
    L.backward()
    got = orc.ref_bwd(q, k, x, y, v, do, s0=s0, dsT=dsT, scale=0.7, ingate=mode)
    for name in NAMES:
        assert _rel(got[name], t[name[1:]].grad.numpy()) < 1e-11, name
    assert _rel(got["ds0"], S0.grad.numpy()) < 1e-11


@pytest.mark.parametrize("mode", MODES)
def test_single_step_by_hand(mode):
    # T = 1: o = c (q . (alpha s0 + ahat k v)); every derivative is one line
    dk, dv = 4, 3
    q, k, x, y, v, do = _draw(21, 1, 1, 1, dk, dv)
    s0 = np.random.default_rng(22).standard_normal((1, 1, dk, dv))
    c = 1.3
    got = orc.ref_bwd(q, k, x, y, v, do, s0=s0, scale=c, ingate=mode)
    q1, k1, x1, y1, v1, d1 = (a[0, 0, 0].astype(np.float64) for a in (q, k, x, y, v, do))
    S0 = s0[0, 0]
    g = np.logaddexp(0, x1)
    tau = 1 / (1 + np.exp(-y1))
    alpha = np.exp(-g * tau)
    u = g if mode == orc.POW_G else 1 - np.exp(-g)
    du = np.ones_like(g) if mode == orc.POW_G else np.exp(-g)
    ahat = u ** tau
    S1 = alpha[:, None] * S0 + (ahat * k1)[:, None] * v1[None, :]
    sd = S0 @ d1            # sum_j S0[d,j] do[j]
    vd = float(v1 @ d1)
    assert _rel(got["dq"][0, 0, 0], c * (S1 @ d1)) < 1e-13
    assert _rel(got["dk"][0, 0, 0], c * q1 * ahat * vd) < 1e-13
    assert _rel(got["dv"][0, 0, 0], c * float(np.sum(q1 * ahat * k1)) * d1) < 1e-13
    assert _rel(got["ds0"][0, 0], c * (q1 * alpha)[:, None] * d1[None, :]) < 1e-13
    dalpha = c * q1 * sd
    dahat = c * q1 * k1 * vd
    dg = -tau * alpha * dalpha + tau * u ** (tau - 1) * du * dahat
    dtau = -g * alpha * dalpha + ahat * np.log(u) * dahat
    assert _rel(got["dx"][0, 0, 0], dg / (1 + np.exp(-x1))) < 1e-12
    assert _rel(got["dy"][0, 0, 0], dtau * tau * (1 - tau)) < 1e-12


def test_linear_in_the_incoming_gradients():
    B, H, T, dk, dv = 1, 1, 33, 4, 4
    q, k, x, y, v, do1 = _draw(31, B, H, T, dk, dv)
    rng = np.random.default_rng(32)
    do2 = _grid(rng.standard_normal(do1.shape))
    ds1, ds2 = rng.standard_normal((2, B, H, dk, dv))
    s0 = rng.standard_normal((B, H, dk, dv))
    a = orc.ref_bwd(q, k, x, y, v, do1, s0=s0, dsT=ds1)
    b = orc.ref_bwd(q, k, x, y, v, do2, s0=s0, dsT=ds2)
    c = orc.ref_bwd(q, k, x, y, v, _grid(do1 + 2 * do2), s0=s0, dsT=ds1 + 2 * ds2)
    for name in NAMES + ("ds0",):
        assert _rel(c[name], a[name] + 2 * b[name]) < 1e-12, name


@pytest.mark.parametrize("mode", MODES)
def test_two_half_calls_chain_through_the_state_gradient(mode):
    B, H, T, dk, dv = 1, 2, 64, 4, 3
    q, k, x, y, v, do = _draw(41, B, H, T, dk, dv)
    rng = np.random.default_rng(42)
    s0 = rng.standard_normal((B, H, dk, dv))
    dsT = rng.standard_normal((B, H, dk, dv))
    kw = dict(scale=0.5, ingate=mode)
    whole = orc.ref_bwd(q, k, x, y, v, do, s0=s0, dsT=dsT, **kw)
    h = 29
    first = tuple(a[:, :, :h] for a in (q, k, x, y, v))
    second = tuple(a[:, :, h:] for a in (q, k, x, y, v))
    _, s_mid = orc.ref_fwd(*first, s0=s0, **kw)
    g2 = orc.ref_bwd(*second, do[:, :, h:], s0=s_mid, dsT=dsT, **kw)
    g1 = orc.ref_bwd(*first, do[:, :, :h], s0=s0, dsT=g2["ds0"], **kw)
    for name in NAMES:
        assert _rel(np.concatenate([g1[name], g2[name]], axis=2), whole[name]) < 1e-12, name
    assert _rel(g1["ds0"], whole["ds0"]) < 1e-12


def test_packed_sequences_equal_one_by_one():
    H, dk, dv = 2, 4, 3
    lens = [5, 0, 37, 1]
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    T = int(cu[-1])
    q, k, x, y, v, do = _draw(51, 1, H, T, dk, dv)
    rng = np.random.default_rng(52)
    s0 = rng.standard_normal((len(lens), H, dk, dv))
    dsT = rng.standard_normal((len(lens), H, dk, dv))
    packed = orc.ref_bwd(q, k, x, y, v, do, s0=s0, dsT=dsT, cu_seqlens=cu)
    for n, L in enumerate(lens):
        sl = slice(int(cu[n]), int(cu[n + 1]))
        one = orc.ref_bwd(*(a[:, :, sl] for a in (q, k, x, y, v, do)), s0=s0[n:n + 1], dsT=dsT[n:n + 1])
        for name in NAMES:
            assert np.array_equal(packed[name][:, :, sl], one[name]), name
        assert np.array_equal(packed["ds0"][n], one["ds0"][0])
        if L == 0:      # nothing happens to the state: its gradient passes through
            assert np.array_equal(packed["ds0"][n], dsT[n])
