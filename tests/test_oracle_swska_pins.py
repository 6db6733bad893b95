"""Pins for the SW-SKA oracle: brute force, a library routine on the case that reduces to plain
causal attention, the head-compression identity of the paper, and what the window implies.  CPU only.
"""
import math

import numpy as np
import pytest

from oracle import swska_oracle as sw


def _draw(seed, B, H, T, d, dv=None):
    rng = np.random.default_rng(seed)
    dv = d if dv is None else dv
    f = lambda *s: rng.standard_normal(s).astype(np.float32)
    return f(B, H, T, d), f(B, T, d), f(B, H, T, dv)


def _rel(a, b):
    return np.max(np.abs(a - b)) / max(np.max(np.abs(b)), 1e-300)


@pytest.mark.parametrize("window", [1, 3, 7, 50])
def test_brute_force_loops(window):
    q, k, v = _draw(1, 2, 2, 11, 4, 3)
    o = sw.swska_ref(q, k, v, window, scale=0.6)
    for b in range(2):
        for h in range(2):
            for t in range(11):
                lo = max(0, t - window + 1)
                e = [math.exp(0.6 * float(np.dot(q[b, h, t].astype(np.float64), k[b, i].astype(np.float64))))
                     for i in range(lo, t + 1)]
                want = sum(w * v[b, h, lo + n].astype(np.float64) for n, w in enumerate(e)) / sum(e)
                assert np.max(np.abs(o[b, h, t] - want)) < 1e-12


def test_window_covering_everything_is_causal_attention_of_a_library():
    torch = pytest.importorskip("torch")
    q, k, v = _draw(2, 2, 3, 40, 8)
    o = sw.swska_ref(q, k, v, window=40, scale=8 ** -0.5)
    tq, tv = (torch.tensor(a.astype(np.float64)) for a in (q, v))
    tk = torch.tensor(k.astype(np.float64))[:, None].expand(-1, 3, -1, -1)
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True).numpy()
    assert _rel(o, ref) < 1e-12
    assert _rel(sw.swska_ref(q, k, v, window=1000, scale=8 ** -0.5), ref) < 1e-12


def test_shared_key_reproduces_multi_head_attention_with_transformed_queries():
    # Sec. "Shared-Key Attention": Q^h K^h^T = (X W_Q^h W_K^h^T W~^-T)(W~^T X^T), so attention with
    # per-head keys equals attention with the single key X W~ and queries X W_Q^h W_K^h^T W~^-T
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(3)
    T, dm, d, H = 24, 6, 6, 3
    X = rng.standard_normal((T, dm))
    WQ, WK = rng.standard_normal((H, dm, d)), rng.standard_normal((H, dm, d))
    WV = rng.standard_normal((H, dm, 5))
    Wt = rng.standard_normal((dm, d)) + 3 * np.eye(dm)                      # invertible
    k_shared = X @ Wt
    q_tilde = np.stack([X @ WQ[h] @ WK[h].T @ np.linalg.inv(Wt).T for h in range(H)])
    v = np.stack([X @ WV[h] for h in range(H)])
    got = sw.swska_ref(q_tilde[None], k_shared[None], v[None], window=T, scale=1.0)[0]
    for h in range(H):
        qh, kh = torch.tensor(X @ WQ[h])[None], torch.tensor(X @ WK[h])[None]
        ref = torch.nn.functional.scaled_dot_product_attention(qh, kh, torch.tensor(v[h])[None],
                                                               is_causal=True, scale=1.0)[0].numpy()
        assert _rel(got[h], ref) < 1e-9


def test_what_the_window_implies():
    q, k, v = _draw(4, 1, 2, 30, 5)
    W = 6
    o = sw.swska_ref(q, k, v, W, scale=0.5)
    # window 1: every token sees only itself
    assert _rel(sw.swska_ref(q, k, v, 1), v.astype(np.float64)) < 1e-15
    # zero queries: the plain mean of the window's values
    o0 = sw.swska_ref(np.zeros_like(q), k, v, W)
    for t in (0, 3, 17, 29):
        lo = max(0, t - W + 1)
        assert _rel(o0[0, 1, t], v[0, 1, lo:t + 1].astype(np.float64).mean(axis=0)) < 1e-14
    # a token outside (t - W, t] has no influence on o_t; one inside has
    k2, v2 = k.copy(), v.copy()
    k2[0, 10] += 5.0
    v2[0, :, 10] -= 3.0
    o2 = sw.swska_ref(q, k2, v2, W, scale=0.5)
    assert np.array_equal(o2[:, :, :10], o[:, :, :10]) and np.array_equal(o2[:, :, 10 + W:], o[:, :, 10 + W:])
    assert _rel(o2[:, :, 10:10 + W], o[:, :, 10:10 + W]) > 1e-3
    # rows of the softmax sum to one: constant values come back unchanged; adding a constant to
    # all scores of a row (q shifted along a direction all keys share) changes nothing
    vc = np.ones_like(v) * 2.5
    assert _rel(sw.swska_ref(q, k, vc, W, scale=0.5), vc.astype(np.float64)) < 1e-15
    k3 = k.copy()
    k3[..., 0] = 1.0
    q3 = q.copy()
    q3[..., 0] += 7.0
    assert _rel(sw.swska_ref(q3, k3, v, W, scale=0.5), sw.swska_ref(q, k3, v, W, scale=0.5)) < 1e-12
