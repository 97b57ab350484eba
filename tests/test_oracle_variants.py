"""Pins of the oracle's variant estimators (CPU only): both orientations of the trilinear score averaged
(Eq. two-views, App. E first item), value streams of a width other than the key width (Sec. 3.1), and the exact
windowed estimator with separate windows for the two key streams."""
import numpy as np

from oracle import linsimp_ref as R


def _rand(T, d, dv, m, seed, scale=0.7):
    rng = np.random.default_rng(seed)
    q, k, r = (rng.standard_normal((T, d)) * scale for _ in range(3))
    v, u, dO = (rng.standard_normal((T, dv)) * scale for _ in range(3))
    om = rng.standard_normal((d, m))
    return q, k, v, r, u, dO, om


def _pair_loops_two_views(q, k, v, r, u, om, W, eps):
    """Both kernelised views as explicit pair loops: view 1 sums phi(q*r_c).phi(k_j) over c in the window and j <= i,
    view 2 phi(q*k_j).phi(r_c) over j in the window and c <= i; numerators and normalisers are added."""
    T, dv = q.shape[0], v.shape[1]
    o = np.zeros((T, dv))
    for i in range(T):
        N, Z = np.zeros(dv), 0.0
        lo = max(0, i - W + 1)
        for c in range(lo, i + 1):
            for j in range(i + 1):
                w = float(R.phi((q[i] * r[c])[None], om)[0] @ R.phi(k[j][None], om)[0])
                N += w * v[j] * u[c]
                Z += w
        for j in range(lo, i + 1):
            for c in range(i + 1):
                w = float(R.phi((q[i] * k[j])[None], om)[0] @ R.phi(r[c][None], om)[0])
                N += w * v[j] * u[c]
                Z += w
        o[i] = N / (Z + 2 * eps)
    return o


def test_two_views_matches_explicit_pair_loops():
    q, k, v, r, u, dO, om = _rand(14, 4, 4, 6, 3)
    got = R.two_views_ref(q, k, v, r, u, om, 5)
    want = _pair_loops_two_views(q, k, v, r, u, om, 5, R.EPS)
    assert np.abs(got - want).max() < 1e-12 * np.abs(want).max()


def test_two_views_symmetry_and_single_view_special_case():
    q, k, v, r, u, dO, om = _rand(20, 5, 5, 8, 4)
    a = R.two_views_ref(q, k, v, r, u, om, 6)
    b = R.two_views_ref(q, r, u, k, v, om, 6)                   # exchanging the two key streams changes nothing
    assert np.abs(a - b).max() < 1e-13
    # when the two key streams and their values coincide, both views are the same estimator
    c = R.two_views_ref(q, k, v, k, v, om, 6)
    d_ = R.fwd_ref(q, k, v, k, v, om, 6)
    assert np.abs(c - d_).max() < 1e-12 * np.abs(d_).max()
    # full windows and a dense feature bank: both views estimate the same exact kernel sum, so they agree with each
    # other (and with the exact joint softmax) up to the estimator's own error
    q2, k2, v2, r2, u2, _, _ = _rand(6, 3, 3, 4, 5, scale=0.4)
    om2 = np.random.default_rng(6).standard_normal((3, 20000))
    two = R.two_views_ref(q2, k2, v2, r2, u2, om2, 6)
    exact = R.exact_window_ref(q2, k2, v2, r2, u2, 6)
    assert np.abs(two - exact).max() < 3e-2 * np.abs(exact).max()


def test_two_views_gradients_finite_differences():
    T, d, m, W = 10, 4, 6, 3
    q, k, v, r, u, dO, om = _rand(T, d, d, m, 7)
    g = R.two_views_bwd_ref(q, k, v, r, u, om, W, dO)
    args = [q, k, v, r, u]
    h = 1e-6
    for idx in range(5):
        num = np.zeros((T, d))
        for t in range(T):
            for a_ in range(d):
                ap = [x.copy() for x in args]
                am = [x.copy() for x in args]
                ap[idx][t, a_] += h
                am[idx][t, a_] -= h
                num[t, a_] = (np.sum(R.two_views_ref(*ap, om, W) * dO) - np.sum(R.two_views_ref(*am, om, W) * dO)) / (2 * h)
        assert np.abs(num - g[idx]).max() < 2e-8 * max(1.0, np.abs(g[idx]).max()), idx


def test_upstream_form_of_the_backward_reproduces_the_plain_one():
    # bwd_ref with the derivatives of its own sums passed in equals bwd_ref from dO
    q, k, v, r, u, dO, om = _rand(12, 4, 4, 6, 8)
    _, N, Z = R.fwd_ref(q, k, v, r, u, om, 4, return_parts=True)
    o = N / (Z + R.EPS)[:, None]
    up = (dO / (Z + R.EPS)[:, None], -np.sum(dO * o, axis=1) / (Z + R.EPS))
    a = R.bwd_ref(q, k, v, r, u, om, 4, dO)
    b = R.bwd_ref(q, k, v, r, u, om, 4, dO, upstream=up)
    for x, y in zip(a, b):
        assert np.abs(x - y).max() < 1e-13 * max(1.0, np.abs(x).max())


def test_value_width_other_than_key_width():
    """v, u in R^{D_v} with D_v != D (Sec. 3.1): every value channel is an estimator of its own sharing Z_i, so the
    output equals the channel blocks computed separately, and the gradients of q, k, r add up over the blocks."""
    T, d, dv, m, W = 12, 4, 7, 6, 3
    q, k, v, r, u, dO, om = _rand(T, d, dv, m, 9)
    o = R.fwd_ref(q, k, v, r, u, om, W)
    assert o.shape == (T, dv)
    parts = [R.fwd_ref(q, k, v[:, a:b], r, u[:, a:b], om, W) for a, b in ((0, 4), (4, 7))]
    assert np.abs(np.concatenate(parts, axis=1) - o).max() < 1e-13 * np.abs(o).max()
    g = R.bwd_ref(q, k, v, r, u, om, W, dO)
    gs = [R.bwd_ref(q, k, v[:, a:b], r, u[:, a:b], om, W, dO[:, a:b]) for a, b in ((0, 4), (4, 7))]
    for idx in (0, 1, 3):                                        # dq, dk, dr: sums over the channel blocks
        assert np.abs(gs[0][idx] + gs[1][idx] - g[idx]).max() < 1e-12 * max(1.0, np.abs(g[idx]).max())
    for idx in (2, 4):                                           # dv, du: the blocks side by side
        assert np.abs(np.concatenate([gs[0][idx], gs[1][idx]], axis=1) - g[idx]).max() < 1e-12 * max(1.0, np.abs(g[idx]).max())
    # and by finite differences on a value channel beyond the key width
    h = 1e-6
    vp, vm = v.copy(), v.copy()
    vp[5, 6] += h
    vm[5, 6] -= h
    num = (np.sum(R.fwd_ref(q, k, vp, r, u, om, W) * dO) - np.sum(R.fwd_ref(q, k, vm, r, u, om, W) * dO)) / (2 * h)
    assert abs(num - g[2][5, 6]) < 1e-7 * max(1.0, abs(num))


def test_exact_two_window_estimator():
    """The exact layer with windows on both key streams: equals the pair-loop form of Eq. exact-window-app when the
    key window covers the prefix; with one anchor and u = 1 it is sliding-window softmax attention with the query
    q_i * r_i (a library routine); its weights are a joint distribution over the pair plane."""
    import torch
    rng = np.random.default_rng(11)
    T, d = 14, 5
    q, k, v, r, u = (rng.standard_normal((T, d)) * 0.6 for _ in range(5))
    a = R.exact_two_window_ref(q, k, v, r, u, T, 4)
    b = R.exact_window_ref(q, k, v, r, u, 4)
    assert np.abs(a - b).max() < 1e-12
    # w2 = 1, u = 1: banded causal softmax attention
    w1 = 6
    got = R.exact_two_window_ref(q, k, v, r, np.ones_like(u), w1, 1)
    mask = torch.tensor([[0.0 if (j <= i and j > i - w1) else -np.inf for j in range(T)] for i in range(T)], dtype=torch.float64)
    want = torch.nn.functional.scaled_dot_product_attention(torch.tensor(q * r)[None], torch.tensor(k)[None], torch.tensor(v)[None],
                                                            attn_mask=mask[None], scale=1.0)[0].numpy()
    assert np.abs(got - want).max() < 1e-12
    # shifting every score of a query by a constant changes nothing but lse (joint normalisation): scale k so that
    # s -> s + const is not available, so check instead that the output is a convex combination of v_j * u_c
    o, lse = R.exact_two_window_ref(q, k, v, r, u, 5, 3, return_lse=True)
    for i in (0, 3, 13):
        ys = np.array([v[j] * u[c] for j in range(max(0, i - 4), i + 1) for c in range(max(0, i - 2), i + 1)])
        assert np.all(o[i] <= ys.max(axis=0) + 1e-12) and np.all(o[i] >= ys.min(axis=0) - 1e-12)
    # and the normaliser by brute force
    i = 9
    Z = sum(np.exp(np.sum(q[i] * k[j] * r[c])) for j in range(i - 4, i + 1) for c in range(i - 2, i + 1))
    assert abs(lse[i] - np.log(Z)) < 1e-12
