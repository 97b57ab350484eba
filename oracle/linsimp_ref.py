"""fp64 CPU oracle for linearized 2-simplicial attention (LinSimp).

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain statement of what the
CUDA library must compute.  Only tests, the smoke check and the timed CPU
baseline of the benchmark may import it; the product path never does, and this
module imports nothing from the product.

Everything is numpy float64 and follows the paper's recurrent definition in the
paper's order (no chunking, no stabiliser shift, no fusion):

  * feature map           phi(x) = exp(Omega x - |x|^2/2) / sqrt(m)       (Eq. prf)
  * prefix states         M_i = M_{i-1} + phi(k_i) v_i^T,  a_i = a_{i-1} + phi(k_i)
                                                              (Eqs. Mstate, astate)
  * anchor window         C_i = {max(0, i-W+1), ..., i}  (0-based)   (Sec. 3.3)
  * estimator             N_i = sum_c [phi(q_i*r_c)^T M_i] * u_c           (Eq. Ni)
                          Z_i = sum_c  phi(q_i*r_c)^T a_i                  (Eq. Zi)
                          o_i = N_i / (Z_i + eps), eps = 1e-30 (Eq. linearized-output)

Inputs are used exactly as given: L2-normalisation of q, k, r and the
temperature of Sec. 3.1 are the caller's business, as is the output gate.

Layout: one head at a time, arrays [T, d]; `omega` is [d, m] (column p is the
paper's feature row omega_p).  Batched wrappers loop over leading axes.

Pins (see tests/test_oracle_*.py): brute-force double loop over (j, c)
(`brute_ref`, Eq. swap-sum and App. A), Lemma 1 mean and variance law,
convergence to the exact windowed joint softmax (Eq. exact-window-app), the
W=1/u=1 reduction to causal random-feature linear attention, the Omega=0 closed
form, causality / convex-hull / bilinearity invariants, and for the gradients
central finite differences, torch fp64 autograd through the brute-force form
and the Euler identities <dv,v> = <du,u> = <dO,o>.  Every function here has
at least one such pin.
"""
import numpy as np

EPS = 1e-30


def log_features(x, omega):
    """l(x) = Omega x - |x|^2/2 for rows of x [n, d]; returns [n, m] (Sec. B.2)."""
    x = np.asarray(x, dtype=np.float64)
    return x @ omega - 0.5 * np.sum(x * x, axis=-1, keepdims=True)


def phi(x, omega):
    """Positive random feature map of Eq. prf, rows of x [n, d] -> [n, m]."""
    m = omega.shape[1]
    return np.exp(log_features(x, omega)) / np.sqrt(m)


def prefix_state(k, v, omega, M0=None, a0=None):
    """M = sum_j phi(k_j) v_j^T, a = sum_j phi(k_j) over all rows (Eqs. Mstate/astate)."""
    m, d = omega.shape[1], v.shape[1]
    M = np.zeros((m, d)) if M0 is None else np.array(M0, dtype=np.float64)
    a = np.zeros(m) if a0 is None else np.array(a0, dtype=np.float64)
    chi = phi(k, omega)
    for j in range(k.shape[0]):
        M += np.outer(chi[j], v[j])
        a += chi[j]
    return M, a


def fwd_ref(q, k, v, r, u, omega, W, eps=EPS, M0=None, a0=None, t0=0, return_parts=False):
    """Forward for one head.

    q, k, r: [T, d]; v, u: [T, dv]; omega: [d, m].  Rows < t0 are history: their
    keys/values are assumed to be inside (M0, a0) already and they act only as
    anchors (r, u).  Returns o [T, dv] (rows < t0 are zero); with return_parts
    also N [T, dv] and Z [T].
    """
    q, k, v, r, u = (np.asarray(t, dtype=np.float64) for t in (q, k, v, r, u))
    omega = np.asarray(omega, dtype=np.float64)
    T, m, dv = q.shape[0], omega.shape[1], v.shape[1]
    M = np.zeros((m, dv)) if M0 is None else np.array(M0, dtype=np.float64)
    a = np.zeros(m) if a0 is None else np.array(a0, dtype=np.float64)
    chi = phi(k, omega)
    o = np.zeros((T, dv))
    Ns = np.zeros((T, dv))
    Zs = np.zeros(T)
    for i in range(t0, T):
        # the state holds every j <= i before query i reads it
        M += np.outer(chi[i], v[i])
        a += chi[i]
        c0 = max(0, i - W + 1)
        x = q[i][None, :] * r[c0:i + 1]            # composite queries z_ic, [w, d]
        psi = phi(x, omega)                        # [w, m]
        g = psi @ M                                # [w, dv]
        N = np.sum(g * u[c0:i + 1], axis=0)        # Eq. Ni
        Z = np.sum(psi @ a)                        # Eq. Zi
        o[i] = N / (Z + eps)                       # Eq. linearized-output
        Ns[i], Zs[i] = N, Z
    if return_parts:
        return o, Ns, Zs
    return o


def brute_ref(q, k, v, r, u, omega, W, eps=EPS):
    """Explicit double loop over (j, c) of the approximate pair weights (App. A).

    N_i = sum_c sum_{j<=i} [phi(z_ic)^T phi(k_j)] (v_j * u_c), Z_i with value 1.
    O(T^2 W m): tiny T only.  Shares only `phi` with fwd_ref.
    """
    q, k, v, r, u = (np.asarray(t, dtype=np.float64) for t in (q, k, v, r, u))
    T, dv = q.shape[0], v.shape[1]
    o = np.zeros((T, dv))
    for i in range(T):
        N = np.zeros(dv)
        Z = 0.0
        for c in range(max(0, i - W + 1), i + 1):
            f_ic = phi((q[i] * r[c])[None, :], omega)[0]
            for j in range(i + 1):
                f_j = phi(k[j][None, :], omega)[0]
                kappa = float(np.dot(f_ic, f_j))
                N += kappa * (v[j] * u[c])
                Z += kappa
        o[i] = N / (Z + eps)
    return o


def exact_window_ref(q, k, v, r, u, W):
    """Exact windowed joint softmax of Eq. exact-window-app (no random features)."""
    q, k, v, r, u = (np.asarray(t, dtype=np.float64) for t in (q, k, v, r, u))
    T, dv = q.shape[0], v.shape[1]
    o = np.zeros((T, dv))
    for i in range(T):
        N = np.zeros(dv)
        Z = 0.0
        for c in range(max(0, i - W + 1), i + 1):
            for j in range(i + 1):
                kappa = np.exp(np.sum(q[i] * k[j] * r[c]))   # Eq. trilinear-score
                N += kappa * (v[j] * u[c])
                Z += kappa
        o[i] = N / Z
    return o


def exact_two_window_ref(q, k, v, r, u, w1, w2, return_lse=False):
    """Exact joint softmax over the pair plane j in [i-w1+1, i] x c in [i-w2+1, i] (the windowed exact layer the paper
    compares with, Sec. 4.3 "Baselines": Eq. exact-window-app with a window on the key stream too), with the
    trilinear score of Eq. trilinear-score on the inputs as given."""
    q, k, v, r, u = (np.asarray(t, dtype=np.float64) for t in (q, k, v, r, u))
    T, dv = q.shape[0], v.shape[1]
    o = np.zeros((T, dv))
    lse = np.zeros(T)
    for i in range(T):
        j0, c0 = max(0, i - w1 + 1), max(0, i - w2 + 1)
        s = ((q[i][None, :] * r[c0:i + 1]) @ k[j0:i + 1].T)          # [anchors, keys]
        mx = s.max()
        kappa = np.exp(s - mx)
        Z = kappa.sum()
        G = kappa @ v[j0:i + 1]                                       # [anchors, dv]
        o[i] = np.sum(G * u[c0:i + 1], axis=0) / Z
        lse[i] = mx + np.log(Z)
    return (o, lse) if return_lse else o


def bwd_ref(q, k, v, r, u, omega, W, dO, eps=EPS, M0=None, a0=None, t0=0, upstream=None):
    """Analytic gradients of sum(dO * o) for one head (no gradient for omega).

    With upstream = (dN [T, dv], dZ [T]) the gradients of a loss are returned whose
    derivatives with respect to this call's own sums N_i, Z_i (Eqs. Ni, Zi) are given
    directly (dO is then not used): what a combination of several estimators needs.

    Sweep 1 walks queries forward with the running state and yields dq, dr, du;
    sweep 2 walks backward accumulating D_j = sum_{i>=j} dM_i, e_j = sum_{i>=j} da_i
    and yields dk, dv.  d l / d z = omega - z (App. C, backward query sweep).
    Rows < t0 are history (see fwd_ref): their dq, dk, dv are zero and their
    dr, du hold only the contributions of queries >= t0.
    Returns dq, dk, dv, dr, du.
    """
    q, k, v, r, u, dO = (np.asarray(t, dtype=np.float64) for t in (q, k, v, r, u, dO))
    omega = np.asarray(omega, dtype=np.float64)
    T, m, dv_ = q.shape[0], omega.shape[1], v.shape[1]
    M = np.zeros((m, dv_)) if M0 is None else np.array(M0, dtype=np.float64)
    a = np.zeros(m) if a0 is None else np.array(a0, dtype=np.float64)
    chi = phi(k, omega)
    dq, dk, dr = np.zeros_like(q), np.zeros_like(k), np.zeros_like(r)
    dv, du = np.zeros_like(v), np.zeros_like(u)
    dN = np.zeros((T, dv_))
    dZ = np.zeros(T)
    # sweep 1: forward over queries
    for i in range(t0, T):
        M += np.outer(chi[i], v[i])
        a += chi[i]
        c0 = max(0, i - W + 1)
        x = q[i][None, :] * r[c0:i + 1]
        psi = phi(x, omega)
        g = psi @ M
        N = np.sum(g * u[c0:i + 1], axis=0)
        Z = np.sum(psi @ a)
        o_i = N / (Z + eps)
        if upstream is None:
            dN[i] = dO[i] / (Z + eps)
            dZ[i] = -np.dot(dO[i], o_i) / (Z + eps)
        else:
            dN[i], dZ[i] = upstream[0][i], upstream[1][i]
        du[c0:i + 1] += dN[i][None, :] * g
        dg = dN[i][None, :] * u[c0:i + 1]                  # [w, dv]
        dpsi = dg @ M.T + dZ[i] * a[None, :]               # [w, m]
        dl = dpsi * psi                                    # d/d log-feature
        dx = dl @ omega.T - np.sum(dl, axis=1, keepdims=True) * x
        dq[i] = np.sum(dx * r[c0:i + 1], axis=0)
        dr[c0:i + 1] += dx * q[i][None, :]
    # sweep 2: backward over keys/values
    D = np.zeros((m, dv_))
    e = np.zeros(m)
    for i in range(T - 1, t0 - 1, -1):
        c0 = max(0, i - W + 1)
        x = q[i][None, :] * r[c0:i + 1]
        psi = phi(x, omega)
        dg = dN[i][None, :] * u[c0:i + 1]
        D += psi.T @ dg                                    # dM_i
        e += dZ[i] * np.sum(psi, axis=0)                   # da_i
        dchi = D @ v[i] + e
        dv[i] = D.T @ chi[i]
        dlk = dchi * chi[i]
        dk[i] = omega @ dlk - np.sum(dlk) * k[i]
    return dq, dk, dv, dr, du


def two_views_ref(q, k, v, r, u, omega, W, eps=EPS, return_parts=False):
    """Both orientations of the trilinear score (Eq. two-views) kernelised and averaged (App. E, first item), in the
    windowed form of this operator: the first view is fwd_ref as it stands (composite query q*r_c over the window,
    keys k_j global); the second exchanges the two key streams and their values (composite query q*k_j over the
    window, keys r_c global).  The kernel estimates are averaged, i.e. numerators and normalisers are added before the
    division: o_i = (N1_i + N2_i) / (Z1_i + Z2_i + 2 eps).  Needs v and u of the same width."""
    _, N1, Z1 = fwd_ref(q, k, v, r, u, omega, W, eps, return_parts=True)
    _, N2, Z2 = fwd_ref(q, r, u, k, v, omega, W, eps, return_parts=True)
    o = (N1 + N2) / (Z1 + Z2 + 2.0 * eps)[:, None]
    if return_parts:
        return o, N1 + N2, Z1 + Z2
    return o


def two_views_bwd_ref(q, k, v, r, u, omega, W, dO, eps=EPS):
    """Gradients of sum(dO * o) for two_views_ref: both views see the same derivatives with respect to their sums,
    dN_i = dO_i / den_i and dZ_i = -(dO_i . o_i) / den_i with den_i = Z1_i + Z2_i + 2 eps; the second view's
    gradients come back with the streams exchanged.  Returns dq, dk, dv, dr, du."""
    dO = np.asarray(dO, dtype=np.float64)
    o, N, Z = two_views_ref(q, k, v, r, u, omega, W, eps, return_parts=True)
    den = Z + 2.0 * eps
    up = (dO / den[:, None], -np.sum(dO * o, axis=1) / den)
    dq1, dk1, dv1, dr1, du1 = bwd_ref(q, k, v, r, u, omega, W, dO, eps, upstream=up)
    dq2, dr2, du2, dk2, dv2 = bwd_ref(q, r, u, k, v, omega, W, dO, eps, upstream=up)
    return dq1 + dq2, dk1 + dk2, dv1 + dv2, dr1 + dr2, du1 + du2


def decode_ref(q_t, k_t, v_t, r_t, u_t, omega, M, a, ring_r, ring_u, pos, W, eps=EPS):
    """One autoregressive step for one head (Theorem 1: state M, a + rolling (r,u)).

    M [m, dv], a [m] hold phi-weighted sums of the `pos` tokens seen so far
    (with the 1/sqrt(m) factor of Eq. prf); ring_r [W, d], ring_u [W, dv] hold the
    anchors of tokens pos-1, pos-2, ... at slots (pos-1) % W, ...  The state is
    updated first, token `pos` is written to slot pos % W, then the query reads
    min(pos+1, W) anchors.  Returns o_t, M, a, ring_r, ring_u (new copies).
    """
    omega = np.asarray(omega, dtype=np.float64)
    M = np.array(M, dtype=np.float64)
    a = np.array(a, dtype=np.float64)
    ring_r = np.array(ring_r, dtype=np.float64)
    ring_u = np.array(ring_u, dtype=np.float64)
    chi = phi(np.asarray(k_t, dtype=np.float64)[None, :], omega)[0]
    M += np.outer(chi, v_t)
    a += chi
    ring_r[pos % W] = r_t
    ring_u[pos % W] = u_t
    n = min(pos + 1, W)
    slots = [(pos - s) % W for s in range(n)]
    x = np.asarray(q_t, dtype=np.float64)[None, :] * ring_r[slots]
    psi = phi(x, omega)
    N = np.sum((psi @ M) * ring_u[slots], axis=0)
    Z = np.sum(psi @ a)
    return N / (Z + eps), M, a, ring_r, ring_u


def fwd_batched(q, k, v, r, u, omega, W, eps=EPS):
    """fwd_ref over leading [B, H] axes; omega [d, m] shared or [H, d, m] per head."""
    B, H = q.shape[:2]
    o = np.zeros(v.shape, dtype=np.float64)
    for b in range(B):
        for h in range(H):
            om = omega[h] if omega.ndim == 3 else omega
            o[b, h] = fwd_ref(q[b, h], k[b, h], v[b, h], r[b, h], u[b, h], om, W, eps)
    return o


def bwd_batched(q, k, v, r, u, omega, W, dO, eps=EPS):
    """bwd_ref over leading [B, H] axes; returns dq, dk, dv, dr, du."""
    B, H = q.shape[:2]
    outs = [np.zeros(t.shape, dtype=np.float64) for t in (q, k, v, r, u)]
    for b in range(B):
        for h in range(H):
            om = omega[h] if omega.ndim == 3 else omega
            g = bwd_ref(q[b, h], k[b, h], v[b, h], r[b, h], u[b, h], om, W, dO[b, h], eps)
            for dst, src in zip(outs, g):
                dst[b, h] = src
    return tuple(outs)
