"""fp64 CPU oracle for the two steps on either side of the LinSimp estimator.

TEST INFRASTRUCTURE ONLY: imported by tests, the smoke check and the timed CPU
baseline, never by the product; imports nothing from the product.

  * input side (Sec. 3.1, text before the trilinear score):
        q^ = tau * q / |q|_2,   k^ = k / |k|_2,   r^ = r / |r|_2
    with one learned temperature tau per head applied to the query only.
  * output side (Eq. gated-output):
        y_i = sigmoid(gamma) * RMSNorm(o~_i),
        RMSNorm(x) = x / sqrt(mean_e(x_e^2) + rms_eps)
    with one learned gate gamma per head.

Readings where the paper is silent: RMSNorm carries no learned weight here and
uses the model's epsilon 1e-6 (Sec. 4); a row of norm below `norm_floor`
(default 1e-12) is divided by `norm_floor` instead of its norm, so a zero row
maps to zero.

The gradient functions are the chain rule written out for these definitions;
they are pinned by central finite differences of the forward functions, the
forward functions by their defining properties (unit norm, unit mean square,
scale invariance, hand-computed rows).  Every function here has such a pin.
"""
import numpy as np

RMS_EPS = 1e-6
NORM_FLOOR = 1e-12


def l2_normalize(x, scale=1.0, norm_floor=NORM_FLOOR):
    """scale * x / max(|x|_2, norm_floor) for rows of x [..., d]."""
    x = np.asarray(x, dtype=np.float64)
    n = np.sqrt(np.sum(x * x, axis=-1, keepdims=True))
    return scale * x / np.maximum(n, norm_floor)


def l2_normalize_bwd(x, g, scale=1.0, norm_floor=NORM_FLOOR):
    """Gradients of sum(g * l2_normalize(x, scale)) w.r.t. x and w.r.t. scale.

    With e = x/|x|: d/dx = scale/|x| * (g - e (e.g));  d/dscale = sum(g.e).
    A row below the floor is a plain scaling by scale/norm_floor.
    """
    x = np.asarray(x, dtype=np.float64)
    g = np.asarray(g, dtype=np.float64)
    n = np.sqrt(np.sum(x * x, axis=-1, keepdims=True))
    floored = n < norm_floor
    nn = np.maximum(n, norm_floor)
    e = x / nn
    eg = np.sum(e * g, axis=-1, keepdims=True)
    dx = scale / nn * np.where(floored, g, g - e * eg)
    return dx, float(np.sum(eg))


def qkr_normalize(q, k, r, tau):
    """Input side of one head: (tau q/|q|, k/|k|, r/|r|), arrays [T, d]."""
    return l2_normalize(q, tau), l2_normalize(k), l2_normalize(r)


def qkr_normalize_bwd(q, k, r, tau, dqh, dkh, drh):
    """Returns dq, dk, dr and dtau for upstream gradients of the three normalised streams."""
    dq, dtau = l2_normalize_bwd(q, dqh, tau)
    dk, _ = l2_normalize_bwd(k, dkh)
    dr, _ = l2_normalize_bwd(r, drh)
    return dq, dk, dr, dtau


def sigmoid(x):
    return 1.0 / (1.0 + np.exp(-x))


def rmsnorm(x, rms_eps=RMS_EPS):
    x = np.asarray(x, dtype=np.float64)
    return x / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + rms_eps)


def gate_rmsnorm(o, gamma, rms_eps=RMS_EPS):
    """y = sigmoid(gamma) * RMSNorm(o) for rows of o [T, d] of one head (Eq. gated-output)."""
    return sigmoid(gamma) * rmsnorm(o, rms_eps)


def gate_rmsnorm_bwd(o, gamma, dy, rms_eps=RMS_EPS):
    """Gradients of sum(dy * gate_rmsnorm(o, gamma)) w.r.t. o and gamma.

    With s = (mean(o^2) + eps)^(-1/2), n = o s, g = sigmoid(gamma):
      do = g s (dy - n mean(dy n)),   dgamma = g (1 - g) sum(dy n).
    """
    o = np.asarray(o, dtype=np.float64)
    dy = np.asarray(dy, dtype=np.float64)
    s = 1.0 / np.sqrt(np.mean(o * o, axis=-1, keepdims=True) + rms_eps)
    n = o * s
    g = sigmoid(gamma)
    do = g * s * (dy - n * np.mean(dy * n, axis=-1, keepdims=True))
    dgamma = g * (1.0 - g) * float(np.sum(dy * n))
    return do, dgamma
