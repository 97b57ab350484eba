"""Error surveys of the bf16-input / fp32-state path beyond the named configurations: a grid of seeds, lengths and
kernel instances, and a set of seeded random combinations (narrow windows, the zero-padded rank-32 instance, per-head
banks, two-token sequences at m = 256 whose attention is saturated).  Every case is compared with the oracle in the
library's metric, max|gpu - ref| / max|ref| per output tensor.

What the surveys establish: all six tensors stay within the 2e-2 of the named configurations everywhere but in one
regime.  dk has the least margin (its numerator and normaliser parts cancel; the backward therefore divides dZ_i by
the normaliser its own operands give, and what is left is mostly the bf16 rounding of the boundary state): worst
1.7e-2 on the grid.
The one regime held to 4e-2: dq, dk, dr of sequences of two or three tokens at feature ranks above 128.  There a query
sees a handful of pairs, the 128-feature blocks' parts of those gradients are each several times larger than their
sum, and what is left after they cancel carries the blocks' fp16/bf16-operand noise; from a few dozen tokens on the
same rank is back within 2e-2 (the T = 260, 1000 and 1500 cases below)."""
import numpy as np
import pytest
import torch

import paper_2608_09307_b200 as P
from paper_2608_09307_b200 import synth
from oracle import c_ref as C
from tests.util import rel_err, to64, units

pytestmark = pytest.mark.gpu

TOL = 2e-2            # the path's tolerance
TOL_FEW = 4e-2        # dq, dk, dr of two- and three-token sequences at feature ranks above 128
NAMES = ("o", "dq", "dk", "dv", "dr", "du")


def _errors(t, om, W, per_head=False, two_term_state=False):
    """Per-tensor metric over all units of one call, and the worst per-unit ratio of every tensor."""
    g = {k_: v_.cuda() for k_, v_ in t.items()}
    omg = om.cuda()
    o, L, lse = P.fwd(g["q"], g["k"], g["v"], g["r"], g["u"], omg, W=W)
    grads = P.bwd(g["q"], g["k"], g["v"], g["r"], g["u"], omg, o, L, lse, g["dO"], W=W, two_term_state=two_term_state)
    torch.cuda.synchronize()
    B, H = t["q"].shape[:2]
    got, ref = {n: [] for n in NAMES}, {n: [] for n in NAMES}
    for b in range(B):
        for h in range(H):
            cut = {name: to64(t[name][b, h:h + 1]) for name in ("q", "k", "v", "r", "u", "dO")}
            om64 = to64(om[h] if per_head else om)
            refs = (C.fwd(cut["q"], cut["k"], cut["v"], cut["r"], cut["u"], om64, W, 1e-30),) + \
                tuple(C.bwd(cut["q"], cut["k"], cut["v"], cut["r"], cut["u"], om64, W, cut["dO"]))
            for n, x, y in zip(NAMES, (o,) + tuple(grads), refs):
                got[n].append(to64(x[b, h]).ravel())
                ref[n].append(np.asarray(y).ravel())
    per_tensor = {n: rel_err(np.concatenate(got[n]), np.concatenate(ref[n]), floor=1e-2) for n in NAMES}
    per_unit = {n: max(rel_err(a, b_, floor=1e-2) for a, b_ in zip(got[n], ref[n])) for n in NAMES}
    return per_tensor, per_unit


def test_seed_grid():
    """48 cases: T in {40, 300, 1000} x four seeds x (d, m) in {(128,128), (64,128), (64,64), (64,32)}."""
    worst = {}
    for d, m in ((128, 128), (64, 128), (64, 64), (64, 32)):
        for T in (40, 300, 1000):
            for seed in range(4):
                t = synth.make_inputs(1, 2, T, d, seed=7000 + 100 * T + seed + d + m, dtype="bf16", scale="rms")
                om = synth.make_omega(d, m, seed + 2)
                e, _ = _errors(t, om, 64)
                for n in NAMES:
                    worst[(d, m, n)] = max(worst.get((d, m, n), 0.0), e[n])
                    assert e[n] <= TOL, (d, m, T, seed, n, e[n])
    for d, m in ((128, 128), (64, 128), (64, 64), (64, 32)):
        print("d=%d m=%d worst:" % (d, m), " ".join("%s %.1e" % (n, worst[(d, m, n)]) for n in NAMES))


# d, m, T, seed of the grid's recipe: the three cases of 120 further seeds (4..13) whose dk leaves 2e-2 with the
# one-term state (2.2e-2..2.3e-2), and one ordinary case per instance
BEYOND = [(128, 128, 300, 5), (64, 128, 1000, 9), (64, 32, 300, 13), (128, 128, 1000, 11), (64, 64, 40, 4), (64, 32, 40, 11)]


def test_two_term_state():
    """LINSIMP_FLAG_STATE_TWO_TERMS: the boundary state as two bf16 terms in the backward.  dk within 1.2e-2 where
    the one-term state gives up to 2.3e-2; the other tensors keep their bounds."""
    for d, m, T, seed in BEYOND:
        t = synth.make_inputs(1, 2, T, d, seed=7000 + 100 * T + seed + d + m, dtype="bf16", scale="rms")
        om = synth.make_omega(d, m, seed + 2)
        e1, _ = _errors(t, om, 64)
        e2, _ = _errors(t, om, 64, two_term_state=True)
        print((d, m, T, seed), "one term: dk %.1e | two terms:" % e1["dk"], " ".join("%s %.1e" % (n, e2[n]) for n in NAMES))
        assert e1["dk"] <= 2.5e-2
        assert e2["dk"] <= 1.2e-2, (d, m, T, seed, e2["dk"])
        for n in NAMES:
            assert e2[n] <= TOL, (d, m, T, seed, n, e2[n])


def test_two_term_state_other_paths():
    """The same bit through the forward's states left for the backward, the feature blocks and both orientations."""
    t = synth.make_inputs(2, 2, 333, 64, seed=8901, dtype="bf16", scale="rms")
    g = {k_: v_.cuda() for k_, v_ in t.items()}
    om = synth.make_omega(64, 128, 41).cuda()
    args = (g["q"], g["k"], g["v"], g["r"], g["u"], om)
    pb = P.binding.make_params(2, 2, 333, 64, 128, 64, P.BF16, flags=P.binding.FLAG_STATE_TWO_TERMS)
    ws = torch.empty(P.workspace_bytes(pb, P.OP_BWD), dtype=torch.uint8, device="cuda")
    o, L, lse = P.fwd(*args, workspace=ws, two_term_state=True)
    reused = P.bwd(*args, o, L, lse, g["dO"], workspace=ws, reuse_fwd_state=True, two_term_state=True)
    fresh = P.bwd(*args, o, L, lse, g["dO"], two_term_state=True)
    for a, b in zip(reused, fresh):
        assert torch.equal(a, b)
    q, k, v, r, u, dO = (units(t[n]) for n in ("q", "k", "v", "r", "u", "dO"))
    for m, two_views in ((256, False), (128, True)):
        om = synth.make_omega(64, m, 43)
        o, L, lse = P.fwd(*args[:5], om.cuda(), two_views=two_views)
        grads = P.bwd(*args[:5], om.cuda(), o, L, lse, g["dO"], two_views=two_views, two_term_state=True)
        if two_views:
            from oracle import linsimp_ref as R
            ref = [np.stack(x) for x in zip(*[R.two_views_bwd_ref(q[i], k[i], v[i], r[i], u[i], to64(om), 64, dO[i])
                                              for i in range(q.shape[0])])]
        else:
            ref = C.bwd(q, k, v, r, u, to64(om), 64, dO)
        for n, got, want in zip(NAMES[1:], grads, ref):
            e = rel_err(units(got), want, floor=1e-2)
            print(m, two_views, n, "%.1e" % e)
            assert e <= TOL, (m, two_views, n, e)


# B, H, T, d, m, W, per_head, seed
COMBOS = [
    (2, 2, 333, 64, 32, 7, False, 1), (1, 3, 1200, 64, 64, 7, True, 2), (3, 1, 90, 128, 128, 7, False, 3),
    (2, 2, 2, 64, 256, 64, False, 4), (1, 2, 2, 128, 256, 64, False, 5), (2, 3, 2, 64, 256, 33, True, 6),
    (1, 1, 2100, 128, 128, 64, False, 7), (2, 2, 1, 64, 64, 64, False, 8), (1, 2, 65, 128, 64, 64, True, 9),
    (3, 2, 129, 64, 128, 17, False, 10), (1, 3, 700, 64, 32, 33, True, 11), (2, 1, 48, 128, 32, 48, False, 12),
    (1, 2, 1500, 64, 256, 64, False, 13), (2, 2, 260, 128, 256, 16, True, 14), (1, 1, 31, 64, 384, 64, False, 15),
    (2, 3, 15, 128, 128, 1, False, 16), (1, 2, 16, 64, 64, 2, True, 17), (3, 3, 17, 64, 128, 3, False, 18),
    (1, 2, 900, 128, 64, 64, False, 19), (2, 1, 2049, 64, 64, 64, False, 20), (1, 3, 450, 128, 128, 25, True, 21),
    (2, 2, 77, 64, 32, 64, False, 22), (1, 1, 1000, 64, 512, 64, False, 23), (3, 1, 200, 128, 128, 64, True, 24),
]


@pytest.mark.parametrize("B,H,T,d,m,W,per_head,seed", COMBOS)
def test_random_combination(B, H, T, d, m, W, per_head, seed):
    t = synth.make_inputs(B, H, T, d, seed=8800 + seed, dtype="bf16", scale="rms")
    om = synth.make_omega(d, m, 40 + seed, heads=H if per_head else None)
    e, unit = _errors(t, om, W, per_head)
    print("per tensor:", " ".join("%s %.1e" % (n, e[n]) for n in NAMES), "| worst unit:",
          " ".join("%s %.1e" % (n, unit[n]) for n in NAMES))
    few = T <= 3 and m > 128
    for n in NAMES:
        tol = TOL_FEW if (few and n in ("dq", "dk", "dr")) else TOL
        assert e[n] <= tol, (n, e[n])
