"""Serving path: chunked prefill (a segment continuing a sequence) and the hand-off from prefill to decode."""
import numpy as np
import pytest
import torch

import paper_2608_09307_b200 as P
from paper_2608_09307_b200 import synth
from oracle import c_ref as C
from tests.util import rel_err, to64, units

pytestmark = pytest.mark.gpu


def _cuda(t):
    return {k: v.cuda() for k, v in t.items()}


@pytest.mark.parametrize("d,m,W,cuts", [(128, 128, 64, (137, 300)), (64, 128, 64, (16, 77, 200)), (64, 32, 33, (5, 90)),
                                        (128, 64, 64, (1, 2, 150)), (64, 64, 64, (2100, 5000))])   # last: segmented state walks
def test_chunked_prefill_equals_one_forward(d, m, W, cuts):
    B, H, T = 1, 2, cuts[-1]
    t = synth.make_inputs(B, H, T, d, seed=1500 + d + m, dtype="bf16", scale="rms", with_dO=False)
    t["omega"] = synth.make_omega(d, m)
    g = _cuda(t)
    q, k, v, r, u = (units(t[n]) for n in ("q", "k", "v", "r", "u"))
    om = to64(t["omega"])
    o_ref, Z_ref, M_ref, a_ref = C.fwd(q, k, v, r, u, om, W, 1e-30, return_state=True)
    # the whole sequence in one call, for reference
    o_full, L_full, lse_full, S_full, z_full = P.fwd(g["q"], g["k"], g["v"], g["r"], g["u"], g["omega"], W=W,
                                                      return_state=True)
    state, lo, outs, lses = None, 0, [], []
    for hi in cuts:
        seg = [g[n][:, :, lo:hi].contiguous() for n in ("q", "k", "v", "r", "u")]
        nh = min(W - 1, lo)
        hist = None if nh == 0 else (g["r"][:, :, lo - nh:lo].contiguous(), g["u"][:, :, lo - nh:lo].contiguous())
        o, L, lse, S, z = P.fwd_continue(*seg, g["omega"], state=state, history=hist, W=W)
        outs.append(o)
        lses.append(lse)
        state, lo = (S, z), hi
    o_cat = torch.cat(outs, dim=2)
    assert rel_err(units(o_cat), o_ref) <= 2e-2
    assert rel_err(units(o_cat), units(o_full)) <= 2e-2
    # the state after the last segment is the state of the whole sequence
    assert rel_err(to64(state[0]).reshape(B * H, m, d), M_ref * np.sqrt(m)) < 5e-5
    assert rel_err(to64(state[1]).reshape(B * H, m), a_ref * np.sqrt(m)) < 5e-5
    assert rel_err(to64(state[0]), to64(S_full)) < 1e-5
    lse_ref = np.log(m * (Z_ref + 1e-30))
    assert np.abs(to64(torch.cat(lses, dim=2)).reshape(B * H, T) - lse_ref).max() < 5e-2


@pytest.mark.parametrize("d,m,W,cuts", [(128, 128, 64, (137, 300)), (64, 128, 64, (16, 77, 200)), (64, 32, 33, (5, 90)),
                                        (128, 64, 64, (1, 2, 150)), (64, 64, 7, (40, 41, 130)), (128, 128, 64, (2100, 4300))])
def test_chunked_backward_equals_one_backward(d, m, W, cuts):
    """Chunked training: the forward runs segment by segment (linsimp_fwd_continue), the backward walks the segments
    last to first (linsimp_bwd_continue), handing the state gradient and the gradients of the W-1 history anchors
    from each segment to the one before.  The result must be the gradient of the whole sequence, which the oracle
    computes in one piece.  Cut points inside a window, segments of one token and segmented state walks included."""
    B, H, T = 1, 2, cuts[-1]
    t = synth.make_inputs(B, H, T, d, seed=1700 + d + m + W, dtype="bf16", scale="rms")
    t["omega"] = synth.make_omega(d, m)
    g = _cuda(t)
    q, k, v, r, u, dO = (units(t[n]) for n in ("q", "k", "v", "r", "u", "dO"))
    ref = C.bwd(q, k, v, r, u, to64(t["omega"]), W, dO)
    # forward chain: remember what every segment started from
    bounds, lo = [], 0
    for hi in cuts:
        bounds.append((lo, hi))
        lo = hi
    saved, state = [], None
    for lo, hi in bounds:
        seg = [g[n][:, :, lo:hi].contiguous() for n in ("q", "k", "v", "r", "u")]
        nh = min(W - 1, lo)
        hist = None if nh == 0 else (g["r"][:, :, lo - nh:lo].contiguous(), g["u"][:, :, lo - nh:lo].contiguous())
        o, L, lse, S, z = P.fwd_continue(*seg, g["omega"], state=state, history=hist, W=W)
        saved.append((seg, state, hist, L, lse))
        state = (S, z)
    # backward chain
    grads = [torch.zeros(B, H, T, d, device="cuda", dtype=torch.float32) for _ in range(5)]
    d_state = None
    for (lo, hi), (seg, st, hist, L, lse) in reversed(list(zip(bounds, saved))):
        dseg, dh, d_state = P.bwd_continue(*seg, g["omega"], L, lse, g["dO"][:, :, lo:hi].contiguous(), state=st,
                                           history=hist, d_state=d_state, W=W)
        for acc, part in zip(grads, dseg):
            acc[:, :, lo:hi] += part.float()
        if dh is not None:
            nh = dh[0].shape[2]
            grads[3][:, :, lo - nh:lo] += dh[0].float()
            grads[4][:, :, lo - nh:lo] += dh[1].float()
    torch.cuda.synchronize()
    # the state before the first token is empty: nothing may depend on what flows into it, but it must be finite
    assert torch.isfinite(d_state[0]).all() and torch.isfinite(d_state[1]).all()
    for name, got, want in zip(("dq", "dk", "dv", "dr", "du"), grads, ref):
        assert rel_err(units(got), want, floor=1e-2) <= 2e-2, name


def test_state_gradient_of_a_continued_segment():
    """dS_init, dz_init against the oracle: the gradient of sum(dO * o_segment) with respect to the state the segment
    starts from, by central differences of the oracle's forward along random directions of (M0, a0)."""
    B, H, T, d, m, W, T0 = 1, 2, 70, 64, 64, 64, 90
    t = synth.make_inputs(B, H, T0 + T, d, seed=1811, dtype="bf16", scale="rms")
    t["omega"] = synth.make_omega(d, m)
    g = _cuda(t)
    om = to64(t["omega"])
    q, k, v, r, u, dO = (units(t[n]) for n in ("q", "k", "v", "r", "u", "dO"))
    pre = [g[n][:, :, :T0].contiguous() for n in ("q", "k", "v", "r", "u")]
    _, _, _, S0, z0 = P.fwd(*pre, g["omega"], W=W, return_state=True)
    seg = [g[n][:, :, T0:].contiguous() for n in ("q", "k", "v", "r", "u")]
    hist = (g["r"][:, :, T0 - (W - 1):T0].contiguous(), g["u"][:, :, T0 - (W - 1):T0].contiguous())
    o, L, lse, S1, z1 = P.fwd_continue(*seg, g["omega"], state=(S0, z0), history=hist, W=W)
    _, _, (dS0, dz0) = P.bwd_continue(*seg, g["omega"], L, lse, g["dO"][:, :, T0:].contiguous(), state=(S0, z0),
                                      history=hist, W=W)
    torch.cuda.synchronize()
    # oracle: rows T0-(W-1) .. T0+T with the first W-1 as history, state (M0, a0) in its own convention (1/sqrt(m) inside)
    M0 = to64(S0).reshape(B * H, m, d) / np.sqrt(m)
    a0 = to64(z0).reshape(B * H, m) / np.sqrt(m)
    sl = slice(T0 - (W - 1), T0 + T)
    rng = np.random.default_rng(5)

    def loss(Mx, ax):
        oo = C.fwd(q[:, sl], k[:, sl], v[:, sl], r[:, sl], u[:, sl], om, W, 1e-30, M0=Mx, a0=ax, t0=W - 1)
        return float((oo[:, W - 1:] * dO[:, T0:]).sum())

    gS = to64(dS0).reshape(B * H, m, d) * np.sqrt(m)          # d/dM0 = sqrt(m) d/dS (S = sqrt(m) M)
    gz = to64(dz0).reshape(B * H, m) * np.sqrt(m)
    for _ in range(3):
        # directions relative to each entry (the features' magnitudes span many orders): stays in the linear regime
        dM = rng.standard_normal(M0.shape) * M0
        da = rng.standard_normal(a0.shape) * a0
        h = 1e-3
        num = (loss(M0 + h * dM, a0 + h * da) - loss(M0 - h * dM, a0 - h * da)) / (2 * h)
        ana = float((gS * dM).sum() + (gz * da).sum())
        # a directional derivative is a sum of terms of both signs: the error is measured against their total size
        scale = float(np.abs(gS * dM).sum() + np.abs(gz * da).sum())
        assert abs(num - ana) <= 2e-2 * scale, (num, ana, scale)


def test_prefill_then_decode_hand_off():
    # prefix by the forward, ring by linsimp_ring_fill, then single-token steps: the outputs must be the rows a
    # forward over the whole sequence gives
    B, H, d, m, W, T0, n_dec = 2, 2, 128, 128, 64, 150, 40
    T = T0 + n_dec
    t = synth.make_inputs(B, H, T, d, seed=1600, dtype="bf16", scale="rms", with_dO=False)
    t["omega"] = synth.make_omega(d, m)
    g = _cuda(t)
    q, k, v, r, u = (units(t[n]) for n in ("q", "k", "v", "r", "u"))
    o_ref = C.fwd(q, k, v, r, u, to64(t["omega"]), W, 1e-30)
    pre = [g[n][:, :, :T0].contiguous() for n in ("q", "k", "v", "r", "u")]
    o0, L0, lse0, S, z = P.fwd(*pre, g["omega"], W=W, return_state=True)
    rr = torch.zeros(B, H, W, d, device="cuda", dtype=torch.bfloat16)
    ru = torch.zeros_like(rr)
    P.ring_fill(pre[3], pre[4], rr, ru, t_first=0)
    # slot s holds the latest token with t % W == s
    for tok in range(T0 - W, T0):
        assert torch.equal(rr[:, :, tok % W], g["r"][:, :, tok]) and torch.equal(ru[:, :, tok % W], g["u"][:, :, tok])
    ws = P.decode_prepare(B, H, d, g["omega"], W=W)
    rows = []
    for s_ in range(T0, T):
        pos = torch.full((B,), s_, dtype=torch.int32, device="cuda")
        args = [g[n][:, :, s_].contiguous() for n in ("q", "k", "v", "r", "u")]
        rows.append(P.decode_step(*args, g["omega"], S, z, rr, ru, pos, W=W, workspace=ws, omega_image=True).clone())
    o_dec = torch.stack(rows, dim=2)
    assert rel_err(units(o_dec), o_ref[:, T0:]) <= 2e-2
    assert rel_err(units(o0), o_ref[:, :T0]) <= 2e-2


def test_ring_fill_short_prefix_and_offset():
    B, H, d, W = 1, 3, 64, 16
    for T, t_first in ((5, 0), (16, 7), (40, 100)):
        t = synth.make_inputs(B, H, T, d, seed=1700 + T, dtype="bf16", scale="rms", with_dO=False)
        r, u = t["r"].cuda(), t["u"].cuda()
        rr = torch.full((B, H, W, d), 7.0, device="cuda", dtype=torch.bfloat16)
        ru = torch.full_like(rr, 7.0)
        P.ring_fill(r, u, rr, ru, t_first=t_first)
        exp_r, exp_u = torch.full_like(rr, 7.0), torch.full_like(ru, 7.0)
        for tok in range(max(0, T - W), T):
            exp_r[:, :, (t_first + tok) % W] = r[:, :, tok]
            exp_u[:, :, (t_first + tok) % W] = u[:, :, tok]
        assert torch.equal(rr, exp_r) and torch.equal(ru, exp_u)


def test_fwd_continue_argument_checks():
    B, H, T, d, m, W = 1, 1, 20, 64, 256, 64            # rank 256 has no tensor-core forward
    t = _cuda(synth.make_inputs(B, H, T, d, seed=1, dtype="bf16", scale="rms", with_dO=False))
    om = synth.make_omega(d, m).cuda()
    with pytest.raises(P.LinSimpError):
        P.fwd_continue(t["q"], t["k"], t["v"], t["r"], t["u"], om, W=W)
    om = synth.make_omega(d, 64).cuda()
    too_long = (torch.zeros(B, H, W, d, device="cuda", dtype=torch.bfloat16),) * 2
    with pytest.raises(P.LinSimpError):
        P.fwd_continue(t["q"], t["k"], t["v"], t["r"], t["u"], om, history=too_long, W=W)


@pytest.mark.parametrize("d,m,W,T,lens", [(128, 128, 64, 150, [150, 37, 1]), (64, 64, 16, 100, [16, 0, 99]),
                                          (64, 128, 64, 80, [80, 65, 33])])
def test_padded_batch_matches_per_sequence_oracle(d, m, W, T, lens):
    """A batch padded to a common T: every sequence's valid rows, its final state, its decode ring and all gradients equal
    the oracle run on the sequence cut to its own length; gradients of padding rows are zero whatever dO holds there."""
    B, H = len(lens), 2
    t = synth.make_inputs(B, H, T, d, seed=2100 + d + T, dtype="bf16", scale="rms")
    om = synth.make_omega(d, m, 3)
    g = _cuda(t)
    omg = om.cuda()
    sl = torch.tensor(lens, dtype=torch.int32, device="cuda")
    p = P.binding.make_params(B, H, T, d, m, W, P.BF16)
    ws = torch.empty(P.workspace_bytes(p, P.OP_BWD), dtype=torch.uint8, device="cuda")
    o, L, lse, S, z = P.fwd_padded(g["q"], g["k"], g["v"], g["r"], g["u"], omg, sl, W=W, return_state=True, workspace=ws)
    grads = P.bwd_padded(g["q"], g["k"], g["v"], g["r"], g["u"], omg, sl, o, L, lse, g["dO"], W=W, workspace=ws,
                         reuse_fwd_state=True)
    grads2 = P.bwd_padded(g["q"], g["k"], g["v"], g["r"], g["u"], omg, sl, o, L, lse, g["dO"], W=W)
    ring_r, ring_u = P.ring_fill_padded(g["r"], g["u"], sl, W=W)
    torch.cuda.synchronize()
    assert torch.isfinite(o.float()).all()
    om64 = to64(om)
    for b, n in enumerate(lens):
        for got in grads + grads2:
            assert torch.all(got[b, :, n:] == 0)
        if n == 0:
            assert torch.all(S[b] == 0) and torch.all(z[b] == 0)
            assert torch.all(ring_r[b] == 0)
            continue
        cut = {name: to64(t[name][b, :, :n]) for name in ("q", "k", "v", "r", "u", "dO")}
        o_ref, _, M_ref, a_ref = C.fwd(cut["q"], cut["k"], cut["v"], cut["r"], cut["u"], om64, W, return_state=True)
        assert rel_err(to64(o[b, :, :n]), o_ref) <= 2e-2
        assert rel_err(to64(S[b]), M_ref * np.sqrt(m)) < 5e-5
        assert rel_err(to64(z[b]), a_ref * np.sqrt(m)) < 5e-5
        g_ref = C.bwd(cut["q"], cut["k"], cut["v"], cut["r"], cut["u"], om64, W, cut["dO"])
        for name, got, got2, ref in zip(("dq", "dk", "dv", "dr", "du"), grads, grads2, g_ref):
            e = rel_err(to64(got[b, :, :n]), ref, floor=1e-2)
            assert e <= 2e-2, (name, b, e)
            assert rel_err(to64(got2[b, :, :n]), ref, floor=1e-2) <= 2e-2, (name, b)
        last = torch.arange(max(0, n - W), n)
        assert torch.equal(ring_r[b][:, last % W].cpu(), t["r"][b][:, last])
        assert torch.equal(ring_u[b][:, last % W].cpu(), t["u"][b][:, last])


def test_padded_argument_checks():
    x = torch.zeros((2, 1, 32, 64), device="cuda", dtype=torch.bfloat16)
    om = torch.zeros((64, 64), device="cuda")
    with pytest.raises(P.LinSimpError):
        P.fwd_padded(x, x, x, x, x, om, torch.zeros(3, dtype=torch.int32, device="cuda"))
    x32 = x.float()
    with pytest.raises(P.LinSimpError, match="-2"):          # no padded variant on the fp32 kernels
        P.fwd_padded(x32, x32, x32, x32, x32, om, torch.zeros(2, dtype=torch.int32, device="cuda"))


@pytest.mark.parametrize("d,m,W,per_head,lens", [(128, 128, 64, False, [150, 37, 3]), (64, 128, 16, True, [40, 0, 16]),
                                                 (128, 64, 33, True, [5, 90, 64])])
def test_ragged_prefill_then_decode(d, m, W, per_head, lens):
    """A ragged batch through the whole serving chain: padded prefill (state per sequence), padded ring fill, then
    decode steps in which every sequence stands at its own position.  Each sequence's decoded rows equal the rows a
    forward over that sequence (prefix + decoded tokens) gives."""
    B, H, n_dec = len(lens), 2, 20
    T0 = max(lens)
    T = T0 + n_dec
    t = synth.make_inputs(B, H, T, d, seed=2300 + d + m + W, dtype="bf16", scale="rms", with_dO=False)
    om = synth.make_omega(d, m, 7, heads=H if per_head else None)
    g = _cuda(t)
    omg = om.cuda()
    sl = torch.tensor(lens, dtype=torch.int32, device="cuda")
    # sequence b = its first lens[b] rows, then the n_dec rows that follow them in the same tensors
    pre = [g[n][:, :, :T0].contiguous() for n in ("q", "k", "v", "r", "u")]
    o0, L0, lse0, S, z = P.fwd_padded(*pre, omg, sl, W=W, return_state=True)
    rr, ru = P.ring_fill_padded(pre[3], pre[4], sl, W=W)
    ws = P.decode_prepare(B, H, d, omg, W=W)
    rows = []
    idx_b = torch.arange(B, device="cuda")
    for s_ in range(n_dec):
        pos = sl + s_
        args = [g[n][idx_b, :, pos.long()].contiguous() for n in ("q", "k", "v", "r", "u")]
        rows.append(P.decode_step(*args, omg, S, z, rr, ru, pos, W=W, workspace=ws, omega_image=True).clone())
    torch.cuda.synchronize()
    o_dec = torch.stack(rows, dim=2)                       # [B, H, n_dec, d]
    for b, n in enumerate(lens):
        for h in range(H):
            cut = [to64(t[name][b, h:h + 1, :n + n_dec]) for name in ("q", "k", "v", "r", "u")]
            o_ref, _, M_ref, a_ref = C.fwd(*cut, to64(om[h] if per_head else om), W, 1e-30, return_state=True)
            assert rel_err(to64(o_dec[b, h:h + 1]), o_ref[:, n:]) <= 2e-2, (b, h)
            if n:
                assert rel_err(to64(o0[b, h:h + 1, :n]), o_ref[:, :n]) <= 2e-2, (b, h)
            assert rel_err(to64(S[b, h]), M_ref[0] * np.sqrt(m)) < 5e-5
            assert rel_err(to64(z[b, h]), a_ref[0] * np.sqrt(m)) < 5e-5



@pytest.mark.parametrize("d,m,W,lens,per_head", [(128, 128, 64, (130, 0, 1, 257, 64), False), (64, 128, 64, (5, 300, 17), True),
                                                 (64, 32, 7, (40, 41), False)])
def test_packed_batches(d, m, W, lens, per_head):
    """Sequences laid end to end in one token buffer (cu_seqlens), with a gap of unused rows in front and behind:
    forward, backward and ring fill against the oracle run on every sequence alone; lengths 0 and 1 included;
    rows outside every sequence stay untouched."""
    H = 2
    front, back = 3, 5
    starts = np.concatenate([[front], front + np.cumsum(lens)]).astype(np.int32)
    total = int(starts[-1]) + back
    t = synth.make_inputs(1, H, total, d, seed=1900 + d + m, dtype="bf16", scale="rms")
    om = synth.make_omega(d, m, heads=H if per_head else None)
    g = {n: v[0].contiguous().cuda() for n, v in t.items()}             # [H, total, d]
    omg = om.cuda()
    cu = torch.from_numpy(starts).cuda()
    o, L, lse, S, z = P.fwd_packed(g["q"], g["k"], g["v"], g["r"], g["u"], omg, cu, max(lens), W=W, return_state=True)
    grads = P.bwd_packed(g["q"], g["k"], g["v"], g["r"], g["u"], omg, cu, max(lens), L, lse, g["dO"], W=W)
    ring_r, ring_u = P.ring_fill_packed(g["r"], g["u"], cu, W=W)
    torch.cuda.synchronize()
    inside = torch.zeros(total, dtype=torch.bool)
    for b, n in enumerate(lens):
        inside[starts[b]:starts[b] + n] = True
    for got in (o,) + grads:
        assert torch.all(got[:, ~inside.cuda()] == 0)
    for b, n in enumerate(lens):
        if n == 0:
            assert torch.all(S[b] == 0) and torch.all(z[b] == 0) and torch.all(ring_r[b] == 0)
            continue
        lo = int(starts[b])
        for h in range(H):
            cut = {name: to64(t[name][0, h:h + 1, lo:lo + n]) for name in ("q", "k", "v", "r", "u", "dO")}
            omh = to64(om[h] if per_head else om)
            o_ref, _, M_ref, a_ref = C.fwd(cut["q"], cut["k"], cut["v"], cut["r"], cut["u"], omh, W, return_state=True)
            assert rel_err(to64(o[h:h + 1, lo:lo + n]), o_ref) <= 2e-2, (b, h)
            assert rel_err(to64(S[b, h:h + 1]), M_ref * np.sqrt(m)) < 5e-5
            assert rel_err(to64(z[b, h:h + 1]), a_ref * np.sqrt(m)) < 5e-5
            g_ref = C.bwd(cut["q"], cut["k"], cut["v"], cut["r"], cut["u"], omh, W, cut["dO"])
            for name, got, want in zip(("dq", "dk", "dv", "dr", "du"), grads, g_ref):
                assert rel_err(to64(got[h:h + 1, lo:lo + n]), want, floor=1e-2) <= 2e-2, (b, h, name)
            for tok in range(max(0, n - W), n):
                assert torch.equal(ring_r[b, h, tok % W], g["r"][h, lo + tok]) and torch.equal(ring_u[b, h, tok % W], g["u"][h, lo + tok])
