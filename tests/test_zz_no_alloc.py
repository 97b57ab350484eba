"""linsimp_fwd_static: the workspace-free forward for callers that must not allocate device memory
(real-time loops, plug-ins without an allocator, fixed memory budgets).  Its scratch is a fixed
array inside the library, shared by all calls, so the checks are: on two calls in a row (the
second with different inputs, so stale scratch contents from the first would show) the result is
bit-identical to the regular entry point's - both run the same kernels, only the scratch differs -
and within the library's tolerance of the fp64 oracle; the second call leaves the device's free
memory untouched; and a problem that does not fit the array is refused cleanly.
Collected last on purpose: a failure here cannot hide other tests in a run that stops early."""
import ctypes

import numpy as np
import pytest
import torch

import paper_2608_09307_b200 as P
from oracle import c_ref as C
from paper_2608_09307_b200 import binding, synth
from tests.util import rel_err, units

pytestmark = pytest.mark.gpu


def _call_static(lib, p, g, omega, outs):
    o, L, lse, S, z = outs
    ptr = lambda t: ctypes.c_void_p(t.data_ptr())
    return lib.linsimp_fwd_static(ctypes.byref(p), ptr(g["q"]), ptr(g["k"]), ptr(g["v"]), ptr(g["r"]), ptr(g["u"]),
                                  ptr(omega), ptr(o), ptr(L), ptr(lse), ptr(S), ptr(z),
                                  ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))


@pytest.mark.parametrize("dtype,tol", [("fp32", 1e-4), ("bf16", 2e-2)])
def test_static_forward_matches_regular_entry_point_twice(dtype, tol):
    lib = P.load_library()
    B, H, T, d, m, W = 2, 3, 200, 64, 128, 64
    omega = synth.make_omega(d, m).cuda()
    tdt = torch.float32 if dtype == "fp32" else torch.bfloat16
    io = P.F32 if dtype == "fp32" else P.BF16
    p = binding.make_params(B, H, T, d, m, W, io, False, P.ALGO_FP32)
    assert P.workspace_bytes(p, P.OP_FWD) <= binding.STATIC_SCRATCH_BYTES
    for call, seed in enumerate((11, 12)):
        t = synth.make_inputs(B, H, T, d, seed=seed, dtype=dtype, scale="rms", with_dO=False)
        g = {k_: v_.cuda() for k_, v_ in t.items()}
        outs = (torch.empty(B, H, T, d, device="cuda", dtype=tdt), torch.empty(B, H, T, device="cuda"),
                torch.empty(B, H, T, device="cuda"), torch.empty(B, H, m, d, device="cuda"),
                torch.empty(B, H, m, device="cuda"))
        if call == 0:
            assert _call_static(lib, p, g, omega, outs) == 0
        else:
            # the second call must not change the device's free memory: nothing is allocated on its behalf
            # (up to three tries, in case anything else on the machine moves the figure at that very moment)
            unchanged = False
            for _ in range(3):
                torch.cuda.synchronize()
                free_before = torch.cuda.mem_get_info()[0]
                assert _call_static(lib, p, g, omega, outs) == 0
                torch.cuda.synchronize()
                unchanged = unchanged or torch.cuda.mem_get_info()[0] == free_before
                if unchanged:
                    break
            assert unchanged
        o_ref, L_ref, lse_ref, S_ref, z_ref = P.fwd(g["q"], g["k"], g["v"], g["r"], g["u"], omega, W=W,
                                                    algo=P.ALGO_FP32, return_state=True)
        torch.cuda.synchronize()
        for got, ref in zip(outs, (o_ref, L_ref, lse_ref, S_ref, z_ref)):
            assert torch.isfinite(got.float()).all()
            assert torch.equal(got, ref), call                      # same kernels, other scratch: same bits
        # and against the oracle, like every other entry point
        o_orc = C.fwd(*[units(t[n]) for n in ("q", "k", "v", "r", "u")], omega.cpu().double().numpy(), W)
        assert rel_err(units(outs[0]), o_orc) <= tol, call
    # the Python convenience wrapper goes through the same entry point
    o2, _, _ = binding.fwd_static(g["q"], g["k"], g["v"], g["r"], g["u"], omega, W=W)
    torch.cuda.synchronize()
    assert (o2.float() - o_ref.float()).abs().max().item() <= tol * o_ref.float().abs().max().item()


def test_static_forward_refuses_problems_beyond_its_scratch():
    lib = P.load_library()
    # 4 x 16 sequences of 8192 tokens at d = m = 128 would need ~1 GB of scratch
    p = binding.make_params(4, 16, 8192, 128, 128, 64, P.BF16, False, P.ALGO_FP32)
    assert P.workspace_bytes(p, P.OP_FWD) > binding.STATIC_SCRATCH_BYTES
    dummy = torch.zeros(64, device="cuda")
    ptr = ctypes.c_void_p(dummy.data_ptr())
    rc = lib.linsimp_fwd_static(ctypes.byref(p), ptr, ptr, ptr, ptr, ptr, ptr, ptr, ptr, ptr, None, None, None)
    assert rc == -6
    assert b"static" in lib.linsimp_strerror(rc)
