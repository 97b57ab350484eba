"""CPU-only checks of the C ABI: the library loads, exports every declared symbol and
rejects bad arguments on the host before touching CUDA."""
import ctypes
import os
import re

import paper_2608_09307_b200 as P
from paper_2608_09307_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            src = open(os.path.join(ROOT, "include", fn)).read()
            src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
            names |= set(re.findall(r"\b(linsimp_[a-z_0-9]+)\s*\(", src))
    return names


def test_exports_every_declared_symbol():
    lib = P.load_library()
    decl = _declared()
    assert {"linsimp_fwd", "linsimp_bwd", "linsimp_decode_step", "linsimp_workspace_bytes"} <= decl
    for name in decl:
        assert hasattr(lib, name), name
    assert set(binding.EXPORTS) <= decl
    assert lib.linsimp_version() == 6


def test_workspace_and_argument_checks_on_host():
    lib = P.load_library()
    p = binding.make_params(2, 3, 100, 64, 128, 64, P.BF16)
    assert P.workspace_bytes(p, P.OP_FWD) > 0
    assert P.workspace_bytes(p, P.OP_BWD) > P.workspace_bytes(p, P.OP_FWD)
    bad = binding.make_params(2, 3, 100, 48, 128, 64, P.BF16)       # d = 48 has no instance
    assert P.workspace_bytes(bad, P.OP_FWD) == 0
    # null pointers -> EINVAL, nothing launched (no CUDA device needed)
    n = ctypes.c_void_p(None)
    rc = lib.linsimp_fwd(ctypes.byref(p), n, n, n, n, n, n, n, n, n, n, n, n, 0, n)
    assert rc == -1
    assert b"invalid" in lib.linsimp_strerror(rc)
    # non-null but misaligned pointer -> EALIGN; too-small workspace -> EWORKSPACE
    buf = ctypes.create_string_buffer(4096)
    a = ctypes.addressof(buf)
    al = ctypes.c_void_p((a + 255) // 256 * 256)
    mis = ctypes.c_void_p(al.value + 4)
    rc = lib.linsimp_fwd(ctypes.byref(p), mis, al, al, al, al, al, al, al, al, n, n, al, 0, n)
    assert rc == -3
    rc = lib.linsimp_fwd(ctypes.byref(p), al, al, al, al, al, al, al, al, al, n, n, al, 16, n)
    assert rc == -4
    rc = lib.linsimp_fwd(ctypes.byref(bad), al, al, al, al, al, al, al, al, al, n, n, al, 1 << 40, n)
    assert rc == -2
    w65 = binding.make_params(1, 1, 10, 64, 64, 65, P.BF16)
    rc = lib.linsimp_fwd(ctypes.byref(w65), al, al, al, al, al, al, al, al, al, n, n, al, 1 << 40, n)
    assert rc == -2
    # S_final without z_final
    rc = lib.linsimp_fwd(ctypes.byref(p), al, al, al, al, al, al, al, al, al, al, n, al, 1 << 40, n)
    assert rc == -1
    rc = lib.linsimp_decode_step(ctypes.byref(p), n, n, n, n, n, n, n, n, n, n, n, n, n, 0, n)
    assert rc == -1
    rc = lib.linsimp_bwd(ctypes.byref(p), *([n] * 15), n, 0, n)
    assert rc == -1
    # unknown flag bits are refused; the known one changes no size
    odd = binding.make_params(2, 3, 100, 64, 128, 64, P.BF16, flags=64)
    assert P.workspace_bytes(odd, P.OP_BWD) == 0
    keep = binding.make_params(2, 3, 100, 64, 128, 64, P.BF16, flags=binding.FLAG_REUSE_FWD_STATE)
    assert P.workspace_bytes(keep, P.OP_BWD) == P.workspace_bytes(p, P.OP_BWD)
    # both orientations averaged: more scratch; not for the decode step, fp32 streams or ranks above 128
    two = binding.make_params(2, 3, 100, 64, 128, 64, P.BF16, flags=binding.FLAG_TWO_VIEWS)
    assert P.workspace_bytes(two, P.OP_FWD) > P.workspace_bytes(p, P.OP_FWD)
    assert P.workspace_bytes(two, P.OP_BWD) > P.workspace_bytes(p, P.OP_BWD)
    assert P.workspace_bytes(two, P.OP_DECODE) == 0
    assert P.workspace_bytes(binding.make_params(2, 3, 100, 64, 128, 64, P.F32, flags=binding.FLAG_TWO_VIEWS), P.OP_FWD) == 0
    assert P.workspace_bytes(binding.make_params(2, 3, 100, 64, 256, 64, P.BF16, flags=binding.FLAG_TWO_VIEWS), P.OP_FWD) == 0
    # the state as two bf16 terms: a second image (128 x m bf16) per 16-token chunk in the backward's workspace, none
    # in the forward's; fp32 streams take the bit without effect
    terms = binding.make_params(2, 3, 100, 64, 128, 64, P.BF16, flags=binding.FLAG_STATE_TWO_TERMS)
    extra = P.workspace_bytes(terms, P.OP_BWD) - P.workspace_bytes(p, P.OP_BWD)
    assert 2 * 3 * 7 * 128 * 128 * 2 <= extra < 2 * 3 * 7 * 128 * 128 * 2 + 4096
    assert P.workspace_bytes(terms, P.OP_FWD) == P.workspace_bytes(p, P.OP_FWD)
    f32 = binding.make_params(2, 3, 100, 64, 128, 64, P.F32)
    f32t = binding.make_params(2, 3, 100, 64, 128, 64, P.F32, flags=binding.FLAG_STATE_TWO_TERMS)
    assert P.workspace_bytes(f32t, P.OP_BWD) == P.workspace_bytes(f32, P.OP_BWD) > 0
    # normalisation / gate calls: one float per 128 rows of a unit, rounded up to 256 bytes
    assert P.workspace_bytes(p, P.OP_NORM) == 256
    big = binding.make_params(2, 16, 16384, 128, 128, 64, P.BF16)
    assert P.workspace_bytes(big, P.OP_NORM) == 2 * 16 * 128 * 4
    odd_d = binding.make_params(2, 3, 100, 6, 1, 1, P.BF16)
    assert P.workspace_bytes(odd_d, P.OP_NORM) == 0
    f = ctypes.c_float(1e-6)
    assert lib.linsimp_qkr_normalize(ctypes.byref(p), al, al, al, n, al, al, al, n) == -1
    assert lib.linsimp_qkr_normalize(ctypes.byref(odd_d), al, al, al, al, al, al, al, n) == -2
    assert lib.linsimp_qkr_normalize(ctypes.byref(p), al, mis, al, al, al, al, al, n) == -3
    assert lib.linsimp_gate_rmsnorm(ctypes.byref(p), al, al, ctypes.c_float(-1.0), al, n) == -1
    assert lib.linsimp_gate_rmsnorm_bwd(ctypes.byref(p), al, al, f, al, al, al, al, 16, n) == -4
    assert lib.linsimp_qkr_normalize_bwd(ctypes.byref(p), *([al] * 11), n, 0, n) == -4
    # padded batches: seq_lens is required
    assert lib.linsimp_fwd_padded(ctypes.byref(p), al, al, al, al, al, al, n, al, al, al, n, n, al, 1 << 40, n) == -1
    assert lib.linsimp_ring_fill_padded(ctypes.byref(p), al, al, n, al, al, n) == -1


def test_packed_and_continued_calls_check_their_arguments_on_the_host():
    lib = P.load_library()
    n = ctypes.c_void_p(None)
    buf = ctypes.create_string_buffer(4096)
    al = ctypes.c_void_p((ctypes.addressof(buf) + 255) // 256 * 256)
    p = binding.make_params(3, 2, 100, 64, 128, 64, P.BF16)
    f32 = binding.make_params(3, 2, 100, 64, 128, 64, P.F32)
    keep = binding.make_params(3, 2, 100, 64, 128, 64, P.BF16, flags=binding.FLAG_REUSE_FWD_STATE)
    inner = P.workspace_bytes(p, P.OP_BWD)
    assert P.workspace_bytes(p, binding.OP_BWD_PACKED) >= inner + 11 * 3 * 2 * 100 * 64 * 2
    assert P.workspace_bytes(p, binding.OP_FWD_PACKED) >= P.workspace_bytes(p, P.OP_FWD) + 6 * 3 * 2 * 100 * 64 * 2
    assert P.workspace_bytes(f32, binding.OP_FWD_PACKED) == 0 and P.workspace_bytes(keep, binding.OP_BWD_PACKED) == 0
    # forward: cu_seqlens missing -> EINVAL; fp32 streams -> EUNSUPPORTED; workspace too small -> EWORKSPACE
    fwd = lambda pp, cu, ws: lib.linsimp_fwd_packed(ctypes.byref(pp), al, al, al, al, al, al, cu, 300, al, al, al, n, n, al, ws, n)
    assert fwd(p, n, 1 << 40) == -1
    assert fwd(f32, al, 1 << 40) == -2
    assert fwd(p, al, 64) == -4
    assert fwd(keep, al, 1 << 40) == -1
    bwd = lambda pp, cu, ws: lib.linsimp_bwd_packed(ctypes.byref(pp), al, al, al, al, al, al, cu, 300, al, al, al, al, al, al, al, al,
                                                    al, ws, n)
    assert bwd(p, n, 1 << 40) == -1 and bwd(f32, al, 1 << 40) == -2 and bwd(p, al, 64) == -4
    assert lib.linsimp_ring_fill_packed(ctypes.byref(p), al, al, n, 300, al, al, n) == -1
    # continued backward: history without its gradient buffers, state gradient without its partner, reuse flag
    cont = lambda pp, hr, dhr, nh, dSf, dzf: lib.linsimp_bwd_continue(ctypes.byref(pp), al, al, al, al, al, al, al, al, hr, hr, nh,
                                                                       al, al, al, dSf, dzf, al, al, al, al, al, dhr, dhr, al, al,
                                                                       al, 64, n)
    assert cont(p, al, n, 5, n, n) == -1
    assert cont(p, al, al, 64, n, n) == -1                 # more than W - 1 history rows
    assert cont(p, n, n, 0, al, n) == -1
    assert cont(keep, n, n, 0, n, n) == -1
    assert cont(f32, n, n, 0, n, n) == -2
    assert cont(p, al, al, 5, al, al) == -4                # everything in order except the workspace size


def test_value_width_is_taken_by_forward_and_backward_only():
    lib = P.load_library()
    n = ctypes.c_void_p(None)
    buf = ctypes.create_string_buffer(4096)
    al = ctypes.c_void_p((ctypes.addressof(buf) + 255) // 256 * 256)
    same = binding.make_params(2, 3, 100, 64, 128, 64, P.BF16)
    wide = binding.make_params(2, 3, 100, 64, 128, 64, P.BF16, dv=160)       # three blocks of 64 value channels
    assert P.workspace_bytes(wide, P.OP_FWD) > P.workspace_bytes(same, P.OP_FWD)
    assert P.workspace_bytes(wide, P.OP_BWD) > P.workspace_bytes(same, P.OP_BWD)
    assert P.workspace_bytes(binding.make_params(2, 3, 100, 64, 128, 64, P.BF16, dv=64), P.OP_FWD) == P.workspace_bytes(same, P.OP_FWD)
    for op in (P.OP_DECODE, P.OP_STATE, binding.OP_FWD_PACKED):
        assert P.workspace_bytes(wide, op) == 0
    assert P.workspace_bytes(binding.make_params(2, 3, 100, 64, 128, 64, P.BF16, dv=100), P.OP_FWD) == 0     # rows of 200 bytes
    assert P.workspace_bytes(binding.make_params(2, 3, 100, 64, 128, 64, P.BF16, dv=-8), P.OP_FWD) == 0
    assert P.workspace_bytes(binding.make_params(2, 3, 100, 64, 128, 64, P.BF16, dv=160, flags=binding.FLAG_TWO_VIEWS), P.OP_FWD) == 0
    # calls that know one width only refuse the parameter
    assert lib.linsimp_fwd_padded(ctypes.byref(wide), al, al, al, al, al, al, al, al, al, al, n, n, al, 1 << 40, n) == -1
    assert lib.linsimp_decode_step(ctypes.byref(wide), *([al] * 13), 1 << 20, n) == -1
    assert lib.linsimp_fwd(ctypes.byref(wide), al, al, al, al, al, al, al, al, al, n, n, al, 64, n) == -4


def test_large_decode_batches_still_get_every_check():
    """More than 65535 (sequence, head) units are fine for the decode step (its grid does not depend on them), and
    the remaining parameter checks apply to such a batch like to any other."""
    lib = P.load_library()
    n = ctypes.c_void_p(None)
    big = binding.make_params(8192, 16, 0, 128, 128, 64, P.BF16)
    assert lib.linsimp_decode_step(ctypes.byref(big), *([n] * 13), 0, n) == -1        # null pointers, not the size
    assert P.workspace_bytes(big, P.OP_DECODE) > 0
    assert P.workspace_bytes(big, P.OP_FWD) == 0                                       # the chunked kernels' grid limit
    for field, value in (("io_dtype", 7), ("eps", float("nan")), ("eps", -1.0), ("flags", 64), ("algo", 9)):
        bad = binding.make_params(8192, 16, 0, 128, 128, 64, P.BF16)
        setattr(bad, field, value)
        assert P.workspace_bytes(bad, P.OP_DECODE) == 0, field
        buf = ctypes.create_string_buffer(4096)
        al = ctypes.c_void_p((ctypes.addressof(buf) + 255) // 256 * 256)
        assert lib.linsimp_decode_step(ctypes.byref(bad), *([al] * 13), 1 << 20, n) == -1, field


def test_workspace_is_zero_where_no_kernel_serves_the_combination():
    # feature ranks above 128 exist as tensor-core feature blocks for bf16 I/O with the default algo only
    ok = binding.make_params(1, 2, 100, 128, 256, 64, P.BF16)
    assert P.workspace_bytes(ok, P.OP_FWD) > 0
    for io, algo in ((P.F32, P.ALGO_DEFAULT), (P.BF16, P.ALGO_FP32), (P.F32, P.ALGO_FP32)):
        none = binding.make_params(1, 2, 100, 128, 256, 64, io, False, algo)
        assert P.workspace_bytes(none, P.OP_FWD) == 0
        assert P.workspace_bytes(none, P.OP_BWD) == 0
    # d = 64 has a CUDA-core instance at m = 256
    assert P.workspace_bytes(binding.make_params(1, 2, 100, 64, 256, 64, P.F32), P.OP_FWD) > 0


def test_descriptor_probe_refuses_unknown_encodings_on_the_host():
    lib = P.load_library()

    class Probe(ctypes.Structure):
        _fields_ = [("idesc", ctypes.c_uint32),
                    ("a_lbo", ctypes.c_uint32), ("a_sbo", ctypes.c_uint32), ("a_layout", ctypes.c_uint32),
                    ("b_lbo", ctypes.c_uint32), ("b_sbo", ctypes.c_uint32), ("b_layout", ctypes.c_uint32),
                    ("nk", ctypes.c_int), ("a_koff", ctypes.c_int * 16), ("b_koff", ctypes.c_int * 16),
                    ("a_bytes", ctypes.c_int), ("b_bytes", ctypes.c_int), ("n_out", ctypes.c_int),
                    ("a_from_tmem", ctypes.c_int)]

    pr = Probe()
    pr.idesc = (1 << 4) | (0 << 7) | (1 << 10) | (16 << 17) | (8 << 24)                 # fp16 A with bf16 B
    pr.a_lbo, pr.a_sbo, pr.a_layout = 0, 1024, 2
    pr.b_lbo, pr.b_sbo, pr.b_layout = 0, 1024, 2
    pr.nk, pr.a_bytes, pr.b_bytes, pr.n_out = 1, 32768, 32768, 128
    buf = ctypes.create_string_buffer(64)
    al = ctypes.c_void_p(ctypes.addressof(buf))
    assert lib.linsimp_debug_umma(al, al, ctypes.byref(pr), al, None, None) == -2         # refused before any launch
    assert lib.linsimp_debug_wait_expiry(None, 1, 100, None, None) == -1


def test_ops_refuse_cpu_tensors():
    import pytest
    import torch
    x = torch.zeros(1, 1, 4, 32)
    om = torch.zeros(32, 64)
    with pytest.raises(P.LinSimpError):
        P.fwd(x, x, x, x, x, om)
