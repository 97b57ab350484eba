"""ctypes binding of liblinsimp.so: same names as the C ABI, argument marshalling only."""
import ctypes
import os

import torch

F32, BF16 = 0, 1
OP_FWD, OP_BWD, OP_DECODE, OP_STATE, OP_NORM, OP_FWD_PACKED, OP_BWD_PACKED = 0, 1, 2, 3, 4, 5, 6
ALGO_DEFAULT, ALGO_FP32 = 0, 1
FLAG_REUSE_FWD_STATE = 1
FLAG_OMEGA_IMAGE = 2
FLAG_TWO_VIEWS = 4
FLAG_STATE_TWO_TERMS = 8

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "liblinsimp.so")
_lib = None

EXPORTS = ("linsimp_workspace_bytes", "linsimp_fwd", "linsimp_bwd", "linsimp_decode_step",
           "linsimp_prefill_state", "linsimp_decode_prepare", "linsimp_fwd_continue", "linsimp_ring_fill",
           "linsimp_strerror", "linsimp_version", "linsimp_last_launch_count",
           "linsimp_profile_enable", "linsimp_profile_read", "linsimp_read_status", "linsimp_fwd_static",
           "linsimp_qkr_normalize", "linsimp_qkr_normalize_bwd", "linsimp_gate_rmsnorm", "linsimp_gate_rmsnorm_bwd",
           "linsimp_fwd_padded", "linsimp_bwd_padded", "linsimp_ring_fill_padded", "linsimp_bwd_continue",
           "linsimp_fwd_packed", "linsimp_bwd_packed", "linsimp_ring_fill_packed", "linsimp_winsimp_fwd")


class LinSimpError(RuntimeError):
    pass


class Params(ctypes.Structure):
    """Mirror of `linsimp_params`."""
    _fields_ = [("B", ctypes.c_int32), ("H", ctypes.c_int32), ("T", ctypes.c_int32), ("d", ctypes.c_int32),
                ("m", ctypes.c_int32), ("W", ctypes.c_int32), ("io_dtype", ctypes.c_int32),
                ("omega_per_head", ctypes.c_int32), ("algo", ctypes.c_int32), ("eps", ctypes.c_float),
                ("flags", ctypes.c_int32), ("dv", ctypes.c_int32)]


def lib_path():
    return _LIB_PATH


def load_library():
    """Loads liblinsimp.so (built in-tree by paper_2608_09307_b200.build); raises if missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise LinSimpError("liblinsimp.so is not built: run `python -m paper_2608_09307_b200.build` "
                           "(there is no fallback path)")
    lib = ctypes.CDLL(_LIB_PATH)
    vp, fp, ip = ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p
    pp = ctypes.POINTER(Params)
    lib.linsimp_workspace_bytes.restype = ctypes.c_size_t
    lib.linsimp_workspace_bytes.argtypes = [pp, ctypes.c_int]
    lib.linsimp_fwd.restype = ctypes.c_int
    lib.linsimp_fwd.argtypes = [pp, vp, vp, vp, vp, vp, fp, vp, fp, fp, fp, fp, vp, ctypes.c_size_t, vp]
    lib.linsimp_bwd.restype = ctypes.c_int
    lib.linsimp_bwd.argtypes = [pp, vp, vp, vp, vp, vp, fp, vp, fp, fp, vp, vp, vp, vp, vp, vp, vp,
                                ctypes.c_size_t, vp]
    lib.linsimp_decode_step.restype = ctypes.c_int
    lib.linsimp_decode_step.argtypes = [pp, vp, vp, vp, vp, vp, fp, fp, fp, vp, vp, ip, vp, vp,
                                        ctypes.c_size_t, vp]
    lib.linsimp_fwd_continue.restype = ctypes.c_int
    lib.linsimp_fwd_continue.argtypes = [pp, vp, vp, vp, vp, vp, fp, fp, fp, vp, vp, ctypes.c_int32, vp, fp, fp, fp, fp,
                                         vp, ctypes.c_size_t, vp]
    lib.linsimp_bwd_continue.restype = ctypes.c_int
    lib.linsimp_bwd_continue.argtypes = [pp, vp, vp, vp, vp, vp, fp, fp, fp, vp, vp, ctypes.c_int32, fp, fp, vp, fp, fp,
                                         vp, vp, vp, vp, vp, vp, vp, fp, fp, vp, ctypes.c_size_t, vp]
    lib.linsimp_ring_fill.restype = ctypes.c_int
    lib.linsimp_ring_fill.argtypes = [pp, vp, vp, ctypes.c_int64, vp, vp, vp]
    lib.linsimp_decode_prepare.restype = ctypes.c_int
    lib.linsimp_decode_prepare.argtypes = [pp, fp, vp, ctypes.c_size_t, vp]
    lib.linsimp_prefill_state.restype = ctypes.c_int
    lib.linsimp_prefill_state.argtypes = [pp, vp, vp, fp, fp, fp, vp, ctypes.c_size_t, vp]
    lib.linsimp_profile_enable.restype = ctypes.c_int
    lib.linsimp_profile_enable.argtypes = [ctypes.c_int]
    lib.linsimp_profile_read.restype = ctypes.c_int
    lib.linsimp_profile_read.argtypes = [ctypes.c_int, ctypes.c_char_p, ctypes.c_int,
                                         ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_int)]
    lib.linsimp_fwd_static.restype = ctypes.c_int
    lib.linsimp_fwd_static.argtypes = [pp, vp, vp, vp, vp, vp, fp, vp, fp, fp, fp, fp, vp]
    lib.linsimp_qkr_normalize.restype = ctypes.c_int
    lib.linsimp_qkr_normalize.argtypes = [pp, vp, vp, vp, fp, vp, vp, vp, vp]
    lib.linsimp_qkr_normalize_bwd.restype = ctypes.c_int
    lib.linsimp_qkr_normalize_bwd.argtypes = [pp, vp, vp, vp, fp, vp, vp, vp, vp, vp, vp, fp, vp, ctypes.c_size_t, vp]
    lib.linsimp_gate_rmsnorm.restype = ctypes.c_int
    lib.linsimp_gate_rmsnorm.argtypes = [pp, vp, fp, ctypes.c_float, vp, vp]
    lib.linsimp_gate_rmsnorm_bwd.restype = ctypes.c_int
    lib.linsimp_gate_rmsnorm_bwd.argtypes = [pp, vp, fp, ctypes.c_float, vp, vp, fp, vp, ctypes.c_size_t, vp]
    lib.linsimp_fwd_padded.restype = ctypes.c_int
    lib.linsimp_fwd_padded.argtypes = [pp, vp, vp, vp, vp, vp, fp, ip, vp, fp, fp, fp, fp, vp, ctypes.c_size_t, vp]
    lib.linsimp_bwd_padded.restype = ctypes.c_int
    lib.linsimp_bwd_padded.argtypes = [pp, vp, vp, vp, vp, vp, fp, ip, vp, fp, fp, vp, vp, vp, vp, vp, vp, vp,
                                       ctypes.c_size_t, vp]
    lib.linsimp_ring_fill_padded.restype = ctypes.c_int
    lib.linsimp_ring_fill_padded.argtypes = [pp, vp, vp, ip, vp, vp, vp]
    lib.linsimp_fwd_packed.restype = ctypes.c_int
    lib.linsimp_fwd_packed.argtypes = [pp, vp, vp, vp, vp, vp, fp, ip, ctypes.c_int64, vp, fp, fp, fp, fp, vp, ctypes.c_size_t, vp]
    lib.linsimp_bwd_packed.restype = ctypes.c_int
    lib.linsimp_bwd_packed.argtypes = [pp, vp, vp, vp, vp, vp, fp, ip, ctypes.c_int64, fp, fp, vp, vp, vp, vp, vp, vp, vp,
                                       ctypes.c_size_t, vp]
    lib.linsimp_ring_fill_packed.restype = ctypes.c_int
    lib.linsimp_ring_fill_packed.argtypes = [pp, vp, vp, ip, ctypes.c_int64, vp, vp, vp]
    lib.linsimp_winsimp_fwd.restype = ctypes.c_int
    lib.linsimp_winsimp_fwd.argtypes = [pp, ctypes.c_int32, vp, vp, vp, vp, vp, vp, fp, vp]
    lib.linsimp_read_status.restype = ctypes.c_int
    lib.linsimp_read_status.argtypes = [vp, vp]
    lib.linsimp_strerror.restype = ctypes.c_char_p
    lib.linsimp_strerror.argtypes = [ctypes.c_int]
    lib.linsimp_version.restype = ctypes.c_int
    lib.linsimp_last_launch_count.restype = ctypes.c_int
    lib.linsimp_last_launch_count.argtypes = [ctypes.c_int]
    _lib = lib
    return lib


def _check(code):
    if code != 0:
        raise LinSimpError("linsimp error %d: %s" % (code, load_library().linsimp_strerror(code).decode()))


def _io_dtype(t):
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise LinSimpError("unsupported tensor dtype %s" % t.dtype)


def _dev(*tensors):
    for t in tensors:
        if t is None:
            continue
        if not t.is_cuda:
            raise LinSimpError("linsimp ops need CUDA tensors (there is no CPU path)")
        if not t.is_contiguous():
            raise LinSimpError("linsimp ops need contiguous tensors")


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def make_params(B, H, T, d, m, W, io_dtype, omega_per_head=False, algo=ALGO_DEFAULT, eps=1e-30, flags=0, dv=0):
    return Params(B, H, T, d, m, W, io_dtype, 1 if omega_per_head else 0, algo, eps, flags, dv)


def workspace_bytes(params, op):
    return int(load_library().linsimp_workspace_bytes(ctypes.byref(params), op))


def _workspace(params, op, workspace, device):
    need = workspace_bytes(params, op)
    if workspace is None:
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=device)
    return workspace, workspace.numel() * workspace.element_size()


def last_launch_count(op):
    return int(load_library().linsimp_last_launch_count(op))


def fwd(q, k, v, r, u, omega, W=64, eps=1e-30, algo=ALGO_DEFAULT, return_state=False, workspace=None,
        out=None, stream=None, two_views=False, two_term_state=False):
    """linsimp_fwd.  q,k,v,r,u [B,H,T,d] (fp32 or bf16, CUDA); omega fp32 [d,m] or [H,d,m].

    two_views: both orientations of the trilinear score averaged (LINSIMP_FLAG_TWO_VIEWS).
    two_term_state: leave the boundary states for a backward that is called with reuse_fwd_state and two_term_state
    (LINSIMP_FLAG_STATE_TWO_TERMS; the workspace must have the size that backward asks for).
    Returns (o, rowmax_L, lse) and, with return_state, also (S_final, z_final).
    """
    lib = load_library()
    _dev(q, k, v, r, u, omega)
    B, H, T, d = q.shape
    m = omega.shape[-1]
    dv = v.shape[-1]
    p = make_params(B, H, T, d, m, W, _io_dtype(q), omega.dim() == 3, algo, eps,
                    (FLAG_TWO_VIEWS if two_views else 0) | (FLAG_STATE_TWO_TERMS if two_term_state else 0),
                    0 if dv == d else dv)
    o = torch.empty_like(v) if out is None else out
    L = torch.empty((B, H, T), dtype=torch.float32, device=q.device)
    lse = torch.empty((B, H, T), dtype=torch.float32, device=q.device)
    S = z = None
    if return_state:
        S = torch.empty((B, H, m, dv), dtype=torch.float32, device=q.device)
        z = torch.empty((B, H, m), dtype=torch.float32, device=q.device)
    ws, ws_bytes = _workspace(p, OP_FWD, workspace, q.device)
    _check(lib.linsimp_fwd(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(r), _ptr(u), _ptr(omega),
                           _ptr(o), _ptr(L), _ptr(lse), _ptr(S), _ptr(z), _ptr(ws), ws_bytes, _stream(stream)))
    if return_state:
        return o, L, lse, S, z
    return o, L, lse


def fwd_continue(q, k, v, r, u, omega, state=None, history=None, W=64, eps=1e-30, return_state=True, workspace=None,
                 out=None, stream=None):
    """linsimp_fwd_continue: forward of a segment [B,H,T,d] that continues a sequence.

    state = (S, z): prefix state before the segment (None: empty); history = (hist_r, hist_u) [B,H,n,d], n <= W-1:
    r and u of the n tokens before the segment, oldest first (None: none).
    Returns (o, rowmax_L, lse) and, with return_state, also (S_final, z_final).
    """
    lib = load_library()
    _dev(q, k, v, r, u, omega)
    B, H, T, d = q.shape
    m = omega.shape[-1]
    p = make_params(B, H, T, d, m, W, _io_dtype(q), omega.dim() == 3, ALGO_DEFAULT, eps)
    S0, z0 = (None, None) if state is None else state
    hr, hu = (None, None) if history is None else history
    n_hist = 0 if hr is None else int(hr.shape[2])
    if n_hist == 0:
        hr = hu = None
    else:
        _dev(hr, hu)
    if S0 is not None:
        _dev(S0, z0)
    o = torch.empty_like(q) if out is None else out
    L = torch.empty((B, H, T), dtype=torch.float32, device=q.device)
    lse = torch.empty((B, H, T), dtype=torch.float32, device=q.device)
    S = z = None
    if return_state:
        S = torch.empty((B, H, m, d), dtype=torch.float32, device=q.device)
        z = torch.empty((B, H, m), dtype=torch.float32, device=q.device)
    ws, ws_bytes = _workspace(p, OP_FWD, workspace, q.device)
    _check(lib.linsimp_fwd_continue(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(r), _ptr(u), _ptr(omega),
                                    _ptr(S0), _ptr(z0), _ptr(hr), _ptr(hu), n_hist, _ptr(o), _ptr(L), _ptr(lse),
                                    _ptr(S), _ptr(z), _ptr(ws), ws_bytes, _stream(stream)))
    if return_state:
        return o, L, lse, S, z
    return o, L, lse


def bwd_continue(q, k, v, r, u, omega, L, lse, dO, state=None, history=None, d_state=None, W=64, eps=1e-30,
                 workspace=None, stream=None):
    """linsimp_bwd_continue: backward of a segment run with fwd_continue.

    state = (S_init, z_init) or None, history = (hist_r, hist_u) or None as given to fwd_continue;
    d_state = (dS_final, dz_final) or None: the gradient later segments send into the state after this one.
    Returns (dq, dk, dv, dr, du), (d_hist_r, d_hist_u) or None, (dS_init, dz_init)."""
    lib = load_library()
    _dev(q, k, v, r, u, omega, L, lse, dO)
    B, H, T, d = q.shape
    m = omega.shape[-1]
    p = make_params(B, H, T, d, m, W, _io_dtype(q), omega.dim() == 3, ALGO_DEFAULT, eps)
    S0 = z0 = hr = hu = dSf = dzf = None
    n_hist = 0
    if state is not None:
        S0, z0 = state
        _dev(S0, z0)
    if history is not None and history[0].shape[2] > 0:
        hr, hu = history
        _dev(hr, hu)
        n_hist = hr.shape[2]
    if d_state is not None:
        dSf, dzf = d_state
        _dev(dSf, dzf)
    grads = [torch.empty_like(q) for _ in range(5)]
    dh = None
    if n_hist:
        dh = (torch.empty_like(hr), torch.empty_like(hu))
    dS0 = torch.empty((B, H, m, d), dtype=torch.float32, device=q.device)
    dz0 = torch.empty((B, H, m), dtype=torch.float32, device=q.device)
    ws, ws_bytes = _workspace(p, OP_BWD, workspace, q.device)
    _check(lib.linsimp_bwd_continue(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(r), _ptr(u), _ptr(omega),
                                    _ptr(S0), _ptr(z0), _ptr(hr), _ptr(hu), n_hist, _ptr(L), _ptr(lse), _ptr(dO),
                                    _ptr(dSf), _ptr(dzf), *[_ptr(g) for g in grads],
                                    _ptr(dh[0]) if dh else None, _ptr(dh[1]) if dh else None, _ptr(dS0), _ptr(dz0),
                                    _ptr(ws), ws_bytes, _stream(stream)))
    return tuple(grads), dh, (dS0, dz0)


def ring_fill(r, u, ring_r, ring_u, t_first=0, stream=None):
    """linsimp_ring_fill: the last min(T, W) rows of r, u [B,H,T,d] into their slots of ring_r, ring_u [B,H,W,d]."""
    lib = load_library()
    _dev(r, u, ring_r, ring_u)
    B, H, T, d = r.shape
    W = ring_r.shape[2]
    p = make_params(B, H, T, d, 64, W, _io_dtype(r))
    _check(lib.linsimp_ring_fill(ctypes.byref(p), _ptr(r), _ptr(u), int(t_first), _ptr(ring_r), _ptr(ring_u),
                                 _stream(stream)))


def bwd(q, k, v, r, u, omega, o, L, lse, dO, W=64, eps=1e-30, algo=ALGO_DEFAULT, workspace=None, stream=None,
        reuse_fwd_state=False, two_views=False, two_term_state=False):
    """linsimp_bwd.  Returns dq, dk, dv, dr, du (same shape/dtype as the inputs).

    two_term_state: the boundary states enter the backward's products as two bf16 terms (LINSIMP_FLAG_STATE_TWO_TERMS):
    halves the error of dk for a sixth more time in the tile kernel and a second state image in the workspace.

    reuse_fwd_state: `workspace` is the tensor the preceding fwd() call on the same inputs was given
    (sized for the backward) and has not been written since; the backward then skips the state pre-pass.
    """
    lib = load_library()
    _dev(q, k, v, r, u, omega, o, L, lse, dO)
    B, H, T, d = q.shape
    m = omega.shape[-1]
    if reuse_fwd_state and workspace is None:
        raise ValueError("reuse_fwd_state needs the workspace of the forward call")
    dv = v.shape[-1]
    p = make_params(B, H, T, d, m, W, _io_dtype(q), omega.dim() == 3, algo, eps,
                    (FLAG_REUSE_FWD_STATE if reuse_fwd_state else 0) | (FLAG_TWO_VIEWS if two_views else 0) |
                    (FLAG_STATE_TWO_TERMS if two_term_state else 0), 0 if dv == d else dv)
    grads = [torch.empty_like(x) for x in (q, k, v, r, u)]
    ws, ws_bytes = _workspace(p, OP_BWD, workspace, q.device)
    _check(lib.linsimp_bwd(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(r), _ptr(u), _ptr(omega),
                           _ptr(o), _ptr(L), _ptr(lse), _ptr(dO), *[_ptr(g) for g in grads],
                           _ptr(ws), ws_bytes, _stream(stream)))
    return tuple(grads)


def _lens(seq_lens, B):
    if seq_lens.dtype != torch.int32 or seq_lens.numel() != B:
        raise LinSimpError("seq_lens must be an int32 tensor with one entry per batch element")
    _dev(seq_lens)
    return seq_lens


def fwd_padded(q, k, v, r, u, omega, seq_lens, W=64, eps=1e-30, return_state=False, workspace=None, out=None, stream=None):
    """linsimp_fwd_padded: forward of a batch padded to a common T; seq_lens int32 [B] (CUDA).

    Returns (o, rowmax_L, lse) and, with return_state, also (S_final, z_final) after each sequence's own last token."""
    lib = load_library()
    _dev(q, k, v, r, u, omega)
    B, H, T, d = q.shape
    m = omega.shape[-1]
    p = make_params(B, H, T, d, m, W, _io_dtype(q), omega.dim() == 3, ALGO_DEFAULT, eps)
    o = torch.empty_like(q) if out is None else out
    L = torch.empty((B, H, T), dtype=torch.float32, device=q.device)
    lse = torch.empty((B, H, T), dtype=torch.float32, device=q.device)
    S = z = None
    if return_state:
        S = torch.empty((B, H, m, d), dtype=torch.float32, device=q.device)
        z = torch.empty((B, H, m), dtype=torch.float32, device=q.device)
    ws, ws_bytes = _workspace(p, OP_FWD, workspace, q.device)
    _check(lib.linsimp_fwd_padded(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(r), _ptr(u), _ptr(omega),
                                  _ptr(_lens(seq_lens, B)), _ptr(o), _ptr(L), _ptr(lse), _ptr(S), _ptr(z), _ptr(ws), ws_bytes,
                                  _stream(stream)))
    if return_state:
        return o, L, lse, S, z
    return o, L, lse


def bwd_padded(q, k, v, r, u, omega, seq_lens, o, L, lse, dO, W=64, eps=1e-30, workspace=None, stream=None,
               reuse_fwd_state=False):
    """linsimp_bwd_padded.  Returns dq, dk, dv, dr, du; rows of padding are zero."""
    lib = load_library()
    _dev(q, k, v, r, u, omega, o, L, lse, dO)
    B, H, T, d = q.shape
    m = omega.shape[-1]
    if reuse_fwd_state and workspace is None:
        raise ValueError("reuse_fwd_state needs the workspace of the forward call")
    p = make_params(B, H, T, d, m, W, _io_dtype(q), omega.dim() == 3, ALGO_DEFAULT, eps,
                    FLAG_REUSE_FWD_STATE if reuse_fwd_state else 0)
    grads = [torch.empty_like(q) for _ in range(5)]
    ws, ws_bytes = _workspace(p, OP_BWD, workspace, q.device)
    _check(lib.linsimp_bwd_padded(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(r), _ptr(u), _ptr(omega),
                                  _ptr(_lens(seq_lens, B)), _ptr(o), _ptr(L), _ptr(lse), _ptr(dO),
                                  *[_ptr(g) for g in grads], _ptr(ws), ws_bytes, _stream(stream)))
    return tuple(grads)


def ring_fill_padded(r, u, seq_lens, W=64, stream=None):
    """linsimp_ring_fill_padded.  Returns (ring_r, ring_u) [B,H,W,d] built from each sequence's own last rows."""
    lib = load_library()
    _dev(r, u)
    B, H, T, d = r.shape
    p = make_params(B, H, T, d, 1, W, _io_dtype(r))
    ring_r = torch.zeros((B, H, W, d), dtype=r.dtype, device=r.device)
    ring_u = torch.zeros((B, H, W, d), dtype=r.dtype, device=r.device)
    _check(lib.linsimp_ring_fill_padded(ctypes.byref(p), _ptr(r), _ptr(u), _ptr(_lens(seq_lens, B)), _ptr(ring_r),
                                        _ptr(ring_u), _stream(stream)))
    return ring_r, ring_u


def winsimp_fwd(q, k, v, r, u, w1=512, w2=32, return_lse=False, out=None, stream=None):
    """linsimp_winsimp_fwd: exact windowed 2-simplicial attention (joint softmax over w1 keys x w2 anchors), bf16."""
    lib = load_library()
    _dev(q, k, v, r, u)
    B, H, T, d = q.shape
    p = make_params(B, H, T, d, 64, w2, _io_dtype(q))
    o = torch.empty_like(q) if out is None else out
    lse = torch.empty((B, H, T), dtype=torch.float32, device=q.device) if return_lse else None
    _check(lib.linsimp_winsimp_fwd(ctypes.byref(p), int(w1), _ptr(q), _ptr(k), _ptr(v), _ptr(r), _ptr(u), _ptr(o), _ptr(lse),
                                   _stream(stream)))
    return (o, lse) if return_lse else o


def _cu(cu_seqlens):
    if cu_seqlens.dtype != torch.int32 or cu_seqlens.dim() != 1 or cu_seqlens.numel() < 2:
        raise LinSimpError("cu_seqlens must be an int32 tensor [B + 1]")
    _dev(cu_seqlens)
    return cu_seqlens


def fwd_packed(q, k, v, r, u, omega, cu_seqlens, max_len, W=64, eps=1e-30, return_state=False, workspace=None, stream=None):
    """linsimp_fwd_packed: q..u [H, total_tokens, d] bf16, sequence b in rows cu_seqlens[b]:cu_seqlens[b+1] of every head;
    max_len: an upper bound on the longest sequence.  Returns (o, rowmax_L, lse) in the packed layout (rows outside
    every sequence are left untouched) and, with return_state, also per-sequence (S_final, z_final)."""
    lib = load_library()
    _dev(q, k, v, r, u, omega)
    H, total, d = q.shape
    B = cu_seqlens.numel() - 1
    m = omega.shape[-1]
    p = make_params(B, H, max(1, int(max_len)), d, m, W, _io_dtype(q), omega.dim() == 3, ALGO_DEFAULT, eps)
    o = torch.zeros_like(q)
    L = torch.zeros((H, total), dtype=torch.float32, device=q.device)
    lse = torch.zeros((H, total), dtype=torch.float32, device=q.device)
    S = z = None
    if return_state:
        S = torch.empty((B, H, m, d), dtype=torch.float32, device=q.device)
        z = torch.empty((B, H, m), dtype=torch.float32, device=q.device)
    ws, ws_bytes = _workspace(p, OP_FWD_PACKED, workspace, q.device)
    _check(lib.linsimp_fwd_packed(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(r), _ptr(u), _ptr(omega),
                                  _ptr(_cu(cu_seqlens)), total, _ptr(o), _ptr(L), _ptr(lse), _ptr(S), _ptr(z), _ptr(ws),
                                  ws_bytes, _stream(stream)))
    if return_state:
        return o, L, lse, S, z
    return o, L, lse


def bwd_packed(q, k, v, r, u, omega, cu_seqlens, max_len, L, lse, dO, W=64, eps=1e-30, workspace=None, stream=None):
    """linsimp_bwd_packed.  Returns dq, dk, dv, dr, du in the packed layout (rows outside every sequence are zero)."""
    lib = load_library()
    _dev(q, k, v, r, u, omega, L, lse, dO)
    H, total, d = q.shape
    B = cu_seqlens.numel() - 1
    m = omega.shape[-1]
    p = make_params(B, H, max(1, int(max_len)), d, m, W, _io_dtype(q), omega.dim() == 3, ALGO_DEFAULT, eps)
    grads = [torch.zeros_like(q) for _ in range(5)]
    ws, ws_bytes = _workspace(p, OP_BWD_PACKED, workspace, q.device)
    _check(lib.linsimp_bwd_packed(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(r), _ptr(u), _ptr(omega),
                                  _ptr(_cu(cu_seqlens)), total, _ptr(L), _ptr(lse), _ptr(dO), *[_ptr(g) for g in grads],
                                  _ptr(ws), ws_bytes, _stream(stream)))
    return tuple(grads)


def ring_fill_packed(r, u, cu_seqlens, W=64, stream=None):
    """linsimp_ring_fill_packed: decode rings [B,H,W,d] (zero-initialised) from a packed batch."""
    lib = load_library()
    _dev(r, u)
    H, total, d = r.shape
    B = cu_seqlens.numel() - 1
    p = make_params(B, H, 1, d, 64, W, _io_dtype(r))
    ring_r = torch.zeros((B, H, W, d), dtype=r.dtype, device=r.device)
    ring_u = torch.zeros_like(ring_r)
    _check(lib.linsimp_ring_fill_packed(ctypes.byref(p), _ptr(r), _ptr(u), _ptr(_cu(cu_seqlens)), total, _ptr(ring_r),
                                        _ptr(ring_u), _stream(stream)))
    return ring_r, ring_u


def _norm_params(x):
    B, H, T, d = x.shape
    return make_params(B, H, T, d, 1, 1, _io_dtype(x))


def qkr_normalize(q, k, r, tau, out=None, stream=None):
    """linsimp_qkr_normalize: (tau_h q/|q|, k/|k|, r/|r|) for q, k, r [B,H,T,d]; tau fp32 [H]."""
    lib = load_library()
    _dev(q, k, r, tau)
    p = _norm_params(q)
    qh, kh, rh = (torch.empty_like(q), torch.empty_like(k), torch.empty_like(r)) if out is None else out
    _check(lib.linsimp_qkr_normalize(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(r), _ptr(tau), _ptr(qh), _ptr(kh), _ptr(rh),
                                     _stream(stream)))
    return qh, kh, rh


def qkr_normalize_bwd(q, k, r, tau, dqh, dkh, drh, workspace=None, stream=None):
    """linsimp_qkr_normalize_bwd.  Returns dq, dk, dr (like the inputs) and dtau fp32 [H]."""
    lib = load_library()
    _dev(q, k, r, tau, dqh, dkh, drh)
    p = _norm_params(q)
    dq, dk, dr = torch.empty_like(q), torch.empty_like(k), torch.empty_like(r)
    dtau = torch.empty_like(tau)
    ws, ws_bytes = _workspace(p, OP_NORM, workspace, q.device)
    _check(lib.linsimp_qkr_normalize_bwd(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(r), _ptr(tau), _ptr(dqh), _ptr(dkh),
                                         _ptr(drh), _ptr(dq), _ptr(dk), _ptr(dr), _ptr(dtau), _ptr(ws), ws_bytes,
                                         _stream(stream)))
    return dq, dk, dr, dtau


def gate_rmsnorm(o, gamma, rms_eps=1e-6, out=None, stream=None):
    """linsimp_gate_rmsnorm: y = sigmoid(gamma_h) RMSNorm(o) for o [B,H,T,d]; gamma fp32 [H]."""
    lib = load_library()
    _dev(o, gamma)
    p = _norm_params(o)
    y = torch.empty_like(o) if out is None else out
    _check(lib.linsimp_gate_rmsnorm(ctypes.byref(p), _ptr(o), _ptr(gamma), ctypes.c_float(rms_eps), _ptr(y),
                                    _stream(stream)))
    return y


def gate_rmsnorm_bwd(o, gamma, dy, rms_eps=1e-6, workspace=None, stream=None):
    """linsimp_gate_rmsnorm_bwd.  Returns d_o (like o) and dgamma fp32 [H]."""
    lib = load_library()
    _dev(o, gamma, dy)
    p = _norm_params(o)
    d_o = torch.empty_like(o)
    dgamma = torch.empty_like(gamma)
    ws, ws_bytes = _workspace(p, OP_NORM, workspace, o.device)
    _check(lib.linsimp_gate_rmsnorm_bwd(ctypes.byref(p), _ptr(o), _ptr(gamma), ctypes.c_float(rms_eps), _ptr(dy),
                                        _ptr(d_o), _ptr(dgamma), _ptr(ws), ws_bytes, _stream(stream)))
    return d_o, dgamma


def decode_prepare(n_seq, H, d, omega, W=64, dtype=None, algo=ALGO_DEFAULT, stream=None):
    """linsimp_decode_prepare.  Returns the workspace tensor to pass to decode_step(..., workspace=ws,
    omega_image=True): the image of omega the decode kernel copies instead of converting omega in every step."""
    lib = load_library()
    _dev(omega)
    m = omega.shape[-1]
    p = make_params(n_seq, H, 0, d, m, W, BF16 if dtype is None else dtype, omega.dim() == 3, algo, 1e-30)
    need = workspace_bytes(p, OP_DECODE)
    ws = torch.empty(max(need, 256), dtype=torch.uint8, device=omega.device)
    _check(lib.linsimp_decode_prepare(ctypes.byref(p), _ptr(omega), _ptr(ws), ws.numel(), _stream(stream)))
    return ws


def decode_step(q_t, k_t, v_t, r_t, u_t, omega, S, z, ring_r, ring_u, pos, W=64, eps=1e-30,
                algo=ALGO_DEFAULT, out=None, workspace=None, stream=None, omega_image=False):
    """linsimp_decode_step.  Updates S, z, ring_r, ring_u in place; returns o_t [B,H,d].
    omega_image: `workspace` is what decode_prepare returned for this omega."""
    lib = load_library()
    _dev(q_t, k_t, v_t, r_t, u_t, omega, S, z, ring_r, ring_u, pos)
    B, H, d = q_t.shape
    m = omega.shape[-1]
    if pos.dtype != torch.int32:
        raise LinSimpError("pos must be int32")
    if omega_image and workspace is None:
        raise ValueError("omega_image needs the workspace decode_prepare returned")
    p = make_params(B, H, 0, d, m, W, _io_dtype(q_t), omega.dim() == 3, algo, eps,
                    FLAG_OMEGA_IMAGE if omega_image else 0)
    o = torch.empty_like(q_t) if out is None else out
    ws, ws_bytes = _workspace(p, OP_DECODE, workspace, q_t.device)
    _check(lib.linsimp_decode_step(ctypes.byref(p), _ptr(q_t), _ptr(k_t), _ptr(v_t), _ptr(r_t), _ptr(u_t),
                                   _ptr(omega), _ptr(S), _ptr(z), _ptr(ring_r), _ptr(ring_u), _ptr(pos),
                                   _ptr(o), _ptr(ws), ws_bytes, _stream(stream)))
    return o


def prefill_state(k, v, omega, W=64, algo=ALGO_DEFAULT, workspace=None, stream=None):
    """linsimp_prefill_state.  k, v [B,H,T,d]; returns S [B,H,m,d], z [B,H,m] (fp32)."""
    lib = load_library()
    _dev(k, v, omega)
    B, H, T, d = k.shape
    m = omega.shape[-1]
    p = make_params(B, H, T, d, m, W, _io_dtype(k), omega.dim() == 3, algo, 1e-30)
    S = torch.empty((B, H, m, d), dtype=torch.float32, device=k.device)
    z = torch.empty((B, H, m), dtype=torch.float32, device=k.device)
    ws, ws_bytes = _workspace(p, OP_STATE, workspace, k.device)
    _check(lib.linsimp_prefill_state(ctypes.byref(p), _ptr(k), _ptr(v), _ptr(omega), _ptr(S), _ptr(z),
                                     _ptr(ws), ws_bytes, _stream(stream)))
    return S, z


def profile_enable(on=True):
    """Switches per-kernel event timing on (clearing old records) or off for this thread."""
    _check(load_library().linsimp_profile_enable(1 if on else 0))


def profile_read():
    """Returns {kernel name: (total_ms, launches)} for the launches recorded since profile_enable."""
    lib = load_library()
    n = lib.linsimp_profile_read(-1, None, 0, None, None)
    if n < 0:
        _check(n)
    out = {}
    for i in range(n):
        name = ctypes.create_string_buffer(64)
        ms = ctypes.c_float(0)
        cnt = ctypes.c_int(0)
        rc = lib.linsimp_profile_read(i, name, 64, ctypes.byref(ms), ctypes.byref(cnt))
        if rc < 0:
            _check(rc)
        out[name.value.decode()] = (float(ms.value), int(cnt.value))
    return out


def read_status(workspace, stream=None):
    """linsimp_read_status: 0 when no bounded device wait gave up in the last call using `workspace`."""
    return int(load_library().linsimp_read_status(_ptr(workspace), _stream(stream)))


STATIC_SCRATCH_BYTES = 32 << 20


def fwd_static(q, k, v, r, u, omega, W=64, eps=1e-30, return_state=False, stream=None):
    """linsimp_fwd_static: the forward for callers that cannot allocate device scratch memory.

    The library keeps the scratch in a fixed 32 MiB array of its own, so this call takes no
    workspace and allocates nothing in the library (the output tensors created here are this
    binding's convenience, not the entry point's).  Raises LinSimpError (code -6) when the
    problem needs more scratch than the array holds.  Returns what `fwd` returns.
    """
    lib = load_library()
    _dev(q, k, v, r, u, omega)
    B, H, T, d = q.shape
    m = omega.shape[-1]
    p = make_params(B, H, T, d, m, W, _io_dtype(q), omega.dim() == 3, ALGO_FP32, eps)
    o = torch.empty_like(q)
    L = torch.empty((B, H, T), dtype=torch.float32, device=q.device)
    lse = torch.empty((B, H, T), dtype=torch.float32, device=q.device)
    S = z = None
    if return_state:
        S = torch.empty((B, H, m, d), dtype=torch.float32, device=q.device)
        z = torch.empty((B, H, m), dtype=torch.float32, device=q.device)
    _check(lib.linsimp_fwd_static(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(r), _ptr(u), _ptr(omega),
                                  _ptr(o), _ptr(L), _ptr(lse), _ptr(S), _ptr(z), _stream(stream)))
    if return_state:
        return o, L, lse, S, z
    return o, L, lse
