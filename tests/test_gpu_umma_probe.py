"""Pins the tcgen05 descriptor encodings and swizzled operand layouts the tensor-core kernels
rely on: one UMMA accumulation chain on caller-built operand images, checked against a matmul."""
import ctypes

import numpy as np
import pytest
import torch

import paper_2608_09307_b200 as P

pytestmark = pytest.mark.gpu

SW = {128: 2, 64: 4, 32: 6}


class Probe(ctypes.Structure):
    _fields_ = [("idesc", ctypes.c_uint32),
                ("a_lbo", ctypes.c_uint32), ("a_sbo", ctypes.c_uint32), ("a_layout", ctypes.c_uint32),
                ("b_lbo", ctypes.c_uint32), ("b_sbo", ctypes.c_uint32), ("b_layout", ctypes.c_uint32),
                ("nk", ctypes.c_int), ("a_koff", ctypes.c_int * 16), ("b_koff", ctypes.c_int * 16),
                ("a_bytes", ctypes.c_int), ("b_bytes", ctypes.c_int), ("n_out", ctypes.c_int),
                ("a_from_tmem", ctypes.c_int)]


def idesc(M, N, fmt, a_mn, b_mn):
    return (1 << 4) | (fmt << 7) | (fmt << 10) | (a_mn << 15) | (b_mn << 16) | ((N >> 3) << 17) | ((M >> 4) << 24)


def kmajor_image(x, rowb):
    """x: [rows, cols] int16 view of 16-bit data.  Blocks of rowb/2 columns, each block a
    [rows][rowb bytes] tile with the rowb-byte swizzle; blocks follow each other."""
    rows, cols = x.shape
    per = rowb // 2
    nblk = cols // per
    nch = rowb // 16
    sh = {128: 0, 64: 1, 32: 2}[rowb]
    img = np.zeros((nblk, rows, nch, 8), dtype=np.int16)
    r = np.arange(rows)
    for b in range(nblk):
        blk = x[:, b * per:(b + 1) * per].reshape(rows, nch, 8)
        for c in range(nch):
            img[b, r, c ^ ((r >> sh) & (nch - 1))] = blk[:, c]
    return img.reshape(-1)


def run(a_img, b_img, pr, n_out):
    lib = P.load_library()
    a = torch.from_numpy(a_img.copy()).cuda()
    b = torch.from_numpy(b_img.copy()).cuda()
    out = torch.zeros(128, n_out, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    pr.a_bytes = a_img.nbytes
    pr.b_bytes = b_img.nbytes
    pr.n_out = n_out
    rc = lib.linsimp_debug_umma(ctypes.c_void_p(a.data_ptr()), ctypes.c_void_p(b.data_ptr()), ctypes.byref(pr),
                                ctypes.c_void_p(out.data_ptr()), ctypes.c_void_p(status.data_ptr()), None)
    assert rc == 0
    torch.cuda.synchronize()
    assert int(status.item()) == 0, "bounded wait gave up"
    return out.cpu().numpy()


def mats(M, N, K, dtype, seed):
    g = torch.Generator().manual_seed(seed)
    A = torch.randn(M, K, generator=g).to(dtype)
    B = torch.randn(N, K, generator=g).to(dtype)
    ref = A.double() @ B.double().T
    return A, B, ref.numpy()


def i16(t):
    return t.view(torch.int16).numpy()


@pytest.mark.parametrize("dtype,fmt", [(torch.float16, 0), (torch.bfloat16, 1)])
@pytest.mark.parametrize("N,K", [(128, 128), (16, 128), (256, 64), (64, 256)])
def test_kmajor_sw128(dtype, fmt, N, K):
    A, B, ref = mats(128, N, K, dtype, 1)
    pr = Probe()
    pr.idesc = idesc(128, N, fmt, 0, 0)
    pr.a_lbo, pr.a_sbo, pr.a_layout = 0, 1024, SW[128]
    pr.b_lbo, pr.b_sbo, pr.b_layout = 0, 1024, SW[128]
    pr.nk = K // 16
    for k in range(pr.nk):
        pr.a_koff[k] = (k // 4) * 128 * 128 + (k % 4) * 32
        pr.b_koff[k] = (k // 4) * N * 128 + (k % 4) * 32
    out = run(kmajor_image(i16(A), 128), kmajor_image(i16(B), 128), pr, N)
    assert np.abs(out - ref).max() < 2e-2 * np.abs(ref).max()


@pytest.mark.parametrize("rowb", [32, 64])
def test_kmajor_narrow_swizzle(rowb):
    # K extent of one row = rowb/2 elements (16 or 32): the intra-chunk tiles
    K = rowb // 2
    A, B, ref = mats(128, 128, K, torch.bfloat16, 2)
    pr = Probe()
    pr.idesc = idesc(128, 128, 1, 0, 0)
    pr.a_lbo, pr.a_sbo, pr.a_layout = 0, 8 * rowb, SW[rowb]
    pr.b_lbo, pr.b_sbo, pr.b_layout = 0, 8 * rowb, SW[rowb]
    pr.nk = K // 16
    for k in range(pr.nk):
        pr.a_koff[k] = k * 32
        pr.b_koff[k] = k * 32
    out = run(kmajor_image(i16(A), rowb), kmajor_image(i16(B), rowb), pr, 128)
    assert np.abs(out - ref).max() < 2e-2 * np.abs(ref).max()


def test_mnmajor_sw128_both():
    # D[M,N] = sum_k At[k,M] Bt[k,N] with both operands stored K-row / MN-contiguous
    M, N, K = 128, 128, 128
    A, B, ref = mats(M, N, K, torch.bfloat16, 3)
    pr = Probe()
    pr.idesc = idesc(M, N, 1, 1, 1)
    pr.a_lbo, pr.a_sbo, pr.a_layout = K * 128, 1024, SW[128]     # LBO: next 64-wide MN block
    pr.b_lbo, pr.b_sbo, pr.b_layout = K * 128, 1024, SW[128]
    pr.nk = K // 16
    for k in range(pr.nk):
        pr.a_koff[k] = k * 16 * 128
        pr.b_koff[k] = k * 16 * 128
    out = run(kmajor_image(i16(A.T.contiguous()), 128), kmajor_image(i16(B.T.contiguous()), 128), pr, N)
    assert np.abs(out - ref).max() < 2e-2 * np.abs(ref).max()


def test_mnmajor_b_n16_sw32():
    M, N, K = 128, 16, 128
    A, B, ref = mats(M, N, K, torch.bfloat16, 4)
    pr = Probe()
    pr.idesc = idesc(M, N, 1, 1, 1)
    pr.a_lbo, pr.a_sbo, pr.a_layout = K * 128, 1024, SW[128]
    pr.b_lbo, pr.b_sbo, pr.b_layout = 0, 256, SW[32]
    pr.nk = K // 16
    for k in range(pr.nk):
        pr.a_koff[k] = k * 16 * 128
        pr.b_koff[k] = k * 16 * 32
    out = run(kmajor_image(i16(A.T.contiguous()), 128), kmajor_image(i16(B.T.contiguous()), 32), pr, N)
    assert np.abs(out - ref).max() < 2e-2 * np.abs(ref).max()


def test_a_from_tmem():
    M, N, K = 128, 128, 128
    A, B, ref = mats(M, N, K, torch.bfloat16, 5)
    pr = Probe()
    pr.idesc = idesc(M, N, 1, 0, 0)
    pr.b_lbo, pr.b_sbo, pr.b_layout = 0, 1024, SW[128]
    pr.a_from_tmem = 1
    pr.nk = K // 16
    for k in range(pr.nk):
        pr.a_koff[k] = k * 8                 # 16 bf16 = 8 32-bit TMEM columns
        pr.b_koff[k] = (k // 4) * N * 128 + (k % 4) * 32
    out = run(i16(A).reshape(-1), kmajor_image(i16(B), 128), pr, N)
    assert np.abs(out - ref).max() < 2e-2 * np.abs(ref).max()


def test_unknown_descriptors_are_refused_before_launch():
    """The probe accepts only the encodings the production kernels build."""
    lib = P.load_library()
    A, B, _ = mats(128, 128, 128, torch.bfloat16, 6)
    a = torch.from_numpy(kmajor_image(i16(A), 128).copy()).cuda()
    b = torch.from_numpy(kmajor_image(i16(B), 128).copy()).cuda()
    out = torch.zeros(128, 128, device="cuda")

    def call(mutate):
        pr = Probe()
        pr.idesc = idesc(128, 128, 1, 0, 0)
        pr.a_lbo, pr.a_sbo, pr.a_layout = 0, 1024, SW[128]
        pr.b_lbo, pr.b_sbo, pr.b_layout = 0, 1024, SW[128]
        pr.nk = 8
        for k in range(8):
            pr.a_koff[k] = pr.b_koff[k] = (k // 4) * 128 * 128 + (k % 4) * 32
        pr.a_bytes, pr.b_bytes, pr.n_out = a.numel() * 2, b.numel() * 2, 128
        mutate(pr)
        return lib.linsimp_debug_umma(ctypes.c_void_p(a.data_ptr()), ctypes.c_void_p(b.data_ptr()), ctypes.byref(pr),
                                      ctypes.c_void_p(out.data_ptr()), None, None)

    assert call(lambda pr: None) == 0
    torch.cuda.synchronize()
    mixed = (1 << 4) | (0 << 7) | (1 << 10) | (16 << 17) | (8 << 24)          # fp16 A with bf16 B: no such product
    for bad in (lambda pr: setattr(pr, "idesc", mixed),
                lambda pr: setattr(pr, "idesc", idesc(64, 128, 1, 0, 0)),       # M = 64
                lambda pr: setattr(pr, "idesc", idesc(128, 128, 1, 0, 0) | (1 << 2)),   # a reserved bit
                lambda pr: setattr(pr, "idesc", idesc(128, 24, 1, 0, 0)),       # N not a multiple of 16
                lambda pr: setattr(pr, "a_layout", 1),
                lambda pr: setattr(pr, "b_sbo", 1000),
                lambda pr: pr.b_koff.__setitem__(7, pr.b_bytes)):               # a K step beyond the image
        assert call(bad) == -2
    torch.cuda.synchronize()


def test_bounded_wait_gives_up_and_reports():
    """A wait nothing ever satisfies runs out after its poll limit: the kernel returns, the status word holds the
    wait's code, and the context keeps working (a product afterwards is correct)."""
    lib = P.load_library()
    status = torch.zeros(64, dtype=torch.int32, device="cuda")     # laid out like the head of a workspace
    gave_up = torch.zeros(1, dtype=torch.int32, device="cuda")
    assert lib.linsimp_read_status(ctypes.c_void_p(status.data_ptr()), None) == 0
    rc = lib.linsimp_debug_wait_expiry(ctypes.c_void_p(status.data_ptr()), 77, 4096, ctypes.c_void_p(gave_up.data_ptr()), None)
    assert rc == 0
    assert lib.linsimp_read_status(ctypes.c_void_p(status.data_ptr()), None) == 77      # synchronises the stream
    assert int(gave_up.item()) == 1
    assert lib.linsimp_debug_wait_expiry(ctypes.c_void_p(status.data_ptr()), 0, 4096, None, None) == -1
    assert lib.linsimp_debug_wait_expiry(ctypes.c_void_p(status.data_ptr()), 5, 1 << 20, None, None) == -1
    # the device is healthy afterwards
    test_kmajor_sw128(torch.bfloat16, 1, 128, 128)
