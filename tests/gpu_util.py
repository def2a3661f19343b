"""Helpers shared by the GPU parity tests: marshal numpy inputs to the device, call the
library through its C ABI binding and fetch results back."""
import numpy as np
import torch

from paper_2609_24519_b200 import binding as b

TORCH_OUT = {b.C_I32: torch.int32, b.C_I64: torch.int64, b.C_RES_I16: torch.int16, b.C_RES_I32: torch.int32}
_handle = None


def handle():
    global _handle
    if _handle is None:
        _handle = b.awe_create(0)
    return _handle


def pitch_bytes(K):
    return (K + 255) // 256 * 256 // 2


def padded_planes(packed, K):
    """n x R x ceil(K/2) packed bytes -> n x R x pitch with zero padding."""
    n, R, kb = packed.shape
    out = np.zeros((n, R, pitch_bytes(K)), dtype=np.uint8)
    out[:, :, :kb] = packed
    return out


def gpu_encode(enc, modulus, side, X_rk, dt=b.I8, layout=b.ROWMAJOR_RxK, ld_extra=0, offset=0):
    """X_rk is R x K.  Returns the plane buffer as a numpy uint8 array n x R x pitch."""
    h = handle()
    R, K = X_rk.shape
    src = X_rk if layout == b.ROWMAJOR_RxK else np.ascontiguousarray(X_rk.T)
    rows, cols = src.shape
    ld = cols + ld_extra
    buf = np.zeros(rows * ld + offset, dtype=X_rk.dtype)
    view = buf[offset:offset + rows * ld].reshape(rows, ld)
    view[:, :cols] = src
    dX = torch.from_numpy(buf).cuda()
    nbytes = b.awe_planes_bytes(enc, modulus, side, R, K)
    planes = torch.full((nbytes,), 0xAA, dtype=torch.uint8, device="cuda")
    b.awe_encode(h, enc, modulus, side, dX[offset:], dt, layout, R, K, ld, planes)
    torch.cuda.synchronize()
    assert b.awe_last_device_status(h) == (0, 0)
    n = nbytes // (R * pitch_bytes(K))
    return planes.cpu().numpy().reshape(n, R, pitch_bytes(K))


def gpu_gemm_exact(A, B, enc, out_dt, modulus=0, a_dt=b.I8, b_dt=b.I8):
    h = handle()
    M, K = A.shape
    N = B.shape[1]
    ws = torch.empty(b.awe_workspace_bytes(enc, modulus, M, N, K), dtype=torch.uint8, device="cuda")
    C = torch.full((M, N), 77, dtype=TORCH_OUT[out_dt], device="cuda")
    b.awe_gemm_exact(h, torch.from_numpy(A).cuda(), a_dt, torch.from_numpy(B).cuda(), b_dt, M, N, K, enc, modulus,
                     C, out_dt, ws)
    torch.cuda.synchronize()
    assert b.awe_last_device_status(h) == (0, 0)
    return C.cpu().numpy()


def gpu_gemm_planes(planesA, planesB, M, N, K, enc, out_dt, modulus=0, k_chunk=0, ldc=None):
    h = handle()
    ldc = N if ldc is None else ldc
    C = torch.full((M, ldc), 77, dtype=TORCH_OUT[out_dt], device="cuda")
    pa = torch.from_numpy(np.ascontiguousarray(planesA)).cuda()
    pb = torch.from_numpy(np.ascontiguousarray(planesB)).cuda()
    b.awe_gemm_planes(h, enc, modulus, pa, pb, M, N, K, C, out_dt, ldc, k_chunk)
    torch.cuda.synchronize()
    assert b.awe_last_device_status(h) == (0, 0)
    return C.cpu().numpy()


def gpu_fp4_raw(X, Y, pack):
    """X: M x K, Y: N x K matrices of S values; pack: function packing them to E2M1 bytes."""
    h = handle()
    M, K = X.shape
    N = Y.shape[0]
    px = torch.from_numpy(padded_planes(pack(X)[None], K)[0]).cuda()
    py = torch.from_numpy(padded_planes(pack(Y)[None], K)[0]).cuda()
    P = torch.full((M, N), -1.0, dtype=torch.float32, device="cuda")
    b.awe_fp4_product_raw(h, px, py, M, N, K, P, N)
    torch.cuda.synchronize()
    assert b.awe_last_device_status(h) == (0, 0)
    return P.cpu().numpy()
