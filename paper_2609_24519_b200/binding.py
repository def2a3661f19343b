"""ctypes binding of libawe_b200.so: argument marshalling only.

Every function has the name of the C entry point it calls (see include/awe.h) and raises
AweError on a non-zero status.  Device buffers are torch CUDA tensors (their data_ptr() is
passed through); host buffers are numpy arrays or CPU tensors.  There is no fallback: if the
library is missing or no CUDA device is present, the calls fail.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libawe_b200.so")

# enums of awe.h
OK = 0
ENC_INT8_AWE6, ENC_INT8_BASE13_9, ENC_INT4xINT8_AWE4, ENC_MOD_M, ENC_INT8_AWE6_ALT = 1, 2, 3, 4, 5
ENC_TERNARY_INT8_3 = 6
ENC_INT4xINT4_3 = 7
ENC_FP16SIG_AWE12 = 8
ENC_INT8_MIXED_FP8_3 = 9
ENC_FP8SIG_3 = 10
ENC_BF16SIG_8 = 11
ENC_INT8_AWE6_DERIVED = 12
I8, I4_IN_I8, T2_IN_I8, I16, I4_PACKED, I5_IN_I8, I9_IN_I16 = 0, 1, 2, 3, 4, 5, 6
C_I32, C_I64, C_RES_I16, C_RES_I32 = 0, 1, 2, 3
SIDE_A, SIDE_B = 0, 1
ROWMAJOR_RxK, ROWMAJOR_KxR = 0, 1
MAX_PRODUCTS, MAX_PLANES = 16, 8
STATIC_WORKSPACE_BYTES = 24 << 20

EXPORTS = ["awe_create", "awe_destroy", "awe_encoding_info", "awe_encoding_lut", "awe_planes_bytes",
           "awe_workspace_bytes", "awe_host_staging_bytes", "awe_encode", "awe_gemm_planes", "awe_gemm_exact",
           "awe_gemm_exact_host", "awe_gemm_exact_static", "awe_wide_moduli", "awe_wide_select", "awe_wide_workspace_bytes",
           "awe_wide_residues", "awe_wide_crt", "awe_gemm_exact_wide", "awe_reconstruct", "awe_fp4_product_raw", "awe_fp8_product_raw", "awe_last_device_status", "awe_selftest_bounded_wait", "awe_last_gemm_clock_mhz", "awe_launch_count",
           "awe_status_string"]


class EncodingDesc(ctypes.Structure):
    _fields_ = [("r", ctypes.c_int32), ("n_planes_a", ctypes.c_int32), ("n_planes_b", ctypes.c_int32),
                ("ia", ctypes.c_int32 * MAX_PRODUCTS), ("ib", ctypes.c_int32 * MAX_PRODUCTS),
                ("ell", ctypes.c_int32 * MAX_PRODUCTS), ("log2D", ctypes.c_int32), ("modulus", ctypes.c_int32),
                ("c_a", ctypes.c_int32), ("c_b", ctypes.c_int32), ("k_star", ctypes.c_int64),
                ("a_lo", ctypes.c_int32), ("a_hi", ctypes.c_int32), ("b_lo", ctypes.c_int32),
                ("b_hi", ctypes.c_int32), ("plane_bits_a", ctypes.c_int32 * MAX_PLANES),
                ("plane_bits_b", ctypes.c_int32 * MAX_PLANES), ("fp8", ctypes.c_int32 * MAX_PRODUCTS),
                ("ia2", ctypes.c_int32 * MAX_PRODUCTS), ("ib2", ctypes.c_int32 * MAX_PRODUCTS)]


class AweError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


_lib = None


def lib() -> ctypes.CDLL:
    """Load the CUDA library (built in-tree by paper_2609_24519_b200.build)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(f"{LIB_PATH} is missing: run `python -m paper_2609_24519_b200.build`")
    L = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_size_t
    L.awe_create.argtypes = [ctypes.POINTER(vp), i32]
    L.awe_destroy.argtypes = [vp]
    L.awe_encoding_info.argtypes = [i32, i32, ctypes.POINTER(EncodingDesc)]
    L.awe_encoding_lut.argtypes = [i32, i32, i32, i32, vp]
    L.awe_planes_bytes.argtypes = [i32, i32, i32, i64, i64]
    L.awe_planes_bytes.restype = sz
    L.awe_workspace_bytes.argtypes = [i32, i32, i64, i64, i64]
    L.awe_workspace_bytes.restype = sz
    L.awe_host_staging_bytes.argtypes = [i32, i32, i64, i64, i64, i32]
    L.awe_host_staging_bytes.restype = sz
    L.awe_encode.argtypes = [vp, i32, i32, i32, vp, i32, i32, i64, i64, i64, vp, vp]
    L.awe_gemm_planes.argtypes = [vp, i32, i32, vp, vp, i64, i64, i64, vp, i32, i64, i64, vp]
    L.awe_gemm_exact.argtypes = [vp, vp, i32, vp, i32, i64, i64, i64, i32, i32, vp, i32, vp, sz, vp]
    L.awe_gemm_exact_host.argtypes = [vp, vp, i32, vp, i32, i64, i64, i64, i32, i32, vp, i32, vp, sz, vp]
    L.awe_gemm_exact_static.argtypes = [vp, i32, vp, i32, i64, i64, i64, i32, i32, vp, i32, vp]
    L.awe_wide_moduli.argtypes = [vp, i32]
    L.awe_wide_select.argtypes = [i32, i64, vp, i32]
    L.awe_wide_workspace_bytes.argtypes = [i64, i64, i64]
    L.awe_wide_workspace_bytes.restype = sz
    L.awe_wide_residues.argtypes = [vp, vp, i64, vp, vp]
    L.awe_wide_crt.argtypes = [vp, vp, i64, vp, vp]
    L.awe_gemm_exact_wide.argtypes = [vp, vp, vp, i64, i64, i64, i32, vp, vp, sz, vp]
    L.awe_reconstruct.argtypes = [vp, i32, i32, vp, i64, i64, i64, i64, vp, i32, i64, vp]
    L.awe_fp4_product_raw.argtypes = [vp, vp, vp, i64, i64, i64, vp, i64, vp]
    L.awe_fp8_product_raw.argtypes = [vp, vp, vp, i64, i64, i64, vp, i64, vp]
    L.awe_last_device_status.argtypes = [vp, vp, ctypes.POINTER(i32)]
    L.awe_selftest_bounded_wait.argtypes = [vp, i64, vp]
    L.awe_last_gemm_clock_mhz.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_double)]
    L.awe_launch_count.argtypes = [vp]
    L.awe_launch_count.restype = i64
    L.awe_status_string.argtypes = [i32]
    L.awe_status_string.restype = ctypes.c_char_p
    for name in EXPORTS:
        if getattr(L, name).restype is ctypes.c_int:
            getattr(L, name).restype = ctypes.c_int
    _lib = L
    return L


def status_string(status: int) -> str:
    return lib().awe_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != OK:
        raise AweError(status, where)


def _ptr(x) -> int:
    """Address of a torch tensor (device or host) or a numpy array."""
    if x is None:
        return 0
    if isinstance(x, np.ndarray):
        return x.ctypes.data
    return x.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return int(getattr(stream, "cuda_stream", stream))


# ------------------------------------------------------------------ host-only queries
def awe_encoding_info(enc: int, modulus: int = 0) -> EncodingDesc:
    d = EncodingDesc()
    _check(lib().awe_encoding_info(enc, modulus, ctypes.byref(d)), "awe_encoding_info")
    return d


def awe_encoding_lut(enc: int, modulus: int, side: int, dt: int = I8) -> np.ndarray:
    n = awe_encoding_info(enc, modulus)
    n_planes = n.n_planes_a if side == SIDE_A else n.n_planes_b
    out = np.zeros((4096 if dt in (I16, I9_IN_I16) else 256, n_planes), dtype=np.int8)
    _check(lib().awe_encoding_lut(enc, modulus, side, dt, out.ctypes.data), "awe_encoding_lut")
    return out


def awe_planes_bytes(enc: int, modulus: int, side: int, R: int, K: int) -> int:
    return int(lib().awe_planes_bytes(enc, modulus, side, R, K))


def awe_workspace_bytes(enc: int, modulus: int, M: int, N: int, K: int) -> int:
    return int(lib().awe_workspace_bytes(enc, modulus, M, N, K))


def awe_host_staging_bytes(enc: int, modulus: int, M: int, N: int, K: int, out_dt: int) -> int:
    return int(lib().awe_host_staging_bytes(enc, modulus, M, N, K, out_dt))


# ------------------------------------------------------------------ device calls
class Handle:
    """Owns one awe_handle_t (awe_create / awe_destroy)."""

    def __init__(self, device: int = 0):
        self._h = ctypes.c_void_p()
        _check(lib().awe_create(ctypes.byref(self._h), device), "awe_create")

    @property
    def raw(self):
        return self._h

    def close(self):
        if self._h:
            lib().awe_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def awe_create(device: int = 0) -> Handle:
    return Handle(device)


def awe_destroy(h: Handle) -> None:
    h.close()


def awe_encode(h: Handle, enc: int, modulus: int, side: int, X, dt: int, layout: int, R: int, K: int, ld: int,
               planes, stream=None) -> None:
    _check(lib().awe_encode(h.raw, enc, modulus, side, _ptr(X), dt, layout, R, K, ld, _ptr(planes),
                            _stream(stream)), "awe_encode")


def awe_gemm_planes(h: Handle, enc: int, modulus: int, planesA, planesB, M: int, N: int, K: int, C, out_dt: int,
                    ldc: int, k_chunk: int = 0, stream=None) -> None:
    _check(lib().awe_gemm_planes(h.raw, enc, modulus, _ptr(planesA), _ptr(planesB), M, N, K, _ptr(C), out_dt, ldc,
                                 k_chunk, _stream(stream)), "awe_gemm_planes")


def awe_gemm_exact(h: Handle, A, a_dt: int, B, b_dt: int, M: int, N: int, K: int, enc: int, modulus: int, C,
                   out_dt: int, workspace, workspace_bytes: Optional[int] = None, stream=None) -> None:
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    _check(lib().awe_gemm_exact(h.raw, _ptr(A), a_dt, _ptr(B), b_dt, M, N, K, enc, modulus, _ptr(C), out_dt,
                                _ptr(workspace), workspace_bytes, _stream(stream)), "awe_gemm_exact")


def awe_gemm_exact_host(h: Handle, A_host, a_dt: int, B_host, b_dt: int, M: int, N: int, K: int, enc: int,
                        modulus: int, C_host, out_dt: int, scratch, scratch_bytes: Optional[int] = None,
                        stream=None) -> None:
    if scratch_bytes is None:
        scratch_bytes = scratch.numel() * scratch.element_size()
    _check(lib().awe_gemm_exact_host(h.raw, _ptr(A_host), a_dt, _ptr(B_host), b_dt, M, N, K, enc, modulus,
                                     _ptr(C_host), out_dt, _ptr(scratch), scratch_bytes, _stream(stream)),
           "awe_gemm_exact_host")


def awe_gemm_exact_static(A, a_dt: int, B, b_dt: int, M: int, N: int, K: int, enc: int, modulus: int, C,
                          out_dt: int, stream=None) -> None:
    """awe_gemm_exact for callers that must not allocate: no handle, no workspace argument; the
    library's built-in device array (at most STATIC_WORKSPACE_BYTES of planes) is the scratch.
    Runs on the current CUDA device; calls that could overlap on the GPU must be serialised."""
    _check(lib().awe_gemm_exact_static(_ptr(A), a_dt, _ptr(B), b_dt, M, N, K, enc, modulus, _ptr(C), out_dt,
                                       _stream(stream)), "awe_gemm_exact_static")


def awe_wide_moduli():
    n = lib().awe_wide_moduli(None, 0)
    out = (ctypes.c_int32 * n)()
    lib().awe_wide_moduli(out, n)
    return list(out)


def awe_wide_select(in_bits: int, K: int):
    n = lib().awe_wide_select(in_bits, K, None, 0)
    out = (ctypes.c_int32 * max(n, 1))()
    lib().awe_wide_select(in_bits, K, out, n)
    return list(out)[:n]


def awe_wide_workspace_bytes(M: int, N: int, K: int) -> int:
    return int(lib().awe_wide_workspace_bytes(M, N, K))


def awe_wide_residues(h: Handle, X, count: int, res, stream=None) -> None:
    _check(lib().awe_wide_residues(h.raw, _ptr(X), count, _ptr(res), _stream(stream)), "awe_wide_residues")


def awe_wide_crt(h: Handle, res, count: int, out, stream=None) -> None:
    _check(lib().awe_wide_crt(h.raw, _ptr(res), count, _ptr(out), _stream(stream)), "awe_wide_crt")


def awe_gemm_exact_wide(h: Handle, A, B, M: int, N: int, K: int, in_bits: int, C, workspace,
                        workspace_bytes: Optional[int] = None, stream=None) -> None:
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    _check(lib().awe_gemm_exact_wide(h.raw, _ptr(A), _ptr(B), M, N, K, in_bits, _ptr(C), _ptr(workspace),
                                     workspace_bytes, _stream(stream)), "awe_gemm_exact_wide")


def awe_fp4_product_raw(h: Handle, planeX, planeY, M: int, N: int, K: int, P, ldp: int, stream=None) -> None:
    _check(lib().awe_fp4_product_raw(h.raw, _ptr(planeX), _ptr(planeY), M, N, K, _ptr(P), ldp, _stream(stream)),
           "awe_fp4_product_raw")


def awe_fp8_product_raw(h: Handle, planeX, planeY, M: int, N: int, K: int, P, ldp: int, stream=None) -> None:
    _check(lib().awe_fp8_product_raw(h.raw, _ptr(planeX), _ptr(planeY), M, N, K, _ptr(P), ldp, _stream(stream)),
           "awe_fp8_product_raw")


def awe_reconstruct(h: Handle, enc: int, modulus: int, P, plane_stride: int, ldp: int, M: int, N: int, C,
                    out_dt: int, ldc: int, stream=None) -> None:
    _check(lib().awe_reconstruct(h.raw, enc, modulus, _ptr(P), plane_stride, ldp, M, N, _ptr(C), out_dt, ldc,
                                 _stream(stream)), "awe_reconstruct")


def awe_last_device_status(h: Handle, stream=None):
    site = ctypes.c_int(0)
    st = lib().awe_last_device_status(h.raw, _stream(stream), ctypes.byref(site))
    return int(st), int(site.value)


def awe_selftest_bounded_wait(h: Handle, limit_us: int = 1000, stream=None) -> None:
    _check(lib().awe_selftest_bounded_wait(h.raw, limit_us, _stream(stream)), "awe_selftest_bounded_wait")


def awe_last_gemm_clock_mhz(h: Handle, stream=None) -> float:
    mhz = ctypes.c_double(0.0)
    _check(lib().awe_last_gemm_clock_mhz(h.raw, _stream(stream), ctypes.byref(mhz)), "awe_last_gemm_clock_mhz")
    return float(mhz.value)


def awe_launch_count(h: Handle) -> int:
    return int(lib().awe_launch_count(h.raw))
