"""Packed 4-bit operands (two values per byte, low nibble first): the encode kernels must produce the
same planes as for the one-value-per-byte container, and the products must match the oracle."""
import numpy as np
import pytest
import torch

from oracle import matmul as mm
from oracle import pipeline as pl
from oracle import schemes as sc
from paper_2609_24519_b200 import binding as b
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def pack_nibbles(X):
    """Row-major int array with values in [-8, 7] and an even number of columns -> uint8 array with
    half as many columns, element 2j in the low nibble of byte j."""
    u = (np.asarray(X).astype(np.int16) & 0xF).astype(np.uint8)
    return (u[:, 0::2] | (u[:, 1::2] << 4)).astype(np.uint8)


def _encode_packed(enc, side, X_rk, layout, ld_extra=0, offset_bytes=0):
    h = gu.handle()
    R, K = X_rk.shape
    src = X_rk if layout == b.ROWMAJOR_RxK else np.ascontiguousarray(X_rk.T)
    rows, cols = src.shape
    ld = cols + ld_extra
    full = np.zeros((rows, ld), dtype=np.int8)
    full[:, :cols] = src
    packed = pack_nibbles(full).reshape(-1)
    buf = np.concatenate([np.zeros(offset_bytes, np.uint8), packed])
    dX = torch.from_numpy(buf).cuda()
    nbytes = b.awe_planes_bytes(enc, 0, side, R, K)
    planes = torch.full((nbytes,), 0xAA, dtype=torch.uint8, device="cuda")
    b.awe_encode(h, enc, 0, side, dX[offset_bytes:], b.I4_PACKED, layout, R, K, ld, planes)
    torch.cuda.synchronize()
    assert b.awe_last_device_status(h) == (0, 0)
    return planes.cpu().numpy().reshape(-1, R, gu.pitch_bytes(K))


def _want(s, sname, X):
    ref = pl.encode_planes(s, sname, X, -8, 7)
    return gu.padded_planes(np.stack([pl.pack_e2m1(p) for p in ref]), X.shape[1])


@pytest.mark.parametrize("shape", [(2, 2), (200, 300), (256, 2048), (132, 1026), (520, 4100)])
def test_packed_encode_matches_oracle_planes(shape):
    R, K = shape
    X = np.random.default_rng(R + K).integers(-8, 8, (R, K), dtype=np.int8)
    for enc, s, side, sname in ((b.ENC_INT4xINT8_AWE4, sc.AWE4, b.SIDE_A, "A"),
                                (b.ENC_INT4xINT4_3, sc.INT4X4_3, b.SIDE_A, "A"),
                                (b.ENC_INT4xINT4_3, sc.INT4X4_3, b.SIDE_B, "B")):
        want = _want(s, sname, X)
        for layout in (b.ROWMAJOR_RxK, b.ROWMAJOR_KxR):
            got = _encode_packed(enc, side, X, layout)
            assert np.array_equal(got, want), (enc, sname, layout)


def test_packed_encode_odd_alignments_and_padded_ld():
    X = np.random.default_rng(3).integers(-8, 8, (70, 334), dtype=np.int8)
    want = _want(sc.AWE4, "A", X)
    for layout in (b.ROWMAJOR_RxK, b.ROWMAJOR_KxR):
        for ld_extra, off in ((0, 0), (0, 1), (2, 0), (6, 3), (30, 16)):
            got = _encode_packed(b.ENC_INT4xINT8_AWE4, b.SIDE_A, X, layout, ld_extra, off)
            assert np.array_equal(got, want), (layout, ld_extra, off)


def test_odd_leading_dimension_is_rejected():
    h = gu.handle()
    X = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    planes = torch.empty(b.awe_planes_bytes(b.ENC_INT4xINT8_AWE4, 0, b.SIDE_A, 8, 33), dtype=torch.uint8, device="cuda")
    with pytest.raises(b.AweError) as e:
        b.awe_encode(h, b.ENC_INT4xINT8_AWE4, 0, b.SIDE_A, X, b.I4_PACKED, b.ROWMAJOR_RxK, 8, 33, 33, planes)
    assert e.value.status == 1
    # an int8-only side has no 4-bit table
    with pytest.raises(b.AweError) as e:
        b.awe_encode(h, b.ENC_INT8_AWE6, 0, b.SIDE_A, X, b.I4_PACKED, b.ROWMAJOR_RxK, 8, 32, 32, planes)
    assert e.value.status == 2


@pytest.mark.parametrize("shape", [(256, 256, 256), (300, 270, 1000), (1024, 768, 4096)])
def test_int4_x_int8_product_with_packed_a(shape):
    M, N, K = shape
    rng = np.random.default_rng(M + N + K)
    A = rng.integers(-8, 8, (M, K), dtype=np.int8)
    B = rng.integers(-128, 128, (K, N), dtype=np.int8)
    h = gu.handle()
    enc = b.ENC_INT4xINT8_AWE4
    ws = torch.empty(b.awe_workspace_bytes(enc, 0, M, N, K), dtype=torch.uint8, device="cuda")
    C = torch.full((M, N), 77, dtype=torch.int32, device="cuda")
    b.awe_gemm_exact(h, torch.from_numpy(pack_nibbles(A)).cuda(), b.I4_PACKED, torch.from_numpy(B).cuda(), b.I8,
                     M, N, K, enc, 0, C, b.C_I32, ws)
    torch.cuda.synchronize()
    assert b.awe_last_device_status(h) == (0, 0)
    assert np.array_equal(C.cpu().numpy().astype(np.int64), mm.matmul_i64(A, B))


def test_int4_x_int4_product_with_both_operands_packed_from_host_buffers():
    M, N, K = 2048, 512, 1024
    rng = np.random.default_rng(21)
    A = rng.integers(-8, 8, (M, K), dtype=np.int8)
    B = rng.integers(-8, 8, (K, N), dtype=np.int8)
    h = gu.handle()
    enc = b.ENC_INT4xINT4_3
    Ah = torch.from_numpy(pack_nibbles(A)).pin_memory()
    Bh = torch.from_numpy(pack_nibbles(B)).pin_memory()
    Ch = torch.empty((M, N), dtype=torch.int32).pin_memory()
    scratch = torch.empty(b.awe_workspace_bytes(enc, 0, M, N, K) + b.awe_host_staging_bytes(enc, 0, M, N, K, b.C_I32),
                          dtype=torch.uint8, device="cuda")
    b.awe_gemm_exact_host(h, Ah, b.I4_PACKED, Bh, b.I4_PACKED, M, N, K, enc, 0, Ch, b.C_I32, scratch)
    assert b.awe_last_device_status(h) == (0, 0)
    assert np.array_equal(Ch.numpy().astype(np.int64), mm.matmul_i64(A, B))
