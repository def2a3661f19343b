"""INT8 x INT8 through 2 FP8 products and 1 FP4 product (Appendix A) against the CPU oracle:
plane bytes of the encode kernels, exactness of the raw FP8 product up to 2^24 (Section 3.4), and
the fused product bit for bit."""
import numpy as np
import pytest
import torch

from oracle import matmul as mm
from oracle import mixed as mx
from oracle import pipeline as pl
from paper_2609_24519_b200 import binding as b
from paper_2609_24519_b200 import workloads as wl
from tests import gpu_util as gu
from tests.test_gpu_configs import run_three_calls, sampled_rows_match

pytestmark = pytest.mark.gpu
ENC = b.ENC_INT8_MIXED_FP8_3


def _want_planes(X):
    """Oracle planes of an R x K matrix as the library lays them out: two E4M3 planes with rows of
    2 * pitch bytes, then one E2M1 plane with rows of pitch bytes, zero padded."""
    R, K = X.shape
    pitch = gu.pitch_bytes(K)
    ref = mx.encode_planes(X)
    p8 = np.zeros((2, R, 2 * pitch), np.uint8)
    p8[:, :, :K] = np.stack([mx.pack_e4m3(ref[0]), mx.pack_e4m3(ref[1])])
    p4 = gu.padded_planes(pl.pack_e2m1(ref[2])[None], K)[0]
    return np.concatenate([p8.reshape(-1), p4.reshape(-1)])


def _gpu_planes(X, side, layout, ld_extra=0, offset=0):
    h = gu.handle()
    R, K = X.shape
    src = X if layout == b.ROWMAJOR_RxK else np.ascontiguousarray(X.T)
    rows, cols = src.shape
    ld = cols + ld_extra
    buf = np.zeros(rows * ld + offset, dtype=np.int8)
    buf[offset:offset + rows * ld].reshape(rows, ld)[:, :cols] = src
    dX = torch.from_numpy(buf).cuda()
    nbytes = b.awe_planes_bytes(ENC, 0, side, R, K)
    assert nbytes == 5 * R * gu.pitch_bytes(K)
    planes = torch.full((nbytes,), 0xAA, dtype=torch.uint8, device="cuda")
    b.awe_encode(h, ENC, 0, side, dX[offset:], b.I8, layout, R, K, ld, planes)
    torch.cuda.synchronize()
    assert b.awe_last_device_status(h) == (0, 0)
    return planes.cpu().numpy()


@pytest.mark.parametrize("shape", [(1, 1), (200, 300), (256, 2048), (131, 1025), (520, 4100)])
def test_encode_bytes_both_sides_both_layouts(shape):
    R, K = shape
    X = np.random.default_rng(R * 31 + K).integers(-128, 128, (R, K), dtype=np.int8)
    want = _want_planes(X)
    for side in (b.SIDE_A, b.SIDE_B):
        for layout in (b.ROWMAJOR_RxK, b.ROWMAJOR_KxR):
            assert np.array_equal(_gpu_planes(X, side, layout), want), (side, layout)


def test_encode_every_value_and_odd_strides():
    X = np.arange(-128, 128, dtype=np.int8).reshape(1, 256).repeat(3, 0)
    X[1] = X[1, ::-1]
    want = _want_planes(X)
    for layout in (b.ROWMAJOR_RxK, b.ROWMAJOR_KxR):
        for ld_extra, offset in ((0, 0), (0, 3), (5, 0), (7, 1)):
            assert np.array_equal(_gpu_planes(X, b.SIDE_A, layout, ld_extra, offset), want), (layout, ld_extra, offset)


def _fp8_raw(X, Y):
    h = gu.handle()
    M, K = X.shape
    N = Y.shape[0]
    p8 = 2 * gu.pitch_bytes(K)
    px = np.zeros((M, p8), np.uint8)
    py = np.zeros((N, p8), np.uint8)
    px[:, :K] = mx.pack_e4m3(X)
    py[:, :K] = mx.pack_e4m3(Y)
    P = torch.full((M, N), -1.0, dtype=torch.float32, device="cuda")
    b.awe_fp8_product_raw(h, torch.from_numpy(px).cuda(), torch.from_numpy(py).cuda(), M, N, K, P, N)
    torch.cuda.synchronize()
    assert b.awe_last_device_status(h) == (0, 0)
    return P.cpu().numpy().astype(np.int64)


@pytest.mark.parametrize("shape", [(128, 256, 128), (300, 270, 1000), (512, 512, 4096)])
def test_fp8_raw_product_random(shape):
    M, N, K = shape
    rng = np.random.default_rng(M + K)
    X, Y = rng.integers(-14, 15, (M, K)), rng.integers(-14, 15, (N, K))
    assert np.array_equal(_fp8_raw(X, Y), X @ Y.T)


def test_fp8_accumulation_is_exact_up_to_k_star():
    """Section 3.4 for E4M3 operands: partial sums that stay below 2^24 come out exactly, including
    odd totals next to the bound and small addends under a large running sum."""
    K = mx.constants()["K_star"]
    assert K == 85598
    rng = np.random.default_rng(11)
    X = np.full((128, K), 14)
    Y = np.full((256, K), 14)
    Y[1::2] = -14
    ref = X @ Y.T
    assert ref.max() == 196 * K < 2 ** 24
    assert np.array_equal(_fp8_raw(X, Y), ref)
    # large head, then +-1 / +-3 addends: totals of either parity just under the bound
    X[:, 80000:] = rng.integers(-1, 2, (128, K - 80000))
    Y[:, 80000:] = rng.integers(-3, 4, (256, K - 80000))
    ref = X @ Y.T
    assert np.abs(ref).max() < 2 ** 24 and (ref & 1).any()
    assert np.array_equal(_fp8_raw(X, Y), ref)
    # 13 x 13 with sparse 1 x 1: odd addends all along
    X = np.full((128, K), 13)
    Y = np.full((256, K), 13)
    X[:, 1::7] = 1
    Y[:, 1::7] = 1
    assert np.array_equal(_fp8_raw(X, Y), X @ Y.T)


@pytest.mark.parametrize("shape", [(1, 1, 1), (256, 256, 256), (300, 270, 1000), (1024, 768, 4096), (129, 515, 2049)])
def test_exact_product_matches_oracle(shape):
    M, N, K = shape
    rng = np.random.default_rng(M * 3 + N * 5 + K)
    A = rng.integers(-128, 128, (M, K), dtype=np.int8)
    B = rng.integers(-128, 128, (K, N), dtype=np.int8)
    want = mm.matmul_i64(A, B)
    assert np.array_equal(gu.gpu_gemm_exact(A, B, ENC, b.C_I32).astype(np.int64), want)
    assert np.array_equal(gu.gpu_gemm_exact(A, B, ENC, b.C_I64), want)
    if M <= 300:
        # the oracle's own three-product path agrees as well (method, not only the definition)
        assert np.array_equal(mx.mixed_matmul(A, B), want)


def test_extreme_values_and_long_k_in_int64():
    """Entries -128 / 127 only; K beyond both K* = 85,598 (several accumulation segments) and the
    length whose result fits 32 bits (several launches added in int64)."""
    M, N, K = 256, 256, 200000
    rng = np.random.default_rng(12)
    A = rng.choice(np.array([-128, 127], np.int8), (M, K))
    B = rng.choice(np.array([-128, 127], np.int8), (K, N))
    A[0, :] = -128
    B[:, 0] = -128
    want = mm.matmul_i64(A, B)
    assert want[0, 0] == 128 * 128 * K > 2 ** 31
    assert np.array_equal(gu.gpu_gemm_exact(A, B, ENC, b.C_I64), want)
    with pytest.raises(b.AweError):
        gu.gpu_gemm_exact(A, B, ENC, b.C_I32)


def test_forced_small_segments():
    M, N, K = 256, 512, 4096
    rng = np.random.default_rng(13)
    A = rng.integers(-128, 128, (M, K), dtype=np.int8)
    B = rng.integers(-128, 128, (K, N), dtype=np.int8)
    want = mm.matmul_i64(A, B)
    w = wl.Workload("mixed_small", M, N, K, "int8", "int8", 13, "i32")
    for k_chunk in (256, 1024):
        C = run_three_calls(w, A, B, ENC, b.C_I32, k_chunk=k_chunk)
        assert np.array_equal(C.cpu().numpy().astype(np.int64), want)


def test_headline_size_equals_the_six_product_result():
    w = wl.headline()
    A, B = wl.make_inputs(w)
    C3 = run_three_calls(w, A, B, ENC, b.C_I32)
    assert sampled_rows_match(C3, A, B, 8, 9)
    C6 = run_three_calls(w, A, B, b.ENC_INT8_AWE6, b.C_I32)
    assert torch.equal(C3, C6)
