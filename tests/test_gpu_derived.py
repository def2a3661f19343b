"""The 6-product record with its sum planes formed inside the product kernel (Section 6.1's remark on
the cost of producing planes; Algorithm 1's second loop moved into the third): only the three limb
planes per side are stored, and the result must still be the exact product, bit for bit."""
import numpy as np
import pytest
import torch

from oracle import matmul as mm
from oracle import pipeline as pl
from oracle import schemes as sc
from paper_2609_24519_b200 import binding as b
from paper_2609_24519_b200 import workloads as wl
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu
ENC = b.ENC_INT8_AWE6_DERIVED


@pytest.mark.parametrize("shape", [(1, 1), (200, 300), (131, 1025), (520, 4100)])
def test_encode_writes_the_limb_planes_of_the_oracle(shape):
    R, K = shape
    X = np.random.default_rng(R + K).integers(-128, 128, (R, K), dtype=np.int8)
    for side, name in ((b.SIDE_A, "A"), (b.SIDE_B, "B")):
        limbs = pl.encode_limbs(sc.AWE6, name, X)
        want = gu.padded_planes(np.stack([pl.pack_e2m1(p) for p in limbs]), K)
        for layout in (b.ROWMAJOR_RxK, b.ROWMAJOR_KxR):
            got = gu.gpu_encode(ENC, 0, side, X, b.I8, layout)
            assert got.shape == want.shape and np.array_equal(got, want), (name, layout)


@pytest.mark.parametrize("M,N,K", [(256, 256, 256), (1, 1, 1), (100, 200, 300), (384, 520, 1300), (129, 257, 2049),
                                   (700, 300, 5000)])
def test_product_equals_the_definition(M, N, K):
    w = wl.small("d", M, N, K, seed=M + N + K)
    A, B = wl.make_inputs(w)
    assert np.array_equal(gu.gpu_gemm_exact(A, B, ENC, b.C_I32), mm.matmul_i64(A, B))


def test_extreme_values_and_int64_output_with_forced_segments():
    """Every entry -128 or 127 (the largest limb sums the record produces), K cut into forced segments."""
    w = wl.small("dx", 300, 280, 3000, "extreme", "extreme", seed=77)
    A, B = wl.make_inputs(w)
    want = mm.matmul_i64(A, B)
    assert np.array_equal(gu.gpu_gemm_exact(A, B, ENC, b.C_I64), want)
    pa = gu.gpu_encode(ENC, 0, b.SIDE_A, A)
    pb = gu.gpu_encode(ENC, 0, b.SIDE_B, np.ascontiguousarray(B.T))
    for k_chunk in (256, 1024):
        assert np.array_equal(gu.gpu_gemm_planes(pa, pb, w.M, w.N, w.K, ENC, b.C_I64, k_chunk=k_chunk), want)


def test_configuration_2_whole_matrix_and_headline_against_the_stored_plane_record():
    w = wl.config2()
    A, B = wl.make_inputs(w)
    assert np.array_equal(gu.gpu_gemm_exact(A, B, ENC, b.C_I32), mm.matmul_i64(A, B))
    w = wl.headline()
    A, B = wl.make_inputs(w)
    got = gu.gpu_gemm_exact(A, B, ENC, b.C_I32)
    rows = [0, 1, 4095, 4096, 8191]
    assert np.array_equal(got[rows], mm.matmul_i64(A[rows], B))
    assert np.array_equal(got, gu.gpu_gemm_exact(A, B, b.ENC_INT8_AWE6, b.C_I32))
