"""Pins for the oracle's plain product and for Algorithm 1 run on the CPU (no GPU)."""
import numpy as np
import pytest

from oracle import matmul as mm
from oracle import pipeline as pl
from oracle import schemes as sc
from paper_2609_24519_b200 import workloads as wl


def _py_matmul(A, B):
    M, K = A.shape
    N = B.shape[1]
    return np.array([[sum(int(A[i, k]) * int(B[k, j]) for k in range(K)) for j in range(N)]
                     for i in range(M)], dtype=np.int64)


def test_c_loop_nest_against_python_integers_and_numpy():
    rng = np.random.default_rng(11)
    for (M, N, K) in [(1, 1, 1), (3, 5, 7), (9, 4, 33)]:
        A = rng.integers(-128, 128, (M, K), dtype=np.int8)
        B = rng.integers(-128, 128, (K, N), dtype=np.int8)
        C = mm.matmul_i64(A, B)
        assert np.array_equal(C, _py_matmul(A, B))
        assert np.array_equal(C, mm.matmul_i64_numpy(A, B))
        assert np.array_equal(mm.matmul_i64_ijk(A, B), _py_matmul(A, B))
    A = rng.integers(-128, 128, (70, 300), dtype=np.int8)
    B = rng.integers(-128, 128, (300, 50), dtype=np.int8)
    assert np.array_equal(mm.matmul_i64(A, B), mm.matmul_i64_numpy(A, B))
    assert np.array_equal(mm.matmul_i64_rows(A, B, 13, 29), mm.matmul_i64_numpy(A, B)[13:29])
    assert np.array_equal(mm.matmul_i64_ijk(A, B), mm.matmul_i64_numpy(A, B))


def test_closed_forms():
    K = 517
    A = np.full((4, K), -128, dtype=np.int8)
    B = np.full((K, 6), -128, dtype=np.int8)
    assert np.all(mm.matmul_i64(A, B) == 16384 * K)
    B = np.random.default_rng(3).integers(-128, 128, (40, 23), dtype=np.int8)
    assert np.array_equal(mm.matmul_i64(np.eye(40, dtype=np.int8), B), B.astype(np.int64))
    a = np.array([[-128], [5], [127]], dtype=np.int8)
    b = np.array([[-128, 0, 127, -1]], dtype=np.int8)
    assert np.array_equal(mm.matmul_i64(a, b), np.outer(a[:, 0].astype(np.int64), b[0].astype(np.int64)))
    # a transposed operand would fail here: the product is not symmetric
    A = np.array([[1, 2], [3, 4]], dtype=np.int8)
    Bm = np.array([[0, 1], [1, 1]], dtype=np.int8)
    assert mm.matmul_i64(A, Bm).tolist() == [[2, 3], [4, 7]]
    assert mm.matmul_i64_ijk(A, Bm).tolist() == [[2, 3], [4, 7]]


def test_int16_product_against_numpy_and_python():
    rng = np.random.default_rng(12)
    A = rng.integers(-2047, 2048, (9, 33), dtype=np.int16)
    B = rng.integers(-2047, 2048, (33, 7), dtype=np.int16)
    C = mm.matmul_i64_s16(A, B)
    assert np.array_equal(C, A.astype(np.int64) @ B.astype(np.int64))
    assert np.array_equal(C, _py_matmul(A, B))
    assert np.array_equal(mm.matmul_i64_s16(A, B, 2, 5), C[2:5])
    assert np.array_equal(pl.awe_matmul(sc.FP16_M12, A, B, a_range=(-2047, 2047), b_range=(-2047, 2047)), C)


def test_mod_symmetric():
    C = np.arange(-50, 50, dtype=np.int64).reshape(10, 10)
    for m in (7, 8, 13):
        R = mm.mod_symmetric(C, m)
        lo, hi = sc.symmetric_range(m)
        assert R.min() >= lo and R.max() <= hi and not np.any((R - C) % m)


@pytest.mark.parametrize("s", [sc.AWE6, sc.AWE6_ALT, sc.BASE13_9], ids=lambda s: s.name)
def test_algorithm1_equals_the_definition_int8(s):
    A, B = wl.make_inputs(wl.small("t", 33, 17, 150, seed=21))
    assert np.array_equal(pl.awe_matmul(s, A, B), mm.matmul_i64(A, B))
    A, B = wl.make_inputs(wl.small("t", 8, 8, 64, "extreme", "extreme", seed=22))
    assert np.array_equal(pl.awe_matmul(s, A, B), mm.matmul_i64(A, B))


def test_algorithm1_equals_the_definition_int4xint8_and_ternary():
    A, B = wl.make_inputs(wl.small("t", 20, 31, 97, "int4", "int8", seed=23))
    assert np.array_equal(pl.awe_matmul(sc.AWE4, A, B, a_range=(-8, 7)), mm.matmul_i64(A, B))
    T = np.random.default_rng(5).integers(-1, 2, (12, 40), dtype=np.int8)
    assert np.array_equal(pl.awe_matmul(sc.TERNARY3, T, B[:40], a_range=(-1, 1)), mm.matmul_i64(T, B[:40]))


@pytest.mark.parametrize("m", [7, 8, 13, 41, 89, 139, 157])
def test_algorithm1_residue_form(m):
    A, B = wl.make_inputs(wl.small("t", 19, 23, 120, "residue", "residue", seed=24, modulus=m))
    want = mm.mod_symmetric(mm.matmul_i64(A, B), m)
    assert np.array_equal(pl.awe_matmul(sc.mod_scheme(m), A, B), want)


def test_brute_force_all_2x2x2_matrices_over_extreme_values():
    """Every 2x2 by 2x2 product with entries from {-128, 0, 127}: Algorithm 1 (6-product and
    base-13 encodings) against integer arithmetic written out entry by entry."""
    import itertools
    vals = (-128, 0, 127)
    mats = [np.array(c, dtype=np.int8).reshape(2, 2) for c in itertools.product(vals, repeat=4)]
    for s in (sc.AWE6, sc.BASE13_9):
        for A in mats:
            for B in mats[::3]:
                want = [[int(A[i, 0]) * int(B[0, j]) + int(A[i, 1]) * int(B[1, j]) for j in range(2)] for i in range(2)]
                assert pl.awe_matmul(s, A, B).tolist() == want


def test_config1_all_int8_encodings_agree():
    A, B = wl.make_inputs(wl.config1())
    C = mm.matmul_i64(A, B)
    for s in (sc.AWE6, sc.AWE6_ALT, sc.BASE13_9):
        assert np.array_equal(pl.awe_matmul(s, A, B), C)
    assert np.abs(C).max() < 2 ** 31


def test_exactness_guard_fires_beyond_k_star():
    # planes of +-12 only: 144 K reaches 2^24 at K = 116,509 > K* = 116,508
    s = sc.Scheme("one", (1,), (1,), ((1,),), ((1,),), (1,))
    K = sc.k_star(12, 12)
    pa = np.full((1, 1, K + 1), 12, dtype=np.int8)
    pb = np.full((1, 1, K + 1), -12, dtype=np.int8)
    with pytest.raises(AssertionError):
        pl.plane_products(s, pa, pb)
    P = pl.plane_products(s, pa, pb, k_chunk=K)           # segmented at K*: exact again
    assert P[0, 0, 0] == -144 * (K + 1)
    assert 144 * K < 2 ** 24 <= 144 * (K + 1)


def test_workload_generators():
    A, B = wl.make_inputs(wl.small("t", 64, 64, 64, "extreme", "extreme"))
    assert set(np.unique(A)) <= {-128, 127} and set(np.unique(B)) <= {-128, 127}
    A, B = wl.make_inputs(wl.small("t", 64, 64, 64, "int4", "int8"))
    assert A.min() >= -8 and A.max() <= 7
    A, B = wl.make_inputs(wl.small("t", 64, 64, 64, "residue", "residue", modulus=8))
    assert A.min() >= -4 and A.max() <= 3
    A2, _ = wl.make_inputs(wl.small("t", 64, 64, 64, "residue", "residue", modulus=8))
    assert np.array_equal(A, A2)


def test_limbs_and_plane_formation_are_the_two_loops_of_algorithm1():
    """First loop (limbs with w . a = x, every limb in S) and second loop (plane alpha_k = sum of limbs)
    taken apart: together they give the stored planes, for every int8 value."""
    X = np.arange(-128, 128, dtype=np.int8).reshape(1, 256)
    for s in (sc.AWE6, sc.AWE6_ALT, sc.BASE13_9):
        for side in ("A", "B"):
            limbs = pl.encode_limbs(s, side, X).astype(np.int64)
            w, _ = s.side(side)
            assert set(np.unique(limbs)) <= sc.S_SET
            assert np.array_equal(sum(int(w[i]) * limbs[i] for i in range(len(w))), X.astype(np.int64))
            planes = pl.encode_planes(s, side, X).astype(np.int64)
            for j, alpha in enumerate(s.stored_planes(side)):
                assert np.array_equal(sum(int(alpha[i]) * limbs[i] for i in range(len(w))), planes[j])
    # the 6-product record stores the three limbs first, then the three pairwise sums
    assert list(sc.AWE6.stored_planes("A")[:3]) == [(1, 0, 0), (0, 1, 0), (0, 0, 1)]
    assert list(sc.AWE6.stored_planes("A")[3:]) == [(1, 1, 0), (1, 0, 1), (0, 1, 1)]
