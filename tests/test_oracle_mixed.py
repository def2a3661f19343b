"""Pins for the oracle's mixed 2 x FP8 + 1 x FP4 construction (no GPU): printed constants,
exhaustive identity over all INT8 pairs, format round trips, and the plain integer product."""
import json
import os

import numpy as np
import pytest

from oracle import matmul as om
from oracle import mixed as mx
from oracle import schemes as sc

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_constants.json")))["mixed_fp8"]


def test_printed_record():
    assert list(mx.W) == GOLD["weights"] and list(mx.ELL) == GOLD["ell"] and mx.RECORD.D == GOLD["D"]
    assert sorted({abs(e) for e in mx.EPS_SET}) == GOLD["eps_magnitudes"]
    assert set(mx.EPS_SET) <= set(sc.S)
    # Definition 4.1 in matrix form: sum_k l_k alpha_k beta_k^T = w w^T
    assert sc.coefficient_identity_holds(mx.RECORD)
    # an FP8 product costs two FP4 products where FP8 runs at half the FP4 rate
    cost = sum(2 if f8 else 1 for f8 in mx.PLANE_IS_FP8)
    assert cost == GOLD["fp4_equivalent_products"] < sc.AWE6.r


def test_printed_cap_and_k_star():
    c = mx.constants()
    assert c["c_A"] == c["c_B"] == GOLD["c"]
    assert c["K_star"] == GOLD["k_star"] == (1 << 24) // (14 * 14)


def test_e4m3_format():
    # format definition: bias 7, 3 mantissa bits, subnormals, largest finite value 448, one NaN pattern
    assert mx.e4m3_value(0x38) == 1 and mx.e4m3_value(0x40) == 2 and mx.e4m3_value(0x44) == 3
    assert mx.e4m3_value(0x7E) == 448 and mx.e4m3_value(0x7F) is None and mx.e4m3_value(0xFF) is None
    assert mx.e4m3_value(0x01) == 2.0 ** -9 and mx.e4m3_value(0x08) == 2.0 ** -6
    assert mx.e4m3_value(0xB8) == -1
    # every integer up to 16 is exact, 17 is not
    for v in range(-16, 17):
        assert mx.e4m3_value(mx.e4m3_code(v)) == v
    with pytest.raises(ValueError):
        mx.e4m3_code(17)
    assert mx.pack_e4m3(np.array([[0, 1, -1, 14, -14, 5]])).tolist() == [[0x00, 0x38, 0xB8, 0x56, 0xD6, 0x4A]]


def test_every_int8_value_has_exactly_one_pair():
    # 5 eps runs through all 13 residue classes exactly once over the 13 allowed eps, so the pair is unique
    assert sorted((5 * e) % 13 for e in mx.EPS_SET) == list(range(13))
    t = mx.mixed_table()
    assert sorted(t) == list(range(-128, 128))
    for x, (h, eps) in t.items():
        assert 13 * h + 5 * eps == x and eps in mx.EPS_SET
        assert abs(h) <= 14 and abs(h + eps) <= 14
    lut = mx.plane_lut().astype(int)
    assert np.abs(lut[:, :2]).max() == 14 and np.abs(lut[:, 2]).max() == 8


def test_identity_over_all_int8_pairs():
    lut = mx.plane_lut().astype(np.int64)
    x = np.arange(-128, 128, dtype=np.int64)
    P = [np.outer(lut[:, k], lut[:, k]) for k in range(3)]
    assert np.array_equal(104 * P[0] + 65 * P[1] - 40 * P[2], np.outer(x, x))
    # a wrong sign or a swapped coefficient breaks it
    assert not np.array_equal(104 * P[0] + 65 * P[1] + 40 * P[2], np.outer(x, x))
    assert not np.array_equal(65 * P[0] + 104 * P[1] - 40 * P[2], np.outer(x, x))


def test_matmul_against_plain_product():
    rng = np.random.default_rng(5)
    for (M, N, K) in [(1, 1, 1), (7, 5, 33), (64, 48, 300)]:
        A = rng.integers(-128, 128, (M, K), dtype=np.int8)
        B = rng.integers(-128, 128, (K, N), dtype=np.int8)
        assert np.array_equal(mx.mixed_matmul(A, B), om.matmul_i64(A, B))
    A = np.full((3, 500), -128, np.int8)
    B = np.full((500, 2), -128, np.int8)
    assert np.array_equal(mx.mixed_matmul(A, B, k_chunk=128), om.matmul_i64(A, B))


def test_exactness_assert_fires_past_k_star():
    K = 85599
    pa = np.full((3, 1, K), 14, np.int8)
    pb = np.full((3, 1, K), 14, np.int8)
    with pytest.raises(AssertionError):
        mx.products(pa, pb)
    mx.products(pa[:, :, :85598], pb[:, :, :85598])
