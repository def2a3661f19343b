"""Pins for the CPU oracle's number system, schemes and tables (no GPU).

Each check compares the oracle with something it did not produce itself: constants the
paper prints (tests/golden/paper_constants.json), closed forms, or exhaustive enumeration
of the identity the scheme claims."""
import itertools
import json
import os

import numpy as np
import pytest

from oracle import pipeline as pl
from oracle import schemes as sc

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_constants.json")))


def test_storable_set_is_the_printed_one():
    pos = GOLD["storable_set"]["value"]
    assert list(sc.S) == sorted(set(pos) | {-x for x in pos})
    assert len(sc.S) == 15
    # E2M1 magnitudes by the format definition: 0, 1/2, 1, 3/2, 2, 3, 4, 6 for codes 0..7
    assert [float(sc.e2m1_value(c)) for c in range(8)] == [0, 0.5, 1, 1.5, 2, 3, 4, 6]
    assert [float(sc.e2m1_value(c + 8)) for c in range(1, 8)] == [-0.5, -1, -1.5, -2, -3, -4, -6]
    for v in sc.S:
        assert 2 * sc.e2m1_value(sc.e2m1_code(v)) == v
    assert sc.e2m1_code(0) == 0 and sc.e2m1_code(-12) == 0xF and sc.e2m1_code(12) == 0x7


def test_pack_e2m1_nibble_order():
    plane = np.array([[1, -1, 12, 0, 3]], dtype=np.int8)
    packed = pl.pack_e2m1(plane)
    # codes: 1->1, -1->9, 12->7, 0->0, 3->3, pad->0; even index in the low nibble
    assert packed.tolist() == [[0x91, 0x07, 0x03]]


def test_x_carry_recurrence_closed_form_and_enumeration():
    for L, want in GOLD["x_carry"]["value"].items():
        L = int(L)
        assert sc.x_carry(L) == want == (13 ** L - 1) // 3
        w = tuple(13 ** i for i in range(L))
        planes = tuple(tuple(1 if i == j else 0 for i in range(L)) for j in range(L))
        assert sc.coverage(sc.value_table(w, planes)) == want


def test_printed_records_are_what_the_oracle_holds():
    g = GOLD["awe6"]
    assert list(sc.AWE6.w) == g["weights"] == list(sc.AWE6.v)
    assert list(sc.AWE6.ell) == g["ell"] and sc.AWE6.D == g["D"]
    assert list(sc.AWE6_ALT.w) == GOLD["awe6_alt"]["weights"]
    assert list(sc.AWE6_ALT.ell) == GOLD["awe6_alt"]["ell"]
    g = GOLD["awe4"]
    assert list(sc.AWE4.w) == g["w"] and list(sc.AWE4.v) == g["v"]
    assert list(sc.AWE4.ell) == g["two_AB"] and sc.AWE4.D == g["D"]
    pc = GOLD["product_counts"]
    assert sc.BASE13_9.r == pc["int8xint8_prior"] and sc.AWE6.r == pc["int8xint8"]
    assert sc.AWE4.r == pc["int4xint8"] and sc.FP16_M12.r == pc["fp16"]
    assert sc.TERNARY3.r == pc["ternary_x_int8"]
    # the direct decomposition of a 4-limb width needs 4 x 4 products
    assert len(sc.FP16_M12.w) ** 2 == pc["fp16_prior"]


def test_awe6_scalar_coefficient_relations():
    # Expanding (a0+29a1+37a2)(b0+29b1+37b2) against the six products term by term.
    l = dict(zip(GOLD["awe6"]["ell_order"], GOLD["awe6"]["ell"]))
    assert l["P00"] + l["P01"] + l["P02"] == 1
    assert l["P11"] + l["P01"] + l["P12"] == 29 * 29
    assert l["P22"] + l["P02"] + l["P12"] == 37 * 37
    assert (l["P01"], l["P02"], l["P12"]) == (29, 37, 29 * 37)


@pytest.mark.parametrize("s", [sc.AWE6, sc.AWE6_ALT, sc.AWE4, sc.BASE13_9, sc.TERNARY3, sc.INT4X4_3, sc.FP8SIG_3,
                               sc.BF16SIG_8, sc.FP16_M12],
                         ids=lambda s: s.name)
def test_matrix_identity(s):
    assert sc.coefficient_identity_holds(s)


def test_broken_record_is_detected():
    bad = sc.Scheme("bad", sc.AWE6.w, sc.AWE6.v, sc.AWE6.alpha, sc.AWE6.beta,
                    (-65, -261, 259, 29, 37, 1072))
    assert not sc.coefficient_identity_holds(bad)


def test_coverage_and_kstar_pins():
    P6 = sc.AWE6.alpha
    assert sc.coverage(sc.value_table((1, 29, 37), P6)) == GOLD["awe6"]["coverage"]
    assert sc.coverage(sc.value_table((1, 29, 37), P6, cap=6)) == GOLD["awe6"]["coverage_with_cap_6"]
    assert sc.coverage(sc.value_table((1, 29, 37), P6, cap=4)) < 127      # a cap of 4 is too tight
    assert sc.coverage(sc.value_table((1, 11, 39), P6)) == GOLD["awe6_alt"]["coverage"]
    assert sc.k_star(6, 6) == GOLD["awe6"]["k_star_cap_6"]
    assert sc.k_star(12, 12) == GOLD["awe6"]["k_star_all_S"]
    assert sc.k_star(3, 8) == GOLD["awe4"]["k_star"]
    o = GOLD["other_k_star"]
    assert sc.k_star(127, 127) == o["bf16_127x127"] and sc.k_star(1, 8) == o["ternary_x_int8"]
    assert sc.k_star(1, 127) == o["bf16_1x127"] and sc.k_star(14, 14) == o["c14"]
    # canonical encoders reach exactly the printed plane-value bounds
    assert pl.scheme_constants(sc.AWE6) == {"c_A": 6, "c_B": 6, "K_star": GOLD["awe6"]["k_star_cap_6"]}
    c4 = pl.scheme_constants(sc.AWE4, a_range=(-8, 7))
    assert (c4["c_A"], c4["c_B"], c4["K_star"]) == (3, 8, GOLD["awe4"]["k_star"])
    t = sc.value_table(sc.FP16_M12.w, sc.FP16_M12.alpha)
    assert sc.coverage(t) == GOLD["fp16_m12"]["coverage"]
    assert sc.k_star(12, 12) == GOLD["fp16_m12"]["k_star"]


def _all_pairs(s, a_vals, b_vals):
    """Exhaustive check over input pairs: every stored plane in S, every limb in S,
    encoded value correct, and sum_k l_k P_k == D x y (Definition 4.1)."""
    ta, tb = pl.encoder_table(s, "A"), pl.encoder_table(s, "B")
    pa = np.array([[sc.dot(p, ta[x]) for p in s.alpha] for x in a_vals], dtype=np.int64)   # |a| x r
    pb = np.array([[sc.dot(p, tb[y]) for p in s.beta] for y in b_vals], dtype=np.int64)
    for x in a_vals:
        assert sc.dot(s.w, ta[x]) == x and all(l in sc.S_SET for l in ta[x])
    for y in b_vals:
        assert sc.dot(s.v, tb[y]) == y and all(l in sc.S_SET for l in tb[y])
    assert set(np.unique(pa)) <= sc.S_SET and set(np.unique(pb)) <= sc.S_SET
    lhs = np.einsum("k,ak,bk->ab", np.array(s.ell, dtype=np.int64), pa, pb)
    rhs = s.D * np.outer(np.array(a_vals, dtype=np.int64), np.array(b_vals, dtype=np.int64))
    assert np.array_equal(lhs, rhs)


@pytest.mark.parametrize("s", [sc.AWE6, sc.AWE6_ALT, sc.BASE13_9], ids=lambda s: s.name)
def test_all_256x256_int8_pairs(s):
    _all_pairs(s, list(range(-128, 128)), list(range(-128, 128)))


def test_all_int4_x_int8_pairs():
    _all_pairs(sc.AWE4, list(range(-8, 8)), list(range(-128, 128)))


def test_int4_x_int4_in_three_products():
    # the count is the paper's (Section 5.2); the encoding is this oracle's construction
    s = sc.INT4X4_3
    assert s.r == 3 and sc.coefficient_identity_holds(s)
    _all_pairs(s, list(range(-8, 8)), list(range(-8, 8)))
    t = sc.value_table(s.w, s.alpha)
    assert sc.coverage(t) == 16
    assert pl.scheme_constants(s, (-8, 7), (-8, 7)) == {"c_A": 2, "c_B": 2, "K_star": 4194304}
    # w1 = 3 is the weight with the smallest plane values among those that cover [-8, 7]
    best = min((max(abs(sc.dot(p, sc.value_table((1, w), s.alpha)[x])) for x in range(-8, 8) for p in s.alpha), w)
               for w in range(2, 8) if sc.coverage(sc.value_table((1, w), s.alpha)) >= 8)
    assert best == (2, 3)


def test_fp8_significands_in_three_products():
    # Section 6.1: an E4M3 significand with sign (|x| <= 15) fits 2 limbs, hence the 3 products of the
    # (2,2) cell; the weights are this oracle's choice by the same rule as for INT4xINT4
    s = sc.FP8SIG_3
    assert s.r == 3 and sc.coefficient_identity_holds(s)
    _all_pairs(s, list(range(-16, 16)), list(range(-16, 16)))
    t = sc.value_table(s.w, s.alpha)
    assert sc.coverage(t) == 20 >= 15
    assert pl.scheme_constants(s, (-15, 15), (-15, 15)) == {"c_A": 3, "c_B": 3, "K_star": (1 << 24) // 9}
    assert pl.scheme_constants(s, (-16, 15), (-16, 15)) == {"c_A": 4, "c_B": 4, "K_star": 1048576}
    best = min((max(abs(sc.dot(p, sc.value_table((1, w), s.alpha)[x])) for x in range(-15, 16) for p in s.alpha), w)
               for w in range(2, 8) if sc.coverage(sc.value_table((1, w), s.alpha)) >= 15)
    assert best == (3, 4)
    # every E4M3 significand: 8 + mantissa (normal numbers), 0..7 (subnormals)
    assert {8 + m for m in range(8)} | set(range(8)) <= set(range(0, 16))


def test_bf16_significands_in_eight_products():
    # the count is the paper's (Section 6.2, table of native formats); the record is this oracle's construction
    s = sc.BF16SIG_8
    assert s.r == 8 and sc.coefficient_identity_holds(s) and s.D == 1
    assert len(s.stored_planes("A")) == len(s.stored_planes("B")) == 4
    v = list(range(-256, 256))
    _all_pairs(s, v, v)
    t = sc.value_table(s.w, s.stored_planes("A"))
    assert sc.coverage(t) == 268 >= 255
    assert pl.scheme_constants(s, (-256, 255), (-256, 255)) == {"c_A": 4, "c_B": 4, "K_star": 1048576}
    assert sc.n_g(s) == 2 and len(sc.equal_coefficient_sets(s)) == 6
    # one Karatsuba-type step saves exactly one of the nine limb-pair products
    assert s.r == len(s.w) * len(s.v) - 1


def test_all_ternary_x_int8_pairs():
    _all_pairs(sc.TERNARY3, [-1, 0, 1], list(range(-128, 128)))


def test_all_fp16_significand_pairs():
    v = list(range(-2047, 2048))
    _all_pairs(sc.FP16_M12, v, v)


def test_identity_over_all_admissible_tuples_awe6():
    # Definition 4.1 quantifies over T_A x T_B, not only over the tuples an encoder picks.
    s = sc.AWE6
    T = np.array(sc.admissible_tuples(s.w, s.stored_planes("A")), dtype=np.int64)
    al = np.array(s.alpha, dtype=np.int64)
    pv = T @ al.T                                     # |T| x r plane values
    val = T @ np.array(s.w, dtype=np.int64)
    lhs = np.einsum("k,ak,bk->ab", np.array(s.ell, dtype=np.int64), pv, pv)
    assert np.array_equal(lhs, np.outer(val, val))
    assert set(np.unique(pv)) <= sc.S_SET


def test_tie_break_is_the_stated_one():
    # brute force over S^3 with the stated ordering, written out independently for AWE-6
    s = sc.AWE6
    t = pl.encoder_table(s, "A")
    for x in (-128, -77, -1, 0, 5, 29, 66, 127):
        cands = []
        for a in itertools.product(sc.S, repeat=3):
            pv = [a[0], a[1], a[2], a[0] + a[1], a[0] + a[2], a[1] + a[2]]
            if all(v in sc.S_SET for v in pv) and a[0] + 29 * a[1] + 37 * a[2] == x:
                cands.append((max(map(abs, pv)), sum(map(abs, pv)), a))
        assert t[x] == min(cands)[2]


def test_equal_coefficient_sets_and_their_accumulation_bound():
    """Section 3.4: n_g products of equal coefficient share an accumulator and divide K* by n_g."""
    sets = sc.equal_coefficient_sets(sc.BASE13_9)
    assert sorted(len(g) for g in sets) == [1, 1, 2, 2, 3] and sc.n_g(sc.BASE13_9) == 3
    # the anti-diagonals i + j = const of the 3 x 3 limb pairs
    assert sets == [[0], [1, 3], [2, 4, 6], [5, 7], [8]]
    assert sc.k_star(8, 8, n_g=3) == (1 << 24) // 192 == 87381
    assert sc.n_g(sc.AWE6) == sc.n_g(sc.AWE6_ALT) == sc.n_g(sc.AWE4) == 1
    assert sc.n_g(sc.FP16_M12) == 2 and len(sc.equal_coefficient_sets(sc.FP16_M12)) == 9
    assert sc.n_g(sc.mod_scheme(157)) == 2 and sc.mod_scheme(157).r == 4      # coefficients (1, w1, w1, w1^2)
    # merged accumulation reconstructs the same matrix
    rng = np.random.default_rng(8)
    A = rng.integers(-128, 128, (9, 40), dtype=np.int8)
    B = rng.integers(-128, 128, (40, 7), dtype=np.int8)
    for s in (sc.BASE13_9, sc.AWE6):
        pa = pl.encode_planes(s, "A", A)
        pb = pl.encode_planes(s, "B", np.ascontiguousarray(B.T))
        Pm, coeff = pl.merged_plane_products(s, pa, pb)
        C = sum(np.int64(c) * P for c, P in zip(coeff, Pm)) >> s.log2D
        assert np.array_equal(C, A.astype(np.int64) @ B.astype(np.int64))
    # the bound: all-(+8) planes at K = 87,381 stay inside, one more element does not
    K = 87381
    pa = np.full((3, 1, K), 8, dtype=np.int8)
    pl.merged_plane_products(sc.BASE13_9, pa, pa[:, :, :])
    big = np.full((3, 1, K + 1), 8, dtype=np.int8)
    with pytest.raises(AssertionError):
        pl.merged_plane_products(sc.BASE13_9, big, big)
