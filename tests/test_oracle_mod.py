"""Pins for the residue form of the CPU oracle (Section 5.3), no GPU."""
import json
import math
import os

import numpy as np
import pytest

from oracle import pipeline as pl
from oracle import rns
from oracle import schemes as sc

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_constants.json")))["moduli"]


def _two_limb_covers(m, w1):
    return len({(a0 + w1 * a1) % m for a0 in sc.S for a1 in sc.S}) == m


def test_one_product_moduli_are_exactly_the_printed_ones():
    got = [m for m in range(2, 200) if len({a % m for a in sc.S}) == m]
    assert got == GOLD["one_product"]
    assert [m for m in range(2, 200) if sc.mod_scheme(m) is not None and sc.mod_scheme(m).r == 1] == got


def test_two_limb_moduli_with_weight_13():
    ok = [m for m in range(2, 400) if _two_limb_covers(m, 13)]
    top = GOLD["two_limb_weight_13_all_up_to"]
    assert [m for m in ok if m <= top] == list(range(2, top + 1))
    assert [m for m in ok if m > top] == GOLD["two_limb_weight_13_beyond"]


def test_free_weight_primes_and_their_smallest_weights():
    for p, w in zip(GOLD["free_weight_primes"], GOLD["free_weight_smallest"]):
        assert not _two_limb_covers(p, 13)
        assert next(x for x in range(2, p) if _two_limb_covers(p, x)) == w
        assert sc.mod_scheme(p) is not None and sc.mod_scheme(p).r <= 4


def test_symmetric_range():
    assert sc.symmetric_range(7) == (-3, 3) and sc.symmetric_range(8) == (-4, 3)
    for m in (7, 8, 157):
        lo, hi = sc.symmetric_range(m)
        assert hi - lo + 1 == m
        for x in range(-400, 400):
            y = sc.to_symmetric(x, m)
            assert lo <= y <= hi and (x - y) % m == 0


@pytest.mark.parametrize("m", rns.RNS_SET_FP64 + (10, 37, 60, 62, 66, 72, 91, 100, 169))
def test_all_residue_pairs(m):
    """Every residue pair: planes in S, limbs in S, value congruent, and
    sum_k l_k P_k == x y (mod m) with integer coefficients."""
    s = sc.mod_scheme(m)
    assert s is not None and sc.coefficient_identity_holds(s)
    assert all(isinstance(l, int) and 0 <= l < m for l in s.ell)
    ta = pl.encoder_table(s, "A")
    assert sorted(ta) == list(range(m))                       # surjective on T_A
    lo, hi = sc.symmetric_range(m)
    vals = list(range(lo, hi + 1))
    pv = np.array([[sc.dot(p, ta[x % m]) for p in s.alpha] for x in vals], dtype=np.int64)
    pw = np.array([[sc.dot(p, ta[x % m]) for p in s.beta] for x in vals], dtype=np.int64)
    assert set(np.unique(pv)) <= sc.S_SET and set(np.unique(pw)) <= sc.S_SET
    for x in vals:
        assert (sc.dot(s.w, ta[x % m]) - x) % m == 0 and all(l in sc.S_SET for l in ta[x % m])
    lhs = np.einsum("k,ak,bk->ab", np.array(s.ell, dtype=np.int64), pv, pw)
    rhs = np.outer(np.array(vals), np.array(vals))
    assert not np.any((lhs - rhs) % m)


def test_three_product_expansion_by_hand():
    # (a0 + w a1)(b0 + w b1) expanded against P1 = a0 b0, P2 = a1 b1, P3 = (a0-a1)(b0-b1)
    s = sc.mod_scheme(41)
    assert s.r == 3 and s.alpha == ((1, 0), (0, 1), (1, -1))
    w = s.w[1]
    for a0, a1, b0, b1 in [(1, 2, 3, 4), (-6, 3, 8, -2), (12, 8, -12, -8)]:
        full = (a0 + w * a1) * (b0 + w * b1)
        got = s.ell[0] * a0 * b0 + s.ell[1] * a1 * b1 + s.ell[2] * (a0 - a1) * (b0 - b1)
        assert (full - got) % 41 == 0


def test_three_product_moduli_of_the_two_limb_family():
    """Which moduli cost three products when both sides use limbs (a0, a1) and planes a0, a1 and one
    third plane p a0 + q a1 with |p|, |q| <= 4: 10, 12, every modulus from 14 to 67, and
    69, 71, 72, 73, 75, ..., 91 (odd) -- 69 moduli, none above 91.  The third plane a0 - a1 serves all of
    them except 60, 62, 66 and 72, which need 2 a0 - a1.  (Section 5.3 speaks of 82 such moduli without
    printing them: parity with that list is unpinned.)"""
    three = [m for m in range(2, 170) if sc.mod_scheme(m) is not None and sc.mod_scheme(m).r == 3]
    assert three == [10, 12] + list(range(14, 68)) + [69, 71, 72, 73] + list(range(75, 92, 2))
    assert len(three) == 69
    general = [m for m in three if sc.mod_scheme(m).alpha[2] != (1, -1)]
    assert general == [60, 62, 66, 72]
    for m in general:
        s = sc.mod_scheme(m)
        assert s.alpha == s.beta == ((1, 0), (0, 1), (2, -1)) and sc.coefficient_identity_holds(s)
    # the identity behind the coefficients, written out by hand for m = 60:
    # (a0 + w a1)(b0 + w b1) = l1 a0 b0 + l2 a1 b1 + l3 (2 a0 - a1)(2 b0 - b1)  (mod 60)
    s = sc.mod_scheme(60)
    w = s.w[1]
    for a0, a1, b0, b1 in [(1, 2, 3, 4), (-6, 3, 8, -2), (12, 8, -12, -8)]:
        got = s.ell[0] * a0 * b0 + s.ell[1] * a1 * b1 + s.ell[2] * (2 * a0 - a1) * (2 * b0 - b1)
        assert ((a0 + w * a1) * (b0 + w * b1) - got) % 60 == 0


def test_rns_set_for_the_fp64_significand():
    g = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_constants.json")))["rns_fp64"]
    sel = list(rns.RNS_SET_FP64)
    B = 2 ** (g["width"] - 1) - 1
    assert math.prod(sel) > 2 * g["K"] * B * B                 # uniqueness condition of Section 5.3
    assert all(math.gcd(a, b) == 1 for i, a in enumerate(sel) for b in sel[i + 1:])
    total = sum(sc.mod_scheme(m).r for m in sel)
    assert total == 60
    # Parity unpinned: the paper's 59 needs three-product moduli it does not print.  What
    # can be pinned: the total is below prior work's printed count and within one of 59.
    assert total < g["prior_products"] and total - g["awe_products"] == 1


def test_integer_program_reaches_the_same_total():
    costs = rns.cost_table(170)
    total, sel = rns.select_moduli(costs)
    assert total == 60
    assert sum(costs[m] for m in sel) == total


def test_one_more_three_product_modulus_would_give_the_printed_total():
    """Sensitivity of the unpinned total: the program returns the paper's 59 as soon as 95 or 97 costs
    three products, and no two-limb scheme with a third plane p a0 + q a1 (|p|, |q| <= 4) reaches them."""
    g = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_constants.json")))["rns_fp64"]
    costs = rns.cost_table(170)
    assert costs[95] == costs[97] == 4
    for extra in ((95,), (97,), (95, 97)):
        c2 = dict(costs)
        for m in extra:
            c2[m] = 3
        assert rns.select_moduli(c2)[0] == g["awe_products"]
    for p, q in [(p, q) for p in range(1, 5) for q in range(-4, 5) if q]:
        T = [(a0, a1) for a0 in sc.S for a1 in sc.S if (p * a0 + q * a1) in sc.S_SET]
        assert len(T) <= 133
        for m in (95, 97):
            assert all(len({(a0 + w * a1) % m for a0, a1 in T}) < m for w in range(1, m))


# ------------------------------------------------------------------ residue number system, wide integers
def test_crt_textbook_examples():
    # Sunzi's problem: x = 2 (mod 3), 3 (mod 5), 2 (mod 7) -> 23
    assert rns.crt_symmetric([2, 3, 2], [3, 5, 7]) == 23
    assert rns.crt_symmetric([-1, -1, -1], [3, 5, 7]) == -1
    assert rns.crt_symmetric([1, 2, 3, 4], [5, 7, 9, 11]) % 5 == 1
    M = math.prod(rns.RNS_SET_FP64)
    rng = np.random.default_rng(9)
    for _ in range(50):
        x = int(rng.integers(-2 ** 62, 2 ** 62)) * int(rng.integers(1, 2 ** 58)) + int(rng.integers(0, 2 ** 40))
        assert abs(x) < M // 2
        res = [int(rns.residues(np.array([x], dtype=object), m)[0]) for m in rns.RNS_SET_FP64]
        assert rns.crt_symmetric(res, rns.RNS_SET_FP64) == x


def test_residues_are_symmetric_and_congruent():
    xs = np.array([-(2 ** 53 - 1), -12345678901234, -1, 0, 1, 77, 2 ** 53 - 1], dtype=np.int64)
    for m in (7, 8, 157):
        r = rns.residues(xs, m)
        lo, hi = sc.symmetric_range(m)
        assert r.min() >= lo and r.max() <= hi
        assert all((int(x) - int(y)) % m == 0 for x, y in zip(xs, r))


def test_rns_product_of_width_54_integers_equals_the_definition():
    rng = np.random.default_rng(10)
    B53 = 2 ** 53 - 1
    A = rng.integers(-B53, B53 + 1, (5, 9), dtype=np.int64)
    B = rng.integers(-B53, B53 + 1, (9, 4), dtype=np.int64)
    A[0, :] = B53                                       # largest magnitudes, all signs aligned
    B[:, 0] = -B53
    want = rns.wide_matmul(A, B)
    assert want[0, 0] == -9 * B53 * B53
    got = rns.rns_matmul(A, B)
    assert all(int(got[i]) == int(want[i]) for i in np.ndindex(*want.shape))
    # a modulus set that is too small must be refused (uniqueness condition of Section 5.3)
    with pytest.raises(AssertionError):
        rns.rns_matmul(A, B, moduli=rns.RNS_SET_FP64[:-4])
