"""Number system, scheme records and per-value tables of the AWE method (CPU oracle).

Test infrastructure only; never imported by the CUDA product path.

Follows, in the paper's notation:
  * Section 3.1  : S = 2 * {E2M1 values}; E2M1 bit patterns are sign(1) exp(2) mant(1).
  * Section 3.2  : N = sum_i w_i a_i with limbs a_i in S; positional weights (1, 13, 169).
  * Section 3.4  : K* = floor(2^F / (n_g c_A c_B)), F = 24.
  * Definition 4.1: planes alpha_k, beta_k, coefficients lambda_k = l_k / D, weights w, v,
                   admissible tuples T_A, T_B, coverage X.
  * Section 5.3  : the same identity as a congruence mod m with integer coefficients.
  * Appendix A   : the printed INT8xINT8 (6 products), INT4xINT8 (4 products) and
                   FP16-significand (12 products) constructions.
"""
from __future__ import annotations

import itertools
from dataclasses import dataclass, field
from fractions import Fraction
from typing import Dict, List, Optional, Sequence, Tuple

F_ACC = 24  # significand bits of the FP32 accumulator (Section 3.4)


# --------------------------------------------------------------------------- Section 3.1
def e2m1_value(code: int) -> Fraction:
    """Real value of a 4-bit E2M1 pattern (1 sign, 2 exponent, 1 mantissa bit, bias 1,
    no infinities or NaNs): exponent field 0 is subnormal (0 or 1/2)."""
    sign = -1 if (code >> 3) & 1 else 1
    e = (code >> 1) & 3
    m = code & 1
    if e == 0:
        mag = Fraction(m, 2)
    else:
        mag = Fraction(2) ** (e - 1) * (1 + Fraction(m, 2))
    return sign * mag


def storable_set() -> List[int]:
    """S: the E2M1 values doubled, as sorted integers (Section 3.1)."""
    vals = {int(2 * e2m1_value(c)) for c in range(16)}
    assert all(2 * e2m1_value(c) == int(2 * e2m1_value(c)) for c in range(16))
    return sorted(vals)


S: Tuple[int, ...] = tuple(storable_set())
S_SET = frozenset(S)


def e2m1_code(s_value: int) -> int:
    """4-bit E2M1 pattern whose doubled value is s_value (zero is stored as +0)."""
    if s_value == 0:
        return 0
    for c in range(16):
        if 2 * e2m1_value(c) == s_value and c != 8:
            return c
    raise ValueError(f"{s_value} is not in S")


# --------------------------------------------------------------------------- Definition 4.1
@dataclass(frozen=True)
class Scheme:
    """One configuration record: Definition 4.1 plus the modulus of Section 5.3.

    alpha[k] in Z^p and beta[k] in Z^q are the planes of product k, ell[k] its integer
    reconstruction coefficient, D = 2**log2D the common denominator, w and v the limb
    weights.  modulus = 0 means the identity holds over the integers."""
    name: str
    w: Tuple[int, ...]
    v: Tuple[int, ...]
    alpha: Tuple[Tuple[int, ...], ...]
    beta: Tuple[Tuple[int, ...], ...]
    ell: Tuple[int, ...]
    log2D: int = 0
    modulus: int = 0

    @property
    def r(self) -> int:
        return len(self.ell)

    @property
    def D(self) -> int:
        return 1 << self.log2D

    def side(self, side: str):
        """(weights, planes of every product) for side 'A' or 'B'."""
        return (self.w, self.alpha) if side == "A" else (self.v, self.beta)

    def stored_planes(self, side: str) -> List[Tuple[int, ...]]:
        """Distinct planes of one side in order of first use (what has to be stored)."""
        out: List[Tuple[int, ...]] = []
        for p in self.side(side)[1]:
            if p not in out:
                out.append(p)
        return out

    def plane_index(self, side: str) -> List[int]:
        """For each product k, the index of its plane in stored_planes(side)."""
        st = self.stored_planes(side)
        return [st.index(p) for p in self.side(side)[1]]


def coefficient_identity_holds(s: Scheme) -> bool:
    """Matrix form of Definition 4.1: sum_k lambda_k alpha_k beta_k^T = w v^T
    (a congruence mod m, with the D-fold of both sides, for residue schemes)."""
    p, q = len(s.w), len(s.v)
    for i in range(p):
        for j in range(q):
            lhs = sum(s.ell[k] * s.alpha[k][i] * s.beta[k][j] for k in range(s.r))
            rhs = s.D * s.w[i] * s.v[j]
            if s.modulus:
                if (lhs - rhs) % s.modulus:
                    return False
            elif lhs != rhs:
                return False
    return True


def dot(c: Sequence[int], a: Sequence[int]) -> int:
    return sum(ci * ai for ci, ai in zip(c, a))


def admissible_tuples(weights: Sequence[int], planes: Sequence[Sequence[int]],
                      cap: Optional[int] = None) -> List[Tuple[int, ...]]:
    """T of Definition 4.1: limb vectors in S^p whose every plane value lies in S
    (optionally with every plane value capped at |.| <= cap, Appendix A)."""
    out = []
    for a in itertools.product(S, repeat=len(weights)):
        pv = [dot(p, a) for p in planes]
        if all(x in S_SET for x in pv) and (cap is None or all(abs(x) <= cap for x in pv)):
            out.append(a)
    return out


def value_table(weights: Sequence[int], planes: Sequence[Sequence[int]], modulus: int = 0,
                cap: Optional[int] = None) -> Dict[int, Tuple[int, ...]]:
    """The decomposition table of Algorithm 1: represented value -> chosen limb tuple.

    The paper leaves the choice among admissible tuples of equal value open.  Reading
    used here: minimise, in this order, the largest |plane value|, the sum of |plane
    values|, then the limb tuple itself compared lexicographically as integers.
    For a residue scheme the key is (w.a mod m) in [0, m)."""
    best: Dict[int, Tuple[Tuple, Tuple[int, ...]]] = {}
    distinct = []
    for p in planes:
        if tuple(p) not in distinct:
            distinct.append(tuple(p))
    for a in admissible_tuples(weights, distinct, cap):
        pv = [abs(dot(p, a)) for p in distinct]
        x = dot(weights, a)
        if modulus:
            x %= modulus
        key = (max(pv), sum(pv), a)
        if x not in best or key < best[x][0]:
            best[x] = (key, a)
    return {x: a for x, (_, a) in best.items()}


def coverage(table: Dict[int, Tuple[int, ...]]) -> int:
    """Half-width X of the contiguous range [-X, X] the table represents (Section 4.2)."""
    X = 0
    while (X + 1) in table and -(X + 1) in table:
        X += 1
    return X if 0 in table else -1


def max_plane_value(table: Dict[int, Tuple[int, ...]], planes, values) -> int:
    """c of Section 3.4 for an encoder that only ever sees `values`."""
    return max(abs(dot(p, table[x])) for x in values for p in planes)


def k_star(c_a: int, c_b: int, n_g: int = 1, F: int = F_ACC) -> int:
    """Exact-accumulation bound of Section 3.4."""
    return (1 << F) // (n_g * c_a * c_b)


def equal_coefficient_sets(s: "Scheme") -> List[List[int]]:
    """Products that may share one accumulator (Section 3.4, Algorithm 1's third loop): those with the
    same reconstruction coefficient, listed by first occurrence.  n_g is the size of the largest set."""
    sets: Dict[int, List[int]] = {}
    for k, l in enumerate(s.ell):
        sets.setdefault(l, []).append(k)
    return list(sets.values())


def n_g(s: "Scheme") -> int:
    return max(len(g) for g in equal_coefficient_sets(s))


def x_carry(L: int) -> int:
    """Contiguous half-width of L base-13 limbs, by the recurrence of Section 3.2."""
    return 4 if L == 1 else 13 * x_carry(L - 1) + 4


# --------------------------------------------------------------------------- printed records
def _unit(i: int, n: int) -> Tuple[int, ...]:
    return tuple(1 if j == i else 0 for j in range(n))


def _pair(i: int, j: int, n: int) -> Tuple[int, ...]:
    return tuple(1 if t in (i, j) else 0 for t in range(n))


_P6 = (_unit(0, 3), _unit(1, 3), _unit(2, 3), _pair(0, 1, 3), _pair(0, 2, 3), _pair(1, 2, 3))

# Appendix A, "INT8xINT8 in 6 products", product order (P00, P11, P22, P01, P02, P12).
AWE6 = Scheme("int8_awe6", (1, 29, 37), (1, 29, 37), _P6, _P6, (-65, -261, 259, 29, 37, 1073))
# Appendix A, alternative weights (1, 11, 39), same planes.
AWE6_ALT = Scheme("int8_awe6_alt", (1, 11, 39), (1, 11, 39), _P6, _P6, (-49, -319, 1053, 11, 39, 429))
# Appendix A, "INT4xINT8 in 4 products": 2AB = 35 P1 - 42 P2 + 210 P3 + 15 P4.
AWE4 = Scheme("int4xint8_awe4", (3, 5), (5, 3, 42),
              ((0, 1), (1, 0), (1, 2), (2, 1)),
              ((1, 0, 0), (0, 1, -1), (0, 0, 1), (1, 2, 0)),
              (35, -42, 210, 15), log2D=1)
# Prior work (Section 1): positional weights (1, 13, 169), all 3x3 limb pairs.
BASE13_9 = Scheme("int8_base13_9", (1, 13, 169), (1, 13, 169),
                  tuple(_unit(i, 3) for i in range(3) for j in range(3)),
                  tuple(_unit(j, 3) for i in range(3) for j in range(3)),
                  tuple(13 ** (i + j) for i in range(3) for j in range(3)))
# Section 6.2: {0, +-1} x INT8 -- one limb against three positional limbs.
TERNARY3 = Scheme("ternary_x_int8_3", (1,), (1, 13, 169),
                  ((1,), (1,), (1,)), tuple(_unit(j, 3) for j in range(3)), (1, 13, 169))


# Section 5.2 states that INT4xINT4 takes 3 products but does not print the encoding.  Construction
# used here: the Karatsuba-type step on the (2,2) cell with planes (a0, a1, a0 - a1),
#   xy = (1 + w1) a0 b0 + (w1^2 + w1) a1 b1 - w1 (a0 - a1)(b0 - b1),
# with w1 = 3, the weight whose tables need the smallest plane values (|plane| <= 2, coverage 16).
INT4X4_3 = Scheme("int4xint4_3", (1, 3), (1, 3), ((1, 0), (0, 1), (1, -1)), ((1, 0), (0, 1), (1, -1)),
                  (4, 12, -3))


# Section 6.1: an E4M3 significand with sign (|x| <= 15) fits two limbs, so the exact product takes
# the 3 products of the (2,2) cell.  The weights are not printed; same construction as above with
# w1 = 4, the weight with the smallest plane values (3) over [-15, 15] (coverage 20).
FP8SIG_3 = Scheme("fp8sig_3", (1, 4), (1, 4), ((1, 0), (0, 1), (1, -1)), ((1, 0), (0, 1), (1, -1)),
                  (5, 20, -4))


# Section 6.2's table lists BF16 significands (width 9, |x| <= 255) at 8 products; the record is not
# printed.  Construction used here: three limbs, one Karatsuba-type step on the pair (a0, a1) through
# the plane a0 + a1, the other four cross terms as direct products (9 - 1 = 8); weights (4, 9, 61): the
# smallest plane values (4) among the weights up to (7, 59, 199) that cover [-255, 255] (coverage 268).
BF16SIG_8 = Scheme("bf16sig_8", (4, 9, 61), (4, 9, 61),
                   ((1, 0, 0), (0, 1, 0), (0, 0, 1), (1, 1, 0), (1, 0, 0), (0, 0, 1), (0, 1, 0), (0, 0, 1)),
                   ((1, 0, 0), (0, 1, 0), (0, 0, 1), (1, 1, 0), (0, 0, 1), (1, 0, 0), (0, 0, 1), (0, 1, 0)),
                   (16 - 36, 81 - 36, 61 * 61, 36, 4 * 61, 4 * 61, 9 * 61, 9 * 61))


def _fp16_m12() -> Scheme:
    """Appendix A, "FP16xFP16 in 12 products": w = (1, 9, 71, 639),
    2AB = sum_{k,l} 71^(k+l) (-7 P[2k,2l] + 126 P[2k+1,2l+1] + 9 Q[k,l])."""
    alpha, beta, ell = [], [], []
    for k in range(2):
        for l in range(2):
            s = 71 ** (k + l)
            alpha.append(_unit(2 * k, 4)); beta.append(_unit(2 * l, 4)); ell.append(-7 * s)
            alpha.append(_unit(2 * k + 1, 4)); beta.append(_unit(2 * l + 1, 4)); ell.append(126 * s)
            qa = [0] * 4; qa[2 * k] = 1; qa[2 * k + 1] = 2
            qb = [0] * 4; qb[2 * l] = 1; qb[2 * l + 1] = 2
            alpha.append(tuple(qa)); beta.append(tuple(qb)); ell.append(9 * s)
    w = (1, 9, 71, 639)
    return Scheme("fp16sig_awe12", w, w, tuple(alpha), tuple(beta), tuple(ell), log2D=1)


FP16_M12 = _fp16_m12()


# --------------------------------------------------------------------------- Section 5.3
ONE_PRODUCT_MODULI = (2, 3, 4, 5, 6, 7, 8, 9, 11, 13)


def _covers(m: int, weights, planes) -> Optional[int]:
    """Largest |plane value| the canonical table needs if a -> w.a mod m is surjective
    on the admissible tuples (Section 5.3), else None."""
    t = value_table(weights, planes, modulus=m)
    if len(t) != m:
        return None
    return max(abs(dot(p, a)) for a in t.values() for p in planes)


def _best_w1(m: int, planes) -> Optional[int]:
    """Second weight of a two-limb residue scheme x = a0 + w1 a1 (mod m): the paper fixes
    none, so take the w1 in [1, m) with the smallest largest-plane-value, then smallest w1."""
    best = None
    for w1 in range(1, m):
        c = _covers(m, (1, w1), planes)
        if c is not None and (best is None or (c, w1) < best):
            best = (c, w1)
    return None if best is None else best[1]


_K3_PLANES = ((1, 0), (0, 1), (1, -1))
_D4_ALPHA = ((1, 0), (1, 0), (0, 1), (0, 1))
_D4_BETA = ((1, 0), (0, 1), (1, 0), (0, 1))
_mod_cache: Dict[int, Optional[Scheme]] = {}
K3_MAX_COMPONENT = 4


def _k3_general(m: int) -> Optional[Scheme]:
    """Three products on two limbs with a general third plane p a0 + q a1 (same planes and weights
    (1, w1) on both sides).  From
        (a0 + w1 a1)(b0 + w1 b1) = a0 b0 + w1 (a0 b1 + a1 b0) + w1^2 a1 b1,
        (p a0 + q a1)(p b0 + q b1) = p^2 a0 b0 + p q (a0 b1 + a1 b0) + q^2 a1 b1
    the coefficients are l3 with l3 p q = w1, l1 = 1 - l3 p^2, l2 = w1^2 - l3 q^2 (all mod m).
    Candidates in the order (largest plane value, |p| + |q|, p, q, w1); the smallest l3 that solves
    the congruence is taken."""
    best = None
    for p in range(1, K3_MAX_COMPONENT + 1):          # (p, q) and (-p, -q) are the same plane up to sign
        for q in range(-K3_MAX_COMPONENT, K3_MAX_COMPONENT + 1):
            if q == 0:
                continue
            planes = ((1, 0), (0, 1), (p, q))
            pairs = [(a0, a1) for a0 in S for a1 in S if p * a0 + q * a1 in S_SET]
            if len(pairs) < m:
                continue                               # too few admissible tuples to reach every residue
            for w1 in range(1, m):
                if len({(a0 + w1 * a1) % m for a0, a1 in pairs}) < m:
                    continue
                l3 = next((l for l in range(m) if (l * p * q - w1) % m == 0), None)
                if l3 is None:
                    continue
                c = _covers(m, (1, w1), planes)
                assert c is not None
                key = (c, abs(p) + abs(q), p, q, w1)
                if best is None or key < best[0]:
                    best = (key, planes, w1, l3)
    if best is None:
        return None
    (_, _, p, q, _), planes, w1, l3 = best
    ell = ((1 - l3 * p * p) % m, (w1 * w1 - l3 * q * q) % m, l3 % m)
    return Scheme(f"mod{m}_3g", (1, w1), (1, w1), planes, planes, ell, modulus=m)


def mod_scheme(m: int) -> Optional[Scheme]:
    """Residue scheme for modulus m (Section 5.3), cheapest of these constructions:

      1 product : one limb a = x (mod m), only for the moduli S covers by itself;
      3 products: limbs (a0, a1), planes (a0, a1, a0 - a1) on both sides, from
                  xy = (1 + w1) a0 b0 + (w1^2 + w1) a1 b1 - w1 (a0 - a1)(b0 - b1);
                  where no weight works with that third plane, any third plane p a0 + q a1 with
                  |p|, |q| <= 4 (_k3_general);
      4 products: limbs (a0, a1), all four limb pairs, coefficients (1, w1, w1, w1^2).
    The paper prints no residue table; these are constructions of Definition 4.1 relaxed
    to a congruence, each checked exhaustively by the tests."""
    if m in _mod_cache:
        return _mod_cache[m]
    sch = None
    if m >= 2 and len({a % m for a in S}) == m:
        sch = Scheme(f"mod{m}_1", (1,), (1,), ((1,),), ((1,),), (1,), modulus=m)
    if sch is None and m >= 2:
        w1 = _best_w1(m, _K3_PLANES)
        if w1 is not None:
            ell = ((1 + w1) % m, (w1 * w1 + w1) % m, (-w1) % m)
            sch = Scheme(f"mod{m}_3", (1, w1), (1, w1), _K3_PLANES, _K3_PLANES, ell, modulus=m)
    if sch is None and 2 <= m <= 4 * 133:
        # at most 133 limb pairs are admissible with a third plane, so larger moduli cannot be covered
        sch = _k3_general(m)
    if sch is None and m >= 2:
        w1 = _best_w1(m, ((1, 0), (0, 1)))
        if w1 is not None:
            ell = (1, w1 % m, w1 % m, (w1 * w1) % m)
            sch = Scheme(f"mod{m}_4", (1, w1), (1, w1), _D4_ALPHA, _D4_BETA, ell, modulus=m)
    _mod_cache[m] = sch
    return sch


def symmetric_range(m: int) -> Tuple[int, int]:
    """Canonical symmetric residues of m: [-floor(m/2), ceil(m/2) - 1]."""
    return -(m // 2), (m + 1) // 2 - 1


def to_symmetric(x: int, m: int) -> int:
    lo, _ = symmetric_range(m)
    return (x - lo) % m + lo
