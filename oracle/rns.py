"""Choice of the residue-number-system moduli (Section 5.3), CPU oracle side.

Test infrastructure only; never imported by the CUDA product path.

The paper selects, by an integer program over a per-modulus cost table, the pairwise
coprime moduli with the fewest FP4 products in total whose product exceeds 2 K B_A B_B
(B = 2^(M-1) - 1).  It prints the totals (75 for prior work, 59 for this method at width
54 and K = 16,384) but neither the selected set nor its list of 82 three-product moduli.
PARITY UNPINNED: with the three-product moduli this oracle can construct (planes a0, a1,
a0 - a1; see schemes.mod_scheme) the program below reaches 60, not 59; the value 60 and
the selected set are what the tests assert, and the set is the one the residue benchmark
configuration uses.  (One more three-product modulus, 95 or 97, would make the program return 59;
tests/test_oracle_mod.py checks that sensitivity.)
"""
from __future__ import annotations

import math
from typing import Dict, List, Sequence, Tuple

import numpy as np

from .schemes import mod_scheme


def cost_table(max_m: int = 200) -> Dict[int, int]:
    """modulus -> number of FP4 products of the cheapest residue scheme constructed."""
    out = {}
    for m in range(2, max_m + 1):
        s = mod_scheme(m)
        if s is not None:
            out[m] = s.r
    return out


def required_log2(width: int, K: int) -> float:
    """log2 of the bound 2 K B^2 the product of the moduli must exceed."""
    B = 2 ** (width - 1) - 1
    return math.log2(2 * K * B * B)


def select_moduli(costs: Dict[int, int], width: int = 54, K: int = 16384) -> Tuple[int, List[int]]:
    """Minimise the total cost over pairwise coprime subsets with prod(m) > 2 K B^2."""
    from scipy.optimize import Bounds, LinearConstraint, milp

    ms = sorted(costs)
    c = np.array([costs[m] for m in ms], dtype=float)
    need = required_log2(width, K)
    cons = [LinearConstraint(np.array([[math.log2(m) for m in ms]]), need + 1e-9, np.inf)]
    primes = [p for p in range(2, max(ms) + 1) if all(p % q for q in range(2, int(p ** 0.5) + 1))]
    for p in primes:
        row = np.array([[1.0 if m % p == 0 else 0.0 for m in ms]])
        if row.sum() > 1:
            cons.append(LinearConstraint(row, 0, 1))
    res = milp(c, constraints=cons, integrality=np.ones(len(ms)), bounds=Bounds(0, 1))
    sel = [m for m, x in zip(ms, res.x) if x > 0.5]
    # exact re-check of what the floating-point program returned
    B = 2 ** (width - 1) - 1
    assert math.prod(sel) > 2 * K * B * B
    assert all(math.gcd(a, b) == 1 for i, a in enumerate(sel) for b in sel[i + 1:])
    return sum(costs[m] for m in sel), sel


# The set the residue configuration runs (width 54, K = 16,384): 5 one-product, 13
# three-product and 4 four-product moduli, 60 products.
RNS_SET_FP64 = (7, 8, 9, 11, 13, 41, 43, 47, 53, 59, 61, 67, 71, 73, 79, 83, 85, 89, 139, 149, 151, 157)


# --------------------------------------------------------------------------- wide integers
# Section 5.3: a residue number system splits the inputs into residues modulo pairwise coprime
# moduli, computes the per-modulus products in parallel and reconstructs by the Chinese remainder
# theorem; unique reconstruction of the accumulated product requires prod(m) > 2 K B_A B_B.
def residues(X, m: int) -> np.ndarray:
    """Entrywise symmetric residue of an integer array (any integer dtype or Python ints), int8."""
    lo = -(m // 2)
    flat = [((int(x) - lo) % m) + lo for x in np.asarray(X, dtype=object).ravel()]
    return np.array(flat, dtype=np.int8).reshape(np.shape(X))


def crt_symmetric(res: Sequence[int], moduli: Sequence[int]) -> int:
    """The integer x with |x| <= prod(m)/2 and x = res[t] (mod moduli[t]) for every t, by the
    textbook formula x = sum_t res_t M_t (M_t^-1 mod m_t) mod M with M_t = M / m_t."""
    M = math.prod(moduli)
    x = 0
    for r, m in zip(res, moduli):
        Mt = M // m
        x += int(r) * Mt * pow(Mt, -1, m)
    x %= M
    return x - M if x > M // 2 else x


def wide_matmul(A, B) -> np.ndarray:
    """The definition: exact product of integer matrices in unbounded Python integers."""
    return np.asarray(A, dtype=object) @ np.asarray(B, dtype=object)


def rns_matmul(A, B, moduli: Sequence[int] = RNS_SET_FP64, width: int = 54) -> np.ndarray:
    """The method of Section 5.3 step by step: residues, one residue product per modulus through
    Algorithm 1 (mod-m scheme), CRT.  A: M x K, B: K x N integers of the given width."""
    from . import pipeline
    A = np.asarray(A, dtype=object)
    B = np.asarray(B, dtype=object)
    K = A.shape[1]
    bound = 2 ** (width - 1) - 1
    assert all(abs(int(x)) <= bound for x in A.ravel()) and all(abs(int(x)) <= bound for x in B.ravel())
    assert math.prod(moduli) > 2 * K * bound * bound, "moduli too small for a unique result"
    per_mod = []
    for m in moduli:
        s = mod_scheme(m)
        per_mod.append(pipeline.awe_matmul(s, residues(A, m), residues(B, m)))
    out = np.empty(per_mod[0].shape, dtype=object)
    for idx in np.ndindex(*out.shape):
        out[idx] = crt_symmetric([int(c[idx]) for c in per_mod], moduli)
    return out
