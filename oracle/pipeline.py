"""Algorithm 1 (run-time procedure) on the CPU, step by step, in integers.

Test infrastructure only; never imported by the CUDA product path.

Steps, in the paper's order: (1) decompose every entry into limbs by table lookup,
(2) form the combination planes by adding limbs, (3) P_k = plane alpha_k of A times plane
beta_k of B, accumulated over the reduction dimension, (4) C = (sum_k l_k P_k) / D, one
exact shift -- or, for the residue form of Section 5.3, the same sum reduced mod m.
Plane values are kept as small integers (elements of S); their E2M1 bit patterns are
produced only by pack_e2m1, which mirrors what the hardware stores (Section 3.1).
"""
from __future__ import annotations

import functools
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

from .schemes import (F_ACC, S_SET, Scheme, dot, e2m1_code, k_star, symmetric_range,
                      to_symmetric, value_table)


@functools.lru_cache(maxsize=None)
def encoder_table(s: Scheme, side: str) -> Dict[int, Tuple[int, ...]]:
    """Decomposition table of one side of a scheme (first loop of Algorithm 1).  Built once per
    (scheme, side): the table is a constant of the configuration record."""
    weights, planes = s.side(side)
    return value_table(weights, planes, modulus=s.modulus)


def plane_values(s: Scheme, side: str, x: int) -> List[int]:
    """Stored plane values of the input value x (first two loops of Algorithm 1)."""
    t = encoder_table(s, side)
    key = x % s.modulus if s.modulus else x
    a = t[key]
    return [dot(p, a) for p in s.stored_planes(side)]


@functools.lru_cache(maxsize=None)
def plane_lut(s: Scheme, side: str, lo: int, hi: int) -> np.ndarray:
    """(hi-lo+1) x n_planes int8 array of stored plane values for inputs lo..hi."""
    t = encoder_table(s, side)
    st = s.stored_planes(side)
    out = np.zeros((hi - lo + 1, len(st)), dtype=np.int8)
    for x in range(lo, hi + 1):
        a = t[x % s.modulus if s.modulus else x]
        for j, p in enumerate(st):
            out[x - lo, j] = dot(p, a)
    return out


def encode_planes(s: Scheme, side: str, X: np.ndarray, lo: int = -128, hi: int = 127) -> np.ndarray:
    """Encode an integer matrix X (R x K, reduction dimension last) into its stored planes:
    result[j] is the R x K int8 matrix of plane j, every entry an element of S."""
    lut = plane_lut(s, side, lo, hi)
    Xi = np.asarray(X).astype(np.int64)
    assert Xi.min(initial=0) >= lo and Xi.max(initial=0) <= hi
    pl = lut[Xi - lo]                     # R x K x n_planes
    return np.ascontiguousarray(np.moveaxis(pl, -1, 0))


def encode_limbs(s: Scheme, side: str, X: np.ndarray, lo: int = -128, hi: int = 127) -> np.ndarray:
    """First loop of Algorithm 1 alone: result[i] is the R x K int8 matrix of limb i (elements of S) with
    w . limbs = X (congruent mod m for a residue scheme).  The second loop -- forming plane alpha_k as
    sum_i alpha_k[i] * limb i -- applied to this gives the planes encode_planes returns."""
    t = encoder_table(s, side)
    n = len(s.side(side)[0])
    lut = np.zeros((hi - lo + 1, n), dtype=np.int8)
    for x in range(lo, hi + 1):
        lut[x - lo] = t[x % s.modulus if s.modulus else x]
    Xi = np.asarray(X).astype(np.int64)
    assert Xi.min(initial=0) >= lo and Xi.max(initial=0) <= hi
    return np.ascontiguousarray(np.moveaxis(lut[Xi - lo], -1, 0))


def pack_e2m1(plane: np.ndarray) -> np.ndarray:
    """Pack an R x K matrix of S values into E2M1 nibbles, two per byte along K, the
    element with the even K index in the low nibble; K is zero-padded to even."""
    code = np.zeros(25, dtype=np.uint8)
    for v in S_SET:
        code[v + 12] = e2m1_code(v)
    c = code[np.asarray(plane).astype(np.int64) + 12]
    if c.shape[-1] % 2:
        c = np.concatenate([c, np.zeros(c.shape[:-1] + (1,), np.uint8)], axis=-1)
    return (c[..., 0::2] | (c[..., 1::2] << 4)).astype(np.uint8)


def plane_products(s: Scheme, pa: np.ndarray, pb: np.ndarray, k_chunk: Optional[int] = None,
                   check_exact: bool = True) -> np.ndarray:
    """Third loop of Algorithm 1.  pa: planes of A (n x M x K), pb: planes of B (n x N x K).
    Returns P (r x M x N, int64).  With check_exact, asserts that over every K segment of
    length k_chunk the sum of |products| stays below 2^24, i.e. an FP32 accumulator would
    have held every partial sum exactly (Section 3.4)."""
    ia, ib = s.plane_index("A"), s.plane_index("B")
    K = pa.shape[-1]
    kc = K if not k_chunk else k_chunk
    out = []
    for k in range(s.r):
        a = pa[ia[k]].astype(np.int64)
        b = pb[ib[k]].astype(np.int64)
        if check_exact:
            for k0 in range(0, K, kc):
                worst = np.abs(a[:, k0:k0 + kc]) @ np.abs(b[:, k0:k0 + kc]).T
                assert worst.max(initial=0) < (1 << F_ACC), "partial sum leaves the exact range"
        out.append(a @ b.T)
    return np.stack(out) if out else np.zeros((0, pa.shape[1], pb.shape[1]), np.int64)


def merged_plane_products(s: Scheme, pa: np.ndarray, pb: np.ndarray) -> Tuple[np.ndarray, List[int]]:
    """Third loop of Algorithm 1 with products of equal coefficient sharing an accumulator
    (Section 3.4, n_g > 1): returns one sum per set and the sets' coefficients, asserting that the sum
    of |products| of every set stays below 2^24 over the whole reduction (one segment)."""
    from .schemes import equal_coefficient_sets
    ia, ib = s.plane_index("A"), s.plane_index("B")
    out, coeff = [], []
    for members in equal_coefficient_sets(s):
        acc = np.zeros((pa.shape[1], pb.shape[1]), dtype=np.int64)
        worst = np.zeros_like(acc)
        for k in members:
            a = pa[ia[k]].astype(np.int64)
            b = pb[ib[k]].astype(np.int64)
            acc += a @ b.T
            worst += np.abs(a) @ np.abs(b).T
        assert worst.max(initial=0) < (1 << F_ACC), "merged partial sum leaves the exact range"
        out.append(acc)
        coeff.append(s.ell[members[0]])
    return np.stack(out), coeff


def reconstruct(s: Scheme, P: np.ndarray) -> np.ndarray:
    """Last step of Algorithm 1: C = (sum_k l_k P_k) / D in Python-width integers
    (int64 suffices for every case the tests run), D an exact shift; residue form:
    the canonical symmetric representative of sum_k l_k P_k mod m."""
    acc = np.zeros(P.shape[1:], dtype=np.int64)
    for k in range(s.r):
        acc += np.int64(s.ell[k]) * P[k]
    if s.modulus:
        lo, _ = symmetric_range(s.modulus)
        return (acc - lo) % s.modulus + lo
    assert not np.any(acc & (s.D - 1)), "sum is not divisible by D"
    return acc >> s.log2D


def awe_matmul(s: Scheme, A: np.ndarray, B: np.ndarray, k_chunk: Optional[int] = None,
               a_range=(-128, 127), b_range=(-128, 127)) -> np.ndarray:
    """Whole of Algorithm 1: A is M x K, B is K x N (integers); returns the M x N product
    (or its symmetric residues for a residue scheme)."""
    pa = encode_planes(s, "A", A, *a_range)
    pb = encode_planes(s, "B", np.ascontiguousarray(np.asarray(B).T), *b_range)
    return reconstruct(s, plane_products(s, pa, pb, k_chunk))


def scheme_constants(s: Scheme, a_range=(-128, 127), b_range=(-128, 127)) -> dict:
    """c_A, c_B and K* of the canonical encoder over the stated input ranges, with n_g = 1."""
    ca = int(np.abs(plane_lut(s, "A", *a_range)).max())
    cb = int(np.abs(plane_lut(s, "B", *b_range)).max())
    return {"c_A": ca, "c_B": cb, "K_star": k_star(ca, cb)}
