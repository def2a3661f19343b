"""INT8 x INT8 with 2 FP8 products and 1 FP4 product (Appendix A, last construction) on the CPU.

Test infrastructure only; never imported by the CUDA product path.

Each input of width 8 is written x = 13 h + 5 eps with eps in {0, +-1, +-2, +-3, +-4, +-6, +-8}
(a subset of S, stored in E2M1) and h an integer stored in FP8 (E4M3).  The three products are
P1 = h h' and P2 = (h + eps)(h' + eps') on FP8 planes and P3 = eps eps' on FP4 planes, with
    x y = 104 P1 + 65 P2 - 40 P3,   D = 1.
In the notation of Definition 4.1 this is the record with limbs (h, eps), weights (13, 5), planes
(1,0), (1,1), (0,1) on both sides and l = (104, 65, -40); what differs from the FP4-only records is
the admissibility rule: a plane stored in FP8 must be an integer E4M3 represents exactly and is
kept within +-14, the bound the paper states (c_A = c_B = 14, K* = floor(2^24 / 14^2)).
"""
from __future__ import annotations

import functools
from fractions import Fraction
from typing import Dict, Tuple

import numpy as np

from .schemes import F_ACC, S, Scheme, k_star

W = (13, 5)
ELL = (104, 65, -40)
FP8_CAP = 14
EPS_SET: Tuple[int, ...] = tuple(s for s in S if abs(s) <= 8)
# the same record in the generic form, for the coefficient identity of Definition 4.1
RECORD = Scheme("int8_mixed_fp8_3", W, W, ((1, 0), (1, 1), (0, 1)), ((1, 0), (1, 1), (0, 1)), ELL)
# planes 0 and 1 are stored as E4M3 bytes, plane 2 as E2M1 nibbles
PLANE_IS_FP8 = (True, True, False)


def e4m3_value(code: int):
    """Real value of an 8-bit E4M3 pattern (1 sign, 4 exponent, 3 mantissa bits, bias 7; no
    infinities, the all-ones exponent with all-ones mantissa is NaN -> None)."""
    sign = -1 if (code >> 7) & 1 else 1
    e = (code >> 3) & 0xF
    m = code & 7
    if e == 0xF and m == 7:
        return None
    if e == 0:
        return sign * Fraction(m, 8) * Fraction(1, 64)
    return sign * (1 + Fraction(m, 8)) * Fraction(2) ** (e - 7)


@functools.lru_cache(maxsize=None)
def e4m3_code(v: int) -> int:
    """8-bit E4M3 pattern whose value is the integer v (zero is stored as +0)."""
    if v == 0:
        return 0
    for c in range(256):
        if e4m3_value(c) == v:
            return c
    raise ValueError(f"{v} is not an E4M3 value")


@functools.lru_cache(maxsize=None)
def mixed_table() -> Dict[int, Tuple[int, int]]:
    """x -> (h, eps) for every int8 x.  Among the pairs with 13 h + 5 eps = x whose FP8 planes h and
    h + eps stay within +-14, take the one minimising (largest |plane|, sum of |planes|, (h, eps)):
    the same tie-break reading as for the FP4-only tables."""
    out: Dict[int, Tuple[int, int]] = {}
    for x in range(-128, 128):
        best = None
        for eps in EPS_SET:
            if (x - 5 * eps) % 13:
                continue
            h = (x - 5 * eps) // 13
            planes = (h, h + eps, eps)
            if abs(h) > FP8_CAP or abs(h + eps) > FP8_CAP:
                continue
            key = (max(abs(p) for p in planes), sum(abs(p) for p in planes), (h, eps))
            if best is None or key < best[0]:
                best = (key, (h, eps))
        if best is None:
            raise ValueError(f"{x} has no admissible pair")
        out[x] = best[1]
    return out


@functools.lru_cache(maxsize=None)
def plane_lut() -> np.ndarray:
    """256 x 3 int8: stored plane values (h, h + eps, eps) of x = -128 .. 127."""
    t = mixed_table()
    out = np.zeros((256, 3), np.int8)
    for x in range(-128, 128):
        h, eps = t[x]
        out[x + 128] = (h, h + eps, eps)
    return out


def encode_planes(X: np.ndarray) -> np.ndarray:
    """R x K int8 matrix -> 3 x R x K int8 planes (h, h + eps, eps)."""
    Xi = np.asarray(X).astype(np.int64)
    assert Xi.min(initial=0) >= -128 and Xi.max(initial=0) <= 127
    return np.ascontiguousarray(np.moveaxis(plane_lut()[Xi + 128], -1, 0))


def pack_e4m3(plane: np.ndarray) -> np.ndarray:
    """Integer plane -> E4M3 bytes, one per element."""
    lut = np.zeros(2 * FP8_CAP + 1, np.uint8)
    for v in range(-FP8_CAP, FP8_CAP + 1):
        lut[v + FP8_CAP] = e4m3_code(v)
    return lut[np.asarray(plane).astype(np.int64) + FP8_CAP]


def constants() -> dict:
    lut = plane_lut().astype(np.int64)
    c = int(np.abs(lut).max())
    return {"c_A": c, "c_B": c, "K_star": k_star(c, c)}


def products(pa: np.ndarray, pb: np.ndarray, k_chunk=None) -> np.ndarray:
    """P_k = plane_k(A) plane_k(B)^T, k = 0..2 (int64), asserting that over every K segment the sum
    of |products| stays below 2^24 (Section 3.4)."""
    K = pa.shape[-1]
    kc = K if not k_chunk else k_chunk
    out = []
    for k in range(3):
        a = pa[k].astype(np.int64)
        b = pb[k].astype(np.int64)
        for k0 in range(0, K, kc):
            worst = np.abs(a[:, k0:k0 + kc]) @ np.abs(b[:, k0:k0 + kc]).T
            assert worst.max(initial=0) < (1 << F_ACC), "partial sum leaves the exact range"
        out.append(a @ b.T)
    return np.stack(out)


def reconstruct(P: np.ndarray) -> np.ndarray:
    return ELL[0] * P[0] + ELL[1] * P[1] + ELL[2] * P[2]


def mixed_matmul(A: np.ndarray, B: np.ndarray, k_chunk=None) -> np.ndarray:
    """A: M x K, B: K x N int8 -> exact M x N product through the three products."""
    pa = encode_planes(A)
    pb = encode_planes(np.ascontiguousarray(np.asarray(B).T))
    return reconstruct(products(pa, pb, k_chunk))
