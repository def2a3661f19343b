"""Seeded synthetic inputs for the tests and the benchmark.

This module only draws random integer matrices; it contains none of the method's
arithmetic, so both the CUDA path and the independent CPU checker can be fed from it.
Every workload is described by a small record; `make_inputs` returns host numpy arrays
A (M x K) and B (K x N), both int8 containers (an INT4 operand holds one value in [-8, 7]
per byte).
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Optional, Tuple

import numpy as np


@dataclass(frozen=True)
class Workload:
    name: str
    M: int
    N: int
    K: int
    a_kind: str           # "int8" | "int4" | "int5" | "int9" | "int12" | "ternary" | "extreme" | "residue"
    b_kind: str
    seed: int
    out: str              # "i32" | "i64" | "res_i16"
    modulus: int = 0


def _draw(rng: np.random.Generator, kind: str, shape: Tuple[int, int], modulus: int) -> np.ndarray:
    if kind == "int8":
        return rng.integers(-128, 128, size=shape, dtype=np.int8)
    if kind == "int4":
        return rng.integers(-8, 8, size=shape, dtype=np.int8)
    if kind == "int5":                         # FP8 (E4M3) significands with sign, uniform in [-15, 15]
        return rng.integers(-15, 16, size=shape, dtype=np.int8)
    if kind == "int9":                         # BF16 significands with sign, uniform in [-255, 255], int16 container
        return rng.integers(-255, 256, size=shape, dtype=np.int16)
    if kind == "int12":                        # width-12 symmetric range (FP16 significand with sign), int16 container
        return rng.integers(-2047, 2048, size=shape, dtype=np.int16)
    if kind == "ternary":                      # uniform in {-1, 0, 1}
        return rng.integers(-1, 2, size=shape, dtype=np.int8)
    if kind == "extreme":                      # every entry is -128 or 127, each with probability 1/2
        pick = rng.integers(0, 2, size=shape, dtype=np.int8)
        return np.where(pick == 1, np.int8(127), np.int8(-128)).astype(np.int8)
    if kind == "residue":                      # uniform in [-floor(m/2), ceil(m/2) - 1]
        lo, hi = -(modulus // 2), (modulus + 1) // 2 - 1
        return rng.integers(lo, hi + 1, size=shape, dtype=np.int8)
    raise ValueError(kind)


def make_inputs(w: Workload) -> Tuple[np.ndarray, np.ndarray]:
    rng = np.random.default_rng(w.seed)
    A = _draw(rng, w.a_kind, (w.M, w.K), w.modulus)
    B = _draw(rng, w.b_kind, (w.K, w.N), w.modulus)
    return A, B


def config1() -> Workload:
    return Workload("c1_int8_256", 256, 256, 256, "int8", "int8", 0, "i32")


def config2() -> Workload:
    return Workload("c2_int8_4096", 4096, 4096, 4096, "int8", "int8", 2, "i32")


def config3() -> Workload:
    return Workload("c3_int4xint8_8192", 8192, 8192, 8192, "int4", "int8", 3, "i32")


def config4() -> Workload:
    return Workload("c4_extreme_4096x4096x16384", 4096, 4096, 16384, "extreme", "extreme", 4, "i64")


def config5(modulus: int, size: int = 8192) -> Workload:
    return Workload(f"c5_mod{modulus}_{size}", size, size, size, "residue", "residue",
                    5000 + modulus, "res_i16", modulus)


def headline(size: int = 8192) -> Workload:
    return Workload(f"hd_int8_{size}", size, size, size, "int8", "int8", 6, "i32")


def small(name: str, M: int, N: int, K: int, a_kind: str = "int8", b_kind: str = "int8",
          seed: int = 1, out: str = "i32", modulus: int = 0) -> Workload:
    return Workload(name, M, N, K, a_kind, b_kind, seed, out, modulus)
