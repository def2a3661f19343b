"""The C-ABI library loads, exports every symbol include/awe.h declares, and its host-side
tables agree with the oracle's independently built ones (no GPU, no compute calls)."""
import os
import re

import numpy as np
import pytest

from oracle import pipeline as pl
from oracle import rns
from oracle import schemes as sc

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def b():
    from paper_2609_24519_b200 import build
    build.build()
    from paper_2609_24519_b200 import binding
    return binding


def test_every_declared_symbol_is_exported(b):
    header = open(os.path.join(ROOT, "include", "awe.h")).read()
    declared = set(re.findall(r"\b(awe_[a-z0-9_]+)\s*\(", header))
    assert declared == set(b.EXPORTS)
    L = b.lib()
    for name in declared:
        assert hasattr(L, name), name


def test_records_match_the_paper_and_the_oracle(b):
    for enc, s in ((b.ENC_INT8_AWE6, sc.AWE6), (b.ENC_INT8_AWE6_ALT, sc.AWE6_ALT),
                   (b.ENC_INT8_BASE13_9, sc.BASE13_9), (b.ENC_INT4xINT8_AWE4, sc.AWE4)):
        d = b.awe_encoding_info(enc)
        assert d.r == s.r and list(d.ell)[:d.r] == list(s.ell) and d.log2D == s.log2D
        assert list(d.ia)[:d.r] == s.plane_index("A") and list(d.ib)[:d.r] == s.plane_index("B")
        assert d.n_planes_a == len(s.stored_planes("A")) and d.n_planes_b == len(s.stored_planes("B"))
    d = b.awe_encoding_info(b.ENC_TERNARY_INT8_3)
    s = sc.TERNARY3
    assert d.r == 3 and list(d.ell)[:3] == list(s.ell) and list(d.ib)[:3] == s.plane_index("B")
    assert (d.n_planes_a, d.n_planes_b, d.c_a, d.c_b, d.k_star) == (1, 3, 1, 8, 2097152)
    d = b.awe_encoding_info(b.ENC_FP16SIG_AWE12)
    s = sc.FP16_M12
    assert d.r == 12 and list(d.ell)[:12] == list(s.ell) and d.log2D == 1
    assert list(d.ia)[:12] == s.plane_index("A") and list(d.ib)[:12] == s.plane_index("B")
    assert (d.n_planes_a, d.n_planes_b, d.c_a, d.c_b, d.k_star) == (6, 6, 12, 12, 116508)
    lut = b.awe_encoding_lut(b.ENC_FP16SIG_AWE12, 0, b.SIDE_A, b.I16)
    assert np.array_equal(lut[np.arange(-2047, 2048) & 0xFFF], pl.plane_lut(sc.FP16_M12, "A", -2047, 2047))
    d = b.awe_encoding_info(b.ENC_INT4xINT4_3)
    assert d.r == 3 and list(d.ell)[:3] == list(sc.INT4X4_3.ell) and (d.c_a, d.c_b, d.k_star) == (2, 2, 4194304)
    lut = b.awe_encoding_lut(b.ENC_INT4xINT4_3, 0, b.SIDE_B, b.I4_IN_I8)
    assert np.array_equal(lut[np.arange(-8, 8) & 0xFF], pl.plane_lut(sc.INT4X4_3, "B", -8, 7))
    d = b.awe_encoding_info(b.ENC_FP8SIG_3)
    assert d.r == 3 and list(d.ell)[:3] == list(sc.FP8SIG_3.ell) and (d.c_a, d.c_b, d.k_star) == (4, 4, 1048576)
    lut = b.awe_encoding_lut(b.ENC_FP8SIG_3, 0, b.SIDE_A, b.I5_IN_I8)
    assert np.array_equal(lut[np.arange(-16, 16) & 0x1F], pl.plane_lut(sc.FP8SIG_3, "A", -16, 15))
    assert np.array_equal(lut[(np.arange(-16, 16) & 0x1F) | 0xE0], pl.plane_lut(sc.FP8SIG_3, "A", -16, 15))
    d = b.awe_encoding_info(b.ENC_BF16SIG_8)
    s = sc.BF16SIG_8
    assert d.r == 8 and list(d.ell)[:8] == list(s.ell) and (d.c_a, d.c_b, d.k_star, d.log2D) == (4, 4, 1048576, 0)
    assert list(d.ia)[:8] == s.plane_index("A") and list(d.ib)[:8] == s.plane_index("B")
    lut = b.awe_encoding_lut(b.ENC_BF16SIG_8, 0, b.SIDE_B, b.I9_IN_I16)
    assert np.array_equal(lut[np.arange(-256, 256) & 0x1FF], pl.plane_lut(s, "B", -256, 255))
    d = b.awe_encoding_info(b.ENC_INT8_AWE6)
    assert (d.c_a, d.c_b, d.k_star) == (6, 6, 466033)
    d = b.awe_encoding_info(b.ENC_INT4xINT8_AWE4)
    assert (d.c_a, d.c_b, d.k_star) == (3, 8, 699050)


def test_record_with_sum_planes_formed_in_the_kernel(b):
    """AWE_ENC_INT8_AWE6_DERIVED is the 6-product record with only its limb planes stored: same
    coefficients, three planes per side, products 4..6 name the two limb planes they add, and the table
    holds the limbs of the oracle's decomposition (whose tuples keep all six plane values in S)."""
    d6, dd = b.awe_encoding_info(b.ENC_INT8_AWE6), b.awe_encoding_info(b.ENC_INT8_AWE6_DERIVED)
    assert dd.r == 6 and list(dd.ell)[:6] == list(d6.ell)[:6] and (dd.n_planes_a, dd.n_planes_b) == (3, 3)
    assert (dd.c_a, dd.c_b, dd.k_star) == (d6.c_a, d6.c_b, d6.k_star)
    assert list(dd.ia)[:6] == [0, 1, 2, 0, 0, 1] and list(dd.ia2)[:6] == [-1, -1, -1, 1, 2, 2]
    assert list(dd.ib)[:6] == list(dd.ia)[:6] and list(dd.ib2)[:6] == list(dd.ia2)[:6]
    assert list(d6.ia2)[:6] == [-1] * 6
    X = np.arange(-128, 128, dtype=np.int8).reshape(1, 256)
    for side, name in ((b.SIDE_A, "A"), (b.SIDE_B, "B")):
        lut = b.awe_encoding_lut(b.ENC_INT8_AWE6_DERIVED, 0, side)
        assert np.array_equal(lut[np.arange(-128, 128) & 0xFF].T, pl.encode_limbs(sc.AWE6, name, X)[:, 0, :])
    assert b.awe_planes_bytes(b.ENC_INT8_AWE6_DERIVED, 0, b.SIDE_A, 100, 300) == 3 * 100 * 256


def test_tables_match_the_oracle_tables(b):
    idx = np.arange(-128, 128) & 0xFF
    for enc, s in ((b.ENC_INT8_AWE6, sc.AWE6), (b.ENC_INT8_AWE6_ALT, sc.AWE6_ALT), (b.ENC_INT8_BASE13_9, sc.BASE13_9)):
        for side, name in ((b.SIDE_A, "A"), (b.SIDE_B, "B")):
            assert np.array_equal(b.awe_encoding_lut(enc, 0, side)[idx], pl.plane_lut(s, name, -128, 127))
    lut = b.awe_encoding_lut(b.ENC_INT4xINT8_AWE4, 0, b.SIDE_A, b.I4_IN_I8)
    assert np.array_equal(lut[np.arange(-8, 8) & 0xFF], pl.plane_lut(sc.AWE4, "A", -8, 7))
    assert np.array_equal(b.awe_encoding_lut(b.ENC_INT4xINT8_AWE4, 0, b.SIDE_B)[idx],
                          pl.plane_lut(sc.AWE4, "B", -128, 127))
    lut = b.awe_encoding_lut(b.ENC_TERNARY_INT8_3, 0, b.SIDE_A, b.T2_IN_I8)
    assert np.array_equal(lut[np.arange(-1, 2) & 0xFF], pl.plane_lut(sc.TERNARY3, "A", -1, 1))
    assert not lut[2:255].any()                                   # non-ternary bytes are read as 0
    assert np.array_equal(b.awe_encoding_lut(b.ENC_TERNARY_INT8_3, 0, b.SIDE_B)[idx],
                          pl.plane_lut(sc.TERNARY3, "B", -128, 127))
    for m in rns.RNS_SET_FP64 + (2, 10, 37, 60, 66, 72, 91, 100, 169):
        s = sc.mod_scheme(m)
        d = b.awe_encoding_info(b.ENC_MOD_M, m)
        assert d.r == s.r and list(d.ell)[:d.r] == list(s.ell) and d.modulus == m
        assert np.array_equal(b.awe_encoding_lut(b.ENC_MOD_M, m, b.SIDE_A)[idx], pl.plane_lut(s, "A", -128, 127))


def test_sizes_and_host_side_rejections(b):
    assert b.awe_planes_bytes(b.ENC_INT8_AWE6, 0, b.SIDE_A, 100, 300) == 6 * 100 * 256
    assert b.awe_planes_bytes(b.ENC_INT8_BASE13_9, 0, b.SIDE_B, 8192, 8192) == 3 * 8192 * 4096
    assert b.awe_workspace_bytes(b.ENC_INT8_AWE6, 0, 8192, 8192, 8192) == 2 * 6 * 8192 * 4096
    assert b.awe_planes_bytes(99, 0, b.SIDE_A, 10, 10) == 0
    assert b.awe_workspace_bytes(b.ENC_MOD_M, 170, 10, 10, 10) == 0
    with pytest.raises(b.AweError):
        b.awe_encoding_info(b.ENC_INT8_AWE6, 7)
    assert "workspace" in b.status_string(3)


def test_modulus_selection_matches_the_integer_program(b):
    """awe_wide_select against the oracle's integer program restricted to the built-in moduli."""
    import math
    costs = {m: sc.mod_scheme(m).r for m in rns.RNS_SET_FP64}
    for width, K in [(54, 16384), (54, 59000), (32, 8192), (24, 4096), (12, 1024), (9, 100000), (2, 1)]:
        sel = b.awe_wide_select(width, K)
        want_cost, _ = rns.select_moduli(costs, width=width, K=K)
        B = 2 ** (width - 1) - 1
        assert set(sel) <= set(rns.RNS_SET_FP64) and len(set(sel)) == len(sel)
        assert math.prod(sel) > 2 * K * B * B
        assert sum(costs[m] for m in sel) == want_cost, (width, K, sel)
    assert b.awe_wide_select(54, 16384) == list(rns.RNS_SET_FP64)       # the full set is needed there
    assert b.awe_wide_select(54, 70000) == []                           # beyond the built-in set


def test_header_is_plain_c():
    """include/awe.h must compile as C (no C++ in the boundary)."""
    import subprocess
    src = '#include "awe.h"\nint main(void) { awe_encoding_desc d; (void)d; return (int)AWE_OK; }\n'
    r = subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", "-fsyntax-only", "-I", os.path.join(ROOT, "include"),
                        "-x", "c", "-"], input=src, capture_output=True, text=True)
    assert r.returncode == 0, r.stderr


def test_range_errors_are_returned_before_any_device_work(b):
    """Definition 4.1's denominator D enters the 32-bit range check, and a forced accumulation
    segment may not exceed K* (Section 3.4).  Both rejections happen on the host before the handle
    or any pointer is touched, so a placeholder handle and placeholder addresses reach them."""
    import ctypes
    L = b.lib()
    fake = ctypes.c_void_p(0x10000)          # never dereferenced: the calls return first
    ptr = ctypes.c_void_p(0x20000)

    def planes(enc, K, out_dt, k_chunk=0, modulus=0):
        return L.awe_gemm_planes(fake, enc, modulus, ptr, ptr, 256, 256, K, ptr, out_dt, 256, k_chunk, None)

    RANGE = 5
    # INT4 x INT8 in 4 products has D = 2: |2 C| <= 2 * 8 * 128 * K must stay below 2^31
    assert planes(b.ENC_INT4xINT8_AWE4, 2 ** 20, b.C_I32) == RANGE
    assert planes(b.ENC_INT4xINT8_AWE4, 2 ** 21 - 256, b.C_I32) == RANGE
    # INT8 x INT8 (D = 1): |C| <= 128 * 128 * K
    assert planes(b.ENC_INT8_AWE6, 2 ** 17, b.C_I32) == RANGE
    # forced segments beyond K* = 466,033 (6-product record) and beyond K*/4 for a residue record
    d = b.awe_encoding_info(b.ENC_INT8_AWE6)
    assert planes(b.ENC_INT8_AWE6, 8192, b.C_I32, k_chunk=(d.k_star // 256 + 1) * 256) == RANGE
    dm = b.awe_encoding_info(b.ENC_MOD_M, 89)
    assert planes(b.ENC_MOD_M, 8192, b.C_RES_I16, k_chunk=(dm.k_star // 4 // 256 + 1) * 256, modulus=89) == RANGE
    # the whole-procedure entry point applies the same range rule before its first launch
    rc = L.awe_gemm_exact(fake, ptr, b.I4_IN_I8, ptr, b.I8, 256, 256, 2 ** 20, b.ENC_INT4xINT8_AWE4, 0, ptr, b.C_I32,
                          ptr, ctypes.c_size_t(1 << 62), None)
    assert rc == RANGE
