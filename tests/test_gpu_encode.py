"""Encode kernel (Algorithm 1, first two loops) against the CPU oracle, byte for byte."""
import numpy as np
import pytest

from oracle import pipeline as pl
from oracle import schemes as sc
from paper_2609_24519_b200 import binding as b
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu

CASES = [
    (b.ENC_INT8_AWE6, sc.AWE6, 0, b.I8, (-128, 127)),
    (b.ENC_INT8_AWE6_ALT, sc.AWE6_ALT, 0, b.I8, (-128, 127)),
    (b.ENC_INT8_BASE13_9, sc.BASE13_9, 0, b.I8, (-128, 127)),
    (b.ENC_INT4xINT8_AWE4, sc.AWE4, 0, None, None),
    (b.ENC_MOD_M, None, 7, b.I8, (-128, 127)),
    (b.ENC_MOD_M, None, 89, b.I8, (-128, 127)),
    (b.ENC_MOD_M, None, 157, b.I8, (-128, 127)),
]


def _want(s, side, X, lo, hi):
    ref = pl.encode_planes(s, side, X, lo, hi)
    return gu.padded_planes(np.stack([pl.pack_e2m1(p) for p in ref]), X.shape[1])


@pytest.mark.parametrize("enc,s,modulus,dt,rng_", CASES, ids=lambda x: getattr(x, "name", str(x)))
@pytest.mark.parametrize("shape", [(1, 1), (200, 300), (256, 2048), (131, 1025), (520, 4100)])
def test_encode_both_sides_both_layouts(enc, s, modulus, dt, rng_, shape):
    s = s or sc.mod_scheme(modulus)
    R, K = shape
    rng = np.random.default_rng(R * 7919 + K)
    for side, sname in ((b.SIDE_A, "A"), (b.SIDE_B, "B")):
        if enc == b.ENC_INT4xINT8_AWE4:
            sdt, (lo, hi) = (b.I4_IN_I8, (-8, 7)) if side == b.SIDE_A else (b.I8, (-128, 127))
        else:
            sdt, (lo, hi) = dt, rng_
        X = rng.integers(lo, hi + 1, (R, K), dtype=np.int8)
        want = _want(s, sname, X, lo, hi)
        for layout in (b.ROWMAJOR_RxK, b.ROWMAJOR_KxR):
            got = gu.gpu_encode(enc, modulus, side, X, sdt, layout)
            assert got.shape == want.shape
            assert np.array_equal(got, want), (sname, layout)


def test_encode_unaligned_source_and_padded_ld():
    s, enc = sc.AWE6, b.ENC_INT8_AWE6
    X = np.random.default_rng(5).integers(-128, 128, (70, 333), dtype=np.int8)
    want = _want(s, "A", X, -128, 127)
    for layout in (b.ROWMAJOR_RxK, b.ROWMAJOR_KxR):
        for ld_extra, offset in ((0, 3), (5, 0), (16, 16), (7, 1)):
            got = gu.gpu_encode(enc, 0, b.SIDE_A, X, b.I8, layout, ld_extra, offset)
            assert np.array_equal(got, want), (layout, ld_extra, offset)


def test_int4_container_reads_only_the_low_nibble():
    X = np.random.default_rng(6).integers(-8, 8, (64, 256), dtype=np.int8)
    dirty = ((X.astype(np.uint8) & 0xF) | 0x50).astype(np.uint8).view(np.int8)      # junk in the high nibble
    a = gu.gpu_encode(b.ENC_INT4xINT8_AWE4, 0, b.SIDE_A, X, b.I4_IN_I8)
    c = gu.gpu_encode(b.ENC_INT4xINT8_AWE4, 0, b.SIDE_A, dirty, b.I4_IN_I8)
    assert np.array_equal(a, c)


def test_every_nibble_decodes_into_S_and_recomposes():
    """Property check that does not rely on the tie-break: decode the GPU planes and recompute
    the encoded value from the single-limb planes (AWE-6 stores a0, a1, a2 as planes 0..2)."""
    X = np.random.default_rng(8).integers(-128, 128, (96, 512), dtype=np.int8)
    got = gu.gpu_encode(b.ENC_INT8_AWE6, 0, b.SIDE_A, X)
    dec = np.array([int(2 * sc.e2m1_value(c)) for c in range(16)], dtype=np.int64)
    lo, hi = dec[got & 0xF], dec[got >> 4]
    vals = np.empty(got.shape[:2] + (got.shape[2] * 2,), dtype=np.int64)
    vals[..., 0::2], vals[..., 1::2] = lo, hi
    vals = vals[:, :, :512]
    assert set(np.unique(vals)) <= sc.S_SET
    assert np.array_equal(vals[0] + 29 * vals[1] + 37 * vals[2], X.astype(np.int64))
    assert np.array_equal(vals[3], vals[0] + vals[1]) and np.array_equal(vals[5], vals[1] + vals[2])
