"""Seeded random sweep: every encoding on random shapes (ragged tiles, tiny and odd sizes), random
leading dimensions of C and random value mixes, against the plain int64 product of the CPU oracle."""
import os
import time

import numpy as np
import pytest
import torch

from oracle import matmul as mm
from oracle import rns
from paper_2609_24519_b200 import binding as b
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu

# encoding, dtype and value range of A, dtype and value range of B
KINDS = [
    ("awe6", b.ENC_INT8_AWE6, b.I8, (-128, 127), b.I8, (-128, 127)),
    ("awe6_alt", b.ENC_INT8_AWE6_ALT, b.I8, (-128, 127), b.I8, (-128, 127)),
    ("base13", b.ENC_INT8_BASE13_9, b.I8, (-128, 127), b.I8, (-128, 127)),
    ("mixed", b.ENC_INT8_MIXED_FP8_3, b.I8, (-128, 127), b.I8, (-128, 127)),
    ("awe4", b.ENC_INT4xINT8_AWE4, b.I4_IN_I8, (-8, 7), b.I8, (-128, 127)),
    ("int4x4", b.ENC_INT4xINT4_3, b.I4_IN_I8, (-8, 7), b.I4_IN_I8, (-8, 7)),
    ("ternary", b.ENC_TERNARY_INT8_3, b.T2_IN_I8, (-1, 1), b.I8, (-128, 127)),
    ("fp8sig", b.ENC_FP8SIG_3, b.I5_IN_I8, (-16, 15), b.I5_IN_I8, (-16, 15)),
    ("fp16sig", b.ENC_FP16SIG_AWE12, b.I16, (-2047, 2047), b.I16, (-2047, 2047)),
    ("bf16sig", b.ENC_BF16SIG_8, b.I9_IN_I16, (-256, 255), b.I9_IN_I16, (-256, 255)),
]


def _draw(rng, lo, hi, shape, dtype, style):
    if style == 0:
        X = rng.integers(lo, hi + 1, shape)
    elif style == 1:                                   # extremes only
        X = rng.choice(np.array([lo, hi]), shape)
    elif style == 2:                                   # sparse: mostly zeros
        X = rng.integers(lo, hi + 1, shape) * (rng.random(shape) < 0.1)
    else:                                              # small magnitudes
        X = rng.integers(max(lo, -2), min(hi, 2) + 1, shape)
    return X.astype(dtype)


@pytest.mark.parametrize("case", range(60))
def test_random_shape_and_values(case):
    rng = np.random.default_rng(1000 + case)
    name, enc, a_dt, (alo, ahi), b_dt, (blo, bhi) = KINDS[case % len(KINDS)]
    M, N = int(rng.integers(1, 700)), int(rng.integers(1, 700))
    K = int(rng.integers(1, 3000))
    wide_in = a_dt in (b.I16, b.I9_IN_I16)
    np_dt = np.int16 if wide_in else np.int8
    A = _draw(rng, alo, ahi, (M, K), np_dt, int(rng.integers(0, 4)))
    B = _draw(rng, blo, bhi, (K, N), np_dt, int(rng.integers(0, 4)))
    want = mm.matmul_i64_s16(A, B) if wide_in else mm.matmul_i64(A, B)
    out_dt = b.C_I64 if (a_dt == b.I16 or case % 3 == 0) else b.C_I32
    got = gu.gpu_gemm_exact(A, B, enc, out_dt, a_dt=a_dt, b_dt=b_dt)
    assert np.array_equal(got.astype(np.int64), want), (name, M, N, K)


@pytest.mark.parametrize("case", range(16))
def test_random_modulus_shape_and_values(case):
    rng = np.random.default_rng(2000 + case)
    m = int(rng.choice(np.array(rns.RNS_SET_FP64)))
    M, N, K = int(rng.integers(1, 600)), int(rng.integers(1, 600)), int(rng.integers(1, 5000))
    A = rng.integers(-128, 128, (M, K), dtype=np.int8)
    B = rng.integers(-128, 128, (K, N), dtype=np.int8)
    want = mm.mod_symmetric(mm.matmul_i64(A, B), m)
    out_dt = b.C_RES_I16 if case % 2 else b.C_RES_I32
    got = gu.gpu_gemm_exact(A, B, b.ENC_MOD_M, out_dt, modulus=m)
    assert np.array_equal(got.astype(np.int64), want), (m, M, N, K)


@pytest.mark.parametrize("case", range(8))
def test_planes_entry_with_random_leading_dimension(case):
    """awe_gemm_planes with ldc > N: the columns beyond N must stay untouched."""
    rng = np.random.default_rng(3000 + case)
    enc = [b.ENC_INT8_AWE6, b.ENC_INT8_MIXED_FP8_3][case % 2]
    M, N, K = int(rng.integers(1, 500)), int(rng.integers(1, 500)), int(rng.integers(1, 2000))
    ldc = N + int(rng.integers(0, 9))
    A = rng.integers(-128, 128, (M, K), dtype=np.int8)
    B = rng.integers(-128, 128, (K, N), dtype=np.int8)
    h = gu.handle()
    nA = b.awe_planes_bytes(enc, 0, b.SIDE_A, M, K)
    ws = torch.empty(b.awe_workspace_bytes(enc, 0, M, N, K), dtype=torch.uint8, device="cuda")
    pa, pb = ws[:nA], ws[(nA + 255) // 256 * 256:]
    b.awe_encode(h, enc, 0, b.SIDE_A, torch.from_numpy(A).cuda(), b.I8, b.ROWMAJOR_RxK, M, K, K, pa)
    b.awe_encode(h, enc, 0, b.SIDE_B, torch.from_numpy(B).cuda(), b.I8, b.ROWMAJOR_KxR, N, K, N, pb)
    C = torch.full((M, ldc), 77, dtype=torch.int32, device="cuda")
    b.awe_gemm_planes(h, enc, 0, pa, pb, M, N, K, C, b.C_I32, ldc, 0)
    torch.cuda.synchronize()
    assert b.awe_last_device_status(h) == (0, 0)
    got = C.cpu().numpy()
    assert np.array_equal(got[:, :N].astype(np.int64), mm.matmul_i64(A, B))
    assert (got[:, N:] == 77).all()


# ---- a campaign over every route into the library, as long as AWE_FUZZ_SECONDS allows (default 15 s) ----
CAMPAIGN_KINDS = KINDS + [
    ("derived", b.ENC_INT8_AWE6_DERIVED, b.I8, (-128, 127), b.I8, (-128, 127)),
    ("mod", b.ENC_MOD_M, b.I8, (-128, 127), b.I8, (-128, 127)),
]
HOST_ROUTE = (b.ENC_INT8_AWE6, b.ENC_INT8_BASE13_9, b.ENC_INT8_MIXED_FP8_3, b.ENC_MOD_M)


def _campaign_shape(rng):
    r = rng.random()
    if r < 0.25:                                       # tiny
        return int(rng.integers(1, 40)), int(rng.integers(1, 40)), int(rng.integers(1, 600))
    if r < 0.7:                                        # a few tiles with ragged edges
        return int(rng.integers(1, 700)), int(rng.integers(1, 700)), int(rng.integers(1, 3000))
    if r < 0.85:                                       # long reductions (several K segments for int64 output)
        return int(rng.integers(1, 160)), int(rng.integers(1, 160)), int(rng.integers(3000, 70000))
    return int(rng.integers(500, 2100)), int(rng.integers(500, 2100)), int(rng.integers(1, 1500))


def _campaign_case(seed, moduli):
    """One random case: encoding, shape, value mix, output type and route (whole procedure on device
    buffers, on host buffers, encode + awe_gemm_planes with a forced K segment length and a padded
    leading dimension, or the entry point without allocations), compared with the oracle."""
    rng = np.random.default_rng(seed)
    name, enc, a_dt, (alo, ahi), b_dt, (blo, bhi) = CAMPAIGN_KINDS[int(rng.integers(0, len(CAMPAIGN_KINDS)))]
    M, N, K = _campaign_shape(rng)
    wide_in = a_dt in (b.I16, b.I9_IN_I16)
    np_dt = np.int16 if wide_in else np.int8
    modulus = int(rng.choice(moduli)) if enc == b.ENC_MOD_M else 0
    A = _draw(rng, alo, ahi, (M, K), np_dt, int(rng.integers(0, 4)))
    B = _draw(rng, blo, bhi, (K, N), np_dt, int(rng.integers(0, 4)))
    want = mm.matmul_i64_s16(A, B) if wide_in else mm.matmul_i64(A, B)
    if modulus:
        want = mm.mod_symmetric(want, modulus)
        out_dt = b.C_RES_I16 if rng.random() < 0.5 else b.C_RES_I32
    else:
        fits32 = max(abs(alo), ahi) * max(abs(blo), bhi) * K * 2 < 2 ** 31
        out_dt = b.C_I64 if (a_dt == b.I16 or not fits32 or rng.random() < 0.35) else b.C_I32
    h = gu.handle()
    r = rng.random()
    ws_bytes = b.awe_workspace_bytes(enc, modulus, M, N, K)
    if r < 0.15 and enc in HOST_ROUTE:
        route = "host"
        Ah, Bh = torch.from_numpy(A).pin_memory(), torch.from_numpy(B).pin_memory()
        Ch = torch.full((M, N), 77, dtype=gu.TORCH_OUT[out_dt]).pin_memory()
        sc = torch.empty(ws_bytes + b.awe_host_staging_bytes(enc, modulus, M, N, K, out_dt), dtype=torch.uint8,
                         device="cuda")
        b.awe_gemm_exact_host(h, Ah, a_dt, Bh, b_dt, M, N, K, enc, modulus, Ch, out_dt, sc)
        torch.cuda.synchronize()
        got = Ch.numpy()
    elif r < 0.3 and not wide_in and enc != b.ENC_INT8_AWE6_DERIVED:
        kc = [0, 256, 512, 1024, 4096][int(rng.integers(0, 5))]
        if modulus and kc > b.awe_encoding_info(enc, modulus).k_star // 4:
            kc = 256
        route = "planes, k_chunk %d" % kc
        ldc = N + int(rng.integers(0, 9))
        nA = b.awe_planes_bytes(enc, modulus, b.SIDE_A, M, K)
        ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
        pa, pb = ws[:nA], ws[(nA + 255) // 256 * 256:]
        b.awe_encode(h, enc, modulus, b.SIDE_A, torch.from_numpy(A).cuda(), a_dt, b.ROWMAJOR_RxK, M, K, K, pa)
        b.awe_encode(h, enc, modulus, b.SIDE_B, torch.from_numpy(B).cuda(), b_dt, b.ROWMAJOR_KxR, N, K, N, pb)
        C = torch.full((M, ldc), 77, dtype=gu.TORCH_OUT[out_dt], device="cuda")
        b.awe_gemm_planes(h, enc, modulus, pa, pb, M, N, K, C, out_dt, ldc, kc)
        torch.cuda.synchronize()
        got = C.cpu().numpy()
        assert (got[:, N:] == 77).all(), (seed, name, route, M, N, K)
        got = got[:, :N]
    elif r < 0.4 and not wide_in and not modulus and ws_bytes <= b.STATIC_WORKSPACE_BYTES:
        route = "static"
        C = torch.full((M, N), 77, dtype=gu.TORCH_OUT[out_dt], device="cuda")
        b.awe_gemm_exact_static(torch.from_numpy(A).cuda(), a_dt, torch.from_numpy(B).cuda(), b_dt, M, N, K, enc,
                                modulus, C, out_dt)
        torch.cuda.synchronize()
        got = C.cpu().numpy()
    else:
        route = "device"
        got = gu.gpu_gemm_exact(A, B, enc, out_dt, modulus=modulus, a_dt=a_dt, b_dt=b_dt)
    assert b.awe_last_device_status(h) == (0, 0), (seed, name, route, M, N, K, modulus)
    assert np.array_equal(got.astype(np.int64), want), (seed, name, route, M, N, K, modulus, out_dt)


def test_random_campaign_over_all_routes():
    """Runs random cases until the time is up: AWE_FUZZ_SECONDS (default 15) and AWE_FUZZ_SEED (default
    50000) select how long and where the seed sequence starts."""
    seconds = float(os.environ.get("AWE_FUZZ_SECONDS", "15"))
    seed = int(os.environ.get("AWE_FUZZ_SEED", "50000"))
    moduli = [m for m in range(2, 170) if b.awe_workspace_bytes(b.ENC_MOD_M, m, 256, 256, 256) > 0]
    assert len(moduli) > 100
    t_end = time.time() + seconds
    cases = 0
    while time.time() < t_end or cases < 50:
        _campaign_case(seed + cases, moduli)
        cases += 1
    print("campaign: %d cases from seed %d" % (cases, seed))
