"""The benchmark configurations at full size, through the same three C-ABI calls bench.py times.
Configuration 2 and the headline shape are compared with the CPU oracle over the WHOLE matrix (the
plain int64 product takes seconds there); the larger ones on sampled rows the oracle computes one by
one, plus properties that hold at any size: every INT8 encoding must give the same matrix, and the
residue of the exact product must equal the residue product."""
import numpy as np
import pytest
import torch

from oracle import matmul as mm
from oracle import rns
from paper_2609_24519_b200 import binding as b
from paper_2609_24519_b200 import workloads as wl
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu

TORCH_OUT = gu.TORCH_OUT


def run_three_calls(w, A, B, enc, out_dt, modulus=0, a_dt=b.I8, k_chunk=0):
    """encode A, encode B, products + reconstruction: the launch configuration bench.py times."""
    h = gu.handle()
    M, N, K = w.M, w.N, w.K
    dA, dB = torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda()
    nA = b.awe_planes_bytes(enc, modulus, b.SIDE_A, M, K)
    ws = torch.empty(b.awe_workspace_bytes(enc, modulus, M, N, K), dtype=torch.uint8, device="cuda")
    pa, pb = ws[:nA], ws[(nA + 255) // 256 * 256:]
    C = torch.full((M, N), 99, dtype=TORCH_OUT[out_dt], device="cuda")
    b.awe_encode(h, enc, modulus, b.SIDE_A, dA, a_dt, b.ROWMAJOR_RxK, M, K, K, pa)
    b.awe_encode(h, enc, modulus, b.SIDE_B, dB, b.I8, b.ROWMAJOR_KxR, N, K, N, pb)
    b.awe_gemm_planes(h, enc, modulus, pa, pb, M, N, K, C, out_dt, N, k_chunk)
    torch.cuda.synchronize()
    assert b.awe_last_device_status(h) == (0, 0)
    return C


def sampled_rows_match(C, A, B, n_rows, seed, modulus=0):
    M = A.shape[0]
    rows = sorted(set(np.random.default_rng(seed).integers(0, M, n_rows).tolist() + [0, M - 1]))
    got = C[rows].cpu().numpy().astype(np.int64)
    for i, r in enumerate(rows):
        want = mm.matmul_i64_rows(A, B, r, r + 1)[0]
        if modulus:
            want = mm.mod_symmetric(want[None], modulus)[0]
        if not np.array_equal(got[i], want):
            return False
    return True


def test_config2_awe6_and_base13_on_identical_inputs():
    w = wl.config2()
    A, B = wl.make_inputs(w)
    C6 = run_three_calls(w, A, B, b.ENC_INT8_AWE6, b.C_I32)
    assert np.array_equal(C6.cpu().numpy(), mm.matmul_i64(A, B))          # every entry, against the definition
    C9 = run_three_calls(w, A, B, b.ENC_INT8_BASE13_9, b.C_I32)
    assert torch.equal(C6, C9)
    Calt = run_three_calls(w, A, B, b.ENC_INT8_AWE6_ALT, b.C_I32)
    assert torch.equal(C6, Calt)
    # secondary, non-oracle cross-check of the whole matrix: the library INT8 tensor-core GEMM
    assert torch.equal(C6, torch._int_mm(torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda()))


def test_config3_int4_x_int8_8192():
    w = wl.config3()
    A, B = wl.make_inputs(w)
    C = run_three_calls(w, A, B, b.ENC_INT4xINT8_AWE4, b.C_I32, a_dt=b.I4_IN_I8)
    assert sampled_rows_match(C, A, B, 12, 3)
    assert torch.equal(C, torch._int_mm(torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda()))


@pytest.mark.parametrize("k_chunk", [0, 256, 4096])
def test_config4_worst_case_accumulation_int64(k_chunk):
    w = wl.config4()
    A, B = wl.make_inputs(w)
    C = run_three_calls(w, A, B, b.ENC_INT8_AWE6, b.C_I64, k_chunk=k_chunk)
    assert sampled_rows_match(C, A, B, 12, 4)
    ref = torch._int_mm(torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda())
    assert torch.equal(C, ref.to(torch.int64))


def test_config5_every_modulus_of_the_rns_set_8192():
    for m in rns.RNS_SET_FP64:
        w = wl.config5(m)
        A, B = wl.make_inputs(w)
        C = run_three_calls(w, A, B, b.ENC_MOD_M, b.C_RES_I16, modulus=m)
        assert sampled_rows_match(C, A, B, 3, m, modulus=m), m
        # whole matrix: residue of the exact product (library INT8 GEMM) equals the residue product
        ref = torch._int_mm(torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda()).to(torch.int64)
        lo = -(m // 2)
        assert torch.equal(C.to(torch.int64), (ref - lo) % m + lo), m
        del C, ref


def test_headline_8192_int8():
    w = wl.headline()
    A, B = wl.make_inputs(w)
    C = run_three_calls(w, A, B, b.ENC_INT8_AWE6, b.C_I32)
    # every entry against the definition, in row bands so the int64 reference stays small
    got = C.cpu().numpy()
    for r0 in range(0, w.M, 1024):
        assert np.array_equal(got[r0:r0 + 1024], mm.matmul_i64_rows(A, B, r0, min(w.M, r0 + 1024))), r0
    assert torch.equal(C, run_three_calls(w, A, B, b.ENC_INT8_BASE13_9, b.C_I32))
