"""The 12-product encoding of width-12 integers (FP16 significands with sign, Appendix A):
16-bit inputs, 6 planes per side, D = 2, 64-bit reconstruction -- against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import matmul as mm
from oracle import pipeline as pl
from oracle import schemes as sc
from paper_2609_24519_b200 import binding as b
from paper_2609_24519_b200 import workloads as wl
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu
ENC = b.ENC_FP16SIG_AWE12


def _want_planes(side, X):
    ref = pl.encode_planes(sc.FP16_M12, side, X, -2047, 2047)
    return gu.padded_planes(np.stack([pl.pack_e2m1(p) for p in ref]), X.shape[1])


@pytest.mark.parametrize("shape", [(1, 1), (70, 333), (256, 2048), (131, 1025)])
def test_encode_16_bit_operands_both_layouts(shape):
    R, K = shape
    X = np.random.default_rng(R + K).integers(-2047, 2048, (R, K), dtype=np.int16)
    for side, name in ((b.SIDE_A, "A"), (b.SIDE_B, "B")):
        want = _want_planes(name, X)
        for layout in (b.ROWMAJOR_RxK, b.ROWMAJOR_KxR):
            for ld_extra, offset in ((0, 0), (3, 1)):
                got = gu.gpu_encode(ENC, 0, side, X, b.I16, layout, ld_extra, offset)
                assert np.array_equal(got, want), (name, layout, ld_extra, offset)


def _run(A, B, out_dt):
    return gu.gpu_gemm_exact(A, B, ENC, out_dt, a_dt=b.I16, b_dt=b.I16)


@pytest.mark.parametrize("shape", [(1, 1, 1), (130, 270, 300), (256, 384, 2048), (257, 129, 1030)])
def test_products_of_width_12_integers(shape):
    M, N, K = shape
    A, B = wl.make_inputs(wl.small("t", M, N, K, "int12", "int12", seed=M + K))
    want = mm.matmul_i64_s16(A, B)
    assert np.array_equal(_run(A, B, b.C_I64), want)
    if 2048 * 2048 * K < 2 ** 31:
        assert np.array_equal(_run(A, B, b.C_I32), want)
    else:
        with pytest.raises(b.AweError) as e:
            _run(A, B, b.C_I32)
        assert e.value.status == 5


def test_extreme_significands_need_more_than_32_bits():
    M, N, K = 128, 128, 4096
    A = np.full((M, K), 2047, dtype=np.int16)
    B = np.full((K, N), -2047, dtype=np.int16)
    B[:, 1::2] = 2047
    got = _run(A, B, b.C_I64)
    assert np.all(got[:, 0::2] == -2047 * 2047 * K) and np.all(got[:, 1::2] == 2047 * 2047 * K)
    assert 2047 * 2047 * K > 2 ** 33


def test_matches_algorithm_1_on_the_cpu_and_only_low_12_bits_are_read():
    A, B = wl.make_inputs(wl.small("t", 40, 30, 200, "int12", "int12", seed=3))
    want = pl.awe_matmul(sc.FP16_M12, A, B, a_range=(-2047, 2047), b_range=(-2047, 2047))
    assert np.array_equal(_run(A, B, b.C_I64), want)
    dirty = ((A.astype(np.uint16) & 0xFFF) | 0x5000).astype(np.uint16).view(np.int16)   # junk above bit 11
    assert np.array_equal(_run(dirty, B, b.C_I64), want)


def test_fp16sig_8192_sampled_rows():
    h = gu.handle()
    w = wl.small("t", 8192, 8192, 8192, "int12", "int12", seed=8)
    A, B = wl.make_inputs(w)
    ws = torch.empty(b.awe_workspace_bytes(ENC, 0, w.M, w.N, w.K), dtype=torch.uint8, device="cuda")
    C = torch.zeros((w.M, w.N), dtype=torch.int64, device="cuda")
    b.awe_gemm_exact(h, torch.from_numpy(A).cuda(), b.I16, torch.from_numpy(B).cuda(), b.I16, w.M, w.N, w.K, ENC, 0, C,
                     b.C_I64, ws)
    torch.cuda.synchronize()
    assert b.awe_last_device_status(h) == (0, 0)
    for r in (0, 4097, 8191):
        assert np.array_equal(C[r].cpu().numpy(), mm.matmul_i64_s16(A, B, r, r + 1)[0])


def test_bf16_significands_eight_products():
    """Width-9 integers (BF16 significands with sign) in a 16-bit container: planes byte for byte, junk
    above bit 8 ignored, 32- and 64-bit outputs, K long enough for several 64-bit launches."""
    enc = b.ENC_BF16SIG_8
    rng = np.random.default_rng(19)
    A = rng.integers(-255, 256, (300, 1000), dtype=np.int16)
    B = rng.integers(-255, 256, (1000, 270), dtype=np.int16)
    A[0, :] = -256
    B[:, 0] = -256
    want = mm.matmul_i64_s16(A, B)
    run = lambda X, Y, out: gu.gpu_gemm_exact(X, Y, enc, out, a_dt=b.I9_IN_I16, b_dt=b.I9_IN_I16).astype(np.int64)
    assert np.array_equal(run(A, B, b.C_I32), want)
    assert np.array_equal(run(A, B, b.C_I64), want)
    dirty = ((A.astype(np.uint16) & 0x1FF) | 0x5A00).astype(np.uint16).view(np.int16)
    assert np.array_equal(run(dirty, B, b.C_I64), want)
    ref = pl.encode_planes(sc.BF16SIG_8, "A", A, -256, 255)
    packed = gu.padded_planes(np.stack([pl.pack_e2m1(p) for p in ref]), A.shape[1])
    for layout in (b.ROWMAJOR_RxK, b.ROWMAJOR_KxR):
        assert np.array_equal(gu.gpu_encode(enc, 0, b.SIDE_A, A, b.I9_IN_I16, layout), packed)
    # extremes over a K that needs 64 bits and several launches
    K = 40000
    A = rng.choice(np.array([-256, 255], np.int16), (130, K))
    B = rng.choice(np.array([-256, 255], np.int16), (K, 140))
    A[0, :] = -256
    B[:, 0] = -256
    want = mm.matmul_i64_s16(A, B)
    assert want[0, 0] == 65536 * K > 2 ** 31
    assert np.array_equal(run(A, B, b.C_I64), want)
    with pytest.raises(b.AweError):
        run(A, B, b.C_I32)


def test_long_k_runs_in_several_launches_and_keeps_every_cell_within_32_bits():
    """K beyond the length over which a cell of the grouped reconstruction fits 32 bits (37,120):
    the launches add into the 64-bit result; all-extreme inputs (including -2048) make every cell as
    large as it can get."""
    M, N, K = 256, 128, 45000
    rng = np.random.default_rng(77)
    A = rng.choice(np.array([-2048, 2047], np.int16), (M, K))
    B = rng.choice(np.array([-2048, 2047], np.int16), (K, N))
    A[0, :] = -2048
    B[:, 0] = -2048
    want = mm.matmul_i64_s16(A, B)
    assert want[0, 0] == 2048 * 2048 * K
    assert np.array_equal(_run(A, B, b.C_I64), want)


def test_many_tiles_per_worker_both_product_orders():
    """More tiles than workers: every worker walks the products forwards on one tile and backwards on
    the next, so the groups reach C in either order."""
    M, N, K = 2560, 2816, 512
    A, B = wl.make_inputs(wl.small("t", M, N, K, "int12", "int12", seed=9))
    got = _run(A, B, b.C_I64)
    rows = [0, 255, 256, 1279, 2559]
    want = mm.matmul_i64_s16(A[rows], B)
    assert np.array_equal(got[rows], want)
    cols = [0, 255, 256, 2815]
    assert np.array_equal(got[:, cols], mm.matmul_i64_s16(A, np.ascontiguousarray(B[:, cols])))
