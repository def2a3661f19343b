"""FP4 products + fused reconstruction (Algorithm 1, third loop and last step; Section 3.4;
Section 5.3) against the CPU oracle.  Integer results: the bar is bit-exact."""
import numpy as np
import pytest
import torch

from oracle import matmul as mm
from oracle import pipeline as pl
from oracle import rns
from oracle import schemes as sc
from paper_2609_24519_b200 import binding as b
from paper_2609_24519_b200 import workloads as wl
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu

INT8_ENCS = [(b.ENC_INT8_AWE6, "awe6"), (b.ENC_INT8_BASE13_9, "base13"), (b.ENC_INT8_AWE6_ALT, "alt")]


# ------------------------------------------------------------------ raw FP4 product (Section 3.4)
def _raw(X, Y):
    got = gu.gpu_fp4_raw(X, Y, pl.pack_e2m1)
    want = X.astype(np.int64) @ Y.astype(np.int64).T
    assert np.array_equal(got, want.astype(np.float32)) and np.array_equal(got.astype(np.int64), want)


def test_raw_product_random_planes():
    rng = np.random.default_rng(2)
    S = np.array(sc.S, dtype=np.int8)
    for (M, N, K) in [(128, 256, 256), (100, 200, 300), (384, 512, 4096), (1, 1, 64), (129, 257, 257)]:
        _raw(rng.choice(S, (M, K)), rng.choice(S, (N, K)))


def test_raw_product_single_nonzero_and_position():
    X = np.zeros((128, 512), dtype=np.int8)
    Y = np.zeros((256, 512), dtype=np.int8)
    X[77, 301] = -6
    Y[200, 301] = 12
    Y[13, 300] = 8
    _raw(X, Y)


def test_accumulation_is_exact_up_to_2_24():
    """Section 3.4: planes of +-12 at K = 116,480 give |P| = 144 K = 16,773,120 < 2^24."""
    K = 116480
    assert 144 * K < 2 ** 24 and K <= sc.k_star(12, 12)
    X = np.full((128, K), 12, dtype=np.int8)
    Y = np.full((256, K), 12, dtype=np.int8)
    Y[1::2] = -12
    _raw(X, Y)


def test_small_terms_survive_next_to_a_large_partial_sum():
    """Adversarial order: the sum first climbs close to 2^24, then only tiny products of
    both signs follow.  Any alignment that dropped low bits would lose them."""
    rng = np.random.default_rng(3)
    K1, K2 = 116000, 448
    X = np.full((128, K1 + K2), 12, dtype=np.int8)
    Y = np.full((256, K1 + K2), 12, dtype=np.int8)
    X[:, K1:] = rng.choice(np.array([-1, 1, 2, -3], dtype=np.int8), (128, K2))
    Y[:, K1:] = rng.choice(np.array([-1, 1, 3, -2], dtype=np.int8), (256, K2))
    X[64:, :K1] = -12                                   # half the rows climb towards -2^24
    assert 144 * K1 + 9 * K2 < 2 ** 24
    _raw(X, Y)
    # and the reverse order: small terms first, large ones after
    _raw(np.ascontiguousarray(X[:, ::-1]), np.ascontiguousarray(Y[:, ::-1]))


# ------------------------------------------------------------------ whole procedure
@pytest.mark.parametrize("enc,name", INT8_ENCS)
def test_config1_bit_exact(enc, name):
    A, B = wl.make_inputs(wl.config1())
    assert np.array_equal(gu.gpu_gemm_exact(A, B, enc, b.C_I32), mm.matmul_i64(A, B))


@pytest.mark.parametrize("shape", [(1, 1, 1), (130, 270, 300), (257, 513, 1030), (640, 768, 2304), (127, 255, 257)])
@pytest.mark.parametrize("enc,name", INT8_ENCS)
def test_ragged_shapes_int8(enc, name, shape):
    M, N, K = shape
    A, B = wl.make_inputs(wl.small("t", M, N, K, seed=M + N + K))
    want = mm.matmul_i64(A, B)
    assert np.array_equal(gu.gpu_gemm_exact(A, B, enc, b.C_I32), want)
    assert np.array_equal(gu.gpu_gemm_exact(A, B, enc, b.C_I64), want)


def test_closed_forms_on_gpu():
    K = 777
    A = np.full((130, K), -128, dtype=np.int8)
    B = np.full((K, 260), -128, dtype=np.int8)
    assert np.all(gu.gpu_gemm_exact(A, B, b.ENC_INT8_AWE6, b.C_I32) == 16384 * K)
    Bm = np.random.default_rng(3).integers(-128, 128, (200, 300), dtype=np.int8)
    C = gu.gpu_gemm_exact(np.eye(200, dtype=np.int8), Bm, b.ENC_INT8_AWE6, b.C_I32)
    assert np.array_equal(C, Bm.astype(np.int32))


def test_int4_x_int8():
    for (M, N, K) in [(256, 512, 512), (130, 270, 300)]:
        A, B = wl.make_inputs(wl.small("t", M, N, K, "int4", "int8", seed=9))
        got = gu.gpu_gemm_exact(A, B, b.ENC_INT4xINT8_AWE4, b.C_I32, a_dt=b.I4_IN_I8)
        assert np.array_equal(got, mm.matmul_i64(A, B))


def test_int4_x_int4_three_products():
    for (M, N, K) in [(256, 512, 1024), (130, 270, 300)]:
        A, B = wl.make_inputs(wl.small("t", M, N, K, "int4", "int4", seed=29))
        got = gu.gpu_gemm_exact(A, B, b.ENC_INT4xINT4_3, b.C_I32, a_dt=b.I4_IN_I8, b_dt=b.I4_IN_I8)
        assert np.array_equal(got, mm.matmul_i64(A, B))


def test_fp8_significands_three_products():
    """E4M3 significands with sign (Section 6.1): |x| <= 15 in a 5-bit container; junk above bit 4 is
    ignored; planes byte for byte against the oracle."""
    rng = np.random.default_rng(15)
    A = rng.integers(-15, 16, (300, 1000), dtype=np.int8)
    B = rng.integers(-15, 16, (1000, 270), dtype=np.int8)
    A[0, :] = -16
    B[:, 0] = -16
    want = mm.matmul_i64(A, B)
    got = gu.gpu_gemm_exact(A, B, b.ENC_FP8SIG_3, b.C_I32, a_dt=b.I5_IN_I8, b_dt=b.I5_IN_I8)
    assert np.array_equal(got.astype(np.int64), want)
    dirty = ((A.astype(np.uint8) & 0x1F) | 0xA0).astype(np.uint8).view(np.int8)
    got = gu.gpu_gemm_exact(dirty, B, b.ENC_FP8SIG_3, b.C_I32, a_dt=b.I5_IN_I8, b_dt=b.I5_IN_I8)
    assert np.array_equal(got.astype(np.int64), want)
    ref = pl.encode_planes(sc.FP8SIG_3, "A", A, -16, 15)
    packed = gu.padded_planes(np.stack([pl.pack_e2m1(p) for p in ref]), A.shape[1])
    for layout in (b.ROWMAJOR_RxK, b.ROWMAJOR_KxR):
        assert np.array_equal(gu.gpu_encode(b.ENC_FP8SIG_3, 0, b.SIDE_A, A, b.I5_IN_I8, layout), packed)


def test_ternary_x_int8():
    """Section 6.2: {0, +-1} x INT8 in 3 products (one limb against the three base-13 limbs)."""
    for (M, N, K) in [(256, 512, 1024), (130, 270, 300), (1, 1, 1)]:
        A, B = wl.make_inputs(wl.small("t", M, N, K, "ternary", "int8", seed=19))
        got = gu.gpu_gemm_exact(A, B, b.ENC_TERNARY_INT8_3, b.C_I32, a_dt=b.T2_IN_I8)
        assert np.array_equal(got, mm.matmul_i64(A, B))
        assert np.array_equal(got, pl.awe_matmul(sc.TERNARY3, A, B, a_range=(-1, 1)))
    # bytes that are not ternary values are read as 0
    A, B = wl.make_inputs(wl.small("t", 128, 256, 256, "ternary", "int8", seed=20))
    dirty = A.copy()
    dirty[::3, ::5] = 77
    clean = dirty.copy()
    clean[clean == 77] = 0
    assert np.array_equal(gu.gpu_gemm_exact(dirty, B, b.ENC_TERNARY_INT8_3, b.C_I32, a_dt=b.T2_IN_I8),
                          mm.matmul_i64(clean, B))


@pytest.mark.parametrize("m", rns.RNS_SET_FP64)
def test_residue_form_every_modulus_of_the_set(m):
    A, B = wl.make_inputs(wl.small("t", 192, 320, 1100, "residue", "residue", seed=m, modulus=m))
    want = mm.mod_symmetric(mm.matmul_i64(A, B), m)
    assert np.array_equal(gu.gpu_gemm_exact(A, B, b.ENC_MOD_M, b.C_RES_I16, modulus=m), want)
    assert np.array_equal(gu.gpu_gemm_exact(A, B, b.ENC_MOD_M, b.C_RES_I32, modulus=m), want)


@pytest.mark.parametrize("m,K,k_chunk", [(157, 49152, 256), (89, 8192, 512), (13, 4096, 256)])
def test_residue_form_with_many_k_segments(m, K, k_chunk):
    """Many exact-accumulation segments per product: the running residue sum must be reduced on
    the way (for m = 157 and 192 segments it would otherwise leave the exact float range)."""
    w = wl.small("t", 128, 256, K, "residue", "residue", seed=m, modulus=m)
    A, B = wl.make_inputs(w)
    want = mm.mod_symmetric(mm.matmul_i64(A, B), m)
    pa = gu.gpu_encode(b.ENC_MOD_M, m, b.SIDE_A, A)
    pb = gu.gpu_encode(b.ENC_MOD_M, m, b.SIDE_B, np.ascontiguousarray(B.T))
    got = gu.gpu_gemm_planes(pa, pb, w.M, w.N, w.K, b.ENC_MOD_M, b.C_RES_I16, modulus=m, k_chunk=k_chunk)
    assert np.array_equal(got, want)


def test_tall_and_wide_shapes():
    for (M, N, K) in [(5000, 64, 320), (64, 5000, 320), (3, 1030, 7), (1030, 3, 7)]:
        A, B = wl.make_inputs(wl.small("t", M, N, K, seed=M + N))
        assert np.array_equal(gu.gpu_gemm_exact(A, B, b.ENC_INT8_AWE6, b.C_I32), mm.matmul_i64(A, B))


def test_residue_form_accepts_any_int8_input():
    A, B = wl.make_inputs(wl.small("t", 128, 256, 512, seed=4))
    want = mm.mod_symmetric(mm.matmul_i64(A, B), 61)
    assert np.array_equal(gu.gpu_gemm_exact(A, B, b.ENC_MOD_M, b.C_RES_I16, modulus=61), want)


@pytest.mark.parametrize("k_chunk", [0, 256, 512, 2048])
def test_forced_k_segments_worst_case_inputs(k_chunk):
    """Section 3.4 / 6.1: segmenting K and adding the segments in integers changes nothing."""
    w = wl.small("t", 256, 512, 4096, "extreme", "extreme", seed=4)
    A, B = wl.make_inputs(w)
    want = mm.matmul_i64(A, B)
    pa = gu.gpu_encode(b.ENC_INT8_AWE6, 0, b.SIDE_A, A)
    pb = gu.gpu_encode(b.ENC_INT8_AWE6, 0, b.SIDE_B, np.ascontiguousarray(B.T))
    for out in (b.C_I32, b.C_I64):
        got = gu.gpu_gemm_planes(pa, pb, w.M, w.N, w.K, b.ENC_INT8_AWE6, out, k_chunk=k_chunk)
        assert np.array_equal(got, want)


@pytest.mark.parametrize("K", [116480, 232960])
def test_planes_of_extreme_values_at_and_beyond_k_star(K):
    """Section 3.4 through awe_gemm_planes: every stored plane value +-12 (the width-12 record, c = 12,
    K* = 116,508).  K = 116,480 fits one segment with |P| = 144 K just below 2^24; K = 232,960 must be
    cut.  Closed form: every product is +-144 K, so C = +-144 K (sum of the coefficients) / D."""
    enc = b.ENC_FP16SIG_AWE12
    d = b.awe_encoding_info(enc)
    assert d.c_a == 12 and d.c_b == 12 and d.k_star == 116508 and (K <= d.k_star) == (K == 116480)
    M, N = 40, 72
    pa = np.full((d.n_planes_a, M, K), 12, dtype=np.int8)
    pb = np.full((d.n_planes_b, N, K), 12, dtype=np.int8)
    pb[:, 1::2] = -12
    packed_a = gu.padded_planes(np.stack([pl.pack_e2m1(x) for x in pa]), K)
    packed_b = gu.padded_planes(np.stack([pl.pack_e2m1(x) for x in pb]), K)
    got = gu.gpu_gemm_planes(packed_a, packed_b, M, N, K, enc, b.C_I64)
    total = sum(int(l) for l in d.ell[:d.r]) * 144 * K
    assert total % (1 << d.log2D) == 0
    want = total >> d.log2D
    assert np.all(got[:, 0::2] == want) and np.all(got[:, 1::2] == -want)


def test_int64_output_beyond_32_bits():
    """K = 2^18 with all entries -128: C = 2^14 K = 2^32, needs the 64-bit path."""
    M, N, K = 128, 256, 1 << 18
    A = np.full((M, K), -128, dtype=np.int8)
    B = np.full((K, N), -128, dtype=np.int8)
    B[:, 1::2] = 127
    got = gu.gpu_gemm_exact(A, B, b.ENC_INT8_AWE6, b.C_I64)
    assert np.all(got[:, 0::2] == (1 << 32)) and np.all(got[:, 1::2] == -128 * 127 * K)
    with pytest.raises(b.AweError) as e:
        gu.gpu_gemm_exact(A, B, b.ENC_INT8_AWE6, b.C_I32)
    assert e.value.status == 5


def test_planes_entry_with_leading_dimension_and_guard_columns():
    w = wl.small("t", 130, 200, 300, seed=12)
    A, B = wl.make_inputs(w)
    pa = gu.gpu_encode(b.ENC_INT8_AWE6, 0, b.SIDE_A, A)
    pb = gu.gpu_encode(b.ENC_INT8_AWE6, 0, b.SIDE_B, np.ascontiguousarray(B.T))
    for ldc in (200, 203, 208):
        got = gu.gpu_gemm_planes(pa, pb, w.M, w.N, w.K, b.ENC_INT8_AWE6, b.C_I32, ldc=ldc)
        assert np.array_equal(got[:, :200], mm.matmul_i64(A, B))
        assert np.all(got[:, 200:] == 77)                  # nothing written past N


@pytest.mark.parametrize("enc,modulus,out_dt,kinds", [
    (b.ENC_INT8_AWE6, 0, b.C_I32, ("int8", "int8")),
    (b.ENC_INT8_BASE13_9, 0, b.C_I64, ("extreme", "extreme")),
    (b.ENC_INT4xINT8_AWE4, 0, b.C_I32, ("int4", "int8")),
    (b.ENC_MOD_M, 89, b.C_RES_I16, ("residue", "residue")),
])
def test_unfused_products_plus_standalone_reconstruction_equal_the_fused_kernel(enc, modulus, out_dt, kinds):
    """Algorithm 1 with its steps apart: every product k as a raw FP32 matrix (one FP4 GEMM each),
    then the stand-alone reconstruction -- must equal the fused kernel and the oracle."""
    h = gu.handle()
    w = wl.small("t", 200, 333, 900, kinds[0], kinds[1], seed=27, modulus=modulus)
    A, B = wl.make_inputs(w)
    d = b.awe_encoding_info(enc, modulus)
    a_dt = b.I4_IN_I8 if enc == b.ENC_INT4xINT8_AWE4 else b.I8
    pa = gu.gpu_encode(enc, modulus, b.SIDE_A, A, a_dt)
    pb = gu.gpu_encode(enc, modulus, b.SIDE_B, np.ascontiguousarray(B.T))
    dpa, dpb = torch.from_numpy(pa).cuda(), torch.from_numpy(pb).cuda()
    ldp = 336
    P = torch.zeros((d.r, w.M, ldp), dtype=torch.float32, device="cuda")
    for k in range(d.r):
        b.awe_fp4_product_raw(h, dpa[d.ia[k]], dpb[d.ib[k]], w.M, w.N, w.K, P[k], ldp)
    C = torch.full((w.M, w.N), 9, dtype=gu.TORCH_OUT[out_dt], device="cuda")
    b.awe_reconstruct(h, enc, modulus, P, w.M * ldp, ldp, w.M, w.N, C, out_dt, w.N)
    torch.cuda.synchronize()
    want = mm.matmul_i64(A, B)
    if modulus:
        want = mm.mod_symmetric(want, modulus)
    assert np.array_equal(C.cpu().numpy().astype(np.int64), want)
    fused = gu.gpu_gemm_exact(A, B, enc, out_dt, modulus=modulus, a_dt=a_dt)
    assert np.array_equal(fused, C.cpu().numpy())


def test_results_are_reproducible_run_to_run():
    A, B = wl.make_inputs(wl.small("t", 512, 768, 2048, seed=31))
    first = gu.gpu_gemm_exact(A, B, b.ENC_INT8_AWE6, b.C_I32)
    for _ in range(10):
        assert np.array_equal(gu.gpu_gemm_exact(A, B, b.ENC_INT8_AWE6, b.C_I32), first)


def test_host_buffer_entry_point():
    h = gu.handle()
    w = wl.small("t", 300, 520, 1000, seed=17)
    A, B = wl.make_inputs(w)
    Ah, Bh = torch.from_numpy(A).pin_memory(), torch.from_numpy(B).pin_memory()
    Ch = torch.zeros((w.M, w.N), dtype=torch.int32).pin_memory()
    nbytes = b.awe_workspace_bytes(b.ENC_INT8_AWE6, 0, w.M, w.N, w.K) + \
        b.awe_host_staging_bytes(b.ENC_INT8_AWE6, 0, w.M, w.N, w.K, b.C_I32)
    scratch = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    b.awe_gemm_exact_host(h, Ah, b.I8, Bh, b.I8, w.M, w.N, w.K, b.ENC_INT8_AWE6, 0, Ch, b.C_I32, scratch)
    assert np.array_equal(Ch.numpy(), mm.matmul_i64(A, B))


@pytest.mark.parametrize("enc,out_dt,tdt,modulus,kinds", [
    (b.ENC_INT8_AWE6, b.C_I32, torch.int32, 0, ("int8", "int8")),
    (b.ENC_INT8_AWE6, b.C_I64, torch.int64, 0, ("extreme", "extreme")),
    (b.ENC_MOD_M, b.C_RES_I16, torch.int16, 89, ("residue", "residue")),
])
def test_host_buffer_entry_point_chunked(enc, out_dt, tdt, modulus, kinds):
    """M large enough that the rows go through in several overlapped chunks (ragged last chunk)."""
    h = gu.handle()
    w = wl.small("t", 3300, 520, 700, kinds[0], kinds[1], seed=23, modulus=modulus)
    A, B = wl.make_inputs(w)
    Ah, Bh = torch.from_numpy(A).pin_memory(), torch.from_numpy(B).pin_memory()
    Ch = torch.full((w.M, w.N), 5, dtype=tdt).pin_memory()
    nbytes = b.awe_workspace_bytes(enc, modulus, w.M, w.N, w.K) + \
        b.awe_host_staging_bytes(enc, modulus, w.M, w.N, w.K, out_dt)
    scratch = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    want = mm.matmul_i64(A, B)
    if modulus:
        want = mm.mod_symmetric(want, modulus)
    for _ in range(2):                                  # the second call reuses the handle's copy streams
        Ch.fill_(5)
        b.awe_gemm_exact_host(h, Ah, b.I8, Bh, b.I8, w.M, w.N, w.K, enc, modulus, Ch, out_dt, scratch)
        assert np.array_equal(Ch.numpy().astype(np.int64), want)
    assert b.awe_last_device_status(h) == (0, 0)
    # pageable host memory works too
    Cp = np.zeros((w.M, w.N), dtype=Ch.numpy().dtype)
    b.awe_gemm_exact_host(h, A, b.I8, B, b.I8, w.M, w.N, w.K, enc, modulus, Cp, out_dt, scratch)
    assert np.array_equal(Cp.astype(np.int64), want)


@pytest.mark.parametrize("enc,out_dt,tdt,kinds,a_dt", [
    (b.ENC_INT8_AWE6, b.C_I32, torch.int32, ("int8", "int8"), b.I8),
    (b.ENC_INT8_MIXED_FP8_3, b.C_I64, torch.int64, ("int8", "int8"), b.I8),
    (b.ENC_INT4xINT8_AWE4, b.C_I32, torch.int32, ("int4", "int8"), b.I4_IN_I8),
])
def test_host_buffer_entry_point_row_chunks_and_column_blocks(enc, out_dt, tdt, kinds, a_dt):
    """M and N large enough for several row chunks and several column blocks, both ragged: the blocks
    of C come back through two-dimensional copies and must tile the matrix exactly."""
    h = gu.handle()
    w = wl.small("t", 4500, 6400, 300, kinds[0], kinds[1], seed=29)
    A, B = wl.make_inputs(w)
    Ah, Bh = torch.from_numpy(A).pin_memory(), torch.from_numpy(B).pin_memory()
    Ch = torch.full((w.M, w.N), 5, dtype=tdt).pin_memory()
    nbytes = b.awe_workspace_bytes(enc, 0, w.M, w.N, w.K) + b.awe_host_staging_bytes(enc, 0, w.M, w.N, w.K, out_dt)
    scratch = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    b.awe_gemm_exact_host(h, Ah, a_dt, Bh, b.I8, w.M, w.N, w.K, enc, 0, Ch, out_dt, scratch)
    assert b.awe_last_device_status(h) == (0, 0)
    got = Ch.numpy().astype(np.int64)
    rows = [0, 511, 512, 1023, 1024, 2047, 2048, 2303, 4095, 4096, 4499]      # both sides of every chunk edge
    assert np.array_equal(got[rows], mm.matmul_i64(A[rows], B))
    cols = [0, 2047, 2048, 2559, 2560, 3071, 3072, 4095, 4096, 6143, 6144, 6399]
    assert np.array_equal(got[:, cols], mm.matmul_i64(A, np.ascontiguousarray(B[:, cols])))
    # whole matrix against the device-buffer entry point
    assert np.array_equal(got, gu.gpu_gemm_exact(A, B, enc, out_dt, a_dt=a_dt).astype(np.int64))


def test_merged_accumulators_stay_exact_at_their_bound():
    """Section 3.4 with n_g > 1: base-13 has up to three products of equal coefficient, which share one
    accumulator when 3 * 8 * 8 * K < 2^24.  All-(+8) planes at the largest such K (a multiple of 256)
    put 16,760,832 into the merged accumulators; one K block further the library no longer merges.
    The planes are not images of int8 data, so the 32-bit result is compared modulo 2^32."""
    enc = b.ENC_INT8_BASE13_9
    d = b.awe_encoding_info(enc)
    assert (d.c_a, d.c_b, d.r) == (8, 8, 9)
    coeff = sum(int(d.ell[k]) for k in range(d.r))
    assert coeff == (1 + 13 + 169) ** 2
    M, N = 128, 256
    for K in (87296, 87552):
        assert (3 * 64 * K < 2 ** 24) == (K == 87296)
        planes = lambda R: np.full((3, R, gu.pitch_bytes(K)), 0x66, dtype=np.uint8)   # E2M1 code 6 = 4.0 -> 8
        got = gu.gpu_gemm_planes(planes(M), planes(N), M, N, K, enc, b.C_I32)
        want = np.int64(64 * K * coeff)
        assert np.all(got.astype(np.int64) & 0xFFFFFFFF == int(want) & 0xFFFFFFFF)


def test_equal_coefficient_products_with_real_inputs_and_long_k():
    """x = 112 = 8 + 13 * 8 on both sides: the merged pair (a0 b1 + a1 b0) is as large as int8 inputs can
    make it; K just below and above the merging bound of base-13, and the 12-product record alike."""
    for K in (87296, 87552):
        A = np.full((130, K), 112, dtype=np.int8)
        B = np.full((K, 140), -112, dtype=np.int8)
        B[:, ::2] = 112
        want = mm.matmul_i64(A, B)
        assert np.array_equal(gu.gpu_gemm_exact(A, B, b.ENC_INT8_BASE13_9, b.C_I64), want)


def test_int32_output_next_to_the_range_limit_of_the_record_with_D_2():
    """INT4 x INT8 in 4 products has D = 2 (Appendix A): the 32-bit sums hold 2 C, so int32 output is
    served while 2 * 8 * 128 * K < 2^31.  K = 2^20 - 256 with the extreme inputs (C = 2^30 - 2^18) is the
    largest served multiple of 256 and must be exact; K = 2^20 is refused."""
    K = 2 ** 20 - 256
    A = np.full((8, K), -8, dtype=np.int8)
    B = np.full((K, 24), -128, dtype=np.int8)
    B[:, 1::2] = 127
    got = gu.gpu_gemm_exact(A, B, b.ENC_INT4xINT8_AWE4, b.C_I32, a_dt=b.I4_IN_I8)
    want = mm.matmul_i64(A, B)
    assert want.max() == 2 ** 30 - 2 ** 18 and np.array_equal(got, want)
    h = gu.handle()
    x = torch.zeros(16, dtype=torch.int8, device="cuda")
    with pytest.raises(b.AweError) as e:
        b.awe_gemm_exact(h, x, b.I4_IN_I8, x, b.I8, 8, 24, 2 ** 20, b.ENC_INT4xINT8_AWE4, 0, x.view(torch.int32), b.C_I32,
                         torch.empty(b.awe_workspace_bytes(b.ENC_INT4xINT8_AWE4, 0, 8, 24, 2 ** 20), dtype=torch.uint8,
                                     device="cuda"))
    assert e.value.status == 5


def test_argument_errors_are_reported_before_any_launch():
    h = gu.handle()
    n0 = b.awe_launch_count(h)
    A = torch.zeros((256, 256), dtype=torch.int8, device="cuda")
    C = torch.zeros((256, 256), dtype=torch.int32, device="cuda")
    ws = torch.empty(b.awe_workspace_bytes(b.ENC_INT8_AWE6, 0, 256, 256, 256) + 256, dtype=torch.uint8, device="cuda")
    def call(**kw):
        args = dict(A=A, a_dt=b.I8, B=A, b_dt=b.I8, M=256, N=256, K=256, enc=b.ENC_INT8_AWE6, modulus=0, C=C,
                    out_dt=b.C_I32, workspace=ws)
        args.update(kw)
        b.awe_gemm_exact(h, **args)
    for kw, status in [(dict(M=0), 1), (dict(enc=99), 2), (dict(modulus=7), 2), (dict(out_dt=b.C_RES_I16), 2),
                       (dict(workspace=ws[:1024]), 3), (dict(workspace=ws[1:]), 4), (dict(A=None), 1),
                       (dict(enc=b.ENC_INT4xINT8_AWE4), 2)]:     # int8 data on the int4 side
        with pytest.raises(b.AweError) as e:
            call(**kw)
        assert e.value.status == status, kw
    with pytest.raises(b.AweError):
        b.awe_encoding_info(b.ENC_MOD_M, 170)
    assert b.awe_launch_count(h) == n0


def test_a_wait_that_runs_out_is_reported_and_the_handle_stays_usable():
    """Failure path without a fault: a bounded wait on a barrier nothing signals gives up after its
    budget, the kernel returns, the host reads AWE_ERR_TIMEOUT + site, and work continues."""
    import time
    h = b.awe_create(0)
    t0 = time.time()
    b.awe_selftest_bounded_wait(h, 2000)                       # 2 ms budget
    assert b.awe_last_device_status(h) == (7, 1000)
    assert time.time() - t0 < 5.0
    assert b.awe_last_device_status(h) == (0, 0)               # the read cleared it
    A, B = wl.make_inputs(wl.small("t", 128, 256, 256, seed=33))
    ws = torch.empty(b.awe_workspace_bytes(b.ENC_INT8_AWE6, 0, 128, 256, 256), dtype=torch.uint8, device="cuda")
    C = torch.zeros((128, 256), dtype=torch.int32, device="cuda")
    b.awe_gemm_exact(h, torch.from_numpy(A).cuda(), b.I8, torch.from_numpy(B).cuda(), b.I8, 128, 256, 256,
                     b.ENC_INT8_AWE6, 0, C, b.C_I32, ws)
    torch.cuda.synchronize()
    assert b.awe_last_device_status(h) == (0, 0)
    assert np.array_equal(C.cpu().numpy(), mm.matmul_i64(A, B))
    b.awe_destroy(h)


def test_whole_procedure_can_be_captured_in_a_cuda_graph_and_replayed():
    """After the first call (which uploads the tables) awe_gemm_exact only enqueues kernels, so a
    launch-bound small product can be captured once and replayed."""
    h = gu.handle()
    w = wl.config1()
    A, B = wl.make_inputs(w)
    dA, dB = torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda()
    ws = torch.empty(b.awe_workspace_bytes(b.ENC_INT8_AWE6, 0, w.M, w.N, w.K), dtype=torch.uint8, device="cuda")
    C = torch.zeros((w.M, w.N), dtype=torch.int32, device="cuda")
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        b.awe_gemm_exact(h, dA, b.I8, dB, b.I8, w.M, w.N, w.K, b.ENC_INT8_AWE6, 0, C, b.C_I32, ws)   # warm-up
    side.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        b.awe_gemm_exact(h, dA, b.I8, dB, b.I8, w.M, w.N, w.K, b.ENC_INT8_AWE6, 0, C, b.C_I32, ws)
    want = mm.matmul_i64(A, B)
    for rep in range(3):
        dA.copy_(torch.from_numpy(np.roll(A, rep, axis=0)).cuda())       # new data, same buffers
        C.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert np.array_equal(C.cpu().numpy(), np.roll(want, rep, axis=0))
    assert b.awe_last_device_status(h) == (0, 0)
