"""Wide-integer product through the residue number system (Section 5.3): residues, the 22
per-modulus products on the FP4 kernels, CRT -- against the oracle's Python-integer results."""
import math

import numpy as np
import pytest
import torch

from oracle import rns
from paper_2609_24519_b200 import binding as b
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu

B53 = 2 ** 53 - 1


def _to_python_ints(C128: np.ndarray) -> np.ndarray:
    """M x N x 2 int64 (low word, high word) -> object array of Python integers."""
    lo = C128[..., 0].astype(np.uint64).astype(object)
    hi = C128[..., 1].astype(object)
    return hi * (1 << 64) + lo


def _wide_inputs(M, N, K, seed):
    rng = np.random.default_rng(seed)
    A = rng.integers(-B53, B53 + 1, (M, K), dtype=np.int64)
    B = rng.integers(-B53, B53 + 1, (K, N), dtype=np.int64)
    return A, B


def test_moduli_are_the_oracle_set():
    assert tuple(b.awe_wide_moduli()) == rns.RNS_SET_FP64


def test_residues_kernel():
    h = gu.handle()
    rng = np.random.default_rng(1)
    for count in (1, 7, 4096, 100003):
        X = rng.integers(-B53, B53 + 1, count, dtype=np.int64)
        X[:3] = [B53, -B53, 0][:min(3, count)]
        res = torch.empty((len(rns.RNS_SET_FP64), count), dtype=torch.int8, device="cuda")
        b.awe_wide_residues(h, torch.from_numpy(X).cuda(), count, res)
        got = res.cpu().numpy()
        for t, m in enumerate(rns.RNS_SET_FP64):
            lo = -(m // 2)
            want = ((X.astype(object) - lo) % m + lo).astype(np.int8)
            assert np.array_equal(got[t], want), (count, m)


def test_crt_kernel():
    h = gu.handle()
    rng = np.random.default_rng(2)
    M = math.prod(rns.RNS_SET_FP64)
    xs = [0, 1, -1, M // 2, -(M // 2) + 1, 9 * B53 * B53, -59000 * B53 * B53]   # representatives lie in (-M/2, M/2]
    xs += [int(rng.integers(-2 ** 62, 2 ** 62)) * int(rng.integers(1, 2 ** 59)) + int(rng.integers(0, 2 ** 50))
           for _ in range(500)]
    assert all(abs(x) <= M // 2 for x in xs)
    res = np.array([[((x + m // 2) % m) - m // 2 for x in xs] for m in rns.RNS_SET_FP64], dtype=np.int16)
    out = torch.empty((len(xs), 2), dtype=torch.int64, device="cuda")
    b.awe_wide_crt(h, torch.from_numpy(res).cuda(), len(xs), out)
    got = _to_python_ints(out.cpu().numpy())
    assert [int(g) for g in got] == xs
    assert [rns.crt_symmetric(res[:, i], rns.RNS_SET_FP64) for i in range(20)] == xs[:20]
    # an even count takes the path with one 4-byte load per modulus and pair of elements
    assert len(xs) % 2 == 1
    even = torch.empty((len(xs) - 1, 2), dtype=torch.int64, device="cuda")
    b.awe_wide_crt(h, torch.from_numpy(np.ascontiguousarray(res[:, :-1])).cuda(), len(xs) - 1, even)
    assert [int(g) for g in _to_python_ints(even.cpu().numpy())] == xs[:-1]
    # other representatives of the same residue classes give the same integers
    # (|r| < m: the non-negative one, or that minus m)
    shifted = np.array([[x % m - (m if (i + m) % 3 == 0 and x % m else 0) for i, x in enumerate(xs)]
                        for m in rns.RNS_SET_FP64], dtype=np.int16)
    assert (np.abs(shifted) < np.array(rns.RNS_SET_FP64)[:, None]).all() and (shifted < 0).any()
    b.awe_wide_crt(h, torch.from_numpy(shifted).cuda(), len(xs), out)
    assert [int(g) for g in _to_python_ints(out.cpu().numpy())] == xs


def test_residues_of_values_on_the_rounding_boundaries():
    """x = q m + r for every symmetric residue r of every modulus, at small and at 53-bit magnitudes and
    both signs: covers the ties of the even modulus and the ends of every range."""
    h = gu.handle()
    xs = []
    for m in rns.RNS_SET_FP64:
        for r in range(-(m // 2), (m + 1) // 2):
            for q in (0, 1, -1, 3, (B53 // m) - 2, -((B53 // m) - 2), 2 ** 40 + 1, -(2 ** 40) - 5):
                xs.append(q * m + r)
    X = np.array(xs, dtype=np.int64)
    assert np.abs(X).max() <= B53
    res = torch.empty((len(rns.RNS_SET_FP64), len(xs)), dtype=torch.int8, device="cuda")
    b.awe_wide_residues(h, torch.from_numpy(X).cuda(), len(xs), res)
    got = res.cpu().numpy()
    for t, m in enumerate(rns.RNS_SET_FP64):
        lo = -(m // 2)
        want = ((X.astype(object) - lo) % m + lo).astype(np.int8)
        assert np.array_equal(got[t], want), m


@pytest.mark.parametrize("shape", [(1, 1, 1), (60, 40, 200), (130, 270, 513)])
def test_wide_product_equals_python_integers(shape):
    h = gu.handle()
    M, N, K = shape
    A, B = _wide_inputs(M, N, K, seed=M + K)
    A[0, :] = B53
    B[:, 0] = -B53                                    # the extreme entry: -K (2^53 - 1)^2
    ws = torch.empty(b.awe_wide_workspace_bytes(M, N, K), dtype=torch.uint8, device="cuda")
    C = torch.zeros((M, N, 2), dtype=torch.int64, device="cuda")
    b.awe_gemm_exact_wide(h, torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda(), M, N, K, 54, C, ws)
    torch.cuda.synchronize()
    assert b.awe_last_device_status(h) == (0, 0)
    got = _to_python_ints(C.cpu().numpy())
    want = rns.wide_matmul(A, B)
    assert want[0, 0] == -K * B53 * B53
    assert all(int(got[i]) == int(want[i]) for i in np.ndindex(M, N))


@pytest.mark.parametrize("bits,K", [(32, 700), (24, 300), (12, 2000), (5, 64)])
def test_narrower_inputs_use_a_cheaper_subset_and_stay_exact(bits, K):
    h = gu.handle()
    M, N = 70, 90
    Bd = 2 ** (bits - 1) - 1
    rng = np.random.default_rng(bits)
    A = rng.integers(-Bd, Bd + 1, (M, K), dtype=np.int64)
    B = rng.integers(-Bd, Bd + 1, (K, N), dtype=np.int64)
    A[0, :], B[:, 0] = Bd, -Bd
    sel = b.awe_wide_select(bits, K)
    assert 0 < len(sel) < len(rns.RNS_SET_FP64)
    ws = torch.empty(b.awe_wide_workspace_bytes(M, N, K), dtype=torch.uint8, device="cuda")
    C = torch.zeros((M, N, 2), dtype=torch.int64, device="cuda")
    b.awe_gemm_exact_wide(h, torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda(), M, N, K, bits, C, ws)
    got = _to_python_ints(C.cpu().numpy())
    want = rns.wide_matmul(A, B)
    assert all(int(got[i]) == int(want[i]) for i in np.ndindex(M, N))


def test_wide_product_agrees_with_the_oracle_pipeline_on_a_tiny_case():
    h = gu.handle()
    A, B = _wide_inputs(4, 3, 6, seed=5)
    ws = torch.empty(b.awe_wide_workspace_bytes(4, 3, 6), dtype=torch.uint8, device="cuda")
    C = torch.zeros((4, 3, 2), dtype=torch.int64, device="cuda")
    b.awe_gemm_exact_wide(h, torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda(), 4, 3, 6, 54, C, ws)
    got = _to_python_ints(C.cpu().numpy())
    want = rns.rns_matmul(A, B)
    assert all(int(got[i]) == int(want[i]) for i in np.ndindex(4, 3))


def test_wide_product_refuses_k_beyond_the_uniqueness_bound():
    h = gu.handle()
    x = torch.zeros(64, dtype=torch.int64, device="cuda")
    ws = torch.empty(1 << 20, dtype=torch.uint8, device="cuda")
    with pytest.raises(b.AweError) as e:              # 2 K B^2 >= prod(m) for width 54 at K = 70,000
        b.awe_gemm_exact_wide(h, x, x, 1, 1, 70000, 54, x, ws)
    assert e.value.status == 5
    with pytest.raises(b.AweError) as e:
        b.awe_gemm_exact_wide(h, x, x, 8, 8, 8, 55, x, ws)
    assert e.value.status == 1


def test_wide_product_8192_sampled_entries():
    h = gu.handle()
    M = N = K = 8192
    gen = torch.Generator(device="cuda")
    gen.manual_seed(11)
    A = torch.randint(-B53, B53 + 1, (M, K), dtype=torch.int64, device="cuda", generator=gen)
    B = torch.randint(-B53, B53 + 1, (K, N), dtype=torch.int64, device="cuda", generator=gen)
    ws = torch.empty(b.awe_wide_workspace_bytes(M, N, K), dtype=torch.uint8, device="cuda")
    C = torch.zeros((M, N, 2), dtype=torch.int64, device="cuda")
    b.awe_gemm_exact_wide(h, A, B, M, N, K, 54, C, ws)
    torch.cuda.synchronize()
    assert b.awe_last_device_status(h) == (0, 0)
    rng = np.random.default_rng(3)
    for _ in range(24):
        i, j = int(rng.integers(0, M)), int(rng.integers(0, N))
        a = A[i].cpu().numpy().astype(object)
        bb = B[:, j].cpu().numpy().astype(object)
        got = _to_python_ints(C[i, j].cpu().numpy()[None])[0]
        assert int(got) == int((a * bb).sum())
