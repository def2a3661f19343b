"""awe_gemm_exact_static -- the entry point for callers that may not allocate device memory --
against awe_gemm_exact and against the CPU oracle, through the C ABI, bit for bit, on two calls in a
row.

Kept in a file that sorts last so that a run stopping at the first failure has already run every
other test.  The check is self-contained: it passes alone in a fresh process and after the others."""
import numpy as np
import pytest
import torch

from oracle import matmul as mm
from paper_2609_24519_b200 import binding as b
from paper_2609_24519_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _reference(h, A, B, enc, out_dt, tdt, modulus=0, a_dt=b.I8):
    M, K = A.shape
    N = B.shape[1]
    ws = torch.empty(b.awe_workspace_bytes(enc, modulus, M, N, K), dtype=torch.uint8, device="cuda")
    C = torch.zeros((M, N), dtype=tdt, device="cuda")
    b.awe_gemm_exact(h, A, a_dt, B, b.I8, M, N, K, enc, modulus, C, out_dt, ws)
    torch.cuda.synchronize()
    return C


def test_static_scratch_entry_matches_awe_gemm_exact_twice_in_a_row():
    h = b.awe_create(0)
    cases = [
        (wl.small("na1", 384, 520, 1300, seed=41), b.ENC_INT8_AWE6, b.C_I32, torch.int32, 0, b.I8),
        (wl.small("na2", 200, 260, 700, "residue", "residue", seed=42, modulus=89), b.ENC_MOD_M, b.C_RES_I16,
         torch.int16, 89, b.I8),
        (wl.small("na3", 300, 260, 900, seed=43), b.ENC_INT8_MIXED_FP8_3, b.C_I32, torch.int32, 0, b.I8),
    ]
    for w, enc, out_dt, tdt, modulus, a_dt in cases:          # two calls in a row share the one array
        A_np, B_np = wl.make_inputs(w)
        A, B = torch.from_numpy(A_np).cuda(), torch.from_numpy(B_np).cuda()
        want = _reference(h, A, B, enc, out_dt, tdt, modulus, a_dt)
        got = torch.full((w.M, w.N), 55, dtype=tdt, device="cuda")
        b.awe_gemm_exact_static(A, a_dt, B, b.I8, w.M, w.N, w.K, enc, modulus, got, out_dt)
        torch.cuda.synchronize()
        assert torch.equal(got, want), w.name
        exact = mm.matmul_i64(A_np, B_np)                     # the definition: plain int64 product
        if modulus:
            exact = mm.mod_symmetric(exact, modulus)
        assert np.array_equal(got.cpu().numpy().astype(np.int64), exact), w.name
    # the same problem again: stale planes of the previous (different) problem are in the array
    w, enc, out_dt, tdt, modulus, a_dt = cases[0]
    A_np, B_np = wl.make_inputs(w)
    A, B = torch.from_numpy(A_np).cuda(), torch.from_numpy(B_np).cuda()
    got = torch.full((w.M, w.N), 55, dtype=tdt, device="cuda")
    b.awe_gemm_exact_static(A, a_dt, B, b.I8, w.M, w.N, w.K, enc, modulus, got, out_dt)
    torch.cuda.synchronize()
    assert torch.equal(got, _reference(h, A, B, enc, out_dt, tdt, modulus, a_dt))
    assert np.array_equal(got.cpu().numpy().astype(np.int64), mm.matmul_i64(A_np, B_np))
    b.awe_destroy(h)


def test_static_scratch_entry_does_not_wait_for_other_streams_and_replays_from_a_graph():
    """The call never blocks on the GPU: with a long kernel queue on another stream it returns at once
    and its product still completes correctly on its own stream.  A warmed-up call recorded into a
    graph gives the right product on every replay."""
    w = wl.small("na4", 256, 384, 1024, seed=44)
    A_np, B_np = wl.make_inputs(w)
    A, B = torch.from_numpy(A_np).cuda(), torch.from_numpy(B_np).cuda()
    want = mm.matmul_i64(A_np, B_np)
    C = torch.zeros((w.M, w.N), dtype=torch.int32, device="cuda")
    side, busy = torch.cuda.Stream(), torch.cuda.Stream()
    with torch.cuda.stream(side):
        b.awe_gemm_exact_static(A, b.I8, B, b.I8, w.M, w.N, w.K, b.ENC_INT8_AWE6, 0, C, b.C_I32)   # warm-up
    side.synchronize()
    big = torch.empty(1 << 28, dtype=torch.uint8, device="cuda")
    with torch.cuda.stream(busy):
        for _ in range(200):
            big.fill_(1)                                       # tens of milliseconds of queued work
    C.zero_()
    with torch.cuda.stream(side):
        b.awe_gemm_exact_static(A, b.I8, B, b.I8, w.M, w.N, w.K, b.ENC_INT8_AWE6, 0, C, b.C_I32)
    assert not busy.query()                                    # returned while the other stream still runs
    side.synchronize()
    assert np.array_equal(C.cpu().numpy(), want)
    busy.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        b.awe_gemm_exact_static(A, b.I8, B, b.I8, w.M, w.N, w.K, b.ENC_INT8_AWE6, 0, C, b.C_I32)
    for rep in range(2):
        A.copy_(torch.from_numpy(np.roll(A_np, rep, axis=0)).cuda())
        C.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert np.array_equal(C.cpu().numpy(), np.roll(want, rep, axis=0))


def test_static_scratch_entry_rejects_problems_beyond_its_array():
    need = b.awe_workspace_bytes(b.ENC_INT8_AWE6, 0, 4096, 4096, 4096)
    assert need > b.STATIC_WORKSPACE_BYTES
    x = torch.zeros(16, dtype=torch.int8, device="cuda")      # never touched: the call must refuse first
    with pytest.raises(b.AweError) as e:
        b.awe_gemm_exact_static(x, b.I8, x, b.I8, 4096, 4096, 4096, b.ENC_INT8_AWE6, 0, x, b.C_I32)
    assert e.value.status == 3
    assert b.awe_workspace_bytes(b.ENC_INT8_AWE6, 0, 2048, 2048, 2048) == b.STATIC_WORKSPACE_BYTES
