"""Back-to-back launches at full size: every repetition must reproduce the first result bit for
bit (the first one is checked against the CPU oracle on sampled rows).  Catches hand-over races
between the roles of the persistent kernel that a single launch would rarely show."""
import pytest
import torch

from paper_2609_24519_b200 import binding as b
from paper_2609_24519_b200 import workloads as wl
from tests import gpu_util as gu
from tests.test_gpu_configs import sampled_rows_match

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("enc,reps", [(b.ENC_INT8_AWE6, 150), (b.ENC_INT8_MIXED_FP8_3, 150), (b.ENC_INT8_BASE13_9, 60)])
def test_repeated_full_size_products_are_identical(enc, reps):
    w = wl.headline()
    A, B = wl.make_inputs(w)
    h = gu.handle()
    M, N, K = w.M, w.N, w.K
    dA, dB = torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda()
    ws = torch.empty(b.awe_workspace_bytes(enc, 0, M, N, K), dtype=torch.uint8, device="cuda")
    first = torch.empty((M, N), dtype=torch.int32, device="cuda")
    b.awe_gemm_exact(h, dA, b.I8, dB, b.I8, M, N, K, enc, 0, first, b.C_I32, ws)
    torch.cuda.synchronize()
    assert sampled_rows_match(first, A, B, 6, 31)
    C = torch.empty_like(first)
    bad = 0
    for i in range(reps):
        C.fill_(-1)
        b.awe_gemm_exact(h, dA, b.I8, dB, b.I8, M, N, K, enc, 0, C, b.C_I32, ws)
        if i % 10 == 9 or i == reps - 1:
            bad += int(not torch.equal(C, first))
    torch.cuda.synchronize()
    assert b.awe_last_device_status(h) == (0, 0)
    assert bad == 0


def test_repeated_residue_products_are_identical():
    m = 89
    w = wl.small("soak_mod89", 4096, 4096, 4096, "residue", "residue", seed=17, modulus=m)
    A, B = wl.make_inputs(w)
    h = gu.handle()
    dA, dB = torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda()
    ws = torch.empty(b.awe_workspace_bytes(b.ENC_MOD_M, m, w.M, w.N, w.K), dtype=torch.uint8, device="cuda")
    first = torch.empty((w.M, w.N), dtype=torch.int16, device="cuda")
    b.awe_gemm_exact(h, dA, b.I8, dB, b.I8, w.M, w.N, w.K, b.ENC_MOD_M, m, first, b.C_RES_I16, ws)
    torch.cuda.synchronize()
    assert sampled_rows_match(first, A, B, 6, 32, modulus=m)
    C = torch.empty_like(first)
    for i in range(200):
        b.awe_gemm_exact(h, dA, b.I8, dB, b.I8, w.M, w.N, w.K, b.ENC_MOD_M, m, C, b.C_RES_I16, ws)
        if i % 20 == 19:
            assert torch.equal(C, first)
    assert b.awe_last_device_status(h) == (0, 0)
