"""The tcgen05 projection kernel on its own, against a plain PyTorch fp32 matmul of the same bf16 operands."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

SHAPES = [
    # n_tok, n_feat, k, forced splits (0 = library's choice)
    (51, 2560, 1024, 0), (51, 1024, 2048, 0), (51, 1024, 4096, 0), (51, 1024, 4096, 1),
    (17, 128, 64, 0), (34, 384, 256, 0), (34, 384, 256, 3),
    (816, 2560, 1024, 0), (816, 1024, 2048, 0), (1632, 1024, 4096, 0), (408, 4608, 1536, 0),
    (50, 1000, 1024, 0), (300, 130, 192, 2),
    # splits = -2: the two-SM kernel (pairs of thread blocks; 256 features x tile tokens per pair): one and several
    # tiles per pair, an odd number of feature tiles, ragged token tails, rings shorter and longer than the k loop
    (64, 256, 128, -2), (1632, 2560, 1024, -2), (1632, 1024, 4096, -2), (816, 1024, 2048, -2), (300, 130, 192, -2),
    (500, 384, 256, -2), (408, 4608, 1536, -2), (8192, 2048, 2048, -2),
]


@pytest.fixture(scope="module")
def adit():
    from paper_2609_12075_b200 import build
    build.build()
    from paper_2609_12075_b200 import adit as mod
    return mod


@pytest.mark.parametrize("n_tok,n_feat,k,splits", SHAPES)
@pytest.mark.parametrize("budget", [0, 13])
def test_projection_kernel_matches_fp32_matmul(adit, n_tok, n_feat, k, splits, budget):
    import torch
    g = torch.Generator().manual_seed(n_tok * 7 + n_feat + k + splits)
    a = torch.randn(n_tok, k, generator=g).to(torch.bfloat16).cuda()
    w = (torch.randn(n_feat, k, generator=g) * 0.05).to(torch.bfloat16).cuda()
    out = torch.full((n_tok, n_feat), float("nan"), device="cuda")
    rc = adit.lib.adit_debug_gemm(0, n_tok, n_feat, k, a.data_ptr(), w.data_ptr(), out.data_ptr(), splits, budget,
                                  None)
    assert rc > 0, rc
    ref = a.float() @ w.float().T
    err = (out - ref).abs().max().item()
    scale = ref.abs().max().item()
    assert torch.isfinite(out).all()
    assert err <= 2e-5 * k ** 0.5 * max(scale, 1.0) / 10 + 1e-4, (rc, err, scale)


def test_two_sm_kernel_budget_does_not_change_a_single_bit(adit):
    import torch
    g = torch.Generator().manual_seed(2)
    a = torch.randn(1632, 1024, generator=g).to(torch.bfloat16).cuda()
    w = torch.randn(2560, 1024, generator=g).to(torch.bfloat16).cuda()
    outs = []
    for budget in (0, 1, 2, 7, 74, 148):  # (a pair needs two SMs: a budget of one is served with two)
        out = torch.empty(1632, 2560, device="cuda")
        rc = adit.lib.adit_debug_gemm(0, 1632, 2560, 1024, a.data_ptr(), w.data_ptr(), out.data_ptr(), -2, budget, None)
        assert rc // 1000000 == 9, rc
        outs.append(out.cpu().numpy())
    for o in outs[1:]:
        assert np.array_equal(o.view(np.uint32), outs[0].view(np.uint32))


def test_budget_does_not_change_a_single_bit(adit):
    import torch
    g = torch.Generator().manual_seed(1)
    a = torch.randn(51, 2048, generator=g).to(torch.bfloat16).cuda()
    w = torch.randn(1024, 2048, generator=g).to(torch.bfloat16).cuda()
    outs = []
    for budget in (0, 1, 7, 148):
        out = torch.empty(51, 1024, device="cuda")
        assert adit.lib.adit_debug_gemm(0, 51, 1024, 2048, a.data_ptr(), w.data_ptr(), out.data_ptr(), 0, budget, None) > 0
        outs.append(out.cpu().numpy())
    for o in outs[1:]:
        assert np.array_equal(o.view(np.uint32), outs[0].view(np.uint32))


def test_an_expired_wait_ends_the_kernel_with_a_status_and_the_next_launch_is_fine(adit):
    """Failure detection on the kernel-per-phase path: one block of a small projection is denied one operand copy, its
    bounded wait runs out (two seconds), the kernel returns by itself with ADIT_E_TIMEOUT in the status word, and the
    same projection launched again completes with a clean status.  Nothing faults and no wait is unbounded."""
    import ctypes as C
    import time
    import torch
    first = C.c_int(123)
    t0 = time.time()
    rc = adit.lib.adit_debug_gemm_timeout(0, C.byref(first), None)
    elapsed = time.time() - t0
    assert first.value == adit.E_TIMEOUT, first.value
    assert rc == adit.OK, rc
    assert 1.5 < elapsed < 20.0, elapsed
    # the device is in working order afterwards
    x = torch.ones(1024, device="cuda")
    assert float(x.sum().item()) == 1024.0
