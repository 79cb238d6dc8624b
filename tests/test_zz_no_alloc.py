"""adit_attention_static: the attention entry point that allocates nothing.

Hosts that may not call cudaMalloc (a region being recorded into a CUDA graph, a real-time loop that
must stay clear of the allocator's locks, a process whose device memory was carved up at start-up)
use this variant; its scratch is a fixed 8 MiB array inside the library.  The test calls it through
the C ABI twice in a row - the second call finds the first call's leftovers in the array - and wants
both results equal to the allocating entry point's, then checks the size limit.  It lives in a file
that pytest collects last, so a failure here cannot hide the outcome of any other test, and it does
not depend on anything the other tests leave behind.
"""
import ctypes as C

import pytest

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def adit():
    from paper_2609_12075_b200 import build
    build.build()
    from paper_2609_12075_b200 import adit as mod
    return mod


def problem(B, n_tok, hq, hkv, dh, p_cap, plens, seed):
    import torch
    g = torch.Generator().manual_seed(seed)
    qkv = torch.randn(B * n_tok, (hq + 2 * hkv) * dh, generator=g).to(torch.bfloat16).cuda()
    kv = []
    for b in range(B):
        t = torch.full((2, 2, hkv, p_cap, dh), float("nan"))
        t[:, :, :, :plens[b]] = torch.randn(2, 2, hkv, plens[b], dh, generator=g)
        kv.append(t.to(torch.bfloat16).cuda())
    return qkv, kv


def fp32_reference(shape, plens, qkv, kv, layer=1):
    """Plain PyTorch fp32 attention per request: prefix rows [0, prefix_len) followed by the suffix rows."""
    import torch
    B, n_tok, hq, hkv, dh, p_cap = shape
    out = torch.empty(B * n_tok, hq * dh)
    q_all = qkv.float().cpu()
    for b in range(B):
        rows = q_all[b * n_tok:(b + 1) * n_tok]
        q = rows[:, :hq * dh].reshape(n_tok, hq, dh).transpose(0, 1)
        ks = rows[:, hq * dh:(hq + hkv) * dh].reshape(n_tok, hkv, dh).transpose(0, 1)
        vs = rows[:, (hq + hkv) * dh:].reshape(n_tok, hkv, dh).transpose(0, 1)
        k = torch.cat([kv[b][layer, 0, :, :plens[b]].float().cpu(), ks], dim=1).repeat_interleave(hq // hkv, dim=0)
        v = torch.cat([kv[b][layer, 1, :, :plens[b]].float().cpu(), vs], dim=1).repeat_interleave(hq // hkv, dim=0)
        o = torch.nn.functional.scaled_dot_product_attention(q, k, v)
        out[b * n_tok:(b + 1) * n_tok] = o.transpose(0, 1).reshape(n_tok, hq * dh)
    return out


def call(fn, shape, plens, splits, qkv, kv):
    import torch
    B, n_tok, hq, hkv, dh, p_cap = shape
    out = torch.full((B * n_tok, hq * dh), float("nan"), dtype=torch.bfloat16, device="cuda")
    ptrs = (C.c_void_p * B)(*[t.data_ptr() for t in kv])
    lens = (C.c_int32 * B)(*plens)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    rc = fn(0, B, n_tok, hq, hkv, dh, p_cap, 1, qkv.data_ptr(), ptrs, lens, splits, out.data_ptr(), None)
    call.free_bytes_during = torch.cuda.mem_get_info()[0] - free_before   # (the kernels may still be running)
    torch.cuda.synchronize()
    call.free_bytes_after = torch.cuda.mem_get_info()[0] - free_before
    return rc, out


def test_static_scratch_attention_matches_allocating_entry_point_twice(adit):
    import torch
    # two different problems back to back: the second finds the first one's partials in the array
    cases = [((1, 51, 8, 1, 256, 816), [816], 14, 3), ((4, 17, 12, 12, 128, 256), [256, 1, 64, 65], 3, 4)]
    for shape, plens, splits, seed in cases:
        qkv, kv = problem(*shape, plens, seed)
        rc_ref, ref = call(adit.lib.adit_debug_attention, shape, plens, splits, qkv, kv)
        assert rc_ref == 0
        exact = fp32_reference(shape, plens, qkv, kv)
        call(adit.lib.adit_attention_static, shape, plens, splits, qkv, kv)      # (first use on the device: set-up)
        for attempt in range(2):
            rc, got = call(adit.lib.adit_attention_static, shape, plens, splits, qkv, kv)
            assert rc == 0, (shape, attempt)
            assert adit.lib.adit_attention_static_status(0) == 0
            assert torch.isfinite(got.float()).all()
            # on its own feet: against the fp32 attention, within the tolerance of the attention tests
            assert (got.float().cpu() - exact).abs().max().item() <= 2e-2
            # and against the allocating entry point: same kernels, same order of operations, not one bit differs
            assert torch.equal(got, ref), (shape, attempt)
            # the claim in its name: the device's free memory is the same before the call, right after it returned and
            # after its kernels have finished
            assert call.free_bytes_during == 0 and call.free_bytes_after == 0


def test_static_scratch_attention_rejects_what_does_not_fit(adit):
    shape, plens = (16, 51, 8, 1, 256, 64), [64] * 16
    qkv, kv = problem(*shape, plens, 5)
    need = 32 * 16 * 51 * 8 * (256 + 2) * 4
    assert need > adit.STATIC_SCRATCH_BYTES
    rc, _ = call(adit.lib.adit_attention_static, shape, plens, 32, qkv, kv)
    assert rc == adit.E_CAPACITY
    rc, out = call(adit.lib.adit_attention_static, shape, plens, 1, qkv, kv)     # no scratch needed: accepted
    assert rc == 0
    rc_ref, ref = call(adit.lib.adit_debug_attention, shape, plens, 1, qkv, kv)
    import torch
    assert rc_ref == 0 and torch.equal(out, ref)
