"""adit_denoise recorded into the caller's CUDA graph (paper section 4.1.1: one graph per stage and batch size):
replays must give the bits of direct calls on whatever the captured buffers hold at replay time."""
import gc

import numpy as np
import pytest

from paper_2609_12075_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("persistent", [False, True])
def test_call_can_be_captured_and_replayed(persistent):
    import torch
    from paper_2609_12075_b200 import build
    build.build()
    from paper_2609_12075_b200 import adit
    cfg = W.scaled(W.TINY, dtype="bf16") if persistent else W.scaled(W.PI0, n_layers=2)
    plens, cap, steps = ([64, 5], 96, 3) if persistent else ([130, 0, 257], 320, 2)
    wl = W.make_workload("capture", cfg, seed=71, batch=len(plens), n_steps=steps, prefix_len=plens, max_prefix_len=cap)
    eng = adit.ADiT(cfg, max_batch=len(plens), max_prefix_len=cap, flags=adit.FLAG_PERSISTENT_LOOP if persistent else 0)
    eng.load_weights(W.make_weights(cfg, wl.seed))
    assert (eng.persistent_blocks(len(plens)) > 0) == persistent
    kv = adit.upload_prefix_kv(wl)
    state, noise = torch.from_numpy(wl.state).cuda(), torch.from_numpy(wl.noise).cuda()
    out = torch.empty_like(noise)
    s = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    # a call that has not been made before cannot be captured: nothing is recorded, the status says so
    with torch.cuda.stream(s):
        s.synchronize()
    fresh = adit.ADiT(cfg, max_batch=len(plens), max_prefix_len=cap, flags=adit.FLAG_PERSISTENT_LOOP if persistent else 0)
    fresh.load_weights(W.make_weights(cfg, wl.seed))
    # (objects of earlier tests that are collected while a capture is open would free device memory inside it and
    # invalidate the capture: collect them now)
    gc.collect()
    torch.cuda.synchronize()
    refused = torch.cuda.CUDAGraph()
    with torch.cuda.graph(refused, stream=s, capture_error_mode="thread_local"):
        with pytest.raises(adit.AditError) as e:
            fresh.denoise(kv, wl.prefix_len, state, noise, steps, stream=s, out=out)
        assert e.value.code == adit.E_UNSUPPORTED
    fresh.close()
    # warm-up outside the capture, then record
    direct0 = eng.denoise(kv, wl.prefix_len, state, noise, steps, stream=s, out=torch.empty_like(noise))
    s.synchronize()
    gc.collect()
    with torch.cuda.graph(g, stream=s, capture_error_mode="thread_local"):
        eng.denoise(kv, wl.prefix_len, state, noise, steps, stream=s, out=out)
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(out, direct0)
    # new contents in the captured buffers: the replay computes on them
    rng = np.random.default_rng(3)
    noise.copy_(torch.from_numpy(rng.standard_normal(wl.noise.shape).astype(np.float32)))
    state.copy_(torch.from_numpy(rng.standard_normal(wl.state.shape).astype(np.float32)))
    for _ in range(2):
        out.zero_()
        g.replay()
        torch.cuda.synchronize()
    direct1 = eng.denoise(kv, wl.prefix_len, state, noise, steps)
    torch.cuda.synchronize()
    assert torch.equal(out, direct1) and not torch.equal(direct1, direct0)
    assert eng.poll_status() == 0
    eng.close()
    del g, refused
    gc.collect()
