"""Lockstep executor on the GPU: the ADiT stage of batch k-1 beside the VLM stand-in of batch k, on two streams, under
an SM restriction; results must equal direct calls bit for bit and the two stages of a lockstep must overlap."""
import numpy as np
import pytest

from paper_2609_12075_b200 import workloads as W

pytestmark = pytest.mark.gpu


def test_locksteps_on_two_streams_match_direct_calls():
    import torch
    from paper_2609_12075_b200 import build
    build.build()
    from paper_2609_12075_b200 import adit, lockstep as LS
    cfg = W.scaled(W.PI0, n_layers=2)
    pool = 6
    wl = W.make_workload("lockstep-test", cfg, seed=61, batch=pool, n_steps=3, prefix_len=[100, 0, 257, 64, 31, 200],
                         max_prefix_len=320)
    eng = adit.ADiT(cfg, max_batch=2, max_prefix_len=320)
    eng.load_weights(W.make_weights(cfg, wl.seed))
    inputs = {"m": {"kv": adit.upload_prefix_kv(wl), "len": wl.prefix_len, "state": torch.from_numpy(wl.state).cuda(),
                    "noise": torch.from_numpy(wl.noise).cuda(), "steps": wl.n_steps}}
    stages = LS.GpuStages(adit, {"m": eng}, inputs, vlm_iters_per_request=40, gemm_shape=(4096, 2048, 2048))
    table = LS.SmTable(stages.n_sm, {(2, 2): 112, (1, 2): 112, (2, 1): 120, (1, 1): 120})
    ex = LS.LockstepExecutor(stages.vlm, stages.adit_stage, 2, table, {"m": 100_000})
    reqs = [LS.Request("m", i, 0, payload=i) for i in range(5)]
    [ex.submit(r) for r in reqs]
    rec = ex.run()
    assert [(r.vlm_ids, r.adit_ids) for r in rec] == [([0, 1], []), ([2, 3], [0, 1]), ([4], [2, 3]), ([], [4])]
    assert [(r.vlm_sms, r.adit_sms) for r in rec][1:3] == [(112, stages.n_sm - 112), (112, stages.n_sm - 112)]
    assert eng.poll_status() == 0
    # the same batches, called directly with the same SM budgets
    for ids, budget in (([0, 1], stages.n_sm - 112), ([2, 3], stages.n_sm - 112), ([4], 0)):
        idx = torch.tensor(ids, device="cuda")
        want = eng.denoise([inputs["m"]["kv"][i] for i in ids], wl.prefix_len[ids], inputs["m"]["state"][idx].contiguous(),
                           inputs["m"]["noise"][idx].contiguous(), wl.n_steps, sm_budget=budget)
        torch.cuda.synchronize()
        for j, i in enumerate(ids):
            assert torch.equal(reqs[i].result, want[j]), i
    # in the locksteps with both stages, their execution intervals overlap (the two host threads launch them together)
    for r in rec[1:3]:
        (v0, v1), (a0, a1) = r.vlm_interval, r.adit_interval
        assert max(v0, a0) < min(v1, a1)
    stages.close()
    eng.close()


def test_green_stream_confines_a_kernel_that_asks_for_the_whole_chip():
    """A stream on a green context (paper section 4.1.2: the VLM stream restricted to a number of SMs in multiples of 8):
    the stand-in GEMM launched with its full grid takes about as long as with its grid capped to that many SMs, and
    much longer than on the whole chip; the partition is what was asked for, rounded up to the driver's granularity."""
    import torch
    from paper_2609_12075_b200 import build
    build.build()
    from paper_2609_12075_b200 import adit

    def per_launch_us(stream, g, cap):
        g.launch(3, cap, stream)
        stream.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        g.launch(10, cap, stream)
        e1.record(stream)
        stream.synchronize()
        return e0.elapsed_time(e1) * 100.0

    g = adit.BackgroundGemm(8192, 2048, 2048)
    plain = torch.cuda.Stream()
    full, capped = per_launch_us(plain, g, 0), per_launch_us(plain, g, 24)
    try:
        gs = adit.GreenStream(20)
    except adit.AditError as e:
        if e.code == adit.E_UNSUPPORTED:
            pytest.skip("no green contexts on this driver")
        raise
    assert gs.sm_count >= 20 and gs.sm_count % 8 == 0 and gs.sm_count <= 32
    confined = per_launch_us(gs.stream, g, 0)
    gs.close()
    g.close()
    assert confined > 2.5 * full            # (24 of 148 SMs: about six times the whole-chip time)
    assert 0.6 * capped < confined * gs.sm_count / 24 < 1.8 * capped
    with pytest.raises(adit.AditError) as e:
        adit.GreenStream(100000)
    assert e.value.code == adit.E_CAPACITY
