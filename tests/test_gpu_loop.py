"""The persistent small-batch kernel (ADIT_FLAG_PERSISTENT_LOOP): one resident kernel for the whole call.

Same bar as the kernel-per-phase path: oracle tolerance on every shape family, bit-exact ragged indexing
(padding contents, batch slot, batch size, SM budget, repetition), plus the bounded-wait path: a
completion signal is withheld on purpose (host-set switch, millisecond limit), the kernel must return
by itself with ADIT_E_TIMEOUT and the handle must serve the next call correctly.
"""
import numpy as np
import pytest

from oracle import adit_oracle as O
from paper_2609_12075_b200 import workloads as W

pytestmark = pytest.mark.gpu

FAMILIES = {
    "pi0": (W.scaled(W.PI0, n_layers=2), [130], 320, 3),
    "pi0-no-prefix": (W.scaled(W.PI0, n_layers=1), [0], 64, 2),
    "expert2": (W.scaled(W.EXPERT2, n_layers=2), [256, 31, 1], 256, 2),
    "tiny-bf16": (W.scaled(W.TINY, dtype="bf16"), [64, 0, 65], 96, 4),
}


@pytest.fixture(scope="module")
def adit():
    from paper_2609_12075_b200 import build
    build.build()
    from paper_2609_12075_b200 import adit as mod
    return mod


def run(adit, eng, wl, kv=None, budget=0, idx=None):
    import torch
    idx = list(range(wl.batch)) if idx is None else idx
    kv = adit.upload_prefix_kv(wl) if kv is None else kv
    out = eng.denoise([kv[i] for i in idx], wl.prefix_len[idx], torch.from_numpy(wl.state[idx]).cuda(),
                      torch.from_numpy(wl.noise[idx]).cuda(), wl.n_steps, sm_budget=budget)
    torch.cuda.synchronize()
    return out.cpu().numpy()


def bits(a):
    return a.view(np.uint32)


@pytest.mark.parametrize("family", sorted(FAMILIES))
def test_parity_and_invariances(adit, family):
    cfg, plens, cap, steps = FAMILIES[family]
    wl = W.make_workload(family, cfg, seed=23, batch=len(plens), n_steps=steps, prefix_len=plens, max_prefix_len=cap)
    w = W.make_weights(cfg, wl.seed)
    eng = adit.ADiT(cfg, max_batch=len(plens), max_prefix_len=cap, flags=adit.FLAG_PERSISTENT_LOOP)
    eng.load_weights(w)
    assert eng.persistent_blocks(len(plens)) >= 8
    kv = adit.upload_prefix_kv(wl)
    before = eng.kernel_launches()
    base = run(adit, eng, wl, kv)
    assert eng.poll_status() == 0
    ref = O.adit_denoise(cfg, w, wl.prefix_kv, wl.prefix_len, wl.state, wl.noise, steps)
    got = base.astype(np.float64)
    assert np.isfinite(got).all()
    assert np.abs(got - ref).max() <= 3e-2 and np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 1e-2
    # the whole call is a handful of launches (time vectors on the first call, set-up kernel, the loop kernel)
    assert eng.kernel_launches() - before <= 5
    # repetition, SM budget (any number of 8-block clusters), slot and batch size: not one bit changes
    assert np.array_equal(bits(run(adit, eng, wl, kv)), bits(base))
    for budget in (8, 17, 64, 1000):
        assert eng.persistent_blocks(len(plens), budget) == min(budget // 8, eng.persistent_blocks(len(plens)) // 8) * 8
        assert np.array_equal(bits(run(adit, eng, wl, kv, budget=budget)), bits(base)), budget
    if len(plens) > 1:
        perm = list(range(len(plens)))[::-1]
        assert np.array_equal(bits(run(adit, eng, wl, kv, idx=perm)), bits(base[perm]))
        for b in range(len(plens)):
            assert np.array_equal(bits(run(adit, eng, wl, kv, idx=[b]))[0], bits(base)[b]), b
    # padding rows of the prefix caches never matter
    for kw in ({"pad_value": 0.0}, {"pad_value": float("inf")}, {"pad_seed": 5}):
        other = W.make_workload(family, cfg, seed=23, batch=len(plens), n_steps=steps, prefix_len=plens, max_prefix_len=cap, **kw)
        assert np.array_equal(bits(run(adit, eng, other)), bits(base)), kw
    eng.close()


def test_wait_limit_runs_out_and_the_handle_recovers(adit):
    cfg, plens, cap, steps = FAMILIES["tiny-bf16"]
    wl = W.make_workload("timeout", cfg, seed=29, batch=len(plens), n_steps=steps, prefix_len=plens, max_prefix_len=cap)
    w = W.make_weights(cfg, wl.seed)
    eng = adit.ADiT(cfg, max_batch=len(plens), max_prefix_len=cap, flags=adit.FLAG_PERSISTENT_LOOP)
    eng.load_weights(w)
    kv = adit.upload_prefix_kv(wl)
    good = run(adit, eng, wl, kv)
    assert eng.poll_status() == adit.OK
    for level in (2, 3, 7):                      # qkv projection, attention, read-out
        eng.debug_wait_limit(5, withhold_level=level)
        run(adit, eng, wl, kv)                   # returns by itself: every wait gives up after 5 ms
        assert eng.poll_status() == adit.E_TIMEOUT
        eng.clear_status()
        eng.debug_wait_limit(2000, withhold_level=-1)
        assert np.array_equal(bits(run(adit, eng, wl, kv)), bits(good))
        assert eng.poll_status() == adit.OK
    eng.close()


def test_c2_full_size(adit):
    wl = W.config_c2()
    w = W.make_weights(wl.cfg, wl.seed)
    eng = adit.ADiT(wl.cfg, max_batch=1, max_prefix_len=wl.max_prefix_len, flags=adit.FLAG_PERSISTENT_LOOP)
    eng.load_weights(w)
    got = run(adit, eng, wl).astype(np.float64)
    assert eng.poll_status() == 0
    ref = O.adit_denoise(wl.cfg, w, wl.prefix_kv, wl.prefix_len, wl.state, wl.noise, wl.n_steps)
    assert np.abs(got - ref).max() <= 3e-2 and np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 1e-2
    eng.close()
