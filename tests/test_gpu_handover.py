"""Hidden-state hand-over (paper section 2.1: the VLM hands over "hidden states or a small KV cache"): the expert
projects the prefix keys and values of every layer itself (adit_project_prefix), then runs the loop on them.
Checked against the oracle's projection and, end to end, against the oracle's loop on the oracle's projection."""
import numpy as np
import pytest

from oracle import adit_oracle as O
from paper_2609_12075_b200 import workloads as W

pytestmark = pytest.mark.gpu

DH = 192  # hidden width of the stand-in VLM (a multiple of 64)


@pytest.fixture(scope="module")
def adit():
    from paper_2609_12075_b200 import build
    build.build()
    from paper_2609_12075_b200 import adit as mod
    return mod


def _setup(adit, cfg, plens, cap, seed=91):
    import torch
    wl = W.make_workload("handover", cfg, seed=seed, batch=len(plens), n_steps=3, prefix_len=plens, max_prefix_len=cap,
                         with_kv=False)
    w = W.make_weights(cfg, wl.seed)
    pw = W.make_prefix_projection(cfg, wl.seed, DH)
    eng = adit.ADiT(cfg, max_batch=len(plens), max_prefix_len=cap)
    eng.load_weights(w)
    hidden = [W.make_prefix_hidden(wl.seed, b, int(p), DH) for b, p in enumerate(plens)]
    hidden_dev = [torch.from_numpy(h).to(torch.bfloat16).cuda() if len(h) else None for h in hidden]
    return wl, w, pw, eng, hidden, hidden_dev


def _empty_caches(cfg, n, cap, fill=-3.0):
    import torch
    return [torch.full((cfg.n_layers, 2, cfg.n_kv_heads, cap, cfg.head_dim), fill, dtype=torch.bfloat16, device="cuda")
            for _ in range(n)]


def test_projection_matches_the_oracle_and_leaves_padding_rows_alone(adit):
    import torch
    cfg = W.scaled(W.PI0, n_layers=2)
    plens, cap = [0, 1, 63, 64, 65, 200, 131], 200
    wl, w, pw, eng, hidden, hidden_dev = _setup(adit, cfg, plens, cap)
    caches = _empty_caches(cfg, len(plens), cap)
    with pytest.raises(adit.AditError) as e:   # nothing loaded yet
        eng.project_prefix(hidden_dev, plens, caches)
    assert e.value.code == adit.E_NOT_LOADED
    eng.load_prefix_projection(pw)
    eng.project_prefix(hidden_dev, plens, caches)
    torch.cuda.synchronize()
    assert eng.poll_status() == 0
    for b, P in enumerate(plens):
        got = caches[b].float().cpu().numpy().astype(np.float64)
        ref = O.project_prefix_kv(cfg, hidden[b], pw, cap, pad_value=-3.0)
        assert np.all(got[:, :, :, P:, :] == -3.0), b            # rows at or beyond the prefix length: untouched
        if P:
            # fp32 accumulation over 192 terms of unit-variance products, then one rounding to bf16 (2^-9 relative)
            err = np.abs(got[:, :, :, :P] - ref[:, :, :, :P])
            assert np.all(err <= 2.0 ** -8 * np.abs(ref[:, :, :, :P]) + 1e-3), (b, err.max())
    # a request's cache does not depend on its neighbours, the SM budget or a repetition: bit for bit
    for b in (2, 5):
        alone = _empty_caches(cfg, 1, cap)
        eng.project_prefix([hidden_dev[b]], [plens[b]], alone, sm_budget=5)
        torch.cuda.synchronize()
        assert torch.equal(alone[0].view(torch.int16), caches[b].view(torch.int16))
    eng.close()


def test_loop_on_the_projected_cache_matches_the_oracle(adit):
    import torch
    cfg = W.scaled(W.PI0, n_layers=2)
    plens, cap = [37, 0, 150], 160
    wl, w, pw, eng, hidden, hidden_dev = _setup(adit, cfg, plens, cap, seed=92)
    eng.load_prefix_projection(pw)
    caches = _empty_caches(cfg, len(plens), cap, fill=float("nan"))
    s = torch.cuda.current_stream()
    eng.project_prefix(hidden_dev, plens, caches, stream=s)   # same stream: the loop reads what the projection wrote
    out = eng.denoise(caches, wl.prefix_len, torch.from_numpy(wl.state).cuda(), torch.from_numpy(wl.noise).cuda(), wl.n_steps, stream=s)
    torch.cuda.synchronize()
    assert eng.poll_status() == 0
    got = out.cpu().numpy().astype(np.float64)
    # the oracle's loop on the oracle's projection (handed over as bf16, as the boundary says)
    kv = [W.round_to_bf16(np.nan_to_num(O.project_prefix_kv(cfg, hidden[b], pw, cap), nan=0.0).astype(np.float32)) for b in range(len(plens))]
    ref = O.adit_denoise(cfg, w, kv, wl.prefix_len, wl.state, wl.noise, wl.n_steps)
    assert np.isfinite(got).all()
    assert np.abs(got - ref).max() <= 3e-2 and np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 1e-2
    # the hidden states matter: other hidden states, other actions
    other = [torch.from_numpy(W.make_prefix_hidden(7, b, int(p), DH)).to(torch.bfloat16).cuda() if p else None for b, p in enumerate(plens)]
    eng.project_prefix(other, plens, caches, stream=s)
    out2 = eng.denoise(caches, wl.prefix_len, torch.from_numpy(wl.state).cuda(), torch.from_numpy(wl.noise).cuda(), wl.n_steps, stream=s)
    torch.cuda.synchronize()
    d = (out2 - out).abs().amax(dim=(1, 2)).cpu().numpy()
    assert d[0] > 1e-3 and d[2] > 1e-3 and d[1] == 0.0   # (request 1 has no prefix)
    eng.close()


def test_hand_over_errors(adit):
    import torch
    cfg = W.scaled(W.TINY, dtype="bf16")
    eng = adit.ADiT(cfg, max_batch=2, max_prefix_len=32)
    eng.load_weights(W.make_weights(cfg, 3))
    pw = W.make_prefix_projection(cfg, 3, 64)
    missing = dict(list(pw.items())[:-1])
    with pytest.raises(adit.AditError) as e:
        eng.load_prefix_projection(missing)
    assert e.value.code == adit.E_INVALID
    bad = dict(pw)
    k0 = next(iter(bad))
    bad[k0] = np.zeros((96, bad[k0].shape[1]), dtype=np.float32)   # another hidden width for one matrix
    with pytest.raises(adit.AditError) as e:
        eng.load_prefix_projection(bad)
    assert e.value.code == adit.E_INVALID
    eng.load_prefix_projection(pw)
    # (the smallest shape family, head_dim 64 and a hidden width of one k-block, also projects correctly)
    hid = [W.make_prefix_hidden(3, b, p, 64) for b, p in enumerate((32, 7))]
    small = _empty_caches(cfg, 2, 32)
    eng.project_prefix([torch.from_numpy(x).to(torch.bfloat16).cuda() for x in hid], [32, 7], small)
    torch.cuda.synchronize()
    for b, P in enumerate((32, 7)):
        got = small[b].float().cpu().numpy().astype(np.float64)
        ref = O.project_prefix_kv(cfg, hid[b], pw, 32, pad_value=-3.0)
        assert np.all(got[:, :, :, P:, :] == -3.0)
        assert np.all(np.abs(got[:, :, :, :P] - ref[:, :, :, :P]) <= 2.0 ** -8 * np.abs(ref[:, :, :, :P]) + 1e-3)
    caches = _empty_caches(cfg, 3, 32)
    h = [torch.zeros(8, 64, dtype=torch.bfloat16, device="cuda") for _ in range(3)]
    with pytest.raises(adit.AditError) as e:
        eng.project_prefix(h, [8, 8, 8], caches)       # B > max_batch
    assert e.value.code == adit.E_CAPACITY
    with pytest.raises(adit.AditError) as e:
        eng.project_prefix(h[:2], [8, 33], caches[:2])  # longer than the capacity
    assert e.value.code == adit.E_INVALID
    eng.close()
    fp32 = adit.ADiT(W.scaled(W.TINY, dtype="fp32"), max_batch=1, max_prefix_len=8)
    with pytest.raises(adit.AditError) as e:
        fp32.load_prefix_projection(W.make_prefix_projection(W.scaled(W.TINY, dtype="fp32"), 3, 64))
    assert e.value.code == adit.E_UNSUPPORTED
    fp32.close()
