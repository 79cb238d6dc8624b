"""Model variants of the ADiT stage (state-block mask, rotary embedding on the suffix) on every kernel set, against
the oracle with the same variant switched on; and that the variants really change the result."""
import numpy as np
import pytest

from oracle import adit_oracle as O
from paper_2609_12075_b200 import workloads as W

pytestmark = pytest.mark.gpu

VARIANTS = {"mask": dict(state_block_mask=True), "rope": dict(suffix_rope=True),
            "mask+rope": dict(state_block_mask=True, suffix_rope=True)}
FAMILIES = {
    "pi0": (W.scaled(W.PI0, n_layers=2), [130, 0, 257], 320, 2),
    "expert2": (W.scaled(W.EXPERT2, n_layers=2), [256, 31, 64, 1], 256, 2),
    "tiny-fp32": (W.TINY, [64, 17, 0], 64, 3),
}


@pytest.fixture(scope="module")
def adit():
    from paper_2609_12075_b200 import build
    build.build()
    from paper_2609_12075_b200 import adit as mod
    return mod


def run(adit, cfg, wl, w, flags=0):
    import torch
    eng = adit.ADiT(cfg, max_batch=wl.batch, max_prefix_len=wl.max_prefix_len, flags=flags)
    eng.load_weights(w)
    out = eng.denoise(adit.upload_prefix_kv(wl), wl.prefix_len, torch.from_numpy(wl.state).cuda(),
                      torch.from_numpy(wl.noise).cuda(), wl.n_steps)
    torch.cuda.synchronize()
    assert eng.poll_status() == 0
    blocks = eng.persistent_blocks(wl.batch)
    eng.close()
    return out.cpu().numpy().astype(np.float64), blocks


def close(got, ref, dtype):
    tol = (3e-2, 1e-2) if dtype == "bf16" else (1e-4, 1e-4)
    assert np.isfinite(got).all()
    return np.abs(got - ref).max() <= tol[0] and np.linalg.norm(got - ref) / np.linalg.norm(ref) <= tol[1]


@pytest.mark.parametrize("variant", sorted(VARIANTS))
@pytest.mark.parametrize("family", sorted(FAMILIES))
def test_variants_match_the_oracle(adit, family, variant):
    base, plens, cap, steps = FAMILIES[family]
    cfg = W.scaled(base, **VARIANTS[variant])
    wl = W.make_workload(family, cfg, seed=81, batch=len(plens), n_steps=steps, prefix_len=plens, max_prefix_len=cap)
    w = W.make_weights(cfg, wl.seed)
    ref = O.adit_denoise(cfg, w, wl.prefix_kv, wl.prefix_len, wl.state, wl.noise, steps)
    plain = O.adit_denoise(base, w, wl.prefix_kv, wl.prefix_len, wl.state, wl.noise, steps)
    effect = np.abs(ref - plain).max()
    got, _ = run(adit, cfg, wl, w)
    assert close(got, ref, cfg.dtype)
    # where the variant moves the actions by clearly more than the tolerance, the result must side with the variant
    # (the mask alone moves them little in the two-layer pi0 case: the state token's own stream is checked below)
    if effect > 3 * (3e-2 if cfg.dtype == "bf16" else 1e-4):
        assert np.abs(got - ref).max() * 3 < np.abs(got - plain).max()
    else:
        assert variant == "mask"
    if cfg.dtype == "bf16":
        got, _ = run(adit, cfg, wl, w, flags=adit.FLAG_REFERENCE_KERNELS)
        assert close(got, ref, cfg.dtype)


@pytest.mark.parametrize("flags_name", ["tensor-core", "reference", "persistent"])
def test_mask_reaches_the_state_tokens_stream(adit, flags_name):
    """One Euler step: the residual stream after the last layer (library workspace) against the oracle's, row by row.
    Under the mask the state token's row differs strongly from the unmasked model's."""
    import torch
    flags = {"tensor-core": 0, "reference": adit.FLAG_REFERENCE_KERNELS, "persistent": adit.FLAG_PERSISTENT_LOOP}[flags_name]
    base = W.scaled(W.PI0, n_layers=2)
    cfg = W.scaled(base, state_block_mask=True)
    wl = W.make_workload("mask-h", cfg, seed=85, batch=1, n_steps=1, prefix_len=[130], max_prefix_len=192)
    w = W.make_weights(cfg, wl.seed)
    tr_m, tr_p = [], []
    O.adit_denoise(cfg, w, wl.prefix_kv, wl.prefix_len, wl.state, wl.noise, 1, traces=tr_m)
    O.adit_denoise(base, w, wl.prefix_kv, wl.prefix_len, wl.state, wl.noise, 1, traces=tr_p)
    want, plain = tr_m[0]["h1"], tr_p[0]["h1"]
    assert np.abs(want[0] - plain[0]).max() > 0.2           # the state token's stream feels the mask
    eng = adit.ADiT(cfg, max_batch=1, max_prefix_len=192, flags=flags)
    eng.load_weights(w)
    eng.denoise(adit.upload_prefix_kv(wl), wl.prefix_len, torch.from_numpy(wl.state).cuda(), torch.from_numpy(wl.noise).cuda(), 1)
    torch.cuda.synchronize()
    assert (eng.persistent_blocks(1) > 0) == (flags_name == "persistent")
    h = eng.debug_copy("h", cfg.n_tokens * cfg.d_model).reshape(cfg.n_tokens, cfg.d_model).astype(np.float64)
    eng.close()
    assert np.abs(h - want).max() <= 5e-2 and np.linalg.norm(h - want) / np.linalg.norm(want) <= 1e-2
    assert np.abs(h[0] - want[0]).max() * 3 < np.abs(h[0] - plain[0]).max()


def test_state_block_mask_on_the_persistent_kernel(adit):
    for base, plens, cap, steps in ((W.scaled(W.PI0, n_layers=2), [130], 320, 2), (W.scaled(W.EXPERT2, n_layers=2), [70, 0, 5], 128, 2),
                                    (W.scaled(W.TINY, dtype="bf16"), [64, 0, 65], 96, 3)):
        cfg = W.scaled(base, state_block_mask=True)
        wl = W.make_workload("mask-loop", cfg, seed=83, batch=len(plens), n_steps=steps, prefix_len=plens, max_prefix_len=cap)
        w = W.make_weights(cfg, wl.seed)
        ref = O.adit_denoise(cfg, w, wl.prefix_kv, wl.prefix_len, wl.state, wl.noise, steps)
        got, blocks = run(adit, cfg, wl, w, flags=adit.FLAG_PERSISTENT_LOOP)
        assert blocks >= 8 and close(got, ref, "bf16")
    # the rotary variant is served by the kernel-per-phase path
    cfg = W.scaled(W.scaled(W.TINY, dtype="bf16"), suffix_rope=True)
    wl = W.make_workload("rope-loop", cfg, seed=84, batch=2, n_steps=2, prefix_len=[9, 40], max_prefix_len=64)
    w = W.make_weights(cfg, wl.seed)
    got, blocks = run(adit, cfg, wl, w, flags=adit.FLAG_PERSISTENT_LOOP)
    assert blocks == 0 and close(got, O.adit_denoise(cfg, w, wl.prefix_kv, wl.prefix_len, wl.state, wl.noise, 2), "bf16")


def test_unsupported_combination_is_refused(adit):
    cfg = W.scaled(W.scaled(W.TINY, dtype="bf16"), state_block_mask=True)
    with pytest.raises(adit.AditError) as e:
        adit.ADiT(cfg, max_batch=1, max_prefix_len=16, flags=adit.FLAG_MMA_SYNC_ATTENTION)
    assert e.value.code == adit.E_UNSUPPORTED
