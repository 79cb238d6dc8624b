"""Pins for the CPU oracle: closed forms, brute force, library special cases and invariants.

None of these re-types the oracle's own formula: each expected value comes from
mathematics (closed-form Euler sums, the mean of value rows), from a scalar
brute-force loop, from a torch CPU fp64 library routine, or from tabulated
constants.
"""
import math

import numpy as np
import pytest
import torch

from oracle import adit_oracle as O
from paper_2609_12075_b200 import workloads as W

SMALL = W.ADiTConfig(n_layers=2, d_model=32, n_q_heads=4, n_kv_heads=2, head_dim=8, d_ff=48,
                     horizon=5, action_dim=3, state_dim=4, time_emb_dim=32, dtype="fp32")


def small_inputs(cfg=SMALL, seed=11, batch=3, plens=(7, 0, 4), cap=9, **kw):
    wl = W.make_workload("small", cfg, seed=seed, batch=batch, n_steps=3, prefix_len=list(plens),
                         max_prefix_len=cap, **kw)
    w = W.make_weights(cfg, seed)
    # larger weights than the 0.02 default so that every term matters at 1e-12
    w = {k: (v if k.endswith(".g") else v * 10.0) for k, v in w.items()}
    return wl, w


def run(wl, w, n_steps=None):
    return O.adit_denoise(wl.cfg, w, wl.prefix_kv, wl.prefix_len, wl.state, wl.noise,
                          wl.n_steps if n_steps is None else n_steps)


# ---- P1: closed-form Euler trajectories for a linear field --------------------------------

@pytest.mark.parametrize("K", [1, 4, 10])
def test_euler_linear_field_closed_form(K):
    a, b, c = -0.7, 0.3, 1.9
    x0 = np.array([[1.5, -2.0], [0.25, 4.0]])
    got = O.euler_integrate(lambda x, t: a * x + b + c * t, x0, K)
    r = 1.0 + a / K
    want = r ** K * x0 + sum(r ** (K - 1 - k) * (b + c * k / K) / K for k in range(K))
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-14)


def test_euler_pure_drift_special_case():
    # a = 0: x_K = x_0 + b + c (K-1)/(2K); for K = 4 the time term is 3c/8.
    b, c = 0.5, 2.0
    got = O.euler_integrate(lambda x, t: b + c * t + 0 * x, np.zeros(3), 4)
    np.testing.assert_allclose(got, np.full(3, b + 3 * c / 8), atol=1e-15)


def test_euler_time_grid_is_left_endpoint():
    seen = []
    O.euler_integrate(lambda x, t: (seen.append(t), 0 * x)[1], np.zeros(1), 4)
    assert seen == [0.0, 0.25, 0.5, 0.75]


def test_euler_single_step():
    # P10: K = 1 is x_1 = x_0 + v(x_0, 0)
    wl, w = small_inputs()
    wf = O.as_f64_weights(w)
    got = run(wl, w, n_steps=1)
    for b in range(wl.batch):
        v = O.velocity(wl.cfg, wf, wl.noise[b].astype(np.float64), wl.state[b].astype(np.float64), 0.0,
                       wl.prefix_kv[b], int(wl.prefix_len[b]))
        np.testing.assert_allclose(got[b], wl.noise[b] + v, atol=1e-14)


# ---- P2: constant-velocity network -----------------------------------------------------------

def test_zero_readout_gives_noise_plus_bias():
    wl, w = small_inputs()
    w["action_out.w"] = np.zeros_like(w["action_out.w"])
    got = run(wl, w, n_steps=7)
    want = wl.noise.astype(np.float64) + w["action_out.b"].astype(np.float64)[None, None, :]
    np.testing.assert_allclose(got, want, atol=1e-14)


# ---- P3: identity layers ---------------------------------------------------------------------

def test_identity_layers_velocity_by_hand():
    wl, w = small_inputs()
    cfg = wl.cfg
    for l in range(cfg.n_layers):
        w[f"layers.{l}.wo"] = np.zeros_like(w[f"layers.{l}.wo"])
        w[f"layers.{l}.wd"] = np.zeros_like(w[f"layers.{l}.wd"])
    b, t = 0, 0.0
    x = wl.noise[b].astype(np.float64)
    v = O.velocity(cfg, O.as_f64_weights(w), x, wl.state[b].astype(np.float64), t, wl.prefix_kv[b], int(wl.prefix_len[b]))
    # hand computation with scalar loops for the action-token embedding and the read-out
    D, half = cfg.d_model, cfg.time_emb_dim // 2
    tau = [0.0] * half + [1.0] * half          # t = 0: sines 0, cosines 1
    want = np.zeros((cfg.horizon, cfg.action_dim))
    for i in range(cfg.horizon):
        a = [sum(float(x[i, j]) * float(w["action_in.w"][j, d]) for j in range(cfg.action_dim)) + float(w["action_in.b"][d])
             for d in range(D)]
        cat = a + tau
        pre = [sum(cat[r] * float(w["time_mlp.w1"][r, d]) for r in range(len(cat))) + float(w["time_mlp.b1"][d]) for d in range(D)]
        z = [p / (1.0 + math.exp(-p)) for p in pre]
        h = [sum(z[r] * float(w["time_mlp.w2"][r, d]) for r in range(D)) + float(w["time_mlp.b2"][d]) for d in range(D)]
        rms = math.sqrt(sum(e * e for e in h) / D + cfg.rms_eps)
        u = [h[d] / rms * float(w["final_norm.g"][d]) for d in range(D)]
        for j in range(cfg.action_dim):
            want[i, j] = sum(u[d] * float(w["action_out.w"][d, j]) for d in range(D)) + float(w["action_out.b"][j])
    np.testing.assert_allclose(v, want, rtol=1e-12, atol=1e-13)


# ---- P4: brute-force attention ---------------------------------------------------------------

def brute_attention(q, ks, vs, kp, vp, plen):
    n, hq, dh = q.shape
    hkv = ks.shape[1]
    out = np.zeros((n, hq, dh))
    for i in range(n):
        for h in range(hq):
            kv = h // (hq // hkv)
            keys = [kp[kv, r] for r in range(plen)] + [ks[r, kv] for r in range(n)]
            vals = [vp[kv, r] for r in range(plen)] + [vs[r, kv] for r in range(n)]
            scores = [sum(float(q[i, h, d]) * float(k[d]) for d in range(dh)) / math.sqrt(dh) for k in keys]
            m = max(scores)
            e = [math.exp(s - m) for s in scores]
            z = sum(e)
            for d in range(dh):
                out[i, h, d] = sum(e[r] * float(vals[r][d]) for r in range(len(vals))) / z
    return out


@pytest.mark.parametrize("plen", [0, 1, 7])
def test_attention_brute_force(plen):
    rng = np.random.default_rng(5)
    n, hq, hkv, dh, cap = 5, 4, 2, 4, 7
    q = rng.standard_normal((n, hq, dh)) * 2
    ks, vs = rng.standard_normal((2, n, hkv, dh))
    kp, vp = rng.standard_normal((2, hkv, cap, dh))
    got = O.attention(q, ks, vs, kp, vp, plen)
    np.testing.assert_allclose(got, brute_attention(q, ks, vs, kp, vp, plen), rtol=1e-12, atol=1e-13)


# ---- P5: uniform scores -> mean of the valid value rows --------------------------------------

@pytest.mark.parametrize("plen", [0, 3, 6, 7])
def test_zero_queries_average_valid_values(plen):
    rng = np.random.default_rng(6)
    n, hq, hkv, dh, cap = 4, 2, 1, 3, 7
    ks, vs = rng.standard_normal((2, n, hkv, dh))
    kp, vp = rng.standard_normal((2, hkv, cap, dh))
    vp[:, plen:, :] = 1e6          # any leak of a padding row would be loud
    got = O.attention(np.zeros((n, hq, dh)), ks, vs, kp, vp, plen)
    want = (vp[0, :plen].sum(0) + vs[:, 0].sum(0)) / (plen + n)
    np.testing.assert_allclose(got, np.broadcast_to(want, got.shape), rtol=1e-12)


# ---- P6: library special cases ---------------------------------------------------------------

def test_attention_matches_torch_sdpa():
    rng = np.random.default_rng(7)
    n, hq, hkv, dh, cap, plen = 6, 4, 2, 8, 10, 9
    q = rng.standard_normal((n, hq, dh))
    ks, vs = rng.standard_normal((2, n, hkv, dh))
    kp, vp = rng.standard_normal((2, hkv, cap, dh))
    got = O.attention(q, ks, vs, kp, vp, plen)
    g = hq // hkv
    k_all = torch.from_numpy(np.concatenate([kp[:, :plen], ks.transpose(1, 0, 2)], axis=1)).repeat_interleave(g, dim=0)
    v_all = torch.from_numpy(np.concatenate([vp[:, :plen], vs.transpose(1, 0, 2)], axis=1)).repeat_interleave(g, dim=0)
    ref = torch.nn.functional.scaled_dot_product_attention(torch.from_numpy(q.transpose(1, 0, 2)), k_all, v_all)
    np.testing.assert_allclose(got, ref.numpy().transpose(1, 0, 2), rtol=1e-12, atol=1e-13)


def test_pointwise_functions_match_torch():
    y = np.linspace(-6, 6, 97)
    t = torch.from_numpy(y)
    np.testing.assert_allclose(O.gelu_tanh(y), torch.nn.functional.gelu(t, approximate="tanh").numpy(), atol=1e-14)
    np.testing.assert_allclose(O.silu(y), torch.nn.functional.silu(t).numpy(), atol=1e-14)
    h = np.random.default_rng(8).standard_normal((5, 16))
    g = np.random.default_rng(9).standard_normal(16)
    ref = torch.nn.functional.rms_norm(torch.from_numpy(h), (16,), torch.from_numpy(g), eps=1e-6)
    np.testing.assert_allclose(O.rmsnorm(h, g, 1e-6), ref.numpy(), atol=1e-14)


def test_gelu_variant_is_tanh_not_erf():
    # tabulated: gelu_tanh(1) = 0.841192, gelu_erf(1) = 0.841345
    assert abs(float(O.gelu_tanh(np.array(1.0))) - 0.841192) < 5e-7
    assert abs(float(O.gelu_tanh(np.array(1.0))) - 0.841345) > 1e-4


def test_rmsnorm_eps_inside_sqrt_and_plain_gain():
    h = np.zeros((1, 4))
    np.testing.assert_array_equal(O.rmsnorm(h, np.ones(4), 1e-6), h)
    h = np.full((1, 4), 2.0)
    np.testing.assert_allclose(O.rmsnorm(h, np.full(4, 3.0), 0.0), np.full((1, 4), 3.0))
    np.testing.assert_allclose(O.rmsnorm(np.full((1, 4), 1e-3), np.ones(4), 1e-6), np.full((1, 4), 1e-3 / math.sqrt(2e-6)))


# ---- P7: grouped-query attention equals multi-head attention with replicated K/V --------------

def test_gqa_equals_replicated_mha():
    cfg_g = W.scaled(SMALL, n_q_heads=4, n_kv_heads=1)
    cfg_m = W.scaled(SMALL, n_q_heads=4, n_kv_heads=4)
    wl, w = small_inputs(cfg=cfg_g)
    got = run(wl, w)
    w2 = dict(w)
    for l in range(cfg_g.n_layers):
        for nm in ("wk", "wv"):
            w2[f"layers.{l}.{nm}"] = np.tile(w[f"layers.{l}.{nm}"], (1, 4))
    kv2 = [np.repeat(kv, 4, axis=2) for kv in wl.prefix_kv]
    want = O.adit_denoise(cfg_m, w2, kv2, wl.prefix_len, wl.state, wl.noise, wl.n_steps)
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-13)


def test_gqa_head_mapping_is_blockwise():
    # With 2 kv heads and 4 query heads, heads {0,1} read kv head 0 and {2,3} read kv head 1.
    rng = np.random.default_rng(10)
    n, dh = 3, 2
    ks = np.zeros((n, 2, dh)); kp = np.zeros((2, 1, dh))
    vs = np.zeros((n, 2, dh)); vs[:, 0] = 1.0; vs[:, 1] = 2.0
    vp = np.zeros((2, 1, dh)); vp[0] = 1.0; vp[1] = 2.0
    out = O.attention(rng.standard_normal((n, 4, dh)), ks, vs, kp, vp, 1)
    np.testing.assert_allclose(out[:, 0], 1.0); np.testing.assert_allclose(out[:, 1], 1.0)
    np.testing.assert_allclose(out[:, 2], 2.0); np.testing.assert_allclose(out[:, 3], 2.0)


# ---- P8: invariants --------------------------------------------------------------------------

def test_batch_permutation():
    wl, w = small_inputs()
    base = run(wl, w)
    perm = [2, 0, 1]
    got = O.adit_denoise(wl.cfg, w, [wl.prefix_kv[i] for i in perm], wl.prefix_len[perm], wl.state[perm],
                         wl.noise[perm], wl.n_steps)
    np.testing.assert_array_equal(got, base[perm])


def test_request_alone_equals_request_in_batch():
    wl, w = small_inputs()
    base = run(wl, w)
    for b in range(wl.batch):
        got = O.adit_denoise(wl.cfg, w, [wl.prefix_kv[b]], wl.prefix_len[b:b + 1], wl.state[b:b + 1],
                             wl.noise[b:b + 1], wl.n_steps)
        np.testing.assert_array_equal(got[0], base[b])


def test_padding_and_capacity_do_not_matter():
    wl_nan, w = small_inputs(cap=9)
    wl_zero, _ = small_inputs(cap=9, pad_value=0.0)
    wl_rand, _ = small_inputs(cap=9, pad_seed=99)
    wl_big, _ = small_inputs(cap=16)
    base = run(wl_nan, w)
    assert np.isfinite(base).all()
    assert np.isnan(wl_nan.prefix_kv[0][:, :, :, 7:, :]).all()
    for other in (wl_zero, wl_rand, wl_big):
        np.testing.assert_array_equal(run(other, w), base)


def test_prefix_rows_do_matter():
    wl, w = small_inputs()
    base = run(wl, w)
    wl.prefix_kv[0][1, 1, 0, 6, :] += 1.0      # last valid V row of request 0, layer 1
    changed = run(wl, w)
    assert np.abs(changed[0] - base[0]).max() > 1e-9
    np.testing.assert_array_equal(changed[1:], base[1:])


def test_softmax_rows():
    s = np.random.default_rng(12).standard_normal((4, 9)) * 30
    p = O.softmax_rows(s)
    np.testing.assert_allclose(p.sum(-1), 1.0, atol=1e-15)
    np.testing.assert_allclose(O.softmax_rows(s + 123.0), p, rtol=1e-12)
    np.testing.assert_allclose(O.softmax_rows(np.log(np.array([[1.0, 2.0, 5.0]]))), [[0.125, 0.25, 0.625]], rtol=1e-14)


def test_state_token_matters_but_is_not_read_out():
    wl, w = small_inputs()
    base = run(wl, w)
    assert base.shape == (wl.batch, wl.cfg.horizon, wl.cfg.action_dim)
    wl.state[1] += 0.5
    changed = run(wl, w)
    assert np.abs(changed[1] - base[1]).max() > 1e-9       # reaches the actions through attention
    np.testing.assert_array_equal(changed[0], base[0])


def test_state_token_has_no_time_conditioning():
    wl, w = small_inputs()
    wf = O.as_f64_weights(w)
    x = wl.noise[0].astype(np.float64)
    s = wl.state[0].astype(np.float64)
    e0 = O.embed_tokens(wl.cfg, wf, x, s, 0.0)
    e1 = O.embed_tokens(wl.cfg, wf, x, s, 0.6)
    np.testing.assert_array_equal(e0[0], e1[0])
    np.testing.assert_allclose(e0[0], s @ wf["state_in.w"] + wf["state_in.b"])
    assert np.abs(e0[1:] - e1[1:]).max() > 1e-6


# ---- P9: time embedding ----------------------------------------------------------------------

def test_time_embedding_special_values():
    dim, pmin, pmax = 16, 4e-3, 4.0
    half = dim // 2
    t0 = O.time_embedding(0.0, dim, pmin, pmax)
    np.testing.assert_array_equal(t0[:half], 0.0)
    np.testing.assert_array_equal(t0[half:], 1.0)
    t = 0.3
    e = O.time_embedding(t, dim, pmin, pmax)
    assert abs(e[0] - math.sin(2 * math.pi * t / 4e-3)) < 1e-9
    assert abs(e[half - 1] - math.sin(2 * math.pi * t / 4.0)) < 1e-12
    assert abs(e[half] - math.cos(2 * math.pi * t / 4e-3)) < 1e-9
    np.testing.assert_allclose(e[:half] ** 2 + e[half:] ** 2, 1.0, atol=1e-12)
    # geometric spacing of the periods: middle sine uses sqrt(pmin*pmax) when half is odd
    e9 = O.time_embedding(t, 18, pmin, pmax)
    assert abs(e9[4] - math.sin(2 * math.pi * t / math.sqrt(pmin * pmax))) < 1e-10


def test_time_embedding_differs_from_base_10000_form():
    e = O.time_embedding(0.5, 8, 4e-3, 4.0)
    alt = np.array([math.sin(0.5 / 10000 ** (j / 4)) for j in range(4)])
    assert np.abs(e[:4] - alt).max() > 0.1


# ---- P11: earliest-SLO-first ordering --------------------------------------------------------

def test_esf_matches_brute_force():
    import itertools
    rng = np.random.default_rng(13)
    for _ in range(20):
        n = int(rng.integers(1, 6))
        arr = rng.integers(0, 5, size=n) * 1000
        ids = list(range(n))
        now, slo = 7000, 50000
        got = O.esf_order(arr, slo, now, ids)
        key = lambda i: (arr[i] + slo - now, arr[i], ids[i])
        ok = [list(p) for p in itertools.permutations(range(n)) if all(key(p[j]) <= key(p[j + 1]) for j in range(n - 1))]
        assert got in ok and len(ok) == 1


# ---- P12: the wiring of one layer, with non-zero Wo and Wd -----------------------------------------

def _layer_by_torch(cfg, w, l, h, kv_l, plen):
    """One pre-norm block composed from torch CPU fp64 library routines and explicit products, written from the
    definition (attention sub-block, then GeGLU MLP sub-block), without calling the oracle."""
    import torch
    import torch.nn.functional as F
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.float64))
    p = f"layers.{l}."
    x = t(h)
    n, D = x.shape
    Hq, Hkv, dh = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    u = F.rms_norm(x, (D,), weight=t(w[p + "norm1.g"]), eps=cfg.rms_eps)
    q = (u @ t(w[p + "wq"])).view(n, Hq, dh).transpose(0, 1)                       # [Hq, n, dh]
    k = (u @ t(w[p + "wk"])).view(n, Hkv, dh).transpose(0, 1)
    v = (u @ t(w[p + "wv"])).view(n, Hkv, dh).transpose(0, 1)
    k_all = torch.cat([t(kv_l[0][:, :plen]), k], dim=1).repeat_interleave(Hq // Hkv, dim=0)   # [Hq, plen + n, dh]
    v_all = torch.cat([t(kv_l[1][:, :plen]), v], dim=1).repeat_interleave(Hq // Hkv, dim=0)
    o = F.scaled_dot_product_attention(q, k_all, v_all)                              # no mask, scale 1/sqrt(dh)
    x = x + o.transpose(0, 1).reshape(n, Hq * dh) @ t(w[p + "wo"])
    u = F.rms_norm(x, (D,), weight=t(w[p + "norm2.g"]), eps=cfg.rms_eps)
    x = x + (F.gelu(u @ t(w[p + "wg"]), approximate="tanh") * (u @ t(w[p + "wu"]))) @ t(w[p + "wd"])
    return x.numpy()


def _layer_case():
    cfg = W.scaled(W.TINY, n_layers=1, d_model=32, n_q_heads=4, n_kv_heads=2, head_dim=8, d_ff=48, horizon=5,
                   time_emb_dim=32)
    rng = np.random.default_rng(99)
    w = {k: np.asarray(v, dtype=np.float64) for k, v in W.make_weights(cfg, 7).items()}
    for k in list(w):                       # weights large enough for every term to matter
        if k.startswith("layers.0.w"):
            w[k] = rng.standard_normal(w[k].shape) * 0.3
        if k.endswith(".g"):
            w[k] = 1.0 + 0.5 * rng.standard_normal(w[k].shape)
    h = rng.standard_normal((cfg.n_tokens, cfg.d_model))
    plen, cap = 7, 9
    kv = rng.standard_normal((2, cfg.n_kv_heads, cap, cfg.head_dim))
    kv[:, :, plen:] = np.nan
    return cfg, w, h, kv, plen


def test_layer_forward_matches_library_composition():
    cfg, w, h, kv, plen = _layer_case()
    got = O.layer_forward(cfg, w, 0, h, kv, plen)
    want = _layer_by_torch(cfg, w, 0, h, kv, plen)
    assert np.isfinite(got).all()
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-12)
    assert np.abs(got - h).max() > 0.5      # both residual branches contribute: the layer is far from the identity


def test_layer_wiring_mistakes_are_visible():
    """Each plausible wiring mistake changes the library composition's result by far more than the tolerance of the
    comparison above, so the oracle cannot contain it and still pass: gate/up swapped, the first norm's gain in the
    second norm, value weights used for the keys, un-normalised input to the query projection, a dropped residual."""
    cfg, w, h, kv, plen = _layer_case()
    want = _layer_by_torch(cfg, w, 0, h, kv, plen)
    p = "layers.0."
    swaps = {"gate/up": {p + "wg": w[p + "wu"], p + "wu": w[p + "wg"]},
             "norm gains": {p + "norm2.g": w[p + "norm1.g"]},
             "wk<-wv": {p + "wk": w[p + "wv"]}}
    for name, repl in swaps.items():
        w2 = dict(w)
        w2.update(repl)
        assert np.abs(O.layer_forward(cfg, w2, 0, h, kv, plen) - want).max() > 1e-3, name
    # un-normalised input to wq == folding 1/rms out of the query: emulate by scaling the rows of h for q only
    w3 = dict(w)
    w3[p + "wq"] = w[p + "wq"] * 1.7
    assert np.abs(O.layer_forward(cfg, w3, 0, h, kv, plen) - want).max() > 1e-3
    w4 = dict(w)
    w4[p + "wo"] = np.zeros_like(w[p + "wo"])
    assert np.abs(O.layer_forward(cfg, w4, 0, h, kv, plen) - want).max() > 1e-3


# ---- P13: model-fidelity variants (state-block mask, rotary embedding on the suffix) ---------------------------

def test_state_block_mask_against_library_and_scalar_loop():
    import torch
    import torch.nn.functional as F
    rng = np.random.default_rng(31)
    n, hq, hkv, dh, plen, cap = 4, 4, 2, 8, 5, 7
    q = rng.standard_normal((n, hq, dh)); ks = rng.standard_normal((n, hkv, dh)); vs = rng.standard_normal((n, hkv, dh))
    kp = rng.standard_normal((hkv, cap, dh)); vp = rng.standard_normal((hkv, cap, dh))
    kp[:, plen:] = np.nan; vp[:, plen:] = np.nan
    got = O.attention(q, ks, vs, kp, vp, plen, state_block_mask=True)
    plain = O.attention(q, ks, vs, kp, vp, plen)
    # library: boolean mask, True = may attend
    allow = torch.ones(n, plen + n, dtype=torch.bool)
    allow[0, plen + 1:] = False
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a))
    k_all = torch.cat([t(kp[:, :plen]), t(ks).transpose(0, 1)], dim=1).repeat_interleave(hq // hkv, dim=0)
    v_all = torch.cat([t(vp[:, :plen]), t(vs).transpose(0, 1)], dim=1).repeat_interleave(hq // hkv, dim=0)
    want = F.scaled_dot_product_attention(t(q).transpose(0, 1), k_all, v_all, attn_mask=allow).transpose(0, 1).numpy()
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-12)
    # the action tokens are not affected; the state token is
    np.testing.assert_array_equal(got[1:], plain[1:])
    assert np.abs(got[0] - plain[0]).max() > 1e-3
    # scalar loop for the state row of head 3: prefix keys and its own key only
    h, kvh = 3, 1
    keys = [kp[kvh, j] for j in range(plen)] + [ks[0, kvh]]
    vals = [vp[kvh, j] for j in range(plen)] + [vs[0, kvh]]
    sc = [sum(q[0, h, c] * kk[c] for c in range(dh)) / math.sqrt(dh) for kk in keys]
    mx = max(sc)
    ws = [math.exp(v - mx) for v in sc]
    for c in range(dh):
        assert abs(got[0, h, c] - sum(wj * vj[c] for wj, vj in zip(ws, vals)) / sum(ws)) < 1e-12


def test_state_token_stream_ignores_the_action_tokens_under_the_mask():
    cfg, w, h, kv, plen = _layer_case()
    cfg_m = W.scaled(cfg, state_block_mask=True)
    h2 = h.copy()
    h2[1:] += 3.0 * np.random.default_rng(5).standard_normal(h2[1:].shape)
    a, b = O.layer_forward(cfg_m, w, 0, h, kv, plen), O.layer_forward(cfg_m, w, 0, h2, kv, plen)
    np.testing.assert_allclose(a[0], b[0], rtol=0, atol=1e-13)          # row 0 never saw rows 1..
    a, b = O.layer_forward(cfg, w, 0, h, kv, plen), O.layer_forward(cfg, w, 0, h2, kv, plen)
    assert np.abs(a[0] - b[0]).max() > 1e-3                             # without the mask it does


def test_rotary_embedding_closed_forms():
    # two channels: one pair, angle = position (10000 ** 0 = 1)
    for pos in (0.0, 1.0, 2.5, 817.0):
        np.testing.assert_allclose(O.rope(np.array([1.0, 0.0]), pos), [math.cos(pos), math.sin(pos)], atol=1e-12)
        np.testing.assert_allclose(O.rope(np.array([0.0, 1.0]), pos), [-math.sin(pos), math.cos(pos)], atol=1e-12)
    rng = np.random.default_rng(41)
    x, y = rng.standard_normal(16), rng.standard_normal(16)
    np.testing.assert_array_equal(O.rope(x, 0), x)                                   # position 0: identity
    assert abs(np.linalg.norm(O.rope(x, 123.0)) - np.linalg.norm(x)) < 1e-12          # a rotation
    # channel j is paired with channel j + dh/2, and pair j turns by pos * 10000 ** (-2 j / dh)
    j, pos = 3, 7.0
    e = np.zeros(16); e[j] = 1.0
    r = O.rope(e, pos)
    ang = pos * 10000.0 ** (-2 * j / 16)
    assert abs(r[j] - math.cos(ang)) < 1e-12 and abs(r[j + 8] - math.sin(ang)) < 1e-12 and abs(np.abs(r).sum() - abs(math.cos(ang)) - abs(math.sin(ang))) < 1e-12
    # a score depends on the difference of the positions only
    s1 = O.rope(x, 900.0) @ O.rope(y, 893.0)
    s2 = O.rope(x, 12.0) @ O.rope(y, 5.0)
    assert abs(s1 - s2) < 1e-9


def test_suffix_rope_changes_the_layer_and_reduces_to_plain_at_identity_positions():
    cfg, w, h, kv, plen = _layer_case()
    cfg_r = W.scaled(cfg, suffix_rope=True)
    plain, rot = O.layer_forward(cfg, w, 0, h, kv, plen), O.layer_forward(cfg_r, w, 0, h, kv, plen)
    assert np.isfinite(rot).all() and np.abs(rot - plain).max() > 1e-3
    # a single suffix token without a prefix sits at position 0, where the rotation is the identity
    one, empty = h[:1], kv[:, :, :0]
    np.testing.assert_allclose(O.layer_forward(cfg_r, w, 0, one, empty, 0), O.layer_forward(cfg, w, 0, one, empty, 0), atol=1e-13)


# ---- the full configurations run and are healthy --------------------------------------------

def test_prefix_projection_against_scalar_loops_and_selection_weights():
    """P14: the hidden-state hand-over.  (a) every cache element recomputed by a scalar triple loop that indexes the
    cache layout itself; (b) with selection matrices as weights, keys are the first and values the last KV
    columns of the hidden states, reversed for the values - a transposed operand, a swapped K/V plane or a
    head-minor column order fails one of them; (c) rows at or beyond the prefix length keep the padding."""
    cfg = SMALL
    rng = np.random.default_rng(140)
    Dh, P, cap = 12, 5, 7
    KV = cfg.n_kv_heads * cfg.head_dim
    H = rng.standard_normal((P, Dh))
    pw = {f"layers.{l}.{leaf}": rng.standard_normal((Dh, KV)) for l in range(cfg.n_layers) for leaf in ("prefix_wk", "prefix_wv")}
    kv = O.project_prefix_kv(cfg, H, pw, cap, pad_value=-7.0)
    assert kv.shape == (cfg.n_layers, 2, cfg.n_kv_heads, cap, cfg.head_dim)
    for l in range(cfg.n_layers):
        for which, leaf in enumerate(("prefix_wk", "prefix_wv")):
            Wm = pw[f"layers.{l}.{leaf}"]
            for g in range(cfg.n_kv_heads):
                for p in range(P):
                    for c in range(cfg.head_dim):
                        acc = 0.0
                        for i in range(Dh):
                            acc += H[p, i] * Wm[i, g * cfg.head_dim + c]
                        assert abs(kv[l, which, g, p, c] - acc) < 1e-12
    assert np.all(kv[:, :, :, P:, :] == -7.0)
    # (b) selection weights
    Dh2 = 2 * KV
    H2 = rng.standard_normal((P, Dh2))
    sel_k = np.zeros((Dh2, KV)); sel_v = np.zeros((Dh2, KV))
    for j in range(KV):
        sel_k[j, j] = 1.0                 # key column j = hidden column j
        sel_v[Dh2 - 1 - j, j] = 1.0       # value column j = hidden column Dh2 - 1 - j
    pw2 = {}
    for l in range(cfg.n_layers):
        pw2[f"layers.{l}.prefix_wk"] = sel_k * (l + 1)
        pw2[f"layers.{l}.prefix_wv"] = sel_v * (l + 1)
    kv2 = O.project_prefix_kv(cfg, H2, pw2, P)
    for l in range(cfg.n_layers):
        for g in range(cfg.n_kv_heads):
            lo = g * cfg.head_dim
            np.testing.assert_allclose(kv2[l, 0, g], (l + 1) * H2[:, lo:lo + cfg.head_dim], atol=0, rtol=0)
            np.testing.assert_allclose(kv2[l, 1, g], (l + 1) * H2[:, ::-1][:, lo:lo + cfg.head_dim], atol=0, rtol=0)
    # an empty prefix projects to nothing
    assert np.all(np.isnan(O.project_prefix_kv(cfg, np.zeros((0, Dh)), pw, 3)))


def test_config_c1_runs_and_signal_is_healthy():
    wl = W.config_c1()
    w = W.make_weights(wl.cfg, wl.seed)
    out = run(wl, w)
    assert out.shape == (2, 16, 7) and np.isfinite(out).all()
    assert 0.05 < np.abs(out - wl.noise).mean() < 5.0      # the network actually moves x


def test_config_c1_matches_stored_fixture():
    # regression fixture written by tests/golden/make_golden.py (calls only the oracle)
    import os
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "c1_oracle.txt")
    want = np.loadtxt(path).reshape(2, 16, 7)
    wl = W.config_c1()
    got = run(wl, W.make_weights(wl.cfg, wl.seed))
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-13)
