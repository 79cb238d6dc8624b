"""CPU oracle (fp64, numpy) for the batched ADiT denoising loop.  TEST INFRASTRUCTURE ONLY.

This is the slow, plain definition the CUDA library is checked against.  Only
tests, the smoke check and the benchmark's CPU-baseline leg may import it; the
product path never does, and this file imports nothing from the CUDA side.

What the paper fixes (section 2.1, "Vision-Language-Action Models"): the ADiT
stage follows the VLM, consumes per-request intermediate tensors such as a small
KV cache, and runs a fixed number of diffusion steps (typically 5-10) to emit a
chunk of 10-50 future actions; section 4.1.1 fixes the batch for the duration of
the stage and keeps each request's VLM tensors separate (not packed).  The
paper gives no equations for the network itself.  Everything below is therefore
the following reading, taken step by step, one request at a time:

* sampler: deterministic forward Euler on a flow-matching velocity field,
  t_k = k/K for k = 0..K-1, dt = 1/K, velocity evaluated at the left end point,
  x_0 = noise, result x_K;
* tokens: one state token (state @ Ws + bs, first, no time conditioning) then
  `horizon` action tokens  W2 . silu(W1 . [Wa x + ba ; tau(t)] + b1) + b2;
* tau(t): sinusoidal, `time_emb_dim` wide, log-spaced periods from t_min_period
  to t_max_period, all sines first, then all cosines;
* layer: pre-norm residual block, attention then GeGLU MLP; RMSNorm over the
  width with eps inside the square root and a plain multiplicative gain;
* attention: every suffix token (state included) attends to the request's
  prefix keys [0, prefix_len) followed by all suffix keys, no mask inside that
  set, no positional term, scale 1/sqrt(head_dim), query head h reads kv head
  h // (n_q_heads / n_kv_heads);
* variants, off unless the configuration asks for them: `state_block_mask` - the state token's query attends to
  the prefix keys and its own key only (the action tokens still attend to everything); `suffix_rope` - the
  suffix queries and keys of every head are rotated by the angles pos * 10000**(-2j/head_dim), j < head_dim/2,
  pairing channel j with channel j + head_dim/2, at position pos = prefix_len + (index of the token in the
  suffix); prefix keys are used as given (their producer has rotated them);
* hidden-state hand-over (section 2.1 names hidden states beside the KV cache as what the VLM may hand over):
  `project_prefix_kv` - the expert projects the handed-over hidden states H [P, Dh] to each layer's prefix keys
  and values itself, K_l = H Wk_l, V_l = H Wv_l (no norm, bias or rotation), once per call; the loop then runs on
  that cache;
* GeGLU: tanh-approximate GELU on the gate times the up projection;
* read-out: final RMSNorm, then Wout, bout, on the action tokens only.

Pins (tests/test_oracle_pins.py): closed-form Euler trajectories for linear
fields; Wout = 0 gives x_K = x_0 + bout; zeroed Wo/Wd give a hand-computable
velocity; one whole layer with non-zero Wo/Wd against a composition of torch
CPU fp64 library routines (norm -> q/k/v, attention, residual, norm ->
GeGLU, residual); scalar-loop softmax attention on tiny shapes; zero queries give the
mean of the valid value rows; torch CPU fp64 library routines for attention,
RMSNorm, GELU(tanh) and SiLU; grouped-query = replicated multi-head; batch
permutation, padding and capacity invariance; time-embedding special values;
for the variants: the masked attention against torch's masked attention and a
scalar loop, the state token's independence of the action tokens; the rotary
embedding against its closed form in two dimensions, norm preservation, the
identity at position 0 and the dependence of a score on the position difference only;
the hand-over projection against scalar loops and, with selection matrices as weights, against slices of the
hidden states themselves.
Parity unpinned: the behaviour of a *trained* model (no weights or reference
outputs exist); the oracle pins the computation, not robot behaviour.
"""
from __future__ import annotations

import math
from typing import Callable, Dict, List, Optional, Sequence

import numpy as np

F64 = np.float64


def time_embedding(t: float, dim: int, min_period: float, max_period: float) -> np.ndarray:
    """tau(t) = [sin(2 pi t / p_j) for j < dim/2] ++ [cos(2 pi t / p_j) for j < dim/2],
    p_j = min_period * (max_period / min_period) ** (j / (dim/2 - 1))."""
    half = dim // 2
    assert dim == 2 * half and half >= 2
    frac = np.arange(half, dtype=F64) / F64(half - 1)
    period = F64(min_period) * (F64(max_period) / F64(min_period)) ** frac
    ang = 2.0 * math.pi * F64(t) / period
    return np.concatenate([np.sin(ang), np.cos(ang)])


def silu(y: np.ndarray) -> np.ndarray:
    return y / (1.0 + np.exp(-y))


def gelu_tanh(y: np.ndarray) -> np.ndarray:
    return 0.5 * y * (1.0 + np.tanh(math.sqrt(2.0 / math.pi) * (y + 0.044715 * y ** 3)))


def rmsnorm(h: np.ndarray, g: np.ndarray, eps: float) -> np.ndarray:
    """Row-wise h / sqrt(mean(h^2) + eps) * g."""
    ms = np.mean(h * h, axis=-1, keepdims=True)
    return h / np.sqrt(ms + eps) * g


def softmax_rows(s: np.ndarray) -> np.ndarray:
    e = np.exp(s - np.max(s, axis=-1, keepdims=True))
    return e / np.sum(e, axis=-1, keepdims=True)


ROPE_BASE = 10000.0


def rope(x: np.ndarray, pos: float) -> np.ndarray:
    """Rotary embedding of the last axis at position pos: channel pair (j, j + dh/2) is rotated by the angle
    pos * ROPE_BASE ** (-2 j / dh)."""
    dh = x.shape[-1]
    half = dh // 2
    assert dh == 2 * half
    ang = F64(pos) * ROPE_BASE ** (-np.arange(half, dtype=F64) / F64(half))
    c, s_ = np.cos(ang), np.sin(ang)
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s_, x2 * c + x1 * s_], axis=-1)


def attention(q: np.ndarray, k_suffix: np.ndarray, v_suffix: np.ndarray,
              k_prefix: np.ndarray, v_prefix: np.ndarray, prefix_len: int,
              state_block_mask: bool = False) -> np.ndarray:
    """One request, one layer.

    q [N, Hq, dh]; k_suffix, v_suffix [N, Hkv, dh]; k_prefix, v_prefix
    [Hkv, capacity, dh] of which only rows [0, prefix_len) are read.
    With state_block_mask the first suffix token (the state token) does not see the suffix keys 1..N-1.
    Returns [N, Hq, dh].
    """
    n, hq, dh = q.shape
    hkv = k_suffix.shape[1]
    group = hq // hkv
    assert group * hkv == hq
    out = np.empty((n, hq, dh), dtype=F64)
    for h in range(hq):
        kv = h // group
        k_all = np.concatenate([k_prefix[kv, :prefix_len, :], k_suffix[:, kv, :]], axis=0)
        v_all = np.concatenate([v_prefix[kv, :prefix_len, :], v_suffix[:, kv, :]], axis=0)
        s = (q[:, h, :] @ k_all.T) / math.sqrt(dh)
        if state_block_mask:
            s[0, prefix_len + 1:] = -np.inf
        out[:, h, :] = softmax_rows(s) @ v_all
    return out


def project_prefix_kv(cfg, hidden: np.ndarray, prefix_w: Dict[str, np.ndarray], max_prefix_len: int,
                      pad_value: float = float("nan")) -> np.ndarray:
    """Hidden-state hand-over (section 2.1): hidden [P, Dh] -> the request's prefix cache
    [n_layers, 2, n_kv_heads, max_prefix_len, head_dim] with K_l = H Wk_l and V_l = H Wv_l in rows < P
    (columns of the products are head-major: column = kv head * head_dim + channel); rows >= P hold pad_value."""
    hidden = np.asarray(hidden, dtype=F64)
    P = hidden.shape[0]
    kv = np.full((cfg.n_layers, 2, cfg.n_kv_heads, max_prefix_len, cfg.head_dim), pad_value, dtype=F64)
    for l in range(cfg.n_layers):
        for which, leaf in enumerate(("prefix_wk", "prefix_wv")):
            y = hidden @ np.asarray(prefix_w[f"layers.{l}.{leaf}"], dtype=F64)  # [P, n_kv_heads * head_dim]
            for g in range(cfg.n_kv_heads):
                kv[l, which, g, :P, :] = y[:, g * cfg.head_dim:(g + 1) * cfg.head_dim]
    return kv


def embed_tokens(cfg, w: Dict[str, np.ndarray], x: np.ndarray, state: np.ndarray, t: float) -> np.ndarray:
    """Residual-stream input [1 + horizon, D]: row 0 the state token, rows 1.. the action tokens."""
    tau = time_embedding(t, cfg.time_emb_dim, cfg.t_min_period, cfg.t_max_period)
    a = x @ w["action_in.w"] + w["action_in.b"]                                  # [Ta, D]
    cat = np.concatenate([a, np.broadcast_to(tau, (a.shape[0], tau.shape[0]))], axis=1)
    z = silu(cat @ w["time_mlp.w1"] + w["time_mlp.b1"])
    h_act = z @ w["time_mlp.w2"] + w["time_mlp.b2"]
    h_state = state @ w["state_in.w"] + w["state_in.b"]
    return np.concatenate([h_state[None, :], h_act], axis=0)


def layer_forward(cfg, w: Dict[str, np.ndarray], l: int, h: np.ndarray,
                  kv_prefix_l: np.ndarray, prefix_len: int) -> np.ndarray:
    """One pre-norm block.  kv_prefix_l is [2, Hkv, capacity, dh] (0 = K, 1 = V)."""
    p = f"layers.{l}."
    n = h.shape[0]
    u = rmsnorm(h, w[p + "norm1.g"], cfg.rms_eps)
    q = (u @ w[p + "wq"]).reshape(n, cfg.n_q_heads, cfg.head_dim)
    kc = (u @ w[p + "wk"]).reshape(n, cfg.n_kv_heads, cfg.head_dim)
    vc = (u @ w[p + "wv"]).reshape(n, cfg.n_kv_heads, cfg.head_dim)
    if getattr(cfg, "suffix_rope", False):
        for i in range(n):
            q[i] = rope(q[i], prefix_len + i)
            kc[i] = rope(kc[i], prefix_len + i)
    o = attention(q, kc, vc, kv_prefix_l[0], kv_prefix_l[1], prefix_len,
                  state_block_mask=getattr(cfg, "state_block_mask", False))
    h = h + o.reshape(n, cfg.q_dim) @ w[p + "wo"]
    u = rmsnorm(h, w[p + "norm2.g"], cfg.rms_eps)
    h = h + (gelu_tanh(u @ w[p + "wg"]) * (u @ w[p + "wu"])) @ w[p + "wd"]
    return h


def velocity(cfg, w: Dict[str, np.ndarray], x: np.ndarray, state: np.ndarray, t: float,
             kv_prefix: np.ndarray, prefix_len: int, trace: Optional[dict] = None) -> np.ndarray:
    """v(x, t) for one request: [horizon, action_dim]."""
    h = embed_tokens(cfg, w, x, state, t)
    if trace is not None:
        trace["embed"] = h.copy()
    for l in range(cfg.n_layers):
        h = layer_forward(cfg, w, l, h, np.asarray(kv_prefix[l], dtype=F64), prefix_len)
        if trace is not None:
            trace[f"h{l}"] = h.copy()
    u = rmsnorm(h[1:], w["final_norm.g"], cfg.rms_eps)
    return u @ w["action_out.w"] + w["action_out.b"]


def euler_integrate(field: Callable[[np.ndarray, float], np.ndarray], x0: np.ndarray, n_steps: int) -> np.ndarray:
    """x_{k+1} = x_k + (1/K) field(x_k, k/K), k = 0..K-1; returns x_K."""
    x = np.array(x0, dtype=F64, copy=True)
    dt = 1.0 / n_steps
    for k in range(n_steps):
        x = x + dt * field(x, k / n_steps)
    return x


def as_f64_weights(weights: Dict[str, np.ndarray]) -> Dict[str, np.ndarray]:
    return {k: np.asarray(v, dtype=F64) for k, v in weights.items()}


def adit_denoise(cfg, weights: Dict[str, np.ndarray], prefix_kv: Sequence[np.ndarray],
                 prefix_len: Sequence[int], state: np.ndarray, noise: np.ndarray, n_steps: int,
                 traces: Optional[List[dict]] = None) -> np.ndarray:
    """Action chunks [B, horizon, action_dim] (fp64) for a batch of independent requests.

    prefix_kv[b] is [n_layers, 2, n_kv_heads, capacity, head_dim]; only rows below
    prefix_len[b] are read.
    """
    w = as_f64_weights(weights)
    batch = len(prefix_len)
    out = np.empty((batch, cfg.horizon, cfg.action_dim), dtype=F64)
    for b in range(batch):
        st = np.asarray(state[b], dtype=F64)
        kv = prefix_kv[b]
        plen = int(prefix_len[b])
        tr = None
        if traces is not None:
            tr = {}
            traces.append(tr)

        def field(x, t, _st=st, _kv=kv, _plen=plen, _tr=tr):
            return velocity(cfg, w, x, _st, t, _kv, _plen, trace=_tr if t == 0.0 else None)

        out[b] = euler_integrate(field, np.asarray(noise[b], dtype=F64), n_steps)
    return out


# ---- request ordering used by the two-expert trace driver (paper section 4.1.3) --------------

def esf_order(arrival_us: Sequence[int], slo_us: int, now_us: int, request_id: Sequence[int]) -> List[int]:
    """Earliest-SLO-first: indices sorted by remaining slack arrival + slo - now (integer
    microseconds), ties by earlier arrival, then lower request id."""
    idx = list(range(len(arrival_us)))
    idx.sort(key=lambda i: (int(arrival_us[i]) + int(slo_us) - int(now_us), int(arrival_us[i]), int(request_id[i])))
    return idx
