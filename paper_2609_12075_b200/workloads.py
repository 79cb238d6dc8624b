"""Seeded synthetic inputs for the ADiT denoising loop.

This module only *draws* numbers and lays them out; it contains none of the
method's arithmetic (no projections, norms, attention or integration), so the
CPU oracle and the CUDA path can both consume it without sharing any of the
computation under test.

Every tensor comes from its own generator ``numpy.random.default_rng([seed,
tensor_id])`` (PCG64), so the order in which tensors are generated never
matters.  ``tensor_id`` table:

    0            prefix lengths
    1            noise          [B, horizon, action_dim]
    2            state          [B, state_dim]
    3            request arrival times (trace workloads)
    10 + i       the i-th weight tensor in ``weight_names(cfg)`` order
    1000 + 1000*b + l   request b, layer l prefix K then V (valid rows only)

Distributions: matrices and biases 0.02 * N(0,1); norm gains 1 + 0.02 * N(0,1);
prefix K, V, noise and state N(0,1).  For ``dtype == "bf16"`` weights and
prefix K/V are rounded once (round-to-nearest-even) to bfloat16 and both the
oracle and the GPU consume those rounded values.

The paper evaluates on trained models fed from a robot-manipulation dataset;
neither is needed for (or available to) this path, whose cost depends only on
shapes.  These inputs stand in for it.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, List, Optional, Sequence

import numpy as np

WEIGHT_STD = 0.02


@dataclass(frozen=True)
class ADiTConfig:
    """Shape family of one action expert (paper section 2.1: the ADiT stage)."""

    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ff: int
    horizon: int
    action_dim: int
    state_dim: int
    time_emb_dim: int
    dtype: str = "bf16"  # "fp32" (debug path) or "bf16" (bf16 operands, fp32 accumulation)
    rms_eps: float = 1e-6
    t_min_period: float = 4e-3
    t_max_period: float = 4.0
    # model-fidelity variants (off in the configurations of the benchmark)
    state_block_mask: bool = False   # the state token attends to the prefix and itself only, not to the action tokens
    suffix_rope: bool = False        # rotary position embedding on the suffix queries/keys at positions prefix_len + i

    @property
    def n_tokens(self) -> int:
        """Suffix tokens per request: one state token then the action tokens."""
        return 1 + self.horizon

    @property
    def q_dim(self) -> int:
        return self.n_q_heads * self.head_dim

    @property
    def kv_dim(self) -> int:
        return self.n_kv_heads * self.head_dim


TINY = ADiTConfig(n_layers=2, d_model=256, n_q_heads=4, n_kv_heads=1, head_dim=64, d_ff=1024,
                  horizon=16, action_dim=7, state_dim=7, time_emb_dim=256, dtype="fp32")
PI0 = ADiTConfig(n_layers=18, d_model=1024, n_q_heads=8, n_kv_heads=1, head_dim=256, d_ff=4096,
                 horizon=50, action_dim=32, state_dim=32, time_emb_dim=1024, dtype="bf16")
EXPERT2 = ADiTConfig(n_layers=16, d_model=1536, n_q_heads=12, n_kv_heads=12, head_dim=128, d_ff=6144,
                     horizon=16, action_dim=32, state_dim=32, time_emb_dim=1536, dtype="bf16")


def weight_names(cfg: ADiTConfig) -> List[str]:
    names = ["action_in.w", "action_in.b", "state_in.w", "state_in.b",
             "time_mlp.w1", "time_mlp.b1", "time_mlp.w2", "time_mlp.b2"]
    for l in range(cfg.n_layers):
        p = f"layers.{l}."
        names += [p + "norm1.g", p + "wq", p + "wk", p + "wv", p + "wo",
                  p + "norm2.g", p + "wg", p + "wu", p + "wd"]
    names += ["final_norm.g", "action_out.w", "action_out.b"]
    return names


def weight_shape(cfg: ADiTConfig, name: str):
    """All matrices are row-major ``[in, out]`` (y = x @ W)."""
    D, F, A, S = cfg.d_model, cfg.d_ff, cfg.action_dim, cfg.state_dim
    leaf = name.split(".")[-1] if name.startswith("layers.") else name
    table = {
        "action_in.w": (A, D), "action_in.b": (D,), "state_in.w": (S, D), "state_in.b": (D,),
        "time_mlp.w1": (D + cfg.time_emb_dim, D), "time_mlp.b1": (D,),
        "time_mlp.w2": (D, D), "time_mlp.b2": (D,),
        "g": (D,), "wq": (D, cfg.q_dim), "wk": (D, cfg.kv_dim), "wv": (D, cfg.kv_dim),
        "wo": (cfg.q_dim, D), "wg": (D, F), "wu": (D, F), "wd": (F, D),
        "final_norm.g": (D,), "action_out.w": (D, A), "action_out.b": (A,),
    }
    return table[leaf]


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16 (ties to even); result stays float32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    bits = a.view(np.uint32)
    rounded = (bits + np.uint32(0x7FFF) + ((bits >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    nan = np.isnan(a)
    out = rounded.view(np.float32).copy()
    out[nan] = np.nan
    return out


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of values that are already bfloat16-representable float32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    return (a.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def _rng(seed: int, tensor_id: int) -> np.random.Generator:
    return np.random.default_rng([int(seed), int(tensor_id)])


def make_weights(cfg: ADiTConfig, seed: int) -> Dict[str, np.ndarray]:
    """Random-initialised weights as float32 arrays (bf16-representable when cfg.dtype == 'bf16')."""
    out: Dict[str, np.ndarray] = {}
    for i, name in enumerate(weight_names(cfg)):
        shape = weight_shape(cfg, name)
        w = _rng(seed, 10 + i).standard_normal(shape).astype(np.float32) * np.float32(WEIGHT_STD)
        if name.endswith(".g"):
            w = np.float32(1.0) + w
        if cfg.dtype == "bf16":
            w = round_to_bf16(w)
        out[name] = w
    return out


def make_prefix_projection(cfg: ADiTConfig, seed: int, hidden_dim: int) -> Dict[str, np.ndarray]:
    """Random-initialised prefix K/V projections of the hidden-state hand-over: layers.<l>.prefix_wk / prefix_wv
    [hidden_dim, n_kv_heads * head_dim], float32 (bf16-representable), scaled so that the projected keys and values
    have about unit variance like the generated caches."""
    out: Dict[str, np.ndarray] = {}
    kv = cfg.n_kv_heads * cfg.head_dim
    for l in range(cfg.n_layers):
        for j, leaf in enumerate(("prefix_wk", "prefix_wv")):
            w = _rng(seed, 50000 + 2 * l + j).standard_normal((hidden_dim, kv)).astype(np.float32)
            out[f"layers.{l}.{leaf}"] = round_to_bf16(w * np.float32(1.0 / np.sqrt(hidden_dim)))
    return out


def make_prefix_hidden(seed: int, b: int, prefix_len: int, hidden_dim: int) -> np.ndarray:
    """Hidden states the VLM stand-in hands over for request ``b``: float32 [prefix_len, hidden_dim], unit variance,
    bf16-representable; depends on (seed, b) only."""
    g = _rng(seed, 70000 + b)
    return round_to_bf16(g.standard_normal((prefix_len, hidden_dim)).astype(np.float32))


@dataclass
class Workload:
    """One batch of requests for ``adit_denoise``.

    ``prefix_kv[b]`` has shape ``[n_layers, 2, n_kv_heads, max_prefix_len, head_dim]``
    (index 0 of the second axis is K, 1 is V); rows at or beyond
    ``prefix_len[b]`` hold ``pad_value`` and must never influence a result.
    """

    name: str
    cfg: ADiTConfig
    seed: int
    batch: int
    n_steps: int
    max_prefix_len: int
    prefix_len: np.ndarray                      # int32 [B]
    noise: np.ndarray                           # float32 [B, horizon, action_dim]
    state: np.ndarray                           # float32 [B, state_dim]
    prefix_kv: List[np.ndarray] = field(default_factory=list)  # float32, see above


def make_prefix_kv(cfg: ADiTConfig, seed: int, b: int, prefix_len: int, max_prefix_len: int,
                   pad_value: float = float("nan"), pad_seed: Optional[int] = None) -> np.ndarray:
    """Prefix K/V of request ``b``.  Valid rows depend only on (seed, b, layer)."""
    kv = np.empty((cfg.n_layers, 2, cfg.n_kv_heads, max_prefix_len, cfg.head_dim), dtype=np.float32)
    if pad_seed is None:
        kv[...] = pad_value
    else:  # random finite garbage in the padding (for padding-independence tests)
        kv[...] = np.random.default_rng([pad_seed, b]).standard_normal(kv.shape).astype(np.float32) * 7.0
    for l in range(cfg.n_layers):
        g = _rng(seed, 1000 + 1000 * b + l)
        vals = g.standard_normal((2, cfg.n_kv_heads, prefix_len, cfg.head_dim)).astype(np.float32)
        if cfg.dtype == "bf16":
            vals = round_to_bf16(vals)
        kv[l, :, :, :prefix_len, :] = vals
    if cfg.dtype == "bf16" and pad_seed is not None:
        kv_pad = round_to_bf16(kv)
        kv = kv_pad
    return kv


def make_workload(name: str, cfg: ADiTConfig, seed: int, batch: int, n_steps: int,
                  prefix_len: Sequence[int] | int | None = None, prefix_range=(600, 900),
                  max_prefix_len: Optional[int] = None, pad_value: float = float("nan"),
                  pad_seed: Optional[int] = None, with_kv: bool = True) -> Workload:
    if prefix_len is None:
        lo, hi = prefix_range
        plen = _rng(seed, 0).integers(lo, hi + 1, size=batch).astype(np.int32)
    elif np.isscalar(prefix_len):
        plen = np.full(batch, int(prefix_len), dtype=np.int32)
    else:
        plen = np.asarray(prefix_len, dtype=np.int32)
        assert plen.shape == (batch,)
    cap = int(max_prefix_len) if max_prefix_len is not None else int(plen.max(initial=0))
    assert cap >= int(plen.max(initial=0))
    noise = _rng(seed, 1).standard_normal((batch, cfg.horizon, cfg.action_dim)).astype(np.float32)
    state = _rng(seed, 2).standard_normal((batch, cfg.state_dim)).astype(np.float32)
    wl = Workload(name=name, cfg=cfg, seed=seed, batch=batch, n_steps=n_steps, max_prefix_len=cap,
                  prefix_len=plen, noise=noise, state=state)
    if with_kv:
        wl.prefix_kv = [make_prefix_kv(cfg, seed, b, int(plen[b]), cap, pad_value, pad_seed)
                        for b in range(batch)]
    return wl


# ----- the named configurations -------------------------------------------------------------

def config_c1(max_prefix_len: int = 64, **kw) -> Workload:
    """Tiny fp32 expert: batch 2, 64 prefix tokens, 4 Euler steps, seed 0."""
    return make_workload("C1-tiny-fp32-B2", TINY, seed=0, batch=2, n_steps=4, prefix_len=64,
                         max_prefix_len=max_prefix_len, **kw)


def config_c2(**kw) -> Workload:
    """pi0-scale expert, batch 1, 816 prefix tokens (3x256 image + 48 text), 10 steps, seed 1."""
    return make_workload("C2-pi0-bf16-B1-P816", PI0, seed=1, batch=1, n_steps=10, prefix_len=816,
                         max_prefix_len=816, **kw)


def config_c3(**kw) -> Workload:
    """pi0-scale expert, batch 16, ragged prefixes uniform in [600, 900], 10 steps, seed 2."""
    return make_workload("C3-pi0-bf16-B16-ragged", PI0, seed=2, batch=16, n_steps=10,
                         prefix_range=(600, 900), max_prefix_len=1024, **kw)


def config_c4(**kw) -> Workload:
    """pi0-scale expert, batch 32, ragged prefixes uniform in [600, 900], 10 steps, seed 3."""
    return make_workload("C4-pi0-bf16-B32-ragged", PI0, seed=3, batch=32, n_steps=10,
                         prefix_range=(600, 900), max_prefix_len=1024, **kw)


def config_c5_expert2(**kw) -> Workload:
    """Second co-located expert: 16 layers, width 1536, 12/12 heads of 128, batch 24, 256 prefix, 4 steps, seed 4."""
    return make_workload("C5-expert2-bf16-B24-P256", EXPERT2, seed=4, batch=24, n_steps=4, prefix_len=256,
                         max_prefix_len=256, **kw)


def config_c5_expert1(**kw) -> Workload:
    """First co-located expert of the two-expert configuration (pi0-scale, batch 16, seed 4)."""
    return make_workload("C5-expert1-bf16-B16-ragged", PI0, seed=4, batch=16, n_steps=10,
                         prefix_range=(600, 900), max_prefix_len=1024, **kw)


def poisson_arrivals_us(seed: int, rate_per_s: float, duration_s: float, stream: int = 0) -> np.ndarray:
    """Arrival timestamps in integer microseconds: exponential gaps at ``rate_per_s`` for ``duration_s``."""
    g = np.random.default_rng([int(seed), 3, int(stream)])
    n = max(16, int(rate_per_s * duration_s * 1.5) + 16)
    t = np.cumsum(g.exponential(1.0 / rate_per_s, size=n))
    t = t[t < duration_s]
    return np.floor(t * 1e6).astype(np.int64)


def scaled(cfg: ADiTConfig, **kw) -> ADiTConfig:
    """A variant of a shape family (tests use small variants of the large ones)."""
    return replace(cfg, **kw)
