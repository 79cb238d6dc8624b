"""ctypes binding of libadit.so: argument marshalling only, every step of the path runs in the
library's CUDA kernels.  torch is used for device memory and streams.

Importing this module loads the shared library and raises if it has not been built
(`python -m paper_2609_12075_b200.build`); there is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

import numpy as np

from . import workloads as W

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libadit.so")
if not os.path.exists(_LIB_PATH):
    raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2609_12075_b200.build`")
lib = C.CDLL(_LIB_PATH)

OK, E_INVALID, E_CAPACITY, E_NOT_LOADED, E_UNSUPPORTED, E_CUDA, E_TIMEOUT = 0, -1, -2, -3, -4, -5, -6
DTYPE_FP32, DTYPE_BF16 = 0, 1
FLAG_REFERENCE_KERNELS, FLAG_NO_GRAPH, FLAG_NO_PDL, FLAG_MMA_SYNC_ATTENTION, FLAG_PERSISTENT_LOOP = 1, 2, 4, 8, 16
FLAG_STATE_BLOCK_MASK, FLAG_SUFFIX_ROPE, FLAG_ONE_SM_GEMM = 32, 64, 128
MAX_BATCH, MAX_STEPS = 64, 64

EXPORTS = ["adit_create", "adit_load_weights", "adit_denoise", "adit_denoise_host", "adit_destroy",
           "adit_poll_status", "adit_last_cuda_error", "adit_kernel_launches", "adit_strerror",
           "adit_debug_copy", "adit_debug_gemm", "adit_debug_gemm_timeout", "adit_debug_plan", "adit_debug_plan_projection", "adit_debug_gemm_stamps", "adit_debug_attention", "adit_attention_static", "adit_profile_enable", "adit_profile_read", "adit_profile_class_name", "adit_trace_enable", "adit_trace_read",
           "adit_load_prefix_projection", "adit_project_prefix", "adit_green_stream_create", "adit_green_stream_handle", "adit_green_stream_sm_count", "adit_green_stream_destroy", "adit_bg_gemm_create", "adit_bg_gemm_create_kind", "adit_bg_gemm_launch", "adit_bg_gemm_destroy",
           "adit_debug_stream_read", "adit_attention_static_status", "adit_debug_stamps_selected",
           "adit_clear_status", "adit_uses_persistent_loop", "adit_debug_wait_limit", "adit_loop_trace_read"]


class Config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "d_ff",
                                         "horizon", "action_dim", "state_dim", "time_emb_dim", "max_batch",
                                         "max_prefix_len", "dtype")] + \
               [("rms_eps", C.c_float), ("t_min_period", C.c_float), ("t_max_period", C.c_float), ("flags", C.c_int32)]


class Tensor(C.Structure):
    _fields_ = [("name", C.c_char_p), ("data", C.c_void_p), ("dtype", C.c_int32), ("ndim", C.c_int32),
                ("shape", C.c_int64 * 4), ("on_device", C.c_int32)]


lib.adit_create.argtypes = [C.POINTER(Config), C.c_int, C.POINTER(C.c_void_p)]
lib.adit_load_weights.argtypes = [C.c_void_p, C.POINTER(Tensor), C.c_int]
_DENOISE_ARGS = [C.c_void_p, C.c_int, C.POINTER(C.c_void_p), C.POINTER(C.c_int32), C.c_void_p, C.c_void_p,
                 C.c_int, C.c_int, C.c_void_p, C.c_void_p]
lib.adit_denoise.argtypes = _DENOISE_ARGS
lib.adit_denoise_host.argtypes = _DENOISE_ARGS
lib.adit_load_prefix_projection.argtypes = [C.c_void_p, C.POINTER(Tensor), C.c_int]
lib.adit_project_prefix.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_void_p), C.POINTER(C.c_int32), C.POINTER(C.c_void_p), C.c_int, C.c_void_p]
lib.adit_destroy.argtypes = [C.c_void_p]
lib.adit_poll_status.argtypes = [C.c_void_p]
lib.adit_last_cuda_error.argtypes = [C.c_void_p]
lib.adit_kernel_launches.argtypes = [C.c_void_p]
lib.adit_kernel_launches.restype = C.c_int64
lib.adit_strerror.argtypes = [C.c_int]
lib.adit_strerror.restype = C.c_char_p
lib.adit_debug_copy.argtypes = [C.c_void_p, C.c_char_p, C.c_void_p, C.c_size_t]
lib.adit_debug_copy.restype = C.c_int64
N_KERNEL_CLASSES = 11
lib.adit_debug_gemm_stamps.argtypes = [C.c_void_p, C.c_int]
lib.adit_debug_plan.argtypes = [C.c_int] * 5 + [C.POINTER(C.c_int32)]
lib.adit_debug_plan.restype = C.c_int
lib.adit_debug_plan_projection.argtypes = [C.c_int] * 6 + [C.POINTER(C.c_int32)]
lib.adit_debug_plan_projection.restype = C.c_int
lib.adit_debug_gemm_timeout.argtypes = [C.c_int, C.POINTER(C.c_int), C.c_void_p]
lib.adit_debug_gemm.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int,
                                C.c_void_p]
lib.adit_profile_enable.argtypes = [C.c_void_p, C.c_int]
lib.adit_profile_read.argtypes = [C.c_void_p, C.POINTER(C.c_double), C.POINTER(C.c_int64)]
lib.adit_profile_class_name.argtypes = [C.c_int]
lib.adit_profile_class_name.restype = C.c_char_p
_ATTN_ARGS = [C.c_int] * 8 + [C.c_void_p, C.POINTER(C.c_void_p), C.POINTER(C.c_int32), C.c_int, C.c_void_p, C.c_void_p]
lib.adit_debug_attention.argtypes = _ATTN_ARGS
lib.adit_attention_static.argtypes = _ATTN_ARGS
STATIC_SCRATCH_BYTES = 8 << 20
lib.adit_trace_enable.argtypes = [C.c_void_p, C.c_int]
lib.adit_trace_read.argtypes = [C.c_void_p, C.POINTER(C.c_int64), C.c_int64]
lib.adit_trace_read.restype = C.c_int64
lib.adit_debug_stream_read.argtypes = [C.c_int, C.c_size_t, C.c_int, C.c_int, C.POINTER(C.c_double)]
lib.adit_attention_static_status.argtypes = [C.c_int]
lib.adit_debug_stamps_selected.argtypes = [C.c_int] * 4
lib.adit_clear_status.argtypes = [C.c_void_p]
lib.adit_uses_persistent_loop.argtypes = [C.c_void_p, C.c_int, C.c_int]
lib.adit_debug_wait_limit.argtypes = [C.c_void_p, C.c_int, C.c_int]
lib.adit_loop_trace_read.argtypes = [C.c_void_p, C.POINTER(C.c_int64), C.c_int64]
lib.adit_loop_trace_read.restype = C.c_int64
lib.adit_bg_gemm_create.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int, C.POINTER(C.c_void_p)]
lib.adit_green_stream_create.argtypes = [C.c_int, C.c_int, C.POINTER(C.c_void_p)]
lib.adit_green_stream_handle.argtypes = [C.c_void_p]
lib.adit_green_stream_handle.restype = C.c_void_p
lib.adit_green_stream_sm_count.argtypes = [C.c_void_p]
lib.adit_green_stream_destroy.argtypes = [C.c_void_p]
lib.adit_bg_gemm_create_kind.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.POINTER(C.c_void_p)]
lib.adit_bg_gemm_launch.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p]
lib.adit_bg_gemm_destroy.argtypes = [C.c_void_p]


class AditError(RuntimeError):
    def __init__(self, code: int, cuda: int = 0):
        self.code, self.cuda = code, cuda
        msg = lib.adit_strerror(code).decode()
        super().__init__(f"adit status {code} ({msg})" + (f", CUDA error {cuda}" if cuda else ""))


def make_config(cfg: W.ADiTConfig, max_batch: int, max_prefix_len: int, flags: int = 0) -> Config:
    flags |= (FLAG_STATE_BLOCK_MASK if getattr(cfg, "state_block_mask", False) else 0) | \
             (FLAG_SUFFIX_ROPE if getattr(cfg, "suffix_rope", False) else 0)
    return Config(n_layers=cfg.n_layers, d_model=cfg.d_model, n_q_heads=cfg.n_q_heads, n_kv_heads=cfg.n_kv_heads,
                  head_dim=cfg.head_dim, d_ff=cfg.d_ff, horizon=cfg.horizon, action_dim=cfg.action_dim,
                  state_dim=cfg.state_dim, time_emb_dim=cfg.time_emb_dim, max_batch=max_batch,
                  max_prefix_len=max_prefix_len, dtype=DTYPE_BF16 if cfg.dtype == "bf16" else DTYPE_FP32,
                  rms_eps=cfg.rms_eps, t_min_period=cfg.t_min_period, t_max_period=cfg.t_max_period, flags=flags)


class ADiT:
    """One action expert on one device: adit_create / adit_load_weights / adit_denoise / adit_destroy."""

    def __init__(self, cfg: W.ADiTConfig, max_batch: int, max_prefix_len: int, device: int = 0, flags: int = 0):
        self.cfg, self.device = cfg, device
        self.max_batch, self.max_prefix_len = max_batch, max_prefix_len
        self._h = C.c_void_p()
        c = make_config(cfg, max_batch, max_prefix_len, flags)
        rc = lib.adit_create(C.byref(c), device, C.byref(self._h))
        if rc != OK:
            self._h = C.c_void_p()
            raise AditError(rc)

    # -- lifetime -----------------------------------------------------------------------------
    def close(self):
        if getattr(self, "_h", None) is not None and self._h:
            lib.adit_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc: int):
        if rc != OK:
            raise AditError(rc, lib.adit_last_cuda_error(self._h) if rc == E_CUDA else 0)

    # -- weights ------------------------------------------------------------------------------
    def load_weights(self, weights: Dict[str, np.ndarray]):
        """weights: name -> float32 numpy array (row-major [in, out] matrices)."""
        keep, arr = [], (Tensor * len(weights))()
        for i, (name, w) in enumerate(weights.items()):
            w = np.ascontiguousarray(w, dtype=np.float32)
            keep.append(w)
            shape = (C.c_int64 * 4)(*(list(w.shape) + [1] * (4 - w.ndim)))
            arr[i] = Tensor(name=name.encode(), data=w.ctypes.data, dtype=DTYPE_FP32, ndim=w.ndim, shape=shape,
                            on_device=0)
        self._check(lib.adit_load_weights(self._h, arr, len(weights)))

    # -- hidden-state hand-over ---------------------------------------------------------------
    def load_prefix_projection(self, weights: Dict[str, np.ndarray]):
        """weights: layers.<l>.prefix_wk / prefix_wv -> float32 [Dh, KV] (all layers, one call)."""
        keep, arr = [], (Tensor * len(weights))()
        for i, (name, w) in enumerate(weights.items()):
            w = np.ascontiguousarray(w, dtype=np.float32)
            keep.append(w)
            shape = (C.c_int64 * 4)(*(list(w.shape) + [1] * (4 - w.ndim)))
            arr[i] = Tensor(name=name.encode(), data=w.ctypes.data, dtype=DTYPE_FP32, ndim=w.ndim, shape=shape,
                            on_device=0)
        self._check(lib.adit_load_prefix_projection(self._h, arr, len(weights)))

    def project_prefix(self, hidden: Sequence, prefix_len: Sequence[int], prefix_kv_out: Sequence, sm_budget: int = 0,
                       stream=None):
        """hidden[b]: bf16 cuda [prefix_len[b], Dh]; writes rows < prefix_len[b] of the caches prefix_kv_out[b] (async)."""
        import torch
        n = len(prefix_len)
        hp = (C.c_void_p * n)(*[int(t.data_ptr()) if t is not None else None for t in hidden])
        op = (C.c_void_p * n)(*[int(t.data_ptr()) for t in prefix_kv_out])
        lens = (C.c_int32 * n)(*[int(v) for v in prefix_len])
        st = stream if stream is not None else torch.cuda.current_stream(self.device)
        self._check(lib.adit_project_prefix(self._h, n, hp, lens, op, int(sm_budget), C.c_void_p(st.cuda_stream)))
        return prefix_kv_out

    # -- the call -----------------------------------------------------------------------------
    @staticmethod
    def _marshal_prefix(prefix_kv: Sequence, prefix_len: Sequence[int]):
        n = len(prefix_len)
        ptrs = (C.c_void_p * n)(*[int(t.data_ptr()) if hasattr(t, "data_ptr") else int(t) for t in prefix_kv])
        lens = (C.c_int32 * n)(*[int(v) for v in prefix_len])
        return ptrs, lens

    def denoise(self, prefix_kv: Sequence, prefix_len: Sequence[int], state, noise, n_steps: int,
                sm_budget: int = 0, stream=None, out=None):
        """state [B, S] fp32 cuda, noise [B, Ta, A] fp32 cuda -> actions [B, Ta, A] fp32 cuda (async)."""
        import torch
        B = len(prefix_len)
        assert state.is_cuda and noise.is_cuda and state.dtype == torch.float32 and noise.dtype == torch.float32
        assert state.is_contiguous() and noise.is_contiguous()
        if out is None:
            out = torch.empty_like(noise)
        ptrs, lens = self._marshal_prefix(prefix_kv, prefix_len)
        st = stream if stream is not None else torch.cuda.current_stream(self.device)
        self._check(lib.adit_denoise(self._h, B, ptrs, lens, state.data_ptr(), noise.data_ptr(), int(n_steps),
                                     int(sm_budget), C.c_void_p(st.cuda_stream), out.data_ptr()))
        return out

    def denoise_host(self, prefix_kv: Sequence, prefix_len: Sequence[int], state, noise, n_steps: int,
                     sm_budget: int = 0, stream=None, out=None):
        """Same with HOST (ideally pinned) torch tensors for state/noise/out; blocks until done."""
        import torch
        B = len(prefix_len)
        assert not state.is_cuda and not noise.is_cuda
        if out is None:
            out = torch.empty_like(noise, pin_memory=True)
        ptrs, lens = self._marshal_prefix(prefix_kv, prefix_len)
        st = stream if stream is not None else torch.cuda.current_stream(self.device)
        self._check(lib.adit_denoise_host(self._h, B, ptrs, lens, state.data_ptr(), noise.data_ptr(), int(n_steps),
                                          int(sm_budget), C.c_void_p(st.cuda_stream), out.data_ptr()))
        return out

    # -- introspection ------------------------------------------------------------------------
    def poll_status(self) -> int:
        return lib.adit_poll_status(self._h)

    def kernel_launches(self) -> int:
        return int(lib.adit_kernel_launches(self._h))

    def profile_enable(self, on: bool):
        self._check(lib.adit_profile_enable(self._h, 1 if on else 0))

    def profile_read(self) -> Dict[str, tuple]:
        """class name -> (total milliseconds, launches) since the last read."""
        ms = (C.c_double * N_KERNEL_CLASSES)()
        n = (C.c_int64 * N_KERNEL_CLASSES)()
        self._check(lib.adit_profile_read(self._h, ms, n))
        return {lib.adit_profile_class_name(i).decode(): (ms[i], int(n[i])) for i in range(N_KERNEL_CLASSES)}

    def trace_enable(self, on: bool):
        self._check(lib.adit_trace_enable(self._h, 1 if on else 0))

    def trace_read(self, max_records: int = 4096) -> np.ndarray:
        """[n_launches, 10] int64: class, grid, first/last block start, first/last block end, first/last wait
        release, first/last main loop finished (ns)."""
        buf = np.zeros((max_records, 10), dtype=np.int64)
        n = lib.adit_trace_read(self._h, buf.ctypes.data_as(C.POINTER(C.c_int64)), max_records)
        if n < 0:
            raise AditError(int(n))
        return buf[:n]

    def clear_status(self):
        self._check(lib.adit_clear_status(self._h))

    def persistent_blocks(self, batch: int, sm_budget: int = 0) -> int:
        """Thread blocks of the single persistent kernel for such a call, 0 if it takes the kernel-per-phase path."""
        return int(lib.adit_uses_persistent_loop(self._h, int(batch), int(sm_budget)))

    def debug_wait_limit(self, limit_ms: int, withhold_level: int = -1):
        self._check(lib.adit_debug_wait_limit(self._h, int(limit_ms), int(withhold_level)))

    def loop_trace_read(self, max_records: int = 8192) -> np.ndarray:
        """[n_levels, 11] int64 per level of the last traced persistent call: type, blocks, earliest start, then
        the latest over blocks of: start, accumulator complete, partials sent, partials received, epilogue stored,
        published, first activation tile landed, last product issued (ns)."""
        buf = np.zeros((max_records, 11), dtype=np.int64)
        n = lib.adit_loop_trace_read(self._h, buf.ctypes.data_as(C.POINTER(C.c_int64)), max_records)
        if n < 0:
            raise AditError(int(n))
        return buf[:n]

    def debug_copy(self, name: str, n_elems: int, dtype=np.float32) -> np.ndarray:
        buf = np.empty(n_elems, dtype=dtype)
        got = lib.adit_debug_copy(self._h, name.encode(), buf.ctypes.data, buf.nbytes)
        if got < 0:
            raise AditError(int(got))
        return buf[: got // buf.itemsize]


def debug_plan(n_tok: int, n_feat: int, k: int, dual: bool = False, sm_count: int = 148) -> dict:
    """The projection tiling the library would choose (host-only)."""
    out = (C.c_int32 * 12)()
    rc = lib.adit_debug_plan(n_tok, n_feat, k, int(dual), sm_count, out)
    if rc != 0:
        raise AditError(rc)
    names = ("tile_tok", "n_ttiles", "n_ftiles", "splits", "stages", "kb_total", "acc_bufs", "issuers", "tmem_cols",
             "smem_bytes", "ring_bytes", "est_ns")
    return dict(zip(names, out))


def debug_plan_projection(n_tok: int, n_feat: int, k: int, dual: bool = False, sm_count: int = 148,
                          allow_pair: bool = True) -> dict:
    """The plan a projection of the loop runs with, `pair` = 1 where it is the two-SM kernel (host-only)."""
    out = (C.c_int32 * 13)()
    rc = lib.adit_debug_plan_projection(n_tok, n_feat, k, int(dual), sm_count, int(allow_pair), out)
    if rc != 0:
        raise AditError(rc)
    names = ("tile_tok", "n_ttiles", "n_ftiles", "splits", "stages", "kb_total", "acc_bufs", "issuers", "tmem_cols",
             "smem_bytes", "ring_bytes", "est_ns", "pair")
    return dict(zip(names, out))


def stream_read_gbs(sm_count: int, n_bytes: int = 1 << 30, iters: int = 5, device: int = 0) -> float:
    """Read bandwidth (GB/s) of a plain streaming read from `sm_count` SMs."""
    out = C.c_double(0.0)
    rc = lib.adit_debug_stream_read(device, n_bytes, sm_count, iters, C.byref(out))
    if rc != OK:
        raise AditError(rc)
    return float(out.value)


def upload_prefix_kv(wl: W.Workload, device: int = 0) -> List:
    """Copy a workload's per-request prefix caches to the device in the compute dtype (one tensor each)."""
    import torch
    dt = torch.bfloat16 if wl.cfg.dtype == "bf16" else torch.float32
    return [torch.from_numpy(kv).to(dt).to(f"cuda:{device}") for kv in wl.prefix_kv]


class GreenStream:
    """A stream confined by the driver to a partition of at least `sm_count` SMs (green context)."""

    def __init__(self, sm_count: int, device: int = 0):
        import torch
        self._g = C.c_void_p()
        rc = lib.adit_green_stream_create(device, int(sm_count), C.byref(self._g))
        if rc != OK:
            self._g = C.c_void_p()
            raise AditError(rc)
        self.sm_count = int(lib.adit_green_stream_sm_count(self._g))
        self.stream = torch.cuda.ExternalStream(int(lib.adit_green_stream_handle(self._g)), device=device)

    def close(self):
        if self._g:
            lib.adit_green_stream_destroy(self._g)
            self._g = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class BackgroundGemm:
    """Looping bf16 GEMM on a capped number of SMs (the VLM-stage stand-in on the other stream)."""

    def __init__(self, m: int, n: int, k: int, device: int = 0, two_sm: bool = False):
        self._g = C.c_void_p()
        rc = lib.adit_bg_gemm_create_kind(device, m, n, k, 1 if two_sm else 0, C.byref(self._g))
        if rc != OK:
            self._g = C.c_void_p()
            raise AditError(rc)

    def launch(self, iters: int, sm_count: int, stream):
        rc = lib.adit_bg_gemm_launch(self._g, iters, sm_count, C.c_void_p(stream.cuda_stream))
        if rc != OK:
            raise AditError(rc)

    def close(self):
        if self._g:
            lib.adit_bg_gemm_destroy(self._g)
            self._g = C.c_void_p()
