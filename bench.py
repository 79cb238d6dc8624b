#!/usr/bin/env python
"""Benchmark of the batched ADiT denoising loop: action chunks/s, per-chunk latency, roofline.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2|c3|c4|c5e2] [--impl ours|reference]

A "step" is one adit_denoise call: the whole K_euler-step loop for one batch of synthetic requests
(prologue, K_euler x (embed, all layers, read-out + Euler update)).  Default workload: the
pi0-scale expert at batch 1 with an 816-token prefix and 10 Euler steps.  Prints ONE JSON line.

With N > 1 (launched under torch.distributed.run) every rank runs an independent replica of the
expert on its own GPU and its own requests; there is no collective on the data path.

`--impl reference` times the fp64 CPU oracle on the host cores instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2609_12075_b200 import workloads as W  # noqa: E402

METRIC = "adit_action_chunks_per_s"
UNIT = "chunks/s"
L2_BYTES = 126e6
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# dram__bytes_read.sum + dram__bytes_write.sum per launch, averaged over the kernel's launches of one layer, from the
# ncu capture summarised in profiles/ (pi0-scale expert, batch 1)
NCU_TRAFFIC_PER_LAUNCH = {("c2", "gemm_tc_kernel"): 9.08e6, ("c2", "attn_tc_kernel"): 1.21e6}
WORKLOADS = {"c2": W.config_c2, "c3": W.config_c3, "c4": W.config_c4, "c5e2": W.config_c5_expert2}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return p, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


# ---- algorithmic work (what the method must move and compute) -------------------------------------

def layer_weight_params(cfg):
    D, F, Q, KV = cfg.d_model, cfg.d_ff, cfg.q_dim, cfg.kv_dim
    return {"gemm_qkv": D * (Q + 2 * KV), "gemm_o": Q * D, "gemm_gateup": 2 * D * F, "gemm_down": F * D}


def algorithmic_work(cfg, prefix_len, n_euler):
    """bytes and flops of ONE Euler step, and per kernel class per launch (bf16 weights and prefix K/V)."""
    B = len(prefix_len)
    N, M, Ma = cfg.n_tokens, len(prefix_len) * cfg.n_tokens, len(prefix_len) * cfg.horizon
    D = cfg.d_model
    esz = 2 if cfg.dtype == "bf16" else 4
    lw = layer_weight_params(cfg)
    embed_params = 2 * D * D + cfg.action_dim * D + D * cfg.action_dim
    w_bytes = (sum(lw.values()) * cfg.n_layers + embed_params) * esz
    kv_bytes_layer = int(sum(prefix_len)) * cfg.n_kv_heads * cfg.head_dim * 2 * esz
    keys = sum(int(p) + N for p in prefix_len)
    att_flops_layer = 4 * N * cfg.n_q_heads * cfg.head_dim * keys
    gemm_flops_layer = 2 * M * sum(lw.values())
    step_bytes = w_bytes + kv_bytes_layer * cfg.n_layers
    step_flops = (gemm_flops_layer + att_flops_layer) * cfg.n_layers + 2 * Ma * embed_params
    per_class = {k: {"bytes": v * esz, "flops": 2 * M * v} for k, v in lw.items()}
    per_class["attention"] = {"bytes": kv_bytes_layer + M * (cfg.q_dim + 2 * cfg.kv_dim) * esz, "flops": att_flops_layer}
    return {"step_bytes": step_bytes, "step_flops": step_flops, "per_class": per_class, "B": B}


# ---- clocks ---------------------------------------------------------------------------------------

class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons every 200 ms while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.idx, self.lines, self.proc = gpu_index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "200", "-i", str(self.idx)], stdout=subprocess.PIPE, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2])); pw.append(float(f[3]))
            except ValueError:
                continue
            for nm, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(pw) if pw else None, "samples": len(sm), "reasons": sorted(reasons)}


def bench_config(base, sm_budget, world, step_bytes, n_sets):
    """The `config` object of the JSON line: the same keys for the GPU arm and the reference arm."""
    return {"workload": base.name, "batch": base.batch, "euler_steps": base.n_steps,
            "prefix_len_mean": float(np.mean(base.prefix_len)), "sm_budget": sm_budget, "parallelism": f"replicas x{world}",
            "l2": f"inputs larger than L2: {step_bytes / 1e6:.0f} MB streamed per Euler step vs 126 MB L2; "
                  f"{n_sets} rotating input sets"}


# ---- CPU oracle legs ------------------------------------------------------------------------------

def oracle_sample_seconds(wl, weights_f64, n_euler_sample, requests):
    """Run the oracle as it stands on a bounded sample: `n_euler_sample` Euler steps of `requests`."""
    from oracle import adit_oracle as O
    t0 = time.perf_counter()
    for b in requests:
        st = np.asarray(wl.state[b], dtype=np.float64)
        O.euler_integrate(lambda x, t: O.velocity(wl.cfg, weights_f64, x, st, t, wl.prefix_kv[b], int(wl.prefix_len[b])),
                          np.asarray(wl.noise[b], dtype=np.float64), n_euler_sample)
    return time.perf_counter() - t0


def run_reference(args):
    """The CPU oracle, timed on the host cores; each step is one Euler step of one request of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import adit_oracle as O
    wl = WORKLOADS[args.workload]()
    weights = O.as_f64_weights(W.make_weights(wl.cfg, wl.seed))
    cores = len(os.sched_getaffinity(0))
    # Size the per-step sample so that the whole run stays within a few minutes: one Euler step of one
    # request, cut down to the first n_l layers (time scaled back by L / n_l) when K + W steps would not fit.
    t1 = oracle_sample_seconds(wl, weights, 1, [0])
    L = wl.cfg.n_layers
    n_l = L
    budget_s = 180.0
    if (args.steps + args.warmup) * t1 > budget_s:
        n_l = max(1, int(L * budget_s / ((args.steps + args.warmup) * t1)))
    wl_s = wl if n_l == L else W.Workload(**{**wl.__dict__, "cfg": W.scaled(wl.cfg, n_layers=n_l)})
    for _ in range(args.warmup):
        oracle_sample_seconds(wl_s, weights, 1, [0])
    t = [oracle_sample_seconds(wl_s, weights, 1, [0]) for _ in range(args.steps)]
    per_chunk = float(np.mean(t)) * wl.n_steps * (L / n_l)   # one request = one chunk = n_steps Euler steps
    value = 1.0 / per_chunk
    sample = (f"per step: 1 of {wl.n_steps} Euler steps of request 0 of {wl.name}, first {n_l} of {L} layers "
              f"(time scaled x{wl.n_steps * L / n_l:g})")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": per_chunk * 1e3 * wl.batch,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": bench_config(wl, args.sm_budget, max(1, args.gpus),
                               algorithmic_work(wl.cfg, wl.prefix_len, wl.n_steps)["step_bytes"], 4),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# ---- the GPU arm ----------------------------------------------------------------------------------

def make_sets(adit, base, n_sets, rank, local, dev, torch):
    """n_sets input sets (own prefix caches, states, noise) of the workload's shape; each rank draws its own."""
    sets = []
    for s in range(n_sets):
        wl = W.make_workload(base.name, base.cfg, seed=base.seed + 1000 * (1 + s + n_sets * rank), batch=base.batch,
                             n_steps=base.n_steps, prefix_len=base.prefix_len, max_prefix_len=base.max_prefix_len)
        sets.append({"kv": adit.upload_prefix_kv(wl, local), "len": wl.prefix_len,
                     "state": torch.from_numpy(wl.state).to(dev), "noise": torch.from_numpy(wl.noise).to(dev),
                     "state_h": torch.from_numpy(wl.state).pin_memory(), "noise_h": torch.from_numpy(wl.noise).pin_memory(),
                     "out_h": torch.empty(wl.noise.shape, dtype=torch.float32).pin_memory(),
                     "out": torch.empty(wl.noise.shape, dtype=torch.float32, device=dev)})
    return sets


def step_roofline(cfg, prefix_len, n_euler, ms_per_call, peaks):
    """Whole call: the slower of bytes at the HBM peak and flops at the sustained bf16 peak, against the measured time."""
    work = algorithmic_work(cfg, prefix_len, n_euler)
    t_hbm = work["step_bytes"] / (peaks["hbm_gbs"] * 1e9)
    t_tc = work["step_flops"] / (peaks["bf16_tflops_sustained"] * 1e12)
    floor_ms = max(t_hbm, t_tc) * n_euler * 1e3
    return work, {"bound": "hbm" if t_hbm >= t_tc else "tensor", "floor_ms_per_call": floor_ms, "frac": floor_ms / ms_per_call,
                  "bytes_per_euler_step": work["step_bytes"], "flops_per_euler_step": work["step_flops"],
                  "achieved_gbs": work["step_bytes"] * n_euler / (ms_per_call * 1e-3) / 1e9,
                  "achieved_tflops": work["step_flops"] * n_euler / (ms_per_call * 1e-3) / 1e12}


def layer_timeline(trace, names):
    """Per kernel class, medians in microseconds over the traced launches of: `interval` = this kernel's dependency
    release to the next kernel's (what the kernel adds to the call), `main` = release to the last accumulator complete,
    `epilogue` = from there to the last block's end, `handover` = the rest of the interval.  Rows of `trace`: class,
    blocks, first/last block start, first/last block end, first/last release, first/last accumulator complete (ns;
    0 where a kernel has no such stamp)."""
    out = {}
    for c in sorted(set(int(x) for x in trace[:-1, 0])):
        idx = np.where(trace[:-1, 0] == c)[0]
        m, nxt = trace[idx], trace[idx + 1]
        ok = (m[:, 7] > 0) & (nxt[:, 7] > 0)
        if not ok.any():
            continue
        m, nxt = m[ok], nxt[ok]
        row = {"launches": int(len(m)), "blocks": int(np.median(m[:, 1])), "interval": float(np.median(nxt[:, 7] - m[:, 7])) / 1e3}
        has_main = m[:, 9] > 0
        if has_main.all():
            row["main"] = float(np.median(m[:, 9] - m[:, 7])) / 1e3
            row["epilogue"] = float(np.median(m[:, 5] - m[:, 9])) / 1e3
            row["handover"] = row["interval"] - row["main"] - row["epilogue"]
        else:
            row["release_to_end"] = float(np.median(m[:, 5] - m[:, 7])) / 1e3
        out[names[c]] = row
    return out


def sample_latency(torch, eng, sets, n_euler, budget, stream, n_calls, wall_s):
    """Per-call device latency (CUDA events on the call's stream) of up to n_calls back-to-back calls, stopped early
    when the wall budget is spent."""
    lat, t0, i = [], time.perf_counter(), 0
    while i < n_calls and time.perf_counter() - t0 < wall_s:
        chunk = min(100, n_calls - i)
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(chunk + 1)]
        ev[0].record(stream)
        for j in range(chunk):
            s = sets[(i + j) % len(sets)]
            eng.denoise(s["kv"], s["len"], s["state"], s["noise"], n_euler, sm_budget=budget, stream=stream, out=s["out"])
            ev[j + 1].record(stream)
        stream.synchronize()
        lat += [ev[j].elapsed_time(ev[j + 1]) for j in range(chunk)]
        i += chunk
    return np.array(lat)


def traffic_from_profile(kernel, workload):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch as recorded in the kernel's ncu summary under profiles/
    (a line `dram_bytes_per_launch: <number>`), or None."""
    import re
    path = os.path.join(ROOT, "profiles", f"{kernel}_{workload}.md")
    if not os.path.exists(path):
        return None
    m = re.search(r"dram_bytes_per_launch:\s*([0-9.eE+]+)", open(path).read())
    return float(m.group(1)) if m else None


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2609_12075_b200 import build
    build.build()
    from paper_2609_12075_b200 import adit

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    torch.cuda.set_device(local)
    dev = torch.device(f"cuda:{local}")

    n_sets = 4
    base = WORKLOADS[args.workload]()
    cfg = base.cfg
    weights = W.make_weights(cfg, base.seed)
    flags = (adit.FLAG_NO_GRAPH if args.no_graph else 0) | (adit.FLAG_PERSISTENT_LOOP if args.persistent else 0) | \
        (adit.FLAG_ONE_SM_GEMM if args.one_sm_gemm else 0)
    eng = adit.ADiT(cfg, max_batch=base.batch, max_prefix_len=base.max_prefix_len, device=local, flags=flags)
    eng.load_weights(weights)
    sets = make_sets(adit, base, n_sets, rank, local, dev, torch)
    stream = torch.cuda.Stream(device=dev)
    K_e, B = base.n_steps, base.batch

    def call(i, budget=args.sm_budget):
        s = sets[i % n_sets]
        eng.denoise(s["kv"], s["len"], s["state"], s["noise"], K_e, sm_budget=budget, stream=stream, out=s["out"])

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    with torch.cuda.stream(stream):
        for i in range(args.warmup):
            call(i)
        barrier()
        # ---- timed region: exactly `steps` calls, device time on the launching stream -------------
        sampler = ClockSampler(local)
        if rank == 0:
            sampler.start()
        launches0 = eng.kernel_launches()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record(stream)
        for i in range(args.steps):
            call(i)
        ev1.record(stream)
        barrier()
        total_ms = ev0.elapsed_time(ev1)
        launches = eng.kernel_launches() - launches0
        clocks = sampler.stop() if rank == 0 else None
        if world > 1:
            t = torch.tensor([total_ms], device=dev, dtype=torch.float64)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            total_ms = float(t.item())
        assert eng.poll_status() == 0

        # ---- per-call latency distribution (its own calls: p99 needs many samples whatever --steps is) ----
        lat = sample_latency(torch, eng, sets, K_e, args.sm_budget, stream, args.latency_calls, args.latency_seconds)
        if len(lat) == 0:       # (--latency-calls 0, for profiler runs: one call's latency from the timed region)
            lat = np.array([total_ms / args.steps])

        # ---- end to end through the host-buffer entry point (pinned host in, host out) ------------
        for i in range(3):
            s = sets[i % n_sets]
            eng.denoise_host(s["kv"], s["len"], s["state_h"], s["noise_h"], K_e, args.sm_budget, stream, s["out_h"])
        barrier()
        n_e2e = max(3, min(args.steps, 50))
        t0 = time.perf_counter()
        for i in range(n_e2e):
            s = sets[i % n_sets]
            eng.denoise_host(s["kv"], s["len"], s["state_h"], s["noise_h"], K_e, args.sm_budget, stream, s["out_h"])
        e2e_s = time.perf_counter() - t0
        if world > 1:
            t = torch.tensor([e2e_s], device=dev, dtype=torch.float64)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            e2e_s = float(t.item())

        # ---- per-kernel-class device times (separate instrumented calls, after the timed region) --
        eng.profile_enable(True)
        n_prof = 3
        for i in range(n_prof):
            call(i)
        prof = eng.profile_read()
        eng.profile_enable(False)
        # ---- in-situ kernel durations: %globaltimer stamps written by every block inside the replayed graph --
        trace = None
        if not args.no_trace and not args.persistent:
            eng.trace_enable(True)
            call(0)
            call(1)
            torch.cuda.synchronize()
            trace = eng.trace_read()
            eng.trace_enable(False)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks, peaks_kind = load_peaks()
    ms_per_step = total_ms / args.steps
    value = world * B * args.steps / (total_ms * 1e-3)
    work, step_roof = step_roofline(cfg, base.prefix_len, K_e, ms_per_step, peaks)
    # dominant kernel: the four per-layer projections (and the two embedding projections) are launches of the
    # same kernel, gemm_tc_kernel; attention (+ merge) is the other candidate; the persistent path is one kernel
    tot = sum(v[0] for v in prof.values()) or 1.0
    shares = {k: {"ms_per_call": v[0] / n_prof, "launches_per_call": v[1] // n_prof, "share": v[0] / tot}
              for k, v in prof.items() if v[1]}
    gemm_classes = [k for k in ("gemm_qkv", "gemm_o", "gemm_gateup", "gemm_down") if k in shares]
    groups = {"gemm_tc_kernel": gemm_classes, "attn_tc_kernel": [k for k in ("attention",) if k in shares],
              "adit_loop_kernel": [k for k in ("loop",) if k in shares]}
    gtime = {g: sum(prof[k][0] for k in ks) for g, ks in groups.items() if ks}
    dom = max(gtime, key=gtime.get) if gtime else None
    roofline = None
    if dom:
        ks = groups[dom]
        n_launch = sum(prof[k][1] for k in ks)
        if dom == "adit_loop_kernel":       # one launch carries the whole call
            bytes_l, flops_l = work["step_bytes"] * K_e, work["step_flops"] * K_e
        else:
            bytes_l = sum(work["per_class"][k]["bytes"] * prof[k][1] for k in ks) / n_launch
            flops_l = sum(work["per_class"][k]["flops"] * prof[k][1] for k in ks) / n_launch
        hbm_bound = bytes_l / (peaks["hbm_gbs"] * 1e9) >= flops_l / (peaks["bf16_tflops"] * 1e12)
        peak, unit = (peaks["hbm_gbs"], "GB/s") if hbm_bound else (peaks["bf16_tflops"], "TFLOP/s")
        per_s = (lambda sec: bytes_l / sec / 1e9) if hbm_bound else (lambda sec: flops_l / sec / 1e12)
        # serialised figure: CUDA events around every launch (adds the launch gap, removes the overlap of the replay)
        ser_s = gtime[dom] / n_launch * 1e-3
        serialised = {"avg_launch_us": ser_s * 1e6, "achieved": per_s(ser_s), "frac": per_s(ser_s) / peak,
                      "timing": "CUDA events around every launch on the call's stream (serialised launches, 3 calls)"}
        # in-situ figure: the kernel as it runs inside the timed replay, from device timestamps of every block
        dur_s, timing = None, None
        if dom == "adit_loop_kernel":
            dur_s, timing = ms_per_step * 1e-3, "the timed region itself (the call is this one kernel plus a set-up kernel)"
        elif trace is not None and len(trace):
            names = [adit.lib.adit_profile_class_name(i).decode() for i in range(adit.N_KERNEL_CLASSES)]
            sel = [r for r in trace if names[int(r[0])] in ks and r[6] > 0]
            if sel:
                dur_s = float(np.mean([(r[5] - r[6]) for r in sel])) * 1e-9
                timing = ("device %globaltimer stamps of every block inside the replayed graph (dependency released -> "
                          "last block done; instrumented kernels)")
        if dur_s is None:
            dur_s, timing = ser_s, serialised["timing"]
        roofline = {"kernel": dom, "bound": "hbm" if hbm_bound else "tensor", "achieved": per_s(dur_s), "peak": peak,
                    "unit": unit, "frac": per_s(dur_s) / peak, "traffic": traffic_from_profile(dom, args.workload),
                    "avg_launch_us": dur_s * 1e6, "launches": n_launch // n_prof,
                    "algorithmic_bytes_per_launch": bytes_l, "algorithmic_flops_per_launch": flops_l, "timing": timing,
                    "launch_time_share_of_call": (n_launch // n_prof) * dur_s * 1e3 / ms_per_step,
                    "serialised_events": serialised,
                    "peak_source": f"{peaks_kind} (MEASURED_PEAKS.json)" if peaks_kind == "measured" else "fallback"}

    # ---- where a call's time goes: per kernel class, from the same in-situ stamps (medians over the traced launches) ----
    timeline = None
    if trace is not None and len(trace) > 1:
        timeline = layer_timeline(np.asarray(trace, dtype=np.int64),
                                  [adit.lib.adit_profile_class_name(i).decode() for i in range(adit.N_KERNEL_CLASSES)])

    # ---- the other batch sizes of the metric, briefly (same expert, its own handle sized for 32 requests) ----
    by_workload = {}
    if world == 1 and args.workload == "c2" and not args.no_extra:
        big = adit.ADiT(cfg, max_batch=32, max_prefix_len=1024, device=local)
        big.load_weights(weights)
        for name, n_calls in (("c3", 150), ("c4", 80)):
            wl = WORKLOADS[name]()
            bsets = make_sets(adit, wl, 1, rank, local, dev, torch)
            with torch.cuda.stream(stream):
                for i in range(3):
                    big.denoise(bsets[0]["kv"], bsets[0]["len"], bsets[0]["state"], bsets[0]["noise"], wl.n_steps, stream=stream,
                                out=bsets[0]["out"])
                l2 = sample_latency(torch, big, bsets, wl.n_steps, 0, stream, n_calls, 6.0)
            _, roof = step_roofline(wl.cfg, wl.prefix_len, wl.n_steps, float(l2.mean()), peaks)
            by_workload[name] = {"batch": wl.batch, "calls": int(len(l2)), "ms_p50": float(np.percentile(l2, 50)),
                                 "ms_p99": float(np.percentile(l2, 99)), "ms_mean": float(l2.mean()),
                                 "chunks_per_s": wl.batch / (float(l2.mean()) * 1e-3), "roofline_step": roof}
            del bsets
        # hidden-state hand-over (the expert projects the prefix K/V itself, once per call): the projection alone, for the
        # batch-1 and batch-32 prefixes, from hidden states of width 2048
        big.load_prefix_projection(W.make_prefix_projection(cfg, base.seed, 2048))
        for name in ("c2", "c4"):
            wl = WORKLOADS[name](with_kv=False) if name != "c2" else base
            hid = [torch.from_numpy(W.make_prefix_hidden(wl.seed, b, int(p), 2048)).to(torch.bfloat16).to(dev) for b, p in enumerate(wl.prefix_len)]
            caches = [torch.zeros((cfg.n_layers, 2, cfg.n_kv_heads, 1024, cfg.head_dim), dtype=torch.bfloat16, device=dev) for _ in hid]
            with torch.cuda.stream(stream):
                for i in range(3):
                    big.project_prefix(hid, wl.prefix_len, caches, stream=stream)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                for i in range(20):
                    big.project_prefix(hid, wl.prefix_len, caches, stream=stream)
                e1.record(stream)
                stream.synchronize()
            ms = e0.elapsed_time(e1) / 20
            flops = 2.0 * float(np.sum(wl.prefix_len)) * 2048 * (2 * cfg.n_layers * cfg.n_kv_heads * cfg.head_dim)
            by_workload[f"{name}_prefix_projection"] = {"batch": int(len(hid)), "hidden_dim": 2048, "ms": ms, "tflops": flops / (ms * 1e-3) / 1e12,
                                                        "launches": int(len(hid))}
            del hid, caches
        assert big.poll_status() == 0
        big.close()
        # the same call as one persistent kernel (opt-in path), for the record
        pl = adit.ADiT(cfg, max_batch=base.batch, max_prefix_len=base.max_prefix_len, device=local, flags=adit.FLAG_PERSISTENT_LOOP)
        pl.load_weights(weights)
        if pl.persistent_blocks(B) > 0:
            with torch.cuda.stream(stream):
                l0 = pl.kernel_launches()
                l3 = sample_latency(torch, pl, sets, K_e, 0, stream, 40, 3.0)
            by_workload["c2_persistent_loop"] = {"batch": B, "calls": int(len(l3)), "ms_p50": float(np.percentile(l3, 50)),
                                                 "ms_p99": float(np.percentile(l3, 99)), "blocks": pl.persistent_blocks(B),
                                                 "launches_per_call": (pl.kernel_launches() - l0) / max(1, len(l3))}
        pl.close()

    # CPU baseline: the oracle as it stands, bounded sample, rank 0 at N = 1 only
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        from oracle import adit_oracle as O
        wl0 = WORKLOADS[args.workload]()
        wf = O.as_f64_weights(weights)
        reps, secs = 0, 0.0
        while secs < 10.0 and reps < 8:          # whole chunks of request 0 until about 10 s of CPU work
            secs += oracle_sample_seconds(wl0, wf, wl0.n_steps, [0])
            reps += 1
        cpu = {"value": reps / secs, "unit": UNIT, "cores": len(os.sched_getaffinity(0)), "kind": "oracle",
               "sample": f"{reps} full chunk(s) ({wl0.n_steps} Euler steps) of request 0 of {wl0.name}",
               "seconds": secs}

    s0 = sets[0]
    h2d = s0["state_h"].numel() * 4 + s0["noise_h"].numel() * 4
    d2h = s0["out_h"].numel() * 4
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if cfg.dtype == "bf16" else "f32", "data": "synthetic",
        "config": bench_config(base, args.sm_budget, world, work["step_bytes"], n_sets),
        "latency_ms": {"p50": float(np.percentile(lat, 50)), "p99": float(np.percentile(lat, 99)),
                       "mean": float(lat.mean()), "min": float(lat.min()), "calls": int(len(lat))},
        "roofline": roofline, "roofline_step": step_roof, "kernel_shares": shares, "timeline_us": timeline, "by_workload": by_workload,
        "cpu_baseline": cpu,
        "e2e": {"value": world * B * n_e2e / e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "calls": n_e2e},
        "gpu_launches": int(launches), "clocks": clocks, "peaks": {"kind": peaks_kind, "hbm_gbs": peaks["hbm_gbs"],
                                                                    "bf16_tflops": peaks["bf16_tflops"],
                                                                    "bf16_tflops_sustained": peaks["bf16_tflops_sustained"]},
    }
    print(json.dumps(line))
    eng.close()
    if world > 1:
        dist.destroy_process_group()


# ---- SM-budget sweep under a concurrent GEMM load (pi0-scale expert, batch 32) -------------------------

def run_budget_sweep(args):
    """p50/p99 chunk latency per sm_budget, with and without a bf16 GEMM 8192x2048x2048 looping on the
    remaining SMs of a second stream (the stand-in for the VLM stage that shares the GPU)."""
    import torch
    from paper_2609_12075_b200 import build
    build.build()
    from paper_2609_12075_b200 import adit
    base = WORKLOADS[args.workload]()
    cfg = base.cfg
    eng = adit.ADiT(cfg, max_batch=base.batch, max_prefix_len=base.max_prefix_len)
    eng.load_weights(W.make_weights(cfg, base.seed))
    kv = adit.upload_prefix_kv(base)
    st_in, nz = torch.from_numpy(base.state).cuda(), torch.from_numpy(base.noise).cuda()
    out = torch.empty_like(nz)
    s_adit, s_load = torch.cuda.Stream(), torch.cuda.Stream()
    bg = adit.BackgroundGemm(8192, 2048, 2048)
    n_sm = torch.cuda.get_device_properties(0).multi_processor_count
    # duration of one background GEMM on the whole chip, to size the top-ups
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    bg.launch(3, 0, s_load); e0.record(s_load); bg.launch(10, 0, s_load); e1.record(s_load)
    torch.cuda.synchronize()
    bg_ms_full = e0.elapsed_time(e1) / 10
    results = {}
    peaks, _ = load_peaks()
    work = algorithmic_work(cfg, base.prefix_len, base.n_steps)
    roof = {}
    for budget in [int(b) for b in args.budgets.split(",")]:
        # memory roofline of a run confined to `budget` SMs: what a plain streaming read reaches from that many SMs
        read_gbs = adit.stream_read_gbs(min(budget, n_sm))
        tc = peaks["bf16_tflops_sustained"] * 1e12 * min(budget, n_sm) / n_sm
        floor_ms = max(work["step_bytes"] / (read_gbs * 1e9), work["step_flops"] / tc) * base.n_steps * 1e3
        roof[str(budget)] = {"stream_read_gbs": read_gbs, "floor_ms_per_call": floor_ms,
                             "bound": "hbm" if work["step_bytes"] / (read_gbs * 1e9) >= work["step_flops"] / tc else "tensor"}
    for budget in [int(b) for b in args.budgets.split(",")]:
        # load: "" = none; "+load" = the stand-in's grid capped to the SMs outside the budget (persistent-grid form, the
        # call's own grids capped to the budget); "+green" = the stand-in's full grid on a stream that the driver
        # confines to the SMs outside the budget (green context, section 4.1.2), the call itself unrestricted
        modes = ["", "+load"] + (["+green"] if args.green and budget < n_sm else [])
        for mode in modes:
            lat = []
            load_sms = n_sm - budget if budget < n_sm else 0        # budget = all SMs: the load is not capped
            est_ms = None
            green = None
            if mode == "+green":
                try:
                    green = adit.GreenStream(load_sms)
                except adit.AditError as e:
                    results[f"{budget}+green"] = {"unavailable": str(e)}
                    continue
            ls = green.stream if green else s_load
            for i in range(args.warmup + args.steps):
                if mode:
                    # keep the load stream busy well past the end of this call
                    per_iter = bg_ms_full * (n_sm / max(load_sms, 1) if load_sms else 2.0)
                    need_ms = (est_ms or 200.0) * 2.0
                    bg.launch(max(4, int(need_ms / per_iter)), 0 if green else load_sms, ls)
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(s_adit)
                eng.denoise(kv, base.prefix_len, st_in, nz, base.n_steps, sm_budget=0 if green else budget, stream=s_adit, out=out)
                b.record(s_adit)
                b.synchronize()
                est_ms = a.elapsed_time(b)
                if i >= args.warmup:
                    lat.append(est_ms)
            torch.cuda.synchronize()
            if green:
                load_granted = green.sm_count
                green.close()
            lat = np.array(lat)
            results[f"{budget}{mode}"] = {
                "p50_ms": float(np.percentile(lat, 50)), "p99_ms": float(np.percentile(lat, 99)),
                "chunks_per_s": base.batch / (float(lat.mean()) * 1e-3),
                "roofline_frac_at_budget": roof[str(budget)]["floor_ms_per_call"] / float(np.percentile(lat, 50))}
            if mode == "+green":  # (the call itself is not confined: no roofline of a budget applies)
                results[f"{budget}{mode}"]["load_sms_granted"] = load_granted
                results[f"{budget}{mode}"]["roofline_frac_at_budget"] = None
    assert eng.poll_status() == 0
    budgets = [int(b) for b in args.budgets.split(",")]
    ratios = {}
    for b in budgets:
        ratios[f"isolation_p99_{b}"] = results[f"{b}+load"]["p99_ms"] / results[f"{b}"]["p99_ms"]
    for lo in budgets:  # every pair of budgets where one is half the other
        for hi in budgets:
            if hi == 2 * lo:
                ratios[f"halving_p99_{lo}_vs_{hi}_load"] = results[f"{lo}+load"]["p99_ms"] / results[f"{hi}+load"]["p99_ms"]
                ratios[f"halving_p99_{lo}_vs_{hi}_idle"] = results[f"{lo}"]["p99_ms"] / results[f"{hi}"]["p99_ms"]
    print(json.dumps({"metric": "adit_chunk_latency_vs_sm_budget", "unit": "ms", "config": {
        "workload": base.name, "batch": base.batch, "euler_steps": base.n_steps,
        "load": "bf16 GEMM 8192x2048x2048 looping on a second stream, grid capped to the SMs outside the budget ('+load'); "
                "with --green also its full grid on a green-context stream of those SMs while the call runs unrestricted ('+green')",
        "bg_gemm_ms_full_chip": bg_ms_full}, "steps": args.steps, "warmup": args.warmup, "n_sm": n_sm,
        "results": results, "ratios": ratios, "roofline_per_budget": roof}))
    bg.close()
    eng.close()


# ---- two co-located experts on two streams, Poisson arrivals, earliest-SLO-first ---------------------

def run_colocated(args):
    """Expert 1 (pi0-scale, batch <= 16) on `s` SMs and expert 2 (batch <= 24) on the rest, each on its own
    stream and host thread; requests arrive as a Poisson process and each round serves the waiting
    requests with the least remaining slack first (SLO 50 ms)."""
    import torch
    from paper_2609_12075_b200 import build, scheduler
    build.build()
    from paper_2609_12075_b200 import adit
    n_sm = torch.cuda.get_device_properties(0).multi_processor_count
    slo_us, duration_s = 50_000, args.trace_seconds
    experts = []
    for wl_fn in (W.config_c5_expert1, W.config_c5_expert2):
        wl = wl_fn()
        eng = adit.ADiT(wl.cfg, max_batch=wl.batch, max_prefix_len=wl.max_prefix_len)
        eng.load_weights(W.make_weights(wl.cfg, wl.seed))
        experts.append({"wl": wl, "eng": eng, "kv": adit.upload_prefix_kv(wl), "stream": torch.cuda.Stream(),
                        "state": torch.from_numpy(wl.state).cuda(), "noise": torch.from_numpy(wl.noise).cuda()})

    def serve(ex, ids, budget):
        """One round: the requests `ids` (indices into the expert's pool of synthetic requests)."""
        wl = ex["wl"]
        pool = [i % wl.batch for i in ids]
        idx = torch.tensor(pool, device="cuda")
        ex["eng"].denoise([ex["kv"][i] for i in pool], [int(wl.prefix_len[i]) for i in pool], ex["state"][idx].contiguous(),
                          ex["noise"][idx].contiguous(), wl.n_steps, sm_budget=budget, stream=ex["stream"])
        ex["stream"].synchronize()

    out = {}
    for s in [int(v) for v in args.splits.split(",")]:
        budgets = (s, n_sm - s)
        # closed-loop capacity of each expert on its share (also records every batch size's launch graph)
        rates = []
        for ex, budget in zip(experts, budgets):
            with torch.cuda.stream(ex["stream"]):
                for nb in range(1, ex["wl"].batch + 1):
                    serve(ex, list(range(nb)), budget)
                t0 = time.perf_counter()
                for _ in range(5):
                    serve(ex, list(range(ex["wl"].batch)), budget)
                rates.append(0.8 * 5 * ex["wl"].batch / (time.perf_counter() - t0))
        import threading
        stats = [None, None]

        def run_expert(k):
            ex, budget = experts[k], budgets[k]
            arrivals = W.poisson_arrivals_us(4, rates[k], duration_s, stream=k)
            done_us = np.full(len(arrivals), -1, dtype=np.int64)
            served, t_start = 0, time.perf_counter()
            with torch.cuda.stream(ex["stream"]):
                while served < len(arrivals):
                    now = int((time.perf_counter() - t_start) * 1e6)
                    waiting = [i for i in range(served, len(arrivals)) if arrivals[i] <= now]
                    if not waiting:
                        time.sleep(max(0.0, (arrivals[served] - now) * 1e-6))
                        continue
                    pick = scheduler.take_batch([arrivals[i] for i in waiting], slo_us, now, waiting, ex["wl"].batch)
                    ids = sorted(waiting[j] for j in pick)   # FIFO queue: the picked set is a prefix of the waiting list
                    serve(ex, ids, budget)
                    t_done = int((time.perf_counter() - t_start) * 1e6)
                    done_us[ids] = t_done
                    served = ids[-1] + 1
            lat = (done_us - arrivals) / 1e3
            stats[k] = {"requests": int(len(arrivals)), "rate_per_s": rates[k], "p50_ms": float(np.percentile(lat, 50)),
                        "p99_ms": float(np.percentile(lat, 99)), "slo_attainment": float((lat <= slo_us / 1e3).mean()),
                        "chunks_per_s": float(len(arrivals) / (done_us.max() * 1e-6))}

        th = [threading.Thread(target=run_expert, args=(k,)) for k in range(2)]
        [t.start() for t in th]
        [t.join() for t in th]
        out[f"split_{s}_{n_sm - s}"] = {"expert1": stats[0], "expert2": stats[1]}
    for ex in experts:
        assert ex["eng"].poll_status() == 0
        ex["eng"].close()
    print(json.dumps({"metric": "colocated_experts_slo", "config": {
        "experts": [e["wl"].name for e in experts], "slo_ms": slo_us / 1e3, "trace_seconds": duration_s,
        "arrivals": "Poisson, rate = 0.8 x closed-loop chunks/s of the expert on its SM share", "policy": "earliest-SLO-first"},
        "results": out}))


# ---- lockstep execution with a profiled SM restriction (paper section 4.1.2) ---------------------------

def run_lockstep(args):
    """VLM stand-in (capped GEMM loop) and the ADiT stage in locksteps on two streams: the offline table of the best
    SM restriction per (VLM batch, ADiT batch) pair, then a saturated trace with and without the restriction."""
    import torch
    from paper_2609_12075_b200 import build, lockstep as LS
    build.build()
    from paper_2609_12075_b200 import adit
    max_batch = args.max_batch
    cfg = W.PI0
    pool = 8
    wl = W.make_workload("lockstep", cfg, seed=7, batch=pool, n_steps=10, prefix_len=[816] * pool, max_prefix_len=816)
    eng = adit.ADiT(cfg, max_batch=max_batch, max_prefix_len=816)
    eng.load_weights(W.make_weights(cfg, wl.seed))
    inputs = {"pi0": {"kv": adit.upload_prefix_kv(wl), "len": wl.prefix_len, "state": torch.from_numpy(wl.state).cuda(),
                      "noise": torch.from_numpy(wl.noise).cuda(), "steps": wl.n_steps}}
    stages = LS.GpuStages(adit, {"pi0": eng}, inputs, vlm_iters_per_request=args.vlm_iters, restriction="green" if args.green else "grid")
    for b in LS.batch_sizes(max_batch):               # record every batch size's launch graph first
        stages.time_lockstep("pi0", b, b, 0, reps=1)
    t0 = time.perf_counter()
    # the paper's arrangement: only the VLM stream is restricted, the ADiT call runs unrestricted
    table = LS.SmTable.profile(stages.n_sm, max_batch, lambda vb, ab, cap: stages.time_lockstep("pi0", vb, ab, cap, reps=2, arrangement="vlm_only"),
                               arrangement="vlm_only")
    # both stages with an explicit allotment (the ADiT call's sm_budget = the SMs outside the VLM's)
    table_c = LS.SmTable.profile(stages.n_sm, max_batch, lambda vb, ab, cap: stages.time_lockstep("pi0", vb, ab, cap, reps=2))
    profile_s = time.perf_counter() - t0
    out = {}
    for name, tab in (("guarded", table), ("guarded_complement", table_c), ("unguarded", LS.SmTable(stages.n_sm))):
        ex = LS.LockstepExecutor(stages.vlm, stages.adit_stage, max_batch, tab, {"pi0": 156_000})
        reqs = [LS.Request("pi0", i, 0, payload=i % pool) for i in range(args.requests)]
        [ex.submit(r) for r in reqs]
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        rec = ex.run()
        total = time.perf_counter() - t0
        full = [r.seconds for r in rec if r.vlm_ids and r.adit_ids]
        out[name] = {"requests": len(reqs), "locksteps": len(rec), "total_s": total, "chunks_per_s": len(reqs) / total,
                     "mean_lockstep_ms": 1e3 * float(np.mean(full)) if full else None,
                     "p99_latency_ms": float(np.percentile([r.done_us for r in reqs], 99)) / 1e3}
    assert eng.poll_status() == 0
    print(json.dumps({"metric": "lockstep_time_with_profiled_sm_restriction", "unit": "ms", "config": {
        "expert": "pi0-scale, 816-token prefixes, 10 Euler steps", "max_batch": max_batch,
        "vlm_stand_in": f"bf16 GEMM 8192x2048x2048 x {args.vlm_iters} per request, " +
                        ("full grid on a green-context stream of the restriction's SMs" if args.green else "grid capped to the restriction"),
        "arrangements": "guarded = only the VLM stream restricted (the paper's); guarded_complement = the ADiT call's sm_budget is the rest",
        "candidates": "multiples of 8 SMs and no restriction", "n_sm": stages.n_sm, "profile_seconds": profile_s},
        "table": {f"{vb},{ab}": c for (vb, ab), c in sorted(table.entries.items())},
        "table_ms": {f"{vb},{ab}": {"best": 1e3 * t[table.entries[(vb, ab)]], "unrestricted": 1e3 * t[0]}
                     for (vb, ab), t in sorted(table.times.items())},
        "table_complement": {f"{vb},{ab}": c for (vb, ab), c in sorted(table_c.entries.items())},
        "table_complement_ms": {f"{vb},{ab}": {"best": 1e3 * t[table_c.entries[(vb, ab)]], "unrestricted": 1e3 * t[0]}
                                for (vb, ab), t in sorted(table_c.times.items())},
        "trace": out, "speedup_guarded_vs_unguarded": out["unguarded"]["total_s"] / out["guarded"]["total_s"]}))
    stages.close()
    eng.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", choices=sorted(WORKLOADS), default=None)
    ap.add_argument("--sm-budget", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--mode", choices=["throughput", "sweep", "colocate", "lockstep"], default="throughput",
                    help="sweep: latency per sm_budget with/without a concurrent GEMM load; colocate: two experts, two streams; "
                         "lockstep: VLM stand-in and ADiT in locksteps with the profiled SM restriction")
    ap.add_argument("--max-batch", type=int, default=4, help="lockstep mode: largest batch admitted per lockstep")
    ap.add_argument("--vlm-iters", type=int, default=60, help="lockstep mode: GEMM repetitions per request of the VLM stand-in")
    ap.add_argument("--requests", type=int, default=64, help="lockstep mode: requests in the saturated trace")
    ap.add_argument("--budgets", default="16,32,64,74,148")
    ap.add_argument("--no-trace", action="store_true", help="skip the in-situ timeline of one call")
    ap.add_argument("--no-extra", action="store_true", help="skip the brief runs of the other batch sizes (c3, c4)")
    ap.add_argument("--no-graph", action="store_true", help="enqueue kernels one by one (ADIT_FLAG_NO_GRAPH): for profilers")
    ap.add_argument("--green", action="store_true", help="sweep: also run the load on a green-context stream confined to the SMs outside the budget, the call unrestricted; lockstep: restrict the VLM stand-in with green-context streams instead of grid caps")
    ap.add_argument("--one-sm-gemm", action="store_true", help="projections on the one-SM kernel at every batch size (ADIT_FLAG_ONE_SM_GEMM): comparison")
    ap.add_argument("--persistent", action="store_true", help="small batches as one persistent kernel (ADIT_FLAG_PERSISTENT_LOOP)")
    ap.add_argument("--latency-calls", type=int, default=None, help="calls sampled for p50/p99 (default 1000 at batch 1)")
    ap.add_argument("--latency-seconds", type=float, default=12.0, help="wall budget of the latency sampling")
    ap.add_argument("--splits", default="48,74,100")
    ap.add_argument("--trace-seconds", type=float, default=2.0)
    args = ap.parse_args()
    if args.workload is None:
        args.workload = "c4" if args.mode == "sweep" else "c2"
    if args.mode == "sweep":
        args.steps = 50 if args.steps is None else args.steps
        args.warmup = 5 if args.warmup is None else args.warmup
        return run_budget_sweep(args)
    if args.mode == "colocate":
        return run_colocated(args)
    if args.mode == "lockstep":
        return run_lockstep(args)
    if args.impl == "reference":
        args.steps = 10 if args.steps is None else args.steps
        args.warmup = 1 if args.warmup is None else args.warmup
        run_reference(args)
    else:
        args.steps = 200 if args.steps is None else args.steps
        args.warmup = 10 if args.warmup is None else max(args.warmup, 3)
        if args.latency_calls is None:
            args.latency_calls = {"c2": 1000, "c3": 500, "c4": 200}.get(args.workload, 300)
        run_ours(args)


if __name__ == "__main__":
    main()
