"""Lockstep execution of the two stages of a VLA model on two streams, with a profiled SM restriction
(paper section 4.1.2) and per-model queues served earliest-SLO-first (section 4.1.3).

At lockstep k the VLM stage of batch k runs on one stream while the ADiT stage of batch k-1 runs on the other;
two host threads (one per stream) launch them and meet at a barrier; the next lockstep starts when both stages
have finished.  At the start of a lockstep the queue whose head request has the least time left to its deadline is
chosen, up to max_batch requests are taken from it - the largest power of two that is available, so that only
O(log max_batch) batch sizes occur - and the number of SMs the VLM stream may use is read from a table indexed by
(VLM batch size, ADiT batch size).  The table comes from an offline sweep that times a lockstep for every batch-size
pair under every restriction in multiples of 8 SMs, and under no restriction, and keeps the fastest.

In the paper the restriction is applied to the VLM stream (Green Contexts) and the ADiT kernels find the remaining
SMs free: the table's arrangement "vlm_only".  The arrangement "complement" gives both stages an explicit SM
allotment instead - the ADiT call gets sm_budget = the rest.  "No restriction" means both may use the whole chip.
The VLM stand-in is a GEMM loop; its restriction is a cap on its grid or, as in the paper, a green-context stream.

The executor is host code and independent of CUDA: a stage is any callable that runs a batch to completion on its
own stream.  `GpuStages` supplies the two callables used on a B200.
"""
from __future__ import annotations

import json
import threading
import time
from collections import deque
from dataclasses import dataclass, field
from typing import Callable, Deque, Dict, List, Optional, Sequence, Tuple

from . import scheduler


def admit_batch_size(pending: int, max_batch: int) -> int:
    """Requests admitted from a queue with `pending` waiting: the largest power of two that is at most
    min(pending, max_batch); 0 when nothing waits."""
    n = min(int(pending), int(max_batch))
    if n < 1:
        return 0
    return 1 << (n.bit_length() - 1)


def batch_sizes(max_batch: int) -> List[int]:
    """The batch sizes that can occur: powers of two up to max_batch."""
    out, b = [], 1
    while b <= max_batch:
        out.append(b)
        b *= 2
    return out


def sm_candidates(n_sm: int, step: int = 8) -> List[int]:
    """SM counts tried for the VLM stream: multiples of `step` below the chip's SM count, and 0 = no restriction."""
    return list(range(step, n_sm, step)) + [0]


class SmTable:
    """(VLM batch size, ADiT batch size) -> SMs the VLM stream is restricted to (0: no restriction)."""

    def __init__(self, n_sm: int, entries: Optional[Dict[Tuple[int, int], int]] = None,
                 times: Optional[Dict[Tuple[int, int], Dict[int, float]]] = None, arrangement: str = "complement"):
        # arrangement: what the ADiT call gets beside a restricted VLM stream - "complement": an sm_budget of the
        # remaining SMs (both stages take an explicit allotment); "vlm_only": no restriction (the paper's arrangement:
        # only the VLM stream is confined, the ADiT kernels run wherever SMs are free)
        assert arrangement in ("complement", "vlm_only")
        self.arrangement = arrangement
        self.n_sm = int(n_sm)
        self.entries: Dict[Tuple[int, int], int] = dict(entries or {})
        self.times: Dict[Tuple[int, int], Dict[int, float]] = dict(times or {})

    def lookup(self, vlm_batch: int, adit_batch: int) -> int:
        """Restriction for this pair; pairs that were not profiled (for instance an idle stage) run unrestricted."""
        return self.entries.get((int(vlm_batch), int(adit_batch)), 0)

    def budgets(self, vlm_batch: int, adit_batch: int) -> Tuple[int, int]:
        """(SMs for the VLM stream, sm_budget of the ADiT call); (0, 0) = both unrestricted."""
        cap = self.lookup(vlm_batch, adit_batch)
        if cap <= 0:
            return (0, 0)
        return (cap, self.n_sm - cap) if self.arrangement == "complement" else (cap, 0)

    @classmethod
    def profile(cls, n_sm: int, max_batch: int, time_lockstep: Callable[[int, int, int], float], step: int = 8,
                candidates: Optional[Sequence[int]] = None, arrangement: str = "complement") -> "SmTable":
        """Offline sweep: for every pair of batch sizes time a lockstep under every candidate restriction
        (`time_lockstep(vlm_batch, adit_batch, vlm_sms)` returns seconds; vlm_sms = 0 means unrestricted) and keep the
        fastest.  Ties go to the smaller restriction index, i.e. to the candidate tried first."""
        cand = list(candidates) if candidates is not None else sm_candidates(n_sm, step)
        table = cls(n_sm, arrangement=arrangement)
        for vb in batch_sizes(max_batch):
            for ab in batch_sizes(max_batch):
                t = {c: float(time_lockstep(vb, ab, c)) for c in cand}
                best = min(cand, key=lambda c: (t[c], cand.index(c)))
                table.entries[(vb, ab)] = best
                table.times[(vb, ab)] = t
        return table

    def to_json(self) -> str:
        return json.dumps({"n_sm": self.n_sm, "arrangement": self.arrangement,
                           "entries": [[vb, ab, c] for (vb, ab), c in sorted(self.entries.items())],
                           "times": [[vb, ab, {str(c): v for c, v in t.items()}] for (vb, ab), t in sorted(self.times.items())]})

    @classmethod
    def from_json(cls, text: str) -> "SmTable":
        d = json.loads(text)
        return cls(d["n_sm"], {(vb, ab): c for vb, ab, c in d["entries"]},
                   {(vb, ab): {int(c): v for c, v in t.items()} for vb, ab, t in d.get("times", [])},
                   arrangement=d.get("arrangement", "complement"))


@dataclass
class Request:
    model: str
    request_id: int
    arrival_us: int
    payload: object = None
    vlm_output: object = None      # what the VLM stage hands to the ADiT stage (the temporary buffer of the paper)
    result: object = None
    done_us: int = -1


@dataclass
class LockstepRecord:
    index: int
    vlm_model: Optional[str]
    vlm_ids: List[int]
    adit_model: Optional[str]
    adit_ids: List[int]
    vlm_sms: int
    adit_sms: int
    seconds: float
    vlm_interval: Tuple[float, float] = (0.0, 0.0)
    adit_interval: Tuple[float, float] = (0.0, 0.0)


class LockstepExecutor:
    """Runs queued requests through VLM and ADiT stages in locksteps.

    vlm_stage(model, requests, vlm_sms) runs the VLM stage of the batch to completion on the VLM stream and stores
    each request's hand-over in request.vlm_output; adit_stage(model, requests, adit_sms) runs the ADiT stage on the
    ADiT stream and stores request.result.  sms = 0 means unrestricted.  Both are called from their own thread.
    """

    def __init__(self, vlm_stage: Callable, adit_stage: Callable, max_batch: int, table: SmTable,
                 slo_us: Dict[str, int], clock: Callable[[], float] = time.perf_counter):
        self.vlm_stage, self.adit_stage = vlm_stage, adit_stage
        self.max_batch, self.table, self.slo_us, self.clock = int(max_batch), table, dict(slo_us), clock
        self.queues: Dict[str, Deque[Request]] = {m: deque() for m in slo_us}
        self.records: List[LockstepRecord] = []

    def submit(self, req: Request):
        self.queues[req.model].append(req)

    def _pick_queue(self, now_us: int) -> Optional[str]:
        """Earliest-SLO-first over the heads of the non-empty queues that have arrived."""
        heads = [(m, q[0]) for m, q in self.queues.items() if q and q[0].arrival_us <= now_us]
        if not heads:
            return None
        order = scheduler.esf_order([h.arrival_us for _, h in heads], [self.slo_us[m] for m, _ in heads], now_us,
                                    [h.request_id for _, h in heads])
        return heads[order[0]][0]

    def _admit(self, now_us: int) -> Tuple[Optional[str], List[Request]]:
        model = self._pick_queue(now_us)
        if model is None:
            return None, []
        q = self.queues[model]
        waiting = sum(1 for r in q if r.arrival_us <= now_us)     # FIFO: the arrived requests are a prefix of the queue
        n = admit_batch_size(waiting, self.max_batch)
        return model, [q.popleft() for _ in range(n)]

    def run(self, until_idle: bool = True, max_locksteps: int = 1 << 30) -> List[LockstepRecord]:
        """Locksteps until every queue is empty and the last VLM batch has gone through the ADiT stage."""
        t_start = self.clock()
        now_us = lambda: int((self.clock() - t_start) * 1e6)
        barrier = threading.Barrier(3)              # the two stage threads and this thread
        work = {"vlm": None, "adit": None, "stop": False}
        spans = {"vlm": (0.0, 0.0), "adit": (0.0, 0.0)}
        errors: List[BaseException] = []

        def stage_thread(which: str, fn: Callable):
            while True:
                barrier.wait()                      # lockstep start
                if work["stop"]:
                    return
                job = work[which]
                t0 = self.clock()
                try:
                    if job is not None:
                        fn(*job)
                except BaseException as e:          # noqa: BLE001 - reported by run()
                    errors.append(e)
                spans[which] = (t0 - t_start, self.clock() - t_start)
                barrier.wait()                      # lockstep end: both stages have finished

        threads = [threading.Thread(target=stage_thread, args=("vlm", self.vlm_stage), daemon=True),
                   threading.Thread(target=stage_thread, args=("adit", self.adit_stage), daemon=True)]
        [t.start() for t in threads]
        handed: Tuple[Optional[str], List[Request]] = (None, [])    # batch k-1: through the VLM stage, waiting for ADiT
        k = 0
        try:
            while k < max_locksteps:
                model, batch = self._admit(now_us())
                a_model, a_batch = handed
                if not batch and not a_batch:
                    pending = [q[0].arrival_us for q in self.queues.values() if q]
                    if not pending:
                        break
                    time.sleep(max(0.0, (min(pending) - now_us()) * 1e-6))      # nothing has arrived yet
                    continue
                vlm_sms, adit_sms = self.table.budgets(len(batch), len(a_batch)) if batch and a_batch else (0, 0)
                work["vlm"] = (model, batch, vlm_sms) if batch else None
                work["adit"] = (a_model, a_batch, adit_sms) if a_batch else None
                t0 = self.clock()
                barrier.wait()
                barrier.wait()
                t1 = self.clock()
                if errors:
                    raise errors[0]
                for r in a_batch:
                    r.done_us = now_us()
                self.records.append(LockstepRecord(k, model if batch else None, [r.request_id for r in batch], a_model if a_batch else None,
                                                   [r.request_id for r in a_batch], vlm_sms, adit_sms, t1 - t0,
                                                   spans["vlm"] if batch else (0.0, 0.0), spans["adit"] if a_batch else (0.0, 0.0)))
                handed = (model, batch)
                k += 1
        finally:
            work["stop"] = True
            barrier.wait()
            [t.join() for t in threads]
        return self.records


class GpuStages:
    """The two stage callables on a B200: a capped GEMM loop as the VLM stand-in (its work grows with the batch) and
    adit_denoise as the ADiT stage, each on its own stream and synchronised by its own thread."""

    def __init__(self, adit_mod, engines: Dict[str, object], inputs: Dict[str, dict], vlm_iters_per_request: int = 6,
                 gemm_shape: Tuple[int, int, int] = (8192, 2048, 2048), device: int = 0, restriction: str = "grid"):
        # restriction: how the VLM stream is held to its SMs - "grid": the stand-in's grid is capped (it honours a cap);
        # "green": its full grid runs on a green-context stream of that many SMs (the paper's mechanism, which also
        # confines kernels that were not written for a budget)
        import torch
        assert restriction in ("grid", "green")
        self.restriction, self.device, self._green = restriction, device, {}
        self.torch, self.adit = torch, adit_mod
        self.engines, self.inputs = engines, inputs
        self.vlm_iters = int(vlm_iters_per_request)
        self.bg = adit_mod.BackgroundGemm(*gemm_shape, device=device)
        self.s_vlm, self.s_adit = torch.cuda.Stream(device=device), torch.cuda.Stream(device=device)
        self.n_sm = torch.cuda.get_device_properties(device).multi_processor_count

    def vlm(self, model: str, requests: List[Request], sms: int):
        stream = self.s_vlm
        if self.restriction == "green" and sms > 0:
            if sms not in self._green:
                self._green[sms] = self.adit.GreenStream(sms, device=self.device)
            stream, sms = self._green[sms].stream, 0     # the driver confines the full grid
        self.bg.launch(self.vlm_iters * len(requests), sms, stream)
        for r in requests:                              # hand-over: the request's (precomputed) prefix cache
            r.vlm_output = r.payload
        stream.synchronize()

    def adit_stage(self, model: str, requests: List[Request], sms: int):
        torch = self.torch
        inp, eng = self.inputs[model], self.engines[model]
        idx = [r.vlm_output for r in requests]
        sel = torch.tensor(idx, device=inp["state"].device)
        out = eng.denoise([inp["kv"][i] for i in idx], [int(inp["len"][i]) for i in idx], inp["state"][sel].contiguous(),
                          inp["noise"][sel].contiguous(), inp["steps"], sm_budget=sms, stream=self.s_adit)
        self.s_adit.synchronize()
        for j, r in enumerate(requests):
            r.result = out[j]

    def time_lockstep(self, model: str, vlm_batch: int, adit_batch: int, vlm_sms: int, reps: int = 3,
                      arrangement: str = "complement") -> float:
        """Seconds for one lockstep of this pair (both stages launched together, until both are done), best of reps."""
        best = float("inf")
        reqs_v = [Request(model, i, 0, payload=i % len(self.inputs[model]["kv"])) for i in range(vlm_batch)]
        reqs_a = [Request(model, i, 0, payload=i % len(self.inputs[model]["kv"])) for i in range(adit_batch)]
        for r in reqs_a:
            r.vlm_output = r.payload
        adit_sms = self.n_sm - vlm_sms if (vlm_sms > 0 and arrangement == "complement") else 0
        for _ in range(reps + 1):
            self.torch.cuda.synchronize()
            t0 = time.perf_counter()
            tv = threading.Thread(target=self.vlm, args=(model, reqs_v, vlm_sms))
            ta = threading.Thread(target=self.adit_stage, args=(model, reqs_a, adit_sms))
            tv.start(); ta.start(); tv.join(); ta.join()
            best = min(best, time.perf_counter() - t0)
        return best

    def close(self):
        for g in self._green.values():
            g.close()
        self._green = {}
        self.bg.close()
