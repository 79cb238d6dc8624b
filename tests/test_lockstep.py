"""Lockstep executor and SM-restriction table (paper sections 4.1.2 and 4.1.3): host logic with fake stages."""
import threading
import time

import pytest

from paper_2609_12075_b200 import lockstep as L


def test_admission_takes_the_largest_power_of_two():
    assert [L.admit_batch_size(p, 8) for p in range(0, 11)] == [0, 1, 2, 2, 4, 4, 4, 4, 8, 8, 8]
    assert [L.admit_batch_size(p, 2) for p in range(0, 5)] == [0, 1, 2, 2, 2]
    assert L.admit_batch_size(5, 3) == 2 and L.admit_batch_size(100, 1) == 1
    assert L.batch_sizes(8) == [1, 2, 4, 8] and L.batch_sizes(2) == [1, 2] and L.batch_sizes(6) == [1, 2, 4]


def test_sm_candidates_are_multiples_of_eight_plus_unrestricted():
    c = L.sm_candidates(148)
    assert c[-1] == 0 and c[:-1] == list(range(8, 148, 8)) and all(v % 8 == 0 for v in c)
    assert L.sm_candidates(188)[-2] == 184          # the paper's GPU: 188 SMs


def test_profile_keeps_the_fastest_restriction_per_batch_pair():
    # a lockstep's time: the slower of a compute-bound VLM stage (work / SMs) and an ADiT stage that needs a few SMs;
    # unrestricted, the VLM stage blocks the ADiT stage, which then runs after it (section 4.1.2, the unguarded case)
    n_sm = 64

    def t(vb, ab, cap):
        if cap == 0:
            return vb * 64.0 / n_sm + ab * 0.25
        return max(vb * 64.0 / cap, ab * 0.25 * max(1.0, 8.0 / (n_sm - cap)))
    table = L.SmTable.profile(n_sm, 4, t)
    assert set(table.entries) == {(v, a) for v in (1, 2, 4) for a in (1, 2, 4)}
    for (vb, ab), cap in table.entries.items():
        assert all(t(vb, ab, cap) <= t(vb, ab, c) for c in L.sm_candidates(n_sm)), (vb, ab)
    # a light VLM batch beside a heavy ADiT batch: leaving 8 SMs to the ADiT stage wins; a heavy VLM batch beside a
    # light ADiT batch: giving up an eighth of the chip costs more than running the ADiT stage afterwards
    assert table.lookup(1, 4) == 56 and table.lookup(4, 1) == 0
    assert table.budgets(1, 4) == (56, 8) and table.budgets(8, 8) == (0, 0)      # unprofiled pair: unrestricted
    # the paper's arrangement: only the VLM stream is restricted, the ADiT call gets no budget (0 = unrestricted)
    paper = L.SmTable.profile(n_sm, 4, t, arrangement="vlm_only")
    assert paper.entries == table.entries and paper.budgets(1, 4) == (56, 0) and paper.budgets(4, 1) == (0, 0)
    assert L.SmTable.from_json(paper.to_json()).arrangement == "vlm_only" and L.SmTable.from_json(table.to_json()).arrangement == "complement"
    back = L.SmTable.from_json(table.to_json())
    assert back.entries == table.entries and back.n_sm == n_sm and back.times[(2, 1)][56] == t(2, 1, 56) and back.lookup(1, 4) == 56
    # when restricting never pays, the table says "no restriction"
    flat = L.SmTable.profile(n_sm, 2, lambda vb, ab, cap: 1.0 if cap == 0 else 1.5)
    assert set(flat.entries.values()) == {0}


class FakeStages:
    def __init__(self):
        self.log, self.lock, self.active = [], threading.Lock(), set()
        self.overlaps = 0

    def _run(self, which, model, reqs, sms):
        with self.lock:
            self.active.add(which)
            if len(self.active) == 2:
                self.overlaps += 1
            self.log.append((which, "start", model, [r.request_id for r in reqs], sms))
        time.sleep(0.003)
        for r in reqs:
            if which == "vlm":
                r.vlm_output = ("kv", r.request_id)
            else:
                assert r.vlm_output == ("kv", r.request_id)          # the ADiT stage sees what the VLM stage handed over
                r.result = ("act", r.request_id)
        with self.lock:
            self.active.discard(which)
            self.log.append((which, "end", model, [r.request_id for r in reqs], sms))

    def vlm(self, model, reqs, sms): self._run("vlm", model, reqs, sms)
    def adit(self, model, reqs, sms): self._run("adit", model, reqs, sms)


def test_locksteps_pair_vlm_batch_k_with_adit_batch_k_minus_1():
    st = FakeStages()
    table = L.SmTable(148, {(2, 2): 120, (1, 2): 136, (2, 1): 112})
    ex = L.LockstepExecutor(st.vlm, st.adit, max_batch=2, table=table, slo_us={"A": 50_000})
    reqs = [L.Request("A", i, 0) for i in range(5)]
    [ex.submit(r) for r in reqs]
    rec = ex.run()
    # batches 2, 2, 1 -> four locksteps: the last one only drains the ADiT stage
    assert [(r.vlm_ids, r.adit_ids) for r in rec] == [([0, 1], []), ([2, 3], [0, 1]), ([4], [2, 3]), ([], [4])]
    assert [(r.vlm_sms, r.adit_sms) for r in rec] == [(0, 0), (120, 28), (136, 12), (0, 0)]
    assert all(r.result == ("act", r.request_id) and r.done_us >= 0 for r in reqs)
    assert st.overlaps >= 2                          # the two stages of a lockstep ran at the same time
    # a lockstep starts only when both stages of the previous one have ended
    depth = 0
    for which, what, *_ in st.log:
        depth += 1 if what == "start" else -1
        assert 0 <= depth <= 2
    starts = [i for i, e in enumerate(st.log) if e[1] == "start"]
    ends = [i for i, e in enumerate(st.log) if e[1] == "end"]
    assert starts[1] > ends[0]                       # lockstep 1 (two stages) begins after lockstep 0's only stage ended
    assert min(starts[3:5]) > max(ends[1:3])         # lockstep 2 after both stages of lockstep 1


def test_earliest_slo_first_across_model_queues():
    st = FakeStages()
    ex = L.LockstepExecutor(st.vlm, st.adit, max_batch=2, table=L.SmTable(148), slo_us={"slow": 150_000, "fast": 50_000})
    # both queues have waited equally long: the tighter deadline goes first; then the other queue's head has less
    # time left than the remaining fast request that arrived later
    ex.submit(L.Request("slow", 0, 0)); ex.submit(L.Request("slow", 1, 0))
    ex.submit(L.Request("fast", 10, 0))
    rec = ex.run()
    assert [r.vlm_model for r in rec if r.vlm_ids] == ["fast", "slow"]
    assert [r.vlm_ids for r in rec if r.vlm_ids] == [[10], [0, 1]]


def test_stage_errors_surface_and_threads_stop():
    def boom(model, reqs, sms):
        raise RuntimeError("stage failed")
    ex = L.LockstepExecutor(boom, lambda *a: None, max_batch=1, table=L.SmTable(8), slo_us={"A": 1})
    ex.submit(L.Request("A", 0, 0))
    with pytest.raises(RuntimeError):
        ex.run()
    assert threading.active_count() < 8
