"""Traffic controller: how many robots of each model every GPU serves (paper section 4.2.2, Eq. 1-3).

Inputs: the robot population N_i of every model, the largest population C_i one GPU sustains for that model at the
target SLO attainment, the number of GPUs and (optionally) which GPU hosts which model.  Output: integers r_ij with
sum_j r_ij = N_i (Eq. 1) and sum_i r_ij / C_i <= 1 on every GPU (Eq. 2) that minimise the number of robot pairs of
distinct models sharing a GPU, sum_j sum_{i<k} r_ij r_kj (Eq. 3), so that a GPU serves a single model wherever the
limits allow and a model's requests concentrate in one queue.  Infeasible inputs raise, as the paper's engine
reports them to the programmer.  Runs on the host; exact.

Method: models are placed one after the other.  With T_j the robots already on GPU j, placing r_kj robots of model k
adds sum_j r_kj T_j to Eq. 3, so the cost-to-go depends only on (k, per-GPU robot counts, per-GPU load); a depth-first
search over each model's splits with that memo, an admissible bound (cost so far) and largest-first model order.
Loads are integers on the common denominator lcm(C), so Eq. 2 is tested exactly.
"""
from __future__ import annotations

from functools import lru_cache
from math import lcm
from typing import List, Optional, Sequence


class Infeasible(ValueError):
    """Eq. 1 and Eq. 2 cannot both hold: choose another placement or add GPUs (paper section 4.2.2)."""


def _splits(n: int, caps: Sequence[int]):
    """Ordered ways to split n robots over GPUs with per-GPU room caps[j]."""
    if len(caps) == 1:
        if n <= caps[0]:
            yield (n,)
        return
    rest_room = sum(caps[1:])
    for first in range(min(n, caps[0]), max(0, n - rest_room) - 1, -1):
        for rest in _splits(n - first, caps[1:]):
            yield (first,) + rest


def assign_robots(n: Sequence[int], c: Sequence[int], n_gpus: int,
                  hosts: Optional[Sequence[Sequence[bool]]] = None) -> List[List[int]]:
    """r[i][j]: robots of model i served by GPU j.  Raises Infeasible when no assignment satisfies Eq. 1 and Eq. 2."""
    m = len(n)
    if len(c) != m or n_gpus < 1 or any(v < 0 for v in n) or any(v < 1 for v in c):
        raise ValueError("bad arguments")
    unit = lcm(*c) if m else 1
    weight = [unit // ci for ci in c]                    # load of one robot of model i, in units of 1 / lcm(C)
    order = sorted(range(m), key=lambda i: -n[i] * weight[i])
    host = [[True] * n_gpus for _ in range(m)] if hosts is None else [list(map(bool, row)) for row in hosts]

    # GPUs that host the same models are interchangeable: states are kept with such GPUs in sorted order, which
    # collapses the symmetric branches (the splits returned are permuted back at the end).
    sig = [tuple(host[i][j] for i in range(m)) for j in range(n_gpus)]

    @lru_cache(maxsize=None)
    def cost_to_go(pos: int, state: tuple):
        """state[j] = (hosting signature, robots, load) of GPU slot j, sorted.  Returns (minimal additional Eq.-3 cost,
        per remaining model its split over the slots of ITS state, and the slot permutations) or None if infeasible."""
        if pos == m:
            return 0, ()
        i = order[pos]
        caps = [((unit - st[2]) // weight[i]) if st[0][i] else 0 for st in state]
        found = None
        for split in _splits(n[i], caps):
            add = sum(split[j] * state[j][1] for j in range(n_gpus))
            if found is not None and add >= found[0]:
                continue
            nxt = [(state[j][0], state[j][1] + split[j], state[j][2] + split[j] * weight[i]) for j in range(n_gpus)]
            perm = sorted(range(n_gpus), key=lambda j: nxt[j])          # slot of the sorted next state <- slot here
            sub = cost_to_go(pos + 1, tuple(nxt[j] for j in perm))
            if sub is None:
                continue
            if found is None or add + sub[0] < found[0]:
                found = (add + sub[0], ((split, tuple(perm)),) + sub[1])
                if found[0] == 0:
                    break
        return found

    start = sorted(range(n_gpus), key=lambda j: (sig[j], 0, 0))
    res = cost_to_go(0, tuple((sig[j], 0, 0) for j in start))
    if res is None:
        raise Infeasible("no assignment keeps every GPU within its robot limits")
    rows = [[0] * n_gpus for _ in range(m)]
    slot_gpu = list(start)                                  # physical GPU behind each slot of the current state
    for pos, (split, perm) in enumerate(res[1]):
        for j in range(n_gpus):
            rows[order[pos]][slot_gpu[j]] = split[j]
        slot_gpu = [slot_gpu[j] for j in perm]
    return rows


def shared_pairs(r: Sequence[Sequence[int]]) -> int:
    """Eq. 3 for an assignment."""
    m, g = len(r), len(r[0]) if r else 0
    return sum(r[i][j] * r[k][j] for j in range(g) for i in range(m) for k in range(i + 1, m))
