"""Brute-force oracle for the traffic controller's integer program.  TEST INFRASTRUCTURE ONLY.

Paper section 4.2.2 ("Adaptive Traffic Controller"): for M models with robot populations N_i and per-GPU robot
limits C_i on G GPUs, find integers r_ij >= 0 with

    sum_j r_ij = N_i                      for every model i          (Eq. 1)
    sum_i r_ij / C_i <= 1                 for every GPU j            (Eq. 2)
    minimise  sum_j sum_{i<k} r_ij r_kj                              (Eq. 3)

and r_ij = 0 where GPU j does not host model i.  This file is the definition written out: it enumerates every
assignment of every model's robots to the GPUs, keeps the feasible ones and returns the smallest objective.  Only
usable for tiny instances; only tests may import it.

Pins (tests/test_traffic.py): the worked example of the paper's traffic figure (two GPUs, models A and B with 6 and 2
robots, limit 4: 4 x A on one GPU, 2 x A + 2 x B on the other; stored under tests/golden/), instances whose optimum is
known in closed form (one model per GPU fits: objective 0; a single GPU: objective sum_{i<k} N_i N_k), infeasibility
by total load.  Fractions are compared exactly (integer arithmetic on the common denominator).
"""
from __future__ import annotations

from fractions import Fraction
from itertools import product
from typing import List, Optional, Sequence, Tuple


def compositions(n: int, parts: int):
    """All ways to write n as an ordered sum of `parts` non-negative integers."""
    if parts == 1:
        yield (n,)
        return
    for first in range(n + 1):
        for rest in compositions(n - first, parts - 1):
            yield (first,) + rest


def objective(r: Sequence[Sequence[int]]) -> int:
    """Eq. 3: robots of distinct models that share a GPU, counted in pairs."""
    m, g = len(r), len(r[0])
    return sum(r[i][j] * r[k][j] for j in range(g) for i in range(m) for k in range(i + 1, m))


def feasible(r, n, c, hosts) -> bool:
    m, g = len(r), len(r[0])
    if any(sum(r[i]) != n[i] for i in range(m)):
        return False
    if hosts is not None and any(r[i][j] and not hosts[i][j] for i in range(m) for j in range(g)):
        return False
    return all(sum(Fraction(r[i][j], c[i]) for i in range(m)) <= 1 for j in range(g))


def solve(n: Sequence[int], c: Sequence[int], n_gpus: int, hosts=None) -> Optional[Tuple[int, List[List[int]]]]:
    """(minimum of Eq. 3, one minimiser) over all assignments satisfying Eq. 1 and Eq. 2, or None if there is none."""
    best = None
    for r in product(*[list(compositions(n[i], n_gpus)) for i in range(len(n))]):
        if not feasible(r, n, c, hosts):
            continue
        val = objective(r)
        if best is None or val < best[0]:
            best = (val, [list(row) for row in r])
    return best
