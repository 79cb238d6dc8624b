"""Traffic controller (paper section 4.2.2, Eq. 1-3): the exact solver against the brute-force oracle, and the
oracle against what the paper and the mathematics fix."""
import numpy as np
import pytest

from oracle import traffic_oracle as TO
from paper_2609_12075_b200 import traffic as T

import os
GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "traffic_example.txt")


def canon(r):
    """An assignment up to the naming of the GPUs."""
    return sorted(tuple(col) for col in zip(*r))


# ---- the oracle against the paper's worked example and closed forms ---------------------------------------------

def test_oracle_reproduces_the_papers_worked_example():
    want = np.loadtxt(GOLDEN, dtype=int).tolist()
    val, r = TO.solve([6, 2], [4, 4], 2)
    assert val == TO.objective(want) == 4
    assert canon(r) == canon(want)
    # the two schemes the paper rejects: one model per GPU overloads GPU 0, the even split shares more pairs
    assert not TO.feasible([[6, 0], [0, 2]], [6, 2], [4, 4], None)
    assert TO.feasible([[3, 3], [1, 1]], [6, 2], [4, 4], None) and TO.objective([[3, 3], [1, 1]]) == 6 > val


def test_oracle_closed_forms():
    # every model fits a GPU of its own: nothing is shared
    assert TO.solve([3, 2, 4], [4, 4, 4], 3)[0] == 0
    # a single GPU: every pair of robots of distinct models shares it
    n = [2, 1, 3]
    assert TO.solve(n, [12, 12, 12], 1)[0] == 2 * 1 + 2 * 3 + 1 * 3
    # total load above the number of GPUs: infeasible (Eq. 2 summed over the GPUs)
    assert TO.solve([5, 4], [4, 4], 2) is None
    # limits differ per model: 2 robots of a model with limit 2 fill a GPU completely
    val, r = TO.solve([2, 3], [2, 6], 2)
    assert val == 0 and canon(r) == canon([[2, 0], [0, 3]])
    # hosting restriction: model 1 may only use GPU 0
    val, r = TO.solve([2, 2], [4, 4], 2, hosts=[[True, True], [True, False]])
    assert r[1] == [2, 0] and val == 0


# ---- the solver against the oracle ---------------------------------------------------------------------------------

def test_solver_reproduces_the_papers_worked_example():
    want = np.loadtxt(GOLDEN, dtype=int).tolist()
    r = T.assign_robots([6, 2], [4, 4], 2)
    assert canon(r) == canon(want) and T.shared_pairs(r) == 4


def test_solver_matches_brute_force_on_small_instances():
    rng = np.random.default_rng(17)
    seen_infeasible = seen_shared = 0
    for _ in range(120):
        m, g = int(rng.integers(1, 4)), int(rng.integers(1, 4))
        n = [int(v) for v in rng.integers(0, 6, size=m)]
        c = [int(v) for v in rng.integers(1, 7, size=m)]
        hosts = None
        if rng.random() < 0.3:
            hosts = [[bool(v) for v in rng.integers(0, 2, size=g)] for _ in range(m)]
        want = TO.solve(n, c, g, hosts)
        if want is None:
            seen_infeasible += 1
            with pytest.raises(T.Infeasible):
                T.assign_robots(n, c, g, hosts)
            continue
        r = T.assign_robots(n, c, g, hosts)
        assert TO.feasible(r, n, c, hosts), (n, c, g, hosts, r)
        assert T.shared_pairs(r) == want[0], (n, c, g, hosts, r, want)
        seen_shared += want[0] > 0
    assert seen_infeasible > 5 and seen_shared > 5


def test_solver_on_a_multi_model_server():
    # six models of two architectures on three GPUs (the shape of the paper's multi-GPU experiments, scaled down):
    # two whole models per GPU is feasible, and sharing a GPU between two models of 6 robots costs 36 pairs
    n, c = [6] * 6, [27, 27, 27, 32, 32, 32]
    r = T.assign_robots(n, c, 3)
    assert [sum(row) for row in r] == n
    assert all(sum(r[i][j] / c[i] for i in range(6)) <= 1 + 1e-12 for j in range(3))
    assert T.shared_pairs(r) == 3 * 36
