"""Algorithm 2, Phase A (budgeted joint planning of bits and kept timesteps): pins for the oracle's
restatement and CPU parity of the library's heap-based implementation against it. No GPU needed:
the planner is host arithmetic (its latency table is measured elsewhere)."""
import os

import numpy as np
import pytest

import oracle
from paper_2511_11446_b200 import binding as B

GOLD = os.path.join(os.path.dirname(__file__), "golden", "phase_a_small.txt")


def _fixture():
    drift = cost = budgets = None
    layers, sens, exp = [], [], {}
    for line in open(GOLD):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, *rest = line.split()
        if key == "drift":
            drift = [float(v) for v in rest]
        elif key == "step_cost":
            cost = [float(v) for v in rest]
        elif key == "layer":
            sens.append(float(rest[0]))
            layers.append([tuple(float(v) if i else int(v) for i, v in enumerate(o.split(":"))) for o in rest[1:]])
        elif key == "budgets":
            budgets = [float(v) for v in rest]
        else:
            exp[key] = [float(v) for v in rest]
    return drift, cost, layers, sens, budgets, exp


@pytest.mark.parametrize("impl", [oracle.phase_a, B.dp_plan_phase_a], ids=["oracle", "library"])
def test_hand_worked_example(impl):
    drift, cost, layers, sens, (B_lat, B_mem), exp = _fixture()
    plan, kept, tot, ok = impl(drift, cost, layers, sens, B_lat, B_mem, 0.2, 0.0)
    assert ok
    assert plan == [int(v) for v in exp["expect_bits"]]
    assert kept == [int(v) for v in exp["expect_kept"]]
    assert list(tot) == exp["expect_totals"]


def _random_problem(rng, T, L):
    drift = (rng.random(T) ** 3 * 10 + 0.01).tolist()
    cost = (rng.random(T) * 3 + 0.5).tolist()
    options = []
    for _ in range(L):
        n = int(rng.integers(1, 4))
        bits = sorted(rng.choice([3, 4, 6, 8, 16], size=n, replace=False).tolist(), reverse=True)
        base_lat, base_mem = rng.random() * 5 + 1, rng.random() * 50 + 5
        options.append([(b, base_lat * (0.5 + b / 16), base_mem * b / 16) for b in bits])
    sens = (rng.random(L) * 4 + 0.05).tolist()
    return drift, cost, options, sens


def test_invariants_of_the_greedy_plan():
    """Whatever the instance: the protected tail is kept; each layer's bits are one of its options;
    the totals equal a recomputation from the outputs; the budgets hold whenever the run is
    feasible and an infeasible run has used every move; looser budgets than the start change
    nothing; dropped steps are exactly the least-drift prunable ones (a prefix of R)."""
    rng = np.random.default_rng(2511)
    for case in range(200):
        T, L = int(rng.integers(2, 40)), int(rng.integers(1, 30))
        drift, cost, options, sens = _random_problem(rng, T, L)
        rho = float(rng.choice([0.0, 0.2, 0.5]))
        lat0 = sum(cost) + sum(o[0][1] for o in options)
        mem0 = sum(o[0][2] for o in options)
        B_lat, B_mem = lat0 * float(rng.uniform(0.3, 1.1)), mem0 * float(rng.uniform(0.3, 1.1))
        plan, kept, (c_lat, c_mem), ok = oracle.phase_a(drift, cost, options, sens, B_lat, B_mem, rho, 1e-6)
        n_tail = int(np.floor(rho * T))
        assert all(kept[t] for t in range(T - n_tail, T))
        chosen = []
        for l, o in enumerate(options):
            match = [x for x in o if x[0] == plan[l]]
            assert len(match) == 1
            chosen.append(match[0])
        assert c_lat == pytest.approx(sum(c for c, k in zip(cost, kept) if k) + sum(x[1] for x in chosen), rel=1e-9)
        assert c_mem == pytest.approx(sum(x[2] for x in chosen), rel=1e-9, abs=1e-9)
        if ok:
            assert c_lat <= B_lat and c_mem <= B_mem
        else:
            assert not any(kept[: T - n_tail]) and all(x == o[-1] for x, o in zip(chosen, options))
        dropped = [t for t in range(T - n_tail) if not kept[t]]
        by_drift = sorted(range(T - n_tail), key=lambda t: (drift[t], t))
        assert sorted(dropped) == sorted(by_drift[:len(dropped)])
        if B_lat >= lat0 and B_mem >= mem0:
            assert all(kept) and plan == [o[0][0] for o in options]


def test_single_resource_cases_reduce_to_sorting():
    """Closed forms. (i) No bit options and a latency budget: the plan drops least-drift prunable steps
    one by one until the budget holds. (ii) No prunable step (rho = 1) and equal sensitivities: layers
    move in order of latency saving until the budget holds."""
    drift = [4.0, 0.5, 2.0, 8.0, 1.0, 3.0]
    cost = [1.0] * 6
    plan, kept, (c_lat, _), ok = oracle.phase_a(drift, cost, [[(8, 2.0, 1.0)]], [1.0], 5.5, 10.0, 0.0, 0.0)
    # start 6 + 2 = 8 > 5.5: drop t=1 (7), t=4 (6), t=2 (5) -> stop
    assert ok and kept == [1, 0, 0, 1, 0, 1] and plan == [8] and c_lat == 5.0
    options = [[(8, 5.0, 1.0), (4, 1.0, 1.0)], [(8, 5.0, 1.0), (4, 4.0, 1.0)], [(8, 5.0, 1.0), (4, 2.0, 1.0)]]
    plan, kept, (c_lat, _), ok = oracle.phase_a([1.0, 1.0], [0.0, 0.0], options, [1.0, 1.0, 1.0], 9.0, 10.0, 1.0, 0.0)
    # savings 4, 1, 3: layer 0 first (15 -> 11), then layer 2 (11 -> 8 <= 9)
    assert ok and plan == [4, 8, 4] and kept == [1, 1] and c_lat == 8.0


def test_memory_clause_prefers_moves_that_reach_the_budget():
    """Two next moves: the better-scored one leaves C_mem above B_mem, the other brings it under: the
    clause makes the second the bit candidate; with no move able to reach the budget the best-scored
    one is taken (reading recorded in the header)."""
    options = [[(8, 10.0, 10.0), (4, 2.0, 9.0)], [(8, 10.0, 10.0), (4, 9.0, 2.0)]]
    plan, kept, (c_lat, c_mem), ok = oracle.phase_a([1.0], [0.0], options, [1.0, 1.0], 100.0, 12.0, 1.0, 0.0)
    assert ok and plan == [8, 4] and c_mem == 12.0
    plan, kept, (c_lat, c_mem), ok = oracle.phase_a([1.0], [0.0], options, [1.0, 1.0], 100.0, 11.5, 1.0, 0.0)
    # neither single move reaches 11.5 from 20: the best-scored (layer 0) goes first, then layer 1 reaches 11
    assert ok and plan == [4, 4] and c_mem == 11.0


def test_library_planner_equals_oracle_on_random_instances():
    rng = np.random.default_rng(7)
    for case in range(300):
        T, L = int(rng.integers(1, 60)), int(rng.integers(1, 150))
        drift, cost, options, sens = _random_problem(rng, T, L)
        if case % 5 == 0:  # ties in scores and drifts
            sens = [1.0] * L
            drift = [float(int(d)) for d in drift]
        rho = float(rng.choice([0.0, 0.2, 1.0]))
        lat0 = sum(cost) + sum(o[0][1] for o in options)
        mem0 = sum(o[0][2] for o in options)
        B_lat, B_mem = lat0 * float(rng.uniform(0.2, 1.05)), mem0 * float(rng.uniform(0.2, 1.05))
        a = oracle.phase_a(drift, cost, options, sens, B_lat, B_mem, rho, 1e-6)
        b = B.dp_plan_phase_a(drift, cost, options, sens, B_lat, B_mem, rho, 1e-6)
        assert a[0] == b[0] and a[1] == b[1] and a[3] == b[3], case
        assert a[2] == pytest.approx(b[2], rel=1e-12)
    with pytest.raises(B.DiffproError):
        B.dp_plan_phase_a([1.0], [1.0], [[]], [1.0], 1.0, 1.0, 0.2, 0.0)
