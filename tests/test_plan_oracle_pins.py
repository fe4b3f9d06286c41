"""Pins of the plan-search oracle (oracle/plan.py) against what the paper's cost model fixes: a
hand-worked instance, closed forms, special cases and properties.  CPU only."""
import os
import random

import pytest

from oracle import plan as OP

HERE = os.path.dirname(os.path.abspath(__file__))
A = (40.0, 5.0, 2.0, 8.0, 3.0)
B = (24.0, 10.0, 1.0, 16.0, 2.0)


def _golden():
    plans, best, answer = [], [], None
    for line in open(os.path.join(HERE, "golden", "plan_example.txt")):
        f = line.split()
        if not f or f[0].startswith("#"):
            continue
        if f[0] == "plan":
            plans.append((int(f[1]), (int(f[2]), int(f[3])), float(f[4]), float(f[5])))
        elif f[0] == "best":
            best.append((int(f[1]), (int(f[2]), int(f[3])), float(f[4])))
        elif f[0] == "answer":
            answer = (int(f[1]), (int(f[2]), int(f[3])), float(f[4]))
    return plans, best, answer


def test_hand_worked_instance_costs():
    plans, _, _ = _golden()
    assert len(plans) == 21
    for b, modes, mem, t in plans:
        assert OP.memory_cost([A, B], modes, b, 4) == mem, (b, modes)
        assert OP.time_cost([A, B], modes, b, 4, 1.0, 0.5) == t, (b, modes)


def test_hand_worked_instance_search():
    _, best, answer = _golden()
    modes, b, t, cands = OP.search([A, B], 4, 1.0, 0.5, 100.0, 50)
    assert [(c[2], c[1], c[0]) for c in cands] == best          # stops after b = 5: nothing fits at b = 6
    assert (b, modes, t) == answer


def test_one_rank_has_no_communication_and_no_saving():
    ops = [A, B, (7.0, 1.0, 0.0, 3.0, 0.5)]
    for modes in ((0, 0, 0), (1, 0, 1), (1, 1, 1)):
        assert OP.time_cost(ops, modes, 3, 1, 2.0, 5.0) == 3 * (3.0 + 2.0 + 0.5)
        assert OP.memory_cost(ops, modes, 3, 1) == OP.memory_cost(ops, (0, 0, 0), 3, 1)


def test_zdp_costs_one_more_collective_and_saves_the_other_ranks_share():
    rng = random.Random(5)
    for _ in range(50):
        world = rng.randint(2, 64)
        op = tuple(rng.uniform(0.1, 100.0) for _ in range(5))
        alpha, beta, b = rng.uniform(0, 1), rng.uniform(0, 1), rng.randint(1, 9)
        dt = OP.time_cost([op], (1,), b, world, alpha, beta) - OP.time_cost([op], (0,), b, world, alpha, beta)
        assert dt == pytest.approx((world - 1) * (alpha + op[3] / world * beta), rel=1e-12)
        dm = OP.memory_cost([op], (0,), b, world) - OP.memory_cost([op], (1,), b, world)
        assert dm == pytest.approx(op[0] * (1 - 1 / world), rel=1e-12)


def test_unlimited_memory_gives_all_dp_and_the_largest_batch():
    ops = [A, B, (9.0, 2.0, 1.0, 30.0, 1.0)]
    modes, b, t, cands = OP.search(ops, 8, 0.3, 0.01, float("inf"), 12)
    assert modes == (0, 0, 0) and b == 12 and len(cands) == 12
    comm = sum(2 * 7 * (0.3 + op[3] / 8 * 0.01) for op in ops)
    assert t == pytest.approx(comm / 12 + sum(op[4] for op in ops), rel=1e-12)


def test_nothing_fits():
    assert OP.search([A, B], 4, 1.0, 0.5, 33.9, 10) == (None, 0, float("inf"), [])
    # 34 is exactly the all-ZDP footprint at b = 1: the bound is inclusive
    modes, b, _, _ = OP.search([A, B], 4, 1.0, 0.5, 34.0, 10)
    assert modes == (1, 1) and b == 1


def test_memory_picks_which_operators_stay_replicated():
    # three operators with the same communication saving; only two fit replicated: the optimum keeps
    # the two SMALLEST replicated (a knapsack whose answer is clear by inspection)
    ops = [(30.0, 0.0, 0.0, 10.0, 1.0), (50.0, 0.0, 0.0, 10.0, 1.0), (20.0, 0.0, 0.0, 10.0, 1.0)]
    world = 10                                   # ZDP footprints 3, 5, 2
    modes, b, _, _ = OP.search(ops, world, 1.0, 1.0, 30 + 20 + 5 + 0.5, 1)
    assert modes == (0, 1, 0) and b == 1


def test_smaller_batch_can_win():
    # one operator: replicated it fits b <= 3 (10 + 20 b <= 85), sharded also b = 4 (1 + 80), nothing at b = 5;
    # per sample 2C/3 < 3C/4, so the scheduler must not simply return the last candidate
    op = (10.0, 20.0, 0.0, 40.0, 1.0)
    modes, b, t, cands = OP.search([op], 10, 0.0, 1.0, 85.0, 100)
    assert [(c[2], c[1]) for c in cands] == [(1, (0,)), (2, (0,)), (3, (0,)), (4, (1,))]
    C = 9 * 4.0
    assert (modes, b) == ((0,), 3) and t == pytest.approx(2 * C / 3 + 1.0)
    assert cands[3][0] == pytest.approx(3 * C / 4 + 1.0)


def test_expand_slices_preserves_totals():
    op = (64.0, 8.0, 4.0, 32.0, 2.0)
    sl = OP.expand_slices(op, 4, overhead=0.25)
    assert len(sl) == 4
    for j in range(4):
        assert sum(s[j] for s in sl) == pytest.approx(op[j])
    assert sum(s[4] for s in sl) == pytest.approx(op[4] * 1.25)
    # slicing makes mixed plans possible: with room for three quarters of the states replicated, the
    # sliced operator beats both whole-operator choices
    world, alpha, beta = 8, 0.0, 1.0
    limit = 0.75 * 64 + 0.25 * 64 / world + 8 + 4
    t_whole = OP.search([op], world, alpha, beta, limit, 1)[2]
    t_sliced = OP.search(OP.expand_slices(op, 4), world, alpha, beta, limit, 1)[2]
    assert OP.search([op], world, alpha, beta, limit, 1)[0] == (1,)
    assert sorted(OP.search(OP.expand_slices(op, 4), world, alpha, beta, limit, 1)[0]) == [0, 0, 0, 1]
    assert t_sliced < t_whole


# ---- granularity left free (Section 3.3, last paragraph)

def _granularity_golden():
    rows = []
    with open(os.path.join(os.path.dirname(__file__), "golden", "plan_granularity_example.txt")) as f:
        for line in f:
            if line.startswith("best"):
                v = line.split()
                rows.append((float(v[1]), int(v[2]), int(v[3]), int(v[4]), float(v[5])))
    return rows


def test_hand_worked_granularity_instance():
    op = (8.0, 3.0, 0.0, 4.0, 10.0)
    rows = _granularity_golden()
    assert len(rows) == 2
    for alpha, k, dp, b, t in rows:
        ks, dps, bb, tt, _ = OP.search_granularity([op], [[(1, 0.0), (2, 0.02)]], 2, alpha, 1.0, 9.5, 8)
        assert (ks, dps, bb) == ([k], [dp], b)
        assert tt == pytest.approx(t, rel=1e-13)


def test_hand_worked_instance_with_the_gathered_slice_counted():
    op = (8.0, 3.0, 0.0, 4.0, 10.0)
    rows = []
    with open(os.path.join(os.path.dirname(__file__), "golden", "plan_granularity_example.txt")) as f:
        rows = [line.split()[1:] for line in f if line.startswith("surge")]
    assert len(rows) == 3
    for factor, limit, alpha, k, dp, b, t in rows:
        ks, dps, bb, tt, _ = OP.search_granularity([op], [[(1, 0.0), (2, 0.02)]], 2, float(alpha), 1.0, float(limit), 8,
                                                   surge_factor=float(factor))
        assert (ks, dps, bb) == ([int(k)], [int(dp)], int(b))
        assert tt == pytest.approx(float(t), rel=1e-13)


def test_one_whole_candidate_reduces_to_the_plain_search():
    rng = random.Random(77)
    for _ in range(20):
        n = rng.randint(1, 6)
        ops = [(rng.uniform(0, 100), rng.uniform(0, 9), rng.uniform(0, 3), rng.uniform(0, 50), rng.uniform(0.1, 2))
               for _ in range(n)]
        world, alpha, beta = rng.choice([2, 4, 8]), rng.uniform(0, 1), rng.uniform(0, 0.3)
        limit = rng.uniform(0.5, 1.2) * OP.memory_cost(ops, [0] * n, 2, world)
        modes, b, t, _ = OP.search(ops, world, alpha, beta, limit, 6)
        ks, dps, b2, t2, _ = OP.search_granularity(ops, [[(1, 0.0)]] * n, world, alpha, beta, limit, 6)
        assert b2 == b and t2 == t
        if b:
            assert ks == [1] * n and dps == [1 - m for m in modes]


def test_more_candidates_never_cost_more_and_latency_decides():
    op = (40.0, 2.0, 1.0, 20.0, 3.0)
    ops = [op, op]
    limit = OP.memory_cost(ops, [0, 1], 2, 4)            # room for one of the two in DP at b = 2, not both
    for alpha in (0.0, 0.5, 5.0):
        whole = OP.search_granularity(ops, [[(1, 0.0)]] * 2, 4, alpha, 0.1, limit, 3)
        free = OP.search_granularity(ops, [[(1, 0.0), (2, 0.0), (4, 0.0)]] * 2, 4, alpha, 0.1, limit, 3)
        assert free[3] <= whole[3] * (1 + 1e-15)
    # without latency, finer slices cost nothing; with a large latency per step every extra slice is a loss
    assert OP.search_granularity(ops, [[(1, 0.0), (4, 0.0)]] * 2, 4, 50.0, 0.1, limit, 3)[0] == [1, 1]
