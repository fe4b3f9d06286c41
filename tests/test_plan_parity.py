"""The library's plan search (osdp_plan_*: host code behind the C ABI) against the exhaustive oracle
(oracle/plan.py) on seeded random instances, and properties on instances too large to enumerate.
Where several plans share the optimal time, the time and batch size are compared and the returned
plan is checked to be feasible and to cost exactly that time.  CPU only."""
import random
import time

import pytest

from oracle import plan as OP


@pytest.fixture(scope="module")
def P():
    import paper_2209_13258_b200 as pkg
    pkg.lib()
    return pkg


def random_instance(rng, n):
    kinds = []
    for _ in range(rng.randint(1, 4)):      # a few operator shapes, repeated: duplicates exercise the grouping
        S = rng.choice([0.0, rng.uniform(1, 100)])
        states = S * rng.choice([1.0, 4.0, 8.0]) if rng.random() < 0.7 else rng.uniform(0, 300)
        kinds.append((states, rng.uniform(0, 20), rng.uniform(0, 5), S, rng.uniform(0.01, 3)))
    ops = [rng.choice(kinds) if rng.random() < 0.7 else
           (rng.uniform(0, 300), rng.uniform(0, 20), rng.uniform(0, 5), rng.uniform(0, 100), rng.uniform(0.01, 3))
           for _ in range(n)]
    world = rng.choice([1, 2, 3, 4, 8, 16])
    alpha, beta = rng.choice([0.0, rng.uniform(0, 2)]), rng.uniform(0, 0.5)
    lo = OP.memory_cost(ops, [1] * n, 1, world)
    hi = OP.memory_cost(ops, [0] * n, 4, world)
    limit = rng.uniform(0.8 * lo, 1.1 * hi)
    return ops, world, alpha, beta, limit


@pytest.mark.parametrize("seed", range(120))
def test_search_matches_exhaustive_enumeration(P, seed):
    rng = random.Random(1000 + seed)
    n = rng.randint(1, 11)
    ops, world, alpha, beta, limit = random_instance(rng, n)
    max_batch = rng.randint(1, 6)
    o_modes, o_b, o_t, _ = OP.search(ops, world, alpha, beta, limit, max_batch)
    rc, modes, b, t, nodes = P.osdp_plan_search(ops, world, alpha, beta, limit, max_batch)
    assert rc == 0
    if o_modes is None:
        assert b == 0 and t == float("inf")
        return
    assert b == o_b
    assert t == pytest.approx(o_t, rel=1e-12)
    # the plan itself: feasible and of exactly that cost, by the oracle's own pricing
    assert OP.memory_cost(ops, modes, b, world) <= limit
    assert OP.time_cost(ops, modes, b, world, alpha, beta) / b == pytest.approx(o_t, rel=1e-12)


def test_plan_cost_matches_oracle(P):
    rng = random.Random(77)
    for _ in range(200):
        n = rng.randint(1, 20)
        ops, world, alpha, beta, _ = random_instance(rng, n)
        modes = [rng.randint(0, 1) for _ in range(n)]
        b = rng.randint(1, 9)
        rc, m, t = P.osdp_plan_cost(ops, world, alpha, beta, modes, b)
        assert rc == 0
        assert m == pytest.approx(OP.memory_cost(ops, modes, b, world), rel=1e-14)
        assert t == pytest.approx(OP.time_cost(ops, modes, b, world, alpha, beta), rel=1e-14)


def test_hand_worked_instance(P):
    A, B = (40.0, 5.0, 2.0, 8.0, 3.0), (24.0, 10.0, 1.0, 16.0, 2.0)
    assert P.osdp_plan_search([A, B], 4, 1.0, 0.5, 100.0, 50)[:4] == (0, (1, 0), 4, 14.0)
    assert P.osdp_plan_cost([A, B], 4, 1.0, 0.5, (1, 0), 4) == (0, 97.0, 56.0)


def test_expand_slices_matches_oracle(P):
    op = (64.0, 8.0, 4.0, 32.0, 2.0)
    for k, ov in ((1, 0.0), (4, 0.25), (7, 0.1)):
        rc, sl = P.osdp_plan_expand_slices(op, k, ov)
        assert rc == 0 and len(sl) == k
        for a, b in zip(sl, OP.expand_slices(op, k, ov)):
            assert a == pytest.approx(b, rel=1e-15)
    assert P.osdp_plan_expand_slices(op, 0)[0] == 3 and P.osdp_plan_expand_slices(op, 2, -1.0)[0] == 2


def gpt_layers(layers, hidden, bytes_per_param_state=16.0):
    """Four linears per layer (QKV, out-projection, two MLP layers), states = 16 bytes per parameter
    (fp32 master weights, Adam moments, bf16 weights and gradients), bf16 parameters on the wire."""
    ops = []
    for _ in range(layers):
        for n_out, n_in in ((3 * hidden, hidden), (hidden, hidden), (4 * hidden, hidden), (hidden, 4 * hidden)):
            params = float(n_out * n_in)
            ops.append((params * bytes_per_param_state, 2.0 * 1024 * (n_in + n_out), 0.0, 2.0 * params,
                        6.0 * 1024 * params / 1.2e15))
    return ops


def test_transformer_sized_instance_is_solved_exactly_and_fast(P):
    ops = gpt_layers(24, 2048)
    world, alpha, beta = 8, 10e-6, 1 / 400e9
    dp = OP.memory_cost(ops, [0] * len(ops), 1, world)
    zdp = OP.memory_cost(ops, [1] * len(ops), 1, world)
    limit = zdp + 0.37 * (dp - zdp)
    t0 = time.time()
    rc, modes, b, t, nodes = P.osdp_plan_search(ops, world, alpha, beta, limit, 64)
    assert rc == 0 and b >= 1 and time.time() - t0 < 20.0
    assert OP.memory_cost(ops, modes, b, world) <= limit
    assert OP.time_cost(ops, modes, b, world, alpha, beta) / b == pytest.approx(t, rel=1e-12)
    # optimality at the chosen batch size: no single switch to DP fits, and no swap of one DP operator for a
    # ZDP one that saves more time fits either (necessary conditions the exact answer must satisfy)
    mem = OP.memory_cost(ops, modes, b, world)
    w = [op[0] * (1 - 1 / world) for op in ops]
    c = [(world - 1) * (alpha + op[3] / world * beta) for op in ops]
    for i, m in enumerate(modes):
        if m == 1:
            assert mem + w[i] > limit or c[i] == 0.0
            for j, mj in enumerate(modes):
                if mj == 0 and c[i] > c[j] * (1 + 1e-12):
                    assert mem + w[i] - w[j] > limit
    # Planning slice by slice: every slice pays the per-step latency alpha of its own collectives, so with
    # alpha = 0 it can only help (every whole-operator plan is still available), and with alpha > 0 it can
    # cost at most the added latency of the whole-operator plan lifted to slices.
    sliced = [s for op in ops for s in OP.expand_slices(op, 4)]
    rc, _, b0, t0_, _ = P.osdp_plan_search(ops, world, 0.0, beta, limit, 64)
    rc4, modes4, b4, t4, _ = P.osdp_plan_search(sliced, world, 0.0, beta, limit, 64)
    assert rc == 0 and rc4 == 0 and t4 <= t0_ * (1 + 1e-12)
    assert OP.memory_cost(sliced, modes4, b4, world) <= limit
    rc4, modes4, b4, t4, _ = P.osdp_plan_search(sliced, world, alpha, beta, limit, 64)
    lifted = [m for m in modes for _ in range(4)]
    assert rc4 == 0 and t4 <= OP.time_cost(sliced, lifted, b, world, alpha, beta) / b * (1 + 1e-12)


def test_node_budget_is_reported_and_the_plan_still_fits(P):
    rng = random.Random(3)
    ops = [(rng.uniform(10, 20), 1.0, 0.0, rng.uniform(10, 20), 1.0) for _ in range(40)]
    world = 4
    limit = OP.memory_cost(ops, [1] * 40, 1, world) + 123.4
    rc, modes, b, t, nodes = P.osdp_plan_search(ops, world, 0.0, 1.0, limit, 1, max_nodes=50)
    assert rc == 10 and b == 1
    assert OP.memory_cost(ops, modes, 1, world) <= limit
    rc2, _, _, t2, _ = P.osdp_plan_search(ops, world, 0.0, 1.0, limit, 1)
    assert rc2 == 0 and t2 <= t


def test_argument_errors(P):
    A = (40.0, 5.0, 2.0, 8.0, 3.0)
    assert P.osdp_plan_search([A], 0, 1.0, 0.5, 100.0, 5)[0] == 2            # world < 1
    assert P.osdp_plan_search([A], 2, -1.0, 0.5, 100.0, 5)[0] == 2           # negative latency
    assert P.osdp_plan_search([A], 2, 1.0, 0.5, 100.0, 0)[0] == 2            # no batch size to try
    assert P.osdp_plan_search([(1.0, 1.0, float("nan"), 1.0, 1.0)], 2, 1.0, 0.5, 100.0, 5)[0] == 2
    assert P.osdp_plan_cost([A], 2, 1.0, 0.5, (0,), 0)[0] == 2
    assert P.lib().osdp_plan_search(None, 1, 2, 1.0, 0.5, 100.0, 5, 0, None, None, None, None) == 1


# ---- granularity left free (osdp_plan_search_granularity)

def _priced(ops, ks, dps, ovh_of, b, world, alpha, beta):
    """Memory and time of a (granularity, DP count) assignment, priced by the oracle on the expanded slices."""
    expanded, modes = [], []
    for op, k, dp, i in zip(ops, ks, dps, range(len(ops))):
        expanded += OP.expand_slices(op, k, ovh_of(i, k))
        modes += [0] * dp + [1] * (k - dp)
    return OP.memory_cost(expanded, modes, b, world), OP.time_cost(expanded, modes, b, world, alpha, beta)


@pytest.mark.parametrize("seed", range(60))
def test_granularity_search_matches_exhaustive_enumeration(P, seed):
    rng = random.Random(5000 + seed)
    n = rng.randint(1, 3)
    kinds = [(rng.uniform(5, 200), rng.uniform(0, 20), rng.uniform(0, 5), rng.uniform(1, 100), rng.uniform(0.05, 3))
             for _ in range(2)]
    ops = [rng.choice(kinds) for _ in range(n)]
    pool = [(1, 0.0), (2, rng.uniform(0, 0.1)), (3, rng.uniform(0, 0.2)), (4, rng.uniform(0, 0.3))]
    shared = sorted(rng.sample(pool, rng.randint(1, 3)))
    cands = [shared if rng.random() < 0.6 else sorted(rng.sample(pool, rng.randint(1, 3))) for _ in range(n)]
    world = rng.choice([2, 3, 4, 8])
    alpha, beta = rng.choice([0.0, rng.uniform(0, 1.5)]), rng.uniform(0, 0.5)
    lo = OP.memory_cost(ops, [1] * n, 1, world)
    hi = OP.memory_cost(ops, [0] * n, 3, world)
    limit = rng.uniform(0.9 * lo, 1.05 * hi)
    factor = rng.choice([0.0, 0.0, 1.0, 2.0, rng.uniform(0, 3)])
    ks_o, dps_o, b_o, t_o, _ = OP.search_granularity(ops, cands, world, alpha, beta, limit, 4, surge_factor=factor)
    rc, ks, dps, b, t, nodes = P.osdp_plan_search_granularity(ops, cands, world, alpha, beta, limit, 4,
                                                              surge_factor=factor)
    assert rc == 0 and b == b_o
    if b_o == 0:
        assert t == float("inf")
        return
    assert t == pytest.approx(t_o, rel=1e-12)
    ovh = lambda i, k: dict(cands[i])[k]
    assert all(k in dict(c) for k, c in zip(ks, cands)) and all(0 <= d <= k for d, k in zip(dps, ks))
    mem, tt = _priced(ops, ks, dps, ovh, b, world, alpha, beta)
    surge = max([op[3] / k for op, k, d in zip(ops, ks, dps) if d < k] + [0.0])
    assert mem + factor * surge <= limit * (1 + 1e-12) and tt / b == pytest.approx(t, rel=1e-12)


def test_granularity_hand_worked_instance(P):
    op = (8.0, 3.0, 0.0, 4.0, 10.0)
    assert P.osdp_plan_search_granularity([op], [[(1, 0.0), (2, 0.02)]], 2, 0.25, 1.0, 9.5, 8)[:5] == \
        (0, [2], [1], 1, pytest.approx(16.45, rel=1e-13))
    assert P.osdp_plan_search_granularity([op], [[(1, 0.0), (2, 0.02)]], 2, 1.0, 1.0, 9.5, 8)[:5] == \
        (0, [1], [0], 1, pytest.approx(19.0, rel=1e-13))
    for limit, want in ((9.5, ([2], [0], 1, 17.7)), (11.0, ([1], [1], 1, 14.5)), (10.5, ([2], [0], 1, 17.7))):
        got = P.osdp_plan_search_granularity([op], [[(1, 0.0), (2, 0.02)]], 2, 0.25, 1.0, limit, 8, surge_factor=1.0)
        assert got[0] == 0 and tuple(got[1:4]) == want[:3] and got[4] == pytest.approx(want[3], rel=1e-13)


def test_granularity_with_whole_operators_only_is_the_plain_search(P):
    rng = random.Random(11)
    for _ in range(30):
        ops, world, alpha, beta, limit = random_instance(rng, rng.randint(1, 12))
        rc, modes, b, t, _ = P.osdp_plan_search(ops, world, alpha, beta, limit, 8)
        rc2, ks, dps, b2, t2, _ = P.osdp_plan_search_granularity(ops, [[(1, 0.0)]] * len(ops), world, alpha, beta,
                                                                 limit, 8)
        assert rc == 0 and rc2 == 0 and b2 == b
        if b:
            assert t2 == pytest.approx(t, rel=1e-12) and ks == [1] * len(ops)


def test_granularity_on_a_transformer_sized_instance(P):
    ops = gpt_layers(24, 2048)
    world, alpha, beta = 8, 10e-6, 1 / 400e9
    dp = OP.memory_cost(ops, [0] * len(ops), 1, world)
    zdp = OP.memory_cost(ops, [1] * len(ops), 1, world)
    limit = zdp + 0.37 * (dp - zdp)
    cands = [[(1, 0.0), (2, 0.01), (4, 0.03), (8, 0.08)]] * len(ops)
    t0 = time.time()
    rc, ks, dps, b, t, nodes = P.osdp_plan_search_granularity(ops, cands, world, alpha, beta, limit, 64)
    assert rc in (0, 10) and b >= 1 and time.time() - t0 < 60.0
    mem, tt = _priced(ops, ks, dps, lambda i, k: dict(cands[i])[k], b, world, alpha, beta)
    assert mem <= limit * (1 + 1e-12) and tt / b == pytest.approx(t, rel=1e-12)
    # the whole-operator plan is among the candidates: leaving the granularity free cannot cost more
    rc1, _, b1, t1, _ = P.osdp_plan_search(ops, world, alpha, beta, limit, 64)
    assert rc1 == 0 and (rc != 0 or t <= t1 * (1 + 1e-12))
    # without latency and overhead, finer slices only add choices: at least as good as the uniform k = 4 plan
    free = [[(1, 0.0), (4, 0.0)]] * len(ops)
    sliced = [s for op in ops for s in OP.expand_slices(op, 4)]
    rc4, _, _, t4, _ = P.osdp_plan_search(sliced, world, 0.0, beta, limit, 64)
    rcf, _, _, _, tf, _ = P.osdp_plan_search_granularity(ops, free, world, 0.0, beta, limit, 64)
    assert rc4 == 0 and (rcf != 0 or tf <= t4 * (1 + 1e-12))


def test_granularity_node_budget_and_argument_errors(P):
    rng = random.Random(4)
    ops = [(rng.uniform(10, 20), 1.0, 0.0, rng.uniform(10, 20), 1.0) for _ in range(30)]
    cands = [[(1, 0.0), (2, 0.0), (4, 0.01)]] * 30
    limit = OP.memory_cost(ops, [1] * 30, 1, 4) + 77.7
    rc, ks, dps, b, t, nodes = P.osdp_plan_search_granularity(ops, cands, 4, 0.0, 1.0, limit, 1, max_nodes=40)
    assert rc == 10 and b == 1
    mem, _ = _priced(ops, ks, dps, lambda i, k: dict(cands[i])[k], 1, 4, 0.0, 1.0)
    assert mem <= limit * (1 + 1e-12)
    A = (40.0, 5.0, 2.0, 8.0, 3.0)
    assert P.osdp_plan_search_granularity([A], [[]], 2, 1.0, 0.5, 100.0, 5)[0] == 2          # no candidate
    assert P.osdp_plan_search_granularity([A], [[(0, 0.0)]], 2, 1.0, 0.5, 100.0, 5)[0] == 3   # k < 1
    assert P.osdp_plan_search_granularity([A], [[(2, -1.0)]], 2, 1.0, 0.5, 100.0, 5)[0] == 2  # overhead <= -1
    assert P.osdp_plan_search_granularity([A], [[(1, 0.0)]], 0, 1.0, 0.5, 100.0, 5)[0] == 2   # world < 1
    assert P.osdp_plan_search_granularity([A], [[(1, 0.0)]], 2, 1.0, 0.5, 1.0, 5)[3] == 0     # nothing fits
    assert P.osdp_plan_search_granularity([A], [[(1, 0.0)]], 2, 1.0, 0.5, 100.0, 5, surge_factor=-1.0)[0] == 2
