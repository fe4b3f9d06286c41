"""Oracle of the execution-plan search (Section 3.1 problem formulation, Algorithm 1).  TEST
INFRASTRUCTURE ONLY: imported by tests alone; shares no code with the library's planner.

Plain Python, fp64, exhaustive: every plan in {DP, ZDP}^n is priced with the paper's memory
and time model and the cheapest feasible one is kept, batch size by batch size, exactly in the
order of Algorithm 1.  No pruning, no bounds, no reordering.  Usable up to n of about 16.

An operator is a tuple (model, act, extra, S, gamma):
    model  M_i^(model)  bytes of model states (parameters and optimiser states)
    act    M_i^(act)    activation bytes per sample
    extra  M_i^(extra)  other bytes (temporary workspace)
    S      S_i          bytes of the operator's parameters (what the collectives move)
    gamma  gamma_i      computation time per sample
A mode is 0 (DP) or 1 (ZDP).
"""
from __future__ import annotations

import itertools

DP, ZDP = 0, 1


def memory_cost(ops, modes, b, world):
    """M(p, b) = sum_i M_i(p_i, b), Section 3.1: ZDP keeps 1/N of the model states."""
    total = 0.0
    for (model, act, extra, _S, _gamma), p in zip(ops, modes):
        states = model / world if p == ZDP else model
        total += states + b * act + extra
    return total


def time_cost(ops, modes, b, world, alpha, beta):
    """sum_i T_i(p_i, b), Section 3.1: ring collectives of N - 1 steps moving S_i / N each; DP runs two
    of them per operator (reduce-scatter + all-gather), ZDP three; computation b * gamma_i."""
    total = 0.0
    for (_model, _act, _extra, S, gamma), p in zip(ops, modes):
        collectives = 3 if p == ZDP else 2
        total += collectives * (world - 1) * (alpha + S / world * beta) + b * gamma
    return total


def best_plan_for_batch(ops, b, world, alpha, beta, mem_limit):
    """Inner loop of Algorithm 1: the feasible plan of least time for one batch size, or None."""
    best_t, best_p = float("inf"), None
    for modes in itertools.product((DP, ZDP), repeat=len(ops)):
        m = memory_cost(ops, modes, b, world)
        t = time_cost(ops, modes, b, world, alpha, beta)
        if m <= mem_limit and t < best_t:
            best_t, best_p = t, modes
    return best_t, best_p


def search(ops, world, alpha, beta, mem_limit, max_batch):
    """Algorithm 1.  Batch sizes 1, 2, 3, ... until no plan fits (or max_batch, which the paper's loop
    does not have: it keeps the loop finite when memory never runs out).  Returns
    (modes, b, time per sample, candidates) with candidates = [(T*(b) / b, modes, b), ...];
    (None, 0, inf, []) if nothing fits at b = 1.  The objective is T(p, b) = (1/b) sum_i T_i(p_i, b)."""
    candidates = []
    for b in range(1, max_batch + 1):
        t, modes = best_plan_for_batch(ops, b, world, alpha, beta, mem_limit)
        if modes is None:
            break
        candidates.append((t / b, modes, b))
    if not candidates:
        return None, 0, float("inf"), []
    best = candidates[0]
    for c in candidates[1:]:
        if c[0] < best[0]:
            best = c
    return best[1], best[2], best[0], candidates


def expand_slices(op, k, overhead=0.0):
    """Section 3.3, last paragraph: an operator cut into k slices is planned slice by slice.  Every
    slice carries 1/k of the operator's bytes and of its computation, the computation inflated by
    the measured relative time overhead of running the operator split k ways."""
    model, act, extra, S, gamma = op
    return [(model / k, act / k, extra / k, S / k, gamma * (1.0 + overhead) / k) for _ in range(k)]


def search_granularity(ops, candidates, world, alpha, beta, mem_limit, max_batch, surge_factor=0.0):
    """Section 3.3, last paragraph, with the slice granularity of every operator left free as well (the
    paper takes it as given): candidates[i] lists the (k, overhead) pairs allowed for operator i.  For
    each batch size of Algorithm 1 every combination of granularities is tried, each operator replaced by
    its slices (expand_slices) and every assignment of DP / ZDP to the slices priced.

    surge_factor: Section 3.3 describes the gathered parameters of a ZDP operator as a memory surge that
    splitting cuts from size(operator) to size(operator) / granularity; the sums of Section 3.1 have no
    term for it.  Here the largest gathered slice S_i / k_i among the operators with at least one ZDP
    slice, times surge_factor, is added to the memory a plan needs (0: the paper's model as it stands).

    Returns (ks, dp_counts, b, time per sample, per_batch): ks[i] the granularity chosen for operator i,
    dp_counts[i] how many of its slices run in DP; (None, None, 0, inf, []) if nothing fits at b = 1.
    Tiny instances only: the work is prod_i |candidates[i]| * 2^(sum of k)."""
    per_batch = []
    for b in range(1, max_batch + 1):
        best = None
        for choice in itertools.product(*candidates):
            expanded, owner = [], []
            for i, (op, (k, overhead)) in enumerate(zip(ops, choice)):
                expanded += expand_slices(op, k, overhead)
                owner += [i] * k
            for modes in itertools.product((DP, ZDP), repeat=len(expanded)):
                surge = 0.0
                for i, p in zip(owner, modes):
                    if p == ZDP:
                        surge = max(surge, ops[i][3] / choice[i][0])
                m = memory_cost(expanded, modes, b, world) + surge_factor * surge
                t = time_cost(expanded, modes, b, world, alpha, beta)
                if m <= mem_limit and (best is None or t < best[0]):
                    dp = [0] * len(ops)
                    for i, p in zip(owner, modes):
                        dp[i] += 1 if p == DP else 0
                    best = (t, [k for k, _ in choice], dp)
        if best is None:
            break
        per_batch.append((best[0] / b, best[1], best[2], b))
    if not per_batch:
        return None, None, 0, float("inf"), []
    top = per_batch[0]
    for c in per_batch[1:]:
        if c[0] < top[0]:
            top = c
    return top[1], top[2], top[3], top[0], per_batch
