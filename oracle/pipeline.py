"""Exact-integer oracle for the 1F1B pipeline timing model (TEST INFRASTRUCTURE ONLY).

Only the tests, the smoke entry and the benchmark's cpu_baseline / reference
legs may import this; it shares no code with the C++ simulator in the library.

The paper evaluates KV-Pipe under the non-interleaved 1F1B schedule (section
"Results on Ascend 910B NPUs": "1F1B pipeline schedule (no interleaving)") and
argues that the iteration time follows the stage imbalance FIR (Eq. 4-5).  It
prints no timing model, so this file restates the schedule itself, the one of
the works the paper cites for 1F1B, as a dependency graph and takes the
iteration time to be the graph's longest path:

* Stage i of P (0-based) runs w_i = min(P - 1 - i, M) warm-up forwards, then
  alternates one forward and one backward until all M forwards are done, then
  drains the remaining backwards; every stage executes its operations strictly
  in that order.
* Forward of micro-batch m on stage i needs the forward of m on stage i - 1;
  backward of m on stage i needs the backward of m on stage i + 1 (on the last
  stage: its own forward of m).  Transfers cost nothing.
* An operation starts when its predecessors have finished; the iteration time
  (makespan) is the finish time of the last operation.

Times are integers (any unit), so every result is exact.  The longest path is
computed by memoised recursion over the graph as defined above: there is no
event loop, no per-stage program counter and no closed form in here.

Pins (tests/test_oracle_pipeline.py): the closed form (M + P - 1)(t_f + t_b)
for equal stages, P = 1, M = 1, the critical-path lower bounds, monotonicity,
a hand-traced 2-stage / 3-micro-batch case, and a second, independently
written event-driven evaluation on random small cases.
"""
from __future__ import annotations

import sys
from functools import lru_cache


def stage_order(P, M, i):
    """Operations of stage i in execution order: list of ('F' | 'B', micro-batch)."""
    warm = min(P - 1 - i, M)
    ops = [("F", m) for m in range(warm)]
    for k in range(M - warm):
        ops.append(("F", warm + k))
        ops.append(("B", k))
    ops += [("B", m) for m in range(M - warm, M)]
    return ops


def sim_1f1b(tf, tb, M):
    """Iteration time of the 1F1B schedule with per-stage forward times tf[i] and backward times tb[i]
    (integers) over M micro-batches.  Returns (makespan, idle) where idle[i] = makespan - M*(tf[i]+tb[i])
    is the time stage i spends not computing (its pipeline bubble)."""
    P = len(tf)
    assert len(tb) == P and P >= 1 and M >= 1
    orders = [stage_order(P, M, i) for i in range(P)]
    pos = [{op: n for n, op in enumerate(orders[i])} for i in range(P)]
    sys.setrecursionlimit(max(10000, 8 * P * M + 1000))

    @lru_cache(maxsize=None)
    def finish(i, kind, m):
        start = 0
        n = pos[i][(kind, m)]
        if n > 0:                                   # the stage runs its operations in order
            pk, pm = orders[i][n - 1]
            start = max(start, finish(i, pk, pm))
        if kind == "F":
            if i > 0:
                start = max(start, finish(i - 1, "F", m))
            return start + tf[i]
        if i + 1 < P:
            start = max(start, finish(i + 1, "B", m))
        else:
            start = max(start, finish(i, "F", m))
        return start + tb[i]

    makespan = max(finish(i, *orders[i][-1]) for i in range(P))
    idle = [makespan - M * (tf[i] + tb[i]) for i in range(P)]
    return makespan, idle


def bubble_fraction(tf, tb, M):
    """Share of the P * makespan stage-time budget in which stages idle, as an exact fraction (num, den)."""
    makespan, idle = sim_1f1b(tf, tb, M)
    return sum(idle), len(tf) * makespan
