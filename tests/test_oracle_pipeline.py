"""Pins for the 1F1B timing oracle (oracle/pipeline.py): closed forms, a hand trace, bounds, and an
independently written event-driven evaluation of the same schedule."""
import random

import pytest

from oracle import pipeline as PL


def event_driven(tf, tb, M):
    """Second opinion, written without looking at the oracle's recursion: every stage keeps a program counter
    into its operation list and a clock; an operation is executed as soon as its remote input exists."""
    P = len(tf)
    orders = [PL.stage_order(P, M, i) for i in range(P)]
    pc = [0] * P
    clock = [0] * P
    done = {}
    remaining = sum(len(o) for o in orders)
    while remaining:
        progressed = False
        for i in range(P):
            while pc[i] < len(orders[i]):
                kind, m = orders[i][pc[i]]
                if kind == "F":
                    dep = (i - 1, "F", m) if i > 0 else None
                else:
                    dep = (i + 1, "B", m) if i + 1 < P else (i, "F", m)
                if dep is not None and dep not in done:
                    break
                start = max(clock[i], done[dep] if dep is not None else 0)
                clock[i] = start + (tf[i] if kind == "F" else tb[i])
                done[(i, kind, m)] = clock[i]
                pc[i] += 1
                remaining -= 1
                progressed = True
        assert progressed, "schedule deadlocked"
    return max(clock)


def test_stage_order_counts_and_warmup():
    P, M = 4, 6
    for i in range(P):
        ops = PL.stage_order(P, M, i)
        assert sorted(m for k, m in ops if k == "F") == list(range(M))
        assert sorted(m for k, m in ops if k == "B") == list(range(M))
        warm = 0
        while ops[warm][0] == "F":
            warm += 1
        # the forward that opens the first 1F1B pair follows the warm-up forwards directly
        assert warm == min(P - 1 - i, M) + (1 if P - 1 - i < M else 0)
    # more stages than micro-batches: the early stages run all forwards first
    assert PL.stage_order(8, 2, 0) == [("F", 0), ("F", 1), ("B", 0), ("B", 1)]


def test_hand_trace_two_stages_three_microbatches():
    # stage 0: F0 0-2, F1 2-4, B0 10-14, F2 14-16, B1 18-22, B2 26-30
    # stage 1: F0 2-5, B0 5-10, F1 10-13, B1 13-18, F2 18-21, B2 21-26
    makespan, idle = PL.sim_1f1b([2, 3], [4, 5], 3)
    assert makespan == 30
    assert idle == [30 - 3 * 6, 30 - 3 * 8]
    assert PL.bubble_fraction([2, 3], [4, 5], 3) == (18, 60)


@pytest.mark.parametrize("P,M,tf,tb", [(1, 5, 7, 9), (2, 4, 3, 6), (4, 8, 5, 10), (8, 8, 11, 23), (8, 32, 1, 2),
                                       (6, 3, 4, 4)])
def test_equal_stages_closed_form(P, M, tf, tb):
    makespan, idle = PL.sim_1f1b([tf] * P, [tb] * P, M)
    assert makespan == (M + P - 1) * (tf + tb)
    assert idle == [(P - 1) * (tf + tb)] * P
    num, den = PL.bubble_fraction([tf] * P, [tb] * P, M)
    assert num * (M + P - 1) == den * (P - 1)          # the textbook bubble share (P-1)/(M+P-1)


def test_single_stage_and_single_microbatch():
    assert PL.sim_1f1b([5], [8], 7)[0] == 7 * 13
    tf, tb = [3, 1, 4, 1, 5], [9, 2, 6, 5, 3]
    assert PL.sim_1f1b(tf, tb, 1)[0] == sum(tf) + sum(tb)


def test_dominant_stage_closed_form():
    # a stage that is slower than every other in both directions is never starved once it has started:
    # fill (forwards before it) + M of its own F+B + drain (backwards before it)
    tf, tb, M = [2, 3, 20, 2], [4, 5, 40, 3], 6
    b = 2
    expect = sum(tf[:b]) + M * (tf[b] + tb[b]) + sum(tb[:b])
    assert PL.sim_1f1b(tf, tb, M)[0] == expect
    # heavy LAST stage (the LM-head case the paper is about)
    tf, tb, M = [10, 10, 10, 13], [20, 20, 20, 26], 8
    assert PL.sim_1f1b(tf, tb, M)[0] == 30 + 8 * 39 + 60


def test_bounds_monotonicity_and_second_opinion():
    rng = random.Random(1234)
    for _ in range(200):
        P = rng.randint(1, 6)
        M = rng.randint(1, 7)
        tf = [rng.randint(1, 20) for _ in range(P)]
        tb = [rng.randint(1, 40) for _ in range(P)]
        makespan, idle = PL.sim_1f1b(tf, tb, M)
        assert makespan == event_driven(tf, tb, M)
        assert makespan >= M * max(a + b for a, b in zip(tf, tb))
        assert makespan >= sum(tf) + sum(tb)
        for b in range(P):
            assert makespan >= sum(tf[:b]) + M * (tf[b] + tb[b]) + sum(tb[:b])
        assert all(x >= 0 for x in idle)
        i = rng.randrange(P)
        tf2 = list(tf)
        tf2[i] += rng.randint(1, 5)
        assert PL.sim_1f1b(tf2, tb, M)[0] >= makespan
        # scaling every time by c scales the makespan by c
        assert PL.sim_1f1b([3 * x for x in tf], [3 * x for x in tb], M)[0] == 3 * makespan


def test_balancing_the_tail_stage_shortens_the_iteration():
    # the paper's setting: the last stage carries the LM head; lightening it towards the average lowers the
    # iteration time by M times the saving; over-lightening it only shortens the fill/drain path (the other
    # stages are the bottleneck by then)
    base_f, base_b, M = 100, 200, 16
    times = []
    for tail_extra in (36, 18, 0, -18):
        tf = [base_f] * 7 + [base_f + tail_extra]
        tb = [base_b] * 7 + [base_b + 2 * tail_extra]
        times.append(PL.sim_1f1b(tf, tb, M)[0])
    assert times[0] - times[1] == M * 54 and times[1] - times[2] == M * 54
    assert 0 <= times[2] - times[3] <= 2 * 54
