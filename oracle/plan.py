"""Exact-integer oracle for the offline planner (TEST INFRASTRUCTURE ONLY).

Only the tests, the smoke entry and the benchmark's cpu_baseline / reference
legs may import this; it shares no code with the C++ planner in the library.

It restates, in Python integers (arbitrary precision, so no rounding anywhere):

* Eq. 4-5  FIR = max_i F_stage_i / F_avg, F_avg the mean over the P stages of
           the stage totals, the LM head counted on the last stage.  Kept as the
           exact rational (max_i F_i * P) / (sum_i F_i).
* Eq. 6-7  stage totals under a conversion mask z and the budget sum z <= m.
* Algorithm 1 (Architecture-Balanced KV-Pipe): start at the tail stage; once
  the tail is within (1+eps) of the average retarget to the arg-max stage;
  convert the deepest unconverted layer of the chosen stage; stop on
  FIR <= 1+eps, on the budget, or when the chosen stage has no convertible
  layer.  The state is the set of converted layers and every quantity is
  recomputed from Eq. 4-7 each round.
* Appendix "Optional Safe-Layer Guardrail": only layers with (1-indexed)
  l >= ceil(alpha L) are admissible.
* Appendix "Attention FLOPs under MHA and GQA": per-token forward FLOPs and the
  saving 4 h^2 / r of a converted layer.
* The Uniform and Symmetric-Bipolar placements of the stage tables in the
  appendix "Stage-level splits".  The paper gives each a sentence and one
  stage table (m = 4, P = 8); how they continue beyond that instance (more
  conversions than stages, a full stage) is this build's definition.

Readings where the paper is silent (each is also a documented reading of the
library): tau(l) is the nearest preceding unconverted layer; global layer 0 is
never convertible; arg-max ties go to the highest stage index; an optional
"stop when FIR does not strictly improve" rule reverts the tentative
conversion; an optional rule keeps the first layer of every stage unconverted
so every donor lives on the consumer's stage.

Pins (tests/test_oracle_plan.py): the FIR values and selected layers the paper
prints (tests/golden/plan_pins.txt), hand traces, and exhaustive search over
all conversion subsets on small layer counts.
"""
from __future__ import annotations

from itertools import combinations

STOP_TOLERANCE = 0      # FIR <= 1 + eps reached
STOP_BUDGET = 1         # t == m
STOP_EXHAUSTED = 2      # chosen stage has no admissible unconverted layer
STOP_NO_IMPROVE = 3     # optional rule: conversion would not lower FIR


def layer_flops(h, f, a, g, dh, s, vocab, causal_half=True):
    """Per-token forward FLOPs (a MAC counts 2) of one decoder layer.

    Attention part from the appendix' per-token totals: Q and output projections
    2*h*(a*dh) each, K and V projections 2*h*(g*dh) each (together 4h^2/r when
    a*dh = h), scores and weighted sum 2*s*(a*dh) each -- halved under the
    causal mask when causal_half is set, which is the count that reproduces the
    paper's printed baseline FIR -- plus a gated MLP 6*h*f.  Returns
    (F_full, F_share, F_lm_head) with F_share = F_full - 4*h*(g*dh) and
    F_lm_head = 2*h*vocab."""
    qd, kvd = a * dh, g * dh
    attn_scores = (2 if causal_half else 4) * s * qd
    f_full = 2 * h * qd + 4 * h * kvd + 2 * qd * h + attn_scores + 6 * h * f
    f_share = f_full - 4 * h * kvd
    return f_full, f_share, 2 * h * vocab


def stage_totals(stage_begin, f_full, f_share, stage_extra, z):
    """Eq. 6: F_stage_i(z) = sum_{l in S_i} F_l(z_l) + extra_i (LM head on the tail)."""
    P = len(stage_begin) - 1
    out = []
    for i in range(P):
        t = stage_extra[i]
        for l in range(stage_begin[i], stage_begin[i + 1]):
            t += f_share[l] if z[l] else f_full[l]
        out.append(t)
    return out


def fir_rational(stage):
    """Eq. 4-5 as an exact fraction (numerator, denominator) = (max*P, sum)."""
    return max(stage) * len(stage), sum(stage)


def donor_from_z(z):
    """tau(l): nearest preceding layer with z = 0 (an owner); owners map to themselves."""
    donor, last = [], -1
    for l, zl in enumerate(z):
        if not zl:
            last = l
        if last < 0:
            raise ValueError("layer 0 cannot be a KV-sharing layer")
        donor.append(last)
    return donor


def _admissible(l, stage_begin, i, L, alpha, stage_local_donor):
    if l == 0:
        return False
    if stage_local_donor and l == stage_begin[i]:
        return False
    if alpha is not None and alpha[0] > 0:
        num, den = alpha
        need = -((-num * L) // den)          # ceil(alpha * L), 1-indexed threshold
        if l + 1 < need:
            return False
    return True


def kvp_plan(stage_begin, f_full, f_share, stage_extra, eps=(0, 1), max_conv=0,
             stop_on_no_improve=False, stage_local_donor=False, alpha=None):
    """Algorithm 1 (Architecture-Balanced KV-Pipe).  eps = (num, den) rational; max_conv 0 means L.

    Stated through the paper's definitions rather than through incremental bookkeeping: the state is the SET of
    converted layers; every round recomputes the stage totals of that set from Eq. 6 and the imbalance from
    Eq. 4-5, then
      * stops if FIR <= 1 + eps, or if the budget sum z = m of Eq. 7 is spent;
      * targets the tail stage while the tail is still heavier than (1 + eps) times the average stage, and
        otherwise the heaviest stage (the deepest one among equals);
      * converts the deepest layer of the target stage that is still unconverted and admissible, or stops if
        there is none;
      * under the optional no-improve rule, keeps the conversion only if the FIR of the enlarged set is strictly
        smaller.
    All comparisons are between exact integer cross-products.

    Returns dict(z, donor, stage, fir_num, fir_den, n_conv, stop_reason)."""
    P = len(stage_begin) - 1
    L = stage_begin[P]
    budget = max_conv if max_conv else L
    en, ed = eps

    def totals(converted):
        return stage_totals(stage_begin, f_full, f_share, stage_extra, [int(l in converted) for l in range(L)])

    def above_tolerance(value_times_p, total):        # value / (total / P) > 1 + eps
        return value_times_p * ed > (ed + en) * total

    converted = set()
    while True:
        stage = totals(converted)
        num, den = fir_rational(stage)
        if not above_tolerance(num, den):
            reason = STOP_TOLERANCE
            break
        if len(converted) >= budget:
            reason = STOP_BUDGET
            break
        if above_tolerance(stage[P - 1] * P, den):
            target = P - 1
        else:
            target = max(range(P), key=lambda j: (stage[j], j))
        pool = {l for l in range(stage_begin[target], stage_begin[target + 1])
                if l not in converted and _admissible(l, stage_begin, target, L, alpha, stage_local_donor)}
        if not pool:
            reason = STOP_EXHAUSTED
            break
        pick = max(pool)
        if stop_on_no_improve:
            num_after, den_after = fir_rational(totals(converted | {pick}))
            if not (num_after * den < num * den_after):
                reason = STOP_NO_IMPROVE
                break
        converted.add(pick)
    z = [int(l in converted) for l in range(L)]
    stage = totals(converted)
    num, den = fir_rational(stage)
    return dict(z=z, donor=donor_from_z(z), stage=stage, fir_num=num, fir_den=den,
                n_conv=len(converted), stop_reason=reason)


def exhaustive_min_fir(stage_begin, f_full, f_share, stage_extra, max_conv=0):
    """Brute force over every subset of layers 1..L-1 (size <= max_conv):
    the smallest FIR, as a fraction, and one subset reaching it."""
    P = len(stage_begin) - 1
    L = stage_begin[P]
    m = max_conv if max_conv else L - 1
    best = None
    for k in range(0, m + 1):
        for sub in combinations(range(1, L), k):
            z = [0] * L
            for l in sub:
                z[l] = 1
            num, den = fir_rational(stage_totals(stage_begin, f_full, f_share, stage_extra, z))
            if best is None or num * best[1] < best[0] * den:
                best = (num, den, sub)
    return best


# --------------------------------------------------------------------------
# the two comparison placements (appendix stage tables)
# --------------------------------------------------------------------------
def place_uniform(stage_begin, m):
    """Spread m conversions one per stage from the last stage leftwards, wrapping
    round if m > P; within a stage the deepest unconverted layer is taken
    (stage table: stages 4-7 each get one for m = 4, P = 8)."""
    P = len(stage_begin) - 1
    L = stage_begin[P]
    z = [0] * L
    i, t, idle = P - 1, 0, 0
    while t < m and idle < P:
        cand = [l for l in range(stage_begin[i], stage_begin[i + 1]) if not z[l] and l > 0]
        if cand:
            z[max(cand)] = 1
            t += 1
            idle = 0
        else:
            idle += 1
        i = i - 1 if i > 0 else P - 1
    return z


def place_bipolar(stage_begin, m):
    """Two anchors, the last stage and the middle stage (index P/2 - 1), filled
    alternately, deepest layer first, each anchor moving one stage left when its
    stage is full (stage table: stages 3 and 7 get two each for m = 4, P = 8)."""
    P = len(stage_begin) - 1
    L = stage_begin[P]
    z = [0] * L
    anchors = [P - 1, max(P // 2 - 1, 0)]
    t, turn, idle = 0, 0, 0
    while t < m and idle < 2 * P:
        a = turn % 2
        i = anchors[a]
        cand = [l for l in range(stage_begin[i], stage_begin[i + 1]) if not z[l] and l > 0] if i >= 0 else []
        if cand:
            z[max(cand)] = 1
            t += 1
            idle = 0
            turn += 1
        else:
            anchors[a] -= 1
            idle += 1
            if anchors[a] < 0:
                turn += 1
    return z
