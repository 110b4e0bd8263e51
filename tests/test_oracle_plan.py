"""Pins for the planner oracle: values the paper prints, hand traces, exhaustive search."""
import os
import random
from fractions import Fraction

import pytest

from oracle import plan as P

GOLD = {}
with open(os.path.join(os.path.dirname(__file__), "golden", "plan_pins.txt")) as fh:
    for line in fh:
        if line.startswith("#") or not line.strip():
            continue
        name, val, tol, _ = [s.strip() for s in line.split("|")]
        GOLD[name] = (val, tol)


def gold(name):
    v, t = GOLD[name]
    return float(v), float(t)


def llama7b(s, pp, V=32000):
    """LLaMA2-7B geometry of the paper's case study: h=4096, f=11008, MHA (r=1)."""
    ff, fs, flm = P.layer_flops(4096, 11008, 32, 32, 128, s, V, causal_half=True)
    L = 32
    sb = [i * (L // pp) for i in range(pp + 1)]
    extra = [0] * pp
    extra[-1] = flm
    return sb, [ff] * L, [fs] * L, extra


def fir(stage):
    n, d = P.fir_rational(stage)
    return n / d


def test_flops_helper_matches_appendix_formulas():
    h, f, a, g, dh, s, V = 4096, 11008, 32, 8, 128, 4096, 32000
    r = a // g
    ff, fs, flm = P.layer_flops(h, f, a, g, dh, s, V, causal_half=False)
    # boxed per-token GQA total 4h^2 + 4h^2/r + 4sh, plus the MLP term
    assert ff == 4 * h * h + 4 * h * h // r + 4 * s * h + 6 * h * f
    assert ff - fs == 4 * h * h // r            # Delta F_GQA
    assert flm == 2 * h * V
    ff1, fs1, _ = P.layer_flops(h, f, 32, 32, 128, s, V, causal_half=False)
    assert ff1 == 8 * h * h + 4 * s * h + 6 * h * f   # boxed MHA total
    assert ff1 - fs1 == 4 * h * h
    ffc, _, _ = P.layer_flops(h, f, 32, 32, 128, s, V, causal_half=True)
    assert ff1 - ffc == 2 * s * h


def test_printed_baseline_fir_values():
    sb, ff, fs, ex = llama7b(8192, 8)
    st = P.stage_totals(sb, ff, fs, ex, [0] * 32)
    v, t = gold("fir_baseline_pp8_s8k")
    assert abs(fir(st) - v) <= t
    v, t = gold("fir_baseline_pp8_s8k_short")
    assert abs(fir(st) - v) <= t
    sb, ff, fs, ex = llama7b(4096, 2)
    v, t = gold("fir_baseline_pp2_s4k")
    assert abs(fir(P.stage_totals(sb, ff, fs, ex, [0] * 32)) - v) <= t
    sb, ff, fs, ex = llama7b(8192, 4)
    v, t = gold("fir_baseline_pp4_s8k")
    assert abs(fir(P.stage_totals(sb, ff, fs, ex, [0] * 32)) - v) <= t


def test_printed_stage_flops():
    sb, ff, fs, ex = llama7b(8192, 8)
    tokens = 8192  # MBS = 1, S = 8K
    st = [x * tokens for x in P.stage_totals(sb, ff, fs, ex, [0] * 32)]
    v, t = gold("stage_flops_body")
    assert all(abs(x - v) <= t for x in st[:7])
    v, t = gold("stage_flops_tail")
    assert abs(st[7] - v) <= t
    z = [0] * 28 + [1] * 4
    st = [x * tokens for x in P.stage_totals(sb, ff, fs, ex, z)]
    v, t = gold("stage_flops_tail_archbal")
    assert abs(st[7] - v) <= t


def test_algorithm1_selects_printed_layers_and_fir():
    sb, ff, fs, ex = llama7b(8192, 8)
    out = P.kvp_plan(sb, ff, fs, ex, eps=(0, 1), stop_on_no_improve=True)
    want = [int(x) for x in GOLD["selected_layers_pp8_s8k"][0].split()]
    assert [l + 1 for l, z in enumerate(out["z"]) if z] == want
    assert out["stop_reason"] == P.STOP_NO_IMPROVE
    v, t = gold("fir_archbal_pp8_s8k_m4")
    assert abs(out["fir_num"] / out["fir_den"] - v) <= t
    v, t = gold("fir_kvpipe_pp8_s8k_short")
    assert abs(out["fir_num"] / out["fir_den"] - v) <= t
    counts = [sum(out["z"][sb[i]:sb[i + 1]]) for i in range(8)]
    assert counts == [int(x) for x in GOLD["archbal_stage_counts_pp8_m4"][0].split()]
    # literal Algorithm 1 with a budget of 4 gives the same mask
    out2 = P.kvp_plan(sb, ff, fs, ex, eps=(1, 10000), max_conv=4)
    assert out2["z"] == out["z"] and out2["stop_reason"] == P.STOP_BUDGET
    # donors: nearest preceding unconverted layer
    assert out["donor"] == list(range(28)) + [27] * 4


def test_fir_is_v_shaped_in_the_tail_budget():
    sb, ff, fs, ex = llama7b(8192, 8)
    vals = []
    for k in range(0, 7):
        out = P.kvp_plan(sb, ff, fs, ex, eps=(0, 1), max_conv=k) if k else None
        z = out["z"] if out else [0] * 32
        vals.append(fir(P.stage_totals(sb, ff, fs, ex, z)))
    assert vals[0] > vals[1] > vals[2] > vals[3] > vals[4]
    # after the tail is balanced the greedy retargets; FIR no longer drops below vals[4]
    assert min(vals[5:]) >= vals[4] - 1e-12


def test_comparison_placements_match_stage_tables():
    sb, ff, fs, ex = llama7b(8192, 8)
    zu = P.place_uniform(sb, 4)
    zb = P.place_bipolar(sb, 4)
    cu = [sum(zu[sb[i]:sb[i + 1]]) for i in range(8)]
    cb = [sum(zb[sb[i]:sb[i + 1]]) for i in range(8)]
    assert cu == [int(x) for x in GOLD["uniform_stage_counts_pp8_m4"][0].split()]
    assert cb == [int(x) for x in GOLD["bipolar_stage_counts_pp8_m4"][0].split()]
    v, t = gold("fir_uniform_pp8_s8k_m4")
    assert abs(fir(P.stage_totals(sb, ff, fs, ex, zu)) - v) <= t
    v, t = gold("fir_bipolar_pp8_s8k_m4")
    assert abs(fir(P.stage_totals(sb, ff, fs, ex, zb)) - v) <= t


def test_hand_trace_small():
    # L=4, P=2, uniform layer cost 10 (shared 7), tail extra 6.
    sb, ff, fs = [0, 2, 4], [10] * 4, [7] * 4
    out = P.kvp_plan(sb, ff, fs, [0, 6], eps=(0, 1), stop_on_no_improve=True)
    # stages (20, 26): FIR 52/46.  convert layer 3 -> (20, 23): 46/43 < 52/46.
    # convert layer 2 -> (20, 20): FIR 1 -> stop on tolerance.
    assert out["z"] == [0, 0, 1, 1] and out["stage"] == [20, 20]
    assert (out["fir_num"], out["fir_den"]) == (40, 40) and out["stop_reason"] == P.STOP_TOLERANCE
    assert out["donor"] == [0, 1, 1, 1]
    # stage-local donors: layer 2 (first of stage 1) stays an owner
    out = P.kvp_plan(sb, ff, fs, [0, 6], eps=(0, 1), stop_on_no_improve=True, stage_local_donor=True)
    assert out["z"] == [0, 0, 0, 1] and out["donor"] == [0, 1, 2, 2]
    assert out["stop_reason"] == P.STOP_EXHAUSTED
    # no tail extra: already balanced, nothing converted
    out = P.kvp_plan(sb, ff, fs, [0, 0], eps=(0, 1))
    assert out["z"] == [0, 0, 0, 0] and out["n_conv"] == 0 and out["fir_num"] == out["fir_den"]
    # budget
    out = P.kvp_plan(sb, ff, fs, [0, 6], eps=(0, 1), max_conv=1)
    assert out["z"] == [0, 0, 0, 1] and out["stop_reason"] == P.STOP_BUDGET
    # literal algorithm over-corrects: tail extra 1 -> (20,21); convert 3 -> (20,18): tail below
    # average, retarget to stage 0, convert layer 1 -> (17,18); tail is argmax ... until exhausted
    out = P.kvp_plan(sb, ff, fs, [0, 1], eps=(0, 1))
    assert out["z"] == [0, 1, 1, 1] and out["stop_reason"] == P.STOP_EXHAUSTED
    # guardrail alpha = 3/4: only (1-indexed) layers >= 3 are admissible
    out = P.kvp_plan(sb, ff, fs, [0, 1], eps=(0, 1), alpha=(3, 4))
    assert out["z"][1] == 0


def test_tolerance_stop_and_retarget_tie_break():
    # three equal stages + small extra on the tail; eps = 5 %
    sb = [0, 2, 4, 6]
    ff, fs = [100] * 6, [90] * 6
    out = P.kvp_plan(sb, ff, fs, [0, 0, 4], eps=(5, 100))
    assert out["n_conv"] == 0 and out["stop_reason"] == P.STOP_TOLERANCE   # 204*3/604 = 1.013
    # eps = 0: convert 5 -> (200,200,194): tail under average; argmax tie between stages 0 and 1
    # goes to the higher index (stage 1, layer 3) -> (200,190,194); then stage 0, layer 1.
    out = P.kvp_plan(sb, ff, fs, [0, 0, 4], eps=(0, 1), max_conv=3)
    assert out["z"] == [0, 1, 0, 1, 0, 1]


@pytest.mark.parametrize("seed", range(40))
def test_greedy_equals_exhaustive_on_paper_family(seed):
    """Equal layers, equal stage sizes, extra cost only on the tail: the greedy with the
    no-improve stop reaches the minimum FIR over all subsets."""
    rng = random.Random(seed)
    Pn = rng.choice([2, 3, 4])
    per = rng.choice([1, 2, 3])
    L = Pn * per
    if L > 10 or L < 2:
        pytest.skip("size")
    full = rng.randint(50, 200)
    share = full - rng.randint(1, 40)
    extra = [0] * Pn
    extra[-1] = rng.randint(0, 4 * (full - share) + 5)
    sb = [i * per for i in range(Pn + 1)]
    out = P.kvp_plan(sb, [full] * L, [share] * L, extra, eps=(0, 1), stop_on_no_improve=True)
    bn, bd, _ = P.exhaustive_min_fir(sb, [full] * L, [share] * L, extra)
    assert Fraction(out["fir_num"], out["fir_den"]) == Fraction(bn, bd)


@pytest.mark.parametrize("seed", range(20))
def test_exhaustive_never_worse_on_heterogeneous(seed):
    rng = random.Random(1000 + seed)
    Pn, per = 3, 2
    L = Pn * per
    full = [rng.randint(50, 200) for _ in range(L)]
    share = [f - rng.randint(1, 40) for f in full]
    extra = [rng.randint(0, 50) for _ in range(Pn)]
    sb = [i * per for i in range(Pn + 1)]
    out = P.kvp_plan(sb, full, share, extra, eps=(0, 1), stop_on_no_improve=True)
    bn, bd, _ = P.exhaustive_min_fir(sb, full, share, extra)
    assert Fraction(bn, bd) <= Fraction(out["fir_num"], out["fir_den"])
    # the greedy never increases FIR relative to doing nothing
    n0, d0 = P.fir_rational(P.stage_totals(sb, full, share, extra, [0] * L))
    assert Fraction(out["fir_num"], out["fir_den"]) <= Fraction(n0, d0)


def test_donor_maps_of_the_benchmark_configs():
    assert P.donor_from_z([0, 1, 0, 1]) == [0, 0, 2, 2]
    assert P.donor_from_z([0, 0, 0, 0, 0, 1, 1, 1]) == [0, 1, 2, 3, 4, 4, 4, 4]
    z = [0] * 16 + [0, 1] * 8
    d = P.donor_from_z(z)
    assert d[:16] == list(range(16)) and all(d[2 * k + 1] == 2 * k and d[2 * k] == 2 * k for k in range(8, 16))
    with pytest.raises(ValueError):
        P.donor_from_z([1, 0])


def test_stage_workload_plan_gqa():
    """32-layer GQA 32/8 decoder, PP=8, s=4096: the LM head outweighs four K/V savings, so the
    whole tail stage converts and the stage is exhausted."""
    ff, fs, flm = P.layer_flops(4096, 11008, 32, 8, 128, 4096, 32000)
    assert ff == 387973120 and ff - fs == 16777216
    sb = [4 * i for i in range(9)]
    ex = [0] * 7 + [flm]
    out = P.kvp_plan(sb, [ff] * 32, [fs] * 32, ex, eps=(0, 1), stop_on_no_improve=True)
    assert [l for l, z in enumerate(out["z"]) if z] == [28, 29, 30, 31]
    assert out["stop_reason"] == P.STOP_EXHAUSTED
    assert abs(out["fir_num"] / out["fir_den"] - 1.108265) < 1e-6
    out = P.kvp_plan(sb, [ff] * 32, [fs] * 32, ex, eps=(0, 1), stop_on_no_improve=True, stage_local_donor=True)
    assert out["donor"][28:] == [28, 28, 28, 28]
