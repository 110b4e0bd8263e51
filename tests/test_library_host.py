"""Host-side checks that need no GPU: the C-ABI library loads, exports every symbol the header
declares, rejects bad arguments, and its planner is bit-exact against the integer oracle."""
import ctypes as C
import os
import random
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def kvp():
    from paper_2608_15943_b200 import build
    build.build()
    from paper_2608_15943_b200 import kvp as mod
    return mod


def test_every_declared_symbol_is_exported(kvp):
    text = open(os.path.join(ROOT, "include", "kvp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(kvp_[a-z0-9_]+)\s*\(", text))
    assert {"kvp_plan", "kvp_proj_fwd", "kvp_proj_bwd", "kvp_attn_fwd", "kvp_attn_bwd", "kvp_decode",
            "kvp_cache_append", "kvp_layer_flops", "kvp_workspace_bytes", "kvp_status_string"} <= declared
    for name in declared:
        assert hasattr(kvp.lib, name), f"{name} declared in kvp.h but not exported"
    assert set(kvp.EXPORTS) <= declared


def test_status_strings(kvp):
    assert kvp.status_string(kvp.OK) == "ok"
    assert "donor" in kvp.status_string(kvp.ERR_BAD_DONOR)
    assert kvp.status_string(99) == "unknown status"


def test_workspace_queries_and_argument_validation_without_gpu(kvp):
    sh = kvp.Shape(8, 2, 8192, 4096, 32, 8, 128)
    donor = [0, 1, 2, 3, 4, 4, 4, 4]
    ws = kvp.workspace_bytes(kvp.OP_ATTN_BWD, sh, donor)
    # Delta [B,Hq,S] fp32 per layer + fp32 dQ accumulators for the member layers of one launch (at most 8)
    assert ws == 8 * (2 * 32 * 8192 * 4) + 8 * (2 * 32 * 8192 * 128 * 4)
    # bf16 copies of the fp32 dK / dV sums of the owners of one grouped launch (5 owners here, at most 8)
    assert kvp.workspace_bytes(kvp.OP_PROJ_BWD, sh, donor) == 5 * 2 * (2 * 8192 * 8 * 128 * 2)
    assert kvp.workspace_bytes(kvp.OP_PROJ_BWD, kvp.Shape(12, 2, 8192, 4096, 32, 8, 128), list(range(12))) \
        == 8 * 2 * (2 * 8192 * 8 * 128 * 2)
    assert kvp.workspace_bytes(kvp.OP_ATTN_FWD, sh, donor) == 0
    assert kvp.workspace_bytes(kvp.OP_ATTN_BWD, sh, [0, 0, 1, 0, 0, 0, 0, 0]) == 0   # invalid donor chain
    # entry points validate before touching the device
    nul = [None] * 8
    with pytest.raises(kvp.KvpError) as e:
        kvp.attn_fwd(sh, [0, 0, 1, 0, 0, 0, 0, 0], nul, nul, nul, nul, nul)
    assert e.value.status == kvp.ERR_BAD_DONOR
    with pytest.raises(kvp.KvpError) as e:
        kvp.attn_fwd(kvp.Shape(8, 2, 8192, 4096, 32, 8, 96), donor, nul, nul, nul, nul, nul)
    assert e.value.status == kvp.ERR_UNSUPPORTED
    with pytest.raises(kvp.KvpError) as e:
        kvp.attn_fwd(sh, donor, nul, nul, nul, nul, nul)
    assert e.value.status == kvp.ERR_INVALID_ARG
    d = kvp.DecodeDesc(4, 2, 8, 2, 128, 128, 10, 20)
    assert kvp.decode_workspace_bytes(d, [0, 0, 2, 2]) > 0
    assert kvp.decode_workspace_bytes(kvp.DecodeDesc(4, 2, 8, 2, 128, 100, 10, 20), [0, 0, 2, 2]) == 0


def test_self_tests_and_tile_mode_switch_validate_before_touching_the_device(kvp):
    # both bounded-wait self-tests refuse a missing or too small scratch buffer before any launch
    for fn, need in ((kvp.lib.kvp_selftest_bounded_wait, 512 * 1024), (kvp.lib.kvp_selftest_bounded_wait_pair, 768 * 1024)):
        assert fn(None, need, None) == kvp.ERR_WORKSPACE
        assert fn(0x1000, need - 1, None) == kvp.ERR_WORKSPACE
        assert fn(0x1008, need, None) == kvp.ERR_WORKSPACE          # not 16-byte aligned
    # the pair self-test is refused while CTA pairs are switched off; the switch clamps its argument
    try:
        kvp.set_gemm_pair_mode(0)
        assert kvp.lib.kvp_selftest_bounded_wait_pair(0x1000, 768 * 1024, None) == kvp.ERR_UNSUPPORTED
        kvp.set_gemm_pair_mode(7)
        kvp.set_gemm_pair_mode(-3)
    finally:
        kvp.set_gemm_pair_mode(1)


def _rand_instance(rng):
    Pn = rng.randint(1, 6)
    sizes = [rng.randint(1, 5) for _ in range(Pn)]
    sb = [0]
    for s in sizes:
        sb.append(sb[-1] + s)
    L = sb[-1]
    if rng.random() < 0.5:
        f = rng.randint(10, 10 ** 9)
        d = rng.randint(1, f - 1)
        full, share = [f] * L, [f - d] * L
    else:
        full = [rng.randint(10, 10 ** 12) for _ in range(L)]
        share = [x - rng.randint(1, x - 1) for x in full]
    extra = [rng.randint(0, 10 ** 9) if rng.random() < 0.4 else 0 for _ in range(Pn)]
    return sb, full, share, extra


@pytest.mark.parametrize("seed", range(200))
def test_plan_bit_exact_against_oracle(kvp, seed):
    from oracle import plan as OP
    rng = random.Random(seed)
    sb, full, share, extra = _rand_instance(rng)
    L = sb[-1]
    eps = rng.choice([(0, 1), (1, 100), (5, 100), (1, 10), (3, 7)])
    kw = dict(eps=eps, max_conv=rng.choice([0, 0, 1, 2, 3, L]), stop_on_no_improve=rng.random() < 0.5,
              stage_local_donor=rng.random() < 0.3, alpha=rng.choice([None, None, (1, 2), (3, 4), (1, 3)]))
    want = OP.kvp_plan(sb, full, share, extra, **kw)
    got = kvp.plan(sb, full, share, extra, **kw)
    assert got["z"] == want["z"]
    assert got["donor"] == want["donor"]
    assert got["stage"] == want["stage"]
    assert (got["fir_num"], got["fir_den"]) == (want["fir_num"], want["fir_den"])
    assert (got["n_conv"], got["stop_reason"]) == (want["n_conv"], want["stop_reason"])
    assert got["fir"] == want["fir_num"] / want["fir_den"]
    P = len(sb) - 1
    assert got["stage_ratio"] == [s * P / want["fir_den"] for s in want["stage"]]


@pytest.mark.parametrize("seed", range(120))
def test_comparison_placements_bit_exact(kvp, seed):
    """The library computes the two comparison placements in closed form / with two descending cursors, the oracle
    by stepping through the visits one at a time: two independent formulations must agree, also where more layers
    are converted than there are stages, where a stage fills up, and where everything convertible is converted."""
    from oracle import plan as OP
    rng = random.Random(500 + seed)
    sb, full, share, extra = _rand_instance(rng)
    m = sb[-1] if seed % 7 == 0 else rng.randint(0, sb[-1])
    for placement, fn in ((kvp.PLACE_UNIFORM, OP.place_uniform), (kvp.PLACE_BIPOLAR, OP.place_bipolar)):
        z = fn(sb, m) if m else [0] * sb[-1]
        got = kvp.plan(sb, full, share, extra, max_conv=m, placement=placement) if m else None
        if got is None:
            continue
        assert got["z"] == z
        assert got["stage"] == OP.stage_totals(sb, full, share, extra, z)
        assert got["donor"] == OP.donor_from_z(z)


def test_plan_paper_case_and_flops_helper(kvp):
    from oracle import plan as OP
    for args in [(4096, 11008, 32, 32, 128, 8192, 32000, True), (4096, 11008, 32, 8, 128, 4096, 32000, True),
                 (5120, 13824, 40, 40, 128, 16384, 32000, False)]:
        assert kvp.layer_flops(*args) == OP.layer_flops(*args)
    ff, fs, flm = kvp.layer_flops(4096, 11008, 32, 32, 128, 8192, 32000)
    sb = [4 * i for i in range(9)]
    out = kvp.plan(sb, [ff] * 32, [fs] * 32, [0] * 7 + [flm], stop_on_no_improve=True)
    assert [l + 1 for l, z in enumerate(out["z"]) if z] == [29, 30, 31, 32]
    assert abs(out["fir"] - 1.00040391) < 5e-5


def test_plan_rejects_bad_input(kvp):
    with pytest.raises(kvp.KvpError):
        kvp.plan([0, 2, 4], [10] * 4, [10] * 4, [0, 0])            # f_share must be < f_full
    with pytest.raises(kvp.KvpError):
        kvp.plan([0, 2, 2, 4], [10] * 4, [5] * 4, [0, 0, 0])       # empty stage
    with pytest.raises(kvp.KvpError):
        kvp.plan([0, 2, 4], [10] * 4, [5] * 4, [0, 0], eps=(1, 0))  # zero denominator
    with pytest.raises(kvp.KvpError):
        kvp.plan([0, 2, 4], [2 ** 63] * 4, [5] * 4, [0, 0])        # totals overflow 64 bits


@pytest.mark.parametrize("seed", range(6))
def test_sim_1f1b_bit_exact_against_oracle(kvp, seed):
    import random
    from oracle import pipeline as PL
    rng = random.Random(seed)
    for _ in range(40):
        P, M = rng.randint(1, 9), rng.randint(1, 12)
        tf = [rng.randint(0, 10 ** 6) for _ in range(P)]
        tb = [rng.randint(0, 2 * 10 ** 6) for _ in range(P)]
        assert kvp.sim_1f1b(tf, tb, M) == tuple(PL.sim_1f1b(tf, tb, M))
    # the paper's setting: 8 stages, the last one heavier
    tf, tb = [100] * 7 + [118], [200] * 7 + [236]
    assert kvp.sim_1f1b(tf, tb, 32) == tuple(PL.sim_1f1b(tf, tb, 32))
    assert kvp.sim_1f1b([5] * 8, [10] * 8, 16)[0] == (16 + 7) * 15


def test_sim_1f1b_rejects_bad_input(kvp):
    for args in (([], [], 4), ([1, 2], [1], 4), ([1, 2], [1, 2], 0), ([1, -2], [1, 2], 3)):
        with pytest.raises(kvp.KvpError):
            kvp.sim_1f1b(*args)
