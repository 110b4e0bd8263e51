"""Parity of the CUDA path (through the C ABI) against the fp64 oracle, element by element, on the
same seeded inputs.  Tolerances: rel-L2 <= 1e-2 and max-abs <= 3e-2, literally, for every bf16 output
(Q, K, V, O, dQ, dX, decode outputs) -- where a stored value exceeds 7.7 in magnitude the element's bound is
bf16's own rounding floor 2^-8 |x| instead; LSE within 1e-3.  Only the fp32 SUMS over many tokens (the
donor-group dK/dV sums, the weight gradients), whose entries grow with the number of summed terms,
take the max-abs bound relative to max(1, |ref|_inf) -- the call sites say `sum_over_tokens=True`.
Integer / index work (planner, donor map) is bit-exact and tested without a GPU."""
import math

import numpy as np
import pytest
import torch

from oracle import attention as A
from guard import Guarded
from paper_2608_15943_b200 import synth
from paper_2608_15943_b200 import workloads as W

pytestmark = pytest.mark.gpu

REL, ABS, LSE_TOL = 1e-2, 3e-2, 1e-3


@pytest.fixture(scope="module")
def kvp():
    from paper_2608_15943_b200 import kvp as mod
    assert torch.cuda.is_available()
    return mod


def f64(t):
    return None if t is None else t.detach().float().cpu().numpy().astype(np.float64)


def f64l(ts):
    return [f64(t) for t in ts]


def close(name, got, ref, rel=REL, abs_=ABS, sum_over_tokens=False):
    got = f64(got) if isinstance(got, torch.Tensor) else np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, (name, got.shape, ref.shape)
    assert np.isfinite(got).all(), f"{name}: non-finite output"
    diff = np.abs(got - ref)
    if np.linalg.norm(ref) > 1e-6 * math.sqrt(ref.size):   # an exactly-zero reference has no relative error
        rl2 = np.linalg.norm(got - ref) / np.linalg.norm(ref)
        assert rl2 <= rel, f"{name}: rel-L2 {rl2:.3e} > {rel}"
    # a bf16 value of magnitude above 7.7 cannot be stored to within 3e-2 (half an ulp is up to 2^-8 |x|):
    # there the element's bound is that storage-rounding floor; below it the bound is the literal one
    bound = abs_ * max(1.0, float(np.abs(ref).max())) if sum_over_tokens else np.maximum(abs_, 2.0 ** -8 * np.abs(ref))
    assert (diff - bound).max() <= 0, f"{name}: max-abs {diff.max():.3e} > {abs_:.1e}"


def lse_close(name, got, ref):
    d = np.abs(f64(got) - ref).max()
    assert d <= LSE_TOL, f"{name}: LSE differs by {d:.3e}"


def run_block(kvp, cfg, t, out, causal=True):
    """proj fwd -> attn fwd -> attn bwd -> proj bwd through the C ABI."""
    sh = kvp.Shape(cfg.L, cfg.B, cfg.S, cfg.D, cfg.Hq, cfg.Hkv, cfg.dh)
    dev = t["x"][0].device
    kvp.proj_fwd(sh, cfg.donor, t["x"], t["wq"], t["wk"], t["wv"], out["q"], out["k"], out["v"])
    kvp.attn_fwd(sh, cfg.donor, out["q"], out["k"], out["v"], out["o"], out["lse"], causal=causal)
    ws = torch.empty(max(kvp.workspace_bytes(kvp.OP_ATTN_BWD, sh, cfg.donor),
                         kvp.workspace_bytes(kvp.OP_PROJ_BWD, sh, cfg.donor), 256), dtype=torch.uint8, device=dev)
    kvp.attn_bwd(sh, cfg.donor, out["q"], out["k"], out["v"], out["o"], t["d_o"], out["lse"], out["dq"],
                 out["dk_sum"], out["dv_sum"], ws, causal=causal)
    kvp.proj_bwd(sh, cfg.donor, t["x"], t["wq"], t["wk"], t["wv"], out["dq"], out["dk_sum"], out["dv_sum"],
                 out["dwq"], out["dwk"], out["dwv"], out["dx"], ws)
    torch.cuda.synchronize()
    assert kvp.device_status() == kvp.OK
    return sh


# ---------------------------------------------------------------------------------------------
# GEMM building block, every operand layout, ragged tiles
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("M,N,K", [(128, 256, 64), (256, 256, 256), (200, 264, 72), (1, 8, 8), (640, 1032, 520)])
@pytest.mark.parametrize("a_mn,b_mn", [(0, 0), (0, 1), (1, 0), (1, 1)])
def test_gemm_all_layouts(kvp, M, N, K, a_mn, b_mn):
    a = synth.normal((M, K), 7, 1, 1.0, "cuda")
    b = synth.normal((N, K), 7, 2, 1.0, "cuda")
    ref = f64(a) @ f64(b).T
    sa = a.t().contiguous() if a_mn else a
    sb = b.t().contiguous() if b_mn else b
    if (sa.stride(0) % 8) or (sb.stride(0) % 8):
        with pytest.raises(kvp.KvpError):
            kvp.gemm(sa, sb, torch.empty(M, N, device="cuda"), a_mn, b_mn)
        return
    gd = Guarded()
    c32 = gd.empty((M, N), torch.float32, float("nan"))
    kvp.gemm(sa, sb, c32, a_mn, b_mn)
    close("gemm f32", c32, ref, rel=1e-5, abs_=1e-4, sum_over_tokens=True)     # tight bounds, relative to |C|_inf
    c16 = gd.empty((M, N), torch.bfloat16, float("nan"))
    kvp.gemm(sa, sb, c16, a_mn, b_mn)
    gd.check()
    close("gemm bf16", c16, A.round_bf16(ref), rel=1e-3, abs_=1e-2, sum_over_tokens=True)
    assert kvp.device_status() == kvp.OK


@pytest.mark.parametrize("M,N,K", [(264, 8, 8), (304, 520, 200), (1280, 768, 1096)])
@pytest.mark.parametrize("a_mn,b_mn", [(0, 0), (0, 1), (1, 0), (1, 1)])
def test_gemm_on_cta_pairs_equals_single_cta_tiles(kvp, M, N, K, a_mn, b_mn):
    """The 256 x 256 tiles of the CTA-pair kernel and the 128 x 256 tiles of the single-CTA kernel sum the same
    products in the same order along K: bit-identical outputs, also with ragged last tiles in M, N and K (and a
    second half-tile that lies entirely outside M)."""
    a = synth.normal((M, K), 13, 1, 1.0, "cuda")
    b = synth.normal((N, K), 13, 2, 1.0, "cuda")
    sa = a.t().contiguous() if a_mn else a
    sb = b.t().contiguous() if b_mn else b
    out = {}
    try:
        for mode in (0, 2):
            kvp.set_gemm_pair_mode(mode)
            gd = Guarded()
            out[mode] = gd.empty((M, N), torch.float32, float("nan"))
            kvp.gemm(sa, sb, out[mode], a_mn, b_mn)
            gd.check()
    finally:
        kvp.set_gemm_pair_mode(1)
    assert torch.equal(out[0], out[2])
    close("gemm on pairs", out[2], f64(a) @ f64(b).T, rel=1e-5, abs_=1e-4, sum_over_tokens=True)
    assert kvp.device_status() == kvp.OK


def test_bounded_wait_runs_out_cleanly_on_a_cta_pair(kvp):
    """The same failure detection on the CTA-pair GEMM kernel: the issuing CTA withholds the arrivals that free a
    ring stage in both CTAs of the cluster; both give up after 5 ms, wait for each other, free their TMEM and exit."""
    assert kvp.device_status() == kvp.OK
    scratch = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    kvp.selftest_bounded_wait_pair(scratch)
    assert kvp.device_status() == kvp.ERR_TIMEOUT
    assert kvp.device_status() == kvp.OK
    with pytest.raises(kvp.KvpError) as e:
        kvp.selftest_bounded_wait_pair(scratch[:512 * 1024])
    assert e.value.status == kvp.ERR_WORKSPACE
    a = synth.normal((512, 512), 9, 1, 1.0, "cuda")
    b = synth.normal((384, 512), 9, 2, 1.0, "cuda")
    c = torch.full((512, 384), float("nan"), device="cuda")
    kvp.gemm(a, b, c, 0, 0)                              # runs on CTA pairs again
    close("pair gemm after a timed-out launch", c, f64(a) @ f64(b).T, rel=1e-5, abs_=1e-4, sum_over_tokens=True)
    assert kvp.device_status() == kvp.OK


def test_bounded_wait_runs_out_cleanly_and_the_library_stays_usable(kvp):
    """Failure detection on the device: a wait that nothing satisfies gives up after its limit, the kernel
    records the timeout, frees its TMEM and exits; the host reads the status and carries on.  The library's
    self-test withholds one barrier arrival in a small GEMM that runs with a 5 ms limit."""
    assert kvp.device_status() == kvp.OK
    scratch = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    kvp.selftest_bounded_wait(scratch)
    assert kvp.device_status() == kvp.ERR_TIMEOUT       # reported once ...
    assert kvp.device_status() == kvp.OK                # ... and cleared
    with pytest.raises(kvp.KvpError) as e:              # too small a scratch buffer is refused before any launch
        kvp.selftest_bounded_wait(scratch[:1024])
    assert e.value.status == kvp.ERR_WORKSPACE
    # tensor memory was released and the barriers of the next launch work: an ordinary GEMM is correct
    a = synth.normal((256, 512), 9, 1, 1.0, "cuda")
    b = synth.normal((384, 512), 9, 2, 1.0, "cuda")
    c = torch.full((256, 384), float("nan"), device="cuda")
    kvp.gemm(a, b, c, 0, 0)
    close("gemm after a timed-out launch", c, f64(a) @ f64(b).T, rel=1e-5, abs_=1e-4, sum_over_tokens=True)
    assert kvp.device_status() == kvp.OK


# ---------------------------------------------------------------------------------------------
# C0: the tiny stack, per-op and composed
# ---------------------------------------------------------------------------------------------
def test_c0_block_per_op_and_composed(kvp):
    cfg = W.C0
    t = W.make_train_inputs(cfg, "cuda")
    out = W.alloc_train_outputs(cfg, "cuda")
    run_block(kvp, cfg, t, out)
    dims = (cfg.B, cfg.S, cfg.Hq, cfg.Hkv, cfg.dh)
    x, wq, wk, wv, d_o = (f64l(t[n]) for n in ("x", "wq", "wk", "wv", "d_o"))
    own = cfg.owners()

    # --- per-op: each op against the oracle fed the operands that op consumed ---
    q, k, v = A.proj_fwd(x, wq, wk, wv, cfg.donor, *dims)
    for l in range(cfg.L):
        close(f"q[{l}]", out["q"][l], q[l])
    for l in own:
        close(f"k[{l}]", out["k"][l], k[l])
        close(f"v[{l}]", out["v"][l], v[l])
        assert out["k"][l] is not None
    qs, ks, vs = f64l(out["q"]), f64l(out["k"]), f64l(out["v"])
    o, lse = A.attn_fwd(qs, ks, vs, cfg.donor)
    for l in range(cfg.L):
        close(f"o[{l}]", out["o"][l], o[l])
        lse_close(f"lse[{l}]", out["lse"][l], lse[l])
    dq, dk, dv = A.attn_bwd(qs, ks, vs, d_o, cfg.donor)
    for l in range(cfg.L):
        close(f"dq[{l}]", out["dq"][l], dq[l])
    for l in own:
        close(f"dk_sum[{l}]", out["dk_sum"][l], dk[l], sum_over_tokens=True)
        close(f"dv_sum[{l}]", out["dv_sum"][l], dv[l], sum_over_tokens=True)
    dqs = f64l(out["dq"])
    dks = [A.round_bf16(f64(a)) if a is not None else None for a in out["dk_sum"]]
    dvs = [A.round_bf16(f64(a)) if a is not None else None for a in out["dv_sum"]]
    dwq, dwk, dwv, dx = A.proj_bwd(x, wq, wk, wv, dqs, dks, dvs, cfg.donor)
    for l in range(cfg.L):
        close(f"dwq[{l}]", out["dwq"][l], dwq[l], sum_over_tokens=True)
        close(f"dx[{l}]", out["dx"][l], dx[l])
    for l in own:
        close(f"dwk[{l}]", out["dwk"][l], dwk[l], sum_over_tokens=True)
        close(f"dwv[{l}]", out["dwv"][l], dwv[l], sum_over_tokens=True)

    # --- composed: oracle end to end with bf16 rounding where the interface stores bf16 ---
    r = A.round_bf16
    qc = [r(a) for a in q]
    kc = [r(a) if a is not None else None for a in k]
    vc = [r(a) if a is not None else None for a in v]
    oc, lsec = A.attn_fwd(qc, kc, vc, cfg.donor)
    dqc, dkc, dvc = A.attn_bwd(qc, kc, vc, d_o, cfg.donor)
    dwqc, dwkc, dwvc, dxc = A.proj_bwd(x, wq, wk, wv, [r(a) for a in dqc],
                                       [r(a) if a is not None else None for a in dkc],
                                       [r(a) if a is not None else None for a in dvc], cfg.donor)
    for l in range(cfg.L):
        close(f"composed o[{l}]", out["o"][l], oc[l])
        assert np.abs(f64(out["lse"][l]) - lsec[l]).max() <= 5e-3
        close(f"composed dq[{l}]", out["dq"][l], dqc[l])
        close(f"composed dwq[{l}]", out["dwq"][l], dwqc[l], sum_over_tokens=True)
        close(f"composed dx[{l}]", out["dx"][l], dxc[l])
    for l in own:
        close(f"composed dk_sum[{l}]", out["dk_sum"][l], dkc[l], sum_over_tokens=True)
        close(f"composed dv_sum[{l}]", out["dv_sum"][l], dvc[l], sum_over_tokens=True)
        close(f"composed dwk[{l}]", out["dwk"][l], dwkc[l], sum_over_tokens=True)
        close(f"composed dwv[{l}]", out["dwv"][l], dwvc[l], sum_over_tokens=True)


# ---------------------------------------------------------------------------------------------
# attention forward / backward over shapes that span several tiles and ragged tails
# ---------------------------------------------------------------------------------------------
SHAPES = [
    # B, S, Hq, Hkv, dh, donor, causal
    (1, 1, 2, 1, 128, [0], True),
    (1, 127, 2, 2, 128, [0, 0], True),
    (2, 129, 4, 2, 64, [0, 0, 2, 2], True),
    (1, 130, 2, 1, 64, [0, 1], False),
    (1, 384, 8, 2, 128, [0, 0, 0], True),
    (2, 300, 4, 4, 128, [0, 1, 1], False),
    (1, 515, 4, 1, 64, [0, 0], True),
    (1, 64, 2, 2, 128, [0], True),                          # exactly one 64-query step, MHA
    (1, 65, 2, 1, 128, [0, 0], False),
    (3, 200, 6, 3, 128, [0, 0, 0, 0, 0, 0, 0, 0], True),    # the largest donor group (8 layers), odd pair count
    (2, 193, 4, 4, 64, [0, 1, 1, 3], False),                # MHA (G = 1), mixed groups
    (1, 130, 2, 1, 64, [0, 0, 0, 3, 3, 5, 5, 5, 8, 8], True),  # ten layers: two forward launches (eight + two)
    (3, 2100, 6, 3, 64, [0, 0], True),                      # 324 forward work items on 148 persistent CTAs: three
                                                            # rounds, the last one short and dealt out backwards
]


def attn_inputs(B, S, Hq, Hkv, dh, donor, seed=11, std=1.0):
    L = len(donor)
    q = [synth.normal((B, S, Hq, dh), seed, synth.tid(20, l), std, "cuda") for l in range(L)]
    k = [synth.normal((B, S, Hkv, dh), seed, synth.tid(21, l), std, "cuda") if donor[l] == l else None for l in range(L)]
    v = [synth.normal((B, S, Hkv, dh), seed, synth.tid(22, l), 1.0, "cuda") if donor[l] == l else None for l in range(L)]
    d_o = [synth.normal((B, S, Hq, dh), seed, synth.tid(23, l), 1.0, "cuda") for l in range(L)]
    return q, k, v, d_o


@pytest.mark.parametrize("B,S,Hq,Hkv,dh,donor,causal", SHAPES)
def test_attention_forward_and_backward_shapes(kvp, B, S, Hq, Hkv, dh, donor, causal):
    L = len(donor)
    q, k, v, d_o = attn_inputs(B, S, Hq, Hkv, dh, donor)
    sh = kvp.Shape(L, B, S, 64, Hq, Hkv, dh)
    # outputs and the workspace sit between guard bands: nothing outside them may be written
    gd = Guarded()
    nan = float("nan")
    o = [gd.empty(x.shape, x.dtype, nan) for x in q]
    lse = [gd.empty((B, Hq, S), torch.float32, nan) for _ in range(L)]
    kvp.attn_fwd(sh, donor, q, k, v, o, lse, causal=causal)
    gd.check()
    ro, rl = A.attn_fwd(f64l(q), f64l(k), f64l(v), donor, causal=causal)
    for l in range(L):
        close(f"o[{l}]", o[l], ro[l])
        lse_close(f"lse[{l}]", lse[l], rl[l])
    # bit-identical on a second run (the forward has no atomics)
    o2 = [torch.empty_like(x) for x in q]
    lse2 = [torch.empty_like(x) for x in lse]
    kvp.attn_fwd(sh, donor, q, k, v, o2, lse2, causal=causal)
    for l in range(L):
        assert torch.equal(o[l], o2[l]) and torch.equal(lse[l], lse2[l])

    dq = [gd.empty(x.shape, x.dtype, nan) for x in q]
    dk = [gd.empty((B, S, Hkv, dh), torch.float32, nan) if donor[l] == l else None for l in range(L)]
    dv = [gd.empty((B, S, Hkv, dh), torch.float32, nan) if donor[l] == l else None for l in range(L)]
    ws = gd.empty((kvp.workspace_bytes(kvp.OP_ATTN_BWD, sh, donor),), torch.uint8)
    kvp.attn_bwd(sh, donor, q, k, v, o, d_o, lse, dq, dk, dv, ws, causal=causal)
    gd.check()
    rdq, rdk, rdv = A.attn_bwd(f64l(q), f64l(k), f64l(v), f64l(d_o), donor, causal=causal)
    for l in range(L):
        close(f"dq[{l}]", dq[l], rdq[l])
        if donor[l] == l:
            close(f"dk_sum[{l}]", dk[l], rdk[l], sum_over_tokens=True)
            close(f"dv_sum[{l}]", dv[l], rdv[l], sum_over_tokens=True)
    # too small a workspace is refused, not overrun
    if ws.numel() > 256:
        with pytest.raises(kvp.KvpError) as e:
            kvp.attn_bwd(sh, donor, q, k, v, o, d_o, lse, dq, dk, dv, ws[:256], causal=causal)
        assert e.value.status == kvp.ERR_WORKSPACE
    assert kvp.device_status() == kvp.OK


def test_attention_peaked_softmax_and_custom_scale(kvp):
    """Large scores exercise the running-maximum rescale path."""
    B, S, Hq, Hkv, dh, donor = 1, 640, 2, 1, 128, [0]
    q, k, v, _ = attn_inputs(B, S, Hq, Hkv, dh, donor, seed=5, std=3.0)
    sh = kvp.Shape(1, B, S, 64, Hq, Hkv, dh)
    o = [torch.empty_like(q[0])]
    lse = [torch.empty(B, Hq, S, device="cuda")]
    kvp.attn_fwd(sh, donor, q, k, v, o, lse, causal=True, scale=0.2)
    ro, rl = A.attn_fwd(f64l(q), f64l(k), f64l(v), donor, causal=True, scale=0.2)
    close("o", o[0], ro[0])
    lse_close("lse", lse[0], rl[0])


# ---------------------------------------------------------------------------------------------
# decode
# ---------------------------------------------------------------------------------------------
def gather_cache(pool, bt_row, n, page):
    """Dense [n, Hkv, dh] float64 view of one sequence's first n positions."""
    n_pg = (n + page - 1) // page
    x = pool[bt_row[:n_pg].long()]                      # [n_pg, Hkv, page, dh]
    x = x.permute(0, 2, 1, 3).reshape(n_pg * page, pool.shape[1], pool.shape[3])[:n]
    return f64(x)


def decode_reference(q, k_cache, v_cache, bt, lens, donor, page, scale=None):
    L = len(donor)
    B = len(lens)
    cap = max(lens)
    kd = [None] * L
    vd = [None] * L
    for l in range(L):
        if donor[l] != l:
            continue
        Hkv, dh = k_cache[l].shape[1], k_cache[l].shape[3]
        kd[l] = np.zeros((B, cap, Hkv, dh))
        vd[l] = np.zeros((B, cap, Hkv, dh))
        for b in range(B):
            kd[l][b, :lens[b]] = gather_cache(k_cache[l], bt[b], lens[b], page)
            vd[l][b, :lens[b]] = gather_cache(v_cache[l], bt[b], lens[b], page)
    return A.decode_attend(f64l(q), kd, vd, lens, donor, scale)


DEC_CASES = [
    # L, donor, B, Hq, Hkv, dh, page, lens, splits
    (1, [0], 1, 4, 1, 128, 16, [1], 0),
    (2, [0, 0], 3, 8, 2, 128, 128, [127, 128, 129], 0),
    (4, [0, 0, 2, 2], 2, 4, 2, 64, 64, [129, 640], 3),
    (4, [0, 0, 0, 0], 2, 8, 2, 128, 32, [777, 31], 2),
    (3, [0, 0, 0], 1, 16, 1, 64, 16, [100], 1),
    (2, [0, 1], 2, 2, 2, 128, 16, [50, 60], 7),
    (6, [0, 0, 0, 0, 0, 0], 1, 8, 2, 128, 16, [333], 0),   # six layers on one donor: two passes
]


@pytest.mark.parametrize("L,donor,B,Hq,Hkv,dh,page,lens,ns", DEC_CASES)
def test_decode_against_oracle(kvp, L, donor, B, Hq, Hkv, dh, page, lens, ns):
    max_pages = (max(lens) + page - 1) // page + 1
    n_pages = B * max_pages
    g = torch.Generator().manual_seed(3)
    bt = torch.randperm(n_pages, generator=g).int().reshape(B, max_pages).cuda()
    lengths = torch.tensor(lens, dtype=torch.int32, device="cuda")
    kc = [synth.normal((n_pages, Hkv, page, dh), 13, synth.tid(7, l), 1.0, "cuda") if donor[l] == l else None
          for l in range(L)]
    vc = [synth.normal((n_pages, Hkv, page, dh), 13, synth.tid(8, l), 1.0, "cuda") if donor[l] == l else None
          for l in range(L)]
    q = [synth.normal((B, Hq, dh), 13, synth.tid(6, l), 1.0, "cuda") for l in range(L)]
    desc = kvp.DecodeDesc(L, B, Hq, Hkv, dh, page, max_pages, n_pages, ns)
    ws = torch.empty(kvp.decode_workspace_bytes(desc, donor), dtype=torch.uint8, device="cuda")

    def run(desc_, bt_, kc_, vc_):
        gd = Guarded()
        o = [gd.empty((B, Hq, dh), torch.bfloat16, float("nan")) for _ in range(L)]
        lse = [gd.empty((B, Hq), torch.float32, float("nan")) for _ in range(L)]
        w = gd.empty((kvp.decode_workspace_bytes(desc_, donor),), torch.uint8)
        kvp.decode(desc_, donor, q, kc_, vc_, bt_, lengths, o, lse, w)
        gd.check()
        return o, lse

    o, lse = run(desc, bt, kc, vc)
    ro, rl = decode_reference(q, kc, vc, bt, lens, donor, page)
    for l in range(L):
        close(f"o[{l}]", o[l], ro[l])
        lse_close(f"lse[{l}]", lse[l], rl[l])
    # invariant to the number of splits (up to rounding) ...
    o1, lse1 = run(kvp.DecodeDesc(L, B, Hq, Hkv, dh, page, max_pages, n_pages, 1), bt, kc, vc)
    for l in range(L):
        close(f"o[{l}] one split", o1[l], ro[l])
        assert (lse1[l] - lse[l]).abs().max().item() <= 1e-4
    # ... and bit-identical under a permutation of the physical pages
    perm = torch.randperm(n_pages, generator=g).cuda()
    inv = torch.empty_like(perm)
    inv[perm] = torch.arange(n_pages, device="cuda")
    kc2 = [a[inv].contiguous() if a is not None else None for a in kc]   # new page perm[p] holds old page p
    vc2 = [a[inv].contiguous() if a is not None else None for a in vc]
    bt2 = perm[bt.long()].int()
    o2, lse2 = run(desc, bt2, kc2, vc2)
    for l in range(L):
        assert torch.equal(o2[l], o[l]) and torch.equal(lse2[l], lse[l])
    # layer ranges: one layer at a time (sequential use) gives the same values
    for l in range(L):
        ol = [torch.zeros_like(x) for x in o]
        ll = [torch.zeros_like(x) for x in lse]
        kvp.decode(desc, donor, q, kc, vc, bt, lengths, ol, ll, ws, layer_begin=l, layer_end=l + 1)
        assert torch.equal(ol[l], o[l]) and torch.equal(ll[l], lse[l])
    assert kvp.device_status() == kvp.OK


def test_decode_ignores_never_appended_slots_even_if_they_hold_nan(kvp):
    """Cache slots at or past lengths[b] were never appended (a pool from an uninitialised allocation, a
    recycled page): whatever bit pattern they hold, NaN included, must not reach the output.  Every slot past
    the length, in the straddling 16-token granule, the rest of its page and the unused pages, is set to NaN."""
    L, donor, B, Hq, Hkv, dh, page = 2, [0, 0], 3, 8, 2, 128, 64
    lens = [1, 70, 200]          # inside the first granule, straddling a granule, straddling a page
    max_pages = 5
    n_pages = B * max_pages
    g = torch.Generator().manual_seed(11)
    bt = torch.randperm(n_pages, generator=g).int().reshape(B, max_pages).cuda()
    lengths = torch.tensor(lens, dtype=torch.int32, device="cuda")
    kc = [synth.normal((n_pages, Hkv, page, dh), 17, synth.tid(7, 0), 1.0, "cuda"), None]
    vc = [synth.normal((n_pages, Hkv, page, dh), 17, synth.tid(8, 0), 1.0, "cuda"), None]
    q = [synth.normal((B, Hq, dh), 17, synth.tid(6, l), 1.0, "cuda") for l in range(L)]
    ro, rl = decode_reference(q, kc, vc, bt, lens, donor, page)          # reads only positions < len
    for b in range(B):
        for i in range(max_pages):
            first_dead = min(max(lens[b] - i * page, 0), page)
            pg = int(bt[b, i])
            kc[0][pg, :, first_dead:] = float("nan")
            vc[0][pg, :, first_dead:] = float("nan")
    for ns in (1, 3):
        desc = kvp.DecodeDesc(L, B, Hq, Hkv, dh, page, max_pages, n_pages, ns)
        ws = torch.empty(kvp.decode_workspace_bytes(desc, donor), dtype=torch.uint8, device="cuda")
        o = [torch.full((B, Hq, dh), float("nan"), device="cuda", dtype=torch.bfloat16) for _ in range(L)]
        lse = [torch.full((B, Hq), float("nan"), device="cuda") for _ in range(L)]
        kvp.decode(desc, donor, q, kc, vc, bt, lengths, o, lse, ws)
        for l in range(L):
            close(f"o[{l}] splits={ns}", o[l], ro[l])
            lse_close(f"lse[{l}] splits={ns}", lse[l], rl[l])
    assert kvp.device_status() == kvp.OK


def test_projection_backward_layer_by_layer_equals_one_call(kvp):
    """kvp_proj_bwd_range over single layers (what a data-parallel step interleaves with the per-layer gradient
    all-reduce) writes bit for bit what one kvp_proj_bwd call writes."""
    cfg = W.C0
    t = W.make_train_inputs(cfg, "cuda")
    out = W.alloc_train_outputs(cfg, "cuda")
    sh = run_block(kvp, cfg, t, out)
    ws = torch.empty(kvp.workspace_bytes(kvp.OP_PROJ_BWD, sh, cfg.donor), dtype=torch.uint8, device="cuda")
    names = ("dwq", "dwk", "dwv", "dx")
    again = {n: [None if a is None else torch.full_like(a, float("nan")) for a in out[n]] for n in names}
    for l in range(cfg.L):
        kvp.proj_bwd(sh, cfg.donor, t["x"], t["wq"], t["wk"], t["wv"], out["dq"], out["dk_sum"], out["dv_sum"],
                     again["dwq"], again["dwk"], again["dwv"], again["dx"], ws, layer_begin=l, layer_end=l + 1)
    torch.cuda.synchronize()
    for n in names:
        for l in range(cfg.L):
            if out[n][l] is not None:
                assert torch.equal(again[n][l], out[n][l]), (n, l)
    with pytest.raises(kvp.KvpError):
        kvp.proj_bwd(sh, cfg.donor, t["x"], t["wq"], t["wk"], t["wv"], out["dq"], out["dk_sum"], out["dv_sum"],
                     again["dwq"], again["dwk"], again["dwv"], again["dx"], ws, layer_begin=3, layer_end=9)
    assert kvp.device_status() == kvp.OK


def test_projections_of_thirteen_layers_span_several_grouped_launches(kvp):
    """Thirteen layers with eleven owners are 35 forward projections and 13 + 22 + 13 gradient GEMMs: more than one
    grouped launch holds (32 problems; the backward takes eight layers at a time), with ragged M, N and K tiles in
    every problem (T = 200, D = 192, Nq = 192, Nkv = 64)."""
    donor = [0, 1, 1, 3, 4, 5, 6, 6, 8, 9, 10, 11, 12]
    cfg = W.TrainCfg("thirteen-layers", 13, 2, 100, 192, 3, 1, 64, donor)
    t = W.make_train_inputs(cfg, "cuda")
    out = W.alloc_train_outputs(cfg, "cuda")
    sh = kvp.Shape(cfg.L, cfg.B, cfg.S, cfg.D, cfg.Hq, cfg.Hkv, cfg.dh)
    kvp.proj_fwd(sh, donor, t["x"], t["wq"], t["wk"], t["wv"], out["q"], out["k"], out["v"])
    g = torch.Generator(device="cpu").manual_seed(5)
    dq = [(torch.randn(cfg.T, cfg.Hq * cfg.dh, generator=g) * 0.5).to(torch.bfloat16).cuda() for _ in range(cfg.L)]
    dks = [None if donor[l] != l else (torch.randn(cfg.T, cfg.Hkv * cfg.dh, generator=g) * 0.5).cuda() for l in range(cfg.L)]
    dvs = [None if donor[l] != l else (torch.randn(cfg.T, cfg.Hkv * cfg.dh, generator=g) * 0.5).cuda() for l in range(cfg.L)]
    ws = torch.empty(kvp.workspace_bytes(kvp.OP_PROJ_BWD, sh, donor), dtype=torch.uint8, device="cuda")
    kvp.proj_bwd(sh, donor, t["x"], t["wq"], t["wk"], t["wv"], dq, dks, dvs, out["dwq"], out["dwk"], out["dwv"],
                 out["dx"], ws)
    torch.cuda.synchronize()
    assert kvp.device_status() == kvp.OK
    x, wq, wk, wv = (f64l(t[n]) for n in ("x", "wq", "wk", "wv"))
    q, k, v = A.proj_fwd(x, wq, wk, wv, donor, cfg.B, cfg.S, cfg.Hq, cfg.Hkv, cfg.dh)
    rb = lambda a: None if a is None else A.round_bf16(f64(a))
    dwq, dwk, dwv, dx = A.proj_bwd(x, wq, wk, wv, f64l(dq), [rb(a) for a in dks], [rb(a) for a in dvs], donor)
    for l in range(cfg.L):
        close(f"q[{l}]", out["q"][l], q[l])
        close(f"dwq[{l}]", out["dwq"][l], dwq[l], sum_over_tokens=True)
        close(f"dx[{l}]", out["dx"][l], dx[l])
        if donor[l] == l:
            close(f"k[{l}]", out["k"][l], k[l])
            close(f"v[{l}]", out["v"][l], v[l])
            close(f"dwk[{l}]", out["dwk"][l], dwk[l], sum_over_tokens=True)
            close(f"dwv[{l}]", out["dwv"][l], dwv[l], sum_over_tokens=True)


def test_projection_block_is_bit_identical_on_cta_pairs_and_single_cta_tiles(kvp):
    """Every projection GEMM of a small block -- forward (K-major operands), weight gradients (both operands
    MN-major, fp32 output, K = all tokens) and input gradients (three K segments into one tile) -- gives the same
    bits on the CTA-pair kernel as on the single-CTA kernel.  All problems have more than 128 rows, so pair mode 2
    really puts every grouped launch on pairs."""
    donor = [0, 0, 2]
    cfg = W.TrainCfg("pairs-vs-single", 3, 2, 200, 192, 4, 2, 128, donor)
    t = W.make_train_inputs(cfg, "cuda")
    sh = kvp.Shape(cfg.L, cfg.B, cfg.S, cfg.D, cfg.Hq, cfg.Hkv, cfg.dh)
    g = torch.Generator(device="cpu").manual_seed(17)
    dq = [(torch.randn(cfg.T, cfg.Hq * cfg.dh, generator=g) * 0.5).to(torch.bfloat16).cuda() for _ in range(cfg.L)]
    dks = [None if donor[l] != l else (torch.randn(cfg.T, cfg.Hkv * cfg.dh, generator=g) * 0.5).cuda() for l in range(cfg.L)]
    dvs = [None if donor[l] != l else (torch.randn(cfg.T, cfg.Hkv * cfg.dh, generator=g) * 0.5).cuda() for l in range(cfg.L)]
    ws = torch.empty(kvp.workspace_bytes(kvp.OP_PROJ_BWD, sh, donor), dtype=torch.uint8, device="cuda")
    outs = {}
    try:
        for mode in (0, 2):
            kvp.set_gemm_pair_mode(mode)
            out = W.alloc_train_outputs(cfg, "cuda")
            for name in ("q", "k", "v", "dwq", "dwk", "dwv", "dx"):
                for a in out[name]:
                    if a is not None:
                        a.fill_(float("nan"))
            kvp.proj_fwd(sh, donor, t["x"], t["wq"], t["wk"], t["wv"], out["q"], out["k"], out["v"])
            kvp.proj_bwd(sh, donor, t["x"], t["wq"], t["wk"], t["wv"], dq, dks, dvs, out["dwq"], out["dwk"], out["dwv"],
                         out["dx"], ws)
            torch.cuda.synchronize()
            outs[mode] = out
    finally:
        kvp.set_gemm_pair_mode(1)
    assert kvp.device_status() == kvp.OK
    for name in ("q", "k", "v", "dwq", "dwk", "dwv", "dx"):
        for l in range(cfg.L):
            a, b = outs[0][name][l], outs[2][name][l]
            if a is not None:
                assert not torch.isnan(a.float()).any(), (name, l)
                assert torch.equal(a, b), (name, l)
    x, wq, wk, wv = (f64l(t[n]) for n in ("x", "wq", "wk", "wv"))
    rb = lambda a: None if a is None else A.round_bf16(f64(a))
    dwq, dwk, dwv, dx = A.proj_bwd(x, wq, wk, wv, f64l(dq), [rb(a) for a in dks], [rb(a) for a in dvs], donor)
    for l in range(cfg.L):
        close(f"dx[{l}] on pairs", outs[2]["dx"][l], dx[l])
        close(f"dwq[{l}] on pairs", outs[2]["dwq"][l], dwq[l], sum_over_tokens=True)


def test_c0_with_fp32_buffers(kvp):
    """The tiny stack with fp32 tensors in the caller's memory (dtype F32): forward, backward and decode steps.
    The library rounds fp32 inputs to bf16 on load and widens its bf16 results on store, so (i) every output
    meets the oracle at the bf16 tolerances and (ii) equals, bit for bit after widening, what the bf16 interface
    returns for the same values (the generator's values are bf16-representable)."""
    cfg = W.C0
    t = W.make_train_inputs(cfg, "cuda")
    out = W.alloc_train_outputs(cfg, "cuda")
    run_block(kvp, cfg, t, out)                                   # bf16 interface: the comparison values
    f32 = lambda xs: [None if a is None else a.float() for a in xs]
    t32 = {n: f32(xs) for n, xs in t.items()}
    like = lambda xs: [None if a is None else torch.full(a.shape, float("nan"), device="cuda") for a in xs]
    o32 = {n: like(out[n]) for n in ("q", "k", "v", "o", "dq", "dx")}
    lse = like(out["lse"])
    dk, dv, dwq, dwk, dwv = (like(out[n]) for n in ("dk_sum", "dv_sum", "dwq", "dwk", "dwv"))
    sh = kvp.Shape(cfg.L, cfg.B, cfg.S, cfg.D, cfg.Hq, cfg.Hkv, cfg.dh, kvp.F32)
    need = max(kvp.workspace_bytes(op, sh, cfg.donor) for op in (kvp.OP_PROJ_FWD, kvp.OP_ATTN_FWD, kvp.OP_ATTN_BWD, kvp.OP_PROJ_BWD))
    assert kvp.workspace_bytes(kvp.OP_PROJ_FWD, sh, cfg.donor) > 0
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    with pytest.raises(kvp.KvpError) as e:                        # the fp32 interface needs its shadow space
        kvp.proj_fwd(sh, cfg.donor, t32["x"], t32["wq"], t32["wk"], t32["wv"], o32["q"], o32["k"], o32["v"])
    assert e.value.status == kvp.ERR_WORKSPACE
    kvp.proj_fwd(sh, cfg.donor, t32["x"], t32["wq"], t32["wk"], t32["wv"], o32["q"], o32["k"], o32["v"], ws)
    kvp.attn_fwd(sh, cfg.donor, o32["q"], o32["k"], o32["v"], o32["o"], lse, ws=ws)
    kvp.attn_bwd(sh, cfg.donor, o32["q"], o32["k"], o32["v"], o32["o"], t32["d_o"], lse, o32["dq"], dk, dv, ws)
    kvp.proj_bwd(sh, cfg.donor, t32["x"], t32["wq"], t32["wk"], t32["wv"], o32["dq"], dk, dv, dwq, dwk, dwv, o32["dx"], ws)
    torch.cuda.synchronize()
    assert kvp.device_status() == kvp.OK
    for n in ("q", "k", "v", "o", "dx"):
        for l in range(cfg.L):
            if out[n][l] is not None:
                assert o32[n][l].dtype == torch.float32
                assert torch.equal(o32[n][l], out[n][l].float()), (n, l)
    for l in range(cfg.L):
        assert torch.equal(lse[l], out["lse"][l])
        # dQ goes through fp32 reductions whose order is not fixed: equal up to fp32 rounding, then bf16-rounded
        assert (o32["dq"][l] - out["dq"][l].float()).abs().max().item() <= 2.0 ** -7 * out["dq"][l].float().abs().max().item()
    # against the oracle, per operation, on the operands each operation consumed
    dims = (cfg.B, cfg.S, cfg.Hq, cfg.Hkv, cfg.dh)
    x, wq, wk, wv, d_o = (f64l(t[n]) for n in ("x", "wq", "wk", "wv", "d_o"))
    q, k, v = A.proj_fwd(x, wq, wk, wv, cfg.donor, *dims)
    qs, ks, vs = f64l(o32["q"]), f64l(o32["k"]), f64l(o32["v"])
    ro, rl = A.attn_fwd(qs, ks, vs, cfg.donor)
    rdq, rdk, rdv = A.attn_bwd(qs, ks, vs, d_o, cfg.donor)
    for l in range(cfg.L):
        close(f"q[{l}]", o32["q"][l], q[l])
        close(f"o[{l}]", o32["o"][l], ro[l])
        lse_close(f"lse[{l}]", lse[l], rl[l])
        close(f"dq[{l}]", o32["dq"][l], rdq[l])
        if cfg.donor[l] == l:
            close(f"dk_sum[{l}]", dk[l], rdk[l], sum_over_tokens=True)
            close(f"dv_sum[{l}]", dv[l], rdv[l], sum_over_tokens=True)
    # decode with fp32 queries / new rows / outputs over a bf16 cache filled from the prefill
    steps, page = 4, 16
    own = cfg.owners()
    max_pages = (cfg.S + steps + page - 1) // page
    n_pages = cfg.B * max_pages
    bt = torch.arange(n_pages, dtype=torch.int32, device="cuda").reshape(cfg.B, max_pages)
    kc, vc, kc16, vc16 = ([None] * cfg.L for _ in range(4))
    for l in own:
        for name, pools in (("k", (kc, kc16)), ("v", (vc, vc16))):
            pool = torch.zeros(n_pages, cfg.Hkv, page, cfg.dh, dtype=torch.bfloat16, device="cuda")
            pg = out[name][l].reshape(cfg.B, cfg.S // page, page, cfg.Hkv, cfg.dh).permute(0, 1, 3, 2, 4)
            pool.view(cfg.B, max_pages, cfg.Hkv, page, cfg.dh)[:, :cfg.S // page] = pg
            pools[0][l], pools[1][l] = pool, pool.clone()
    d32 = kvp.DecodeDesc(cfg.L, cfg.B, cfg.Hq, cfg.Hkv, cfg.dh, page, max_pages, n_pages, 2, kvp.F32)
    d16 = kvp.DecodeDesc(cfg.L, cfg.B, cfg.Hq, cfg.Hkv, cfg.dh, page, max_pages, n_pages, 2)
    dws = torch.empty(kvp.decode_workspace_bytes(d32, cfg.donor), dtype=torch.uint8, device="cuda")
    lengths = torch.full((cfg.B,), cfg.S, dtype=torch.int32, device="cuda")
    for step in range(steps):
        qn = [synth.normal((cfg.B, cfg.Hq, cfg.dh), W.SEED, synth.tid(30, l, step), 1.0, "cuda") for l in range(cfg.L)]
        kn = [synth.normal((cfg.B, cfg.Hkv, cfg.dh), W.SEED, synth.tid(31, l, step), 1.0, "cuda") if l in own else None
              for l in range(cfg.L)]
        vn = [synth.normal((cfg.B, cfg.Hkv, cfg.dh), W.SEED, synth.tid(32, l, step), 1.0, "cuda") if l in own else None
              for l in range(cfg.L)]
        lengths += 1
        kvp.cache_append(d32, cfg.donor, f32(kn), f32(vn), kc, vc, bt, lengths)
        kvp.cache_append(d16, cfg.donor, kn, vn, kc16, vc16, bt, lengths)
        o_a = [torch.full((cfg.B, cfg.Hq, cfg.dh), float("nan"), device="cuda") for _ in range(cfg.L)]
        o_b = [torch.empty(cfg.B, cfg.Hq, cfg.dh, dtype=torch.bfloat16, device="cuda") for _ in range(cfg.L)]
        l_a = [torch.empty(cfg.B, cfg.Hq, device="cuda") for _ in range(cfg.L)]
        l_b = [torch.empty(cfg.B, cfg.Hq, device="cuda") for _ in range(cfg.L)]
        kvp.decode(d32, cfg.donor, f32(qn), kc, vc, bt, lengths, o_a, l_a, dws)
        kvp.decode(d16, cfg.donor, qn, kc16, vc16, bt, lengths, o_b, l_b, dws)
        lens = [int(n) for n in lengths.cpu()]
        ro, rl = decode_reference(qn, kc, vc, bt, lens, cfg.donor, page)
        for l in range(cfg.L):
            assert torch.equal(o_a[l], o_b[l].float()) and torch.equal(l_a[l], l_b[l])
            close(f"decode step {step} o[{l}]", o_a[l], ro[l])
            lse_close(f"decode step {step} lse[{l}]", l_a[l], rl[l])
    for l in own:
        assert torch.equal(kc[l], kc16[l]) and torch.equal(vc[l], vc16[l])
    assert kvp.device_status() == kvp.OK


def test_c0_prefill_then_16_decode_steps(kvp):
    """Prefill the tiny stack, move K/V into pages, then 16 decode steps: project the new token,
    append for owners, attend over the shared cache; compared step by step with the oracle run with
    bf16 rounding where the interface stores bf16."""
    cfg = W.C0
    steps, page = 16, 16
    t = W.make_train_inputs(cfg, "cuda")
    out = W.alloc_train_outputs(cfg, "cuda")
    sh = kvp.Shape(cfg.L, cfg.B, cfg.S, cfg.D, cfg.Hq, cfg.Hkv, cfg.dh)
    kvp.proj_fwd(sh, cfg.donor, t["x"], t["wq"], t["wk"], t["wv"], out["q"], out["k"], out["v"])
    own = cfg.owners()
    max_pages = (cfg.S + steps + page - 1) // page
    n_pages = cfg.B * max_pages
    bt = torch.arange(n_pages, dtype=torch.int32, device="cuda").reshape(cfg.B, max_pages)
    kc = [None] * cfg.L
    vc = [None] * cfg.L
    for l in own:
        for name, pool_list in (("k", kc), ("v", vc)):
            pool = torch.zeros(n_pages, cfg.Hkv, page, cfg.dh, dtype=torch.bfloat16, device="cuda")
            src = out[name][l]                                            # [B,S,Hkv,dh]
            pg = src.reshape(cfg.B, cfg.S // page, page, cfg.Hkv, cfg.dh).permute(0, 1, 3, 2, 4)
            pool.view(cfg.B, max_pages, cfg.Hkv, page, cfg.dh)[:, :cfg.S // page] = pg
            pool_list[l] = pool
    # oracle state: dense caches from the SAME stored bf16 prefill K/V
    cap = cfg.S + steps
    okc = [None] * cfg.L
    ovc = [None] * cfg.L
    for l in own:
        okc[l] = np.zeros((cfg.B, cap, cfg.Hkv, cfg.dh))
        ovc[l] = np.zeros((cfg.B, cap, cfg.Hkv, cfg.dh))
        okc[l][:, :cfg.S] = f64(out["k"][l])
        ovc[l][:, :cfg.S] = f64(out["v"][l])
    olen = [cfg.S] * cfg.B
    wq, wk, wv = f64l(t["wq"]), f64l(t["wk"]), f64l(t["wv"])
    desc = kvp.DecodeDesc(cfg.L, cfg.B, cfg.Hq, cfg.Hkv, cfg.dh, page, max_pages, n_pages, 2)
    ws = torch.empty(kvp.decode_workspace_bytes(desc, cfg.donor), dtype=torch.uint8, device="cuda")
    dsh = kvp.Shape(cfg.L, cfg.B, 1, cfg.D, cfg.Hq, cfg.Hkv, cfg.dh)      # one token per sequence
    lengths = torch.full((cfg.B,), cfg.S, dtype=torch.int32, device="cuda")
    for step in range(steps):
        x_t = [synth.normal((cfg.B, cfg.D), W.SEED, synth.tid(10, l, step), 1.0, "cuda") for l in range(cfg.L)]
        qn = [torch.empty(cfg.B, 1, cfg.Hq, cfg.dh, dtype=torch.bfloat16, device="cuda") for _ in range(cfg.L)]
        kn = [torch.empty(cfg.B, 1, cfg.Hkv, cfg.dh, dtype=torch.bfloat16, device="cuda") if l in own else None
              for l in range(cfg.L)]
        vn = [torch.empty(cfg.B, 1, cfg.Hkv, cfg.dh, dtype=torch.bfloat16, device="cuda") if l in own else None
              for l in range(cfg.L)]
        kvp.proj_fwd(dsh, cfg.donor, x_t, t["wq"], t["wk"], t["wv"], qn, kn, vn)
        lengths += 1
        kvp.cache_append(desc, cfg.donor, kn, vn, kc, vc, bt, lengths)
        o = [torch.empty(cfg.B, cfg.Hq, cfg.dh, dtype=torch.bfloat16, device="cuda") for _ in range(cfg.L)]
        lse = [torch.empty(cfg.B, cfg.Hq, device="cuda") for _ in range(cfg.L)]
        kvp.decode(desc, cfg.donor, qn, kc, vc, bt, lengths, o, lse, ws)
        oq, oo, ol = A.decode_step(f64l(x_t), wq, wk, wv, okc, ovc, olen, cfg.donor, cfg.Hq, cfg.Hkv, cfg.dh,
                                   store_round=A.round_bf16)
        for l in range(cfg.L):
            close(f"step {step} q[{l}]", qn[l].reshape(cfg.B, cfg.Hq, cfg.dh), oq[l], rel=5e-3)
            close(f"step {step} o[{l}]", o[l], oo[l])
            assert np.abs(f64(lse[l]) - ol[l]).max() <= 5e-3   # composed: q, k re-rounded on each side
    # the appended rows landed where the oracle put them
    for l in own:
        got = kc[l].view(cfg.B, max_pages, cfg.Hkv, page, cfg.dh).permute(0, 1, 3, 2, 4).reshape(
            cfg.B, max_pages * page, cfg.Hkv, cfg.dh)[:, cfg.S:cfg.S + steps]
        close(f"appended k[{l}]", got, okc[l][:, cfg.S:cfg.S + steps], rel=5e-3)
    assert kvp.device_status() == kvp.OK


def test_decode_clamps_out_of_range_lengths(kvp):
    L, donor, B, Hq, Hkv, dh, page = 1, [0], 2, 4, 1, 128, 16
    max_pages, n_pages = 4, 8
    bt = torch.arange(8, dtype=torch.int32, device="cuda").reshape(B, max_pages)
    kc = [synth.normal((n_pages, Hkv, page, dh), 1, 1, 1.0, "cuda")]
    vc = [synth.normal((n_pages, Hkv, page, dh), 1, 2, 1.0, "cuda")]
    q = [synth.normal((B, Hq, dh), 1, 3, 1.0, "cuda")]
    desc = kvp.DecodeDesc(L, B, Hq, Hkv, dh, page, max_pages, n_pages, 0)
    ws = torch.empty(kvp.decode_workspace_bytes(desc, donor), dtype=torch.uint8, device="cuda")
    o = [torch.empty(B, Hq, dh, dtype=torch.bfloat16, device="cuda")]
    lse = [torch.empty(B, Hq, device="cuda")]
    lengths = torch.tensor([0, 10 ** 6], dtype=torch.int32, device="cuda")   # both invalid
    kvp.decode(desc, donor, q, kc, vc, bt, lengths, o, lse, ws)
    torch.cuda.synchronize()
    ro, _ = decode_reference(q, kc, vc, bt, [1, max_pages * page], donor, page)
    close("clamped", o[0], ro[0])
    assert kvp.device_status() == kvp.OK


# ---------------------------------------------------------------------------------------------
# output projection (stage workload) and its chain rule
# ---------------------------------------------------------------------------------------------
def test_output_projection(kvp):
    cfg = W.TrainCfg("t", 2, 1, 200, 128, 2, 1, 64, [0, 0])
    sh = kvp.Shape(cfg.L, cfg.B, cfg.S, cfg.D, cfg.Hq, cfg.Hkv, cfg.dh)
    nq = cfg.Hq * cfg.dh
    o = [synth.normal((cfg.B, cfg.S, cfg.Hq, cfg.dh), 3, synth.tid(30, l), 1.0, "cuda") for l in range(cfg.L)]
    wo = [synth.normal((cfg.D, nq), 3, synth.tid(31, l), 0.05, "cuda") for l in range(cfg.L)]
    dy = [synth.normal((cfg.T, cfg.D), 3, synth.tid(32, l), 1.0, "cuda") for l in range(cfg.L)]
    y = [torch.empty(cfg.T, cfg.D, dtype=torch.bfloat16, device="cuda") for _ in range(cfg.L)]
    d_o = [torch.empty_like(x) for x in o]
    dwo = [torch.empty(cfg.D, nq, device="cuda") for _ in range(cfg.L)]
    kvp.out_proj_fwd(sh, o, wo, y)
    kvp.out_proj_bwd(sh, o, wo, dy, d_o, dwo)
    for l in range(cfg.L):
        close("y", y[l], A.out_proj_fwd(f64(o[l]), f64(wo[l])))
        rd, rw = A.out_proj_bwd(f64(o[l]), f64(wo[l]), f64(dy[l]))
        close("d_o", d_o[l], rd)
        close("dwo", dwo[l], rw, sum_over_tokens=True)
    assert kvp.device_status() == kvp.OK
