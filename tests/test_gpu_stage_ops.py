"""Parity of the element-wise stage operators (through the C ABI) against the fp64 oracle on seeded inputs.
Outputs are bf16: the bar is the rounding of the exact result (half an ulp, 2^-9 relative) plus the fp32
arithmetic, i.e. |got - ref| <= 2^-8 |ref| + 1e-6 element by element, and rel-L2 <= 4e-3."""
import numpy as np
import pytest
import torch

from oracle import stage as ST
from paper_2608_15943_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def kvp():
    from paper_2608_15943_b200 import kvp as mod
    assert torch.cuda.is_available()
    return mod


def f64(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def close(name, got, ref):
    got, ref = f64(got), np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape and np.isfinite(got).all(), name
    err = np.abs(got - ref)
    bound = 2.0 ** -8 * np.abs(ref) + 1e-6
    assert (err <= bound).all(), f"{name}: worst excess {float((err - bound).max()):.3e} at |ref| {float(np.abs(ref).flat[(err - bound).argmax()]):.3e}"
    assert np.linalg.norm(got - ref) <= 4e-3 * np.linalg.norm(ref) + 1e-9, name


@pytest.mark.parametrize("T,D", [(1, 8), (5, 256), (37, 4096), (3, 8192), (300, 1000)])
def test_rmsnorm(kvp, T, D):
    x = synth.normal((T, D), 3, synth.tid(40), 2.0, "cuda")
    w = synth.normal((D,), 3, synth.tid(41), 1.0, "cuda")
    y = torch.full_like(x, float("nan"))
    kvp.rmsnorm(x, w, 1e-5, y)
    close("rmsnorm", y, ST.rmsnorm(f64(x), f64(w), 1e-5))
    kvp.rmsnorm(x, w, 1e-5, x)                      # in place
    assert torch.equal(x, y)
    assert kvp.device_status() == kvp.OK


@pytest.mark.parametrize("B,S,H,dh,pos0", [(1, 1, 1, 8, 0), (2, 130, 3, 64, 0), (1, 64, 4, 128, 7), (1, 33, 2, 128, 131000),
                                           (1, 16, 1, 256, 262000)])
def test_rope(kvp, B, S, H, dh, pos0):
    x = synth.normal((B, S, H, dh), 5, synth.tid(42), 1.0, "cuda")
    ref = ST.rope(f64(x), 10000.0, pos0)
    kvp.rope(x, 10000.0, pos0)
    close("rope", x, ref)
    assert kvp.device_status() == kvp.OK


@pytest.mark.parametrize("shape", [(1, 8), (7, 11008), (257, 264)])
def test_swiglu_and_add(kvp, shape):
    g = synth.normal(shape, 9, synth.tid(43), 3.0, "cuda")
    u = synth.normal(shape, 9, synth.tid(44), 1.0, "cuda")
    out = torch.full_like(g, float("nan"))
    kvp.swiglu(g, u, out)
    close("swiglu", out, ST.swiglu(f64(g), f64(u)))
    s = torch.full_like(g, float("nan"))
    kvp.add(g, u, s)
    close("add", s, ST.add(f64(g), f64(u)))
    kvp.add(g, u, g)                                # in place
    assert torch.equal(g, s)
    assert kvp.device_status() == kvp.OK


def test_shape_limits_are_refused(kvp):
    x = torch.zeros(4, 12, dtype=torch.bfloat16, device="cuda")
    w = torch.zeros(12, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(kvp.KvpError) as e:
        kvp.rmsnorm(x, w, 1e-5, x)                  # D not a multiple of 8
    assert e.value.status == kvp.ERR_UNSUPPORTED
    with pytest.raises(kvp.KvpError):
        kvp.rope(torch.zeros(1, 2, 1, 12, dtype=torch.bfloat16, device="cuda"))
    with pytest.raises(kvp.KvpError):
        kvp.rope(torch.zeros(1, 2, 1, 16, dtype=torch.bfloat16, device="cuda"), 10000.0, 1 << 18)   # position limit
    y = torch.zeros(12, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(kvp.KvpError):
        kvp.swiglu(y, y, y)                         # n not a multiple of 8
    with pytest.raises(kvp.KvpError):
        kvp.add(y, y, y)


def test_whole_stage_forward_composed(kvp):
    """Two decoder layers (an owner and a consumer that attends to the owner's K/V) and the LM head, every operator of
    the stage chained through the C ABI with real data flow: RMSNorm -> Q (K, V) projections -> rotary embedding ->
    causal attention -> output projection -> residual -> RMSNorm -> gate / up -> SwiGLU -> down -> residual, then the
    final norm and the logits.  The oracle runs the same chain in fp64 and rounds to bf16 wherever the stage stores a
    bf16 tensor, so what is compared is the arithmetic of the kernels, not the storage format.  Bound, element by
    element: 2^-6 of the reference plus 2^-5 of the tensor's rms (a bf16 rounding that falls the other way early in
    the chain is carried through the MLP's matrix products), and rel-L2 <= 1e-2."""
    from oracle import attention as A
    B, S, D, Hq, Hkv, dh, F, V = 1, 192, 256, 4, 2, 64, 512, 384
    T, nq, nkv = B * S, Hq * dh, Hkv * dh
    bf = torch.bfloat16
    rnd = lambda shape, i, std: synth.normal(shape, 21, synth.tid(60, i), std, "cuda")
    h = rnd((T, D), 0, 1.0)
    wn1 = [rnd((D,), 1 + l, 1.0) for l in range(2)]
    wn2 = [rnd((D,), 3 + l, 1.0) for l in range(2)]
    wq = [rnd((nq, D), 5 + l, 0.06) for l in range(2)]
    wk, wv = rnd((nkv, D), 7, 0.06), rnd((nkv, D), 8, 0.06)
    wo = [rnd((D, nq), 9 + l, 0.06) for l in range(2)]
    wg = [rnd((F, D), 11 + l, 0.06) for l in range(2)]
    wu = [rnd((F, D), 13 + l, 0.06) for l in range(2)]
    wd = [rnd((D, F), 15 + l, 0.04) for l in range(2)]
    wnf, wlm = rnd((D,), 17, 1.0), rnd((V, D), 18, 0.06)

    # ---- the kernels ----
    e = lambda *shape: torch.full(shape, float("nan"), dtype=bf, device="cuda")
    sh1 = kvp.Shape(1, B, S, D, Hq, Hkv, dh)
    k_r = v_r = None
    x = h
    for l in range(2):
        n1 = kvp.rmsnorm(x, wn1[l], 1e-5, e(T, D))
        q = kvp.gemm(n1, wq[l], e(T, nq)).view(B, S, Hq, dh)
        kvp.rope(q)
        if l == 0:                                   # the owner projects K and V; the consumer reuses them (Eq. 3)
            k_r = kvp.gemm(n1, wk, e(T, nkv)).view(B, S, Hkv, dh)
            v_r = kvp.gemm(n1, wv, e(T, nkv)).view(B, S, Hkv, dh)
            kvp.rope(k_r)
        o, lse = e(B, S, Hq, dh), torch.empty(B, Hq, S, device="cuda")
        kvp.attn_fwd(sh1, [0], [q], [k_r], [v_r], [o], [lse])
        y = kvp.gemm(o.view(T, nq), wo[l], e(T, D))
        h1 = kvp.add(x, y, e(T, D))
        n2 = kvp.rmsnorm(h1, wn2[l], 1e-5, e(T, D))
        gate, up = kvp.gemm(n2, wg[l], e(T, F)), kvp.gemm(n2, wu[l], e(T, F))
        act = kvp.swiglu(gate, up, e(T, F))
        x = kvp.add(h1, kvp.gemm(act, wd[l], e(T, D)), e(T, D))
    logits = kvp.gemm(kvp.rmsnorm(x, wnf, 1e-5, e(T, D)), wlm, e(T, V))
    torch.cuda.synchronize()
    assert kvp.device_status() == kvp.OK

    # ---- the oracle, bf16 wherever the stage stores bf16 ----
    r = A.round_bf16
    mm = lambda a, w: r(a @ f64(w).T)
    xr = f64(h)
    kr = vr = None
    for l in range(2):
        n1 = r(ST.rmsnorm(xr, f64(wn1[l]), 1e-5))
        q = r(ST.rope(mm(n1, wq[l]).reshape(B, S, Hq, dh)))
        if l == 0:
            kr = r(ST.rope(mm(n1, wk).reshape(B, S, Hkv, dh)))
            vr = mm(n1, wv).reshape(B, S, Hkv, dh)
        o, _ = A.attn_fwd([q], [kr], [vr], [0])
        y = mm(r(o[0]).reshape(T, nq), wo[l])
        h1 = r(ST.add(xr, y))
        n2 = r(ST.rmsnorm(h1, f64(wn2[l]), 1e-5))
        act = r(ST.swiglu(mm(n2, wg[l]), mm(n2, wu[l])))
        xr = r(ST.add(h1, mm(act, wd[l])))
    ref_logits = mm(r(ST.rmsnorm(xr, f64(wnf), 1e-5)), wlm)

    for name, got, ref in (("residual stream after two layers", x, xr), ("logits", logits, ref_logits)):
        got = f64(got)
        assert np.isfinite(got).all(), name
        err = np.abs(got - ref)
        rms = float(np.sqrt(np.mean(ref * ref)))
        bound = 2.0 ** -6 * np.abs(ref) + 2.0 ** -5 * rms
        assert (err <= bound).all(), f"{name}: worst excess {float((err - bound).max()):.3e}"
        rel = np.linalg.norm(got - ref) / np.linalg.norm(ref)
        assert rel <= 1e-2, f"{name}: rel-L2 {rel:.3e}"
