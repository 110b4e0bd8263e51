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
