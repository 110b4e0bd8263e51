"""Pins for the stage-operator oracle (oracle/stage.py): closed forms, invariants and torch's functional
routines as an independent library opinion."""
import numpy as np
import torch

from oracle import stage as ST

RNG = np.random.default_rng(7)


def test_rmsnorm_unit_rms_scale_invariance_and_closed_form():
    x = RNG.normal(size=(5, 64)) * 3.0
    y = ST.rmsnorm(x, np.ones(64), 0.0)
    assert np.allclose(np.sqrt(np.mean(y * y, axis=1)), 1.0, atol=1e-12)
    assert np.allclose(ST.rmsnorm(7.5 * x, np.ones(64), 0.0), y, atol=1e-12)          # invariant to the input's scale
    w = RNG.normal(size=64)
    assert np.allclose(ST.rmsnorm(x, w, 0.0), y * w, atol=1e-12)                       # the weight is a plain factor
    # a constant row c: mean square c^2, so y = c / sqrt(c^2 + eps) * w
    c, eps = 2.0, 0.25
    assert np.allclose(ST.rmsnorm(np.full((1, 8), c), np.arange(8.0), eps), c / np.sqrt(c * c + eps) * np.arange(8.0))
    # eps dominates a zero row
    assert np.all(ST.rmsnorm(np.zeros((1, 8)), np.ones(8), 1e-6) == 0.0)


def test_rmsnorm_against_torch():
    x = RNG.normal(size=(9, 128))
    w = RNG.normal(size=128)
    ref = torch.nn.functional.rms_norm(torch.tensor(x), (128,), torch.tensor(w), 1e-5).numpy()
    assert np.allclose(ST.rmsnorm(x, w, 1e-5), ref, atol=1e-12)


def test_rope_rotation_of_one_pair_written_out():
    # dh = 2: the single pair rotates by pos * theta^0 = pos radians
    x = np.array([1.0, 0.0, 0.0, 2.0]).reshape(1, 2, 1, 2)          # token 0: (1, 0); token 1: (0, 2)
    y = ST.rope(x, theta=10000.0, pos0=0)
    assert np.allclose(y[0, 0, 0], [1.0, 0.0])                        # position 0 is the identity
    assert np.allclose(y[0, 1, 0], [-2.0 * np.sin(1.0), 2.0 * np.cos(1.0)])
    # second pair of dh = 4 turns by pos * theta^(-2/4)
    x4 = np.zeros((1, 3, 1, 4))
    x4[0, 2, 0, 2] = 1.0
    y4 = ST.rope(x4, theta=100.0)
    ang = 2 * 100.0 ** (-0.5)
    assert np.allclose(y4[0, 2, 0], [0.0, 0.0, np.cos(ang), np.sin(ang)])


def test_rope_preserves_norms_and_depends_on_relative_position_only():
    B, S, H, dh = 2, 7, 3, 16
    q = RNG.normal(size=(B, S, H, dh))
    k = RNG.normal(size=(B, S, H, dh))
    rq, rk = ST.rope(q), ST.rope(k)
    pair_norm = lambda a: a.reshape(B, S, H, dh // 2, 2)
    assert np.allclose((pair_norm(rq) ** 2).sum(-1), (pair_norm(q) ** 2).sum(-1), atol=1e-12)
    # <rope(q, m), rope(k, n)> is a function of m - n: shifting both positions leaves every score unchanged
    s0 = np.einsum("bshd,bthd->bhst", rq, rk)
    s5 = np.einsum("bshd,bthd->bhst", ST.rope(q, pos0=5), ST.rope(k, pos0=5))
    assert np.allclose(s0, s5, atol=1e-10)
    # and the same vector placed at two positions scores like its copy at their distance
    v = RNG.normal(size=(1, 1, 1, dh))
    a = ST.rope(v, pos0=9)[0, 0, 0] @ ST.rope(v, pos0=4)[0, 0, 0]
    b = ST.rope(v, pos0=5)[0, 0, 0] @ ST.rope(v, pos0=0)[0, 0, 0]
    assert abs(a - b) < 1e-10


def test_rope_against_complex_multiplication():
    B, S, H, dh = 1, 6, 2, 8
    x = RNG.normal(size=(B, S, H, dh))
    xc = torch.view_as_complex(torch.tensor(x).reshape(B, S, H, dh // 2, 2))
    freqs = 10000.0 ** (-torch.arange(0, dh, 2, dtype=torch.float64) / dh)
    ang = torch.outer(torch.arange(S, dtype=torch.float64), freqs)
    rot = torch.polar(torch.ones_like(ang), ang)[None, :, None, :]
    ref = torch.view_as_real(xc * rot).reshape(B, S, H, dh).numpy()
    assert np.allclose(ST.rope(x), ref, atol=1e-12)


def test_swiglu_closed_forms_and_torch():
    g = np.array([0.0, 1.0, -1.0, 30.0, -30.0])
    u = np.array([5.0, 2.0, 2.0, 1.0, 1.0])
    y = ST.swiglu(g, u)
    assert y[0] == 0.0
    assert np.isclose(y[1], 2.0 / (1.0 + np.exp(-1.0)))
    assert np.isclose(y[1] - y[2], 2.0 * 1.0)                  # silu(t) - silu(-t) = t
    assert np.isclose(y[3], 30.0, rtol=1e-12) and abs(y[4]) < 1e-11
    a, b = RNG.normal(size=(4, 33)), RNG.normal(size=(4, 33))
    ref = (torch.nn.functional.silu(torch.tensor(a)) * torch.tensor(b)).numpy()
    assert np.allclose(ST.swiglu(a, b), ref, atol=1e-13)


def test_add():
    assert np.array_equal(ST.add([1.0, 2.0], [0.5, -2.0]), np.array([1.5, 0.0]))
