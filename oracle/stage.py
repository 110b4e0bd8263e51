"""fp64 oracle for the element-wise operators of a decoder stage (TEST INFRASTRUCTURE ONLY).

Only the tests, the smoke entry and the benchmark's cpu_baseline / reference
legs may import this; it shares no code with the CUDA kernels in the library.

The paper times whole pipeline stages of LLaMA2-7B (the "FWD time" rows of its
stage tables) but defines none of the stage's operators besides attention
(Eq. 1-3).  The three below are the ones of the architecture it names, written
out from their published definitions, so that a stage's forward time can be
measured with the library's own kernels:

* rmsnorm   y = x / sqrt(mean(x^2) + eps) * w          (root-mean-square layer normalisation)
* rope      rotary position embedding: consecutive pairs (x[2i], x[2i+1]) of every head are
            rotated by the angle pos * theta^(-2i/dh)      (the complex-pair form)
* swiglu    h = silu(gate) * up,  silu(t) = t / (1 + exp(-t))
* add       residual sum

Everything is computed in float64 on the values as given; rounding to the
storage type is the caller's business (oracle.attention.round_bf16).

Pins (tests/test_oracle_stage.py): closed forms and invariants (unit RMS,
scale invariance; norm preservation, identity at position 0, the relative-
position property of rotated dot products, the 2-D rotation matrix written out
for one pair; silu at 0, its odd part, its limits), and torch's functional
routines as a library opinion.
"""
from __future__ import annotations

import numpy as np


def rmsnorm(x, w, eps):
    """x [T, D], w [D] -> [T, D]."""
    x = np.asarray(x, dtype=np.float64)
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * np.asarray(w, dtype=np.float64)


def rope(x, theta=10000.0, pos0=0):
    """x [B, S, H, dh] (dh even) -> same shape; token s of every sequence has position pos0 + s."""
    x = np.asarray(x, dtype=np.float64)
    B, S, H, dh = x.shape
    out = np.empty_like(x)
    for s in range(S):
        pos = pos0 + s
        for i in range(dh // 2):
            ang = pos * theta ** (-2.0 * i / dh)
            c, sn = np.cos(ang), np.sin(ang)
            a, b = x[:, s, :, 2 * i], x[:, s, :, 2 * i + 1]
            out[:, s, :, 2 * i] = a * c - b * sn
            out[:, s, :, 2 * i + 1] = a * sn + b * c
    return out


def swiglu(gate, up):
    g = np.asarray(gate, dtype=np.float64)
    return g / (1.0 + np.exp(-g)) * np.asarray(up, dtype=np.float64)


def add(a, b):
    return np.asarray(a, dtype=np.float64) + np.asarray(b, dtype=np.float64)
