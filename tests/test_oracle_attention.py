"""Pins for the fp64 attention oracle: brute force, library third opinions, closed forms,
invariants, finite differences.  None of these re-types the oracle's own formulae."""
import math

import numpy as np
import pytest
import torch

from oracle import attention as A


def rnd(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


def make(L, B, S, Hq, Hkv, dh, donor, seed=0):
    q = [rnd((B, S, Hq, dh), seed + 10 * l) for l in range(L)]
    k = [rnd((B, S, Hkv, dh), seed + 10 * l + 1) if donor[l] == l else None for l in range(L)]
    v = [rnd((B, S, Hkv, dh), seed + 10 * l + 2) if donor[l] == l else None for l in range(L)]
    return q, k, v


def brute_forward(q, k, v, donor, causal, scale):
    """Pure-Python loops with the probability matrix written out."""
    L = len(q)
    out, lse = [], []
    for l in range(L):
        d = donor[l]
        B, S, Hq, dh = q[l].shape
        G = Hq // k[d].shape[2]
        o = np.zeros((B, S, Hq, dh))
        ls = np.zeros((B, Hq, S))
        for b in range(B):
            for h in range(Hq):
                for i in range(S):
                    js = range(i + 1) if causal else range(S)
                    s = [sum(q[l][b, i, h, c] * k[d][b, j, h // G, c] for c in range(dh)) * scale for j in js]
                    m = max(s)
                    w = [math.exp(x - m) for x in s]
                    z = sum(w)
                    for c in range(dh):
                        o[b, i, h, c] = sum(w[n] * v[d][b, j, h // G, c] for n, j in enumerate(js)) / z
                    ls[b, h, i] = m + math.log(z)
        out.append(o)
        lse.append(ls)
    return out, lse


def test_round_bf16_matches_torch_and_ties_to_even():
    x = np.random.default_rng(0).standard_normal(10000) * 3
    want = torch.from_numpy(x).float().to(torch.bfloat16).double().numpy()
    assert np.array_equal(A.round_bf16(x), want)
    # 1 + 2^-8 is exactly half way between 1 and 1 + 2^-7: ties to even -> 1
    assert A.round_bf16(np.array([1.0 + 2.0 ** -8]))[0] == 1.0
    assert A.round_bf16(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 1.0 + 2 * 2.0 ** -7


@pytest.mark.parametrize("causal", [True, False])
def test_forward_brute_force_tiny(causal):
    donor = [0, 0, 2]
    q, k, v = make(3, 2, 5, 4, 2, 3, donor, seed=1)
    o, lse = A.attn_fwd(q, k, v, donor, causal=causal)
    bo, bl = brute_forward(q, k, v, donor, causal, 1 / math.sqrt(3))
    for l in range(3):
        assert np.allclose(o[l], bo[l], rtol=0, atol=1e-12)
        assert np.allclose(lse[l], bl[l], rtol=0, atol=1e-12)


def torch_sdpa(q, k, v, causal, scale=None):
    """Library third opinion: torch fp64 scaled-dot-product attention, KV heads repeated."""
    tq = torch.from_numpy(q).permute(0, 2, 1, 3)
    G = q.shape[2] // k.shape[2]
    tk = torch.from_numpy(k).permute(0, 2, 1, 3).repeat_interleave(G, dim=1)
    tv = torch.from_numpy(v).permute(0, 2, 1, 3).repeat_interleave(G, dim=1)
    o = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=causal, scale=scale)
    return o.permute(0, 2, 1, 3).numpy()


def test_identity_donor_is_standard_attention_vs_library():
    donor = [0, 1]
    q, k, v = make(2, 2, 70, 4, 2, 16, donor, seed=2)
    o, _ = A.attn_fwd(q, k, v, donor, causal=True)
    for l in range(2):
        assert np.allclose(o[l], torch_sdpa(q[l], k[l], v[l], True), atol=1e-12)
    o, _ = A.attn_fwd(q, k, v, donor, causal=False, scale=0.3)
    for l in range(2):
        assert np.allclose(o[l], torch_sdpa(q[l], k[l], v[l], False, 0.3), atol=1e-12)


def test_consumer_equals_standard_attention_on_copy_of_donor_kv():
    donor = [0, 0, 2, 2, 2]
    q, k, v = make(5, 1, 33, 4, 2, 8, donor, seed=3)
    o, lse = A.attn_fwd(q, k, v, donor)
    for l in range(5):
        d = donor[l]
        assert np.allclose(o[l], torch_sdpa(q[l], k[d].copy(), v[d].copy(), True), atol=1e-12)
        # and against the oracle itself run as a one-layer standard stack
        o1, l1 = A.attn_fwd([q[l]], [k[d].copy()], [v[d].copy()], [0])
        assert np.array_equal(o1[0], o[l]) and np.array_equal(l1[0], lse[l])


def test_rows_sum_to_one_and_causal_invariance():
    donor = [0, 0]
    q, k, v = make(2, 1, 40, 2, 1, 8, donor, seed=4)
    ones = [np.ones_like(v[0]), None]
    o, _ = A.attn_fwd(q, k, ones, donor)      # O = P @ 1 = row sums
    assert np.allclose(o[0], 1.0, atol=1e-14) and np.allclose(o[1], 1.0, atol=1e-14)
    o0, l0 = A.attn_fwd(q, k, v, donor)
    i = 17
    q2 = [x.copy() for x in q]
    k2, v2 = [k[0].copy(), None], [v[0].copy(), None]
    for x in q2:
        x[:, i + 1:] += 5.0
    k2[0][:, i + 1:] -= 3.0
    v2[0][:, i + 1:] *= -2.0
    o1, l1 = A.attn_fwd(q2, k2, v2, donor)
    for l in range(2):
        assert np.array_equal(o0[l][:, :i + 1], o1[l][:, :i + 1])
        assert np.array_equal(l0[l][:, :, :i + 1], l1[l][:, :, :i + 1])


def test_closed_forms():
    donor = [0]
    q, k, v = make(1, 1, 9, 2, 1, 4, donor, seed=5)
    # Q = 0: uniform weights over the visible prefix
    o, lse = A.attn_fwd([np.zeros_like(q[0])], k, v, donor)
    for i in range(9):
        assert np.allclose(o[0][0, i, 0], v[0][0, :i + 1, 0].mean(axis=0), atol=1e-14)
        assert abs(lse[0][0, 0, i] - math.log(i + 1)) < 1e-14
    # S = 1: O = V_0, LSE = the single score
    o, lse = A.attn_fwd([q[0][:, :1]], [k[0][:, :1]], [v[0][:, :1]], donor)
    assert np.allclose(o[0][0, 0, 1], v[0][0, 0, 0])
    assert abs(lse[0][0, 1, 0] - q[0][0, 0, 1] @ k[0][0, 0, 0] / 2.0) < 1e-14
    # adding a vector u to every key shifts row i's scores by q_i.u*scale: O unchanged, LSE shifted
    u = rnd((4,), 6)
    o0, l0 = A.attn_fwd(q, k, v, donor)
    o1, l1 = A.attn_fwd(q, [k[0] + u], v, donor)
    assert np.allclose(o0[0], o1[0], atol=1e-12)
    shift = np.einsum("bshc,c->bhs", q[0], u) / 2.0
    assert np.allclose(l1[0] - l0[0], shift, atol=1e-12)


def test_selected_rows_helper_agrees_with_full():
    donor = [0]
    q, k, v = make(1, 1, 50, 2, 1, 8, donor, seed=7)
    o, lse = A.attn_fwd(q, k, v, donor)
    rows = np.array([0, 1, 31, 49])
    orow, lrow = A.attn_fwd_rows(q[0][0, rows, 1], rows, k[0][0, :, 0], v[0][0, :, 0])
    assert np.allclose(orow, o[0][0, rows, 1], atol=1e-14)
    assert np.allclose(lrow, lse[0][0, 1, rows], atol=1e-14)


# ---------------------------------------------------------------------------
# backward
# ---------------------------------------------------------------------------
def loss_of(x, wq, wk, wv, R, donor, dims):
    B, S, Hq, Hkv, dh = dims
    q, k, v = A.proj_fwd(x, wq, wk, wv, donor, B, S, Hq, Hkv, dh)
    o, _ = A.attn_fwd(q, k, v, donor)
    return sum(float((R[l] * o[l]).sum()) for l in range(len(donor)))


def test_gradients_by_central_finite_differences():
    donor = [0, 0, 2]
    L, B, S, Hq, Hkv, dh, D = 3, 1, 6, 4, 2, 3, 5
    dims = (B, S, Hq, Hkv, dh)
    x = [rnd((B * S, D), 20 + l) for l in range(L)]
    wq = [rnd((Hq * dh, D), 30 + l) * 0.5 for l in range(L)]
    wk = [rnd((Hkv * dh, D), 40 + l) * 0.5 if donor[l] == l else None for l in range(L)]
    wv = [rnd((Hkv * dh, D), 50 + l) * 0.5 if donor[l] == l else None for l in range(L)]
    R = [rnd((B, S, Hq, dh), 60 + l) for l in range(L)]
    q, k, v = A.proj_fwd(x, wq, wk, wv, donor, *dims)
    dq, dk, dv = A.attn_bwd(q, k, v, R, donor)
    dwq, dwk, dwv, dx = A.proj_bwd(x, wq, wk, wv, dq, dk, dv, donor)
    eps = 1e-5
    rng = np.random.default_rng(99)

    def check(arrs, grads, name):
        for l, (a, g) in enumerate(zip(arrs, grads)):
            if a is None:
                assert g is None
                continue
            for _ in range(12):
                idx = tuple(rng.integers(0, n) for n in a.shape)
                old = a[idx]
                a[idx] = old + eps
                lp = loss_of(x, wq, wk, wv, R, donor, dims)
                a[idx] = old - eps
                lm = loss_of(x, wq, wk, wv, R, donor, dims)
                a[idx] = old
                fd = (lp - lm) / (2 * eps)
                assert abs(fd - g[idx]) <= 1e-6 * max(1.0, abs(fd)), (name, l, idx, fd, g[idx])

    check(x, dx, "dx")
    check(wq, dwq, "dwq")
    check(wk, dwk, "dwk")
    check(wv, dwv, "dwv")


def test_backward_vs_torch_autograd_and_group_sum_rule():
    donor = [0, 0, 0]
    q, k, v = make(3, 2, 19, 4, 2, 8, donor, seed=8)
    R = [rnd(q[0].shape, 80 + l) for l in range(3)]
    dq, dk, dv = A.attn_bwd(q, k, v, R, donor)
    # third opinion: torch autograd through its own SDPA on a shared leaf K, V
    tk = torch.from_numpy(k[0]).requires_grad_(True)
    tv = torch.from_numpy(v[0]).requires_grad_(True)
    tqs = [torch.from_numpy(x).requires_grad_(True) for x in q]
    loss = 0
    for l in range(3):
        o = torch.nn.functional.scaled_dot_product_attention(
            tqs[l].permute(0, 2, 1, 3), tk.permute(0, 2, 1, 3).repeat_interleave(2, dim=1),
            tv.permute(0, 2, 1, 3).repeat_interleave(2, dim=1), is_causal=True).permute(0, 2, 1, 3)
        loss = loss + (o * torch.from_numpy(R[l])).sum()
    loss.backward()
    assert np.allclose(dk[0], tk.grad.numpy(), atol=1e-11)
    assert np.allclose(dv[0], tv.grad.numpy(), atol=1e-11)
    for l in range(3):
        assert np.allclose(dq[l], tqs[l].grad.numpy(), atol=1e-11)
    # sum rule: the shared gradient is the sum of separate standard attentions on explicit copies
    sk, sv = np.zeros_like(k[0]), np.zeros_like(v[0])
    for l in range(3):
        _, dk1, dv1 = A.attn_bwd([q[l]], [k[0].copy()], [v[0].copy()], [R[l]], [0])
        sk += dk1[0]
        sv += dv1[0]
    assert np.allclose(sk, dk[0], atol=1e-12) and np.allclose(sv, dv[0], atol=1e-12)
    assert dk[1] is None and dv[2] is None


def test_selected_rows_backward_agrees_with_full_and_with_autograd():
    """attn_bwd_rows (the row-sampled backward the full-size GPU tests call): the contributions of
    all rows add up to the full backward; a subset of rows equals torch autograd of a loss that only
    those rows enter; Q = 0 closed form."""
    donor = [0, 0]
    q, k, v = make(2, 1, 37, 4, 2, 8, donor, seed=11)
    R = [rnd(q[0].shape, 90 + l) for l in range(2)]
    dq, dk, dv = A.attn_bwd(q, k, v, R, donor)
    all_rows = np.arange(37)
    sk, sv = np.zeros((37, 8)), np.zeros((37, 8))
    for l in range(2):
        for hq in (2, 3):  # the two query heads of KV head 1
            dq_r, dk_c, dv_c = A.attn_bwd_rows(q[l][0, :, hq], all_rows, k[0][0, :, 1], v[0][0, :, 1], R[l][0, :, hq])
            assert np.allclose(dq_r, dq[l][0, :, hq], atol=1e-13)
            sk += dk_c
            sv += dv_c
    assert np.allclose(sk, dk[0][0, :, 1], atol=1e-12)
    assert np.allclose(sv, dv[0][0, :, 1], atol=1e-12)
    # a subset of rows, non-causal and causal, against autograd of sum(R_rows * O_rows)
    rows = np.array([0, 5, 17, 36])
    for causal in (True, False):
        tq = torch.from_numpy(q[1][0, :, 3].copy()).requires_grad_(True)
        tk = torch.from_numpy(k[0][0, :, 1].copy()).requires_grad_(True)
        tv = torch.from_numpy(v[0][0, :, 1].copy()).requires_grad_(True)
        s = (tq @ tk.T) / math.sqrt(8)
        if causal:
            s = s.masked_fill(torch.triu(torch.ones(37, 37, dtype=torch.bool), 1), float("-inf"))
        o = torch.softmax(s, dim=1) @ tv
        (o[rows] * torch.from_numpy(R[1][0, rows, 3])).sum().backward()
        dq_r, dk_c, dv_c = A.attn_bwd_rows(q[1][0, rows, 3], rows, k[0][0, :, 1], v[0][0, :, 1], R[1][0, rows, 3],
                                           causal=causal)
        assert np.allclose(dq_r, tq.grad.numpy()[rows], atol=1e-12)
        assert np.allclose(dk_c, tk.grad.numpy(), atol=1e-12)
        assert np.allclose(dv_c, tv.grad.numpy(), atol=1e-12)
    # Q = 0: uniform rows, dK contribution vanishes, dV_j = sum_{i >= j} dO_i / (i + 1)
    g = rnd((6, 3), 12)
    kk, vv = rnd((6, 3), 13), rnd((6, 3), 14)
    _, dk0, dv0 = A.attn_bwd_rows(np.zeros((6, 3)), np.arange(6), kk, vv, g)
    assert np.allclose(dk0, 0.0, atol=1e-15)
    for j in range(6):
        assert np.allclose(dv0[j], sum(g[i] / (i + 1) for i in range(j, 6)), atol=1e-14)


def test_backward_closed_form_zero_queries():
    donor = [0]
    _, k, v = make(1, 1, 7, 1, 1, 3, donor, seed=9)
    g = rnd((1, 7, 1, 3), 10)
    dq, dk, dv = A.attn_bwd([np.zeros((1, 7, 1, 3))], k, v, [g], donor)
    assert np.allclose(dk[0], 0.0, atol=1e-15)
    for j in range(7):
        want = sum(g[0, i, 0] / (i + 1) for i in range(j, 7))
        assert np.allclose(dv[0][0, j, 0], want, atol=1e-14)


def test_out_projection_against_autograd():
    o = rnd((2, 5, 3, 4), 11)
    wo = rnd((7, 12), 12)
    dy = rnd((10, 7), 13)
    to = torch.from_numpy(o).requires_grad_(True)
    tw = torch.from_numpy(wo).requires_grad_(True)
    y = to.reshape(10, 12) @ tw.T
    assert np.allclose(A.out_proj_fwd(o, wo), y.detach().numpy(), atol=1e-13)
    (y * torch.from_numpy(dy)).sum().backward()
    d_o, dwo = A.out_proj_bwd(o, wo, dy)
    assert np.allclose(d_o, to.grad.numpy(), atol=1e-13) and np.allclose(dwo, tw.grad.numpy(), atol=1e-13)


# ---------------------------------------------------------------------------
# decode
# ---------------------------------------------------------------------------
def test_decode_step_is_last_row_of_causal_prefill():
    donor = [0, 0, 2, 2]
    L, B, S, Hq, Hkv, dh, D = 4, 2, 12, 4, 2, 4, 6
    x = [rnd((B * (S + 3), D), 100 + l) for l in range(L)]
    wq = [rnd((Hq * dh, D), 110 + l) for l in range(L)]
    wk = [rnd((Hkv * dh, D), 120 + l) if donor[l] == l else None for l in range(L)]
    wv = [rnd((Hkv * dh, D), 130 + l) if donor[l] == l else None for l in range(L)]
    q, k, v = A.proj_fwd(x, wq, wk, wv, donor, B, S + 3, Hq, Hkv, dh)
    o_full, lse_full = A.attn_fwd(q, k, v, donor)
    cap = S + 3
    kc = [np.zeros((B, cap, Hkv, dh)) if donor[l] == l else None for l in range(L)]
    vc = [np.zeros((B, cap, Hkv, dh)) if donor[l] == l else None for l in range(L)]
    for l in A.owners(donor):
        kc[l][:, :S] = k[l][:, :S]
        vc[l][:, :S] = v[l][:, :S]
    lengths = [S] * B
    xr = [a.reshape(B, S + 3, D) for a in x]
    for t in range(3):
        _, o, lse = A.decode_step([a[:, S + t] for a in xr], wq, wk, wv, kc, vc, lengths, donor, Hq, Hkv, dh)
        for l in range(L):
            assert np.allclose(o[l], o_full[l][:, S + t], atol=1e-12)
            assert np.allclose(lse[l], lse_full[l][:, :, S + t], atol=1e-12)
    assert lengths == [S + 3] * B


def test_decode_ragged_lengths_ignore_stale_cache_tail():
    donor = [0, 0]
    B, Hq, Hkv, dh, cap = 3, 4, 2, 8, 20
    q = [rnd((B, Hq, dh), 200 + l) for l in range(2)]
    kc = [rnd((B, cap, Hkv, dh), 210), None]
    vc = [rnd((B, cap, Hkv, dh), 211), None]
    lengths = [1, 7, 20]
    o, lse = A.decode_attend(q, kc, vc, lengths, donor)
    kc2, vc2 = [kc[0].copy(), None], [vc[0].copy(), None]
    for b, n in enumerate(lengths):
        kc2[0][b, n:] = 1e3
        vc2[0][b, n:] = -1e3
    o2, lse2 = A.decode_attend(q, kc2, vc2, lengths, donor)
    for l in range(2):
        assert np.array_equal(o[l], o2[l]) and np.array_equal(lse[l], lse2[l])
    # length 1: output is the single value row
    assert np.allclose(o[1][0, 3], vc[0][0, 0, 1])
