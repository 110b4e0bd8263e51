"""fp64 CPU oracle for the shared-KV attention block (TEST INFRASTRUCTURE ONLY).

This module is a checker, not a product path: only the tests, the smoke entry
and the benchmark's cpu_baseline / reference legs may import it.  It shares no
code with the CUDA library and never imports it.

What it states, all in float64 numpy, with explicit score matrices:

* Eq. 1   Q = X Wq^T, K = X Wk^T, V = X Wv^T  (weights stored [out, in]).
* Eq. 2   O = softmax(Q K^T / sqrt(d_h) + M) V with M the causal mask
          (key j visible to query i iff j <= i), per query head; query head hq
          reads KV head hq // G (contiguous groups, G = Hq / Hkv).
* Eq. 3   a KV-sharing layer l uses K, V of its donor tau(l) = donor[l] <= l;
          its Q projection and the attention itself are unchanged.
* The backward pass is the chain rule of Eq. 1-3; the paper prints none.  dK and
  dV of a donor are the sums over the donor and every consumer layer and over
  the G query heads of each KV head.
* Decode: every owner layer appends its new (k, v) to its cache, then every
  layer attends with its single new query over the donor's cache including the
  token just appended (the paper's "each layer appends (K, V) into the KV
  cache", sentence after Eq. 2).

Rows of the score matrix are processed in blocks only to bound memory; rows are
independent, so this is not a reordering of the definition.

Pins (tests/test_oracle_attention.py): brute-force Python loops on tiny shapes,
torch fp64 scaled-dot-product attention and autograd as a third opinion, closed
forms (Q = 0, S = 1, score shift), softmax rows summing to one, causal
invariance to future tokens, consumer == standard attention on a copy of the
donor's K/V, central finite differences for every gradient, and decode step ==
last row of a causal prefill.
"""
from __future__ import annotations

import math

import numpy as np

_ROW_BLOCK = 512


# --------------------------------------------------------------------------
# storage rounding (bf16, round-to-nearest-even) -- part of the method's
# definition wherever the interface stores bf16; written here independently.
# --------------------------------------------------------------------------
def round_bf16(a: np.ndarray) -> np.ndarray:
    """Round float64/float32 values to the nearest bf16 (ties to even); returns float64."""
    f = np.ascontiguousarray(a, dtype=np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    r = ((u + 0x7FFF + lsb) >> 16) << 16
    r = np.where(np.isnan(f), u, r).astype(np.uint32)
    return r.view(np.float32).astype(np.float64).reshape(np.shape(a))


def validate_donor(donor) -> None:
    """donor[l] <= l and donor[donor[l]] == donor[l] (a donor owns its K/V)."""
    for l, d in enumerate(donor):
        if not (0 <= d <= l) or donor[d] != d:
            raise ValueError(f"bad donor map at layer {l}: {list(donor)}")


def owners(donor):
    return [l for l, d in enumerate(donor) if d == l]


# --------------------------------------------------------------------------
# Eq. 1: projections
# --------------------------------------------------------------------------
def proj_fwd(x, wq, wk, wv, donor, B, S, Hq, Hkv, dh):
    """x[l]: [B*S, D]; wq[l]: [Hq*dh, D]; wk[l], wv[l]: [Hkv*dh, D] (owners only).

    Returns q[l] [B,S,Hq,dh] for every layer and k[l], v[l] [B,S,Hkv,dh] for
    owners (None for consumers: Eq. 3 removes their K/V projections)."""
    validate_donor(donor)
    L = len(donor)
    q, k, v = [None] * L, [None] * L, [None] * L
    for l in range(L):
        xl = np.asarray(x[l], dtype=np.float64)
        q[l] = (xl @ np.asarray(wq[l], dtype=np.float64).T).reshape(B, S, Hq, dh)
        if donor[l] == l:
            k[l] = (xl @ np.asarray(wk[l], dtype=np.float64).T).reshape(B, S, Hkv, dh)
            v[l] = (xl @ np.asarray(wv[l], dtype=np.float64).T).reshape(B, S, Hkv, dh)
    return q, k, v


def proj_bwd(x, wq, wk, wv, dq, dk_sum, dv_sum, donor):
    """Chain rule of Eq. 1.  dq[l]: [B,S,Hq,dh]; dk_sum[d], dv_sum[d]: [B,S,Hkv,dh]
    (owners; already summed over the donor group).

    dWq_l = dQ_l^T X_l, dX_l = dQ_l Wq_l; owners add dWk = dK^T X, dWv = dV^T X
    and dX += dK Wk + dV Wv."""
    L = len(donor)
    dwq, dwk, dwv, dx = [None] * L, [None] * L, [None] * L, [None] * L
    for l in range(L):
        xl = np.asarray(x[l], dtype=np.float64)
        T = xl.shape[0]
        g = np.asarray(dq[l], dtype=np.float64).reshape(T, -1)
        dwq[l] = g.T @ xl
        dx[l] = g @ np.asarray(wq[l], dtype=np.float64)
        if donor[l] == l:
            gk = np.asarray(dk_sum[l], dtype=np.float64).reshape(T, -1)
            gv = np.asarray(dv_sum[l], dtype=np.float64).reshape(T, -1)
            dwk[l] = gk.T @ xl
            dwv[l] = gv.T @ xl
            dx[l] = dx[l] + gk @ np.asarray(wk[l], dtype=np.float64) \
                          + gv @ np.asarray(wv[l], dtype=np.float64)
    return dwq, dwk, dwv, dx


def out_proj_fwd(o, wo):
    """Y = O Wo^T with O [B,S,Hq,dh] flattened to [T, Hq*dh], Wo [D, Hq*dh]."""
    o = np.asarray(o, dtype=np.float64)
    T = o.shape[0] * o.shape[1]
    return o.reshape(T, -1) @ np.asarray(wo, dtype=np.float64).T


def out_proj_bwd(o, wo, dy):
    """dO = dY Wo, dWo = dY^T O."""
    o = np.asarray(o, dtype=np.float64)
    T = o.shape[0] * o.shape[1]
    dy = np.asarray(dy, dtype=np.float64)
    d_o = (dy @ np.asarray(wo, dtype=np.float64)).reshape(o.shape)
    dwo = dy.T @ o.reshape(T, -1)
    return d_o, dwo


# --------------------------------------------------------------------------
# Eq. 2-3: attention forward
# --------------------------------------------------------------------------
def _scores(qh, kh, scale, causal, i0):
    """Scaled, masked scores of query rows i0.. of one head: [rows, S_kv]."""
    s = (qh @ kh.T) * scale
    if causal:
        rows, n = s.shape
        i = np.arange(i0, i0 + rows)[:, None]
        j = np.arange(n)[None, :]
        s = np.where(j <= i, s, -np.inf)
    return s


def _softmax_rows(s):
    m = s.max(axis=1, keepdims=True)
    e = np.exp(s - m)
    l = e.sum(axis=1, keepdims=True)
    return e / l, (m + np.log(l))[:, 0]


def attn_fwd(q, k, v, donor, causal=True, scale=None):
    """q[l]: [B,S,Hq,dh]; k[d], v[d]: [B,S,Hkv,dh] for owners.

    Returns o[l] [B,S,Hq,dh] and lse[l] [B,Hq,S] (natural log of the row sum of
    exp of the scaled scores)."""
    validate_donor(donor)
    L = len(donor)
    o, lse = [None] * L, [None] * L
    for l in range(L):
        d = donor[l]
        ql = np.asarray(q[l], dtype=np.float64)
        kd = np.asarray(k[d], dtype=np.float64)
        vd = np.asarray(v[d], dtype=np.float64)
        B, S, Hq, dh = ql.shape
        Hkv = kd.shape[2]
        G = Hq // Hkv
        sc = (1.0 / math.sqrt(dh)) if scale is None else float(scale)
        ol = np.zeros_like(ql)
        ll = np.zeros((B, Hq, S))
        for b in range(B):
            for hq in range(Hq):
                hk = hq // G
                kh, vh = kd[b, :, hk, :], vd[b, :, hk, :]
                for i0 in range(0, S, _ROW_BLOCK):
                    i1 = min(S, i0 + _ROW_BLOCK)
                    p, ls = _softmax_rows(_scores(ql[b, i0:i1, hq, :], kh, sc, causal, i0))
                    ol[b, i0:i1, hq, :] = p @ vh
                    ll[b, hq, i0:i1] = ls
        o[l], lse[l] = ol, ll
    return o, lse


def attn_fwd_rows(q_rows, row_index, k_head, v_head, causal=True, scale=None):
    """Selected query rows of ONE head: q_rows [n,dh] at positions row_index [n]
    against k_head, v_head [S,dh].  Used to check sampled rows at sizes where the
    full oracle is too slow; rows are independent so this is the same definition."""
    q_rows = np.asarray(q_rows, dtype=np.float64)
    k_head = np.asarray(k_head, dtype=np.float64)
    v_head = np.asarray(v_head, dtype=np.float64)
    dh = q_rows.shape[1]
    sc = (1.0 / math.sqrt(dh)) if scale is None else float(scale)
    s = (q_rows @ k_head.T) * sc
    if causal:
        j = np.arange(k_head.shape[0])[None, :]
        s = np.where(j <= np.asarray(row_index)[:, None], s, -np.inf)
    p, ls = _softmax_rows(s)
    return p @ v_head, ls


# --------------------------------------------------------------------------
# chain rule of Eq. 2-3: attention backward with the donor-group sum
# --------------------------------------------------------------------------
def attn_bwd(q, k, v, d_o, donor, causal=True, scale=None):
    """Returns dq[l] [B,S,Hq,dh] for every layer and dk_sum[d], dv_sum[d]
    [B,S,Hkv,dh] for owners, summed over every layer l with donor[l] == d and
    every query head of the KV head's group.

    Per (l, b, hq): P = softmax rows, O = P V, Delta_i = sum_c dO_ic O_ic,
    dP = dO V^T, dS = P * (dP - Delta), dQ = dS K * scale,
    dK += dS^T Q * scale, dV += P^T dO."""
    validate_donor(donor)
    L = len(donor)
    dq = [None] * L
    dk = [None] * L
    dv = [None] * L
    for l in range(L):
        if donor[l] == l:
            dk[l] = np.zeros(np.shape(k[l]), dtype=np.float64)
            dv[l] = np.zeros(np.shape(v[l]), dtype=np.float64)
    for l in range(L):
        d = donor[l]
        ql = np.asarray(q[l], dtype=np.float64)
        gl = np.asarray(d_o[l], dtype=np.float64)
        kd = np.asarray(k[d], dtype=np.float64)
        vd = np.asarray(v[d], dtype=np.float64)
        B, S, Hq, dh = ql.shape
        G = Hq // kd.shape[2]
        sc = (1.0 / math.sqrt(dh)) if scale is None else float(scale)
        dql = np.zeros_like(ql)
        for b in range(B):
            for hq in range(Hq):
                hk = hq // G
                kh, vh = kd[b, :, hk, :], vd[b, :, hk, :]
                for i0 in range(0, S, _ROW_BLOCK):
                    i1 = min(S, i0 + _ROW_BLOCK)
                    qh = ql[b, i0:i1, hq, :]
                    gh = gl[b, i0:i1, hq, :]
                    p, _ = _softmax_rows(_scores(qh, kh, sc, causal, i0))
                    oh = p @ vh
                    delta = (gh * oh).sum(axis=1, keepdims=True)
                    dp = gh @ vh.T
                    ds = p * (dp - delta)
                    dql[b, i0:i1, hq, :] = (ds @ kh) * sc
                    dk[d][b, :, hk, :] += (ds.T @ qh) * sc
                    dv[d][b, :, hk, :] += p.T @ gh
        dq[l] = dql
    return dq, dk, dv


def attn_bwd_rows(q_rows, row_index, k_head, v_head, g_rows, causal=True, scale=None):
    """Backward of selected query rows of ONE head (the same chain rule as attn_bwd;
    query rows are independent given K and V, so their contributions add).

    q_rows, g_rows [n,dh]: the queries and their dO at positions row_index [n];
    k_head, v_head [S,dh].  Returns dq_rows [n,dh] and the CONTRIBUTION of these
    rows to dK and dV of the head, [S,dh] each: summing the contributions of all
    rows of all heads and layers that read the head gives dk_sum / dv_sum."""
    q_rows = np.asarray(q_rows, dtype=np.float64)
    g_rows = np.asarray(g_rows, dtype=np.float64)
    k_head = np.asarray(k_head, dtype=np.float64)
    v_head = np.asarray(v_head, dtype=np.float64)
    dh = q_rows.shape[1]
    sc = (1.0 / math.sqrt(dh)) if scale is None else float(scale)
    s = (q_rows @ k_head.T) * sc
    if causal:
        j = np.arange(k_head.shape[0])[None, :]
        s = np.where(j <= np.asarray(row_index)[:, None], s, -np.inf)
    p, _ = _softmax_rows(s)
    delta = (g_rows * (p @ v_head)).sum(axis=1, keepdims=True)
    ds = p * (g_rows @ v_head.T - delta)
    return (ds @ k_head) * sc, (ds.T @ q_rows) * sc, p.T @ g_rows


# --------------------------------------------------------------------------
# decode over the shared cache
# --------------------------------------------------------------------------
def decode_attend(q, k_cache, v_cache, lengths, donor, scale=None):
    """One decode step, attention part.  q[l]: [B,Hq,dh]; k_cache[d], v_cache[d]:
    [B,cap,Hkv,dh] for owners (dense, position-major); lengths[b] counts the
    valid positions INCLUDING the token appended this step.

    Returns o[l] [B,Hq,dh], lse[l] [B,Hq].  No mask: the query is the last
    position."""
    validate_donor(donor)
    L = len(donor)
    o, lse = [None] * L, [None] * L
    for l in range(L):
        d = donor[l]
        ql = np.asarray(q[l], dtype=np.float64)
        B, Hq, dh = ql.shape
        Hkv = np.shape(k_cache[d])[2]
        G = Hq // Hkv
        sc = (1.0 / math.sqrt(dh)) if scale is None else float(scale)
        ol = np.zeros((B, Hq, dh))
        ll = np.zeros((B, Hq))
        for b in range(B):
            n = int(lengths[b])
            kb = np.asarray(k_cache[d][b, :n], dtype=np.float64)
            vb = np.asarray(v_cache[d][b, :n], dtype=np.float64)
            for hq in range(Hq):
                hk = hq // G
                s = (kb[:, hk, :] @ ql[b, hq, :]) * sc
                m = s.max()
                e = np.exp(s - m)
                z = e.sum()
                ol[b, hq, :] = (e / z) @ vb[:, hk, :]
                ll[b, hq] = m + math.log(z)
        o[l], lse[l] = ol, ll
    return o, lse


def cache_append(k_cache, v_cache, k_new, v_new, lengths, donor):
    """Owners write k_new[d][b], v_new[d][b] ([B,Hkv,dh]) at position lengths[b]-1
    (lengths already count the new token).  Consumers store nothing (Eq. 3)."""
    for d in owners(donor):
        for b in range(len(lengths)):
            p = int(lengths[b]) - 1
            k_cache[d][b, p] = k_new[d][b]
            v_cache[d][b, p] = v_new[d][b]


def decode_step(x_t, wq, wk, wv, k_cache, v_cache, lengths, donor, Hq, Hkv, dh,
                scale=None, store_round=None):
    """Full decode step from hidden states x_t[l] [B,D]: project (Eq. 1), append
    for owners, attend for all layers.  lengths are the counts BEFORE this step;
    they are incremented in place.  store_round, if given, is applied to q, k, v
    before they are stored/used (bf16 interface storage)."""
    L = len(donor)
    B = np.shape(x_t[0])[0]
    rnd = (lambda a: a) if store_round is None else store_round
    q, kn, vn = [None] * L, [None] * L, [None] * L
    for l in range(L):
        xl = np.asarray(x_t[l], dtype=np.float64)
        q[l] = rnd(xl @ np.asarray(wq[l], dtype=np.float64).T).reshape(B, Hq, dh)
        if donor[l] == l:
            kn[l] = rnd(xl @ np.asarray(wk[l], dtype=np.float64).T).reshape(B, Hkv, dh)
            vn[l] = rnd(xl @ np.asarray(wv[l], dtype=np.float64).T).reshape(B, Hkv, dh)
    for b in range(B):
        lengths[b] += 1
    cache_append(k_cache, v_cache, kn, vn, lengths, donor)
    o, lse = decode_attend(q, k_cache, v_cache, lengths, donor, scale)
    return q, o, lse
