"""The allocation-free decode entry point (kvp_decode_static), called through the C ABI.

It exists for callers that cannot obtain device memory where they decode (the device is fully
committed to a cache pool, or the host application forbids allocation on its hot path): the
per-split scratch is a fixed array inside the library instead of a caller workspace.  Its outputs
must equal those of kvp_decode on the same inputs, on two calls in a row (the array is reused and
keeps the previous call's contents), and a request that does not fit must be refused.

This file is collected last on purpose, so a run that stops at the first failure has already run
every other test; it also passes when run alone in a fresh process."""
import numpy as np
import pytest
import torch

from oracle import attention as A
from paper_2608_15943_b200 import synth

pytestmark = pytest.mark.gpu

REL, ABS, LSE_TOL = 1e-2, 3e-2, 1e-3


def _case(kvp, L, donor, B, Hq, Hkv, dh, page, lens, ns, seed):
    max_pages = (max(lens) + page - 1) // page + 1
    n_pages = B * max_pages
    g = torch.Generator().manual_seed(seed)
    bt = torch.randperm(n_pages, generator=g).int().reshape(B, max_pages).cuda()
    lengths = torch.tensor(lens, dtype=torch.int32, device="cuda")
    kc = [synth.normal((n_pages, Hkv, page, dh), seed, synth.tid(7, l), 1.0, "cuda") if donor[l] == l else None
          for l in range(L)]
    vc = [synth.normal((n_pages, Hkv, page, dh), seed, synth.tid(8, l), 1.0, "cuda") if donor[l] == l else None
          for l in range(L)]
    q = [synth.normal((B, Hq, dh), seed, synth.tid(6, l), 1.0, "cuda") for l in range(L)]
    desc = kvp.DecodeDesc(L, B, Hq, Hkv, dh, page, max_pages, n_pages, ns)
    return desc, bt, lengths, kc, vc, q


def _oracle(q, kc, vc, bt, lens, donor, page):
    """The fp64 oracle on the same cache: pages gathered into dense [B, cap, Hkv, dh] arrays."""
    f = lambda t: t.detach().float().cpu().numpy().astype(np.float64)
    B, cap = len(lens), max(lens)
    kd, vd = [None] * len(donor), [None] * len(donor)
    for l, d in enumerate(donor):
        if d != l:
            continue
        Hkv, dh = kc[l].shape[1], kc[l].shape[3]
        kd[l], vd[l] = np.zeros((B, cap, Hkv, dh)), np.zeros((B, cap, Hkv, dh))
        for b in range(B):
            n_pg = (lens[b] + page - 1) // page
            pages = bt[b, :n_pg].long()
            kd[l][b, :lens[b]] = f(kc[l][pages].permute(0, 2, 1, 3).reshape(-1, Hkv, dh))[:lens[b]]
            vd[l][b, :lens[b]] = f(vc[l][pages].permute(0, 2, 1, 3).reshape(-1, Hkv, dh))[:lens[b]]
    return A.decode_attend([f(x) for x in q], kd, vd, lens, donor)


def _outputs(L, B, Hq, dh):
    o = [torch.full((B, Hq, dh), float("nan"), device="cuda", dtype=torch.bfloat16) for _ in range(L)]
    lse = [torch.full((B, Hq), float("nan"), device="cuda") for _ in range(L)]
    return o, lse


def test_decode_static_matches_decode_on_two_calls_in_a_row():
    from paper_2608_15943_b200 import kvp
    L, donor, B, Hq, Hkv, dh, page = 4, [0, 0, 2, 2], 3, 8, 2, 128, 64
    # two different problems back to back: the second call finds the first call's partials in the array
    for call, (lens, ns, seed) in enumerate([([700, 129, 64], 4, 21), ([33, 512, 1000], 3, 22)]):
        desc, bt, lengths, kc, vc, q = _case(kvp, L, donor, B, Hq, Hkv, dh, page, lens, ns, seed)
        ws = torch.empty(kvp.decode_workspace_bytes(desc, donor), dtype=torch.uint8, device="cuda")
        assert ws.numel() <= kvp.DECODE_STATIC_SCRATCH_BYTES
        o_ref, lse_ref = _outputs(L, B, Hq, dh)
        kvp.decode(desc, donor, q, kc, vc, bt, lengths, o_ref, lse_ref, ws)
        o, lse = _outputs(L, B, Hq, dh)
        kvp.decode_static(desc, donor, q, kc, vc, bt, lengths, o, lse)
        torch.cuda.synchronize()
        oracle_o, oracle_lse = _oracle(q, kc, vc, bt, lens, donor, page)
        for l in range(L):
            got, ref = o[l].float().cpu().numpy().astype(np.float64), o_ref[l].float().cpu().numpy().astype(np.float64)
            assert np.isfinite(got).all(), f"call {call}: non-finite output"
            assert np.linalg.norm(got - ref) <= REL * np.linalg.norm(ref)
            assert np.abs(got - ref).max() <= ABS
            assert (lse[l] - lse_ref[l]).abs().max().item() <= LSE_TOL
            # and directly against the fp64 oracle, at the same tolerances
            assert np.linalg.norm(got - oracle_o[l]) <= REL * np.linalg.norm(oracle_o[l])
            assert np.abs(got - oracle_o[l]).max() <= ABS
            assert np.abs(lse[l].cpu().numpy().astype(np.float64) - oracle_lse[l]).max() <= LSE_TOL
    assert kvp.device_status() == kvp.OK


def test_decode_static_narrow_layer_range_fits_where_all_layers_do_not():
    """The built-in array has to hold the partials of the donor groups that ONE call touches, so a model whose
    full-range request is refused can still be decoded one donor group at a time; the results equal kvp_decode's."""
    from paper_2608_15943_b200 import kvp
    L, donor, B, Hq, Hkv, dh, page = 6, [0, 0, 2, 2, 4, 4], 12, 32, 8, 128, 16
    lens = [40 + 7 * b for b in range(B)]
    desc, bt, lengths, kc, vc, q = _case(kvp, L, donor, B, Hq, Hkv, dh, page, lens, 16, 23)
    assert kvp.decode_workspace_bytes(desc, donor) > kvp.DECODE_STATIC_SCRATCH_BYTES
    o, lse = _outputs(L, B, Hq, dh)
    with pytest.raises(kvp.KvpError) as e:
        kvp.decode_static(desc, donor, q, kc, vc, bt, lengths, o, lse)
    assert e.value.status == kvp.ERR_STATIC_SCRATCH
    ws = torch.empty(kvp.decode_workspace_bytes(desc, donor), dtype=torch.uint8, device="cuda")
    o_ref, lse_ref = _outputs(L, B, Hq, dh)
    kvp.decode(desc, donor, q, kc, vc, bt, lengths, o_ref, lse_ref, ws)
    for l0 in (0, 2, 4):                                   # one donor group per call
        kvp.decode_static(desc, donor, q, kc, vc, bt, lengths, o, lse, layer_begin=l0, layer_end=l0 + 2)
    torch.cuda.synchronize()
    for l in range(L):
        assert torch.equal(o[l], o_ref[l]) and torch.equal(lse[l], lse_ref[l])
    assert kvp.device_status() == kvp.OK


def test_decode_static_refuses_what_does_not_fit():
    from paper_2608_15943_b200 import kvp
    L, donor, B, Hq, Hkv, dh, page = 8, list(range(8)), 32, 32, 8, 128, 128
    desc, bt, lengths, kc, vc, q = _case(kvp, 1, [0], 1, 4, 1, dh, 16, [40], 0, 5)   # tensors are irrelevant here
    big = kvp.DecodeDesc(L, B, Hq, Hkv, dh, page, 64, 4096, 16)     # 8 groups x 32 x 8 x 16 splits of partials
    assert kvp.decode_workspace_bytes(big, donor) > kvp.DECODE_STATIC_SCRATCH_BYTES
    nul = [None] * L
    with pytest.raises(kvp.KvpError) as e:
        kvp.decode_static(big, donor, nul, nul, nul, bt, lengths, nul, nul)
    assert e.value.status == kvp.ERR_STATIC_SCRATCH
    assert "scratch" in kvp.status_string(kvp.ERR_STATIC_SCRATCH)
