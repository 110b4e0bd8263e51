"""Benchmark / test workloads: shapes, seeded synthetic inputs and output buffers.

Nothing here computes any part of the method; it names the configurations, allocates device
memory with torch and fills inputs through ``synth``.  The shapes follow the LLaMA-3-8B-like
attention geometry (d_model 4096, 32 query / 8 KV heads, head_dim 128) the paper's GQA experiments
use; the data are seeded Gaussians (activations ~N(0,1), weights ~N(0,0.02^2)) standing in for the
paper's training text and pretrained weights, which are not needed for throughput or parity.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional

import torch

from . import synth

SEED = synth.DEFAULT_SEED


@dataclass
class TrainCfg:
    name: str
    L: int
    B: int
    S: int
    D: int
    Hq: int
    Hkv: int
    dh: int
    donor: List[int]

    @property
    def T(self) -> int:
        return self.B * self.S

    def owners(self) -> List[int]:
        return [l for l, d in enumerate(self.donor) if d == l]

    # algorithmic FLOPs (a MAC counts 2; causal attention counts the S(S+1)/2 visible pairs)
    def proj_fwd_flops(self) -> int:
        f = 0
        for l, d in enumerate(self.donor):
            f += 2 * self.T * self.D * self.Hq * self.dh
            if d == l:
                f += 2 * 2 * self.T * self.D * self.Hkv * self.dh
        return f

    def attn_fwd_flops(self) -> int:
        pairs = self.S * (self.S + 1) // 2
        return self.L * 4 * self.dh * pairs * self.B * self.Hq

    def step_flops_model(self) -> int:
        """forward + backward, backward counted as 2x forward (4 attention GEMMs, dX and dW)."""
        return 3 * (self.proj_fwd_flops() + self.attn_fwd_flops())


C0 = TrainCfg("C0-tiny", 4, 2, 128, 256, 4, 2, 64, [0, 0, 2, 2])
C1 = TrainCfg("C1-prefill-B4-S4096", 8, 4, 4096, 4096, 32, 8, 128, [0, 1, 2, 3, 4, 4, 4, 4])
C2 = TrainCfg("C2-train-B2-S8192", 8, 2, 8192, 4096, 32, 8, 128, [0, 1, 2, 3, 4, 4, 4, 4])
# reduced shapes of the same kernels for profiler captures (inputs larger than L2, < 2 GB live)
SMALL_TRAIN = TrainCfg("small-train-B1-S4096", 2, 1, 4096, 4096, 32, 8, 128, [0, 0])
# tail pipeline stage of the 32-layer / PP=8 plan, batch 8 x 4096 tokens
C4_UNCONVERTED = TrainCfg("C4-stage-unconverted", 4, 8, 4096, 4096, 32, 8, 128, [0, 1, 2, 3])
C4_STAGE_LOCAL = TrainCfg("C4-stage-local-donor", 4, 8, 4096, 4096, 32, 8, 128, [0, 0, 0, 0])


def make_train_inputs(cfg: TrainCfg, device, seed: int = SEED, with_out_proj: bool = False) -> dict:
    """x[l] [T,D], wq[l] [Hq*dh,D], wk/wv[l] [Hkv*dh,D] (owners), d_o[l] [B,S,Hq,dh]; bf16."""
    own = set(cfg.owners())
    nq, nkv = cfg.Hq * cfg.dh, cfg.Hkv * cfg.dh
    t = dict(x=[], wq=[], wk=[], wv=[], d_o=[])
    for l in range(cfg.L):
        t["x"].append(synth.normal((cfg.T, cfg.D), seed, synth.tid(0, l), 1.0, device))
        t["wq"].append(synth.normal((nq, cfg.D), seed, synth.tid(1, l), 0.02, device))
        t["wk"].append(synth.normal((nkv, cfg.D), seed, synth.tid(2, l), 0.02, device) if l in own else None)
        t["wv"].append(synth.normal((nkv, cfg.D), seed, synth.tid(3, l), 0.02, device) if l in own else None)
        t["d_o"].append(synth.normal((cfg.B, cfg.S, cfg.Hq, cfg.dh), seed, synth.tid(5, l), 1.0, device))
    if with_out_proj:
        t["wo"] = [synth.normal((cfg.D, nq), seed, synth.tid(4, l), 0.02, device) for l in range(cfg.L)]
        t["dy"] = [synth.normal((cfg.T, cfg.D), seed, synth.tid(11, l), 1.0, device) for l in range(cfg.L)]
    return t


def alloc_train_outputs(cfg: TrainCfg, device, with_out_proj: bool = False) -> dict:
    own = set(cfg.owners())
    bf, f32 = torch.bfloat16, torch.float32
    nq, nkv = cfg.Hq * cfg.dh, cfg.Hkv * cfg.dh

    def per_layer(shape, dtype, owners_only=False):
        return [torch.empty(shape, dtype=dtype, device=device) if (not owners_only or l in own) else None
                for l in range(cfg.L)]

    o = dict(q=per_layer((cfg.B, cfg.S, cfg.Hq, cfg.dh), bf), k=per_layer((cfg.B, cfg.S, cfg.Hkv, cfg.dh), bf, True),
             v=per_layer((cfg.B, cfg.S, cfg.Hkv, cfg.dh), bf, True), o=per_layer((cfg.B, cfg.S, cfg.Hq, cfg.dh), bf),
             lse=per_layer((cfg.B, cfg.Hq, cfg.S), f32), dq=per_layer((cfg.B, cfg.S, cfg.Hq, cfg.dh), bf),
             dk_sum=per_layer((cfg.B, cfg.S, cfg.Hkv, cfg.dh), f32, True),
             dv_sum=per_layer((cfg.B, cfg.S, cfg.Hkv, cfg.dh), f32, True), dwq=per_layer((nq, cfg.D), f32),
             dwk=per_layer((nkv, cfg.D), f32, True), dwv=per_layer((nkv, cfg.D), f32, True),
             dx=per_layer((cfg.T, cfg.D), bf))
    if with_out_proj:
        o["y"] = per_layer((cfg.T, cfg.D), bf)
        o["dwo"] = per_layer((cfg.D, nq), f32)
    return o


# ---------------------------------------------------------------------------------------------
# decode
# ---------------------------------------------------------------------------------------------
@dataclass
class DecodeCfg:
    name: str
    L: int
    B: int
    Hq: int
    Hkv: int
    dh: int
    page: int
    len_lo: int
    len_hi: int
    donor: List[int]
    steps: int
    headroom: int = 256   # tokens of capacity beyond len_hi

    def owners(self) -> List[int]:
        return [l for l, d in enumerate(self.donor) if d == l]

    @property
    def max_pages(self) -> int:
        return (self.len_hi + self.headroom + self.page - 1) // self.page


def pair_donor(L: int, first_shared: int) -> List[int]:
    """Layers below first_shared own their K/V; above, odd layers share the even layer below them."""
    return [l if (l < first_shared or (l - first_shared) % 2 == 0) else l - 1 for l in range(L)]


C3 = DecodeCfg("C3-decode-B32-16k-32k", 32, 32, 32, 8, 128, 128, 16384, 32768, pair_donor(32, 16), 256)
SMALL_DECODE = DecodeCfg("small-decode-B8-8k-16k", 4, 8, 32, 8, 128, 128, 8192, 16384, [0, 0, 2, 2], 8)
C3_UNSHARED = DecodeCfg("C3-decode-unshared", 32, 32, 32, 8, 128, 128, 16384, 32768, list(range(32)), 256)


@dataclass
class DecodeState:
    cfg: DecodeCfg
    lengths0: torch.Tensor            # CPU int32 [B], context lengths before the first step
    lengths: torch.Tensor             # device int32 [B]
    block_table: torch.Tensor         # device int32 [B, max_pages]
    n_pages: int
    k_cache: List[Optional[torch.Tensor]]
    v_cache: List[Optional[torch.Tensor]]
    slot_of: List[int] = field(default_factory=list)   # physical pool slot of each owner layer
    seed: int = SEED


def make_decode_state(cfg: DecodeCfg, device, seed: int = SEED, n_slots: Optional[int] = None,
                      shuffle_pages: bool = False) -> DecodeState:
    """Paged cache pools [n_pages, Hkv, page, dh] per owner layer, filled procedurally; each
    sequence gets enough pages for len + steps tokens.  With n_slots < number of owners the owner
    layers are mapped cyclically onto n_slots physical pools (traffic per step is unchanged)."""
    lengths0 = synth.uniform_ints(cfg.B, cfg.len_lo, cfg.len_hi, seed, synth.tid(9))
    need = [(int(n) + cfg.steps + cfg.page - 1) // cfg.page for n in lengths0]
    n_pages = sum(need)
    bt = torch.zeros(cfg.B, cfg.max_pages, dtype=torch.int32)
    order = torch.arange(n_pages, dtype=torch.int32)
    if shuffle_pages:
        key = synth.table_index(seed, synth.tid(12), torch.arange(n_pages, dtype=torch.int64)) * 65536 + \
            synth.table_index(seed, synth.tid(12, 1), torch.arange(n_pages, dtype=torch.int64))
        order = torch.argsort(key).to(torch.int32)
    pid = 0
    for b in range(cfg.B):
        bt[b, :need[b]] = order[pid:pid + need[b]]
        pid += need[b]
    own = cfg.owners()
    n_slots = len(own) if n_slots is None else min(n_slots, len(own))
    pools_k, pools_v = [], []
    for s in range(n_slots):
        pools_k.append(synth.normal((n_pages, cfg.Hkv, cfg.page, cfg.dh), seed, synth.tid(7, s), 1.0, device))
        pools_v.append(synth.normal((n_pages, cfg.Hkv, cfg.page, cfg.dh), seed, synth.tid(8, s), 1.0, device))
    k_cache: List[Optional[torch.Tensor]] = [None] * cfg.L
    v_cache: List[Optional[torch.Tensor]] = [None] * cfg.L
    slot_of = []
    for i, l in enumerate(own):
        k_cache[l] = pools_k[i % n_slots]
        v_cache[l] = pools_v[i % n_slots]
        slot_of.append(i % n_slots)
    return DecodeState(cfg, lengths0, lengths0.to(device), bt.to(device), n_pages, k_cache, v_cache, slot_of, seed)


def decode_queries(cfg: DecodeCfg, device, seed: int, step: int) -> List[torch.Tensor]:
    return [synth.normal((cfg.B, cfg.Hq, cfg.dh), seed, synth.tid(6, l, step), 1.0, device) for l in range(cfg.L)]


def decode_step_bytes(cfg: DecodeCfg, lengths) -> int:
    """Algorithmic HBM bytes of one decode step: every stored (owner) layer's K and V rows of every
    sequence read once, plus queries and outputs."""
    kv = sum(int(n) for n in lengths) * 2 * cfg.Hkv * cfg.dh * 2 * len(cfg.owners())
    qo = 2 * cfg.L * cfg.B * cfg.Hq * cfg.dh * 2
    return kv + qo
