#!/usr/bin/env python
"""Benchmark of the shared-KV attention block on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload train|prefill|decode|stage]
                    [--impl ours|reference] [--no-decode] [--no-cpu-baseline]

Default (no flags): N=1, the training step of the Llama-like block (8 layers, donor map
[0,1,2,3,4,4,4,4], batch 2 x 8192 tokens, bf16): Q / K / V projections, causal flash-attention
forward, backward with the donor-group dK/dV sum, projection backward -- one "step" is one pass
of all of these over one batch.  The decode workload (32 layers, batch 32, 16k-32k contexts,
256 steps over the shared paged cache) is timed in the same run and reported under "decode".
One JSON line is printed by rank 0.  `--impl reference` times the fp64 CPU oracle on a bounded
sample of the same workload instead.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2608_15943_b200 import dist as kdist          # noqa: E402
from paper_2608_15943_b200 import synth                   # noqa: E402
from paper_2608_15943_b200 import workloads as W          # noqa: E402

NOMINAL_BF16_TFLOPS = 2250.0
NOMINAL_HBM_GBS = 8000.0
# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum): STORED CONSTANTS, not measured by this
# program.  They come from ncu captures of the small case of each kernel, scaled to a full-size launch by the units
# one launch processes (traffic grows in proportion); the committed profile summaries give the captures and dates.
NCU_TRAFFIC_BYTES = {"bwd_kernel": 7.45e9, "attn_fwd_kernel": 0.474e9, "decode_kernel": 77.96e9}
NCU_TRAFFIC_NOTE = "bytes per launch; a stored constant from an earlier ncu capture, not measured in this run"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            d = json.load(fh)
        return d, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


# ---------------------------------------------------------------------------------------------
# clocks during the timed region (read-only NVML queries)
# ---------------------------------------------------------------------------------------------
class ClockSampler:
    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self._h = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            vis = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = int(vis.split(",")[index]) if vis and vis.split(",")[index].isdigit() else index
            self._h = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self._h = None

    def _loop(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h)
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(0.05)

    def __enter__(self):
        if self._h is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": 0}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def timed_region(fn, steps, device, sampler_index):
    """barrier + synchronize, CUDA events around `steps` calls, synchronize + barrier; ms total (max over ranks)."""
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    kdist.barrier()
    torch.cuda.synchronize()
    with ClockSampler(sampler_index) as cs:
        e0.record()
        for i in range(steps):
            fn(i)
        e1.record()
        torch.cuda.synchronize()
    kdist.barrier()
    ms = kdist.max_over_ranks(e0.elapsed_time(e1), device)
    return ms, cs.summary()


# ---------------------------------------------------------------------------------------------
# training / prefill / stage workloads
# ---------------------------------------------------------------------------------------------
class TrainRunner:
    def __init__(self, kvp, cfg: W.TrainCfg, device, backward=True, out_proj=False, bucket=True):
        self.kvp, self.cfg, self.device, self.backward, self.out_proj = kvp, cfg, device, backward, out_proj
        self.t = W.make_train_inputs(cfg, device, with_out_proj=out_proj)
        self.out = W.alloc_train_outputs(cfg, device, with_out_proj=out_proj)
        self.sh = kvp.Shape(cfg.L, cfg.B, cfg.S, cfg.D, cfg.Hq, cfg.Hkv, cfg.dh)
        nq, nkv = cfg.Hq * cfg.dh, cfg.Hkv * cfg.dh
        own = set(cfg.owners())
        if backward and bucket:   # weight gradients live in one flat bucket, each layer's entries next to each other
            shapes = [(nq, cfg.D)] * cfg.L + [(nkv, cfg.D) if l in own else None for l in range(cfg.L)] * 2
            layer_of = list(range(cfg.L)) * 3
            if out_proj:
                shapes += [(cfg.D, nq)] * cfg.L
                layer_of += list(range(cfg.L))
            self.bucket = kdist.GradBucket(shapes, device, layer_of=layer_of)
            v = self.bucket.views
            self.out["dwq"], self.out["dwk"], self.out["dwv"] = v[:cfg.L], v[cfg.L:2 * cfg.L], v[2 * cfg.L:3 * cfg.L]
            if out_proj:
                self.out["dwo"] = v[3 * cfg.L:4 * cfg.L]
            if kdist.is_multi():   # the cross-rank sum runs layer by layer on its own stream, behind the gradient GEMMs
                self.s_comm = torch.cuda.Stream()
                self.ev_layer = [torch.cuda.Event() for _ in range(cfg.L)]
        else:
            self.bucket = None
        ws = max(kvp.workspace_bytes(kvp.OP_ATTN_BWD, self.sh, cfg.donor),
                 kvp.workspace_bytes(kvp.OP_PROJ_BWD, self.sh, cfg.donor), 256) if backward else 256
        self.ws = torch.empty(ws, dtype=torch.uint8, device=device)
        if out_proj and backward:
            self.d_o = [torch.empty_like(x) for x in self.out["o"]]

    def step(self, _i=0, before_proj_bwd=None):
        k, c, t, o = self.kvp, self.cfg, self.t, self.out
        k.proj_fwd(self.sh, c.donor, t["x"], t["wq"], t["wk"], t["wv"], o["q"], o["k"], o["v"])
        k.attn_fwd(self.sh, c.donor, o["q"], o["k"], o["v"], o["o"], o["lse"])
        if self.out_proj:
            k.out_proj_fwd(self.sh, o["o"], t["wo"], o["y"])
        if not self.backward:
            return
        d_o = t["d_o"]
        if self.out_proj:
            k.out_proj_bwd(self.sh, o["o"], t["wo"], t["dy"], self.d_o, o["dwo"])
            d_o = self.d_o
        k.attn_bwd(self.sh, c.donor, o["q"], o["k"], o["v"], o["o"], d_o, o["lse"], o["dq"], o["dk_sum"],
                   o["dv_sum"], self.ws)
        if before_proj_bwd is not None:
            before_proj_bwd()
        args = (self.sh, c.donor, t["x"], t["wq"], t["wk"], t["wv"], o["dq"], o["dk_sum"], o["dv_sum"], o["dwq"], o["dwk"],
                o["dwv"], o["dx"], self.ws)
        if self.bucket is not None and kdist.is_multi():
            # one layer's gradient GEMMs, then that layer's slice of the bucket is summed over ranks on the side
            # stream while the next layer's GEMMs run: only the last layer's reduction is exposed
            cur = torch.cuda.current_stream()
            for l in range(c.L):
                k.proj_bwd(*args, layer_begin=l, layer_end=l + 1)
                self.ev_layer[l].record(cur)
                with torch.cuda.stream(self.s_comm):
                    self.s_comm.wait_event(self.ev_layer[l])
                    self.bucket.all_reduce_layer(l)
            cur.wait_stream(self.s_comm)
        else:
            k.proj_bwd(*args)

    def flops(self):
        c = self.cfg
        f = c.proj_fwd_flops() + c.attn_fwd_flops()
        if self.out_proj:
            f += c.L * 2 * c.T * c.D * c.Hq * c.dh
        return 3 * f if self.backward else f

    def gemm_flops(self):
        """FLOPs of the projection GEMM launches of one step (forward; backward = dW and dX, 2x)."""
        c = self.cfg
        f = c.proj_fwd_flops() + (c.L * 2 * c.T * c.D * c.Hq * c.dh if self.out_proj else 0)
        return 3 * f if self.backward else f

    def attn_step(self, ins, before_results=None):
        """Attention only (the headline metric's unit of work): forward, then backward, on the q / k / v / dO given."""
        k, c, o = self.kvp, self.cfg, self.out
        if not self.backward and before_results is not None:
            before_results()
        k.attn_fwd(self.sh, c.donor, ins["q"], ins["k"], ins["v"], o["o"], o["lse"])
        if self.backward:
            if before_results is not None:
                before_results()
            k.attn_bwd(self.sh, c.donor, ins["q"], ins["k"], ins["v"], o["o"], ins["d_o"], o["lse"], o["dq"], o["dk_sum"],
                       o["dv_sum"], self.ws)

    # End to end: every step's inputs come from pinned host memory and its results go back to pinned host memory.
    #   mode "attn":  q, k, v (and dO) in; O (forward only) or dQ, dK/dV sums (with backward) out -- the calls a user
    #                 of kvp_attn_fwd / kvp_attn_bwd with host-resident tensors makes;
    #   mode "block": X (and dO) in; O of every layer (forward only) or dX of every layer and the whole weight-gradient
    #                 bucket (with backward) out.
    # The copies are pipelined the way an input loader does it: while step n computes, a second stream brings step
    # n+1's inputs into the other of two device buffer sets, and a third takes step n's results out.  Every call
    # issues exactly one input copy and one result copy and does not return the compute stream until the input
    # copy it issued has landed, so K timed calls contain K input and K result transfers.
    def setup_e2e(self, mode):
        o, t = self.out, self.t
        self.e2e_mode = mode
        if mode == "attn":
            self.step()                          # q, k, v of this batch
            torch.cuda.synchronize()
            cur_in = {"q": o["q"], "k": o["k"], "v": o["v"]}
            if self.backward:
                cur_in["d_o"] = t["d_o"]
            results = (o["dq"] + [x for x in o["dk_sum"] if x is not None] + [x for x in o["dv_sum"] if x is not None]) \
                if self.backward else list(o["o"])
        else:
            cur_in = {"x": t["x"]}
            if self.backward:
                cur_in["dy" if self.out_proj else "d_o"] = t["dy" if self.out_proj else "d_o"]
            results = (list(o["dx"]) + ([self.bucket.flat] if self.bucket is not None else [])) if self.backward \
                else list(o["o"])
        dup = lambda xs: [None if a is None else torch.empty_like(a) for a in xs]
        self.in_sets = [cur_in, {n: dup(xs) for n, xs in cur_in.items()}]
        self.h_in = {n: [None if a is None else a.cpu().pin_memory() for a in xs] for n, xs in cur_in.items()}
        self.results = results
        self.h_out = [torch.empty_like(a, device="cpu").pin_memory() for a in results]
        nb = lambda xs: sum(a.numel() * a.element_size() for a in xs if a is not None)
        self.h2d = sum(nb(xs) for xs in self.h_in.values())
        self.d2h = nb(self.h_out)
        self.s_in, self.s_out = torch.cuda.Stream(), torch.cuda.Stream()
        self.ev_in = [torch.cuda.Event(), torch.cuda.Event()]      # input set filled
        self.ev_free = [torch.cuda.Event(), torch.cuda.Event()]    # input set no longer read
        self.ev_result, self.ev_out = torch.cuda.Event(), torch.cuda.Event()
        self.e2e_calls = 0
        cur = torch.cuda.current_stream()
        self._copy_in(0, after=None)           # the first call's inputs
        cur.wait_event(self.ev_in[0])
        self.ev_out.record(cur)

    def _copy_in(self, which, after):
        with torch.cuda.stream(self.s_in):
            if after is not None:
                self.s_in.wait_event(after)    # the set's previous reader has finished
            for n, hs in self.h_in.items():
                for dst, src in zip(self.in_sets[which][n], hs):
                    if dst is not None:
                        dst.copy_(src, non_blocking=True)
            self.ev_in[which].record(self.s_in)

    def step_e2e(self, _i=0):
        cur = torch.cuda.current_stream()
        a = self.e2e_calls & 1
        self.e2e_calls += 1
        ins = self.in_sets[a]
        # next step's inputs into the other set, once the step before this one has stopped reading it
        self._copy_in(1 - a, after=self.ev_free[1 - a] if self.e2e_calls > 1 else None)
        # the previous results must have left the device before this step overwrites them
        wait_out = lambda: cur.wait_event(self.ev_out)
        if self.e2e_mode == "attn":
            self.attn_step(ins, before_results=wait_out)
        else:
            for n, xs in ins.items():
                self.t[n] = xs
            if self.backward:
                self.step(before_proj_bwd=wait_out)
            else:
                wait_out()
                self.step()
        self.ev_free[a].record(cur)
        self.ev_result.record(cur)
        with torch.cuda.stream(self.s_out):
            self.s_out.wait_event(self.ev_result)
            for dst, src in zip(self.h_out, self.results):
                dst.copy_(src, non_blocking=True)
            self.ev_out.record(self.s_out)
        cur.wait_event(self.ev_in[1 - a])      # the copy issued by this call is inside this call's time
        if _i == getattr(self, "e2e_last", -1):  # the last timed call also waits for its own result copy
            cur.wait_event(self.ev_out)

    def teardown_e2e(self):
        torch.cuda.synchronize()
        for n in ("in_sets", "h_in", "h_out", "results"):
            if hasattr(self, n):
                delattr(self, n)
        torch.cuda.empty_cache()


def train_config(cfg: W.TrainCfg, world: int, gemm_pair_mode: int) -> dict:
    """The `config` object of a training / prefill line; the reference arm prints the same one."""
    return {"workload": cfg.name, "layers": cfg.L, "donor": cfg.donor, "batch_per_gpu": cfg.B,
            "global_batch": cfg.B * world, "seq_len": cfg.S, "d_model": cfg.D, "heads": [cfg.Hq, cfg.Hkv],
            "head_dim": cfg.dh, "parallelism": f"dp{world}", "l2": "inputs larger than L2 (about 10 GB live)",
            "gemm_tiles": {0: "single-CTA 128x256 everywhere", 1: "CTA pairs 256x256 for the forward GEMMs, single-CTA "
                           "128x256 for the gradient GEMMs", 2: "CTA pairs 256x256 everywhere"}[gemm_pair_mode],
            "flops": "value: attention kernels only, model count (forward 2 GEMMs, backward 4), causal pairs "
                     "S(S+1)/2, over the summed device time of the attention kernels inside the timed block step; "
                     "ms_per_step: the whole block step (projections + attention)"}


def cpu_baseline_train(cfg: W.TrainCfg, backward: bool, heads: int = 4, proj_tokens: int = 1024):
    """The oracle, as it stands, on a bounded exact slice: attention forward (+ backward) of one
    layer, one sequence, `heads` query heads of one KV group at the full sequence length, and the
    projections of one owner layer on `proj_tokens` tokens."""
    from oracle import attention as A
    S, dh, D = cfg.S, cfg.dh, cfg.D
    seed = W.SEED
    q = [synth.normal((1, S, heads, dh), seed, synth.tid(20), 1.0).double().numpy()]
    k = [synth.normal((1, S, 1, dh), seed, synth.tid(21), 1.0).double().numpy()]
    v = [synth.normal((1, S, 1, dh), seed, synth.tid(22), 1.0).double().numpy()]
    g = [synth.normal((1, S, heads, dh), seed, synth.tid(23), 1.0).double().numpy()]
    nq, nkv = cfg.Hq * dh, cfg.Hkv * dh
    x = [synth.normal((proj_tokens, D), seed, synth.tid(0), 1.0).double().numpy()]
    wq = [synth.normal((nq, D), seed, synth.tid(1), 0.02).double().numpy()]
    wk = [synth.normal((nkv, D), seed, synth.tid(2), 0.02).double().numpy()]
    wv = [synth.normal((nkv, D), seed, synth.tid(3), 0.02).double().numpy()]
    t0 = time.perf_counter()
    A.attn_fwd(q, k, v, [0])
    if backward:
        A.attn_bwd(q, k, v, g, [0])
    dt_attn = time.perf_counter() - t0
    qq, kk, vv = A.proj_fwd(x, wq, wk, wv, [0], 1, proj_tokens, cfg.Hq, cfg.Hkv, dh)
    if backward:
        A.proj_bwd(x, wq, wk, wv, qq, kk, vv, [0])
    dt = time.perf_counter() - t0
    f_attn = 4 * dh * (S * (S + 1) // 2) * heads
    f_proj = 2 * proj_tokens * D * (nq + 2 * nkv)
    if backward:
        f_attn, f_proj = 3 * f_attn, 3 * f_proj
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        cores = os.cpu_count() or 1
    sample = (f"attention fwd{'+bwd' if backward else ''} of 1 layer x 1 sequence x {heads} query heads (one KV group) "
              f"at S={S}: {f_attn / 1e9:.1f} model GFLOP in {dt_attn:.2f} s (the value); plus Q/K/V projections "
              f"fwd{'+bwd' if backward else ''} of one owner layer on {proj_tokens} tokens: {f_proj / 1e9:.1f} GFLOP in {dt - dt_attn:.2f} s")
    return {"value": f_attn / dt_attn / 1e12, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": sample,
            "seconds": dt, "block_value": (f_attn + f_proj) / dt / 1e12}


# ---------------------------------------------------------------------------------------------
# decode workload
# ---------------------------------------------------------------------------------------------
class DecodeRunner:
    def __init__(self, kvp, cfg: W.DecodeCfg, device, n_slots=None, q_sets=4, shuffle_pages=True, per_layer=False):
        """per_layer: one kvp_decode call per layer (layer_begin / layer_end), the order a real model's forward
        pass imposes -- a consumer then re-reads its donor's pages -- instead of one grouped call per step."""
        self.kvp, self.cfg, self.device, self.per_layer = kvp, cfg, device, per_layer
        self.state = W.make_decode_state(cfg, device, n_slots=n_slots, shuffle_pages=shuffle_pages)
        st = self.state
        self.desc = kvp.DecodeDesc(cfg.L, cfg.B, cfg.Hq, cfg.Hkv, cfg.dh, cfg.page, cfg.max_pages, st.n_pages, 0)
        self.ws = torch.empty(kvp.decode_workspace_bytes(self.desc, cfg.donor), dtype=torch.uint8, device=device)
        self.q = [W.decode_queries(cfg, device, W.SEED, s) for s in range(q_sets)]
        own = set(cfg.owners())
        self.k_new = [[synth.normal((cfg.B, cfg.Hkv, cfg.dh), W.SEED, synth.tid(13, l, s), 1.0, device) if l in own
                       else None for l in range(cfg.L)] for s in range(q_sets)]
        self.v_new = [[synth.normal((cfg.B, cfg.Hkv, cfg.dh), W.SEED, synth.tid(14, l, s), 1.0, device) if l in own
                       else None for l in range(cfg.L)] for s in range(q_sets)]
        self.o = [torch.empty(cfg.B, cfg.Hq, cfg.dh, dtype=torch.bfloat16, device=device) for _ in range(cfg.L)]
        self.lse = [torch.empty(cfg.B, cfg.Hq, device=device) for _ in range(cfg.L)]
        self.steps_done = 0

    def reset(self):
        self.state.lengths.copy_(self.state.lengths0.to(self.device))
        self.steps_done = 0

    def step(self, i=0):
        k, c, st = self.kvp, self.cfg, self.state
        s = i % len(self.q)
        st.lengths.add_(1)                       # the new token is part of the context it attends to
        k.cache_append(self.desc, c.donor, self.k_new[s], self.v_new[s], st.k_cache, st.v_cache, st.block_table,
                       st.lengths)
        if self.per_layer:
            for l in range(c.L):
                k.decode(self.desc, c.donor, self.q[s], st.k_cache, st.v_cache, st.block_table, st.lengths, self.o,
                         self.lse, self.ws, layer_begin=l, layer_end=l + 1)
        else:
            k.decode(self.desc, c.donor, self.q[s], st.k_cache, st.v_cache, st.block_table, st.lengths, self.o,
                     self.lse, self.ws)
        self.steps_done += 1

    def setup_e2e(self):
        c = self.cfg
        self.h_q = [a.cpu().pin_memory() for a in self.q[0]]
        self.h_kn = [a.cpu().pin_memory() if a is not None else None for a in self.k_new[0]]
        self.h_vn = [a.cpu().pin_memory() if a is not None else None for a in self.v_new[0]]
        self.h_o = [torch.empty_like(a, device="cpu").pin_memory() for a in self.o]
        nb = lambda xs: sum(a.numel() * a.element_size() for a in xs if a is not None)
        self.h2d = nb(self.h_q) + nb(self.h_kn) + nb(self.h_vn)
        self.d2h = nb(self.h_o)

    def step_e2e(self, i=0):
        for dst, src in zip(self.q[0], self.h_q):
            dst.copy_(src, non_blocking=True)
        for dl, sl in ((self.k_new[0], self.h_kn), (self.v_new[0], self.h_vn)):
            for dst, src in zip(dl, sl):
                if dst is not None:
                    dst.copy_(src, non_blocking=True)
        self.step(0)
        for dst, src in zip(self.h_o, self.o):
            dst.copy_(src, non_blocking=True)


def cpu_baseline_decode(cfg: W.DecodeCfg, n_seq: int = 16):
    """The oracle's decode on one stored layer (an owner plus its consumer, if any) and n_seq sequences.
    Only the time matters here, so the slice is filled by numpy's generator (the seeded table generator
    is slow on the host)."""
    from oracle import attention as A
    lens = [int(x) for x in synth.uniform_ints(cfg.B, cfg.len_lo, cfg.len_hi, W.SEED, synth.tid(9))[:n_seq]]
    cap = max(lens)
    members = [l for l in range(cfg.L) if cfg.donor[l] == cfg.owners()[-1]]
    donor = [0] * len(members)
    rng = np.random.default_rng(W.SEED)
    kc = [rng.standard_normal((n_seq, cap, cfg.Hkv, cfg.dh))] + [None] * (len(members) - 1)
    vc = [rng.standard_normal((n_seq, cap, cfg.Hkv, cfg.dh))] + [None] * (len(members) - 1)
    q = [rng.standard_normal((n_seq, cfg.Hq, cfg.dh)) for _ in range(len(members))]
    t0 = time.perf_counter()
    A.decode_attend(q, kc, vc, lens, donor)
    dt = time.perf_counter() - t0
    kv_bytes = sum(lens) * 2 * cfg.Hkv * cfg.dh * 2            # bf16 bytes this slice stands for
    step_bytes = W.decode_step_bytes(cfg, synth.uniform_ints(cfg.B, cfg.len_lo, cfg.len_hi, W.SEED, synth.tid(9)))
    est_step_s = dt * step_bytes / kv_bytes
    return {"value": cfg.B / est_step_s, "unit": "tokens/s", "cores": os.cpu_count() or 1, "kind": "oracle",
            "sample": f"one stored layer ({len(members)} query layers) x {n_seq} sequences (mean length {sum(lens) // len(lens)}) in {dt:.2f} s, "
                      f"extrapolated linearly in cache bytes to a full step", "seconds": dt}


# ---------------------------------------------------------------------------------------------
def run_train_like(args, kvp, rank, local_rank, world, device, peaks, peaks_kind, workload=None, e2e=True):
    """Times the block step (projections + attention, forward [+ backward]) of C2 / C1 and reports, as `value`,
    the ATTENTION-ONLY rate: model FLOPs of the attention kernels (12 dh pairs B Hq per layer with backward, 4 dh
    pairs B Hq forward only, pairs = S(S+1)/2) over the summed device time of those kernels (forward, backward,
    and the backward's helper passes) inside the timed region.  The block rate is reported beside it."""
    workload = workload or args.workload
    if workload == "train":
        cfg, backward, out_proj = (W.SMALL_TRAIN if args.small else W.C2), True, False
    elif workload == "prefill":
        cfg, backward, out_proj = (W.SMALL_TRAIN if args.small else W.C1), False, False
    else:
        raise ValueError(workload)
    runner = TrainRunner(kvp, cfg, device, backward=backward, out_proj=out_proj)
    for i in range(args.warmup):
        runner.step(i)
    torch.cuda.synchronize()
    status = kvp.device_status()
    if status != kvp.OK:
        raise RuntimeError("device status after warm-up: " + kvp.status_string(status))
    n_groups, n_own = len(cfg.owners()), len(cfg.owners())
    pairs = cfg.S * (cfg.S + 1) // 2
    unit = 2 * cfg.dh * pairs * cfg.B * cfg.Hq * cfg.L        # one attention GEMM over every layer
    n_gemm = (cfg.L + 2 * n_own) + ((2 * cfg.L + 2 * n_own) if backward else 0)   # GEMM problems; launches are fewer
    # kernel -> (event pairs to provide per step, algorithmic FLOPs per step, executed FLOPs per step)
    kernels = {"attn_fwd_kernel": (kvp.KERNEL_ATTN_FWD, cfg.L, 2 * unit, 2 * unit),
               "gemm_kernel": (kvp.KERNEL_GEMM, n_gemm, runner.gemm_flops(), runner.gemm_flops())}
    if backward:
        # single-pass backward: dV, dP, dK, dQ of the model count (it also recomputes S); helper passes: Delta,
        # clearing the fp32 accumulators, converting dQ to bf16 (no FLOPs counted)
        kernels["bwd_kernel"] = (kvp.KERNEL_ATTN_BWD, n_groups, 4 * unit, 5 * unit)
        kernels["bwd_aux"] = (kvp.KERNEL_ATTN_BWD_AUX, 1 + 2 * n_groups, 0, 0)
    timers = {name: kvp.KernelTimer(kid, args.steps * n) for name, (kid, n, _a, _e) in kernels.items()}
    l0 = kvp.launch_count()
    for t in timers.values():
        t.__enter__()
    ms, clocks = timed_region(runner.step, args.steps, device, local_rank)
    for t in timers.values():
        t.__exit__(None, None, None)
    launches = kvp.launch_count() - l0
    ms_step = ms / args.steps
    flops = runner.flops()
    block_tflops = world * flops / (ms_step * 1e-3) / 1e12
    peak = peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])
    per_kernel = {}
    for name, (kid, _n, algo, execd) in kernels.items():
        durs = timers[name].durations_ms()
        k_ms = sum(durs) / args.steps
        per_kernel[name] = {"timed_launch_groups_per_step": len(durs) / args.steps, "ms_per_step": k_ms,
                            "share_of_step": k_ms / ms_step,
                            "algorithmic_tflops": algo / (k_ms * 1e-3) / 1e12,
                            "executed_tflops": execd / (k_ms * 1e-3) / 1e12}
    attn_names = [n for n in per_kernel if n != "gemm_kernel"]
    attn_ms = kdist.max_over_ranks(sum(per_kernel[n]["ms_per_step"] for n in attn_names), device)
    attn_units = 6 if backward else 2
    value = world * attn_units * unit / (attn_ms * 1e-3) / 1e12
    flash = world * (7 if backward else 2) * unit / (attn_ms * 1e-3) / 1e12
    top = max((n for n in per_kernel if n != "bwd_aux"), key=lambda k: per_kernel[k]["ms_per_step"])
    achieved = per_kernel[top]["algorithmic_tflops"]
    traffic = None if args.small or cfg is not W.C2 else NCU_TRAFFIC_BYTES.get(top)
    roofline = {"bound": "tensor", "kernel": top + "<128>", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                "frac": achieved / peak, "traffic": traffic,
                "traffic_unit": NCU_TRAFFIC_NOTE,
                "peak_kind": f"{peaks_kind} sustained cuBLAS bf16",
                "launches_per_step": per_kernel[top]["timed_launch_groups_per_step"],
                "kernel_ms_per_step": per_kernel[top]["ms_per_step"],
                "share_of_step": per_kernel[top]["share_of_step"],
                "executed_tflops": per_kernel[top]["executed_tflops"],
                "frac_of_nominal_2250": achieved / NOMINAL_BF16_TFLOPS, "kernels": per_kernel}
    # end to end through the public API with host buffers
    e2e_obj, block_e2e = None, None
    if e2e and not args.small and not args.no_e2e:
        e2e_steps = max(3, min(args.steps, 5))
        for mode in ("attn", "block"):
            runner.setup_e2e(mode)
            for i in range(2):
                runner.step_e2e(i)
            runner.e2e_last = e2e_steps - 1 + 2
            calls0 = runner.e2e_calls
            ms_e2e, _ = timed_region(lambda i: runner.step_e2e(i + 2), e2e_steps, device, local_rank)
            assert runner.e2e_calls - calls0 == e2e_steps
            f = (attn_units * unit) if mode == "attn" else flops
            obj = {"value": world * f / (ms_e2e / e2e_steps * 1e-3) / 1e12, "unit": "TFLOP/s",
                   "h2d_bytes_per_step": runner.h2d, "d2h_bytes_per_step": runner.d2h, "ms_per_step": ms_e2e / e2e_steps,
                   "copies": "pipelined: step n+1's inputs arrive on a second stream while step n computes; "
                             "one input and one result transfer per timed step"}
            if mode == "attn":
                obj["what"] = ("kvp_attn_fwd" + (" + kvp_attn_bwd" if backward else "") + " with q, k, v" +
                               (", dO" if backward else "") + " coming from pinned host memory and " +
                               ("dQ and the fp32 dK/dV sums" if backward else "O") + " going back, every step")
                e2e_obj = obj
            else:
                obj["what"] = ("the whole block step with X" + (", dO" if backward else "") + " from pinned host memory and " +
                               ("dX of every layer and the fp32 weight-gradient bucket" if backward else "O of every layer") +
                               " going back, every step; block model FLOPs")
                block_e2e = obj
            runner.teardown_e2e()
    if e2e_obj is None:
        e2e_obj = {"value": float("nan"), "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    status = kvp.device_status()
    line = {
        "metric": "shared-KV attn fwd+bwd TFLOP/s" if backward else "shared-KV attn prefill fwd TFLOP/s",
        "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": train_config(cfg, world, args.gemm_pair_mode),
        "clocks": clocks, "gpu_launches": int(launches),
        "attn_ms_per_step": attn_ms,
        "attn_flash_convention_tflops": flash,
        "block_tflops": block_tflops,
        "block_model_flops_per_step": flops,
        "tokens_per_s": world * cfg.T / (ms_step * 1e-3),
        "pct_bf16_peak_nominal": 100.0 * value / world / NOMINAL_BF16_TFLOPS,
        "pct_bf16_peak_measured": 100.0 * value / world / peak,
        "e2e": e2e_obj, "block_e2e": block_e2e,
        "roofline": roofline, "device_status": kvp.status_string(status),
    }
    del runner
    torch.cuda.empty_cache()
    return line, cfg, backward


def run_decode(args, kvp, rank, local_rank, world, device, peaks, peaks_kind, steps=None, warmup=None, extra_modes=True):
    cfg = W.SMALL_DECODE if args.small else W.C3
    steps = cfg.steps if steps is None else steps
    warmup = 3 if warmup is None else warmup
    free, _total = torch.cuda.mem_get_info()
    own = len(cfg.owners())
    lens0 = synth.uniform_ints(cfg.B, cfg.len_lo, cfg.len_hi, W.SEED, synth.tid(9))
    pages = sum((int(n) + cfg.steps + cfg.page - 1) // cfg.page for n in lens0)
    per_slot = 2 * pages * cfg.Hkv * cfg.page * cfg.dh * 2
    n_slots = int(max(1, min(own, (free - (6 << 30)) // per_slot)))
    runner = DecodeRunner(kvp, cfg, device, n_slots=n_slots)
    for i in range(warmup):
        runner.step(i)
    torch.cuda.synchronize()
    runner.reset()
    l0 = kvp.launch_count()
    with kvp.KernelTimer(kvp.KERNEL_DECODE, steps) as kt:
        ms, clocks = timed_region(runner.step, steps, device, local_rank)
    launches = kvp.launch_count() - l0
    durs = kt.durations_ms()
    ms_step = ms / steps
    mean_len = float(lens0.double().mean()) + (steps + 1) / 2.0
    step_bytes = W.decode_step_bytes(cfg, [mean_len] * cfg.B)
    k_ms = sum(durs) / len(durs)
    achieved = step_bytes / (k_ms * 1e-3) / 1e9
    peak = peaks["hbm_gbs"]
    unshared_bytes = W.decode_step_bytes(W.C3_UNSHARED, [mean_len] * cfg.B)
    if args.small or args.no_e2e:
        ms_e2e, e2e_steps = float("nan"), 1
        runner.h2d = runner.d2h = 0
    else:
        runner.setup_e2e()
        runner.reset()
        for i in range(2):
            runner.step_e2e(i)
        e2e_steps = min(steps, 32)
        ms_e2e, _ = timed_region(runner.step_e2e, e2e_steps, device, local_rank)
    e2e_h2d, e2e_d2h = runner.h2d, runner.d2h
    # the two other report modes: the same model decoded layer by layer (consumers re-read their donor's pages), and
    # the same model with nothing shared (every layer stores and reads its own K/V); a bounded number of steps each
    modes = {}
    if not args.small and extra_modes and not args.no_e2e:
        m_steps = min(steps, 32)
        unshared_m = W.decode_step_bytes(W.C3_UNSHARED, [float(lens0.double().mean()) + (m_steps + 1) / 2.0] * cfg.B)
        for key, mcfg, per_layer in (("per_layer_sequential", cfg, True), ("unshared", W.C3_UNSHARED, False)):
            if key == "per_layer_sequential":
                runner.per_layer, r2 = True, runner
                bytes_step = unshared_m              # every layer reads a full K/V stream
            else:
                del runner
                torch.cuda.empty_cache()
                free2, _t = torch.cuda.mem_get_info()
                r2 = DecodeRunner(kvp, mcfg, device, n_slots=int(max(1, min(len(mcfg.owners()), (free2 - (6 << 30)) // per_slot))))
                bytes_step = unshared_m
            r2.reset()
            for i in range(3):
                r2.step(i)
            torch.cuda.synchronize()
            r2.reset()
            n_ev = m_steps * (mcfg.L if r2.per_layer else 1)
            with kvp.KernelTimer(kvp.KERNEL_DECODE, n_ev) as kt2:
                ms2, _c = timed_region(r2.step, m_steps, device, local_rank)
            k2 = sum(kt2.durations_ms()) / m_steps
            modes[key] = {"tokens_per_s": world * cfg.B / (ms2 / m_steps * 1e-3), "ms_per_step": ms2 / m_steps,
                          "bytes_per_step": bytes_step, "hbm_gbs": bytes_step / (ms2 / m_steps * 1e-3) / 1e9,
                          "kernel_gbs": bytes_step / (k2 * 1e-3) / 1e9, "steps": m_steps,
                          "decode_calls_per_step": mcfg.L if r2.per_layer else 1,
                          "stored_layers": len(mcfg.owners())}
            if key == "per_layer_sequential":
                runner.per_layer = False
            else:
                runner = r2
        modes["grouped_over_per_layer"] = modes["per_layer_sequential"]["ms_per_step"] / ms_step
        modes["grouped_over_unshared"] = modes["unshared"]["ms_per_step"] / ms_step
    out = {
        "metric": "shared-cache decode tokens/s", "value": world * cfg.B / (ms_step * 1e-3), "unit": "tokens/s",
        "n_gpus": world, "steps": steps, "warmup": warmup, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "hbm_gbs": step_bytes / (ms_step * 1e-3) / 1e9,
        "config": {"workload": cfg.name, "layers": cfg.L, "stored_layers": own, "batch_per_gpu": cfg.B,
                   "context": [cfg.len_lo, cfg.len_hi], "page": cfg.page, "heads": [cfg.Hq, cfg.Hkv],
                   "head_dim": cfg.dh, "physical_layer_pools": n_slots, "mode": "grouped (donor+consumer in one pass)",
                   "block_table": "pages of a sequence scattered over the pool (seeded shuffle)",
                   "l2": "cache slices far larger than L2", "bytes_per_step": step_bytes,
                   "bytes_per_step_unshared": unshared_bytes},
        "clocks": clocks, "gpu_launches": int(launches),
        "e2e": {"value": world * cfg.B / (ms_e2e / e2e_steps * 1e-3), "unit": "tokens/s",
                "h2d_bytes_per_step": e2e_h2d, "d2h_bytes_per_step": e2e_d2h},
        "modes": modes,
        "roofline": {"bound": "hbm", "kernel": "decode_kernel<128>", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak,
                     "traffic": None if args.small else NCU_TRAFFIC_BYTES["decode_kernel"],
                     "traffic_unit": NCU_TRAFFIC_NOTE,
                     "algorithmic_bytes_per_launch": step_bytes, "peak_kind": f"{peaks_kind} copy bandwidth",
                     "kernel_ms_per_step": k_ms, "share_of_step": k_ms / ms_step,
                     "frac_of_nominal_8000": achieved / NOMINAL_HBM_GBS},
        "device_status": kvp.status_string(kvp.device_status()),
    }
    del runner
    torch.cuda.empty_cache()
    return out


def run_decode_sweep(args, kvp, rank, local_rank, world, device, peaks, peaks_kind):
    """The paper's inference case study as a workload shape: LLaMA2-7B geometry with MHA (32 KV heads, so a
    converted layer saves four times the bytes of the GQA case), context 8K ... 128K, half of the layers
    sharing the K/V of the layer below, against the same model with every layer storing its own K/V."""
    B, steps, warmup = 4, 16, 3
    rows = []
    for ctx in (8192, 16384, 32768, 65536, 131072):
        row = {"context": ctx}
        for key, donor in (("shared_50pct", W.pair_donor(32, 0)), ("unshared", list(range(32)))):
            cfg = W.DecodeCfg(f"sweep-mha-{key}-{ctx}", 32, B, 32, 32, 128, 128, ctx, ctx, donor, steps)
            own = len(cfg.owners())
            free, _total = torch.cuda.mem_get_info()
            pages = B * ((ctx + steps + cfg.page - 1) // cfg.page)
            per_slot = 2 * pages * cfg.Hkv * cfg.page * cfg.dh * 2
            n_slots = int(max(1, min(own, (free - (6 << 30)) // per_slot)))
            runner = DecodeRunner(kvp, cfg, device, n_slots=n_slots)
            for i in range(warmup):
                runner.step(i)
            torch.cuda.synchronize()
            runner.reset()
            with kvp.KernelTimer(kvp.KERNEL_DECODE, steps) as kt:
                ms, clocks = timed_region(runner.step, steps, device, local_rank)
            k_ms = float(np.mean(kt.durations_ms()))
            step_bytes = W.decode_step_bytes(cfg, [ctx + (steps + 1) / 2.0] * B)
            row[key] = {"tokens_per_s": world * B / (ms / steps * 1e-3), "ms_per_step": ms / steps, "stored_layers": own,
                        "physical_layer_pools": n_slots, "bytes_per_step": step_bytes,
                        "kernel_gbs": step_bytes / (k_ms * 1e-3) / 1e9, "frac_of_measured_copy": step_bytes / (k_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                        "sm_mhz": clocks.get("sm_mhz")}
            del runner
            torch.cuda.empty_cache()
        row["speedup_shared"] = row["shared_50pct"]["tokens_per_s"] / row["unshared"]["tokens_per_s"]
        rows.append(row)
    last = rows[-1]["shared_50pct"]
    return {"metric": "shared-cache decode tokens/s (MHA, 128K context, 50% sharing)", "value": last["tokens_per_s"],
            "unit": "tokens/s", "n_gpus": world, "steps": steps, "warmup": warmup, "ms_per_step": last["ms_per_step"],
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "decode-sweep-LLaMA2-7B-MHA", "layers": 32, "heads": [32, 32], "head_dim": 128,
                       "batch_per_gpu": B, "page": 128, "l2": "cache slices far larger than L2"},
            "sweep": rows, "device_status": kvp.status_string(kvp.device_status())}


def run_stage(args, kvp, rank, local_rank, world, device, peaks, peaks_kind):
    """Tail pipeline stage of the planned 32-layer decoder: full attention block (Q/K/V projections,
    attention, output projection) forward + backward, converted (stage-local donor) vs unconverted."""
    ff, fs, flm = kvp.layer_flops(4096, 11008, 32, 8, 128, 4096, 32000)
    sb = [4 * i for i in range(9)]
    plan = kvp.plan(sb, [ff] * 32, [fs] * 32, [0] * 7 + [flm], stop_on_no_improve=True)
    plan_local = kvp.plan(sb, [ff] * 32, [fs] * 32, [0] * 7 + [flm], stop_on_no_improve=True, stage_local_donor=True)
    res = {}
    for cfg in (W.C4_UNCONVERTED, W.C4_STAGE_LOCAL):
        runner = TrainRunner(kvp, cfg, device, backward=True, out_proj=True)
        for i in range(args.warmup):
            runner.step(i)
        ms, clocks = timed_region(runner.step, args.steps, device, local_rank)
        res[cfg.name] = {"ms_per_step": ms / args.steps, "tflops": runner.flops() / (ms / args.steps * 1e-3) / 1e12,
                         "model_flops": runner.flops(), "clocks": clocks}
        del runner
        torch.cuda.empty_cache()
    a, b = res[W.C4_UNCONVERTED.name], res[W.C4_STAGE_LOCAL.name]
    return {"metric": "tail-stage attention block fwd+bwd ms (converted vs unconverted)", "value": b["ms_per_step"],
            "unit": "ms", "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": b["ms_per_step"],
            "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "C4-stage", "batch": 8, "seq_len": 4096, "layers": 4,
                       "plan": {"converted": [l for l, z in enumerate(plan["z"]) if z], "fir": plan["fir"],
                                "fir_stage_local": plan_local["fir"],
                                "stage_local_donor": plan_local["donor"][28:]}},
            "stage": res, "speedup_converted": a["ms_per_step"] / b["ms_per_step"],
            "flops_ratio_converted": b["model_flops"] / a["model_flops"]}


def _time_gemm(kvp, M, N, K, a_mn, b_mn, f32_out, device, reps=5):
    """Median device time (ms) of one kvp_gemm launch on fresh random bf16 operands."""
    a = torch.randn((K, M) if a_mn else (M, K), device=device, dtype=torch.bfloat16)
    b = torch.randn((K, N) if b_mn else (N, K), device=device, dtype=torch.bfloat16)
    c = torch.empty((M, N), device=device, dtype=torch.float32 if f32_out else torch.bfloat16)
    for _ in range(2):
        kvp.gemm(a, b, c, a_mn, b_mn)
    ts = []
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        kvp.gemm(a, b, c, a_mn, b_mn)
        e1.record()
        torch.cuda.synchronize()
        ts.append(e0.elapsed_time(e1))
    del a, b, c
    return float(np.median(ts))


def run_pipeline(args, kvp, rank, local_rank, world, device, peaks, peaks_kind):
    """What the measured kernels mean for the paper's headline: per-stage forward / backward times of a
    32-layer, 8-stage decoder (LLaMA2-7B geometry, MHA, S = 8192, one sequence per micro-batch) are assembled
    from MEASURED pieces -- the attention block of a 4-layer stage, unconverted and converted with a
    stage-local donor, through the library's own path; the MLP and LM-head GEMMs through kvp_gemm -- and fed
    to kvp_plan (time-guided) and kvp_sim_1f1b.  Norms, rotary embedding, the SwiGLU activation, the
    embedding and the loss are not timed (they are not built), so every stage is equally too light."""
    D, H, dh, S, F, V, M_MICRO = 4096, 32, 128, 8192, 11008, 32000, 32
    T = S
    cfgs = {"full": W.TrainCfg("stage-mha-unconverted", 4, 1, S, D, H, H, dh, [0, 1, 2, 3]),
            "local": W.TrainCfg("stage-mha-local-donor", 4, 1, S, D, H, H, dh, [0, 0, 0, 0])}
    t_attn = {}
    for key, cfg in cfgs.items():
        for backward in (False, True):
            runner = TrainRunner(kvp, cfg, device, backward=backward, out_proj=True, bucket=False)
            for i in range(args.warmup):
                runner.step(i)
            ms, _ = timed_region(runner.step, args.steps, device, local_rank)
            t_attn[(key, backward)] = ms / args.steps
            del runner
            torch.cuda.empty_cache()
    g = lambda *a: _time_gemm(kvp, *a, device)
    mlp_f = 2 * g(T, F, D, False, False, False) + g(T, D, F, False, False, False)
    mlp_b = (g(T, F, D, False, True, False) + g(D, F, T, True, True, True)            # through the down projection
             + 2 * (g(T, D, F, False, True, False) + g(F, D, T, True, True, True)))   # through gate and up
    lm_f = g(T, V, D, False, False, False)
    lm_b = g(T, D, V, False, True, False) + g(V, D, T, True, True, True)
    ns = lambda ms: int(round(ms * 1e6))
    full_f = t_attn[("full", False)] / 4 + mlp_f
    full_b = (t_attn[("full", True)] - t_attn[("full", False)]) / 4 + mlp_b
    cons_f = (t_attn[("local", False)] - t_attn[("full", False)] / 4) / 3 + mlp_f
    cons_b = ((t_attn[("local", True)] - t_attn[("local", False)]) - (t_attn[("full", True)] - t_attn[("full", False)]) / 4) / 3 + mlp_b
    sb = [4 * i for i in range(9)]
    ff, fs, flm = kvp.layer_flops(D, F, H, H, dh, S, V)
    plans = {
        "baseline": {"z": [0] * 32},
        "flops_guided": kvp.plan(sb, [ff] * 32, [fs] * 32, [0] * 7 + [flm], stop_on_no_improve=True, stage_local_donor=True),
        "time_guided": kvp.plan(sb, [ns(full_f + full_b)] * 32, [ns(cons_f + cons_b)] * 32, [0] * 7 + [ns(lm_f + lm_b)],
                                stop_on_no_improve=True, stage_local_donor=True),
    }
    out = {}
    for name, pl in plans.items():
        z = pl["z"]
        tf = [ns(sum(cons_f if z[l] else full_f for l in range(sb[i], sb[i + 1])) + (lm_f if i == 7 else 0)) for i in range(8)]
        tb = [ns(sum(cons_b if z[l] else full_b for l in range(sb[i], sb[i + 1])) + (lm_b if i == 7 else 0)) for i in range(8)]
        makespan, idle = kvp.sim_1f1b(tf, tb, M_MICRO)
        tot = [a + b for a, b in zip(tf, tb)]
        out[name] = {"converted": [l for l in range(32) if z[l]], "iteration_ms": makespan / 1e6,
                     "bubble_fraction": sum(idle) / (8 * makespan), "time_imbalance": max(tot) * 8 / sum(tot),
                     "fir_flops": pl.get("fir"), "stage_fwd_ms": [x / 1e6 for x in tf], "stage_bwd_ms": [x / 1e6 for x in tb]}
    base, best = out["baseline"], out["flops_guided"]
    return {"metric": "simulated 1F1B iteration ms (PP=8, 32 micro-batches, measured stage kernels)",
            "value": best["iteration_ms"], "unit": "ms", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": best["iteration_ms"], "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "pipeline-LLaMA2-7B-MHA-S8192-PP8", "micro_batches": M_MICRO, "tokens_per_micro_batch": T,
                       "not_timed": "norms, rotary embedding, SwiGLU activation, embedding, loss (not built)"},
            "measured_ms": {"attn_block_4_layers_fwd": t_attn[("full", False)], "attn_block_4_layers_fwd_bwd": t_attn[("full", True)],
                            "attn_block_1_owner_3_consumers_fwd": t_attn[("local", False)],
                            "attn_block_1_owner_3_consumers_fwd_bwd": t_attn[("local", True)],
                            "mlp_fwd": mlp_f, "mlp_bwd": mlp_b, "lm_head_fwd": lm_f, "lm_head_bwd": lm_b},
            "plans": out, "iteration_time_reduction": 1.0 - best["iteration_ms"] / base["iteration_ms"]}


class StageFwdRunner:
    """Forward pass of one pipeline stage of 4 decoder layers built from the library's kernels: per layer
    RMSNorm -> Q/K/V projections (K/V on owners) -> rotary embedding -> attention -> output projection ->
    residual -> RMSNorm -> gate/up GEMMs -> SwiGLU -> down GEMM -> residual; the tail stage adds the final
    norm and the LM head.  The operators run with the launch sequence and byte counts of a real forward pass
    (layer l's kernels read layer l's own buffers rather than layer l-1's output, which does not change a
    kernel's time)."""

    def __init__(self, kvp, cfg, device, F=11008, V=32000, lm_head=False):
        self.kvp, self.cfg, self.F, self.V, self.lm_head = kvp, cfg, F, V, lm_head
        self.attn = TrainRunner(kvp, cfg, device, backward=False, out_proj=True, bucket=False)
        bf = torch.bfloat16
        T, D, L = cfg.T, cfg.D, cfg.L
        rnd = lambda *shape: torch.randn(*shape, device=device, dtype=bf)
        self.h = [rnd(T, D) for _ in range(L)]                     # residual stream entering each layer
        self.wn1 = [rnd(D) for _ in range(L)]
        self.wn2 = [rnd(D) for _ in range(L)]
        self.w_gate = [rnd(F, D) * 0.02 for _ in range(L)]
        self.w_up = [rnd(F, D) * 0.02 for _ in range(L)]
        self.w_down = [rnd(D, F) * 0.02 for _ in range(L)]
        self.gate, self.up = torch.empty(T, F, device=device, dtype=bf), torch.empty(T, F, device=device, dtype=bf)
        self.mid = torch.empty(T, D, device=device, dtype=bf)
        if lm_head:
            self.w_lm = rnd(V, D) * 0.02
            self.logits = torch.empty(T, V, device=device, dtype=bf)
        self.elem_bytes = 0

    def step(self, _i=0):
        k, c, a = self.kvp, self.cfg, self.attn
        t, o = a.t, a.out
        own = set(c.owners())
        eb = 0
        T, D, F = c.T, c.D, self.F
        for l in range(c.L):
            k.rmsnorm(self.h[l], self.wn1[l], 1e-5, t["x"][l])
            eb += 2 * T * D * 2
        k.proj_fwd(a.sh, c.donor, t["x"], t["wq"], t["wk"], t["wv"], o["q"], o["k"], o["v"])
        for l in range(c.L):
            k.rope(o["q"][l])
            eb += 2 * o["q"][l].numel() * 2
            if l in own:
                k.rope(o["k"][l])
                eb += 2 * o["k"][l].numel() * 2
        k.attn_fwd(a.sh, c.donor, o["q"], o["k"], o["v"], o["o"], o["lse"])
        k.out_proj_fwd(a.sh, o["o"], t["wo"], o["y"])
        for l in range(c.L):
            k.add(self.h[l], o["y"][l], self.mid)
            k.rmsnorm(self.mid, self.wn2[l], 1e-5, o["y"][l])
            k.gemm(o["y"][l], self.w_gate[l], self.gate)
            k.gemm(o["y"][l], self.w_up[l], self.up)
            k.swiglu(self.gate, self.up, self.gate)
            k.gemm(self.gate, self.w_down[l], o["y"][l])
            k.add(self.mid, o["y"][l], self.mid)
            eb += (3 + 2 + 3) * T * D * 2 + 3 * T * F * 2
        if self.lm_head:
            k.rmsnorm(self.mid, self.wn1[0], 1e-5, self.mid)
            k.gemm(self.mid, self.w_lm, self.logits)
            eb += 2 * T * D * 2
        self.elem_bytes = eb


def run_stage_fwd(args, kvp, rank, local_rank, world, device, peaks, peaks_kind):
    """Whole-stage forward times (the paper's stage tables list one per stage): a regular stage, the tail stage
    with the LM head, and the tail stage with three of its four layers converted (stage-local donor), LLaMA2-7B
    geometry with MHA, S = 8192, one sequence per micro-batch."""
    D, H, dh, S = 4096, 32, 128, 8192
    full = W.TrainCfg("stage-mha-unconverted", 4, 1, S, D, H, H, dh, [0, 1, 2, 3])
    local = W.TrainCfg("stage-mha-local-donor", 4, 1, S, D, H, H, dh, [0, 0, 0, 0])
    # The three stage kinds are timed in turn, round after round, and each reports the median of its rounds: the
    # SM clock under the power cap drifts over seconds, and back-to-back blocks would put that drift into the ratios.
    kinds = (("regular", full, False), ("tail", full, True), ("tail_converted", local, True))
    runners = {name: StageFwdRunner(kvp, cfg, device, lm_head=lm) for name, cfg, lm in kinds}
    for i in range(max(args.warmup, 20)):           # long enough for the power-capped clock to settle
        for r in runners.values():
            r.step(i)
    rounds, per_round = 7, max(args.steps, 4)
    samples = {name: [] for name in runners}
    mhz = {name: [] for name in runners}
    for _ in range(rounds):
        for name, r in runners.items():
            ms, clocks = timed_region(r.step, per_round, device, local_rank)
            samples[name].append(ms / per_round)
            if clocks.get("sm_mhz") is not None:
                mhz[name].append(clocks["sm_mhz"])
    res = {name: {"ms": float(np.median(samples[name])), "ms_min": min(samples[name]), "ms_max": max(samples[name]),
                  "rounds": rounds, "steps_per_round": per_round, "elementwise_bytes": runners[name].elem_bytes,
                  "sm_mhz": float(np.median(mhz[name])) if mhz[name] else None} for name in runners}
    del runners
    torch.cuda.empty_cache()
    # the element-wise kernels alone, against the measured copy bandwidth
    r = StageFwdRunner(kvp, full, device)
    T, F = full.T, r.F
    def timed(fn, nbytes, reps=20):
        # fn(i) works on the i-th of four sets of buffers in turn: together they are larger than L2
        for i in range(4):
            fn(i)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(reps):
            fn(i)
        e1.record()
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) / reps * 1e3
        return {"us": us, "gbs": nbytes / (us * 1e-6) / 1e9, "frac_of_measured_copy": nbytes / (us * 1e-6) / 1e9 / peaks["hbm_gbs"]}
    qs = r.attn.out["q"]
    elem = {"rmsnorm": timed(lambda i: kvp.rmsnorm(r.h[i % 4], r.wn1[0], 1e-5, r.mid), 2 * T * D * 2),
            "rope": timed(lambda i: kvp.rope(qs[i % 4]), 2 * qs[0].numel() * 2),
            "swiglu": timed(lambda i: kvp.swiglu(r.gate, r.up, r.gate), 3 * T * F * 2),
            "add": timed(lambda i: kvp.add(r.h[i % 4], r.h[(i + 1) % 4], r.mid), 3 * T * D * 2)}
    del r
    torch.cuda.empty_cache()
    ff, fs, flm = kvp.layer_flops(D, 11008, H, H, dh, S, 32000)
    return {"metric": "tail-stage forward ms (LLaMA2-7B MHA, S=8192, converted)", "value": res["tail_converted"]["ms"], "unit": "ms",
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": res["tail_converted"]["ms"],
            "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "stage-forward-LLaMA2-7B-MHA-S8192", "layers_per_stage": 4, "tokens": S,
                       "l2": "working set of a stage far larger than L2"},
            "stages": res, "elementwise_kernels": elem,
            "time_ratio_tail_over_regular": res["tail"]["ms"] / res["regular"]["ms"],
            "time_ratio_converted_tail_over_regular": res["tail_converted"]["ms"] / res["regular"]["ms"],
            "flops_ratio_tail_over_regular": (4 * ff + flm) / (4 * ff),
            "flops_ratio_converted_tail_over_regular": (ff + 3 * fs + flm) / (4 * ff),
            "device_status": kvp.status_string(kvp.device_status())}


def reference_arm(args, rank, world):
    """The fp64 CPU oracle on this machine's host cores; each step is a bounded sample of the workload."""
    if rank != 0:
        return
    steps, warmup = args.steps, args.warmup
    if args.workload == "decode":
        fn = lambda: cpu_baseline_decode(W.C3, n_seq=1)
        metric = "shared-cache decode tokens/s"
        config = {"workload": W.C3.name, "note": "fp64 CPU oracle on a bounded sample per step"}
    else:
        # the same workload, config object and sample as the cpu_baseline of the CUDA arm's line
        backward = args.workload != "prefill"
        cfg = W.C2 if backward else W.C1
        fn = lambda: cpu_baseline_train(cfg, backward)
        metric = "shared-KV attn fwd+bwd TFLOP/s" if backward else "shared-KV attn prefill fwd TFLOP/s"
        config = train_config(cfg, world, args.gemm_pair_mode)
    for _ in range(min(warmup, 1)):
        fn()
    t0 = time.perf_counter()
    last = None
    vals = []
    for _ in range(steps):
        last = fn()
        vals.append(last["value"])
    dt = time.perf_counter() - t0
    value = float(np.mean(vals))
    line = {"impl": "reference", "metric": metric, "value": value, "unit": last["unit"], "n_gpus": world,
            "steps": steps, "warmup": min(warmup, 1), "ms_per_step": dt / steps * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config,
            "cpu_baseline": {"value": value, "unit": last["unit"], "cores": last["cores"], "kind": "oracle",
                             "sample": last["sample"]},
            "e2e": {"value": value, "unit": last["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="train", choices=["train", "prefill", "decode", "stage", "pipeline", "decode_sweep", "stage_fwd"])
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-decode", action="store_true", help="skip the decode workload in the default run")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the shortened prefill and tail-stage runs of the default line")
    ap.add_argument("--no-e2e", action="store_true",
                    help="skip the end-to-end arms and the extra decode modes (for profiler launch lists: fewer launches)")
    ap.add_argument("--gemm-pair-mode", type=int, default=1, choices=[0, 1, 2],
                    help="GEMM tiles: 1 = CTA pairs for the forward GEMMs (the library's default), 0 = single-CTA tiles "
                         "everywhere, 2 = CTA pairs everywhere (for comparison)")
    ap.add_argument("--small", action="store_true",
                    help="reduced shapes of the same kernels (inputs still larger than L2, under 2 GB on the device) "
                         "for profiler captures; implies --no-decode for train and --no-cpu-baseline")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" and not args.small else args.warmup
    if args.small:
        args.no_decode = args.no_cpu_baseline = args.no_extras = True

    rank, local_rank, world = kdist.env_world()
    if args.impl == "reference":
        reference_arm(args, rank, world)
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback for the hot path")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    kdist.init("nccl")
    from paper_2608_15943_b200 import kvp     # loads the CUDA library or raises
    peaks, peaks_kind = measured_peaks()
    kvp.set_gemm_pair_mode(args.gemm_pair_mode)

    if args.workload in ("train", "prefill"):
        line, cfg, backward = run_train_like(args, kvp, rank, local_rank, world, device, peaks, peaks_kind)
        if args.workload == "train" and not args.small and not args.no_extras:
            # the prefill configuration and the tail-stage workload, shortened, so that the default record carries them
            sub = argparse.Namespace(**vars(args))
            sub.steps, sub.warmup = max(3, min(args.steps, 5)), 3
            try:
                pl, _c, _b = run_train_like(sub, kvp, rank, local_rank, world, device, peaks, peaks_kind, workload="prefill", e2e=False)
                line["prefill"] = {k: pl[k] for k in ("metric", "value", "unit", "ms_per_step", "attn_ms_per_step", "block_tflops",
                                                      "pct_bf16_peak_nominal", "tokens_per_s", "steps", "warmup")}
                line["prefill"]["config"] = pl["config"]["workload"]
                line["prefill"]["kernels"] = pl["roofline"]["kernels"]
                st = run_stage(sub, kvp, rank, local_rank, world, device, peaks, peaks_kind)
                line["stage"] = {k: st[k] for k in ("metric", "value", "unit", "stage", "speedup_converted", "flops_ratio_converted", "steps", "warmup")}
                line["stage"]["config"] = st["config"]
            except Exception as exc:
                line["extras_error"] = repr(exc)
        if args.workload == "train" and not args.no_decode:
            try:
                line["decode"] = run_decode(args, kvp, rank, local_rank, world, device, peaks, peaks_kind)
            except Exception as exc:   # report, do not hide: the training line is still valid
                line["decode"] = {"error": repr(exc)}
        if rank == 0 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline_train(cfg, backward)
            if "decode" in line and "error" not in line["decode"]:
                line["decode"]["cpu_baseline"] = cpu_baseline_decode(W.C3)
    elif args.workload == "stage_fwd":
        line = run_stage_fwd(args, kvp, rank, local_rank, world, device, peaks, peaks_kind)
    elif args.workload == "decode_sweep":
        line = run_decode_sweep(args, kvp, rank, local_rank, world, device, peaks, peaks_kind)
    elif args.workload == "pipeline":
        line = run_pipeline(args, kvp, rank, local_rank, world, device, peaks, peaks_kind)
    elif args.workload == "decode":
        line = run_decode(args, kvp, rank, local_rank, world, device, peaks, peaks_kind,
                          steps=args.steps if (args.steps != 10 or args.small) else None,
                          warmup=args.warmup if args.small else None)
        if rank == 0 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline_decode(W.C3)
    else:
        line = run_stage(args, kvp, rank, local_rank, world, device, peaks, peaks_kind)
    if rank == 0:
        print(json.dumps(line), flush=True)
    kdist.barrier()


if __name__ == "__main__":
    main()
