"""World-size-2 gloo test of the multi-rank plumbing the benchmark uses (no GPU)."""
import os
import socket

import torch
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    from paper_2608_15943_b200 import dist as kd
    r, lr, w = kd.init("gloo")
    assert (r, w) == (rank, world)
    # independent units (sequences) are split without overlap or gaps
    mine = list(kd.shard_range(7, rank, world))
    # timings are reported as the slowest rank; throughput as the sum of the ranks' units
    slow = kd.max_over_ranks(10.0 + rank)
    total = kd.sum_over_ranks(float(len(mine)))
    # the one real exchange of a training step: sum of the flat weight-gradient bucket
    b = kd.GradBucket([(4, 8), None, (2, 8)], "cpu")
    assert b.views[1] is None and b.views[0].shape == (4, 8) and b.views[2].shape == (2, 8)
    assert b.views[0].data_ptr() == b.flat.data_ptr()
    b.views[0].fill_(rank + 1.0)
    b.views[2].fill_(10.0 * (rank + 1))
    b.all_reduce()
    # the same exchange layer by layer: entries of a layer are adjacent, the layers' slices partition the bucket,
    # and summing slice by slice gives what one all-reduce of the whole bucket gives
    shapes = [(3, 4)] * 3 + [(2, 4), None, (2, 4)] * 2          # dwq of 3 layers, dwk and dwv of owners 0 and 2
    layer_of = [0, 1, 2] * 3
    lb = kd.GradBucket(shapes, "cpu", layer_of=layer_of)
    assert kd.is_multi()
    spans = sorted(lb.layer_slices.values())
    assert spans[0][0] == 0 and spans[-1][1] == lb.flat.numel() and all(a[1] == b_[0] for a, b_ in zip(spans, spans[1:]))
    assert lb.views[4] is None and lb.layer_slices[1] == (lb.views[1].storage_offset(), lb.views[1].storage_offset() + 12)
    for i, v in enumerate(lb.views):
        if v is not None:
            v.fill_(float((rank + 1) * (i + 1)))
    whole = lb.flat.clone()
    for l in range(3):
        lb.all_reduce_layer(l)
    kd_sum = lb.flat.clone()
    import torch.distributed as td
    td.all_reduce(whole)
    layered_ok = bool(torch.equal(kd_sum, whole)) and float(lb.views[8][1, 3]) == 3.0 * 9
    # the benchmark's argument path: every rank takes its own batch (weak scaling) and reports the job total
    from paper_2608_15943_b200 import workloads as Wl
    per_rank_tokens = Wl.C2.T
    job_tokens = kd.sum_over_ranks(float(per_rank_tokens))
    kd.barrier()
    q.put((rank, mine, slow, total, float(b.views[0][0, 0]), float(b.views[2][1, 7]), layered_ok, job_tokens))


def test_two_ranks_gloo():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, m0, s0, t0, a0, c0, ok0, j0), (r1, m1, s1, t1, a1, c1, ok1, j1) = res
    assert m0 == [0, 1, 2, 3] and m1 == [4, 5, 6]
    assert s0 == s1 == 11.0 and t0 == t1 == 7.0
    assert a0 == a1 == 3.0 and c0 == c1 == 30.0
    assert ok0 and ok1
    assert j0 == j1 == 2 * 2 * 8192


def test_single_rank_is_a_no_op():
    from paper_2608_15943_b200 import dist as kd
    assert kd.max_over_ranks(3.5) == 3.5 and kd.sum_over_ranks(2.0) == 2.0
    assert list(kd.shard_range(5, 0, 1)) == [0, 1, 2, 3, 4]
    b = kd.GradBucket([(2, 2)], "cpu")
    assert b.all_reduce() is None
    assert not kd.is_multi()
    lb = kd.GradBucket([(2, 2), (1, 2)], "cpu", layer_of=[0, 1])
    assert lb.all_reduce_layer(1) is None and lb.layer_slices == {0: (0, 4), 1: (4, 6)}
