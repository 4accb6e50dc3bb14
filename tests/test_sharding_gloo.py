"""The multi-GPU path of the benchmark on CPU ranks: world_size 2 over gloo.

Instances are independent, so the only cross-rank step is the MAX-reduction of the elapsed time; every
rank generates its own workload from a rank-dependent seed."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2603_09221_b200 import sharding, workloads


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        seed = sharding.rank_seed(1, rank)
        w = workloads.make_workload(1, device="cpu", batch=(1, 2, 3), seed=seed)
        local_ms = 10.0 * (rank + 1)                       # rank 1 is the slow one
        value, ms, ws = sharding.aggregate_throughput(6, local_ms)
        out.put((rank, seed, float(w["Q"].double().sum()), value, ms, ws, sharding.max_over_ranks(float(rank))))
    finally:
        dist.destroy_process_group()


def test_two_ranks_weak_scaling_and_max_time():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, s0, q0, v0, ms0, w0, m0), (r1, s1, q1, v1, ms1, w1, m1) = res
    assert (r0, r1) == (0, 1) and s1 - s0 == 1000 and s0 == workloads.SEED0 + 1
    assert q0 != q1                                        # different seeds, different inputs
    assert ms0 == ms1 == 20.0 and w0 == w1 == 2            # the slowest rank sets the time
    assert v0 == v1 == 2 * 6 / 20e-3                       # whole-job instances per second
    assert m0 == m1 == 1.0


def test_single_process_is_the_identity():
    assert sharding.max_over_ranks(3.5) == 3.5
    v, ms, w = sharding.aggregate_throughput(10, 5.0)
    assert (v, ms, w) == (10 / 5e-3, 5.0, 1)
