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


_RANK_SCRIPT = """
import json, os, sys
import torch.distributed as dist
sys.path.insert(0, %r)
from paper_2603_09221_b200 import sharding
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
value, ms, ws = sharding.aggregate_throughput(8, 5.0 * (rank + 1))
with open(os.path.join(sys.argv[1], "rank%%d.json" %% rank), "w") as f:
    json.dump(dict(rank=rank, world=world, value=value, ms=ms, env_world=int(os.environ["WORLD_SIZE"]),
                   local=int(os.environ["LOCAL_RANK"]), addr=os.environ["MASTER_ADDR"]), f)
dist.destroy_process_group()
"""


def test_launcher_starts_one_process_per_rank(tmp_path):
    """The `--gpus N` path of the benchmark outside a launcher: sharding.launch_ranks starts N ranks through torch's
    launcher with a 127.0.0.1 rendezvous.  Two CPU ranks over gloo stand in for two GPUs."""
    import json
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    script = tmp_path / "rank_script.py"
    script.write_text(_RANK_SCRIPT % root)
    cmd = sharding.launcher_command(2, str(script), [str(tmp_path)], port=_free_port())
    assert cmd[1:3] == ["-m", "torch.distributed.run"] and "--nproc-per-node" in cmd and "127.0.0.1" in cmd
    rc = sharding.launch_ranks(2, str(script), [str(tmp_path)])
    assert rc == 0
    res = [json.load(open(tmp_path / ("rank%d.json" % r))) for r in range(2)]
    assert [r["rank"] for r in res] == [0, 1] and all(r["world"] == r["env_world"] == 2 for r in res)
    assert all(r["addr"] == "127.0.0.1" for r in res) and [r["local"] for r in res] == [0, 1]
    assert all(r["ms"] == 10.0 and r["value"] == 2 * 8 / 10e-3 for r in res)
