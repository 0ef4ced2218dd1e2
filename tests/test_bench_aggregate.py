"""The multi-rank part of bench.py on CPU: two gloo ranks, each with its own
timing and work count; the aggregate must be the max time and the summed work
(the path shards by batch with no collective on the data path)."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms, units = bench.aggregate(10.0 + 5.0 * rank, 100.0 * (rank + 1), dist)
    out.put((rank, ms, units))
    dist.barrier()
    dist.destroy_process_group()


def test_aggregate_max_time_sum_work_gloo_world2():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for _, ms, units in res:
        assert ms == 15.0 and units == 300.0


def test_aggregate_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate(3.5, 7.0, None) == (3.5, 7.0)


def test_workload_arithmetic():
    sys.path.insert(0, ROOT)
    import bench
    import wino_inputs as wi
    wl = wi.CONFIGS["cfg3"]
    assert bench.direct_ops(wl, wl.N) == 2 * 256 * 8 * 8 * 256 * 256 * 9
    assert bench.wino_ops(wl, wl.N) == 2 * 1024 * 36 * 256 * 256
    shards = wi.resnet18_layers()
    assert len(shards) == 16 and sum(1 for l in shards if l["stride"] == 2) == 3
    assert [l["C"] for l in shards if l["stride"] == 1].count(512) == 3
