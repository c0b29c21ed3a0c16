"""The N > 1 path of the benchmark is "independent replicas": no data-path collective, only the timing
aggregation (max over ranks of the device time, sum over ranks of the work).  Covered here with two gloo
ranks on CPU."""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms_local = 10.0 + 5.0 * rank          # rank 1 is the slow one
    ms_step, gbs = bench.aggregate_over_ranks(ms_local, 1_000_000, 10, world, dist, "cpu")
    out.put((rank, ms_step, gbs))
    dist.barrier()
    dist.destroy_process_group()


def test_replica_aggregation_two_gloo_ranks():
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
    for rank, ms_step, gbs in res:
        assert ms_step == pytest.approx(1.5)                       # max over ranks (15 ms) / 10 steps
        assert gbs == pytest.approx(2 * 1_000_000 / 1.5 * 1e-6)    # both replicas' bytes over the slower rank's time


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    ms_step, gbs = bench.aggregate_over_ranks(20.0, 2_000_000, 10, 1)
    assert ms_step == 2.0 and gbs == pytest.approx(1.0)
