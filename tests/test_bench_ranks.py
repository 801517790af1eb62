"""The multi-GPU leg of bench.py is "replicas only": no data-path collective, just the aggregation of the ranks'
timings (max) and work (sum).  Checked here with two gloo ranks on the CPU."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    try:
        step, e2e, orders, E = bench.aggregate_over_ranks(dist, torch.device("cpu"), 5.0 + rank, 9.0 - rank,
                                                          [1.0 + rank, 2.0 - rank, 3.0], 1000 * (rank + 1))
        q.put((rank, step, e2e, list(orders), E))
    finally:
        dist.destroy_process_group()


def test_replica_aggregation_two_ranks():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, step, e2e, orders, E in got:
        assert step == 6.0 and e2e == 9.0            # max over the ranks
        assert orders == [2.0, 2.0, 3.0]
        assert E == 3000.0                            # whole-job work: sum over the ranks


def test_single_process_passthrough():
    sys.path.insert(0, ROOT)
    import bench
    step, e2e, orders, E = bench.aggregate_over_ranks(None, None, 5.0, 7.0, [1.0, 2.0, 3.0], 10)
    assert (step, e2e, E) == (5.0, 7.0, 10.0) and np.allclose(orders, [1.0, 2.0, 3.0])
