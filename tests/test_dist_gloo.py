"""world_size-2 check (gloo, CPU) of the benchmark's multi-process plumbing: replicas are
independent, the job's time is the slowest rank's, its throughput the sum of units over it."""
import os
import socket

import torch.multiprocessing as mp


def _worker(rank, world, port, q):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    from paper_2605_17879_b200 import dist as gd
    r, lr, w = gd.init("gloo")
    assert (r, lr, w) == (rank, rank, world)
    gd.barrier()
    secs = 2.0 if rank == 0 else 3.0          # rank 1 is the slower replica
    units = 100.0 * (rank + 1)
    thr, tmax = gd.aggregate_throughput(units, secs)
    q.put((rank, thr, tmax, gd.max_over_ranks(float(rank)), gd.sum_over_ranks(1.0)))
    gd.barrier()
    gd.finish()


def test_two_rank_aggregation():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, thr, tmax, mx, sm in res:
        assert tmax == 3.0
        assert thr == 300.0 / 3.0
        assert mx == 1.0 and sm == 2.0


def test_single_process_is_identity():
    from paper_2605_17879_b200 import dist as gd
    assert gd.aggregate_throughput(10.0, 2.0) == (5.0, 2.0)
    assert gd.env_world()[2] >= 1
