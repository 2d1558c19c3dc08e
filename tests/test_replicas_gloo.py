"""The N > 1 path of the benchmark on CPU: two gloo ranks, independent replicas, max-time / sum-work."""
import os
import socket

import torch
import torch.multiprocessing as mp

from paper_2403_08058_b200 import replicas


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    r = replicas.init_ranks("gloo")
    assert r.world == world and r.rank == rank
    r.barrier()
    # each replica does the same work; rank 1 is slower
    agg = replicas.whole_job_throughput(r, units_local=10.0, seconds_local=1.0 + rank)
    mx = r.max_over_ranks([rank, 5.0 - rank])
    sm = r.sum_over_ranks([1.0, rank])
    out[rank] = (agg, mx, sm)
    r.close()


def test_two_gloo_ranks_aggregate_like_the_benchmark():
    world, port = 2, _free_port()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        for rank in range(world):
            agg, mx, sm = out[rank]
            assert agg["units"] == 20.0 and agg["seconds"] == 2.0 and agg["value"] == 10.0   # sum of work / slowest rank
            assert mx == [1.0, 5.0] and sm == [2.0, 1.0]


def test_single_process_is_the_identity():
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        os.environ.pop(k, None)
    r = replicas.init_ranks("gloo")
    assert r.world == 1 and r.dist is None
    assert r.max_over_ranks([3.0]) == [3.0] and r.sum_over_ranks([3.0]) == [3.0]
    assert replicas.whole_job_throughput(r, 8.0, 2.0)["value"] == 4.0
    r.close()
