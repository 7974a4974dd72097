"""The multi-rank host logic of the benchmark on CPU: two gloo ranks, max-over-ranks timing."""
import os
import socket

import pytest
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from paper_2501_17116_b200 import harness
    r, w = harness.init_process_group("gloo")
    assert (r, w) == (rank, world)
    harness.barrier()
    seconds = 1.0 + rank                      # rank 1 is the slow one
    units = 10.0 * (rank + 1)
    out[rank] = (harness.max_over_ranks(seconds), harness.sum_over_ranks(units),
                 harness.whole_job_throughput(units, seconds))
    harness.barrier()
    import torch.distributed as dist
    dist.destroy_process_group()


def test_two_gloo_ranks_reduce_time_and_work():
    world = 2
    port = _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    for rank in range(world):
        tmax, usum, thr = res[rank]
        assert tmax == 2.0                     # the slowest rank
        assert usum == 30.0                    # whole-job work
        assert thr == pytest.approx(15.0)


def test_single_process_passthrough():
    from paper_2501_17116_b200 import harness
    assert harness.max_over_ranks(3.5) == 3.5
    assert harness.whole_job_throughput(10.0, 2.0) == 5.0
