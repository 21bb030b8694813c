"""The N>1 path of bench.py on CPU: two gloo ranks, each with its own batch, no collective
on the data path - only the timing scalars are reduced (sum of frames, max of time)."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(world))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = bench._workload(rank)                       # every rank draws its own batch
    frames = int(wl.lengths.sum())
    ms_total = 10.0 * (rank + 1)                     # rank 1 is the slow one
    value, ms_per_step = bench.whole_job_throughput(frames, ms_total, 5, dist, "cpu")
    out.put((rank, frames, value, ms_per_step, float(wl.emissions[0, 0, 0])))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_by_batch_and_reduce_timing():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (_, f0, v0, t0, e0), (_, f1, v1, t1, e1) = got
    assert e0 != e1                                  # different seeds per rank: weak scaling
    assert t0 == t1 == 20.0 / 5                      # the slowest rank sets the time
    expect = (f0 + f1) / (4.0e-3)
    assert np.isclose(v0, expect) and np.isclose(v1, expect)


def test_single_rank_is_the_identity():
    import bench
    v, t = bench.whole_job_throughput(1000, 50.0, 10, None, "cpu")
    assert t == 5.0 and np.isclose(v, 1000 / 5e-3)
