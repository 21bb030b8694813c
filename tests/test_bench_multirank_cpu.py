"""The N>1 path on CPU, two gloo ranks: one batch is split over the ranks by total frames
(longest first), every rank decodes its own share, nothing crosses ranks on the data path,
and only the timing scalars are reduced (sum of frames, max of time).  The CUDA library cannot
run here, so the ranks decode their shards with the CPU oracle: what is checked is the host
logic - the partition, its balance, and that sharded results equal unsharded ones."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2510_09085_b200 import sharding


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(world))
    import bench
    import oracle
    from paper_2510_09085_b200 import workloads as W
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # the same global batch on every rank (seeded), each rank takes its shard
    em, ln = W.make_small(77, 12, 5, 60, 8)
    mine = sharding.shard_of_rank(ln, rank, world)
    res = oracle.decode(em[mine], ln[mine], 0, 4, 0.01)
    local = {int(b): res.hyps(i) for i, b in enumerate(mine)}
    gathered = [None] * world
    dist.all_gather_object(gathered, (mine.tolist(), local))      # results only, after the fact
    frames = int(ln[mine].sum())
    ms_total = 10.0 * (rank + 1)                     # rank 1 is the slow one
    value, ms_per_step = bench.whole_job_throughput(frames, ms_total, 5, dist, "cpu")
    # the benchmark's own sharding of its workload
    wl, n_global = bench._workload(rank, world)
    out.put((rank, gathered, frames, value, ms_per_step, int(wl.lengths.sum()), len(wl.lengths),
             n_global))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_split_one_batch_and_reduce_timing():
    import oracle
    from paper_2510_09085_b200 import workloads as W
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=300) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (_, g0, f0, v0, t0, bf0, bn0, ng0), (_, g1, f1, v1, t1, bf1, bn1, ng1) = got
    assert g0 == g1                                  # both ranks saw the same gathered results
    em, ln = W.make_small(77, 12, 5, 60, 8)
    shards = [set(idx) for idx, _ in g0]
    assert shards[0].isdisjoint(shards[1]) and shards[0] | shards[1] == set(range(12))
    assert abs(f0 - f1) <= int(ln.max())             # balanced by total frames
    whole = oracle.decode(em, ln, 0, 4, 0.01)
    merged = {}
    for _, local in g0:
        merged.update(local)
    for b in range(12):
        assert merged[b] == whole.hyps(b)            # sharding changes no result
    assert t0 == t1 == 20.0 / 5                      # the slowest rank sets the time
    expect = (f0 + f1) / (4.0e-3)
    assert np.isclose(v0, expect) and np.isclose(v1, expect)
    # bench.py: a global batch of 64 utterances per rank, split by frames
    assert ng0 == ng1 == 128 and bn0 + bn1 == 128
    longest = int(W.workload_wav2vec2(batch=128).lengths.max())
    assert abs(bf0 - bf1) <= longest


def test_longest_first_partition_properties():
    rng = np.random.default_rng(3)
    for n, m in [(64, 2), (64, 8), (7, 3), (3, 8), (0, 4), (256, 5)]:
        ln = rng.integers(0, 1751, size=n)
        shards = sharding.lpt_shards(ln, m)
        assert len(shards) == m
        flat = np.concatenate(shards) if n else np.zeros(0, dtype=np.int64)
        assert sorted(flat.tolist()) == list(range(n))
        loads = [int(ln[s].sum()) for s in shards]
        if n:
            assert max(loads) - min(loads) <= int(ln.max())
            assert max(loads) <= ln.sum() / m + ln.max()
        again = sharding.lpt_shards(ln, m)
        assert all((a == b).all() for a, b in zip(shards, again))
    # longest first: the two longest utterances never share a shard when there are two shards
    s = sharding.lpt_shards([5, 100, 99, 1, 1], 2)
    assert {1, 2} not in [set(x.tolist()) for x in s] and not {1, 2} <= set(s[0].tolist())


def test_single_rank_is_the_identity():
    import bench
    v, t = bench.whole_job_throughput(1000, 50.0, 10, None, "cpu")
    assert t == 5.0 and np.isclose(v, 1000 / 5e-3)
    assert (sharding.shard_of_rank([3, 1, 2], 0, 1) == np.arange(3)).all()
