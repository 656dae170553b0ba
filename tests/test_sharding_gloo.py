"""The multi-GPU path of the benchmark (replicas: disjoint streams per rank, max over ranks of the time),
exercised with two gloo ranks on the CPU."""
import os

import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2608_21343_b200 import sharding, workloads as W


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    streams = sharding.rank_streams(rank, 4)
    w = W.get_workload(2, B=4, T=12, n_plants=0)
    first_phrase = W.stream_phrases(w, streams[0])[0]            # every rank generates its own inputs
    r = sharding.job_throughput(frames_this_rank=4 * 12, ms_this_rank=1.0 + rank)   # rank 1 is the slow one
    q.put((rank, streams, first_phrase, r))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_partition_streams_and_take_the_slowest_time():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, s0, p0, t0), (r1, s1, p1, t1) = got
    assert s0 == [0, 1, 2, 3] and s1 == [4, 5, 6, 7] and not set(s0) & set(s1)
    assert p0 != p1                                    # different streams, different lists
    for t in (t0, t1):
        assert t["world"] == 2 and t["frames"] == 96 and t["ms"] == 2.0
        assert abs(t["value"] - 96 / 2.0e-3) < 1e-6


def test_single_process_needs_no_group():
    r = sharding.job_throughput(100, 4.0)
    assert r["world"] == 1 and r["value"] == 25000.0
