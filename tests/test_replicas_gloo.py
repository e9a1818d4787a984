"""The N > 1 path is N independent replicas; this covers its host logic with two gloo ranks on CPU:
distinct seeds per rank, max-over-ranks timing, whole-job rate, and the reference arm that only
rank 0 runs."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2607_05147_b200 import replicas


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), LOCAL_RANK=str(rank),
                      WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert replicas.env_ranks() == (rank, rank, world)
        local_ms = [10.0 + 5.0 * rank, 100.0 - 7.0 * rank]           # rank 1 is slower on the first, faster on the second
        dist.barrier()
        got = replicas.max_over_ranks(local_ms, dist, "cpu")
        seeds = [replicas.rank_seed(5000, rank, k) for k in range(3)]
        gathered = [None] * world
        dist.all_gather_object(gathered, seeds)
        out.put((rank, got, gathered, replicas.is_reporting_rank(rank)))
    finally:
        dist.destroy_process_group()


def test_two_ranks_over_gloo():
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    results = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, got, gathered, reporting in results:
        assert got == [15.0, 100.0]                                  # max over ranks, element-wise
        flat = [s for seeds in gathered for s in seeds]
        assert len(set(flat)) == len(flat)                           # no two replicas share a batch seed
        assert reporting == (rank == 0)
    # the job is as slow as its slowest rank and does world x the work
    assert replicas.whole_job_rate(640, 100, 15.0, 2) == 2 * 640 * 100 / 0.015


def test_single_process_defaults(monkeypatch):
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        monkeypatch.delenv(k, raising=False)
    assert replicas.env_ranks() == (0, 0, 1)
    assert replicas.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]


def test_reference_arm_is_silent_on_other_ranks(capsys):
    import bench

    class A:
        workload, steps, warmup, gpus = "cfg3", 1, 3, 2
    bench.run_reference(A, rank=1)
    assert capsys.readouterr().out == ""
