"""The multi-GPU path is replicas only; its host logic (dispatch, slowest-rank time, whole-job rate)
is exercised here with two gloo ranks on the CPU."""
import os
import socket

import pytest

from paper_2602_00608_b200 import replicas


def test_round_robin_dispatch_covers_every_frame_once():
    for n, world in [(0, 1), (1, 2), (7, 2), (8, 4), (9, 8)]:
        got = sorted(i for r in range(world) for i in replicas.frames_of_rank(n, r, world))
        assert got == list(range(n))
        sizes = [len(replicas.frames_of_rank(n, r, world)) for r in range(world)]
        assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        replicas.frames_of_rank(4, 2, 2)


def test_whole_job_rate():
    assert replicas.whole_job_rate(1, 1, 20, 100.0) == pytest.approx(200.0)
    assert replicas.whole_job_rate(8, 2, 10, 50.0) == pytest.approx(3200.0)     # weak scaling: work grows with the ranks
    with pytest.raises(ValueError):
        replicas.whole_job_rate(1, 1, 1, 0.0)
    assert replicas.max_over_ranks(3.5, 1) == 3.5


def _worker(rank, world, port, q):
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ms = 10.0 + 5.0 * rank                                # rank 1 is the slow one
        dist.barrier()
        slowest = replicas.max_over_ranks(ms, world)
        mine = replicas.frames_of_rank(5, rank, world)
        q.put((rank, slowest, replicas.whole_job_rate(world, 1, 4, slowest), mine))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_the_slowest_time():
    import torch.multiprocessing as mp
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    out = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [o[1] for o in out] == [15.0, 15.0]                # both ranks report the slowest rank's time
    assert out[0][2] == out[1][2] == pytest.approx(2 * 1 * 4 / 15e-3)
    assert sorted(out[0][3] + out[1][3]) == [0, 1, 2, 3, 4]
