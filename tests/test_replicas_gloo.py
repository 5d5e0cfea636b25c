"""The N > 1 path on CPU: two gloo ranks run the replica bookkeeping bench.py uses (partition of independent
requests, barrier, max-over-ranks timing, whole-job throughput)."""
import os
import socket

import pytest

torch = pytest.importorskip("torch")
import torch.distributed as dist  # noqa: E402
import torch.multiprocessing as mp  # noqa: E402

from paper_2608_16477_b200 import replicas  # noqa: E402


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        mine = replicas.requests_of_rank(7, world, rank)
        ms = 100.0 + 50.0 * rank                     # rank 1 is the slow one
        dist.barrier()
        slowest = replicas.max_over_ranks(ms)
        value = replicas.whole_job_throughput(4096, world, slowest)
        gathered = [None] * world
        dist.all_gather_object(gathered, mine)
        out.put((rank, mine, slowest, value, gathered))
    finally:
        dist.destroy_process_group()


def test_two_ranks_replicas():
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
    for rank, mine, slowest, value, gathered in results:
        assert slowest == 150.0                                   # every rank sees the slowest rank's time
        assert value == pytest.approx(2 * 4096 / 0.150)
        assert sorted(sum(gathered, [])) == list(range(7))       # every request exactly once, no overlap
    assert results[0][1] == [0, 2, 4, 6] and results[1][1] == [1, 3, 5]


def test_single_process_is_identity():
    assert replicas.max_over_ranks(12.5) == 12.5
    assert replicas.requests_of_rank(3, 1, 0) == [0, 1, 2]
    with pytest.raises(ValueError):
        replicas.requests_of_rank(3, 2, 2)
