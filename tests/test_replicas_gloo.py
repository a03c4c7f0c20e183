"""The N > 1 host logic (barrier, max over ranks, whole-job aggregation) with two gloo ranks on CPU."""
import os
import socket

import pytest
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    from paper_2511_09987_b200.replicas import Replicas
    reps = Replicas("gloo")
    assert (reps.world, reps.rank) == (world, rank)
    reps.barrier()
    local_seconds = 1.0 + rank          # rank 1 is the slow one
    slowest = reps.max_over_ranks(local_seconds)
    total = reps.aggregate_throughput(units_per_replica=10.0, seconds_local=local_seconds)
    reps.barrier()
    reps.close()
    out.put((rank, slowest, total))


def test_two_ranks_aggregate_over_the_slowest():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, slowest, total in results:
        assert slowest == 2.0                      # max over ranks, seen by every rank
        assert total == pytest.approx(2 * 10.0 / 2.0)   # both replicas' units over the slowest time


def test_single_process_needs_no_group(monkeypatch):
    for k in ("WORLD_SIZE", "RANK", "LOCAL_RANK"):
        monkeypatch.delenv(k, raising=False)
    from paper_2511_09987_b200.replicas import Replicas
    reps = Replicas("gloo")
    assert reps.world == 1 and reps.max_over_ranks(3.5) == 3.5
    assert reps.aggregate_throughput(7.0, 2.0) == 3.5
    reps.barrier()
    reps.close()
