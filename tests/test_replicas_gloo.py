"""The N > 1 path of the bench: independent replicas, a barrier around the timed region, the maximum over ranks of
the device time, whole-job throughput.  Two gloo ranks on CPU."""
import os
import socket

import pytest
import torch
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world))
    from paper_2110_02781_b200.replicas import Replicas
    reps = Replicas("gloo")
    assert reps.world == world and reps.rank == rank and reps.dist is not None
    reps.barrier()
    my_ms = 10.0 + 5.0 * rank                     # rank 1 is the slow replica
    ms = reps.max_over_ranks(my_ms)
    value = reps.job_throughput(128 * 50, ms)
    reps.barrier()
    out.put((rank, ms, value))
    reps.close()


def test_two_replicas_report_the_slowest_time_and_the_whole_job_rate():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, value in res:
        assert ms == 15.0                                            # the maximum, on every rank
        assert value == pytest.approx(2 * 128 * 50 / 15e-3)          # both replicas' samples over the slowest time


def test_single_process_needs_no_process_group(monkeypatch):
    for k in ("WORLD_SIZE", "RANK", "LOCAL_RANK"):
        monkeypatch.delenv(k, raising=False)
    from paper_2110_02781_b200.replicas import Replicas
    reps = Replicas("nccl", torch.device("cpu"))
    assert reps.world == 1 and reps.dist is None
    reps.barrier()
    assert reps.max_over_ranks(3.5) == 3.5
    assert reps.job_throughput(100, 50.0) == pytest.approx(2000.0)
    reps.close()
