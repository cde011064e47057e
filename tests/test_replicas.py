"""Two replicas over gloo on the CPU: the reduction that turns per-rank times into the job's figure
(the N > 1 path of the benchmark: no data-path collective, max over ranks, units of all ranks)."""
import os
import socket

import pytest
import torch
import torch.multiprocessing as mp


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    from paper_2405_14371_b200 import replicas
    import torch.distributed as dist

    r, l, w = replicas.setup("gloo")
    assert (r, l, w) == (rank, rank, world)
    replicas.barrier(w)
    ms = 10.0 + 5.0 * rank                       # rank 1 is the slow replica
    slowest = replicas.max_over_ranks(ms, w)
    value = replicas.job_throughput(128.0, ms, w)
    out.put((rank, slowest, value))
    replicas.barrier(w)
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_ranks_time():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, slowest, value in got:
        assert slowest == 15.0
        assert value == pytest.approx(128.0 * 2 / 0.015)


def test_single_process_needs_no_group():
    from paper_2405_14371_b200 import replicas

    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        os.environ.pop(k, None)
    assert replicas.max_over_ranks(3.5, 1) == 3.5
    assert replicas.job_throughput(10.0, 500.0, 1) == pytest.approx(20.0)


def test_launch_plan_starts_ranks_only_when_asked_for_several_gpus_outside_a_job():
    from paper_2405_14371_b200 import replicas

    argv = ["bench.py", "--gpus", "4", "--steps", "2"]
    assert replicas.launch_plan(1, {}, argv) is None                       # one GPU: this process
    assert replicas.launch_plan(4, {"WORLD_SIZE": "4", "RANK": "1"}, argv) is None   # already a rank of a job
    cmd = replicas.launch_plan(4, {}, argv)
    assert cmd[1:3] == ["-m", "torch.distributed.run"] and "--nproc-per-node=4" in cmd and "--standalone" in cmd
    assert cmd[cmd.index("--local-addr") + 1] == "127.0.0.1"
    assert cmd[-len(argv):] == argv                                        # same script, same arguments
    assert replicas.launch_plan(0, {}, argv) is None
