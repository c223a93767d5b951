"""World-size-2 check (gloo, CPU) of the benchmark's multi-process plumbing: replicas draw
different activations, the job time is the slowest rank's, the job throughput counts every
rank's tokens."""
import os
import socket

import torch
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from paper_2505_19645_b200 import replicas, workloads as wl

    r, w = replicas.init("gloo")
    assert (r, w) == (rank, world)
    shape = wl.small_shape("g", 64, 4, 2, 64)
    x = wl.make_tokens(shape, 8, replicas.replica_seed(5, rank))
    replicas.barrier()
    # rank 1 is the slow replica
    tput, ms = replicas.job_throughput(128.0, 2.0 + 3.0 * rank)
    q.put((rank, tput, ms, float(x.float().sum())))
    replicas.shutdown()


def test_two_replicas_over_gloo():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (_, t0, ms0, s0), (_, t1, ms1, s1) = res
    assert ms0 == ms1 == 5.0                      # max over ranks
    assert t0 == t1 == 256.0 / 5e-3               # all ranks' tokens / slowest time
    assert s0 != s1                               # replicas see different activations


def test_single_process_defaults():
    from paper_2505_19645_b200 import replicas

    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        os.environ.pop(k, None)
    assert replicas.env_world() == (0, 0, 1)
    assert replicas.job_throughput(10.0, 2.0) == (5000.0, 2.0)
    assert torch.distributed.is_initialized() is False
