"""The N > 1 plumbing (independent replicas, max-over-ranks timing) with two gloo ranks on the CPU."""
import os
import socket

import torch
import torch.multiprocessing as mp


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out):
    os.environ.update({"RANK": str(rank), "LOCAL_RANK": str(rank), "WORLD_SIZE": str(world),
                       "MASTER_ADDR": "127.0.0.1", "MASTER_PORT": str(port)})
    from paper_2602_22700_b200 import synth
    from paper_2602_22700_b200.replicas import Replicas
    rep = Replicas(backend="gloo")
    assert (rep.rank, rep.world) == (rank, world)
    rep.barrier()
    seconds = 0.010 * (rank + 1)                       # rank 1 is the slow one
    slowest = rep.max_over_ranks(seconds)
    rate = rep.whole_job_rate(1000.0, seconds)
    a = synth.gauss_i8(rep.seed(1), synth.tid(0, synth.ROLE_ACT), 4, 16, synth.Q_SIGMA20)
    out.put((rank, slowest, rate, a.tolist()))
    rep.barrier()
    rep.close()


def test_two_replicas_report_the_slowest_time_and_the_sum_of_units():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, slow0, rate0, data0), (r1, slow1, rate1, data1) = got
    assert (r0, r1) == (0, 1)
    assert slow0 == slow1 == 0.020                      # the maximum over ranks, on every rank
    assert rate0 == rate1 == 2 * 1000.0 / 0.020         # all units over the slowest replica's time
    assert data0 != data1                                # replicas work on different seeded inputs


def test_single_process_needs_no_group():
    from paper_2602_22700_b200.replicas import Replicas
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        os.environ.pop(k, None)
    rep = Replicas(backend="gloo")
    assert rep.world == 1 and rep.dist is None
    assert rep.max_over_ranks(1.5) == 1.5 and rep.whole_job_rate(10.0, 2.0) == 5.0 and rep.seed(7) == 7
    rep.barrier()
