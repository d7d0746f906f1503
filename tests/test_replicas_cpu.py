"""The benchmark's multi-GPU plumbing on two gloo ranks (CPU): the job's time is the slowest rank's,
ranks draw different token batches, the aggregate counts every rank's work, and no rank's data is
touched by another (the only collectives are the barrier and the MAX of one float)."""
import os
import socket

import numpy as np
import torch
import torch.multiprocessing as mp

from paper_2501_01144_b200 import inputs, replicas


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    assert replicas.world_from_env() == (rank, world, rank)
    assert replicas.init("gloo") == world
    replicas.barrier()
    # each rank "measures" its own time; the job's time is the maximum
    mine = 1.5 + rank
    slowest = replicas.max_over_ranks(mine)
    # each rank's token batch comes from its own seed
    xb = inputs.act_student_t(8, 64, seed=replicas.rank_seed(2, rank))
    replicas.barrier()
    out.put((rank, slowest, replicas.whole_job_rate(10.0, slowest, world), int(np.asarray(xb, np.uint16).sum())))
    replicas.shutdown()


def test_two_gloo_ranks_share_only_the_clock():
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
    assert [r[0] for r in results] == [0, 1]
    assert all(abs(r[1] - 2.5) < 1e-12 for r in results)             # max(1.5, 2.5) on both ranks
    assert all(abs(r[2] - 2 * 10.0 / 2.5) < 1e-12 for r in results)  # both ranks' units over the slowest time
    assert results[0][3] != results[1][3]                            # different token batches


def test_single_process_is_a_no_op():
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK"):
        os.environ.pop(k, None)
    assert replicas.world_from_env() == (0, 1, 0)
    assert replicas.init("gloo") == 1
    replicas.barrier()
    assert replicas.max_over_ranks(3.25) == 3.25
    assert replicas.whole_job_rate(4.0, 2.0, 1) == 2.0
    replicas.shutdown()
