"""The multi-GPU plumbing (independent replicas: barrier + maximum over ranks) on two CPU processes over gloo."""
import os
import socket

import torch
import torch.multiprocessing as mp

from paper_2601_22379_b200 import replicas


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), WORLD_SIZE=str(world), RANK=str(rank),
                      LOCAL_RANK=str(rank))
    assert replicas.env_world() == (world, rank, rank)
    assert replicas.init("gloo") == (world, rank)
    replicas.barrier()
    # every rank reports its own times; the slowest one counts
    step_ms, e2e_ms = replicas.max_over_ranks([10.0 + rank, 30.0 - 5.0 * rank])
    rate = replicas.whole_job_rate(units_per_rank_per_step=128, steps=1000, ms_max=step_ms)
    out[rank] = (step_ms, e2e_ms, rate)
    replicas.barrier()
    replicas.shutdown()


def test_two_replicas_report_the_slowest_rank_and_the_whole_job_rate():
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]                                  # every rank ends with the same figures
    step_ms, e2e_ms, rate = res[0]
    assert step_ms == 11.0 and e2e_ms == 30.0
    assert abs(rate - 128 * 2 * 1000 / 11.0e-3) < 1e-6 * rate


def test_single_process_needs_no_process_group():
    for k in ("WORLD_SIZE", "RANK", "LOCAL_RANK"):
        os.environ.pop(k, None)
    assert replicas.env_world() == (1, 0, 0)
    assert replicas.init("gloo") == (1, 0)
    assert replicas.max_over_ranks([3.0, 4.0]) == [3.0, 4.0]
    assert replicas.whole_job_rate(128, 10, 2.0) == 128 * 10 / 2.0e-3
    replicas.barrier()
    replicas.shutdown()
