"""The N>1 host logic (rank seeding, barrier, max-over-ranks timing) on two gloo ranks on CPU."""
import os
import socket

import torch
import torch.multiprocessing as mp

from paper_2603_14303_b200 import dist as scdist
from paper_2603_14303_b200 import synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), LOCAL_RANK=str(rank),
                      WORLD_SIZE=str(world))
    assert scdist.env_rank() == (rank, rank, world)
    scdist.init("gloo")
    w = scdist.rank_workload(synth.config(0, n=512), rank)
    ids, _, _ = synth.token_ids(w)
    scdist.barrier()
    # each rank reports its own timings; every rank must end up with the slowest one
    ms = scdist.max_over_ranks([10.0 + rank, 5.0 - rank, 7.0])
    out.put((rank, w.seed, int(ids.sum()), ms))
    scdist.barrier()
    torch.distributed.destroy_process_group()


def test_two_gloo_ranks_own_batches_and_max_timing():
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
    (r0, s0, sum0, ms0), (r1, s1, sum1, ms1) = got
    assert (r0, r1) == (0, 1) and s1 == s0 + 1000 and sum0 != sum1      # independent seeded batches
    assert ms0 == ms1 == [11.0, 5.0, 7.0]                               # max over ranks, same on both
    assert scdist.whole_job_rate(32, 2, 1000.0) == 64.0


def test_single_process_is_the_identity():
    assert scdist.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    w = synth.config(0)
    assert scdist.rank_workload(w, 0) is w
