"""The N > 1 benchmark path on CPU: two gloo ranks draw different batches, reduce their timings with
the maximum over ranks, and compose the same whole-job figure (no GPU needed)."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2603_06738_b200 import multi, synthetic


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        wl = multi.rank_workload(synthetic.Workload("t", 1, 8, 8, 2, 8, 8, 4, 2, seed=5), rank)
        q = synthetic.make_inputs(wl, False)["q"]
        my_ms = [10.0 + 5.0 * rank, 3.0 - rank]                  # rank 1 is slower on the first, faster on the second
        red = multi.max_over_ranks(my_ms)
        gathered = [None] * world
        dist.all_gather_object(gathered, (wl.seed, float(q.float().sum()), red))
        if rank == 0:
            out.put(gathered)
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_reduce_times_and_draw_distinct_batches():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    gathered = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (seed0, sum0, red0), (seed1, sum1, red1) = gathered
    assert seed0 == 5 and seed1 == 1005 and sum0 != sum1          # independent batches
    assert red0 == red1 == [15.0, 3.0]                            # max over ranks, same on every rank
    assert multi.job_throughput(100.0, red0[0], 2) == pytest.approx(2 * 100.0 / 15e-3)


def test_single_process_is_identity():
    assert multi.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert multi.job_throughput(10.0, 2.0, 1) == pytest.approx(5000.0)
