"""Host logic of the multi-rank path (layers sharded over ranks, no data-path collective), run
as two gloo ranks on the CPU: which layers each rank takes, and that the whole-job figure is
built from the slowest rank's time."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    from paper_2605_08692_b200 import sharding, synth
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        mine = sharding.layers_for_rank(7, rank, world)
        # every rank reports a different step time; all must agree on the slowest
        ms = sharding.max_over_ranks(10.0 + 5.0 * rank)
        # weak scaling: different seeds give different synthetic layers of the same shape
        w = synth.weights(4, 64, sharding.seed_for_rank(0, rank), "shard/W")
        gathered = [None] * world
        dist.all_gather_object(gathered, (mine, ms, int(w.astype("int64").sum())))
        if rank == 0:
            out.put(gathered)
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_layers_and_agree_on_the_step_time():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    got = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (l0, ms0, s0), (l1, ms1, s1) = got
    assert sorted(l0 + l1) == list(range(7)) and not set(l0) & set(l1)
    assert ms0 == ms1 == 15.0
    assert s0 != s1                                   # ranks hold different data


def test_job_throughput_and_single_process_fallback():
    sys.path.insert(0, ROOT)
    from paper_2605_08692_b200 import sharding
    assert sharding.max_over_ranks(3.5) == 3.5                      # no process group: identity
    # two ranks, 1e9 weights each, 20 rounds in 100 ms -> 400 Gweights/s per round
    assert sharding.job_throughput(10**9, 20, 100.0, 2) == pytest.approx(400.0)
    assert sharding.job_throughput([10**9, 3 * 10**9], 1, 1000.0, 2) == pytest.approx(4.0)
    with pytest.raises(ValueError):
        sharding.layers_for_rank(3, 2, 2)
