"""Multi-rank logic of bench.py on CPU (gloo, world_size 2): the whole-job step time is the MAX
over ranks, every rank draws its own input shard, and only rank 0 of the reference arm works."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert bench.dist_env() == (rank, world, rank)
        # rank 1 is the slow one: both ranks must report its time
        ms = bench.max_over_ranks(1.5 + 2.0 * rank, world)
        out[rank] = ms
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_step_time_is_the_max_over_ranks():
    world = 2
    out = mp.Manager().dict()
    port = 29500 + (os.getpid() % 2000)
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    assert out[0] == pytest.approx(3.5) and out[1] == pytest.approx(3.5)


def test_ranks_draw_disjoint_shards_and_single_rank_is_identity():
    import bench
    from paper_2605_26636_b200 import inputs
    a, b = bench.rank_layer_ids(0, 3), bench.rank_layer_ids(1, 3)
    assert not set(a) & set(b)
    w = inputs.WORKLOADS["dinov3_l"]
    seeds = {inputs.seed_for(w.cfg, l, t) for l in a + b for t in range(3)}
    assert len(seeds) == 18                      # no two tensors of the two ranks share a seed
    assert bench.max_over_ranks(2.25, 1) == 2.25


def test_reference_arm_runs_on_rank_zero_only(monkeypatch, capsys):
    import bench
    monkeypatch.setenv("RANK", "1")
    monkeypatch.setenv("WORLD_SIZE", "2")

    class A:
        steps, warmup, gpus = 1, 0, 2
    bench.run_reference(A)                        # returns at once: no oracle work, no output
    assert capsys.readouterr().out == ""
