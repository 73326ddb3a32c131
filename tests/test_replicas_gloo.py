"""The multi-GPU arrangement is N independent replicas; its host-side logic
(barrier, max-over-ranks time, whole-job throughput) runs here on CPU with two
gloo ranks."""
import os

import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2505_10526_b200.replicas import aggregate_throughput, barrier, max_over_ranks, world_size
    barrier()
    assert world_size() == world
    slowest = max_over_ranks(2.0 + rank)                  # rank 0: 2 ms, rank 1: 3 ms
    ms, value = aggregate_throughput(96, 2.0 + rank)
    out[rank] = (slowest, ms, value)
    barrier()
    dist.destroy_process_group()


def test_two_replicas_report_slowest_time_and_whole_job_throughput():
    import __graft_entry__ as entry
    entry.build()
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, 29611, out), nprocs=world, join=True)
        res = dict(out)
    for rank in range(world):
        slowest, ms, value = res[rank]
        assert slowest == 3.0 and ms == 3.0
        assert abs(value - 2 * 96 / 3.0e-3) < 1e-6


def test_single_process_is_a_world_of_one():
    import __graft_entry__ as entry
    entry.build()
    from paper_2505_10526_b200.replicas import aggregate_throughput, world_size
    assert world_size() == 1
    ms, value = aggregate_throughput(6, 0.2)
    assert ms == 0.2 and abs(value - 30000.0) < 1e-6
