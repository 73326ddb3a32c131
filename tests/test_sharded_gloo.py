"""The exchange of the vocabulary-sharded acceptance on two CPU ranks (gloo): the communicator's gather is
rank-major and a rank's phase generator is driven to the end with every rank seeing the same gathered
values.  No kernel runs here; the phases are a stand-in that only exchanges."""
import os

import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _phases(rank):
    a = yield torch.full((6,), float(rank))
    b = yield torch.tensor([rank * 10, -1 if rank == 0 else 7], dtype=torch.int32)
    c = yield torch.arange(4, dtype=torch.float64) + 100 * rank
    return a, b, c


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2505_10526_b200.sharded import DistComm, drive
    comm = DistComm()
    assert (comm.world, comm.rank) == (world, rank)
    a, b, c = drive(_phases(rank), comm)
    out[rank] = (a.tolist(), b.tolist(), c.tolist())
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_exchange_in_rank_order():
    import __graft_entry__ as entry
    entry.build()
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, 29633, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]                                       # every rank sees the same values
    a, b, c = res[0]
    assert a == [0.0] * 6 + [1.0] * 6                             # rank 0's copy, then rank 1's
    assert b == [0, -1, 10, 7]
    assert c == [0.0, 1.0, 2.0, 3.0, 100.0, 101.0, 102.0, 103.0]


def test_lockstep_driver_matches_the_collectives():
    """The single-device stand-in combines the ranks' requests the way the collectives do."""
    import __graft_entry__ as entry
    entry.build()
    from paper_2505_10526_b200.sharded import run_lockstep

    class Rank:
        def __init__(self, r):
            self.r = r

        def phases(self):
            return _phases(self.r)

    res = run_lockstep([Rank(0), Rank(1)], [{}, {}])
    for a, b, c in res:
        assert a.tolist() == [0.0] * 6 + [1.0] * 6
        assert b.tolist() == [0, -1, 10, 7]
        assert c.tolist() == [0.0, 1.0, 2.0, 3.0, 100.0, 101.0, 102.0, 103.0]
