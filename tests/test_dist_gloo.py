"""World-size-2 checks of the multi-GPU plumbing on CPU (gloo): sequence sharding covers the
batch exactly once and the timing reduction is a max over ranks."""
import os
import sys

import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(world))
    import torch.distributed as dist
    from paper_2607_27735_b200 import dist_util

    dist_util.init_process_group("gloo")
    mine = list(dist_util.shard_sequences(7, world, rank))
    t = dist_util.max_over_ranks(10.0 + rank, world)
    gathered = [None] * world
    dist.all_gather_object(gathered, mine)
    dist.barrier()
    q.put((rank, t, gathered))
    dist.destroy_process_group()


def test_two_rank_sharding_and_max_reduce():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29600 + os.getpid() % 300
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = [q.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, t, gathered in res:
        assert t == 11.0
        assert sorted(sum(gathered, [])) == list(range(7))
        assert abs(len(gathered[0]) - len(gathered[1])) <= 1


def test_single_rank_is_identity():
    from paper_2607_27735_b200 import dist_util

    assert dist_util.max_over_ranks(3.5, 1) == 3.5
    assert list(dist_util.shard_sequences(5, 1, 0)) == [0, 1, 2, 3, 4]
