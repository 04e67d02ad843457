"""World-size-2 gloo test of the multi-rank bookkeeping used by bench.py --gpus N."""
import os
import socket

import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2605_06068_b200 import sharding


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank r "measured" (10 + r) ms per step and did (100 + r) units of work
    t, w = sharding.aggregate([10.0 + rank, 5.0 - rank], [100.0 + rank, 1.0])
    own = sharding.shard_sequences(7, rank, world)
    out.put((rank, t, w, list(own), sharding.rank_seed(43, rank)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_aggregation_and_shards():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, t, w, own, seed in res:
        assert t == [11.0, 5.0]          # max over ranks
        assert w == [201.0, 2.0]         # sum over ranks
        assert seed == 43 + 1000 * rank
    assert res[0][3] + res[1][3] == list(range(7)) and len(res[0][3]) == 4


def test_single_process_is_identity():
    t, w = sharding.aggregate([3.0], [7.0])
    assert t == [3.0] and w == [7.0]
    assert list(sharding.shard_sequences(5, 0, 1)) == [0, 1, 2, 3, 4]
    assert sharding.rank_seed(42, 0) == 42
