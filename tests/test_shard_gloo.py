"""Multi-GPU path on CPU: world_size-2 gloo ranks each take an element-range shard (global element
index carried along), reduce it with no data-path collective, and the gathered shards equal the
unsharded result.  The reduction itself is done by the oracle here (no GPU): what is under test is
the partition and the global-index bookkeeping that bench.py --gpus N and trv_allreduce_ex rely on."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, dims, variant, count, ret):
    sys.path.insert(0, ROOT)
    import oracle
    from paper_2602_17254_b200 import shard, synth
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        n = int(np.prod(dims))
        off, ln = shard.element_shard(count, world, rank)
        x = synth.rank_matrix("normal", 7, n, count)[:, off:off + ln]
        mine = oracle.allreduce(dims, variant, np.ascontiguousarray(x), E=count, e0=off)
        # gather (offset, length, values) on every rank: plumbing only, no data-path collective
        meta = [None] * world
        dist.all_gather_object(meta, (off, ln))
        objs = [None] * world
        dist.all_gather_object(objs, mine)
        parts = [torch.from_numpy(o) for o in objs]
        t = torch.tensor([float(rank + 1)])
        dist.all_reduce(t, op=dist.ReduceOp.MAX)          # the max-over-ranks reduction bench.py does on its time
        if rank == 0:
            full = oracle.allreduce(dims, variant, synth.rank_matrix("normal", 7, n, count))
            got = np.concatenate([p.numpy() for p in parts], axis=1)
            ret["ok"] = bool(np.array_equal(got, full)) and meta[0][0] == 0 and sum(m[1] for m in meta) == count \
                and all(m[0] % 4 == 0 for m in meta) and float(t) == world
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("dims,variant,count", [((9,), 0, 1001), ((9, 9), 1, 1003), ((3, 3, 3), 0, 998), ((27,), 1, 64)])
def test_two_rank_element_shards_reproduce_the_unsharded_result(dims, variant, count):
    port = _free_port()
    mgr = mp.Manager()
    ret = mgr.dict()
    mp.spawn(_worker, args=(2, port, dims, variant, count, ret), nprocs=2, join=True)
    assert ret.get("ok") is True


def test_element_shard_tiles_the_vector():
    from paper_2602_17254_b200 import shard
    for count in (0, 1, 3, 4, 5, 1000, 1001, 8388608):
        for world in (1, 2, 3, 4, 8):
            pieces = [shard.element_shard(count, world, r) for r in range(world)]
            assert pieces[0][0] == 0 and sum(p[1] for p in pieces) == count
            for (o1, l1), (o2, _) in zip(pieces, pieces[1:]):
                assert o1 + l1 == o2 and o2 % 4 == 0
    with pytest.raises(ValueError):
        shard.element_shard(10, 2, 2)
