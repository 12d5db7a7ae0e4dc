"""Rank-sharded Trivance on CPU: gloo processes each host a contiguous range of the ranks and exchange, step by
step, the messages the schedule defines (whole slices in the latency form, block sets in the bandwidth form).  What
is under test is the exchange bookkeeping of rank_shard.py; the joint reduction itself is a plain torch stand-in here
(on GPUs it is the library's trv_joint_reduce, see test_gpu_rank_shard.py).  The gathered rows must equal the oracle's
bit for bit."""
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


def cpu_reduce_segments(left, own, right, out):
    """(left + own) + right in binary32 / wrapping int32, one rounding per add; a missing side is left out."""
    for l, o, r, dst in zip(left, own, right, out):
        v = o.clone()
        if l is not None:
            v = l + v
        if r is not None:
            v = v + r
        dst.copy_(v)


def _worker(rank, world, port, cases, ret):
    sys.path.insert(0, ROOT)
    import oracle
    from paper_2602_17254_b200 import binding, rank_shard, synth
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ok = True
    try:
        for dims, variant, count, dist_name in cases:
            plan = binding.Plan(dims, variant)
            n = plan.n
            x = synth.rank_matrix(dist_name, 17, n, count)
            lo, hi = rank_shard.rank_range(n, world, rank)
            local = torch.from_numpy(x[lo:hi].copy())
            engine = rank_shard.RankSharded(plan, world, rank, rank_shard.torch_exchange(), cpu_reduce_segments)
            engine(local)
            rows = [None] * world
            dist.all_gather_object(rows, local.numpy())
            if rank == 0:
                got = np.concatenate(rows, axis=0)
                want = oracle.allreduce(dims, variant, x)
                same = np.array_equal(got.view(np.uint32), want.view(np.uint32))
                if not same:
                    print("MISMATCH", dims, variant, count, flush=True)
                ok = ok and same
        if rank == 0:
            ret["ok"] = ok
    finally:
        dist.destroy_process_group()


CASES = [((9,), 0, 1001, "normal"), ((9,), 1, 1001, "normal"), ((3, 3), 0, 514, "int32"), ((3, 3), 1, 515, "normal"),
         ((27,), 1, 300, "normal"), ((3, 9), 1, 700, "normal"), ((3, 3, 3), 0, 301, "normal"),
         ((7,), 1, 500, "normal"), ((4, 4), 1, 333, "normal"), ((2, 5), 1, 97, "int32"), ((2,), 1, 10, "normal")]


@pytest.mark.parametrize("world", [2, 3])
def test_rank_sharded_allreduce_equals_the_oracle(world):
    port = _free_port()
    mgr = mp.Manager()
    ret = mgr.dict()
    mp.spawn(_worker, args=(world, port, CASES, ret), nprocs=world, join=True)
    assert ret.get("ok") is True


def test_rank_ranges_tile_the_ranks():
    from paper_2602_17254_b200 import rank_shard
    for n in (2, 9, 27, 100, 729):
        for world in (1, 2, 3, 4, 8):
            if world > n:
                continue
            pieces = [rank_shard.rank_range(n, world, g) for g in range(world)]
            assert pieces[0][0] == 0 and pieces[-1][1] == n
            assert all(a[1] == b[0] for a, b in zip(pieces, pieces[1:]))
            for r in range(n):
                g = rank_shard.host_of(n, world, r)
                assert pieces[g][0] <= r < pieces[g][1]


def test_the_product_refuses_cpu_tensors():
    from paper_2602_17254_b200 import rank_shard
    t = torch.zeros(8)
    with pytest.raises(RuntimeError):
        rank_shard.cuda_reduce_segments([None], [t], [None], [t])
