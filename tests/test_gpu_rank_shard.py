"""GPU side of the rank-sharded form: the library's joint-reduction primitive (trv_joint_reduce) against the oracle,
and the whole rank-sharded driver with every rank hosted by this one GPU (the exchange then moves nothing between
processes; with more GPUs it goes through NCCL point-to-point operations, covered on CPU by test_rank_shard_gloo.py)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_17254_b200 import binding, build, rank_shard, synth

from gpu_util import DEV

pytestmark = pytest.mark.gpu
LAT, BW = binding.LATENCY_OPTIMAL, binding.BANDWIDTH_OPTIMAL


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    assert torch.cuda.is_available()
    binding.lib()


@pytest.mark.parametrize("dist,count,shift", [("normal", 10007, 0), ("int32", 4096, 0), ("normal", 5001, 1), ("uniform", 777, 3), ("normal", 3, 2)])
def test_joint_reduce_is_one_trivance_step(dist, count, shift):
    """A ring of three runs ONE latency-form step: rank p ends with (x[p-1] + x[p]) + x[p+1] (Sec. 4.2).  The three
    segments start `shift` elements into their buffers (unaligned starts take the scalar form)."""
    x = synth.rank_matrix(dist, 61, 3, count)
    want = oracle.allreduce((3,), oracle.VARIANT_LATENCY, x)
    tdt = torch.int32 if dist == "int32" else torch.float32
    src = torch.zeros((3, count + 8), dtype=tdt, device=DEV)
    dst = torch.full((3, count + 8), 5, dtype=tdt, device=DEV)
    for r in range(3):
        src[r, shift:shift + count].copy_(torch.from_numpy(x[r]))
    es = src.element_size()
    sp = [src[r].data_ptr() + shift * es for r in range(3)]
    dp = [dst[r].data_ptr() + shift * es for r in range(3)]
    dcode = binding.INT32 if dist == "int32" else binding.FLOAT32
    before = binding.launch_count()
    binding.joint_reduce([sp[2], sp[0], sp[1]], sp, [sp[1], sp[2], sp[0]], dp, [count] * 3, dcode, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert binding.launch_count() == before + 1 and binding.last_kernel_name() == "joint_reduce"
    got = dst[:, shift:shift + count].cpu().numpy()
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    assert (dst[:, :shift] == 5).all().item() and (dst[:, shift + count:] == 5).all().item()    # nothing outside the segments


def test_joint_reduce_missing_sides_mixed_alignment_and_many_segments():
    rng = np.random.default_rng(3)
    k, width = 1300, 41                 # more segments than one launch carries
    a = rng.standard_normal((k, width)).astype(np.float32)
    b = rng.standard_normal((k, width)).astype(np.float32)
    c = rng.standard_normal((k, width)).astype(np.float32)
    ad, bd, cd = (torch.from_numpy(v).to(DEV) for v in (a, b, c))
    od = torch.zeros_like(ad)
    left = [ad[i].data_ptr() if i % 3 != 0 else 0 for i in range(k)]
    right = [cd[i].data_ptr() if i % 5 != 0 else 0 for i in range(k)]
    counts = [width if i % 7 else 0 for i in range(k)]
    before = binding.launch_count()
    binding.joint_reduce(left, [bd[i].data_ptr() for i in range(k)], right, [od[i].data_ptr() for i in range(k)], counts,
                         binding.FLOAT32, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert binding.launch_count() - before == 3
    want = np.zeros_like(a)
    for i in range(k):
        if counts[i]:
            v = b[i]
            if left[i]:
                v = a[i] + v
            if right[i]:
                v = v + c[i]
            want[i] = v
    assert np.array_equal(od.cpu().numpy().view(np.uint32), want.view(np.uint32))
    with pytest.raises(binding.TrivanceError):
        binding.joint_reduce([0], [bd[0].data_ptr() + 2], [0], [od[0].data_ptr()], [4], binding.FLOAT32)    # misaligned


@pytest.mark.parametrize("dims,variant,count,dist", [((27,), LAT, 5003, "normal"), ((9, 9), LAT, 3001, "int32"), ((9, 9), BW, 4001, "normal"),
                                                     ((81,), BW, 9001, "normal"), ((3, 3, 3), BW, 2000, "normal"), ((10,), BW, 3001, "normal"),
                                                     ((4, 4), BW, 1999, "normal")])
def test_rank_sharded_driver_on_one_gpu(dims, variant, count, dist):
    plan = binding.Plan(dims, variant)
    x = synth.rank_matrix(dist, 62, plan.n, count)
    local = torch.from_numpy(x).to(DEV)
    engine = rank_shard.RankSharded(plan, 1, 0, lambda sends, recvs: None)      # one process: nothing to exchange
    before = binding.launch_count()
    engine(local)
    torch.cuda.synchronize()
    assert binding.launch_count() > before and binding.last_kernel_name() == "joint_reduce"
    want = oracle.allreduce(dims, variant, x)
    assert np.array_equal(local.cpu().numpy().view(np.uint32), want.view(np.uint32))
    plan.destroy()
