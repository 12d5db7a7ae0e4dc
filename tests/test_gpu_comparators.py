"""GPU parity for the comparison algorithms as executable data paths (Sec. 2.4, 3.1): Bruck with joint reductions,
Recursive Doubling, Swing, the ring (Bucket) algorithm and their mirrored forms through trv_allreduce_ex / trv_allreduce,
bit-exact against the oracle's message-by-message execution of the same schedules."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_17254_b200 import binding, build, synth

from gpu_util import DEV, torch_dtype

pytestmark = pytest.mark.gpu
LAT, BW = binding.LATENCY_OPTIMAL, binding.BANDWIDTH_OPTIMAL
CASES = [(binding.ALGO_BRUCK, (9,)), (binding.ALGO_BRUCK, (27,)), (binding.ALGO_BRUCK, (81,)), (binding.ALGO_BRUCK, (3, 9)), (binding.ALGO_BRUCK, (9, 9)),
         (binding.ALGO_RECDOUB, (2,)), (binding.ALGO_RECDOUB, (8,)), (binding.ALGO_RECDOUB, (64,)), (binding.ALGO_SWING, (8,)),
         (binding.ALGO_SWING, (32,)), (binding.ALGO_SWING, (128,)), (binding.ALGO_BUCKET, (5,)), (binding.ALGO_BUCKET, (12,)), (binding.ALGO_BUCKET, (30,)),
         (binding.ALGO_BUCKET, (4, 4)), (binding.ALGO_BUCKET, (3, 5)), (binding.ALGO_BUCKET, (2, 3, 4)), (binding.ALGO_BUCKET, (8, 8))]


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    assert torch.cuda.is_available()
    binding.lib()


def _run(algo, dims, variant, count, dist, seed, in_place=True, shard=None, via_allreduce=False):
    plan = binding.Plan(dims, variant, algo)
    n = plan.n
    x = synth.rank_matrix(dist, seed, n, count)
    pad = (count + 3) // 4 * 4
    buf = torch.zeros((n, pad + 4), dtype=torch_dtype(x.dtype), device=DEV)
    xd = buf[:, :count]
    xd.copy_(torch.from_numpy(x))
    obuf = torch.full((n, pad + 4), -77, dtype=buf.dtype, device=DEV)
    gc, go = (count, 0) if shard is None else shard
    stream = torch.cuda.current_stream().cuda_stream
    dcode = binding.INT32 if x.dtype == np.int32 else binding.FLOAT32
    ip = [xd[r].data_ptr() for r in range(n)]
    if via_allreduce:
        plan.allreduce(ip, count, dcode, stream)            # the in-place call; the plan owns the wire buffer
        res = xd
    else:
        need = plan.scratch_bytes(count, binding.KERNEL_AUTO, in_place=in_place)
        assert need > 0
        scratch = torch.empty(need, dtype=torch.uint8, device=DEV)
        op = None if in_place else [obuf[r].data_ptr() for r in range(n)]
        plan.allreduce_ex(ip, op, count, dcode, global_count=gc, global_offset=go, kernel=binding.KERNEL_AUTO,
                          scratch_ptr=scratch.data_ptr(), scratch_bytes=need, stream=stream)
        res = xd if in_place else obuf[:, :count]
    torch.cuda.synchronize()
    assert binding.last_kernel_name() == "comparator_steps"
    want = oracle.allreduce_algo(dims, variant, x, algo, E=gc, e0=go)
    got = res.cpu().numpy()
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    if in_place or via_allreduce:
        assert torch.count_nonzero(buf[:, count:]).item() == 0, "wrote past the end of a rank buffer"
    else:
        assert (obuf[:, count:] == -77).all().item() and np.array_equal(xd.cpu().numpy(), x)
    plan.destroy()


@pytest.mark.parametrize("algo,dims", CASES)
@pytest.mark.parametrize("mirror", [0, binding.ALGO_MIRRORED])
def test_comparator_data_paths_match_the_oracle(algo, dims, mirror):
    if mirror and len(dims) > 1 and algo == binding.ALGO_BRUCK:
        pytest.skip("Bruck's mirrored sub-collective is defined on rings")
    for variant in (LAT, BW):
        if algo == binding.ALGO_BUCKET and variant == LAT:
            continue
        _run(algo | mirror, dims, variant, 3001, "normal", 71)
        _run(algo | mirror, dims, variant, 2049, "int32", 72, in_place=False)


@pytest.mark.parametrize("algo,dims", [(binding.ALGO_BRUCK, (27,)), (binding.ALGO_RECDOUB, (16,)), (binding.ALGO_SWING, (16,)), (binding.ALGO_BUCKET, (7,))])
def test_windows_short_vectors_and_the_in_place_call(algo, dims):
    gcount = 20011
    for variant in (LAT, BW):
        if algo == binding.ALGO_BUCKET and variant == LAT:
            continue
        for lo, hi in ((0, 10004), (10004, gcount), (5000, 5000 + 2048)):
            _run(algo, dims, variant, hi - lo, "int32", 73, shard=(gcount, lo))
        for count in (1, 5, 64):
            _run(algo | binding.ALGO_MIRRORED, dims, variant, count, "normal", 74, in_place=False)
        _run(algo, dims, variant, 4100, "normal", 75, via_allreduce=True)


TORUS_CASES = [(binding.ALGO_RECDOUB, (4, 4)), (binding.ALGO_RECDOUB, (2, 8)), (binding.ALGO_SWING, (8, 8)), (binding.ALGO_SWING, (4, 4, 4)),
               (binding.ALGO_RECDOUB, (4, 4, 4))]


@pytest.mark.parametrize("algo,dims", TORUS_CASES)
@pytest.mark.parametrize("flag", [0, binding.ALGO_MIRRORED, binding.ALGO_SINGLE])
def test_recursive_doubling_and_swing_on_tori(algo, dims, flag):
    """Sec. 2.4, Table 2: one collective per dimension, 2 D when mirrored, or a single one walking through the dimensions:
    data paths bit-exact against the oracle, link loads and cost model equal to its hop-by-hop tally."""
    for variant in (LAT, BW):
        _run(algo | flag, dims, variant, 3001, "normal", 81)
        _run(algo | flag, dims, variant, 1025, "int32", 82, in_place=False)
        plan = binding.Plan(dims, variant, algo | flag)
        got = plan.link_loads(100003, 4)
        want = oracle.link_loads(dims, variant, 100003, 4, algo=algo | flag)
        for k in ("msgs", "bytes", "max_msgs", "max_bytes"):
            assert got[k].dtype == want[k].dtype and np.array_equal(got[k], want[k]), k
        c, w = plan.cost_model(100003, 4, 1.5e-6, 1e-11), oracle.cost_model(dims, variant, 100003, 4, 1.5e-6, 1e-11, algo | flag)
        assert c.steps == w["steps"] and c.tx_bytes == w["tx_bytes"] and c.bytes_sent_per_node == w["bytes_sent_per_node"]
        assert np.isclose(c.theta, w["theta"], rtol=1e-12) and np.isclose(c.delta, w["delta"], rtol=1e-12)
        plan.destroy()


def test_what_the_comparators_do_not_serve():
    plan = binding.Plan((16,), LAT, binding.ALGO_SWING)
    assert plan.kernel_supported(binding.KERNEL_AUTO) and plan.kernel_supported(binding.KERNEL_STEP)
    assert not plan.kernel_supported(binding.KERNEL_FUSED) and not plan.kernel_supported(binding.KERNEL_PIPELINED)
    x = torch.zeros((16, 64), device=DEV)
    with pytest.raises(binding.TrivanceError) as e:
        plan.allreduce_ex([x[r].data_ptr() for r in range(16)], None, 64, binding.FLOAT32, kernel=binding.KERNEL_FUSED)
    assert e.value.status == binding.ERR_UNSUPPORTED
    with pytest.raises(binding.TrivanceError) as e:
        plan.allreduce_ex([x[r].data_ptr() for r in range(16)], None, 64, binding.FLOAT32)      # no wire buffer given
    assert e.value.status == binding.ERR_SCRATCH
    with pytest.raises(binding.TrivanceError) as e:             # the ring algorithm has no latency-optimal form
        binding.Plan((7,), LAT, binding.ALGO_BUCKET)
    assert e.value.status == binding.ERR_UNSUPPORTED
