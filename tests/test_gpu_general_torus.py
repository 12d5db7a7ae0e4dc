"""GPU parity for tori with a side that is no power of three (Sec. 4.4 per dimension, Sec. 5): the STEP kernels, the
fused tree-walk kernel and the link-load tally through the C ABI vs the CPU oracle, bit-exact."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_17254_b200 import binding, build, synth

from gpu_util import DEV, check_case, check_scattered

pytestmark = pytest.mark.gpu

BW = binding.BANDWIDTH_OPTIMAL
AUTO, STEP, FUSED = binding.KERNEL_AUTO, binding.KERNEL_STEP, binding.KERNEL_FUSED
TORI = [(4, 4), (8, 8), (7, 3), (3, 10), (2, 5), (5, 5), (2, 2), (4, 4, 4), (2, 3, 4), (6, 9), (16, 8), (2, 2, 2, 2), (8, 64), (32, 32)]


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    assert torch.cuda.is_available()
    binding.lib()


@pytest.mark.parametrize("dims", TORI)
def test_matches_oracle(dims):
    n = int(np.prod(dims))
    count = 4099 if n <= 128 else 2053      # blocks of ragged length, unaligned block and slice starts
    check_case(dims, BW, count, "normal", 41, FUSED)
    check_case(dims, BW, count, "int32", 42, STEP, in_place=False)
    check_case(dims, BW, count, "int32", 42, FUSED, in_place=False)
    check_case(dims, BW, count, "normal", 41, STEP)
    check_scattered(dims, BW, count, "uniform", 43, AUTO)
    check_scattered(dims, BW, count, "uniform", 43, STEP)


@pytest.mark.parametrize("dims", [(4, 4), (7, 3), (4, 4, 4)])
@pytest.mark.parametrize("count", [1, 2, 5, 31, 63, 64, 65])
def test_short_vectors(dims, count):
    """Fewer elements than ranks x collectives: most blocks are empty, some collectives too."""
    check_case(dims, BW, count, "int32", 44, AUTO)
    check_case(dims, BW, count, "normal", 45, STEP, in_place=False)


@pytest.mark.parametrize("dims,count", [((8, 8), (1 << 20) + 6), ((4, 4, 4), (1 << 20) + 3), ((16, 8), (1 << 20) + 1)])
def test_two_columns_per_thread_path(dims, count):
    """Long vectors take the kernel with two columns per thread; block and slice boundaries fall inside some pairs.
    (The largest tori run this path at full size in test_gpu_full_configs.py, with the oracle on all host threads.)"""
    check_case(dims, BW, count, "normal", 52, FUSED)
    assert binding.last_kernel_name() == "bw_tree<V=2>"
    check_case(dims, BW, count, "int32", 53, FUSED, in_place=False)
    check_scattered(dims, BW, count, "normal", 54, FUSED)


@pytest.mark.parametrize("dims", [(4, 4), (7, 3), (8, 8), (2, 3, 4)])
def test_sharded_window(dims):
    """The buffers hold a window of a longer vector: slice and block bounds follow the global index."""
    gcount = 50021
    for (lo, hi) in ((0, 25008), (25008, gcount), (12344, 12344 + 4096), (16000, 17000)):
        check_case(dims, BW, hi - lo, "int32", 47, AUTO, shard=(gcount, lo))
        check_case(dims, BW, hi - lo, "normal", 48, STEP, in_place=False, shard=(gcount, lo))


def test_launch_counts():
    plan = binding.Plan((4, 4), BW)
    x = torch.zeros((16, 64), dtype=torch.int32, device=DEV)
    ptrs = [x[r].data_ptr() for r in range(16)]
    st = torch.cuda.current_stream().cuda_stream
    before = binding.launch_count()
    plan.allreduce_ex(ptrs, None, 64, binding.INT32, kernel=AUTO, stream=st)
    torch.cuda.synchronize()
    assert binding.last_kernel_name() == "bw_tree<V=1>" and binding.launch_count() - before == 1
    before = binding.launch_count()
    plan.allreduce_ex(ptrs, None, 64, binding.INT32, kernel=STEP, stream=st)
    torch.cuda.synchronize()
    # one launch per row and collective, in place (every row moves blocks in both collectives here)
    assert binding.last_kernel_name() == "step_general" and binding.launch_count() - before == plan.rows * 2
    plan.destroy()


def test_float32_error_bound_against_naive_sum():
    dims, count = (8, 8), 20011
    plan = binding.Plan(dims, BW)
    x = synth.rank_matrix("normal", 51, plan.n, count)
    buf = torch.zeros((plan.n, (count + 3) // 4 * 4), dtype=torch.float32, device=DEV)
    xd = buf[:, :count]
    xd.copy_(torch.from_numpy(x))
    binding.allreduce_tensor(plan, xd)
    torch.cuda.synchronize()
    got = xd.cpu().numpy()
    naive = oracle.naive_sum_f32(x)
    bound = 2e-6 * np.abs(x.astype(np.float64)).sum(0)
    assert (np.abs(got.astype(np.float64) - naive.astype(np.float64)[None]) <= bound[None]).all()
    assert (got == got[0][None]).all()      # every rank ends with the same bits
    plan.destroy()


def _same(a, b):
    for k in ("msgs", "bytes", "max_msgs", "max_bytes"):
        assert a[k].dtype == b[k].dtype and np.array_equal(a[k], b[k]), k


@pytest.mark.parametrize("dims", TORI)
@pytest.mark.parametrize("count", [7, 1024, 100003])
def test_link_loads(dims, count):
    got = binding.Plan(dims, BW).link_loads(count, 4)
    _same(got, oracle.link_loads(dims, oracle.VARIANT_BANDWIDTH, count, 4))


@pytest.mark.parametrize("dims", [(4, 4), (32, 32), (4, 4, 4)])
def test_cost_model(dims):
    alpha, beta = 1.5e-6, 1.0 / 100e9
    got = binding.Plan(dims, BW).cost_model(100003, 4, alpha, beta)
    want = oracle.cost_model(dims, oracle.VARIANT_BANDWIDTH, 100003, 4, alpha, beta)
    assert got.steps == want["steps"] and got.bytes_sent_per_node == want["bytes_sent_per_node"]
    assert got.tx_bytes == want["tx_bytes"]
    for name, key in [("total", "total"), ("lambda_", "lambda"), ("delta", "delta"), ("theta", "theta")]:
        assert np.isclose(getattr(got, name), want[key], rtol=1e-12, atol=0), name
