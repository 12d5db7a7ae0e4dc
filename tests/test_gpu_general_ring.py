"""GPU parity for rings whose size is no power of three (Sec. 4.4): the STEP kernels of that
schedule and its link-load tally through the C ABI vs the CPU oracle, bit-exact."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_17254_b200 import binding, build, synth

from gpu_util import DEV, check_case, check_scattered, compare, torch_dtype

pytestmark = pytest.mark.gpu

BW = binding.BANDWIDTH_OPTIMAL
AUTO, STEP, FUSED = binding.KERNEL_AUTO, binding.KERNEL_STEP, binding.KERNEL_FUSED
SIZES = [2, 4, 5, 6, 7, 8, 10, 13, 26, 28, 32, 33, 80, 82, 100, 244, 257]


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    assert torch.cuda.is_available()
    binding.lib()


@pytest.mark.parametrize("n", SIZES)
def test_matches_oracle(n):
    count = 4099 if n <= 100 else 1531      # several blocks of ragged length, unaligned block starts
    check_case((n,), BW, count, "normal", 21, FUSED)
    check_case((n,), BW, count, "int32", 22, STEP, in_place=False)
    check_case((n,), BW, count, "int32", 22, FUSED, in_place=False)
    check_case((n,), BW, count, "normal", 21, STEP)
    check_scattered((n,), BW, count, "uniform", 23, AUTO)
    check_scattered((n,), BW, count, "uniform", 23, STEP)


@pytest.mark.parametrize("n", [7, 32, 100])
@pytest.mark.parametrize("count", [1, 2, 5, 31, 99, 100, 101])
def test_short_vectors(n, count):
    """Fewer elements than ranks: most blocks are empty."""
    check_case((n,), BW, count, "int32", 24, AUTO)
    check_case((n,), BW, count, "normal", 25, AUTO, in_place=False)


@pytest.mark.parametrize("n", [10, 53])
def test_larger_vector_spans_many_ctas(n):
    check_case((n,), BW, 700001, "normal", 26, STEP)
    check_case((n,), BW, 700001, "normal", 26, FUSED)


@pytest.mark.parametrize("n,count", [(4, 1 << 20), (10, (1 << 20) + 6), (100, (1 << 20) + 3)])
def test_two_columns_per_thread_path(n, count):
    """Long vectors take the kernel with two columns per thread; block boundaries fall inside some pairs."""
    check_case((n,), BW, count, "normal", 32, FUSED)
    assert binding.last_kernel_name() == "bw_tree<V=2>"
    check_case((n,), BW, count, "int32", 33, FUSED, in_place=False)
    check_scattered((n,), BW, count, "normal", 34, FUSED)


@pytest.mark.parametrize("n", [7, 32, 244])
def test_sharded_window(n):
    """The buffers hold a window of a longer vector: block bounds follow the global index."""
    gcount = 50021
    for (lo, hi) in ((0, 25008), (25008, gcount), (12344, 12344 + 4096)):
        check_case((n,), BW, hi - lo, "int32", 27, AUTO, shard=(gcount, lo))
        check_case((n,), BW, hi - lo, "normal", 28, AUTO, in_place=False, shard=(gcount, lo))


def test_largest_ring():
    n, count = 1000, 3001
    check_case((n,), BW, count, "int32", 29, AUTO)


def test_empty_and_kernel_choice():
    plan = binding.Plan((10,), BW)
    assert plan.kernel_supported(STEP) and plan.kernel_supported(FUSED)
    x = torch.zeros((10, 64), dtype=torch.int32, device=DEV)
    ptrs = [x[r].data_ptr() for r in range(10)]
    before = binding.launch_count()
    plan.allreduce_ex(ptrs, None, 0, binding.INT32, kernel=AUTO, stream=torch.cuda.current_stream().cuda_stream)
    assert binding.launch_count() == before
    plan.allreduce_ex(ptrs, None, 64, binding.INT32, kernel=AUTO, stream=torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert binding.last_kernel_name() == "bw_tree<V=1>" and binding.launch_count() - before == 1
    before = binding.launch_count()
    plan.allreduce_ex(ptrs, None, 64, binding.INT32, kernel=STEP, stream=torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert binding.last_kernel_name() == "step_general"
    # one launch per row of the schedule, in place
    assert binding.launch_count() - before == plan.rows
    plan.destroy()


def test_float32_error_bound_against_naive_sum():
    n, count = 100, 20011
    plan = binding.Plan((n,), BW)
    x = synth.rank_matrix("normal", 31, n, count)
    buf = torch.zeros((n, (count + 3) // 4 * 4), dtype=torch.float32, device=DEV)
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


@pytest.mark.parametrize("n", SIZES + [1000])
@pytest.mark.parametrize("count", [7, 1024, 100003])
def test_link_loads(n, count):
    got = binding.Plan((n,), BW).link_loads(count, 4)
    _same(got, oracle.link_loads((n,), oracle.VARIANT_BANDWIDTH, count, 4))


@pytest.mark.parametrize("n", [7, 32, 100])
def test_cost_model(n):
    alpha, beta = 1.5e-6, 1.0 / 100e9
    got = binding.Plan((n,), BW).cost_model(100003, 4, alpha, beta)
    want = oracle.cost_model((n,), oracle.VARIANT_BANDWIDTH, 100003, 4, alpha, beta)
    assert got.steps == want["steps"] and got.bytes_sent_per_node == want["bytes_sent_per_node"]
    assert got.tx_bytes == want["tx_bytes"]
    for name, key in [("total", "total"), ("lambda_", "lambda"), ("delta", "delta"), ("theta", "theta")]:
        assert np.isclose(getattr(got, name), want[key], rtol=1e-12, atol=0), name
