"""trv_allreduce_noalloc: the entry point for callers that may not allocate device memory (code
running under stream capture, inside a framework that owns all device memory, or with a fixed
memory budget).  Its scratch is a fixed 16 MiB array inside the library instead of a cudaMalloc'd
buffer.  The test calls it through the C ABI twice in a row and compares every output bit with
the ordinary entry point's (trv_allreduce_ex) and with the CPU oracle's, then checks that oversized
calls are refused.

Collected last on purpose (file name), so a run that stops at the first failure has already run
every other test; it passes on its own in a fresh process as well."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_17254_b200 import binding, build, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    assert torch.cuda.is_available()


def _reference(plan, x):
    n, count = x.shape          # row stride padded to 4 elements: every rank buffer 16-byte aligned
    xd = torch.zeros((n, (count + 3) // 4 * 4), dtype=torch.from_numpy(x).dtype, device=DEV)[:, :count]
    xd.copy_(torch.from_numpy(x))
    binding.allreduce_tensor(plan, xd, kernel=binding.KERNEL_AUTO)
    torch.cuda.synchronize()
    return xd.cpu().numpy()


@pytest.mark.parametrize("dims,count,dist", [((27,), 4133, "normal"), ((9,), 1024, "int32"), ((9, 9), 2500, "normal"),
                                             ((3,), 777, "normal"), ((243,), 1000, "normal")])
def test_noalloc_matches_the_ordinary_entry_point_twice_in_a_row(dims, count, dist):
    plan = binding.Plan(dims, binding.LATENCY_OPTIMAL)
    n = plan.n
    dcode = binding.INT32 if dist == "int32" else binding.FLOAT32
    pad = (count + 3) // 4 * 4
    stream = torch.cuda.current_stream().cuda_stream
    for call, seed in enumerate((101, 202)):        # the second call finds the first call's leftovers in the scratch
        x = synth.rank_matrix(dist, seed, n, count)
        want = _reference(plan, x)
        buf = torch.zeros((n, pad), dtype=torch.from_numpy(x).dtype, device=DEV)
        xd = buf[:, :count]
        xd.copy_(torch.from_numpy(x))
        plan.allreduce_noalloc([xd[r].data_ptr() for r in range(n)], count, dcode, stream)
        torch.cuda.synchronize()
        got = xd.cpu().numpy()
        assert np.array_equal(got.view(np.uint32), want.view(np.uint32)), "call %d differs" % call
        exact = oracle.allreduce(dims, binding.LATENCY_OPTIMAL, x)
        assert np.array_equal(got.view(np.uint32), exact.view(np.uint32)), "call %d differs from the oracle" % call
        assert binding.last_kernel_name() == "step_latency"


def test_noalloc_refuses_what_does_not_fit_and_what_it_does_not_serve():
    cap = binding.noalloc_max_scratch_bytes()
    assert cap == 16 * 1024 * 1024
    plan = binding.Plan((27,), binding.LATENCY_OPTIMAL)           # odd step count: two scratch buffers
    fits = cap // (2 * 27 * 4) // 64 * 64
    xd = torch.zeros((27, fits + 64), device=DEV)
    ptrs = [xd[r].data_ptr() for r in range(27)]
    before = binding.launch_count()
    with pytest.raises(binding.TrivanceError) as e:
        plan.allreduce_noalloc(ptrs, fits + 64, binding.FLOAT32)
    assert e.value.status == binding.ERR_TOO_LARGE and "capacity" in str(e.value)
    assert binding.launch_count() == before                      # nothing was launched
    plan.allreduce_noalloc(ptrs, fits, binding.FLOAT32)           # the largest size that fits runs
    torch.cuda.synchronize()
    assert binding.launch_count() == before + 3
    with pytest.raises(binding.TrivanceError) as e:
        binding.Plan((27,), binding.BANDWIDTH_OPTIMAL).allreduce_noalloc(ptrs, 64, binding.FLOAT32)
    assert e.value.status == binding.ERR_UNSUPPORTED
    with pytest.raises(binding.TrivanceError) as e:
        plan.allreduce_noalloc(ptrs[:26] + [ptrs[0] + 16], 64, binding.FLOAT32)
    assert e.value.status == binding.ERR_INVALID_ARG
