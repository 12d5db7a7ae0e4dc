"""Randomised GPU parity: shapes, sizes, kernel families, dtypes, in/out of place and element-range
shards drawn from a seeded generator; every case bit-exact against the oracle."""
import numpy as np
import pytest
import torch

from paper_2602_17254_b200 import binding, build

from gpu_util import check_case

pytestmark = pytest.mark.gpu

LAT, BW = binding.LATENCY_OPTIMAL, binding.BANDWIDTH_OPTIMAL
AUTO, STEP, FUSED, PIPE = binding.KERNEL_AUTO, binding.KERNEL_STEP, binding.KERNEL_FUSED, binding.KERNEL_PIPELINED
REGULAR = [(3,), (9,), (27,), (81,), (243,), (3, 3), (9, 3), (3, 9), (9, 9), (27, 3), (3, 27), (3, 3, 3), (3, 3, 9), (9, 3, 3),
           (9, 9, 3), (3, 3, 3, 3), (27, 9), (9, 9, 9)]


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    assert torch.cuda.is_available()
    binding.lib()


def _cases(seed, k):
    rng = np.random.default_rng(seed)
    out = []
    for i in range(k):
        if rng.random() < 0.3:          # a ring of any size, bandwidth form
            dims, variant = (int(rng.integers(2, 300)),), BW
            kernel = [AUTO, STEP, FUSED][int(rng.integers(0, 3))]
        else:
            dims = REGULAR[int(rng.integers(0, len(REGULAR)))]
            variant = LAT if rng.random() < 0.5 else BW
            kernel = [AUTO, STEP, FUSED, PIPE][int(rng.integers(0, 4))]
            if kernel == PIPE and (variant == BW or dims == (3,)):
                kernel = AUTO
            if kernel == FUSED and variant == LAT and dims in ((27, 9),):
                pass                    # served by the line-group kernel
        n = int(np.prod(dims))
        big = rng.random() < 0.2 and n <= 81
        count = int(rng.integers(1, 200000 if big else (6000 if n <= 243 else 1500)))
        in_place = bool(rng.random() < 0.5)
        shard = None
        if rng.random() < 0.3:
            gcount = count + int(rng.integers(1, 5000))
            shard = (gcount, int(rng.integers(0, gcount - count + 1)))
        dist = ["int32", "normal", "uniform"][int(rng.integers(0, 3))]
        out.append((dims, variant, kernel, count, in_place, shard, dist, 1000 + i))
    return out


@pytest.mark.parametrize("case", _cases(20260217, 60), ids=lambda c: "%s-%d-k%d-%d%s%s" % (
    "x".join(map(str, c[0])), c[1], c[2], c[3], "-ip" if c[4] else "-oop", "-shard" if c[5] else ""))
def test_random_case(case):
    dims, variant, kernel, count, in_place, shard, dist, seed = case
    plan = binding.Plan(dims, variant)
    if not plan.kernel_supported(kernel):
        kernel = AUTO
    if kernel == PIPE and in_place and plan.rows == 1:
        kernel = AUTO
    plan.destroy()
    check_case(dims, variant, count, dist, seed, kernel, in_place=in_place, shard=shard)


def _wide_cases(seed, k):
    """The persistent 64-column kernels (729-rank shapes, long vectors): sizes just above their thresholds, ragged, sharded."""
    rng = np.random.default_rng(seed)
    shapes = [((27, 27), "lat_t27x27_wide"), ((9, 81), "lat_t9x81_wide"), ((81, 9), "lat_t81x9_wide"), ((729,), "lat_ring729_wide")]
    out = []
    for i in range(k):
        dims, name = shapes[i % len(shapes)]
        count = int(rng.integers(66000, 140000))
        shard = None
        if rng.random() < 0.5:
            gcount = count + int(rng.integers(1, 300000))
            shard = (gcount, int(rng.integers(0, gcount - count + 1)))
        out.append((dims, name, count, bool(rng.random() < 0.5), shard, ["int32", "normal", "uniform"][int(rng.integers(0, 3))], 2000 + i))
    return out


@pytest.mark.parametrize("case", _wide_cases(20260218, 12), ids=lambda c: "%s-%d%s%s" % (
    "x".join(map(str, c[0])), c[2], "-ip" if c[3] else "-oop", "-shard" if c[4] else ""))
def test_random_case_on_the_wide_kernels(case):
    dims, name, count, in_place, shard, dist, seed = case
    check_case(dims, LAT, count, dist, seed, FUSED, in_place=in_place, shard=shard)
    if shard is None or min(shard[0] - shard[1], count) >= 66000:
        assert binding.last_kernel_name() == name
