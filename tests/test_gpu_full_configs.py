"""Parity at the benchmark configurations' full sizes, in the launch configuration bench.py times.

Where the oracle can afford it (configs 1-3 and the small points of config 5) every element is
compared; for the multi-GiB cases (config 4, config 5 at 8 and 32 MiB) the oracle computes element
windows placed on slice boundaries, block boundaries, tile boundaries and interiors, plus
properties that hold at any size (bandwidth form: all n rows identical)."""
import numpy as np
import pytest
import torch

from paper_2602_17254_b200 import binding, build, synth

from gpu_util import compare, run_gpu, upload_matrix

pytestmark = pytest.mark.gpu
LAT, BW = binding.LATENCY_OPTIMAL, binding.BANDWIDTH_OPTIMAL


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    assert torch.cuda.is_available()


def _windows(w, k=6, width=384):
    """Element windows around slice and block boundaries, at both ends and in the interior."""
    D, n, E = len(w.dims), w.n, w.count
    wins = [(0, width), (E - width, E), (E // 2 - 100, E // 2 - 100 + width)]
    for c in range(1, D):
        b = (c * E) // D
        wins.append((b - width // 2, b + width // 2))
    if w.variant == BW:
        plan = binding.Plan(w.dims, w.variant)
        rng = np.random.default_rng(w.seed)
        for c in range(D):
            bb = plan.block_bounds(E, c)
            for j in rng.integers(1, n, k):
                wins.append((int(bb[j]) - width // 2, int(bb[j]) + width // 2))
    return [(max(0, a), min(E, b)) for a, b in wins]


@pytest.mark.parametrize("name", ["ring9_lat_int32", "ring27_lat_2MiB", "ring81_bw_8MiB", "ring243_lat_32KiB",
                                  "ring243_bw_32KiB", "ring243_lat_512KiB", "ring243_bw_512KiB"])
def test_config_every_element(name):
    w = synth.CONFIGS[name]
    plan = binding.Plan(w.dims, w.variant)
    xd, (xh,) = upload_matrix(w.dist, w.seed, w.n, w.count, [(0, w.count)])
    got = run_gpu(plan, xd).cpu().numpy()
    compare(w.dims, w.variant, xh, got)
    # the step-literal family must agree bit for bit at full size too
    xd.copy_(torch.from_numpy(xh))
    got2 = run_gpu(plan, xd, binding.KERNEL_STEP).cpu().numpy()
    assert np.array_equal(got.view(np.uint32), got2.view(np.uint32))
    # and so must the chunk-level readiness engine (latency form only)
    if w.variant == LAT and plan.kernel_supported(binding.KERNEL_PIPELINED):
        xd.copy_(torch.from_numpy(xh))
        got3 = run_gpu(plan, xd, binding.KERNEL_PIPELINED).cpu().numpy()
        assert np.array_equal(got.view(np.uint32), got3.view(np.uint32))


@pytest.mark.parametrize("name", ["ring243_lat_8MiB", "ring243_bw_8MiB", "ring243_lat_32MiB", "ring243_bw_32MiB",
                                  "torus9x9x9_lat_32MiB", "torus9x9x9_bw_32MiB", "ring32_bw_8MiB", "ring100_bw_8MiB"])
def test_config_sampled_windows(name):
    w = synth.CONFIGS[name]
    plan = binding.Plan(w.dims, w.variant)
    wins = _windows(w)
    xd, keep = upload_matrix(w.dist, w.seed, w.n, w.count, wins)
    res = run_gpu(plan, xd, in_place=False)       # AUTO, separate output: what bench.py launches
    for (w0, w1), xh in zip(wins[:2], keep[:2]):
        compare(w.dims, w.variant, xh, res[:, w0:w1].cpu().numpy(), E=w.count, e0=w0)
    del res
    res = run_gpu(plan, xd)                       # in place, AUTO: trv_allreduce's form
    for (w0, w1), xh in zip(wins, keep):
        compare(w.dims, w.variant, xh, res[:, w0:w1].cpu().numpy(), E=w.count, e0=w0)
    if w.variant == BW:                           # holds at any size: every rank ends with the same bits
        ref = res[0].view(torch.int32)
        for r in range(1, w.n, 7):
            assert torch.equal(res[r].view(torch.int32), ref)
    del xd, res
    torch.cuda.empty_cache()
