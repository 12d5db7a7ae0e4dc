"""Parity at the benchmark configurations' full sizes, in the launch configuration bench.py times.

Every element of every configuration is compared with the oracle.  For the multi-GiB cases (config 4,
config 5 at 8 and 32 MiB) the vector is walked in element-range chunks with the oracle on all host
threads; windows on slice, block and tile boundaries are checked first because they fail fastest."""
import concurrent.futures
import os

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
    # and so must the chunk-level readiness engine
    if plan.kernel_supported(binding.KERNEL_PIPELINED):
        xd.copy_(torch.from_numpy(xh))
        got3 = run_gpu(plan, xd, binding.KERNEL_PIPELINED).cpu().numpy()
        assert np.array_equal(got.view(np.uint32), got3.view(np.uint32))


def _every_element(w, x_dev, res_dev, chunk_bytes=3 << 29):
    """Compares res_dev with the oracle on EVERY element: the vector is walked in element-range chunks;
    inputs and results of a chunk come down through pinned staging buffers and the oracle runs on
    sub-windows over all host threads (columns are independent, so windows change nothing)."""
    n, E = w.n, w.count
    chunk = max(4096, min(E, chunk_bytes // (4 * n)))
    threads = os.cpu_count() or 4
    hin = torch.empty((n, chunk), dtype=x_dev.dtype).pin_memory()
    hout = torch.empty((n, chunk), dtype=x_dev.dtype).pin_memory()

    def one(job):
        xin, got, e0 = job
        compare(w.dims, w.variant, np.ascontiguousarray(xin), np.ascontiguousarray(got), E=E, e0=e0)

    with concurrent.futures.ThreadPoolExecutor(max_workers=threads) as ex:
        for c0 in range(0, E, chunk):
            c1 = min(E, c0 + chunk)
            hin[:, :c1 - c0].copy_(x_dev[:, c0:c1])
            hout[:, :c1 - c0].copy_(res_dev[:, c0:c1])
            torch.cuda.synchronize()
            a, b = hin.numpy(), hout.numpy()
            cuts = [c0 + ((c1 - c0) * i) // threads for i in range(threads + 1)]
            jobs = [(a[:, u - c0:v - c0], b[:, u - c0:v - c0], u) for u, v in zip(cuts, cuts[1:]) if v > u]
            list(ex.map(one, jobs))


@pytest.mark.parametrize("name", ["ring243_lat_8MiB", "ring243_bw_8MiB", "ring243_lat_32MiB", "ring243_bw_32MiB",
                                  "torus9x9x9_lat_32MiB", "torus9x9x9_bw_32MiB", "ring32_bw_8MiB", "ring100_bw_8MiB",
                                  "torus32x32_bw_8MiB", "torus8x64_bw_8MiB", "torus16x16x4_bw_8MiB",
                                  "torus27x27_lat_8MiB", "torus9x81_lat_8MiB", "ring729_lat_8MiB"])
def test_config_full_size_every_element(name):
    """The multi-GiB configurations, in the launch configuration bench.py times (AUTO, separate outputs):
    first the boundary-centred windows (fast to fail), then every element against the oracle, then the
    in-place call (trv_allreduce's form) bit for bit against that verified result."""
    w = synth.CONFIGS[name]
    plan = binding.Plan(w.dims, w.variant)
    wins = _windows(w)
    xd, keep = upload_matrix(w.dist, w.seed, w.n, w.count, wins)
    res = run_gpu(plan, xd, in_place=False)       # AUTO, separate output: what bench.py launches
    for (w0, w1), xh in zip(wins, keep):
        compare(w.dims, w.variant, xh, res[:, w0:w1].cpu().numpy(), E=w.count, e0=w0)
    _every_element(w, xd, res)
    if w.variant == BW:                           # every rank ends with the same bits
        ref = res[0].view(torch.int32)
        for r in range(1, w.n):
            assert torch.equal(res[r].view(torch.int32), ref)
    res2 = run_gpu(plan, xd)                      # in place, AUTO
    assert res2.data_ptr() == xd.data_ptr()
    for r0 in range(0, w.n, 27):                  # in slabs: torch.equal on 22 GiB at once would need a mask as large
        assert torch.equal(res2[r0:r0 + 27].view(torch.int32), res[r0:r0 + 27].view(torch.int32))
    del xd, res, res2
    torch.cuda.empty_cache()
