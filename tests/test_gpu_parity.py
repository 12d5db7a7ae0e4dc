"""GPU parity: the CUDA path through the C ABI vs the CPU oracle, element by element, bit-exact.

Small cases: sizes the oracle finishes in seconds that still span several tiles and ragged tails,
every kernel family, both dtypes, in place and out of place, sharded windows, degenerate sizes.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_17254_b200 import binding, build, synth

from gpu_util import DEV, check_case, check_scattered, compare, run_gpu, torch_dtype, upload_matrix

pytestmark = pytest.mark.gpu

LAT, BW = binding.LATENCY_OPTIMAL, binding.BANDWIDTH_OPTIMAL
AUTO, STEP, FUSED = binding.KERNEL_AUTO, binding.KERNEL_STEP, binding.KERNEL_FUSED


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    assert torch.cuda.is_available()
    binding.lib()


FUSED_LAT = [(3,), (9,), (27,), (81,), (243,), (729,), (3, 3), (9, 9), (3, 3, 3), (3, 3, 3, 3), (9, 9, 9),
             (3, 9), (27, 3), (3, 3, 9), (27, 27), (9, 81), (81, 9), (3, 81), (9, 3, 27), (3, 27, 9)]   # the last ones: line-group kernel
ANY = FUSED_LAT + [(243, 3)]


@pytest.mark.parametrize("dims", ANY)
@pytest.mark.parametrize("variant", [LAT, BW])
def test_step_family_matches_oracle(dims, variant):
    n = int(np.prod(dims))
    count = 1531 if n <= 243 else 517
    check_case(dims, variant, count, "normal", 11, STEP)
    check_case(dims, variant, count, "int32", 12, STEP, in_place=False)
    check_scattered(dims, variant, count, "normal", 13, STEP)


@pytest.mark.parametrize("dims", FUSED_LAT)
def test_fused_latency_matches_oracle(dims):
    n = int(np.prod(dims))
    count = 4133 if n <= 243 else 1029          # several tiles of every kernel + ragged tail
    check_case(dims, LAT, count, "normal", 21, FUSED)
    check_case(dims, LAT, count, "int32", 22, FUSED, in_place=False)
    check_scattered(dims, LAT, count, "normal", 23, FUSED)
    check_scattered(dims, LAT, count, "int32", 24, FUSED)


@pytest.mark.parametrize("dims", ANY)
def test_fused_bandwidth_matches_oracle(dims):
    n = int(np.prod(dims))
    D = len(dims)
    small = 1531 if n <= 243 else 517                     # one column per thread (short blocks)
    check_case(dims, BW, small, "normal", 31, FUSED)
    check_case(dims, BW, small, "int32", 32, FUSED, in_place=False)
    check_scattered(dims, BW, small, "normal", 36, FUSED)
    if n <= 27:                                           # two columns per thread (long blocks, >= 2^20 elements)
        wide = (1 << 20) + 300 * n * D + 7
        check_case(dims, BW, wide, "normal", 33, FUSED)
        check_case(dims, BW, wide, "int32", 34, FUSED, in_place=False)
        check_scattered(dims, BW, wide, "int32", 37, FUSED)


def test_fused_latency_9x9x9_many_tiles_per_cta():
    """The 9x9x9 kernel is persistent (one CTA per SM looping over tiles, two tiles in flight): sizes
    where a CTA gets 1, 2, 3 and about 9 tiles, with ragged slice edges, and scattered buffers."""
    for count in (148 * 32 // 3 * 3 + 96, 9000, 14211, 40003):
        check_case((9, 9, 9), LAT, count, "normal", count, FUSED)
    check_case((9, 9, 9), LAT, 20011, "int32", 5, FUSED, in_place=False)
    check_scattered((9, 9, 9), LAT, 20011, "normal", 6, FUSED)


def test_fused_latency_9x9x9_tiles_of_64_columns():
    """Long vectors on the 9x9x9 torus take the persistent kernel on 64-column tiles (one CTA per SM, the next tile
    loading while group 3 of the current one runs from registers): ragged slice edges that share a tile between two
    slices, many tiles per CTA with both mbarrier parities, both dtypes, in place and not.  Tiles are handed out from a
    per-stream counter; a second stream gets its own; a call captured into a CUDA graph takes the fixed assignment
    instead -- all must give the same bits."""
    x, want = check_case((9, 9, 9), LAT, 800003, "normal", 41, FUSED)
    assert binding.last_kernel_name() == "lat_t999_wide"
    plan = binding.Plan((9, 9, 9), LAT)
    n, count = x.shape
    pad = (count + 3) // 4 * 4
    xin = torch.zeros((n, pad), dtype=torch.float32, device=DEV)
    xin[:, :count].copy_(torch.from_numpy(x))
    xout = torch.zeros_like(xin)
    ip = binding.ptr_array([xin[r].data_ptr() for r in range(n)])
    op = binding.ptr_array([xout[r].data_ptr() for r in range(n)])
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):       # twice on a stream of its own: the counter is back at zero after the first call
        for _ in range(2):
            xout.zero_()
            plan.allreduce_ex(ip, op, count, binding.FLOAT32, kernel=FUSED, stream=side.cuda_stream)
    side.synchronize()
    assert binding.last_kernel_name() == "lat_t999_wide"
    assert np.array_equal(xout[:, :count].cpu().numpy().view(np.uint32), want.view(np.uint32))
    g = torch.cuda.CUDAGraph()
    torch.cuda.synchronize()
    with torch.cuda.graph(g):
        plan.allreduce_ex(ip, op, count, binding.FLOAT32, kernel=FUSED, stream=torch.cuda.current_stream().cuda_stream)
    xout.zero_()
    g.replay()
    torch.cuda.synchronize()
    assert np.array_equal(xout[:, :count].cpu().numpy().view(np.uint32), want.view(np.uint32))
    plan.destroy()
    del xin, xout
    check_case((9, 9, 9), LAT, 786754, "int32", 42, FUSED, in_place=False)
    assert binding.last_kernel_name() == "lat_t999_wide"
    assert binding.tma_giveups() == 0


def test_fused_latency_27x27_tiles_of_64_columns():
    """Long vectors on the 27 x 27 torus take the same persistent 64-column kernel with the 27 x 27 groups: both slices
    (dimension orders), ragged slice edges, both dtypes, in place and not."""
    check_case((27, 27), LAT, 70001, "normal", 51, FUSED)
    assert binding.last_kernel_name() == "lat_t27x27_wide"
    check_case((27, 27), LAT, 300034, "int32", 52, FUSED, in_place=False)
    assert binding.last_kernel_name() == "lat_t27x27_wide"
    # an element-range shard: the buffers hold elements [64999, 135000) of vectors of 200003 (the slice boundary at 100001
    # falls inside the window, at an odd column)
    check_case((27, 27), LAT, 70001, "normal", 53, FUSED, shard=(200003, 64999))
    assert binding.last_kernel_name() == "lat_t27x27_wide"
    check_case((9, 9, 9), LAT, 800003, "int32", 54, FUSED, in_place=False, shard=(2400011, 790001))
    assert binding.last_kernel_name() == "lat_t999_wide"
    assert binding.tma_giveups() == 0


def test_fused_latency_9x81_tiles_of_64_columns():
    """9 x 81 and 81 x 9: the persistent 64-column kernel with steps along the side of 81 streamed as ring stencils across the
    planes; both slices (A1 B1 A3 B3 B9 B27 and B1 A1 B3 A3 B9 B27), ragged edges, both dtypes, in place and not."""
    check_case((9, 81), LAT, 70001, "normal", 61, FUSED)
    assert binding.last_kernel_name() == "lat_t9x81_wide"
    check_case((9, 81), LAT, 300034, "int32", 62, FUSED, in_place=False)
    assert binding.last_kernel_name() == "lat_t9x81_wide"
    check_case((81, 9), LAT, 70001, "int32", 63, FUSED)
    assert binding.last_kernel_name() == "lat_t81x9_wide"
    check_case((81, 9), LAT, 200002, "normal", 64, FUSED, in_place=False)
    assert binding.last_kernel_name() == "lat_t81x9_wide"
    assert binding.tma_giveups() == 0


def test_fused_latency_ring729_tiles_of_64_columns():
    """Ring of 729: the persistent 64-column kernel with the steps 1 and 3 as open-segment stencils with halos (one
    segment of 81 ranks per warp) and 9, 27 as ring stencils; ragged edges, both dtypes, in place and not."""
    check_case((729,), LAT, 70001, "normal", 71, FUSED)
    assert binding.last_kernel_name() == "lat_ring729_wide"
    check_case((729,), LAT, 150034, "int32", 72, FUSED, in_place=False)
    assert binding.last_kernel_name() == "lat_ring729_wide"
    assert binding.tma_giveups() == 0


def test_fused_bandwidth_wide_path_on_729_ranks_sampled():
    """9x9x9 with blocks of >= 256 elements: the oracle checks windows around slice and block
    boundaries and in block interiors."""
    dims, count = (9, 9, 9), (1 << 20) + 5
    plan = binding.Plan(dims, BW)
    wins = [(0, 700), (count // 3 - 400, count // 3 + 400), (2 * count // 3 - 333, 2 * count // 3 + 777),
            (count - 900, count), (123456, 124000)]
    xd, keep = upload_matrix("uniform", 35, 729, count, wins)
    res = run_gpu(plan, xd, FUSED, in_place=False)
    assert binding.last_kernel_name() == "bw_fused<V=2>"
    for (w0, w1), xh in zip(wins, keep):
        compare(dims, BW, xh, res[:, w0:w1].cpu().numpy(), E=count, e0=w0)


@pytest.mark.parametrize("dims,variant", [((27,), LAT), ((9, 9), LAT), ((9, 9, 9), LAT), ((243,), LAT), ((81,), BW), ((9, 9, 9), BW)])
@pytest.mark.parametrize("count", [1, 2, 3, 4, 5, 31, 32, 33, 127])
def test_degenerate_sizes(dims, variant, count):
    """Fewer elements than ranks / than dimensions: empty slices and empty blocks."""
    for kernel in (STEP, FUSED):
        check_case(dims, variant, count, "int32", count, kernel)
        check_case(dims, variant, count, "normal", count, kernel, in_place=False)


@pytest.mark.parametrize("dims,variant", [((27,), LAT), ((9, 9, 9), LAT), ((243,), LAT), ((9, 9), BW), ((9, 9, 9), BW), ((81,), BW)])
def test_sharded_windows_equal_the_unsharded_run(dims, variant):
    """Element-range shards carry the global element index: concatenating the shards' results gives
    the unsharded result (slice and block membership must not move)."""
    n = int(np.prod(dims))
    total = 3001
    for kernel in (STEP, FUSED):
        pieces = []
        for (go, cnt) in [(0, 1000), (1000, 996), (1996, 1005)]:
            x = synth.rank_matrix("normal", 41, n, total)[:, go:go + cnt]
            plan = binding.Plan(dims, variant)
            pad = (cnt + 3) // 4 * 4
            buf = torch.zeros((n, pad), dtype=torch.float32, device=DEV)
            xd = buf[:, :cnt]
            xd.copy_(torch.from_numpy(np.ascontiguousarray(x)))
            got = run_gpu(plan, xd, kernel, True, total, go).cpu().numpy()
            compare(dims, variant, np.ascontiguousarray(x), got, E=total, e0=go)
            pieces.append(got)
        full = oracle.allreduce(dims, variant, synth.rank_matrix("normal", 41, n, total))
        assert np.array_equal(np.concatenate(pieces, axis=1), full)


def test_default_entry_point_and_plan_owned_scratch():
    """trv_allreduce (in place, AUTO) incl. the case where the plan has to allocate scratch itself."""
    for dims, variant in [((27,), LAT), ((243, 3), LAT), ((81,), BW)]:
        plan = binding.Plan(dims, variant)
        n = plan.n
        x = synth.rank_matrix("normal", 51, n, 2048)
        xd = torch.from_numpy(x).to(DEV)
        for _ in range(2):      # second call reuses the plan's scratch
            xd.copy_(torch.from_numpy(x))
            plan.allreduce([xd[r].data_ptr() for r in range(n)], 2048, binding.FLOAT32,
                           torch.cuda.current_stream().cuda_stream)
            torch.cuda.synchronize()
            compare(dims, variant, x, xd.cpu().numpy())
        plan.destroy()


def test_separate_rank_allocations_and_side_stream():
    """Rank buffers need not be rows of one tensor; work is queued on the caller's stream."""
    dims = (9, 9)
    plan = binding.Plan(dims, LAT)
    x = synth.rank_matrix("normal", 61, 81, 1000)
    bufs = [torch.from_numpy(x[r]).to(DEV) for r in range(81)]
    s = torch.cuda.Stream()
    torch.cuda.synchronize()
    with torch.cuda.stream(s):
        plan.allreduce_ex([b.data_ptr() for b in bufs], None, 1000, binding.FLOAT32, stream=s.cuda_stream)
    s.synchronize()
    compare(dims, LAT, x, np.stack([b.cpu().numpy() for b in bufs]))


def test_host_buffer_entry_point():
    dims, count = (27,), 5000
    plan = binding.Plan(dims, LAT)
    x = synth.rank_matrix("normal", 71, 27, count)
    hin = torch.from_numpy(x.copy()).pin_memory()
    hout = torch.empty_like(hin).pin_memory()
    ws = torch.empty(plan.host_workspace_bytes(count), dtype=torch.uint8, device=DEV)
    plan.allreduce_host([hin[r].data_ptr() for r in range(27)], [hout[r].data_ptr() for r in range(27)], count,
                        binding.FLOAT32, ws.data_ptr(), ws.numel(), torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    compare(dims, LAT, x, hout.numpy())
    with pytest.raises(binding.TrivanceError) as e:
        plan.allreduce_host([hin[r].data_ptr() for r in range(27)], None, count, binding.FLOAT32, ws.data_ptr(), 1024)
    assert e.value.status == binding.ERR_SCRATCH


@pytest.mark.parametrize("dims,variant,count,dist", [
    ((27,), LAT, 200003, "normal"),         # 8 windows of 25024 elements + a ragged last one
    ((9, 9), BW, 150001, "int32"),          # block and slice bounds must follow the global element index
    ((9, 9, 9), LAT, 50021, "normal"),      # the TMA-fed kernel on windows of a longer vector
    ((100,), BW, 140000, "normal"),         # ring of another size
    ((243, 3), LAT, 70001, "normal"),       # STEP family: every window slot carries its own scratch
])
def test_host_buffer_entry_point_runs_windows_of_the_vector(dims, variant, count, dist):
    """trv_allreduce_host pipelines element-range windows; the result is the oracle's for the whole vector."""
    plan = binding.Plan(dims, variant)
    n = plan.n
    x = synth.rank_matrix(dist, 72, n, count)
    hin = torch.from_numpy(x.copy()).pin_memory()
    hout = torch.empty_like(hin).pin_memory()
    need = plan.host_workspace_bytes(count)
    assert need < n * count * 4 or count < 8 * 16384        # a few windows, not the whole matrix
    ws = torch.empty(need, dtype=torch.uint8, device=DEV)
    dcode = binding.INT32 if dist == "int32" else binding.FLOAT32
    stream = torch.cuda.current_stream().cuda_stream
    before = binding.launch_count()
    plan.allreduce_host([hin[r].data_ptr() for r in range(n)], [hout[r].data_ptr() for r in range(n)], count, dcode,
                        ws.data_ptr(), ws.numel(), stream)
    torch.cuda.synchronize()
    assert binding.launch_count() - before >= min(8, -(-count // 16384))      # one AllReduce per window
    compare(dims, variant, x, hout.numpy())
    assert np.array_equal(hin.numpy(), x)
    # in place on the host, rows NOT equally spaced (one copy per row), and a workspace a fifth of the preferred size
    rows = [torch.empty(count + 64 * (r % 3), dtype=hin.dtype).pin_memory() for r in range(n)]
    for r in range(n):
        rows[r][:count].copy_(torch.from_numpy(x[r]))
    small = torch.empty(need // 5 // 256 * 256, dtype=torch.uint8, device=DEV)
    plan.allreduce_host([t.data_ptr() for t in rows], None, count, dcode, small.data_ptr(), small.numel(), stream)
    torch.cuda.synchronize()
    got = np.stack([t[:count].numpy() for t in rows])
    assert np.array_equal(got.view(np.uint32), hout.numpy().view(np.uint32))


def test_plan_owned_scratch_is_bound_to_its_device_and_can_be_reserved():
    """trv_allreduce on a shape that needs the STEP family's scratch: reserve first, then the call launches only."""
    dims, count = (243, 3), 777
    plan = binding.Plan(dims, LAT)
    assert plan.scratch_bytes(count) > 0
    plan.reserve_scratch(4 * count)
    x = synth.rank_matrix("normal", 73, plan.n, count)
    xd = torch.zeros((plan.n, 780), device=DEV)[:, :count]
    xd.copy_(torch.from_numpy(x))
    for _ in range(2):
        xd.copy_(torch.from_numpy(x))
        plan.allreduce([xd[r].data_ptr() for r in range(plan.n)], count, binding.FLOAT32, torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        compare(dims, LAT, x, xd.cpu().numpy())
    plan.destroy()
    fused = binding.Plan((27,), LAT)        # nothing to reserve for a fused shape
    fused.reserve_scratch(10 ** 6)


def test_plan_scratch_grows_safely_under_concurrent_host_threads():
    """Two host threads call trv_allreduce on ONE plan whose shape needs the plan-owned scratch, with growing vector
    lengths, on one stream (so the calls do not overlap on the device, as the header asks).  The grow path is
    serialised inside the plan: no double free, no dangling scratch, every result equals the oracle's."""
    import threading
    dims = (243, 3)
    plan = binding.Plan(dims, LAT)
    stream = torch.cuda.current_stream().cuda_stream
    counts = [64, 700, 260, 1500, 128, 3000]
    xs = {c: synth.rank_matrix("int32", 90 + c, plan.n, c) for c in counts}
    bufs = {(t, c): torch.from_numpy(xs[c]).to(DEV) for t in range(2) for c in counts}
    errors = []

    def worker(t):
        try:
            for c in (counts if t == 0 else counts[::-1]):
                xd = bufs[(t, c)]
                plan.allreduce([xd[r].data_ptr() for r in range(plan.n)], c, binding.INT32, stream)
        except Exception as e:      # pragma: no cover
            errors.append(e)

    threads = [threading.Thread(target=worker, args=(t,)) for t in range(2)]
    for th in threads:
        th.start()
    for th in threads:
        th.join()
    torch.cuda.synchronize()
    assert not errors
    for (t, c), xd in bufs.items():
        compare(dims, LAT, xs[c], xd.cpu().numpy())
    plan.destroy()


def test_wide_kernels_on_several_streams_and_threads_at_once():
    """The persistent 64-column kernels draw their tiles from a counter that belongs to the (device, stream) pair.  Three
    host threads, each with a stream of its own, run ONE plan's AllReduce several times at once (the kernels of
    different streams overlap on the device); one more thread shares the first thread's stream (its calls are serialised
    with that thread's).  Every output equals the oracle's bits."""
    import threading
    dims, count, reps = (27, 27), 70001, 4
    plan = binding.Plan(dims, LAT)
    n = plan.n
    x = synth.rank_matrix("normal", 77, n, count)
    want = oracle.allreduce(dims, LAT, x)
    pad = (count + 3) // 4 * 4
    xin = torch.zeros((n, pad), dtype=torch.float32, device=DEV)
    xin[:, :count].copy_(torch.from_numpy(x))
    ip = binding.ptr_array([xin[r].data_ptr() for r in range(n)])
    streams = [torch.cuda.Stream() for _ in range(3)]
    use = [0, 1, 2, 0]
    outs = [torch.zeros((reps, n, pad), dtype=torch.float32, device=DEV) for _ in use]
    torch.cuda.synchronize()
    errors, names = [], []

    def worker(t):
        try:
            st = streams[use[t]].cuda_stream
            for k in range(reps):
                op = binding.ptr_array([outs[t][k, r].data_ptr() for r in range(n)])
                plan.allreduce_ex(ip, op, count, binding.FLOAT32, kernel=FUSED, stream=st)
            names.append(binding.last_kernel_name())
        except Exception as e:      # pragma: no cover
            errors.append(e)

    threads = [threading.Thread(target=worker, args=(t,)) for t in range(len(use))]
    for th in threads:
        th.start()
    for th in threads:
        th.join()
    torch.cuda.synchronize()
    assert not errors and names == ["lat_t27x27_wide"] * len(use)
    for o in outs:
        got = o[:, :, :count].cpu().numpy()
        for k in range(reps):
            assert np.array_equal(got[k].view(np.uint32), want.view(np.uint32))
    assert binding.tma_giveups() == 0
    plan.destroy()


def test_fp32_tolerance_against_naive_and_exact_sums():
    """|err| <= 2e-6 * sum|x| against the naive sequential binary32 sum (and the fp64 sum)."""
    for dims, variant, dist in [((27,), LAT, "normal"), ((81,), BW, "normal"), ((9, 9, 9), LAT, "uniform"),
                                ((9, 9, 9), BW, "uniform"), ((243,), LAT, "normal"), ((243,), BW, "normal")]:
        plan = binding.Plan(dims, variant)
        x = synth.rank_matrix(dist, 81, plan.n, 2048)
        got = run_gpu(plan, torch.from_numpy(x).to(DEV)).cpu().numpy().astype(np.float64)
        sabs = np.abs(x.astype(np.float64)).sum(0)
        assert np.all(np.abs(got - oracle.naive_sum_f32(x).astype(np.float64)) <= 2e-6 * sabs)
        assert np.all(np.abs(got - x.astype(np.float64).sum(0)) <= 2e-6 * sabs)


def test_latency_rows_differ_and_bandwidth_rows_agree():
    x = synth.rank_matrix("normal", 91, 27, 4096)
    lat = run_gpu(binding.Plan((27,), LAT), torch.from_numpy(x).to(DEV)).cpu().numpy()
    bw = run_gpu(binding.Plan((27,), BW), torch.from_numpy(x).to(DEV)).cpu().numpy()
    assert any(not np.array_equal(lat[0], lat[r]) for r in range(1, 27))
    assert all(np.array_equal(bw[0], bw[r]) for r in range(1, 27))


def test_launch_counter_and_kernel_names():
    plan = binding.Plan((27,), LAT)
    xd = torch.zeros((27, 1024), device=DEV)
    before = binding.launch_count()
    run_gpu(plan, xd, FUSED)
    assert binding.launch_count() == before + 1 and binding.last_kernel_name() == "lat_reg<27>"
    run_gpu(plan, xd, STEP)
    assert binding.launch_count() == before + 1 + 3 and binding.last_kernel_name() == "step_latency"


def test_calls_can_be_captured_in_a_cuda_graph():
    """The AllReduce call is a pure launch sequence (no allocation, no synchronisation): it can be
    captured into a CUDA graph and replayed; replays give the oracle's bits."""
    for dims, variant, kernel in [((27,), LAT, FUSED), ((243,), BW, FUSED), ((9, 9), LAT, STEP), ((9, 9, 9), LAT, FUSED),
                                  ((100,), BW, FUSED), ((32,), BW, STEP), ((27,), LAT, binding.KERNEL_PIPELINED),
                                  ((3, 9), LAT, binding.KERNEL_PIPELINED)]:
        plan = binding.Plan(dims, variant)
        n, count = plan.n, 2048
        x = synth.rank_matrix("normal", 77, n, count)
        xin = torch.from_numpy(x).to(DEV)
        xout = torch.zeros_like(xin)
        need = plan.scratch_bytes(count, kernel, in_place=False)
        scratch = torch.empty(max(need, 256), dtype=torch.uint8, device=DEV)
        ip = binding.ptr_array([xin[r].data_ptr() for r in range(n)])
        op = binding.ptr_array([xout[r].data_ptr() for r in range(n)])
        g = torch.cuda.CUDAGraph()
        torch.cuda.synchronize()
        with torch.cuda.graph(g):
            plan.allreduce_ex(ip, op, count, binding.FLOAT32, kernel=kernel, scratch_ptr=scratch.data_ptr() if need else 0,
                              scratch_bytes=need, stream=torch.cuda.current_stream().cuda_stream)
        for _ in range(2):
            xout.zero_()
            g.replay()
            torch.cuda.synchronize()
            compare(dims, variant, x, xout.cpu().numpy())


def test_tma_fed_kernels_never_gave_up():
    """The bounded wait of the TMA-fed 9x9x9 kernel did not run out in any call of this process."""
    check_case((9, 9, 9), LAT, 2051, "normal", 91, FUSED)
    assert binding.last_kernel_name() == "lat_t999_planes"
    check_case((9, 9, 9), LAT, 1031, "int32", 92, FUSED, in_place=False)
    assert binding.tma_giveups() == 0
