"""GPU parity for the PIPELINED family (chunk-level readiness engine, App. D): bit-exact against the
oracle and the other families; its bounded waits give up with a status instead of hanging."""
import numpy as np
import pytest
import torch

from paper_2602_17254_b200 import binding, build, synth

from gpu_util import DEV, compare, torch_dtype

pytestmark = pytest.mark.gpu

LAT, BW = binding.LATENCY_OPTIMAL, binding.BANDWIDTH_OPTIMAL
PIPE = binding.KERNEL_PIPELINED


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    assert torch.cuda.is_available()
    binding.lib()


def _run(dims, count, dist, seed, in_place=True, shard=None, scattered=False, variant=LAT):
    plan = binding.Plan(dims, variant)
    n = plan.n
    x = synth.rank_matrix(dist, seed, n, count)
    pad = (count + 3) // 4 * 4 + 4
    pool = torch.zeros((n + 1, pad), dtype=torch_dtype(x.dtype), device=DEV)
    order = np.random.default_rng(seed).permutation(n + 1)[:n] if scattered else np.arange(n)
    rows = [pool[int(order[r])] for r in range(n)]
    for r in range(n):
        rows[r][:count].copy_(torch.from_numpy(x[r]))
    outp = None
    if not in_place:
        opool = torch.full((n, pad), -77, dtype=pool.dtype, device=DEV)
        outp = [opool[r].data_ptr() for r in range(n)]
    gc, go = (count, 0) if shard is None else shard
    need = plan.scratch_bytes(gc if variant == BW else count, PIPE, in_place=in_place)
    assert need > 0
    scratch = torch.empty(need, dtype=torch.uint8, device=DEV)
    before = binding.launch_count()
    plan.allreduce_ex([rows[r].data_ptr() for r in range(n)], outp, count,
                      binding.INT32 if x.dtype == np.int32 else binding.FLOAT32, global_count=gc, global_offset=go,
                      kernel=PIPE, scratch_ptr=scratch.data_ptr(), scratch_bytes=need,
                      stream=torch.cuda.current_stream().cuda_stream)
    assert binding.last_kernel_name() == ("lat_pipe" if variant == LAT else "bw_pipe") and binding.launch_count() - before == 1
    assert binding.pipeline_status(scratch.data_ptr(), torch.cuda.current_stream().cuda_stream) == binding.OK
    if in_place:
        got = np.stack([rows[r][:count].cpu().numpy() for r in range(n)])
        for r in range(n):
            assert torch.count_nonzero(rows[r][count:]).item() == 0, "wrote past the end of a rank buffer"
    else:
        got = opool[:, :count].cpu().numpy()
        assert (opool[:, count:] == -77).all().item(), "wrote past the end of a rank buffer"
        assert np.array_equal(np.stack([rows[r][:count].cpu().numpy() for r in range(n)]), x), "input modified"
    compare(dims, variant, x, got, E=gc, e0=go)
    plan.destroy()


SHAPES = [(9,), (27,), (81,), (243,), (729,), (3, 3), (9, 9), (3, 9), (27, 3), (3, 3, 3), (9, 9, 9), (3, 3, 9)]


@pytest.mark.parametrize("dims", SHAPES)
def test_matches_oracle(dims):
    n = int(np.prod(dims))
    count = 5003 if n <= 243 else 2051          # several chunks per slice, ragged, unaligned slice starts
    _run(dims, count, "normal", 41)
    _run(dims, count, "int32", 42, in_place=False)
    _run(dims, count, "uniform", 43, scattered=True)


@pytest.mark.parametrize("dims", SHAPES + [(3,)])
def test_bandwidth_form_matches_oracle(dims):
    """Reduce-Scatter and AllGather by the readiness engine: a chunk is a piece of one block (its active block range)."""
    n = int(np.prod(dims))
    count = 40009 if n <= 243 else 9001         # blocks of ragged length; the ring of 27 gets blocks of several chunks below
    _run(dims, count, "normal", 51, variant=BW)
    _run(dims, count, "int32", 52, in_place=False, variant=BW)
    _run(dims, count, "uniform", 53, scattered=True, variant=BW)


def test_bandwidth_form_blocks_of_several_chunks_and_many_groups():
    _run((27,), 200003, "normal", 54, variant=BW)                   # 7408 elements per block: four chunks
    _run((9,), 1500007, "int32", 55, in_place=False, variant=BW)    # 82 chunks per block
    _run((9, 9), 700001, "normal", 56, variant=BW)
    _run((3, 3, 3), 5, "int32", 57, variant=BW)                     # most blocks empty


@pytest.mark.parametrize("dims", [(27,), (9, 9), (9, 9, 9)])
def test_bandwidth_form_sharded_window(dims):
    gcount = 30011
    for lo, hi in ((0, 15004), (15004, gcount), (7000, 7000 + 4096)):
        _run(dims, hi - lo, "int32", 58, shard=(gcount, lo), variant=BW)
        _run(dims, hi - lo, "normal", 59, in_place=False, shard=(gcount, lo), variant=BW)


@pytest.mark.parametrize("dims", [(3,), (9,), (27,)])
@pytest.mark.parametrize("count", [1, 2, 5, 1023, 1024, 1025])
def test_short_vectors(dims, count):
    _run(dims, count, "int32", 44, in_place=False)
    if dims != (3,):
        _run(dims, count, "normal", 45)


def test_many_groups():
    """More chunks than one group holds: several groups of chunks follow one another through all steps."""
    _run((27,), 1500007, "normal", 46)
    _run((9, 9), 300007, "int32", 47, in_place=False)


@pytest.mark.parametrize("dims", [(27,), (9, 9, 9)])
def test_sharded_window(dims):
    gcount = 30011
    for lo, hi in ((0, 15004), (15004, gcount), (7000, 7000 + 4096)):
        _run(dims, hi - lo, "int32", 48, shard=(gcount, lo))
        _run(dims, hi - lo, "normal", 49, in_place=False, shard=(gcount, lo))


def test_unsupported_and_scratch_checks():
    stream = torch.cuda.current_stream().cuda_stream
    x = torch.zeros((27, 64), dtype=torch.int32, device=DEV)
    ptrs = [x[r].data_ptr() for r in range(27)]
    scratch = torch.empty(1 << 20, dtype=torch.uint8, device=DEV)
    assert binding.Plan((27,), BW).kernel_supported(PIPE)
    for dims, variant in (((10,), BW), ((4, 4), BW)):
        plan = binding.Plan(dims, variant)
        assert not plan.kernel_supported(PIPE)
        with pytest.raises(binding.TrivanceError) as e:
            plan.allreduce_ex(ptrs[:plan.n], None, 64, binding.INT32, kernel=PIPE, scratch_ptr=scratch.data_ptr(),
                              scratch_bytes=1 << 20, stream=stream)
        assert e.value.status == binding.ERR_UNSUPPORTED
        plan.destroy()
    plan = binding.Plan((27,), LAT)
    assert plan.kernel_supported(PIPE)
    with pytest.raises(binding.TrivanceError) as e:
        plan.allreduce_ex(ptrs, None, 64, binding.INT32, kernel=PIPE, scratch_ptr=scratch.data_ptr(), scratch_bytes=256, stream=stream)
    assert e.value.status == binding.ERR_SCRATCH
    plan.destroy()
    plan = binding.Plan((3,), LAT)       # a single step cannot run in place
    with pytest.raises(binding.TrivanceError) as e:
        plan.scratch_bytes(64, PIPE, in_place=True)
    assert e.value.status == binding.ERR_UNSUPPORTED
    plan.destroy()


def test_bounded_wait_gives_up_and_the_context_survives():
    """A waiter whose entry nothing sets runs out of polls, records TRV_ERR_TIMEOUT and returns; the
    next call on the same scratch works and reports OK again."""
    stream = torch.cuda.current_stream().cuda_stream
    scratch = torch.empty(1 << 22, dtype=torch.uint8, device=DEV)
    binding.pipeline_selftest_timeout(scratch.data_ptr(), scratch.numel(), stream)
    assert binding.pipeline_status(scratch.data_ptr(), stream) == binding.ERR_TIMEOUT
    assert binding.strerror(binding.ERR_TIMEOUT).startswith("a bounded device-side wait")
    plan = binding.Plan((27,), LAT)
    x = synth.rank_matrix("int32", 50, 27, 4096)
    xd = torch.from_numpy(x).to(DEV)
    need = plan.scratch_bytes(4096, PIPE, in_place=True)
    assert need <= scratch.numel()
    plan.allreduce_ex([xd[r].data_ptr() for r in range(27)], None, 4096, binding.INT32, kernel=PIPE,
                      scratch_ptr=scratch.data_ptr(), scratch_bytes=scratch.numel(), stream=stream)
    assert binding.pipeline_status(scratch.data_ptr(), stream) == binding.OK
    compare((27,), LAT, x, xd.cpu().numpy())
    plan.destroy()
