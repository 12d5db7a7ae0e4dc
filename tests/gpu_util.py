"""Helpers of the GPU parity tests: run the CUDA path through the C ABI, run the oracle on the same
bits, compare element by element."""
import concurrent.futures
import os

import numpy as np
import torch

import oracle
from paper_2602_17254_b200 import binding, synth

DEV = "cuda:0"


def torch_dtype(np_dtype):
    return torch.int32 if np.dtype(np_dtype) == np.int32 else torch.float32


def upload_matrix(dist, seed, n, count, windows=()):
    """Draws rank vectors on the host (thread pool over ranks), uploads them as an [n, count] CUDA
    tensor and keeps the requested element windows on the host for the oracle."""
    dt = np.int32 if dist == "int32" else np.float32
    # row stride padded to a multiple of 4 elements: every rank buffer starts 16-byte aligned
    dev = torch.empty((n, (count + 3) // 4 * 4), dtype=torch_dtype(dt), device=DEV)[:, :count]
    keep = [np.empty((n, w1 - w0), dt) for (w0, w1) in windows]

    def one(r):
        v = synth.rank_vector(dist, seed, r, count)
        for k, (w0, w1) in enumerate(windows):
            keep[k][r] = v[w0:w1]
        return r, v

    with concurrent.futures.ThreadPoolExecutor(max_workers=min(16, os.cpu_count() or 4)) as ex:
        for r, v in ex.map(one, range(n)):
            dev[r].copy_(torch.from_numpy(v))
    torch.cuda.synchronize()
    return dev, keep


def run_gpu(plan, x_dev, kernel=binding.KERNEL_AUTO, in_place=True, global_count=None, global_offset=0):
    """Runs the CUDA path; returns the [n, count] result tensor (x_dev itself when in place)."""
    out = None
    if not in_place:        # rows must stay 16-byte aligned: pad the row stride to a multiple of 4 elements
        n, count = x_dev.shape
        out = torch.full((n, (count + 3) // 4 * 4), -77, dtype=x_dev.dtype, device=x_dev.device)[:, :count]
    res = binding.allreduce_tensor(plan, x_dev, out=out, kernel=kernel, global_count=global_count,
                                   global_offset=global_offset)
    torch.cuda.synchronize()
    return res


def compare(dims, variant, x_host, got_host, E=None, e0=0):
    """Oracle on x_host ([n][w] window starting at e0 of vectors of E elements) vs the GPU's values:
    bit-exact for int32 and for the schedule-ordered float32 sum."""
    want = oracle.allreduce(dims, variant, x_host, E=E, e0=e0)
    assert got_host.dtype == want.dtype and got_host.shape == want.shape
    if not np.array_equal(got_host.view(np.uint32), want.view(np.uint32)):
        bad = np.argwhere(got_host.view(np.uint32) != want.view(np.uint32))
        r, e = bad[0]
        raise AssertionError("%d of %d values differ; first at rank %d element %d: got %r want %r"
                             % (len(bad), want.size, r, e0 + e, got_host[r, e], want[r, e]))
    return want


def check_scattered(dims, variant, count, dist, seed, kernel):
    """Same as check_case, in place, but the rank buffers are NOT equally spaced (rows of a pool
    in shuffled order): exercises the pointer-table addressing of the kernels."""
    plan = binding.Plan(dims, variant)
    n = plan.n
    x = synth.rank_matrix(dist, seed, n, count)
    pad = (count + 3) // 4 * 4 + 4
    pool = torch.zeros((n + 1, pad), dtype=torch_dtype(x.dtype), device=DEV)
    order = np.random.default_rng(seed).permutation(n + 1)[:n]
    rows = [pool[int(order[r])] for r in range(n)]
    for r in range(n):
        rows[r][:count].copy_(torch.from_numpy(x[r]))
    ptrs = [rows[r].data_ptr() for r in range(n)]
    need = plan.scratch_bytes(count, kernel, in_place=True)
    scratch = torch.empty(max(need, 256), dtype=torch.uint8, device=DEV)
    plan.allreduce_ex(ptrs, None, count, binding.INT32 if x.dtype == np.int32 else binding.FLOAT32, kernel=kernel,
                      scratch_ptr=scratch.data_ptr() if need else 0, scratch_bytes=need,
                      stream=torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    got = np.stack([rows[r][:count].cpu().numpy() for r in range(n)])
    compare(dims, variant, x, got)
    for r in range(n):
        assert torch.count_nonzero(rows[r][count:]).item() == 0, "wrote past the end of a rank buffer"
    plan.destroy()


def check_case(dims, variant, count, dist, seed, kernel, in_place=True, shard=None):
    """Full element-by-element parity on a case the oracle finishes quickly.
    shard = (global_count, global_offset): the buffers hold only that window of a longer vector."""
    plan = binding.Plan(dims, variant)
    n = plan.n
    x = synth.rank_matrix(dist, seed, n, count)
    # row stride padded to a multiple of 4 elements so that every row is 16-byte aligned
    pad = (count + 3) // 4 * 4
    buf = torch.zeros((n, pad), dtype=torch_dtype(x.dtype), device=DEV)
    xd = buf[:, :count]
    xd.copy_(torch.from_numpy(x))
    gc, go = (count, 0) if shard is None else shard
    res = run_gpu(plan, xd, kernel, in_place, gc, go)
    got = res.cpu().numpy()
    want = compare(dims, variant, x, got, E=gc, e0=go)
    if not in_place:
        assert np.array_equal(xd.cpu().numpy(), x), "input modified by an out-of-place call"
    if pad > count:
        assert torch.count_nonzero(buf[:, count:]).item() == 0, "wrote past the end of a rank buffer"
    plan.destroy()
    return x, want
