"""ctypes binding of ``libtrivance.so``: same names as the C ABI, argument marshalling only.

Every step of the AllReduce path runs in the library's CUDA kernels.  PyTorch is used by
callers for device memory and streams; this module only needs ``data_ptr()``-like integers.
If the library has not been built, loading fails with an error: there is no CPU fallback.
"""
import ctypes
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtrivance.so")

LATENCY_OPTIMAL, BANDWIDTH_OPTIMAL = 0, 1
ALGO_TRIVANCE, ALGO_BRUCK, ALGO_RECDOUB, ALGO_SWING, ALGO_BUCKET = 0, 1, 2, 3, 4
ALGO_MIRRORED = 16
ALGO_SINGLE = 32
INT32, FLOAT32 = 0, 1
SUM = 0
KERNEL_AUTO, KERNEL_STEP, KERNEL_FUSED, KERNEL_PIPELINED = 0, 1, 2, 3
MAX_RANKS = 1024

(OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_UNDEFINED_SCHEDULE, ERR_ALLOC, ERR_CUDA, ERR_SCRATCH, ERR_TOO_LARGE,
 ERR_TIMEOUT) = range(9)

# every symbol include/trivance.h declares
SYMBOLS = [
    "trv_plan_create", "trv_plan_create_algo", "trv_plan_destroy", "trv_plan_info", "trv_plan_slices", "trv_plan_step",
    "trv_plan_peers", "trv_plan_send_set", "trv_plan_block_bounds", "trv_allreduce", "trv_scratch_bytes",
    "trv_kernel_supported", "trv_allreduce_ex", "trv_allreduce_host", "trv_host_workspace_bytes",
    "trv_link_loads", "trv_plan_message_bytes", "trv_plan_message_bytes_side", "trv_strerror", "trv_launch_count", "trv_last_kernel_name",
    "trv_allreduce_noalloc", "trv_noalloc_max_scratch_bytes", "trv_cost_model", "trv_pipeline_status",
    "trv_pipeline_selftest_timeout", "trv_tma_giveups", "trv_plan_reserve_scratch", "trv_joint_reduce",
]


class Cost(ctypes.Structure):
    """trv_cost_t"""
    _fields_ = [("steps", ctypes.c_int32), ("bytes_sent_per_node", ctypes.c_int64), ("tx_bytes", ctypes.c_int64),
                ("latency_term", ctypes.c_double), ("tx_term", ctypes.c_double), ("total", ctypes.c_double),
                ("lambda_", ctypes.c_double), ("delta", ctypes.c_double), ("theta", ctypes.c_double)]

_lib = None


class TrivanceError(RuntimeError):
    def __init__(self, status, what):
        super().__init__("%s: %s (status %d)" % (what, strerror(status), status))
        self.status = status


def lib():
    """The loaded C-ABI library (loads it on first use; raises if it was never built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("%s is missing: build it with `python -m paper_2602_17254_b200.build` "
                               "(there is no fallback path)" % LIB_PATH)
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t
        L.trv_plan_create.argtypes = [vp, i32, ctypes.c_int, ctypes.POINTER(vp)]
        L.trv_plan_create_algo.argtypes = [vp, i32, ctypes.c_int, ctypes.c_int, ctypes.POINTER(vp)]
        L.trv_plan_destroy.argtypes = [vp]
        L.trv_plan_info.argtypes = [vp, ctypes.POINTER(i32), ctypes.POINTER(i32), ctypes.POINTER(i32)]
        L.trv_plan_step.argtypes = [vp, i32, i32, ctypes.POINTER(i32), ctypes.POINTER(i32)]
        L.trv_plan_peers.argtypes = [vp, i32, i32, vp]
        L.trv_plan_send_set.argtypes = [vp, i32, i32, i32, vp]
        L.trv_plan_block_bounds.argtypes = [vp, sz, i32, vp]
        L.trv_plan_message_bytes.argtypes = [vp, sz, sz, i32, i32, vp]
        L.trv_plan_slices.argtypes = [vp, vp]
        L.trv_plan_message_bytes_side.argtypes = [vp, sz, sz, i32, i32, i32, vp]
        L.trv_pipeline_status.argtypes = [vp, vp]
        L.trv_pipeline_selftest_timeout.argtypes = [vp, sz, vp]
        L.trv_allreduce.argtypes = [vp, vp, sz, ctypes.c_int, ctypes.c_int, vp]
        L.trv_plan_reserve_scratch.argtypes = [vp, sz]
        L.trv_joint_reduce.argtypes = [vp, vp, vp, vp, vp, sz, ctypes.c_int, vp]
        L.trv_scratch_bytes.argtypes = [vp, sz, ctypes.c_int, i32, ctypes.POINTER(sz)]
        L.trv_kernel_supported.argtypes = [vp, ctypes.c_int]
        L.trv_kernel_supported.restype = i32
        L.trv_allreduce_ex.argtypes = [vp, vp, vp, sz, sz, sz, ctypes.c_int, ctypes.c_int, ctypes.c_int, vp, sz, vp]
        L.trv_allreduce_noalloc.argtypes = [vp, vp, sz, ctypes.c_int, ctypes.c_int, vp]
        L.trv_noalloc_max_scratch_bytes.argtypes = []
        L.trv_noalloc_max_scratch_bytes.restype = sz
        L.trv_allreduce_host.argtypes = [vp, vp, vp, sz, ctypes.c_int, ctypes.c_int, vp, sz, vp]
        L.trv_host_workspace_bytes.argtypes = [vp, sz, ctypes.POINTER(sz)]
        L.trv_link_loads.argtypes = [vp, sz, sz, vp, vp, vp, vp]
        L.trv_cost_model.argtypes = [vp, sz, sz, ctypes.c_double, ctypes.c_double, ctypes.POINTER(Cost)]
        L.trv_strerror.argtypes = [ctypes.c_int]
        L.trv_strerror.restype = ctypes.c_char_p
        L.trv_launch_count.argtypes = []
        L.trv_launch_count.restype = ctypes.c_uint64
        L.trv_last_kernel_name.argtypes = []
        L.trv_last_kernel_name.restype = ctypes.c_char_p
        _lib = L
    return _lib


def strerror(status):
    return lib().trv_strerror(int(status)).decode()


def noalloc_max_scratch_bytes():
    return int(lib().trv_noalloc_max_scratch_bytes())


def pipeline_status(scratch_ptr, stream=0):
    """Status code (OK or ERR_TIMEOUT) recorded by the last PIPELINED call that used this device scratch."""
    return int(lib().trv_pipeline_status(scratch_ptr, stream))


def pipeline_selftest_timeout(scratch_ptr, scratch_bytes, stream=0):
    _check(lib().trv_pipeline_selftest_timeout(scratch_ptr, scratch_bytes, stream), "trv_pipeline_selftest_timeout")


def tma_giveups():
    """Thread blocks of TMA-fed kernels that gave up waiting for their tile on the current device (0 in a correct run)."""
    v = ctypes.c_uint32()
    _check(lib().trv_tma_giveups(ctypes.byref(v)), "trv_tma_giveups")
    return v.value


def joint_reduce(left, own, right, out, counts, dtype, stream=0):
    """trv_joint_reduce: out[s] = (left[s] + own[s]) + right[s] on segments given as lists of device addresses (0 = side left out)."""
    k = len(own)
    arr = lambda p: None if p is None else (ctypes.c_void_p * k)(*[int(v) if v else None for v in p])
    cnt = (ctypes.c_size_t * k)(*[int(c) for c in counts])
    _check(lib().trv_joint_reduce(arr(left), arr(own), arr(right), arr(out), cnt, k, int(dtype), ctypes.c_void_p(int(stream))),
           "trv_joint_reduce")


def launch_count():
    return int(lib().trv_launch_count())


def last_kernel_name():
    return lib().trv_last_kernel_name().decode()


def _check(status, what):
    if status != OK:
        raise TrivanceError(status, what)


def ptr_array(ptrs):
    """HOST array of pointers in the form the C ABI takes.  Build it once and pass it to the Plan's
    calls instead of a list when the same buffers are used repeatedly (saves the per-call conversion)."""
    if isinstance(ptrs, ctypes.Array):
        return ptrs
    return (ctypes.c_void_p * len(ptrs))(*[int(p) for p in ptrs])


_ptr_array = ptr_array


def _np_ptr(a):
    return a.ctypes.data_as(ctypes.c_void_p) if a is not None else None


class Plan:
    """trv_plan_t with the C ABI's calls as methods."""

    def __init__(self, dims, variant, algo=ALGO_TRIVANCE):
        d = np.ascontiguousarray(np.asarray(dims, dtype=np.int32).reshape(-1))
        h = ctypes.c_void_p()
        _check(lib().trv_plan_create_algo(_np_ptr(d), d.size, int(variant), int(algo), ctypes.byref(h)), "trv_plan_create")
        self._h = h
        self.dims = tuple(int(v) for v in d)
        self.variant, self.algo = int(variant), int(algo)
        n, nd, rows = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32()
        _check(lib().trv_plan_info(h, ctypes.byref(n), ctypes.byref(nd), ctypes.byref(rows)), "trv_plan_info")
        self.n, self.ndims, self.rows = n.value, nd.value, rows.value
        ns = ctypes.c_int32()
        _check(lib().trv_plan_slices(h, ctypes.byref(ns)), "trv_plan_slices")
        self.nslices = ns.value

    def destroy(self):
        if getattr(self, "_h", None):
            lib().trv_plan_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    # ---- schedule queries (host integer tables)
    def step(self, c, row):
        dim, dist = ctypes.c_int32(), ctypes.c_int32()
        _check(lib().trv_plan_step(self._h, c, row, ctypes.byref(dim), ctypes.byref(dist)), "trv_plan_step")
        return dim.value, dist.value

    def peers(self, c, row):
        out = np.zeros((self.n, 2), np.int32)
        _check(lib().trv_plan_peers(self._h, c, row, _np_ptr(out)), "trv_plan_peers")
        return out

    def send_set(self, c, step, dst):
        out = np.zeros(self.n, np.uint8)
        _check(lib().trv_plan_send_set(self._h, c, step, dst, _np_ptr(out)), "trv_plan_send_set")
        return out.astype(bool)

    def send_mask(self, c, step, dst):
        """Raw bytes of trv_plan_send_set (rings of other sizes: bit 0 = from the left peer, bit 1 = from the right)."""
        out = np.zeros(self.n, np.uint8)
        _check(lib().trv_plan_send_set(self._h, c, step, dst, _np_ptr(out)), "trv_plan_send_set")
        return out

    def block_bounds(self, count, c):
        out = np.zeros(self.n + 1, np.int64)
        _check(lib().trv_plan_block_bounds(self._h, count, c, _np_ptr(out)), "trv_plan_block_bounds")
        return out

    def message_bytes(self, count, elem_size, c, row):
        out = np.zeros(self.n, np.int64)
        _check(lib().trv_plan_message_bytes(self._h, count, elem_size, c, row, _np_ptr(out)), "trv_plan_message_bytes")
        return out

    def message_bytes_side(self, count, elem_size, c, row, side):
        out = np.zeros(self.n, np.int64)
        _check(lib().trv_plan_message_bytes_side(self._h, count, elem_size, c, row, side, _np_ptr(out)),
               "trv_plan_message_bytes_side")
        return out

    def kernel_supported(self, kernel):
        return bool(lib().trv_kernel_supported(self._h, int(kernel)))

    def scratch_bytes(self, count, kernel=KERNEL_AUTO, in_place=True):
        b = ctypes.c_size_t()
        _check(lib().trv_scratch_bytes(self._h, count, int(kernel), 1 if in_place else 0, ctypes.byref(b)), "trv_scratch_bytes")
        return b.value

    def reserve_scratch(self, count):
        """trv_plan_reserve_scratch: allocate the plan-owned scratch trv_allreduce needs up to this count (may wait for
        the device); afterwards trv_allreduce is launch-only for every shape."""
        _check(lib().trv_plan_reserve_scratch(self._h, count), "trv_plan_reserve_scratch")

    def host_workspace_bytes(self, count):
        b = ctypes.c_size_t()
        _check(lib().trv_host_workspace_bytes(self._h, count, ctypes.byref(b)), "trv_host_workspace_bytes")
        return b.value

    # ---- AllReduce (pointers are plain integers: device addresses)
    def allreduce(self, rank_ptrs, count, dtype, stream=0, op=SUM):
        arr = _ptr_array(rank_ptrs)
        _check(lib().trv_allreduce(self._h, arr, count, int(dtype), int(op), ctypes.c_void_p(int(stream))), "trv_allreduce")

    def allreduce_ex(self, in_ptrs, out_ptrs, count, dtype, global_count=None, global_offset=0, kernel=KERNEL_AUTO,
                     scratch_ptr=0, scratch_bytes=0, stream=0, op=SUM):
        a_in = _ptr_array(in_ptrs)
        a_out = a_in if out_ptrs is None or out_ptrs is in_ptrs else _ptr_array(out_ptrs)
        gc = count if global_count is None else global_count
        _check(lib().trv_allreduce_ex(self._h, a_in, a_out, count, gc, global_offset, int(dtype), int(op), int(kernel),
                                      ctypes.c_void_p(int(scratch_ptr)), scratch_bytes, ctypes.c_void_p(int(stream))),
               "trv_allreduce_ex")

    def allreduce_noalloc(self, rank_ptrs, count, dtype, stream=0, op=SUM):
        """trv_allreduce_noalloc: in-place latency-form AllReduce whose scratch is a fixed array inside the
        library (16 MiB), for callers that may not allocate device memory.  Calls sharing a GPU must not overlap."""
        arr = _ptr_array(rank_ptrs)
        _check(lib().trv_allreduce_noalloc(self._h, arr, count, int(dtype), int(op), ctypes.c_void_p(int(stream))),
               "trv_allreduce_noalloc")

    def allreduce_host(self, host_in_ptrs, host_out_ptrs, count, dtype, workspace_ptr, workspace_bytes, stream=0, op=SUM):
        a_in = _ptr_array(host_in_ptrs)
        a_out = a_in if host_out_ptrs is None or host_out_ptrs is host_in_ptrs else _ptr_array(host_out_ptrs)
        _check(lib().trv_allreduce_host(self._h, a_in, a_out, count, int(dtype), int(op), ctypes.c_void_p(int(workspace_ptr)),
                                        workspace_bytes, ctypes.c_void_p(int(stream))), "trv_allreduce_host")

    # ---- link loads
    def link_loads(self, count, elem_size=4):
        T, n, D = self.rows, self.n, self.ndims
        msgs = np.zeros((T, n, D, 2), np.int32)
        byts = np.zeros((T, n, D, 2), np.int64)
        mm = np.zeros(T, np.int32)
        mb = np.zeros(T, np.int64)
        _check(lib().trv_link_loads(self._h, count, elem_size, _np_ptr(msgs), _np_ptr(byts), _np_ptr(mm), _np_ptr(mb)),
               "trv_link_loads")
        return {"msgs": msgs, "bytes": byts, "max_msgs": mm, "max_bytes": mb}


    def cost_model(self, count, elem_size, alpha, beta):
        c = Cost()
        _check(lib().trv_cost_model(self._h, count, elem_size, float(alpha), float(beta), ctypes.byref(c)), "trv_cost_model")
        return c


# ---------------------------------------------------------------- torch conveniences (marshalling only)

def _torch_dtype_code(t):
    import torch
    if t.dtype == torch.float32:
        return FLOAT32
    if t.dtype == torch.int32:
        return INT32
    raise TypeError("only float32 and int32 tensors are supported")


def allreduce_tensor(plan, x, out=None, kernel=KERNEL_AUTO, global_count=None, global_offset=0, scratch=None):
    """AllReduce of a CUDA tensor x of shape [n, count] (row r = rank r), in place unless `out` is given.

    Rows must be 16-byte aligned (count a multiple of 4, or a row stride that is).  Runs on torch's
    current stream.  Returns the tensor holding the result.
    """
    import torch
    if not x.is_cuda or x.dim() != 2 or x.shape[0] != plan.n or x.stride(1) != 1:
        raise ValueError("x must be a CUDA tensor of shape [n, count] with unit inner stride")
    dst = x if out is None else out
    if dst.shape != x.shape or dst.dtype != x.dtype or dst.stride(1) != 1:
        raise ValueError("out must match x")
    count = x.shape[1]
    es = x.element_size()
    in_ptrs = [x.data_ptr() + r * x.stride(0) * es for r in range(plan.n)]
    out_ptrs = in_ptrs if out is None else [dst.data_ptr() + r * dst.stride(0) * es for r in range(plan.n)]
    need = plan.scratch_bytes(count, kernel, in_place=out is None)
    sp, sb = 0, 0
    if need:
        if scratch is None or scratch.numel() * scratch.element_size() < need:
            scratch = torch.empty(need, dtype=torch.uint8, device=x.device)
        sp, sb = scratch.data_ptr(), scratch.numel() * scratch.element_size()
    plan.allreduce_ex(in_ptrs, None if out is None else out_ptrs, count, _torch_dtype_code(x), global_count, global_offset,
                      kernel, sp, sb, torch.cuda.current_stream().cuda_stream)
    return dst
