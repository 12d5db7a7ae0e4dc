#!/usr/bin/env python
"""Benchmark of the Trivance AllReduce hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

Default workload: torus9x9x9_lat_32MiB, the largest single-GPU configuration (729 ranks x 32 MiB).
One "step" is `calls_per_step` passes of the whole hot path, each one trv_allreduce_ex call on one of
`buffer_sets` independent synthetic buffer sets of the workload (plan built once, outside the timed
region); consecutive calls rotate over sets that together exceed several times the L2 capacity, so
every call reads cold data from HBM.  calls_per_step is chosen after the warm-up so that the timed
region lasts at least 0.55 s (clock samples then fall inside it).  Metric: effective AllReduce GB/s =
n * S_bytes / t, S_bytes = per-rank vector size.  Rank 0 prints ONE JSON line; besides the contract's
keys it carries `roofline` (dominant kernel against the measured copy bandwidth), `e2e` (host buffers
through trv_allreduce_host, with the plain pinned-copy rate of the same bytes as ceiling),
`in_place_trv_allreduce_us` (the in-place call), `cpu_baseline` (the oracle on the host cores) and
`per_workload`: the device-resident leg of every other configuration with >= 2 MiB per rank.

With --gpus N > 1 (launched under torchrun) every GPU runs its own batch (element columns are
independent, so a longer vector sharded by element range behaves the same): no collective on the
data path, weak scaling; the time is the max over ranks.

--impl reference times the CPU oracle (oracle/, as it stands) on the host cores for the same
workload and metric; it needs no GPU.
"""
import argparse
import concurrent.futures
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2602_17254_b200 import synth  # noqa: E402

DEFAULT_WORKLOAD = "torus9x9x9_lat_32MiB"
L2_BYTES = 126 * 1024 * 1024
FALLBACK_HBM_GBS = 6650.0


def _peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json, copy bandwidth)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (earlier pool measurement)"


def _traffic(kernel_name, workload):
    """DRAM bytes per launch from the committed ncu capture of this kernel/workload, if there is one."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    try:
        with open(path) as f:
            return json.load(f).get("%s|%s" % (kernel_name, workload))
    except Exception:
        return None


# ------------------------------------------------------------------ CPU oracle leg

def _oracle_pass(w, x, threads):
    """One oracle AllReduce of one buffer set, element windows spread over `threads` host threads."""
    import oracle
    E = w.count
    cuts = [(E * i) // threads for i in range(threads + 1)]
    parts = [(cuts[i], cuts[i + 1]) for i in range(threads) if cuts[i + 1] > cuts[i]]

    def one(rng):
        e0, e1 = rng
        return oracle.allreduce(w.dims, w.variant, np.ascontiguousarray(x[:, e0:e1]), E=E, e0=e0)

    if threads == 1:
        return [one(parts[0])]
    with concurrent.futures.ThreadPoolExecutor(max_workers=threads) as ex:
        return list(ex.map(one, parts))


def _oracle_sample(w):
    """Bounded sample of the workload for the CPU legs: the whole vector if small, else a prefix."""
    max_elems = (64 * 1024 * 1024) // (4 * w.n)           # <= 64 MiB of input
    count = min(w.count, max(1024, max_elems))
    # Timing a prefix keeps the run short; the oracle's cost per element does not depend on E.
    sub = synth.Workload(w.name, w.dims, w.variant, count, w.dist, w.seed)
    return sub, synth.workload_inputs(sub)


def cpu_baseline(w, budget_s=12.0):
    import oracle
    oracle.build()
    cores = os.cpu_count() or 1
    sub, x = _oracle_sample(w)
    _oracle_pass(sub, x, cores)                             # warm-up (page faults, library load)
    t0 = time.perf_counter()
    _oracle_pass(sub, x, 1)
    t1 = time.perf_counter() - t0
    reps, t0 = 0, time.perf_counter()
    while True:
        _oracle_pass(sub, x, cores)
        reps += 1
        el = time.perf_counter() - t0
        if (el >= budget_s and reps >= 3) or el >= 2.5 * budget_s:
            break
    nbytes = sub.n * sub.count * 4
    return {
        "value": nbytes * reps / el / 1e9, "unit": "GB/s", "cores": cores, "kind": "oracle",
        "sample": "%d passes of the oracle over %d of %d elements per rank of %s (%.1f MiB of input per pass), element "
                  "windows over %d threads" % (reps, sub.count, w.count, w.name, nbytes / 2**20, cores),
        "single_thread_value": nbytes / t1 / 1e9,
    }


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    cores = os.cpu_count() or 1
    sub, x = _oracle_sample(w)
    for _ in range(args.warmup):
        _oracle_pass(sub, x, cores)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        _oracle_pass(sub, x, cores)
    el = time.perf_counter() - t0
    nbytes = sub.n * sub.count * 4
    value = nbytes * args.steps / el / 1e9
    sample = "each step = one oracle pass over %d of %d elements per rank (%.1f MiB of input), %d threads" % (
        sub.count, w.count, nbytes / 2**20, cores)
    print(json.dumps({
        "impl": "reference", "metric": "allreduce_effective_GBps", "value": value, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": el / args.steps * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int32" if w.dist == "int32" else "f32", "data": "synthetic",
        "config": {"workload": w.name, "dims": list(w.dims), "variant": "latency" if w.variant == 0 else "bandwidth",
                   "bytes_per_rank": w.bytes_per_rank, "sample": sample},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# ------------------------------------------------------------------ clocks

class ClockSampler:
    """Samples SM clock and clock-event reasons through NVML while the timed region runs."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting", 0x10: "sync_boost"}

    def __init__(self, index):
        self.samples, self.reason_bits, self.max_mhz, self._stop, self._thr, self._h = [], 0, None, threading.Event(), None, None
        self.power = []
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            try:        # CUDA_VISIBLE_DEVICES renumbers CUDA devices but not NVML's: go by UUID
                import torch
                uuid = "GPU-" + str(torch.cuda.get_device_properties(index).uuid)
                self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self._h = None

    def _loop(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                try:
                    self.power.append(nv.nvmlDeviceGetPowerUsage(self._h) / 1e3)
                except Exception:
                    pass
                try:
                    self.reason_bits |= int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
                except Exception:
                    self.reason_bits |= int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
            except Exception:
                break
            time.sleep(0.001)

    def start(self):
        if self._h is not None:
            self._stop.clear()
            self._thr = threading.Thread(target=self._loop, daemon=True)
            self._thr.start()

    def stop(self):
        if self._thr is not None:
            self._stop.set()
            self._thr.join()
            self._thr = None

    def report(self, note):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0, "note": "NVML unavailable"}
        reasons = [name for bit, name in self.REASONS.items() if self.reason_bits & bit]
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz, "reasons": reasons,
                "samples": len(self.samples), "power_w": float(np.median(self.power)) if self.power else None, "note": note}


# ------------------------------------------------------------------ GPU legs

MIN_REGION_S = 0.55     # every timed region lasts at least this long, so that NVML samples fall inside it
PER_WORKLOAD = ["ring27_lat_2MiB", "ring81_bw_8MiB", "torus9x9x9_lat_32MiB", "torus9x9x9_bw_32MiB", "ring243_lat_8MiB",
                "ring243_bw_8MiB", "ring243_lat_32MiB", "ring243_bw_32MiB",      # the configurations with >= 2 MiB per rank
                "torus27x27_lat_8MiB", "torus9x81_lat_8MiB", "ring729_lat_8MiB"]  # the other 729-rank shapes, latency form


class Leg:
    """Device buffers and call arguments of one workload: `batch` independent buffer sets."""

    def __init__(self, torch, binding, w, dev, rank, batch, kfam):
        self.torch, self.binding, self.w, self.kfam = torch, binding, w, kfam
        n, count = w.n, w.count
        self.set_bytes = n * count * 4
        self.batch = batch or max(1, min(64, max(16, -(-4 * L2_BYTES // self.set_bytes)), (24 * 2**30) // self.set_bytes))
        self.tdt = torch.int32 if w.dist == "int32" else torch.float32
        self.dcode = binding.INT32 if w.dist == "int32" else binding.FLOAT32
        self.plan = binding.Plan(w.dims, w.variant)
        # Set 0 carries the workload's seeded vectors in its first columns (all of them when the set is small):
        # they feed the parity spot check.  Everything else is drawn on the device with the same distribution
        # (values do not influence the run time: the path has no data-dependent control flow).
        self.check_cols = count if self.set_bytes <= 2**28 else min(count, 4096)
        self.x0 = np.stack([synth.rank_vector(w.dist, w.seed, r, self.check_cols) for r in range(n)])
        self.ins = torch.empty((self.batch, n, count), dtype=self.tdt, device=dev)
        self.outs = torch.empty((self.batch, n, count), dtype=self.tdt, device=dev)
        g = torch.Generator(device=dev)
        g.manual_seed(1000 * w.seed + rank)
        for b in range(self.batch):
            if w.dist == "int32":
                self.ins[b].copy_(torch.randint(-1000, 1001, (n, count), generator=g, device=dev, dtype=self.tdt))
            elif w.dist == "normal":
                self.ins[b].normal_(generator=g)
            else:
                self.ins[b].uniform_(-1.0, 1.0, generator=g)
        self.ins[0][:, :self.check_cols].copy_(torch.from_numpy(self.x0))
        self.in_ptrs = [binding.ptr_array([self.ins[b, r].data_ptr() for r in range(n)]) for b in range(self.batch)]
        self.out_ptrs = [binding.ptr_array([self.outs[b, r].data_ptr() for r in range(n)]) for b in range(self.batch)]
        self.need = self.plan.scratch_bytes(count, kfam, in_place=False)
        self.scratch = torch.empty(max(self.need, 256), dtype=torch.uint8, device=dev)
        self.plan.reserve_scratch(count)            # trv_allreduce (in place) then only launches
        # per-call Python work is kept off the timed loop: the launch-bound sizes measure the library, not attribute look-ups
        self.stream = torch.cuda.current_stream().cuda_stream
        self.scratch_ptr = self.scratch.data_ptr() if self.need else 0

    def call(self, b):
        self.plan.allreduce_ex(self.in_ptrs[b], self.out_ptrs[b], self.w.count, self.dcode, kernel=self.kfam,
                               scratch_ptr=self.scratch_ptr, scratch_bytes=self.need, stream=self.stream)

    def call_in_place(self, b):     # the call the engine is named for: trv_allreduce on the output buffers of set b
        self.plan.allreduce(self.out_ptrs[b], self.w.count, self.dcode, self.stream)

    def parity(self):
        """Set 0's output of the timed calls against the oracle, on the seeded columns."""
        import oracle
        want = oracle.allreduce(self.w.dims, self.w.variant, self.x0, E=self.w.count, e0=0)
        got = self.outs[0, :, :self.check_cols].cpu().numpy()
        return bool(np.array_equal(got.view(np.uint32), want.view(np.uint32)))

    def free(self):
        self.plan.destroy()
        for name in ("ins", "outs", "scratch"):
            setattr(self, name, None)
        self.torch.cuda.empty_cache()


def _timed(torch, stream, fn, reps, sampler=None):
    """Milliseconds (CUDA events on the launching stream) of `reps` calls of fn(i)."""
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    if sampler:
        sampler.start()
    ev0.record(stream)
    for i in range(reps):
        fn(i)
    ev1.record(stream)
    torch.cuda.synchronize()
    if sampler:
        sampler.stop()
    return ev0.elapsed_time(ev1)


def _timed_in_place(torch, stream, leg, reps):
    """Microseconds per in-place trv_allreduce call.  Every call runs on fresh inputs (set b's outputs are refilled from
    its inputs first, untimed): repeated in place on its own results the data would overflow to inf/NaN within a dozen
    calls, and such data draws less power than the workload's."""
    pairs = []
    for i in range(reps):
        b = i % leg.batch
        leg.outs[b].copy_(leg.ins[b])
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        leg.call_in_place(b)
        e1.record(stream)
        pairs.append((e0, e1))
    torch.cuda.synchronize()
    return sum(a.elapsed_time(b) for a, b in pairs) * 1e3 / reps


def _calls_per_step(torch, stream, leg, steps, fixed):
    """Calls per step: a whole number of passes over the batch, enough for a timed region of MIN_REGION_S."""
    if fixed:
        return leg.batch
    ms = _timed(torch, stream, lambda i: leg.call(i % leg.batch), 2 * leg.batch) / (2 * leg.batch)
    passes = max(1, int(np.ceil(MIN_REGION_S * 1e3 / (ms * steps * leg.batch))))
    return passes * leg.batch


def _roofline(set_bytes, launches, calls, ms, kernel_name, workload):
    per_launch_ms = ms / launches
    algo_bytes = 2 * set_bytes / (launches / calls)         # per launch of the dominant kernel
    peak, peak_src = _peak()
    achieved = algo_bytes / (per_launch_ms * 1e-3) / 1e9
    return {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
            "traffic": _traffic(kernel_name, workload), "peak_source": peak_src, "algorithmic_bytes_per_launch": algo_bytes,
            "avg_launch_us": per_launch_ms * 1e3, "frac_of_nominal_8000": achieved / 8000.0}


def _side_leg(torch, binding, name, dev, local, steps, kfam):
    """One entry of `per_workload`: the device-resident leg of another configuration."""
    w = synth.CONFIGS[name]
    leg = Leg(torch, binding, w, dev, 0, 0, kfam)
    stream = torch.cuda.current_stream()
    for b in range(leg.batch):
        leg.call(b)
    cps = _calls_per_step(torch, stream, leg, steps, False)
    sampler = ClockSampler(local)
    l0 = binding.launch_count()
    ms = _timed(torch, stream, lambda i: leg.call(i % leg.batch), steps * cps, sampler)
    launches, calls = binding.launch_count() - l0, steps * cps
    kernel_name = binding.last_kernel_name()
    parity = leg.parity()
    us_ip = _timed_in_place(torch, stream, leg, max(leg.batch, min(200, calls // 2)))
    roof = _roofline(leg.set_bytes, launches, calls, ms, kernel_name, name)
    out = {"workload": name, "kernel": kernel_name, "calls": calls, "region_ms": ms, "avg_launch_us": roof["avg_launch_us"],
           "value": calls * leg.set_bytes / (ms * 1e-3) / 1e9, "achieved": roof["achieved"], "frac": roof["frac"],
           "frac_of_nominal_8000": roof["frac_of_nominal_8000"], "traffic": roof["traffic"],
           "in_place_trv_allreduce_us": us_ip, "parity_spot_check": parity,
           "clocks": sampler.report("sampled during the timed region")}
    leg.free()
    return out


def _e2e(torch, binding, leg, dev, steps, world):
    """End to end through trv_allreduce_host: pinned host vectors in, pinned host vectors out (in place on the host),
    every step; plus the rate of plain pinned copies of the same bytes in both directions at once, as the ceiling."""
    import psutil
    w, n = leg.w, leg.w.n
    count = w.count
    budget = int(psutil.virtual_memory().available * 0.5 / max(1, world))
    if n * count * 4 > budget:          # a node too small to pin the whole set per GPU: a prefix of the columns
        count = max(4096, budget // (4 * n) // 4096 * 4096)
    sets = 1 if n * count * 4 >= 2**30 else min(leg.batch, 4)
    host = [torch.empty((n, count), dtype=leg.tdt, pin_memory=True) for _ in range(sets)]
    for b in range(sets):
        host[b].copy_(leg.ins[b][:, :count])
    ptrs = [binding.ptr_array([host[b][r].data_ptr() for r in range(n)]) for b in range(sets)]
    wsb = leg.plan.host_workspace_bytes(count)
    ws = torch.empty(wsb, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()

    def step(_):
        for b in range(sets):
            leg.plan.allreduce_host(ptrs[b], None, count, leg.dcode, ws.data_ptr(), wsb, stream.cuda_stream)

    step(0)                                     # first call: from the inputs; checked against the device path
    torch.cuda.synchronize()
    ok = None
    if count == w.count:
        ok = True
        for r0 in range(0, n, 27):
            up = host[0][r0:r0 + 27].to(dev, non_blocking=True)
            ok = ok and bool(torch.equal(up.view(torch.int32), leg.outs[0][r0:r0 + 27].view(torch.int32)))
    step(0)
    steps = max(1, min(steps, 10 if sets > 1 else 5))
    ms = _timed(torch, stream, step, steps)
    nbytes = sets * n * count * 4
    # ceiling: the same bytes up and down at once as plain copies between pinned memory and the device
    chunk = min(n, max(1, (128 << 20) // (count * 4)))
    dbuf = [torch.empty((chunk, count), dtype=leg.tdt, device=dev) for _ in range(2)]
    s_up, s_dn = torch.cuda.Stream(), torch.cuda.Stream()

    def copies(_):
        s_up.wait_stream(stream)
        s_dn.wait_stream(stream)
        for b in range(sets):
            for r0 in range(0, n, chunk):
                r1 = min(n, r0 + chunk)
                with torch.cuda.stream(s_up):
                    dbuf[0][:r1 - r0].copy_(host[b][r0:r1], non_blocking=True)
                with torch.cuda.stream(s_dn):
                    host[b][r0:r1].copy_(dbuf[1][:r1 - r0], non_blocking=True)
        stream.wait_stream(s_up)
        stream.wait_stream(s_dn)

    copies(0)
    ms_copy = _timed(torch, stream, copies, 2) / 2
    return {"value": world * steps * nbytes / (ms * 1e-3) / 1e9, "unit": "GB/s", "h2d_bytes_per_step": nbytes,
            "d2h_bytes_per_step": nbytes, "steps": steps, "ms_per_step": ms / steps,
            "call": "trv_allreduce_host, in place on pinned host vectors (%d set%s of %d x %d elements), element-range "
                    "windows pipelined inside the call" % (sets, "" if sets == 1 else "s", n, count),
            "matches_device_path": ok,
            "pinned_copy_ceiling": {"value": nbytes / (ms_copy * 1e-3) / 1e9, "unit": "GB/s",
                                    "what": "the same bytes host->device and device->host at once, plain copies of 128 MiB"},
            "frac_of_ceiling": (steps * nbytes / ms) / (nbytes / ms_copy)}


def run_ours(args, w):
    import torch
    from paper_2602_17254_b200 import binding, build
    build.build()
    binding.lib()                                       # fails loudly if the CUDA library is missing
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (there is no CPU fallback for the product path)")
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1 or "TORCHELASTIC_RUN_ID" in os.environ:       # launched by torchrun: one rank per GPU over NCCL
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    kfam = {"auto": binding.KERNEL_AUTO, "step": binding.KERNEL_STEP, "fused": binding.KERNEL_FUSED,
            "pipelined": binding.KERNEL_PIPELINED}[args.kernel]
    leg = Leg(torch, binding, w, dev, rank, args.batch, kfam)
    n, count, batch, set_bytes = w.n, w.count, leg.batch, leg.set_bytes
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    for b in range(batch):
        leg.call(b)
    cps = _calls_per_step(torch, stream, leg, args.steps, args.profile or args.graph or args.batch)
    if dist is not None:        # every rank runs the same number of calls
        t = torch.tensor([cps], dtype=torch.int64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        cps = int(t[0])

    def step():
        for i in range(cps):
            leg.call(i % batch)

    for _ in range(args.warmup):
        step()
    barrier()
    kernel_name = binding.last_kernel_name()
    launches_per_step = None
    if args.graph:      # one step captured once, replayed: removes the per-call host cost (launch-bound sizes)
        l_before = binding.launch_count()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            saved, leg.stream = leg.stream, torch.cuda.current_stream().cuda_stream     # the capturing stream
            step()
            leg.stream = saved
        launches_per_step = binding.launch_count() - l_before
        step = graph.replay
        for _ in range(args.warmup):
            step()
        barrier()
    sampler = ClockSampler(local)
    l0 = binding.launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler.start()
    ev0.record(stream)
    for _ in range(args.steps):
        step()
    ev1.record(stream)
    barrier()
    sampler.stop()
    launches = binding.launch_count() - l0
    if launches_per_step is not None:
        launches = launches_per_step * args.steps       # replayed launches are not seen by the library's counter
    ms = ev0.elapsed_time(ev1)

    parity = leg.parity() if rank == 0 and not args.no_check else None
    e2e = None
    if not args.no_e2e:             # before the in-place leg: it compares with the outputs of the timed calls
        e2e = _e2e(torch, binding, leg, dev, args.steps, world)
    in_place_us = None
    if not args.profile:
        in_place_us = _timed_in_place(torch, stream, leg, max(batch, min(200, (args.steps * cps) // 2)))
    barrier()

    # max over ranks, sums over ranks
    t = torch.tensor([ms, e2e["ms_per_step"] if e2e else 0.0], dtype=torch.float64, device=dev)
    cnt = torch.tensor([float(launches)], dtype=torch.float64, device=dev)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(cnt, op=dist.ReduceOp.SUM)
    ms = float(t[0])
    if e2e:
        e2e["value"] *= e2e["ms_per_step"] / float(t[1])
        e2e["ms_per_step"] = float(t[1])
    launches_all = int(cnt[0])
    leg.free()

    if rank == 0:
        calls = args.steps * cps
        out = {
            "metric": "allreduce_effective_GBps", "value": world * calls * set_bytes / (ms * 1e-3) / 1e9, "unit": "GB/s",
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "int32" if w.dist == "int32" else "f32", "data": "synthetic",
            "config": {"workload": w.name, "dims": list(w.dims), "variant": "latency" if w.variant == 0 else "bandwidth",
                       "ranks": n, "bytes_per_rank": w.bytes_per_rank, "calls_per_step": cps, "buffer_sets": batch,
                       "l2": "consecutive calls run on %d distinct buffer set%s; one pass over them reads %.0f MiB and writes "
                             "%.0f MiB (L2 is 126 MiB): inputs larger than L2, no flush"
                             % (batch, "" if batch == 1 else "s", batch * set_bytes / 2**20, batch * set_bytes / 2**20),
                       "timed_region_ms": ms, "kernel": kernel_name,
                       "call": "trv_allreduce_ex, separate output buffers, TRV_KERNEL_%s" % args.kernel.upper()
                       + (", one step captured in a CUDA graph and replayed" if args.graph else ""),
                       "parallelism": "replicas" if world > 1 else "single GPU"},
            "roofline": _roofline(set_bytes, launches, calls, ms, kernel_name, w.name),
            "e2e": e2e if e2e else {"value": None, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": launches_all,
            "clocks": sampler.report("sampled during the timed region"),
            "parity_spot_check": parity,
            "in_place_trv_allreduce_us": in_place_us,
        }
        if world == 1 and not args.no_side and not args.profile:
            out["per_workload"] = [_side_leg(torch, binding, name, dev, local, args.steps, kfam)
                                   for name in PER_WORKLOAD if name != w.name]
        if not args.no_cpu and world == 1:
            out["cpu_baseline"] = cpu_baseline(w)
        elif not args.no_cpu:
            out["cpu_baseline"] = None
        print(json.dumps(out))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(synth.CONFIGS))
    ap.add_argument("--batch", type=int, default=0, help="buffer sets per step (default: enough to exceed 4x L2)")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline leg")
    ap.add_argument("--no-check", action="store_true", help="skip the parity spot check")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end leg")
    ap.add_argument("--no-side", action="store_true", help="skip the per_workload legs of the other configurations")
    ap.add_argument("--dims", default="", help="ad-hoc torus sides, e.g. 27,27 (overrides the workload's topology)")
    ap.add_argument("--variant", default="latency", choices=["latency", "bandwidth"], help="form for --dims")
    ap.add_argument("--kernel", default="auto", choices=["auto", "step", "fused", "pipelined"],
                    help="kernel family (step = one launch per schedule step, as the paper states the steps; "
                         "pipelined = chunk-level readiness engine, latency form only)")
    ap.add_argument("--graph", action="store_true", help="capture one step in a CUDA graph and time its replays")
    ap.add_argument("--count", type=int, default=0, help="override the workload's elements per rank")
    ap.add_argument("--profile", action="store_true",
                    help="for runs under ncu: only warm-up and timed launches (implies --no-cpu --no-check --no-e2e)")
    args = ap.parse_args()
    if args.profile:
        args.no_cpu = args.no_check = args.no_e2e = args.no_side = True
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    w = synth.CONFIGS[args.workload]
    if args.dims or args.count or args.workload != DEFAULT_WORKLOAD or args.kernel != "auto" or args.graph:
        args.no_side = True         # per_workload belongs to the default run only
    if args.dims:       # ad-hoc topology: same recipe (float32 N(0,1)), for shapes outside the named configurations
        dims = tuple(int(v) for v in args.dims.split(","))
        variant = synth.LATENCY if args.variant == "latency" else synth.BANDWIDTH
        w = synth.Workload("adhoc_%s_%s" % ("x".join(map(str, dims)), args.variant), dims, variant, w.count, "normal", 9)
    if args.count:      # same topology and form, shorter vectors (small cases for ncu captures)
        w = synth.Workload(w.name + "@%d" % args.count, w.dims, w.variant, args.count, w.dist, w.seed)
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
