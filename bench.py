#!/usr/bin/env python
"""Benchmark of the Trivance AllReduce hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

One "step" is one pass of the hot path over a batch of independent synthetic buffer sets of the
chosen workload: for every set one trv_allreduce_ex call (plan built once, outside the timed
region).  The batch is sized so that the sets of one step exceed several times the L2 capacity:
every call reads cold data from HBM.  Metric: effective AllReduce GB/s = n * S_bytes / t, where
S_bytes is the per-rank vector size.  Rank 0 prints ONE JSON line.

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

DEFAULT_WORKLOAD = "ring27_lat_2MiB"
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
                "samples": len(self.samples), "note": note}


# ------------------------------------------------------------------ GPU legs

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

    n, count = w.n, w.count
    set_bytes = n * count * 4
    batch = args.batch or max(1, min(64, max(16, -(-4 * L2_BYTES // set_bytes)), (24 * 2**30) // set_bytes))   # >= 4x L2 per step
    tdt = torch.int32 if w.dist == "int32" else torch.float32
    dcode = binding.INT32 if w.dist == "int32" else binding.FLOAT32
    plan = binding.Plan(w.dims, w.variant)

    # synthetic inputs: set 0 is the workload's seeded vectors (and feeds the parity spot check);
    # the other sets are the same recipe with other seeds (rank- and set-specific)
    x0 = synth.workload_inputs(w) if set_bytes <= 2**31 else None
    ins = torch.empty((batch, n, count), dtype=tdt, device=dev)
    outs = torch.empty((batch, n, count), dtype=tdt, device=dev)
    if x0 is not None:
        ins[0].copy_(torch.from_numpy(x0))
        g = torch.Generator(device=dev)
        g.manual_seed(1000 * w.seed + rank)
        for b in range(1, batch):
            if w.dist == "int32":
                ins[b].copy_(torch.randint(-1000, 1001, (n, count), generator=g, device=dev, dtype=tdt))
            elif w.dist == "normal":
                ins[b].normal_(generator=g)
            else:
                ins[b].uniform_(-1.0, 1.0, generator=g)
    else:   # multi-GiB sets: drawn on the device (values do not influence the run time)
        g = torch.Generator(device=dev)
        g.manual_seed(1000 * w.seed + rank)
        for b in range(batch):
            ins[b].normal_(generator=g) if w.dist == "normal" else ins[b].uniform_(-1.0, 1.0, generator=g)
    in_ptrs = [binding.ptr_array([ins[b, r].data_ptr() for r in range(n)]) for b in range(batch)]
    out_ptrs = [binding.ptr_array([outs[b, r].data_ptr() for r in range(n)]) for b in range(batch)]
    kfam = {"auto": binding.KERNEL_AUTO, "step": binding.KERNEL_STEP, "fused": binding.KERNEL_FUSED,
            "pipelined": binding.KERNEL_PIPELINED}[args.kernel]
    need = plan.scratch_bytes(count, kfam, in_place=False)
    scratch = torch.empty(max(need, 256), dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()
    sh = stream.cuda_stream

    def step():
        for b in range(batch):
            plan.allreduce_ex(in_ptrs[b], out_ptrs[b], count, dcode, kernel=kfam,
                              scratch_ptr=scratch.data_ptr() if need else 0, scratch_bytes=need,
                              stream=torch.cuda.current_stream().cuda_stream)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    kernel_name = binding.last_kernel_name()
    launches_per_step = None
    if args.graph:      # one step captured once, replayed: removes the per-call host cost (launch-bound sizes)
        l_before = binding.launch_count()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            step()
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
    launches = binding.launch_count() - l0
    if launches_per_step is not None:
        launches = launches_per_step * args.steps       # replayed launches are not seen by the library's counter
    ms = ev0.elapsed_time(ev1)
    note = "sampled during the timed region"
    if len(sampler.samples) < 8 and not args.profile:        # region too short for NVML: keep the same load running ~0.4 s more
        t_end = time.perf_counter() + 0.4
        while time.perf_counter() < t_end:
            step()
            torch.cuda.synchronize()
        note = "timed region (%.1f ms) plus 0.4 s of the same load right after it" % ms
    sampler.stop()

    # parity spot check of what was just timed: set 0's output against the oracle on a window
    parity = None
    if rank == 0 and x0 is not None and not args.no_check:
        import oracle
        w1 = min(count, 4096)
        want = oracle.allreduce(w.dims, w.variant, np.ascontiguousarray(x0[:, :w1]), E=count, e0=0)
        got = outs[0, :, :w1].cpu().numpy()
        parity = bool(np.array_equal(got.view(np.uint32), want.view(np.uint32)))

    # end to end through the host-buffer entry point: pinned host inputs -> device -> host outputs,
    # two streams so that one set's upload overlaps the previous set's download
    do_e2e = not args.no_e2e and set_bytes <= 4 * 2**30
    e2e_sets = min(batch, 4) if do_e2e else 0
    hin = [torch.empty((n, count), dtype=tdt).pin_memory() for _ in range(e2e_sets)]
    hout = [torch.empty((n, count), dtype=tdt).pin_memory() for _ in range(e2e_sets)]
    for b in range(e2e_sets):
        hin[b].copy_(ins[b])
    wsb = plan.host_workspace_bytes(count)
    ws = [torch.empty(wsb, dtype=torch.uint8, device=dev) for _ in range(2)]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    hin_p = [binding.ptr_array([hin[b][r].data_ptr() for r in range(n)]) for b in range(e2e_sets)]
    hout_p = [binding.ptr_array([hout[b][r].data_ptr() for r in range(n)]) for b in range(e2e_sets)]

    def e2e_step():
        for b in range(e2e_sets):
            plan.allreduce_host(hin_p[b], hout_p[b], count, dcode, ws[b % 2].data_ptr(), wsb, streams[b % 2].cuda_stream)

    e2e_steps = max(1, min(args.steps, 10))
    e2e_ms, e2e_ok = 0.0, None
    if do_e2e:
        for _ in range(2):
            e2e_step()
        barrier()
        e0, e1, eb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True), torch.cuda.Event()
        streams[1].wait_stream(streams[0])
        e0.record(streams[0])
        streams[1].wait_event(e0)
        for _ in range(e2e_steps):
            e2e_step()
        eb.record(streams[1])
        streams[0].wait_event(eb)
        e1.record(streams[0])
        barrier()
        e2e_ms = e0.elapsed_time(e1)
        if parity is not None:
            e2e_ok = bool(torch.equal(hout[0].view(torch.int32), outs[0].cpu().view(torch.int32)))

    # max over ranks, sums over ranks
    t = torch.tensor([ms, e2e_ms], dtype=torch.float64, device=dev)
    cnt = torch.tensor([float(launches)], dtype=torch.float64, device=dev)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(cnt, op=dist.ReduceOp.SUM)
    ms, e2e_ms = float(t[0]), float(t[1])
    launches_all = int(cnt[0])

    if rank == 0:
        calls = args.steps * batch
        value = world * calls * set_bytes / (ms * 1e-3) / 1e9
        per_launch_ms = ms / launches                                          # this rank's launches
        kernels_per_call = launches / calls
        algo_bytes = 2 * set_bytes / kernels_per_call                         # per launch of the dominant kernel
        peak, peak_src = _peak()
        achieved = algo_bytes / (per_launch_ms * 1e-3) / 1e9
        e2e_value = world * e2e_steps * e2e_sets * set_bytes / (e2e_ms * 1e-3) / 1e9 if do_e2e else None
        out = {
            "metric": "allreduce_effective_GBps", "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "int32" if w.dist == "int32" else "f32", "data": "synthetic",
            "config": {"workload": w.name, "dims": list(w.dims), "variant": "latency" if w.variant == 0 else "bandwidth",
                       "ranks": n, "bytes_per_rank": w.bytes_per_rank, "calls_per_step": batch,
                       "l2": "each step touches %d distinct buffer sets = %.0f MiB read + %.0f MiB written (L2 is 126 MiB): "
                             "inputs larger than L2, no flush" % (batch, batch * set_bytes / 2**20, batch * set_bytes / 2**20),
                       "kernel": kernel_name, "call": "trv_allreduce_ex, separate output buffers, TRV_KERNEL_%s" % args.kernel.upper()
                       + (", one step captured in a CUDA graph and replayed" if args.graph else ""),
                       "parallelism": "replicas" if world > 1 else "single GPU"},
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": _traffic(kernel_name, w.name), "peak_source": peak_src,
                         "algorithmic_bytes_per_launch": algo_bytes, "avg_launch_us": per_launch_ms * 1e3,
                         "frac_of_nominal_8000": achieved / 8000.0},
            "e2e": {"value": e2e_value, "unit": "GB/s", "h2d_bytes_per_step": e2e_sets * set_bytes,
                    "d2h_bytes_per_step": e2e_sets * set_bytes, "steps": e2e_steps,
                    "call": "trv_allreduce_host on pinned host buffers, two streams", "matches_device_path": e2e_ok},
            "gpu_launches": launches_all,
            "clocks": sampler.report(note),
            "parity_spot_check": parity,
        }
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
        args.no_cpu = args.no_check = args.no_e2e = True
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    w = synth.CONFIGS[args.workload]
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
