#!/usr/bin/env python
"""Benchmark of the ZVC codec hot path on B200: one JSON line on stdout.

A step is one pass of the whole hot path over one activation map: compress
(load, mask, scan, look-back, compaction, table) then decompress (table read,
staging, mask walk, expansion).  The default workload is the VGG-16
conv1_2-shaped fp32 map (64x64x224x224, 822 MB, per-channel Beta(2,4)
densities); other workloads can be chosen with --workload for the results
table.  Inputs are synthetic and seeded; they are larger than L2 so every step
streams from HBM.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl cdma|reference]
                  [--workload NAME]

N > 1 is launched under torchrun, one rank per GPU.  The codec has no exchange
step: every rank compresses its own tensor (weak scaling, no collective on the
data path).

--impl reference times the CPU oracle (the plain C checker) on the host cores,
on bounded samples of the same workload.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "zvc_compress_decompress_uncompressed_GBps"
UNIT = "GB/s"
FALLBACK_HBM_GBS = 6650.0
BASE_SEED_RELU = 170501626 + 6000
NOMINAL_HBM_GBS = 8000.0

# DRAM bytes per launch measured by ncu (dram__bytes_read.sum + dram__bytes_write.sum, one
# pass, one launch of each kernel) on the workloads the default line reports, at their full
# size; the captures are summarised under profiles/dram_bytes_bench_workloads.md.  Reads
# equal the algorithmic read bytes; writes fall short of the algorithmic figure by what is
# still in the write-back L2 when the kernel ends.
NCU_DRAM_BYTES = {("config2", "compress"): 1060200704, ("config2", "decompress"): 1052529152,
                  ("config5a", "compress"): 2312471808, ("config5a", "decompress"): 2263166464,
                  ("config5c", "compress"): 1465721600, ("config5c", "decompress"): 1408377600}
KERNEL_NAMES = {(4, "compress"): "zvc_compress_kernel", (4, "decompress"): "zvc_decompress_kernel",
                (2, "compress"): "zvc_compress_rows_kernel", (2, "decompress"): "zvc_decompress_groups_kernel",
                (1, "compress"): "zvc_compress_rows_kernel", (1, "decompress"): "zvc_decompress_groups_kernel"}


def env_int(name, default):
    try:
        return int(os.environ.get(name, default))
    except ValueError:
        return default


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# --------------------------------------------------------------------------- #
# workloads
# --------------------------------------------------------------------------- #
def make_workload(name: str, device, rank: int = 0):
    """Returns (tensor, description).  Rank r > 0 draws a different seed."""
    import torch
    from paper_1705_01626_b200 import workloads as wl
    bump = 7919 * rank
    if name == "config1":
        return wl.alexnet_conv1(seed=wl.seed_for(1) + bump, device=device), \
            "config1: fp32 NCHW 32x96x55x55, i.i.d. density 0.5"
    if name == "config2":
        return wl.per_channel_beta(seed=wl.seed_for(2) + bump, device=device), \
            "config2: fp32 NCHW 64x64x224x224 (VGG-16 conv1_2), per-channel Beta(2,4) density"
    if name in ("config5a", "config5b", "config5c"):
        which = name[-1]
        x = wl.large_extremes(which, device=device, seed=wl.seed_for(5, "abc".index(which)) + bump)
        return x, {"a": "config5a: fp32 2^29 elements, i.i.d. density 0.05",
                   "b": "config5b: fp32 2^29 elements, all non-zero",
                   "c": "config5c: fp16 2^29 elements, i.i.d. density 0.3"}[which]
    if name.startswith("config3."):
        i = int(name.split(".")[1])
        c, h, w = wl.VGG16_CONV_SHAPES[i]
        d = 0.5 - 0.4 * i / 12
        return wl.correlated_relu((64, c, h, w), d, wl.seed_for(3, i) + bump, device), \
            "config3 tensor %d: fp32 NCHW 64x%dx%dx%d, clustered zeros, density %.3f" % (i, c, h, w, d)
    if name.startswith("iid:"):
        # iid:<elements>:<density>[:f16|:u8] -- free-size case for profiling and sweeps
        parts = name.split(":")
        cnt, d = int(parts[1]), float(parts[2])
        kind = parts[3] if len(parts) > 3 else "f32"
        if kind == "u8":
            # one-byte elements (an 8-bit float or integer type): non-zero bytes 1..255, zeros i.i.d.
            g = torch.Generator(device=device).manual_seed(wl.seed_for(9) + bump)
            v = torch.randint(1, 256, (cnt,), generator=g, device=device, dtype=torch.int16).to(torch.uint8)
            keep = torch.rand(cnt, generator=g, device=device) < d
            return v * keep, "iid: 1-byte elements, %d elements, i.i.d. density %g" % (cnt, d)
        dt = torch.float16 if kind == "f16" else torch.float32
        return wl.iid_relu_like((cnt,), d, wl.seed_for(9) + bump, device, dtype=dt, floor=2.0 ** -10), \
            "iid: %s %d elements, i.i.d. density %g" % ("fp16" if dt == torch.float16 else "fp32", cnt, d)
    raise SystemExit("unknown workload %r" % name)


# --------------------------------------------------------------------------- #
# clock sampling during the timed region (read-only NVML queries)
# --------------------------------------------------------------------------- #
class ClockSampler:
    REASONS = {
        0x0000000000000004: "sw_power_cap",
        0x0000000000000008: "hw_slowdown",
        0x0000000000000020: "sw_thermal_slowdown",
        0x0000000000000040: "hw_thermal_slowdown",
        0x0000000000000080: "hw_power_brake_slowdown",
    }

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self._h = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._h = None

    def _run(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                bits = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
                for bit, name in self.REASONS.items():
                    if bits & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(0.005)

    def start(self):
        if self._h is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        return {
            "sm_mhz": statistics.median(self.samples) if self.samples else None,
            "sm_max_mhz": self.max_mhz,
            "reasons": sorted(self.reasons),
            "samples": len(self.samples),
        }


# --------------------------------------------------------------------------- #
# CPU oracle timing (cpu_baseline leg and --impl reference)
# --------------------------------------------------------------------------- #
def host_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


class OracleRunner:
    """Times the C oracle's compress and decompress on one sample with buffers
    allocated (and touched) beforehand, so only the two C calls are timed."""

    def __init__(self, sample, threads: int):
        import numpy as np
        from oracle import zvc_c
        self.zvc_c, self.sample, self.threads = zvc_c, sample, threads
        n, s = sample.size, sample.dtype.itemsize
        self.dst = np.zeros(4 * ((n + 31) // 32) + s * n, dtype=np.uint8)
        self.table = np.zeros(zvc_c.table_entries(n), dtype=np.uint64)
        self.out = np.zeros(n, dtype=sample.dtype)
        self.checked = False

    def round_trip(self):
        """Returns (compress seconds, decompress seconds, payload bytes)."""
        t0 = time.perf_counter()
        c = self.zvc_c.compress_into(self.sample, self.dst, self.table, self.threads)
        t1 = time.perf_counter()
        r = self.zvc_c.decompress_into(self.dst[:max(c, 0)], self.table, self.out, self.threads)
        t2 = time.perf_counter()
        if c < 0 or r != self.sample.nbytes:
            raise SystemExit("oracle failed: %d %d" % (c, r))
        if not self.checked:
            assert self.out.tobytes() == self.sample.tobytes()
            self.checked = True
        return t1 - t0, t2 - t1, c


def time_oracle_round_trip(sample, threads: int):
    return OracleRunner(sample, threads).round_trip()


def oracle_sample_elems(host_flat, threads: int, target_seconds: float) -> int:
    """Pick a sample size (multiple of 1024 elements) costing about target_seconds."""
    probe = min(host_flat.size, 4 << 20)
    tc, td, _ = time_oracle_round_trip(host_flat[:probe], threads)
    rate = probe / max(tc + td, 1e-9)
    n = int(rate * target_seconds) // 1024 * 1024
    return max(1024, min(n, host_flat.size // 1024 * 1024 or host_flat.size))


def cpu_baseline(host_flat, target_seconds: float = 12.0):
    """The C oracle on all host cores over a bounded sample, repeated until
    about target_seconds of CPU wall time have been spent."""
    threads = host_cores()
    n = oracle_sample_elems(host_flat, threads, target_seconds)
    sample = host_flat[:n]
    runner = OracleRunner(sample, threads)
    runner.round_trip()                      # untimed: touches every buffer once
    tc = td = 0.0
    reps = 0
    while reps < 1 or (tc + td < target_seconds and reps < 200):
        a, b, c = runner.round_trip()
        tc, td, reps = tc + a, td + b, reps + 1
    total = sample.nbytes * reps
    one = OracleRunner(sample[: min(n, 8 << 20)], 1)
    one.round_trip()
    a1, b1, _ = one.round_trip()
    return {
        "value": total / (tc + td) / 1e9,
        "unit": UNIT,
        "cores": threads,
        "kind": "oracle",
        "sample": "first %d elements (%.1f MB) of the same tensor, %d round trips, compress %.2f s + "
                  "decompress %.2f s in total, chunk-parallel driver over the byte-wise C oracle"
                  % (n, sample.nbytes / 1e6, reps, tc, td),
        "compress_GBps": total / tc / 1e9,
        "decompress_GBps": total / td / 1e9,
        "single_thread_GBps": one.sample.nbytes / (a1 + b1) / 1e9,
    }


def run_reference(args):
    """--impl reference: the CPU oracle as it stands, on bounded samples."""
    rank = env_int("RANK", 0)
    if rank != 0:
        return
    import torch
    x, desc = make_workload(args.workload, "cpu") if args.workload == "config1" else (None, None)
    if x is None:
        # generate a bounded slice of the workload's recipe on the CPU: the first
        # images of the batch (same per-channel statistics), enough for the samples
        from paper_1705_01626_b200 import workloads as wl
        if args.workload == "config2":
            x = wl.per_channel_beta(shape=(8, 64, 224, 224), device="cpu")
            desc = "config2: fp32 NCHW 64x64x224x224 (VGG-16 conv1_2), per-channel Beta(2,4) density"
        else:
            x, desc = make_workload(args.workload, "cpu")
    host = x.contiguous().view(-1).numpy()
    threads = host_cores()
    budget = 150.0 / max(1, args.steps + args.warmup)
    n = oracle_sample_elems(host, threads, min(budget, 15.0))
    sample = host[:n]
    runner = OracleRunner(sample, threads)
    for _ in range(args.warmup):
        runner.round_trip()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        runner.round_trip()
    dt = time.perf_counter() - t0
    value = sample.nbytes * args.steps / dt / 1e9
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u32",
        "data": "synthetic", "config": {"workload": desc},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                         "sample": "each step = first %d elements (%.1f MB) of the workload's recipe" %
                                   (n, sample.nbytes / 1e6)},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------- #
# the CUDA arm
# --------------------------------------------------------------------------- #
def dtype_code(B, x):
    import torch
    return {torch.float32: B.F32, torch.float16: B.F16, torch.bfloat16: B.BF16, torch.uint8: B.U8}[x.dtype]


def raw_view(x):
    import torch
    return x.view(-1).view({4: torch.int32, 2: torch.int16, 1: torch.uint8}[x.element_size()])


def measure_codec(B, x, steps, warmup, repeats, world=1, dev=None, sampler=None):
    """Parity on these very buffers, then `repeats` timed loops of exactly `steps` steps (a step = one
    compress + one decompress of x, device resident) whose only extra work is the event pair the library
    records around each kernel; call-level times (host side of the call + kernel) come from one more pass
    with events around the calls instead.  Returns sizes, the per-repeat loop times, the per-kernel times of
    every timed step, the per-call times, and the launches counted in the timed loops."""
    import torch
    import torch.distributed as dist
    dev = dev or x.device
    n, s = x.numel(), x.element_size()
    code = dtype_code(B, x)
    dense_bytes = n * s
    cap = B.cdma_zvc_max_compressed_bytes(n, code)
    entries = B.cdma_zvc_table_entries(n)
    ws_bytes = B.cdma_zvc_workspace_bytes(n, code)
    payload = torch.empty(cap, dtype=torch.uint8, device=dev)
    table = torch.empty(entries, dtype=torch.int64, device=dev)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    out = torch.empty_like(x)
    res = torch.zeros(2, dtype=torch.int64).pin_memory()
    stream = torch.cuda.current_stream()
    sh = stream.cuda_stream

    def compress():
        st = B.cdma_zvc_compress_async(x.data_ptr(), n, code, B.NCHW, payload.data_ptr(), cap,
                                       table.data_ptr(), ws.data_ptr(), ws_bytes, sh, res.data_ptr())
        if st != B.OK:
            raise B.CdmaError(st, "cdma_zvc_compress_async")

    def decompress(c):
        st = B.cdma_zvc_decompress_async(payload.data_ptr(), c, table.data_ptr(), n, code, B.NCHW,
                                         out.data_ptr(), ws.data_ptr(), ws_bytes, sh, res.data_ptr())
        if st != B.OK:
            raise B.CdmaError(st, "cdma_zvc_decompress_async")

    # ---- correctness on these very buffers before any timing ----------------
    nnz = int(torch.count_nonzero(raw_view(x)))
    c_bytes = B.cdma_zvc_compress(x.data_ptr(), n, code, B.NCHW, payload.data_ptr(), cap, table.data_ptr(),
                                  ws.data_ptr(), ws_bytes, sh)
    if c_bytes != 4 * ((n + 31) // 32) + s * nnz:
        raise SystemExit("compressed size %d differs from 4*ceil(n/32)+s*nnz" % c_bytes)
    r = B.cdma_zvc_decompress(payload.data_ptr(), c_bytes, table.data_ptr(), n, code, B.NCHW, out.data_ptr(),
                              ws.data_ptr(), ws_bytes, sh)
    if r != dense_bytes or not torch.equal(raw_view(out), raw_view(x)):
        raise SystemExit("round trip is not bit-exact")

    # ---- device-resident timing --------------------------------------------
    K = steps
    for _ in range(max(warmup, 3)):
        compress()
        decompress(c_bytes)
    torch.cuda.synchronize()
    loops, tc, td = [], [], []
    launches = 0
    for rep in range(repeats):
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
        # event pairs recorded by the library around each kernel alone
        kev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(K)]
        for row in kev:
            for e in row:
                e.record(stream)                     # creates the underlying cudaEvent_t
        torch.cuda.synchronize()
        launches0 = B.cdma_kernel_launch_count()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        if sampler is not None and rep == 0:
            sampler.start()
        ev[0].record(stream)
        for i in range(K):
            B.cdma_time_next_kernel(kev[i][0].cuda_event, kev[i][1].cuda_event)
            compress()
            B.cdma_time_next_kernel(kev[i][2].cuda_event, kev[i][3].cuda_event)
            decompress(c_bytes)
        ev[1].record(stream)
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        launches = B.cdma_kernel_launch_count() - launches0
        total_ms = ev[0].elapsed_time(ev[1])
        if world > 1:
            t = torch.tensor([total_ms], dtype=torch.float64, device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            total_ms = float(t.item())
        loops.append(total_ms)
        tc += [kev[i][0].elapsed_time(kev[i][1]) for i in range(K)]
        td += [kev[i][2].elapsed_time(kev[i][3]) for i in range(K)]
        if int(res[1]) != 0:
            raise SystemExit("device reported status %d during timing" % int(res[1]))
    # ---- call level (host side of the call + kernel), in a pass of its own after the timed loops:
    # events around every call, none inside it
    Kc = min(K, 50)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2 * Kc + 1)]
    torch.cuda.synchronize()
    ev[0].record(stream)
    for i in range(Kc):
        compress()
        ev[2 * i + 1].record(stream)
        decompress(c_bytes)
        ev[2 * i + 2].record(stream)
    torch.cuda.synchronize()
    tc_call = [ev[2 * i].elapsed_time(ev[2 * i + 1]) for i in range(Kc)]
    td_call = [ev[2 * i + 1].elapsed_time(ev[2 * i + 2]) for i in range(Kc)]
    return {"n": n, "s": s, "dense_bytes": dense_bytes, "c_bytes": c_bytes, "table_bytes": 8 * entries, "nnz": nnz,
            "loops_ms": loops, "tc": tc, "td": td, "tc_call": tc_call, "td_call": td_call, "launches": launches}


def kernel_roofline(workload, direction, m, peak, peak_kind):
    """Roofline record of one kernel: algorithmic bytes per launch over its mean launch time."""
    algo_bytes = m["dense_bytes"] + m["c_bytes"] + m["table_bytes"]      # per launch, either direction
    times = m["tc"] if direction == "compress" else m["td"]
    calls = m["tc_call"] if direction == "compress" else m["td_call"]
    ms = statistics.mean(times)
    ach = algo_bytes / (ms * 1e-3) / 1e9
    traffic = NCU_DRAM_BYTES.get((workload, direction))
    return {"kernel": KERNEL_NAMES[(m["s"], direction)], "bound": "hbm", "achieved": ach, "peak": peak,
            "unit": "GB/s", "frac": ach / peak, "peak_kind": "of " + peak_kind,
            "frac_of_nominal_8TBps": ach / NOMINAL_HBM_GBS,
            "traffic": traffic,
            "traffic_note": ("ncu dram__bytes_read.sum + dram__bytes_write.sum of one launch at this size; "
                             "see profiles/dram_bytes_bench_workloads.md") if traffic else
                            "not captured for this workload",
            "frac_dram": (traffic / (ms * 1e-3) / 1e9 / peak) if traffic else None,
            "algorithmic_bytes": algo_bytes, "mean_launch_ms": ms, "median_launch_ms": statistics.median(times),
            "mean_call_ms": statistics.mean(calls),
            "uncompressed_GBps": m["dense_bytes"] / (ms * 1e-3) / 1e9}


def run_cdma(args):
    import torch
    import torch.distributed as dist
    from paper_1705_01626_b200 import binding as B

    world = env_int("WORLD_SIZE", 1)
    rank = env_int("RANK", 0)
    local = env_int("LOCAL_RANK", 0)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the codec has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    x, desc = make_workload(args.workload, dev, rank)
    x = x.contiguous()
    n, s = x.numel(), x.element_size()
    K, W = args.steps, max(args.warmup, 3)
    sampler = ClockSampler(local)
    m = measure_codec(B, x, K, W, args.repeats, world, dev, sampler)
    clocks = sampler.stop()
    dense_bytes, c_bytes, table_bytes, nnz = m["dense_bytes"], m["c_bytes"], m["table_bytes"], m["nnz"]
    total_ms = statistics.median(m["loops_ms"])          # the median repeat of exactly K steps

    # ---- end to end with host buffers (copies inside the timed region) ------
    e2e = None
    offload = None
    if not args.no_e2e:
        e2e, offload = run_e2e(B, x, dtype_code(B, x), c_bytes, args, world, dev)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peak()
    rc = kernel_roofline(args.workload, "compress", m, peak, peak_kind)
    rd = kernel_roofline(args.workload, "decompress", m, peak, peak_kind)
    dominant = rc if rc["mean_launch_ms"] >= rd["mean_launch_ms"] else rd
    line = {
        "metric": METRIC,
        "value": world * dense_bytes * K / (total_ms * 1e-3) / 1e9,
        "unit": UNIT,
        "n_gpus": world,
        "steps": K,
        "warmup": W,
        "ms_per_step": total_ms / K,
        "higher_is_better": True,
        "scaling": "weak",
        "vs_baseline": None,
        "dtype": {4: "u32", 2: "u16", 1: "u8"}[s],
        "data": "synthetic",
        "config": {"workload": desc, "elements": n, "dense_bytes": dense_bytes,
                   "compressed_bytes": c_bytes, "table_bytes": table_bytes,
                   "density": nnz / n, "ratio_payload": dense_bytes / c_bytes,
                   "ratio_with_table": dense_bytes / (c_bytes + table_bytes),
                   "l2": "inputs larger than L2 (no flush needed)" if dense_bytes > 2 * 126e6
                         else "input fits in L2: warm-cache figure",
                   "parallelism": "replicas x%d, no collective" % world,
                   "repeats": "%d timed loops of %d steps each; value and ms_per_step are the median loop"
                              % (args.repeats, K),
                   "loops_ms_per_step": [t / K for t in m["loops_ms"]]},
        "roofline": dominant,
        "kernels": {"compress": rc, "decompress": rd},
        "clocks": clocks,
        "gpu_launches": int(m["launches"]),
        "e2e": e2e,
        "offload": offload,
    }
    host = None
    if not args.no_cpu_baseline and world == 1:
        host = x.view(-1)[: min(n, 1 << 28)].cpu().numpy()
    del x
    torch.cuda.empty_cache()
    if not args.no_other_configs and world == 1 and args.workload == "config2":
        # the cases furthest from the roofline ride along in the same record: the sparse 2 GiB tensor
        # and the 2-byte tensor of workload 5 (fewer steps; same parity check first)
        other = {}
        for name in ("config5a", "config5c"):
            y, ydesc = make_workload(name, dev, rank)
            mo = measure_codec(B, y.contiguous(), max(4, K // 4), 3, 3)
            other[name] = {"workload": ydesc, "ratio_payload": mo["dense_bytes"] / mo["c_bytes"],
                           "ms_per_step": statistics.median(mo["loops_ms"]) / max(4, K // 4),
                           "compress": kernel_roofline(name, "compress", mo, peak, peak_kind),
                           "decompress": kernel_roofline(name, "decompress", mo, peak, peak_kind)}
            del y
            torch.cuda.empty_cache()
        line["other_configs"] = other
    if host is not None:
        line["cpu_baseline"] = cpu_baseline(host)
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_e2e(B, x, code, c_bytes, args, world, dev):
    """The same round trip through the host-buffer entry points: dense tensor in
    pinned host memory -> device -> compress -> payload in pinned host memory,
    and back.  Also the natural offload/prefetch path (dense stays on the device,
    only compressed bytes cross the link) against a plain pinned copy."""
    import torch
    import torch.distributed as dist
    n, s = x.numel(), x.element_size()
    dense_bytes = n * s
    cap = B.cdma_zvc_max_compressed_bytes(n, code)
    entries = B.cdma_zvc_table_entries(n)
    staging = 2 * (cap + 8 * entries + B.cdma_zvc_workspace_bytes(n, code) + 4096)
    ctx = B.cdma_ctx_create(cap + 8 * entries + 4096, staging)
    h_x = torch.empty(x.shape, dtype=x.dtype).pin_memory()
    h_x.copy_(x)
    h_y = torch.empty(x.shape, dtype=x.dtype).pin_memory()
    h_p = torch.empty(cap, dtype=torch.uint8).pin_memory()
    h_t = torch.empty(entries, dtype=torch.int64).pin_memory()
    steps = max(1, min(args.steps, args.e2e_steps))

    def one():
        c = B.cdma_zvc_compress_host(ctx, h_x.data_ptr(), n, code, B.NCHW, h_p.data_ptr(), cap, h_t.data_ptr())
        if c != c_bytes:
            raise SystemExit("host-buffer compress returned %d, expected %d" % (c, c_bytes))
        r = B.cdma_zvc_decompress_host(ctx, h_p.data_ptr(), c, h_t.data_ptr(), n, code, B.NCHW, h_y.data_ptr())
        if r != dense_bytes:
            raise SystemExit("host-buffer decompress returned %d" % r)

    one()
    itype = {4: torch.int32, 2: torch.int16, 1: torch.uint8}[s]
    if not torch.equal(h_y.view(-1).view(itype), h_x.view(-1).view(itype)):
        raise SystemExit("host-buffer round trip is not bit-exact")
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    t0 = time.perf_counter()
    for _ in range(steps):
        one()
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    if world > 1:
        t = torch.tensor([dt], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dt = float(t.item())
    e2e = {"value": world * dense_bytes * steps / dt / 1e9, "unit": UNIT,
           "h2d_bytes_per_step": dense_bytes + c_bytes + 8 * entries,
           "d2h_bytes_per_step": dense_bytes + c_bytes + 8 * entries,
           "steps": steps, "ms_per_step": 1e3 * dt / steps,
           "path": "cdma_zvc_compress_host + cdma_zvc_decompress_host on pinned host buffers"}

    # natural path: OFF then PRE of the device tensor; only compressed bytes cross the link
    stream = torch.cuda.current_stream()
    out = torch.empty_like(x)

    def off_pre():
        c, t = B.cdma_offload(ctx, x.data_ptr(), n, code, B.NCHW, stream.cuda_stream)
        if c != c_bytes:
            raise SystemExit("cdma_offload returned %d" % c)
        r = B.cdma_prefetch(ctx, t, out.data_ptr(), stream.cuda_stream)
        if r != dense_bytes:
            raise SystemExit("cdma_prefetch returned %d" % r)

    off_pre()
    if not torch.equal(out.view(-1).view(itype), x.view(-1).view(itype)):
        raise SystemExit("offload/prefetch round trip is not bit-exact")
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(steps):
        off_pre()
    B.cdma_ctx_synchronize(ctx)
    torch.cuda.synchronize()
    dt_off = (time.perf_counter() - t0) / steps

    # the uncompressed copy the compressed one replaces (pinned, both directions)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(steps):
        h_y.copy_(x, non_blocking=True)
        torch.cuda.synchronize()
        out.copy_(h_y, non_blocking=True)
        torch.cuda.synchronize()
    dt_raw = (time.perf_counter() - t0) / steps
    offload = {
        "offload_prefetch_GBps": dense_bytes / dt_off / 1e9,
        "plain_copy_round_trip_GBps": dense_bytes / dt_raw / 1e9,
        "speedup_over_plain_copy": dt_raw / dt_off,
        "pcie_round_trip_GBps_per_direction": 2 * dense_bytes / dt_raw / 1e9,
        "link_bytes_per_step": 2 * (c_bytes + 8 * entries),
        "note": "cdma_offload + cdma_prefetch per step vs pinned cudaMemcpy D2H + H2D of the dense tensor",
    }
    B.cdma_ctx_destroy(ctx)
    return e2e, offload


# --------------------------------------------------------------------------- #
# results-table workloads (not the default line): offload set and layout sweep
# --------------------------------------------------------------------------- #
def time_codec(B, x, code, iters=10, codec="zvc"):
    """Device-timed compress and decompress of one tensor: (C, ms_compress, ms_decompress).
    codec: "zvc" (the paper's zero-value compression) or "rle" (the run-length comparison codec)."""
    comp, comp_async = (B.cdma_zvc_compress, B.cdma_zvc_compress_async) if codec == "zvc" else \
        (B.cdma_rle_compress, B.cdma_rle_compress_async)
    dec, dec_async = (B.cdma_zvc_decompress, B.cdma_zvc_decompress_async) if codec == "zvc" else \
        (B.cdma_rle_decompress, B.cdma_rle_decompress_async)
    import torch
    n = x.numel()
    cap = B.cdma_zvc_max_compressed_bytes(n, code)
    entries = B.cdma_zvc_table_entries(n)
    ws_bytes = B.cdma_zvc_workspace_bytes(n, code)
    payload = torch.empty(cap, dtype=torch.uint8, device=x.device)
    table = torch.empty(entries, dtype=torch.int64, device=x.device)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=x.device)
    out = torch.empty_like(x)
    res = torch.zeros(2, dtype=torch.int64).pin_memory()
    sh = torch.cuda.current_stream().cuda_stream
    c = comp(x.data_ptr(), n, code, B.NCHW, payload.data_ptr(), cap, table.data_ptr(),
                            ws.data_ptr(), ws_bytes, sh)
    if c < 0:
        raise B.CdmaError(c, "compress")
    r = dec(payload.data_ptr(), c, table.data_ptr(), n, code, B.NCHW, out.data_ptr(),
                              ws.data_ptr(), ws_bytes, sh)
    it = torch.int32 if x.element_size() == 4 else torch.int16
    if r < 0 or not torch.equal(out.view(-1).view(it), x.view(-1).view(it)):
        raise SystemExit("round trip failed")
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2 * iters + 1)]
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=x.device)
    tc = td = 0.0
    for i in range(iters + 3):
        flush.fill_(i & 0xFF)                      # tensors smaller than L2 are measured cold
        a, b, cc = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        a.record()
        comp_async(x.data_ptr(), n, code, B.NCHW, payload.data_ptr(), cap, table.data_ptr(),
                                  ws.data_ptr(), ws_bytes, sh, res.data_ptr())
        b.record()
        flush.fill_((i + 1) & 0xFF)
        d0 = torch.cuda.Event(enable_timing=True)
        d0.record()
        dec_async(payload.data_ptr(), c, table.data_ptr(), n, code, B.NCHW, out.data_ptr(),
                                    ws.data_ptr(), ws_bytes, sh, res.data_ptr())
        cc.record()
        torch.cuda.synchronize()
        if i >= 3:
            tc += a.elapsed_time(b)
            td += d0.elapsed_time(cc)
    return c, tc / iters, td / iters


def run_sweep(args):
    """config4: ratio and GB/s per (density, layout); tensors (103 MB) are measured with a cold L2.
    Each point also goes through the run-length comparison codec (Section VI-A, Fig. 11: zero-value
    compression gives the same ratio in every layout, run-length encoding does not)."""
    import torch
    from paper_1705_01626_b200 import binding as B
    from paper_1705_01626_b200 import workloads as wl
    torch.cuda.set_device(0)
    peak, kind = measured_peak()
    for d, layout, x in wl.layout_density_sweep(device="cuda"):
        c, tc, td = time_codec(B, x, B.F32)
        rc, rtc, rtd = time_codec(B, x, B.F32, codec="rle")
        dense = x.numel() * 4
        algo = dense + c + 8 * B.cdma_zvc_table_entries(x.numel())
        ralgo = dense + rc + 8 * B.cdma_zvc_table_entries(x.numel())
        # Section VI-A also looks at compression blocks of up to 64 KB: the zero-value stream has no
        # per-block header, so the block size changes nothing but the size of the offset table kept
        # beside it (one 8-byte entry per block)
        blocks = {"%d KB" % kb: dense / (c + 8 * (dense // (kb << 10) + 1)) for kb in (4, 16, 64)}
        print(json.dumps({"workload": "config4", "density": d, "layout": layout, "dense_bytes": dense,
                          "compressed_bytes": c, "ratio": dense / c, "ratio_with_table_by_block": blocks,
                          "compress_GBps": dense / tc / 1e6, "decompress_GBps": dense / td / 1e6,
                          "compress_frac_of_" + kind: algo / tc / 1e6 / peak,
                          "decompress_frac_of_" + kind: algo / td / 1e6 / peak,
                          "rle": {"compressed_bytes": rc, "ratio": dense / rc,
                                  "compress_GBps": dense / rtc / 1e6, "decompress_GBps": dense / rtd / 1e6,
                                  "compress_frac_of_" + kind: ralgo / rtc / 1e6 / peak,
                                  "decompress_frac_of_" + kind: ralgo / rtd / 1e6 / peak},
                          "l2": "flushed between calls"}),
              flush=True)


def run_offload_set(args):
    """config3: OFF of all 13 conv outputs (compress || D2H), then PRE in reverse (H2D || decompress),
    against the same schedule with plain pinned copies."""
    import torch
    from paper_1705_01626_b200 import binding as B
    from paper_1705_01626_b200 import workloads as wl
    torch.cuda.set_device(0)
    tensors = [t for t, _ in wl.vgg16_offload_set(device="cuda")]
    total = sum(t.numel() * 4 for t in tensors)
    worst = max(B.cdma_zvc_max_compressed_bytes(t.numel(), B.F32) + 8 * B.cdma_zvc_table_entries(t.numel())
                + B.cdma_zvc_workspace_bytes(t.numel(), B.F32) + 4096 for t in tensors)
    pinned = sum(B.cdma_zvc_max_compressed_bytes(t.numel(), B.F32) // 2 + 8 * B.cdma_zvc_table_entries(t.numel())
                 + 4096 for t in tensors) + worst      # the direct mode reserves one worst case while it runs
    ctx = B.cdma_ctx_create(pinned, 2 * worst)
    stream = torch.cuda.current_stream()
    outs = [torch.empty_like(t) for t in tensors]
    per_tensor = []

    def cycle():
        tickets, sizes = [], []
        t0 = time.perf_counter()
        for t in tensors:
            c, tk = B.cdma_offload(ctx, t.data_ptr(), t.numel(), B.F32, B.NCHW, stream.cuda_stream)
            if c < 0:
                raise B.CdmaError(c, "cdma_offload")
            tickets.append(tk)
            sizes.append(c)
        if B.cdma_ctx_synchronize(ctx) != 0:
            raise SystemExit("offload failed")
        t1 = time.perf_counter()
        for i in reversed(range(len(tensors))):
            st = B.cdma_prefetch_async(ctx, tickets[i], outs[i].data_ptr(), stream.cuda_stream)
            if st != 0:
                raise B.CdmaError(st, "cdma_prefetch_async")
        if B.cdma_ctx_synchronize(ctx) != 0:
            raise SystemExit("prefetch failed")
        torch.cuda.synchronize()
        t2 = time.perf_counter()
        return t1 - t0, t2 - t1, sizes

    _, _, sizes = cycle()
    for t, o in zip(tensors, outs):
        if not torch.equal(o.view(-1).view(torch.int32), t.view(-1).view(torch.int32)):
            raise SystemExit("offload set round trip is not bit-exact")
    offs, pres = [], []
    for _ in range(3):
        a, b, _ = cycle()
        offs.append(a)
        pres.append(b)

    def cycle_direct():
        """The kernels store into / load from the pinned pool themselves (no staging, no second copy)."""
        tickets = []
        t0 = time.perf_counter()
        for t in tensors:
            c, tk = B.cdma_offload_direct(ctx, t.data_ptr(), t.numel(), B.F32, B.NCHW, stream.cuda_stream)
            if c < 0:
                raise B.CdmaError(c, "cdma_offload_direct")
            tickets.append(tk)
        torch.cuda.synchronize()
        t1 = time.perf_counter()
        for i in reversed(range(len(tensors))):
            r = B.cdma_prefetch_direct(ctx, tickets[i], outs[i].data_ptr(), stream.cuda_stream)
            if r < 0:
                raise B.CdmaError(r, "cdma_prefetch_direct")
        torch.cuda.synchronize()
        t2 = time.perf_counter()
        return t1 - t0, t2 - t1

    for o in outs:
        o.zero_()
    cycle_direct()
    for t, o in zip(tensors, outs):
        if not torch.equal(o.view(-1).view(torch.int32), t.view(-1).view(torch.int32)):
            raise SystemExit("direct offload set round trip is not bit-exact")
    doffs, dpres = [], []
    for _ in range(3):
        a, b = cycle_direct()
        doffs.append(a)
        dpres.append(b)
    hosts = [torch.empty(t.shape, dtype=t.dtype).pin_memory() for t in tensors]
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for t, h in zip(tensors, hosts):
        h.copy_(t, non_blocking=True)
    torch.cuda.synchronize()
    t1 = time.perf_counter()
    for o, h in zip(reversed(outs), reversed(hosts)):
        o.copy_(h, non_blocking=True)
    torch.cuda.synchronize()
    t2 = time.perf_counter()
    for t, c in zip(tensors, sizes):
        per_tensor.append({"shape": list(t.shape), "ratio": t.numel() * 4 / c})
    csum = sum(sizes)
    print(json.dumps({
        "workload": "config3: 13 VGG-16-shaped conv outputs, batch 64, fp32 NCHW, clustered zeros",
        "dense_bytes": total, "compressed_bytes": csum, "ratio_size_weighted": total / csum,
        "ratio_max": max(p["ratio"] for p in per_tensor), "per_tensor": per_tensor,
        "offload_GBps": total / min(offs) / 1e9, "prefetch_GBps": total / min(pres) / 1e9,
        "offload_direct_GBps": total / min(doffs) / 1e9, "prefetch_direct_GBps": total / min(dpres) / 1e9,
        "plain_d2h_GBps": total / (t1 - t0) / 1e9, "plain_h2d_GBps": total / (t2 - t1) / 1e9,
        "offload_speedup": (t1 - t0) / min(offs), "prefetch_speedup": (t2 - t1) / min(pres),
        "paper_context": "paper: 2.6x average / 13.8x maximum ratio, 32 % average training speedup "
                         "(Titan X, PCIe gen3, hybrid measurement + model)"}), flush=True)
    B.cdma_ctx_destroy(ctx)


def run_relu(args):
    """ReLU + compression in one pass against ReLU (torch) followed by compression, on a
    pre-activation tensor of the bench workload's shape whose ReLU has about the same density."""
    import torch
    from paper_1705_01626_b200 import binding as B
    torch.cuda.set_device(0)
    g = torch.Generator(device="cuda").manual_seed(BASE_SEED_RELU)
    x = torch.empty(64, 64, 224, 224, device="cuda")
    for b in range(64):
        x[b] = torch.randn(64, 224, 224, generator=g, device="cuda") - 0.47
    n = x.numel()
    cap = B.cdma_zvc_max_compressed_bytes(n, B.F32)
    entries = B.cdma_zvc_table_entries(n)
    ws_bytes = B.cdma_zvc_workspace_bytes(n, B.F32)
    payload = torch.empty(cap, dtype=torch.uint8, device="cuda")
    payload2 = torch.empty(cap, dtype=torch.uint8, device="cuda")
    table = torch.empty(entries, dtype=torch.int64, device="cuda")
    table2 = torch.empty(entries, dtype=torch.int64, device="cuda")
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    y = torch.empty_like(x)
    y2 = torch.empty_like(x)
    res = torch.zeros(2, dtype=torch.int64).pin_memory()
    sh = torch.cuda.current_stream().cuda_stream

    def separate():
        torch.clamp_min(x, 0.0, out=y)
        B.cdma_zvc_compress_async(y.data_ptr(), n, B.F32, B.NCHW, payload.data_ptr(), cap, table.data_ptr(),
                                  ws.data_ptr(), ws_bytes, sh, res.data_ptr())

    def fused(with_dense):
        B.cdma_zvc_relu_compress_async(x.data_ptr(), n, B.F32, B.NCHW, y2.data_ptr() if with_dense else 0,
                                       payload2.data_ptr(), cap, table2.data_ptr(), ws.data_ptr(), ws_bytes, sh,
                                       res.data_ptr())

    separate()
    torch.cuda.synchronize()
    c = int(res[0])
    fused(True)
    torch.cuda.synchronize()
    if int(res[0]) != c or not torch.equal(payload[:c], payload2[:c]) or not torch.equal(table, table2) \
            or not torch.equal(y.view(torch.int32), y2.view(torch.int32)):
        raise SystemExit("fused ReLU+compress differs from ReLU then compress")

    def timed(fn, iters=30):
        for _ in range(3):
            fn()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(iters):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / iters

    t_sep = timed(separate)
    t_fd = timed(lambda: fused(True))
    t_f = timed(lambda: fused(False))
    dense = n * 4
    peak, kind = measured_peak()

    # backward pass: the gradient gated by the masks of the compressed map, against rebuilding y and
    # running the framework's backward kernel over y and dy
    dy = torch.randn_like(x)
    dx = torch.empty_like(x)
    dx2 = torch.empty_like(x)

    def bwd_separate():
        B.cdma_zvc_decompress_async(payload.data_ptr(), c, table.data_ptr(), n, B.F32, B.NCHW, y.data_ptr(),
                                    ws.data_ptr(), ws_bytes, sh, res.data_ptr())
        torch.ops.aten.threshold_backward.grad_input(dy, y, 0.0, grad_input=dx)

    def bwd_fused():
        B.cdma_zvc_relu_backward_async(payload.data_ptr(), c, table.data_ptr(), n, B.F32, B.NCHW, dy.data_ptr(),
                                       dx2.data_ptr(), ws.data_ptr(), ws_bytes, sh, res.data_ptr())

    bwd_separate()
    bwd_fused()
    torch.cuda.synchronize()
    if not torch.equal(dx.view(torch.int32), dx2.view(torch.int32)):
        raise SystemExit("backward from the masks differs from decompress + threshold_backward")
    t_bs = timed(bwd_separate)
    t_bf = timed(bwd_fused)
    print(json.dumps({
        "workload": "relu: fp32 64x64x224x224 pre-activations N(-0.47,1), ReLU density %.3f" % ((c - 4 * (n // 32)) / 4 / n),
        "dense_bytes": dense, "compressed_bytes": c,
        "relu_then_compress_ms": t_sep, "fused_with_dense_output_ms": t_fd, "fused_payload_only_ms": t_f,
        "speedup_fused_with_dense": t_sep / t_fd, "speedup_payload_only": t_sep / t_f,
        "algorithmic_bytes": {"relu_then_compress": 3 * dense + c, "fused_with_dense": 2 * dense + c,
                              "fused_payload_only": dense + c},
        "frac_of_" + kind: {"relu_then_compress": (3 * dense + c) / t_sep / 1e6 / peak,
                            "fused_with_dense": (2 * dense + c) / t_fd / 1e6 / peak,
                            "fused_payload_only": (dense + c) / t_f / 1e6 / peak},
        "backward": {"decompress_then_threshold_backward_ms": t_bs, "from_masks_ms": t_bf,
                     "speedup": t_bs / t_bf,
                     "algorithmic_bytes": {"decompress_then_threshold_backward": 4 * dense + c,
                                           "from_masks": 2 * dense + c},
                     "frac_of_" + kind: {"decompress_then_threshold_backward": (4 * dense + c) / t_bs / 1e6 / peak,
                                         "from_masks": (2 * dense + c) / t_bf / 1e6 / peak}}}), flush=True)


def run_timeline(args):
    """Training-step estimate of Section VI's model, fed with numbers measured on this GPU: forward and
    backward time of the 13 conv layers of a VGG-16-shaped CNN (batch 64, torch's convolution, used for
    timing only), the codec's time and ratio on each layer's synthetic activation map (the config3 set),
    and the pinned-copy rates of the host link."""
    import torch
    import torch.nn.functional as F
    from paper_1705_01626_b200 import binding as B
    from paper_1705_01626_b200 import timeline as tl
    from paper_1705_01626_b200 import workloads as wl
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    batch = 64
    g = torch.Generator(device="cuda").manual_seed(BASE_SEED_RELU + 1)

    def timed(fn, iters=5):
        for _ in range(2):
            fn()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(iters):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / iters * 1e-3

    # host link, pinned, 1 GiB each way
    hbuf = torch.empty(1 << 30, dtype=torch.uint8).pin_memory()
    dbuf = torch.empty(1 << 30, dtype=torch.uint8, device=dev)
    d2h = (1 << 30) / timed(lambda: hbuf.copy_(dbuf, non_blocking=True)) / 1e9
    h2d = (1 << 30) / timed(lambda: dbuf.copy_(hbuf, non_blocking=True)) / 1e9
    del hbuf, dbuf
    link = min(d2h, h2d)

    rows, plain, packed = [], [], []
    cin = 3
    prev = None                        # (bytes, ratio, compress_s, decompress_s) of the map feeding this layer
    for i, (cout, h, w) in enumerate(wl.VGG16_CONV_SHAPES):
        x = torch.randn(batch, cin, h, w, generator=g, device=dev).requires_grad_(True)
        wt = (torch.randn(cout, cin, 3, 3, generator=g, device=dev) * 0.05).requires_grad_(True)
        gy = torch.randn(batch, cout, h, w, generator=g, device=dev)
        fwd = timed(lambda: F.relu(F.conv2d(x, wt, padding=1)))
        y = F.relu(F.conv2d(x, wt, padding=1))
        bwd = timed(lambda: torch.autograd.grad(y, (x, wt), gy, retain_graph=True))
        del y, gy, wt
        # the map saved for this layer's backward pass: the input images for the first layer, else the
        # previous conv + ReLU output (before any pooling, as in the config3 set)
        if prev is None:
            act_bytes, ratio, t_c, t_d = batch * cin * h * w * 4, 1.0, 0.0, 0.0
        else:
            act_bytes, ratio, t_c, t_d = prev[:4]
        del x
        rows.append({"layer": i, "fwd_ms": fwd * 1e3, "bwd_ms": bwd * 1e3, "input_map_MB": act_bytes / 1e6,
                     "ratio": ratio, "plain_copy_ms": act_bytes / (link * 1e9) * 1e3,
                     "compressed_copy_ms": act_bytes / ratio / (link * 1e9) * 1e3,
                     "compress_ms": t_c * 1e3, "decompress_ms": t_d * 1e3})
        plain.append(tl.Layer(fwd, bwd, act_bytes, 1.0))
        packed.append((fwd, bwd, act_bytes, ratio, t_c, t_d))
        # this layer's output map: synthetic stand-in with the config3 recipe, through the codec
        d = 0.5 - 0.4 * i / (len(wl.VGG16_CONV_SHAPES) - 1)
        a = wl.correlated_relu((batch, cout, h, w), d, wl.seed_for(3, i), dev)
        c, ms_c, ms_d = time_codec(B, a, B.F32, iters=5)
        nbytes = a.numel() * 4
        prev = (nbytes, nbytes / (c + 8 * B.cdma_zvc_table_entries(a.numel())), ms_c * 1e-3, ms_d * 1e-3)
        del a
        cin = cout
        torch.cuda.empty_cache()
    # software codec: compression runs on the GPU in front of the copy (added to the layer that produces the
    # copy's overlap window), decompression of the map a layer below needs runs beside the layer above it
    cdma = []
    for i, (fwd, bwd, act_bytes, ratio, t_c, t_d) in enumerate(packed):
        t_d_above = packed[i - 1][5] if i > 0 else 0.0
        cdma.append(tl.Layer(fwd + t_c, bwd + t_d_above, act_bytes, ratio))

    def both(pcie, dram):
        sp = tl.summary(plain, pcie)
        sc = tl.summary(cdma, pcie, dram)
        return {"pcie_GBps": pcie, "oracle_ms": sp["oracle_s"] * 1e3, "vdnn_ms": sp["vdnn_s"] * 1e3,
                "cdma_ms": sc["cdma_s"] * 1e3, "vdnn_vs_oracle": sp["vdnn_vs_oracle"],
                "cdma_vs_oracle": sp["oracle_s"] / sc["cdma_s"],
                "cdma_speedup_over_vdnn": sp["vdnn_s"] / sc["cdma_s"],
                "traffic_reduction": sc["traffic_reduction"], "max_comp_bw_GBps": sc["max_comp_bw_gbs"]}

    peak, _ = measured_peak()
    print(json.dumps({
        "workload": "timeline: 13 conv layers of a VGG-16-shaped CNN, batch 64, fp32 tensors (TF32 convolutions), "
                    "config3 activation maps",
        "model": "Section VI: copy time = bytes / ratio / PCIe x max(1, ratio x PCIe / DRAM_BW); "
                 "a layer stalls when its copy outlasts it",
        "link": {"d2h_GBps": d2h, "h2d_GBps": h2d},
        "layers": rows,
        "this_box": both(link, peak),
        "same_layers_on_a_16_GBps_link": both(16.0, peak),
        "paper_context": "paper (Titan X, PCIe gen3, six CNNs): vDNN loses 31 % on average, compressed copies win "
                         "back 32 % on average (61 % at most)",
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="cdma", choices=["cdma", "reference"])
    ap.add_argument("--workload", default="config2")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-other-configs", action="store_true")
    ap.add_argument("--repeats", type=int, default=10)
    args = ap.parse_args()
    if args.steps < 1:
        raise SystemExit("--steps must be >= 1")
    if args.impl == "reference":
        run_reference(args)
    elif args.workload == "config3":
        run_offload_set(args)
    elif args.workload == "config4":
        run_sweep(args)
    elif args.workload == "relu":
        run_relu(args)
    elif args.workload == "timeline":
        run_timeline(args)
    else:
        run_cdma(args)


if __name__ == "__main__":
    main()
