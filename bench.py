#!/usr/bin/env python
"""Benchmark of the fused recurrence scan (one JSON line on stdout).

A "step" is one pass of the whole hot path -- one call of the C ABI on one batch of seeded
synthetic input.  Headline workload: configuration 2 of the benchmark contract (16384 rows x 2048
steps, fp32, log-space inputs of a linear-RNN layer), the configuration the metric is quoted on.
`value` is elements/s with the inputs resident in HBM; `e2e` is the same metric through the
host-buffer entry point with pinned host buffers and both copies inside the timed region.

The same line carries, under `workloads`, one record per benchmark configuration measured in the same
process (both kernels: the row-batched one on configurations 2, 4, 5, the look-back one on
configuration 3 and its linear / bf16 variants, the call latency of configuration 1), each with
median / min / mean time per step over repeated batches, the clocks sampled meanwhile, and a
two-legged roofline: algorithmic bytes at the measured HBM copy bandwidth against algorithmic
transcendentals at the MUFU rate that a register-only probe kernel measures in the same run.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 2|3|4|5] [--impl reference]
                  [--only-headline] [--fig1] [--ablation unfused|pairs]

N > 1: one rank per GPU (launched by torchrun, or spawned from here when the torchrun environment is
absent); rows are independent, so every rank runs its own batch (weak scaling) and the only
communication is the barrier and the max-over-ranks of the time.
"""
from __future__ import annotations

import argparse
import ctypes
import json
import os
import socket
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "recurrence_elements_per_s"
UNIT = "elements/s"
ARITHMETIC = "f32"            # every kernel computes in fp32 whatever the storage type
HBM_FALLBACK_GBS = 6650.0     # used only when MEASURED_PEAKS.json is absent
NOMINAL_HBM_GBS = 8000.0      # the figure the benchmark contract quotes for B200
MIN_TIMED_SECONDS = 0.15      # per record: long enough for a few dozen clock samples
MIN_REPEATS = 10


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", type=int, default=2, choices=[2, 3, 4, 5], help="headline workload")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--rows", type=int, default=None, help="override the workload's rows (profiling of small cases)")
    ap.add_argument("--n", type=int, default=None, help="override the workload's n (profiling of small cases)")
    ap.add_argument("--variant", default=None, choices=["linear", "bf16", "complex"],
                    help="with --workload 3: time the linear entry point / bf16 storage on the same sequence; with "
                         "--workload 4: the same signed values as complex logarithms (heinsen_scan_log_complex)")
    ap.add_argument("--only-headline", action="store_true",
                    help="skip the per-configuration records, the MUFU probe, the end-to-end leg and the CPU baselines "
                         "(profiling runs)")
    ap.add_argument("--fig1", action="store_true",
                    help="the paper's only experiment: sequential (CPU oracle, one core) over parallel (this library) "
                         "time for one sequence of n = 2^10..2^28 elements, means of 30 runs; prints one JSON object")
    ap.add_argument("--ablation", default=None, choices=["unfused", "pairs"],
                    help="'unfused': the paper's own recipe (Eq. 7) as separate framework kernels -- torch.cumsum, "
                         "torch.logcumsumexp and elementwise ops, one pass over memory each -- on the same workload; "
                         "'pairs': the linear-domain (alpha, beta) pair scan (no logarithms) beside the log-space "
                         "scan_linear on the signed linear workload (cfg4)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-workloads", action="store_true", help="headline record only (keeps e2e and CPU baseline)")
    return ap.parse_args()


def measured_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return HBM_FALLBACK_GBS, "fallback (no MEASURED_PEAKS.json)"


def ncu_traffic():
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of each workload's kernel, as summarised from the
    ncu captures under profiles/ (absent workload: None)."""
    try:
        with open(os.path.join(ROOT, "profiles", "dram_traffic.json")) as f:
            return json.load(f)
    except Exception:
        return {}


class ClockSampler:
    """Samples SM clock, power and throttle reasons of one GPU through NVML while a timed region runs."""
    REASONS = {
        0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
        0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
        0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting",
    }

    def __init__(self, index: int, period_s: float = 0.003):
        self.samples, self.reasons, self.max_mhz, self.power = [], set(), None, []
        self.period = period_s
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def sample(self):
        if self.nv is None:
            return
        try:
            self.samples.append(int(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM)))
            mask = int(self.nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
            for bit, name in self.REASONS.items():
                if mask & bit and name != "gpu_idle":
                    self.reasons.add(name)
        except Exception:
            pass

    def start(self):
        """One sample now, in the caller's thread; the sampling thread takes its first one a period later (a timed
        region shorter than that is then not disturbed by a second Python thread at all)."""
        def loop():
            while not self._stop.wait(self.period):
                self.sample()
        self.sample()
        self._thread = threading.Thread(target=loop, daemon=True)
        self._thread.start()
        return self

    def stop(self):
        self._stop.set()
        if self._thread:
            self._thread.join()
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2] if s else None, "sm_mhz_min": s[0] if s else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(s)}


# ---------------------------------------------------------------------------------------------- workloads
def describe(cid, w, variant=None):
    call = "scan_linear" if w.kind == "linear" else "scan_log"
    extra = f", variant {variant}" if variant else ""
    return f"cfg{cid}: {w.name} ({w.rows} rows x n={w.n}, {call}, {w.storage} storage{extra})"


def make_workload(cid, variant=None, rows=None, n=None, seed=0):
    """Configuration `cid`, or one of configuration 3's variants: 'linear' = the linear entry point on
    a = fp32(exp(log_a)), b, x0 = 0.5; 'bf16' = the same log-space sequence stored in bf16."""
    from paper_2311_06281_b200 import workloads
    w = workloads.make(cid, rows=rows, n=n, seed=seed)
    if variant == "linear":
        assert cid == 3
        w.kind = "linear"
    elif variant == "bf16":
        assert cid == 3
        for k in ("log_a", "log_b", "log_x0"):
            w.tensors[k] = workloads.to_bf16_bits(w.tensors[k].astype("float64")).reshape(w.tensors[k].shape)
        w.storage = "bf16"
    elif variant == "complex":
        # the signed workload as complex logarithms (log|v|, 0 or pi): the representation the paper names for
        # negative values; the logarithms are taken on the host in float64 (input preparation, not the method)
        import numpy as np
        assert cid == 4
        with np.errstate(divide="ignore"):
            for src, dst in (("a", "log_a"), ("b", "log_b"), ("x0", "log_x0")):
                v = w.tensors.pop(src).astype(np.float64)
                z = np.empty(v.shape, dtype=np.complex64)
                z.real = np.log(np.abs(v))
                z.imag = np.where(v < 0, np.float32(np.pi), np.float32(0))
                w.tensors[dst] = z
        w.kind, w.storage = "log", "c64"
    return w


def input_keys(w):
    return ("a", "b", "x0") if w.kind == "linear" else ("log_a", "log_b", "log_x0")


def mufu_per_element(w):
    """Algorithmic transcendentals per element: scan_log one ex2 for the scan and one lg2 for the output;
    scan_linear two logarithms on the way in, one ex2 for the scan and one for the output."""
    return 4 if w.kind == "linear" else 2


ELEMENT_BYTES = {"f32": 4, "bf16": 2, "c64": 8}


def algorithmic_bytes(w):
    es = ELEMENT_BYTES[w.storage]
    return w.rows * w.n * 3 * es + w.rows * es   # two inputs read once, one output written once, x0


class DeviceWorkload:
    """A workload resident on the device in `nsets` rotating buffer sets, each larger than L2."""

    def __init__(self, w, dev, hs, nsets=3):
        import numpy as np
        import torch
        self.w, self.hs, self.nsets = w, hs, nsets

        def dev_tensor(arr):
            x = torch.from_numpy(np.ascontiguousarray(arr))
            if arr.dtype == np.uint16:
                x = x.view(torch.bfloat16)
            return x.to(dev)

        base = [dev_tensor(w.tensors[k]) for k in input_keys(w)]
        self.sets = [base] + [[x.clone() for x in base] for _ in range(nsets - 1)]
        self.outs = [torch.empty((w.rows, w.n), dtype=base[0].dtype, device=dev) for _ in range(nsets)]
        if w.storage == "c64":
            nbytes = int(hs.lib().heinsen_scan_complex_workspace_bytes(w.rows, w.n))
            self.wss = [torch.empty(nbytes, dtype=torch.uint8, device=dev) for _ in range(nsets)]
        else:
            self.wss = [hs.new_workspace(w.rows, w.n, dev) for _ in range(nsets)]

        # the same calls with their arguments marshalled once: the timed loops then spend about 4 us of host time
        # per step instead of 12, so that a short timed region starts its first kernel early and the clock sampler's
        # thread has little to disturb
        L, vp = hs.lib(), ctypes.c_void_p
        stream = vp(torch.cuda.current_stream(dev).cuda_stream)
        code = {torch.float32: hs.HS_F32, torch.bfloat16: hs.HS_BF16}
        self.calls = []
        for k in range(nsets):
            a, b, x0 = (vp(t.data_ptr()) for t in self.sets[k])
            out, ws, wsn = vp(self.outs[k].data_ptr()), vp(self.wss[k].data_ptr()), self.wss[k].numel()
            if w.storage == "c64":
                self.calls.append((L.heinsen_scan_log_complex, (a, b, x0, out, w.rows, w.n, ws, wsn, stream)))
            elif w.kind == "linear":
                self.calls.append((L.heinsen_scan_linear, (a, b, x0, out, w.rows, w.n, hs.HS_F32, ws, wsn, stream)))
            else:
                dt = code[self.outs[k].dtype]
                self.calls.append((L.heinsen_scan_log, (a, b, x0, out, None, None, None, None, w.rows, w.n, dt, dt, ws, wsn,
                                                        stream)))

    def step(self, i):
        fn, argv = self.calls[i % self.nsets]
        status = fn(*argv)
        if status != 0:
            raise self.hs.HeinsenScanError(status, self.hs.strerror(status))

    def step_through_binding(self, i):
        s, hs = i % self.nsets, self.hs
        if self.w.storage == "c64":
            hs.scan_log_complex(*self.sets[s], log_x=self.outs[s], workspace=self.wss[s])
        elif self.w.kind == "linear":
            hs.scan_linear(*self.sets[s], x=self.outs[s], workspace=self.wss[s])
        else:
            hs.scan_log(*self.sets[s], log_x=self.outs[s], workspace=self.wss[s])

    def check(self):
        for ws in self.wss:
            self.hs.check(ws)


def timed_batches(dw, steps, repeats, local, torch):
    """`repeats` batches of `steps` steps back to back, an event between batches; returns the per-step time of
    every batch (ms) and the clocks sampled meanwhile."""
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(repeats + 1)]
    torch.cuda.synchronize()
    sampler = ClockSampler(local).start()
    k = 0
    ev[0].record()
    for r in range(repeats):
        for _ in range(steps):
            dw.step(k)
            k += 1
        ev[r + 1].record()
    sampler.sample()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    per_step = [ev[r].elapsed_time(ev[r + 1]) / steps for r in range(repeats)]
    return per_step, clocks


def roofline_record(w, us_per_step, clocks, peak, peak_source, mufu_rate, kernel, traffic):
    """Two legs: bytes at the measured HBM bandwidth, transcendentals at the measured MUFU rate at the clock
    sampled during the run; the slower one is the roofline."""
    elements = w.rows * w.n
    alg_bytes = algorithmic_bytes(w)
    t_hbm = alg_bytes / (peak * 1e9) * 1e6
    achieved = alg_bytes / (us_per_step * 1e-6) / 1e9
    rec = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": t_hbm / us_per_step,
           "traffic": traffic, "peak_source": peak_source, "kernel": kernel,
           "algorithmic_bytes_per_launch": alg_bytes, "bytes_per_element": 3 * ELEMENT_BYTES[w.storage],
           "hbm": {"time_us": t_hbm, "frac": t_hbm / us_per_step},
           "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS}
    if mufu_rate and clocks.get("sm_mhz"):
        ops = mufu_per_element(w)
        peak_ops = mufu_rate["results_per_clk_per_sm"] * mufu_rate["sm_count"] * clocks["sm_mhz"] * 1e6
        t_mufu = elements * ops / peak_ops * 1e6
        rec["mufu"] = {"ops_per_element": ops, "peak_ops_per_s": peak_ops, "at_sm_mhz": clocks["sm_mhz"],
                       "time_us": t_mufu, "frac": t_mufu / us_per_step}
        if t_mufu > t_hbm:   # the transcendental leg is the slower one: report against it
            rec.update(bound="mufu", achieved=elements * ops / (us_per_step * 1e-6) / 1e12, peak=peak_ops / 1e12,
                       unit="Tops/s", frac=t_mufu / us_per_step)
    return rec


def stats(values):
    s = sorted(values)
    return {"median": s[len(s) // 2], "min": s[0], "mean": sum(s) / len(s), "max": s[-1]}


def measure_record(cid, variant, dev, local, hs, args, peak, peak_source, mufu_rate, torch):
    """One record of `workloads`: build the configuration, warm up, time repeated batches."""
    w = make_workload(cid, variant)
    dw = DeviceWorkload(w, dev, hs)
    for i in range(max(args.warmup, 3)):
        dw.step(i)
    torch.cuda.synchronize()
    dw.check()
    kernel = "batched_scan_kernel" if hs.last_path() == hs.PATH_BATCHED else "lookback_scan_kernel"
    # a first short batch sizes the run: at least MIN_REPEATS batches and MIN_TIMED_SECONDS of device time
    probe, _ = timed_batches(dw, max(3, min(args.steps, 10)), 1, local, torch)
    steps = max(3, args.steps if cid == 2 else min(args.steps, 100))
    repeats = max(MIN_REPEATS, int(MIN_TIMED_SECONDS / (probe[0] * 1e-3 * steps)) + 1)
    per_step_ms, clocks = timed_batches(dw, steps, repeats, local, torch)
    dw.check()
    st = stats([1e3 * v for v in per_step_ms])
    key = f"cfg{cid}" + (f"_{variant}" if variant else "")
    traffic = ncu_traffic().get(key)
    rec = {"workload": describe(cid, w, variant), "kernel": kernel, "elements_per_s": w.rows * w.n / (st["median"] * 1e-6),
           "us_per_step": st, "repeats": repeats, "steps_per_repeat": steps, "timed_launches": repeats * steps,
           "clocks": clocks, "us_times_sm_ghz": st["median"] * (clocks["sm_mhz"] or 0) * 1e-3,
           "roofline": roofline_record(w, st["median"], clocks, peak, peak_source, mufu_rate, kernel,
                                       traffic["bytes"] if traffic else None)}
    if traffic:
        rec["roofline"]["traffic_source"] = traffic.get("source")
    del dw
    torch.cuda.empty_cache()
    return rec, w


def measure_small_call(dev, hs, torch):
    """Configuration 1 (one sequence of 4096 elements) is bound by the cost of a call, not by bytes: time the
    C ABI itself -- pre-marshalled arguments, no tensor wrapping -- back to back, and one call plus its
    synchronisation."""
    w = make_workload(1)
    t = w.tensors
    a, b, x0 = (torch.from_numpy(t[k]).to(dev) for k in ("a", "b", "x0"))
    x = torch.empty_like(a)
    ws = hs.new_workspace(w.rows, w.n, dev)
    L = hs.lib()
    vp = ctypes.c_void_p
    argv = (vp(a.data_ptr()), vp(b.data_ptr()), vp(x0.data_ptr()), vp(x.data_ptr()), w.rows, w.n, hs.HS_F32,
            vp(ws.data_ptr()), ws.numel(), vp(torch.cuda.current_stream(dev).cuda_stream))
    fn = L.heinsen_scan_linear
    for _ in range(20):
        assert fn(*argv) == 0
    torch.cuda.synchronize()
    runs = []
    for _ in range(10):
        calls = 300
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.perf_counter()
        e0.record()
        for _ in range(calls):
            fn(*argv)
        e1.record()
        host_us = (time.perf_counter() - t0) / calls * 1e6
        torch.cuda.synchronize()
        runs.append((e0.elapsed_time(e1) * 1e3 / calls, host_us))
    lat = []
    for _ in range(30):
        t0 = time.perf_counter()
        fn(*argv)
        torch.cuda.synchronize()
        lat.append((time.perf_counter() - t0) * 1e6)
    hs.check(ws)
    dev_us = stats([r[0] for r in runs])
    return {"workload": describe(1, w), "kernel": "lookback_scan_kernel (one tile)" if hs.last_path() == hs.PATH_LOOKBACK
            else "batched_scan_kernel",
            "us_per_call_back_to_back": dev_us, "host_us_per_call": stats([r[1] for r in runs])["median"],
            "us_call_plus_sync": stats(lat), "calls_per_batch": 300, "batches": 10,
            "elements_per_s": w.rows * w.n / (dev_us["median"] * 1e-6),
            "note": "latency-bound: 48 KB of traffic per call; timed through the C ABI with pre-marshalled arguments"}, w


def cpu_oracle_rate(w, cores, budget_s=2.5, max_elements=1 << 25):
    """The float64 oracle, as it stands, on a bounded sample of workload `w` with `cores` threads."""
    import numpy as np
    from oracle import heinsen_oracle
    heinsen_oracle.build()
    t, keys = w.tensors, input_keys(w)
    if w.rows == 1:
        srows, sn = 1, min(w.n, max_elements if cores > 1 else max_elements // 4)
    else:
        limit = max_elements if cores > 1 else max_elements // 4
        srows, sn = max(1, min(w.rows, limit // w.n)), w.n
    sub = {k: np.ascontiguousarray(t[k][:srows, :sn] if t[k].ndim == 2 else t[k][:srows]) for k in keys}
    threads = cores if srows > 1 else 1
    passes, t0 = 0, time.perf_counter()
    while True:
        if w.kind == "linear":
            heinsen_oracle.scan_linear(sub["a"], sub["b"], sub["x0"], nthreads=threads)
        else:
            heinsen_oracle.scan_log(sub["log_a"], sub["log_b"], sub["log_x0"], nthreads=threads)
        passes += 1
        dt = time.perf_counter() - t0
        if dt > budget_s or passes >= 8:
            break
    return {"value": srows * sn * passes / dt, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"{passes} passes over {srows} rows x n={sn} of the workload "
                      f"({'whole batch' if srows * sn == w.rows * w.n else 'first rows / first elements'}), float64 sequential "
                      f"loop" + (", OpenMP over rows" if threads > 1 else ", one core (the paper's sequential computation)")}


# ---------------------------------------------------------------------------------------------- reference arm
def run_reference(args):
    """Times the float64 CPU oracle, as it stands, on a bounded sample of the same workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import heinsen_oracle
    from paper_2311_06281_b200 import workloads

    cid = args.workload
    full = workloads.CONFIGS[cid]
    # bounded sample: about 2^22 elements per step
    if full["rows"] == 1:
        rows, n = 1, min(full["n"], 1 << 22)
    else:
        rows, n = max(1, min(full["rows"], (1 << 22) // full["n"])), full["n"]
    w = workloads.make(cid, rows=rows, n=n)
    t = w.tensors
    heinsen_oracle.build()
    cores = heinsen_oracle.max_threads() if rows > 1 else 1

    def step():
        if w.kind == "linear":
            heinsen_oracle.scan_linear(t["a"], t["b"], t["x0"], nthreads=cores)
        else:
            heinsen_oracle.scan_log(t["log_a"], t["log_b"], t["log_x0"], nthreads=cores)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t0
    value = rows * n * args.steps / dt
    name = describe(cid, workloads.Workload(**{**full, "tensors": {}}))
    sample = f"{rows} rows x n={n} of {name} per step"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": name, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------------- our arm
def spawn_ranks(args):
    """`--gpus N` without a torchrun environment: start the N ranks from here, the way the contract launches them."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    raise SystemExit(subprocess.call(cmd))


def run_ours(args):
    import numpy as np
    import torch

    from paper_2311_06281_b200 import build_ext, heinsen_scan as hs, sharding

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        spawn_ranks(args)
    rank, world, local = sharding.init_from_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    build_ext.build()
    hs.lib()
    peak, peak_source = measured_peak()
    full = not args.only_headline
    reduced = args.rows is not None or args.n is not None

    # MUFU leg of the roofline: a register-only ex2/lg2 kernel, its rate per clock and SM at the clock sampled meanwhile
    mufu_rate = None
    if full:
        hs.probe_mufu(1024)
        sampler = ClockSampler(local, 0.002).start()
        results, seconds = hs.probe_mufu(1 << 15)
        pc = sampler.stop()
        sms = torch.cuda.get_device_properties(dev).multi_processor_count
        if pc["sm_mhz"]:
            mufu_rate = {"results_per_clk_per_sm": results / seconds / (sms * pc["sm_mhz"] * 1e6), "sm_count": sms,
                         "results_per_s": results / seconds, "probe_seconds": seconds, "probe_clocks": pc,
                         "kernel": "heinsen_scan_probe_mufu: 8 independent ex2/lg2 chains per thread, 64 warps per SM"}

    # ------------------------------------------------------------------ headline: EXACTLY K timed steps
    cid = args.workload
    w = make_workload(cid, args.variant, rows=args.rows, n=args.n, seed=rank)  # weak scaling: every rank its own batch
    rows, n = w.rows, w.n
    dw = DeviceWorkload(w, dev, hs)
    for i in range(max(args.warmup, 3)):
        dw.step(i)
    torch.cuda.synchronize()
    dw.check()
    kernel = "batched_scan_kernel" if hs.last_path() == hs.PATH_BATCHED else "lookback_scan_kernel"

    sampler = ClockSampler(local)
    launches0 = hs.launch_count()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sharding.barrier()
    torch.cuda.synchronize()
    sampler.start()
    start.record()
    for i in range(args.steps):
        dw.step(i)
    stop.record()
    sampler.sample()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    sharding.barrier()
    ms_local = start.elapsed_time(stop)
    ms_total = sharding.max_over_ranks(ms_local, dev)
    launches = hs.launch_count() - launches0
    dw.check()

    elements = rows * n
    ms_per_step = ms_total / args.steps
    value = world * elements / (ms_per_step * 1e-3)
    key = f"cfg{cid}" + (f"_{args.variant}" if args.variant else "")
    traffic = None if reduced else ncu_traffic().get(key)
    roofline = roofline_record(w, 1e3 * ms_local / args.steps, clocks, peak, peak_source, mufu_rate, kernel,
                               traffic["bytes"] if traffic else None)
    if traffic:
        roofline["traffic_source"] = traffic.get("source")
    alg_bytes = algorithmic_bytes(w)

    # ------------------------------------------------------------------ per-configuration records (rank 0 of 1 only)
    records = {}
    cpu_1core = {}
    if full and not args.no_workloads and world == 1 and not reduced:
        # the headline workload again as repeated batches, then the other configurations
        del dw
        torch.cuda.empty_cache()
        for c, variant in ((2, None), (4, None), (4, "complex"), (5, None), (3, None), (3, "linear"), (3, "bf16")):
            rec, wl = measure_record(c, variant, dev, local, hs, args, peak, peak_source, mufu_rate, torch)
            k = f"cfg{c}" + (f"_{variant}" if variant else "")
            if not args.no_cpu_baseline and variant not in ("bf16", "complex"):
                rec["cpu_baseline_1core"] = cpu_oracle_rate(wl, 1, budget_s=1.5)
            records[k] = rec
            del wl
        rec1, w1 = measure_small_call(dev, hs, torch)
        if not args.no_cpu_baseline:
            rec1["cpu_baseline_1core"] = cpu_oracle_rate(w1, 1, budget_s=0.5)
        records["cfg1"] = rec1
        dw = None

    # ------------------------------------------------------------------ end to end: pinned host buffers, H2D + kernel + D2H per step
    e2e = None
    if full and not args.no_e2e:
        t = w.tensors
        keys = input_keys(w)
        host_in = [torch.from_numpy(np.ascontiguousarray(t[k])) for k in keys]
        host_in = [(x.view(torch.bfloat16) if x.dtype == torch.uint16 else x).pin_memory() for x in host_in]
        host_out = torch.empty((rows, n), dtype=host_in[0].dtype).pin_memory()
        scratch = torch.empty(hs.host_scratch_bytes(rows, n, host_in[0].dtype, host_out.dtype, False), dtype=torch.uint8,
                              device=dev)
        host_call = hs.scan_linear_host if w.kind == "linear" else hs.scan_log_host
        e2e_steps = max(3, min(args.steps, 20))
        for _ in range(3):
            host_call(host_in[0], host_in[1], host_in[2], host_out, scratch)
        sharding.barrier()
        torch.cuda.synchronize()
        start.record()
        for _ in range(e2e_steps):
            host_call(host_in[0], host_in[1], host_in[2], host_out, scratch)
        stop.record()
        torch.cuda.synchronize()
        e2e_ms = sharding.max_over_ranks(start.elapsed_time(stop), dev) / e2e_steps
        es = host_in[0].element_size()
        e2e = {"value": world * elements / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": 2 * elements * es + rows * es,
               "d2h_bytes_per_step": elements * host_out.element_size(), "ms_per_step": e2e_ms, "steps": e2e_steps,
               "entry_point": "heinsen_scan_linear_host" if w.kind == "linear" else "heinsen_scan_log_host"}
        del scratch

    cpu_baseline = None
    cpu_baseline_1core = None
    if full and rank == 0 and world == 1 and not args.no_cpu_baseline:
        from oracle import heinsen_oracle
        heinsen_oracle.build()
        cpu_baseline = cpu_oracle_rate(w, heinsen_oracle.max_threads(), budget_s=4.0)
        cpu_baseline_1core = cpu_oracle_rate(w, 1, budget_s=2.0)

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": ARITHMETIC, "data": "synthetic",
            "config": {"workload": describe(cid, w, args.variant) + (" [reduced size]" if reduced else ""), "rows_per_gpu": rows,
                       "n": n, "storage": w.storage,
                       "entry_point": "heinsen_scan_linear" if w.kind == "linear" else "heinsen_scan_log",
                       "l2": f"3 rotating buffer sets of {alg_bytes / 1e6:.0f} MB each (every set exceeds the 126 MB L2)",
                       "parallelism": f"rows sharded, {world} rank(s), no data-path collective"},
            "clocks": clocks, "gpu_launches": launches, "roofline": roofline, "e2e": e2e, "cpu_baseline": cpu_baseline,
            "cpu_baseline_1core": cpu_baseline_1core, "mufu_probe": mufu_rate, "workloads": records or None,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def run_fig1(args):
    """Figure 1 of the paper: time to compute n elements sequentially relative to the parallel evaluation,
    each point the mean of 30 runs.  Sequential = the float64 oracle loop on one host core; parallel =
    heinsen_scan_linear on one B200 with the inputs resident on the device (single sequence, look-back path)."""
    import math

    import numpy as np
    import torch

    from oracle import heinsen_oracle
    from paper_2311_06281_b200 import build_ext, heinsen_scan as hs, workloads

    build_ext.build()
    heinsen_oracle.build()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    points = []
    for e in range(10, 29, 2):
        n = 1 << e
        t = workloads.make(1, rows=1, n=n).tensors
        a, b, x0 = (torch.from_numpy(t[k]).to(dev) for k in ("a", "b", "x0"))
        x = torch.empty_like(a)
        ws = hs.new_workspace(1, n, dev)
        for _ in range(5):
            hs.scan_linear(a, b, x0, x=x, workspace=ws)
        torch.cuda.synchronize()
        gpu = []
        for _ in range(30):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            hs.scan_linear(a, b, x0, x=x, workspace=ws)
            e1.record()
            torch.cuda.synchronize()
            gpu.append(e0.elapsed_time(e1) * 1e-3)
        hs.check(ws)
        reps = 30 if n <= (1 << 24) else 5   # bounded: the largest sizes take ~1 s per sequential run
        cpu = []
        for _ in range(reps):
            t0 = time.perf_counter()
            heinsen_oracle.scan_linear(t["a"], t["b"], t["x0"], nthreads=1)
            cpu.append(time.perf_counter() - t0)
        points.append({"n": n, "sequential_s": float(np.mean(cpu)), "sequential_runs": reps,
                       "parallel_s": float(np.mean(gpu)), "parallel_runs": 30,
                       "ratio": float(np.mean(cpu) / np.mean(gpu)), "n_over_log2n": n / math.log2(n)})
        del a, b, x, ws
    print(json.dumps({"fig1": points, "sequential": "float64 oracle loop, 1 host core", "parallel": "heinsen_scan_linear, 1x B200, "
                      "device-resident inputs, wall time of one call incl. launch"}), flush=True)


def run_unfused(args):
    """Ablation: Eq. 7 literally, as the paper ran it -- a numerical framework's cumulative-sum and
    LogCumSumExp kernels plus elementwise kernels, each a full pass over HBM (not part of the library)."""
    import numpy as np
    import torch

    from oracle import heinsen_oracle
    from paper_2311_06281_b200 import unfused_eq7, workloads

    cid = args.workload
    w = workloads.make(cid, rows=args.rows, n=args.n)
    if w.kind != "log" or w.storage != "f32":
        raise SystemExit("--ablation unfused runs the fp32 log-space workloads (2 or 3)")
    dev = torch.device("cuda", 0)
    t = w.tensors
    la, lb, lx0 = (torch.from_numpy(t[k]).to(dev) for k in ("log_a", "log_b", "log_x0"))

    for _ in range(max(args.warmup, 3)):
        out = unfused_eq7.scan_log_unfused(la, lb, lx0)
    torch.cuda.synchronize()
    torch.cuda.reset_peak_memory_stats()
    base = torch.cuda.memory_allocated()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for _ in range(args.steps):
        out = unfused_eq7.scan_log_unfused(la, lb, lx0)
    stop.record()
    torch.cuda.synchronize()
    ms = start.elapsed_time(stop) / args.steps
    elements = w.rows * w.n
    # accuracy of the literal global form in fp32 against the oracle, on a sample of rows
    rows = list(range(min(w.rows, 64)))
    ref, _ = heinsen_oracle.scan_log(t["log_a"][rows], t["log_b"][rows], t["log_x0"][rows])
    got = out[rows].double().cpu().numpy()
    astar = np.cumsum(t["log_a"][rows].astype(np.float64), axis=1)
    tol = 2e-6 * (1 + np.abs(astar) + np.abs(ref - astar)) + 1e-5
    passes_bytes = unfused_eq7.MIN_BYTES_PER_ELEMENT
    print(json.dumps({
        "ablation": "unfused", "metric": METRIC, "value": elements / (ms * 1e-3), "unit": UNIT, "ms_per_step": ms,
        "steps": args.steps, "config": {"workload": describe(cid, w)},
        "framework_kernels_per_step": unfused_eq7.FRAMEWORK_KERNELS_PER_CALL, "min_bytes_per_element": passes_bytes,
        "achieved_GBs_at_min_bytes": elements * passes_bytes / (ms * 1e-3) / 1e9,
        "extra_device_memory_bytes": int(torch.cuda.max_memory_allocated() - base),
        "max_err_over_tolerance": float(np.max(np.abs(got - ref) / tol)),
    }), flush=True)


def run_pairs(args):
    """Comparison: the linear-domain pair scan (no logarithms) beside the log-space heinsen_scan_linear on the
    same signed linear workload (cfg4 unless --rows/--n say otherwise), three rotating buffer sets."""
    import numpy as np
    import torch

    from oracle import heinsen_oracle
    from paper_2311_06281_b200 import heinsen_scan as hs
    from paper_2311_06281_b200 import workloads

    cid = 4
    w = workloads.make(cid, rows=args.rows, n=args.n)
    dev = torch.device("cuda", 0)
    t = w.tensors
    sets = [[torch.from_numpy(t[k]).to(dev) for k in ("a", "b", "x0")] for _ in range(3)]
    outs = [torch.empty_like(s[0]) for s in sets]
    wss = [hs.new_workspace(w.rows, w.n, dev) for _ in sets]
    elements = w.rows * w.n
    rows = list(range(min(w.rows, 64)))
    ref = heinsen_oracle.scan_linear(t["a"][rows], t["b"][rows], t["x0"][rows])
    result = {}
    for name, fn in (("pairs", hs.scan_linear_pairs), ("log_space", hs.scan_linear)):
        def step(i):
            k = i % 3
            fn(*sets[k], x=outs[k], workspace=wss[k])
        for i in range(max(args.warmup, 3)):
            step(i)
        torch.cuda.synchronize()
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        start.record()
        for i in range(args.steps):
            step(i)
        stop.record()
        torch.cuda.synchronize()
        for ws in wss:
            hs.check(ws)
        ms = start.elapsed_time(stop) / args.steps
        got = outs[0][rows].double().cpu().numpy()
        err = np.abs(got - ref) / (1e-3 * np.abs(ref).max(axis=1, keepdims=True))
        result[name] = {"ms_per_step": ms, "value": elements / (ms * 1e-3), "algorithmic_GBs": elements * 12 / (ms * 1e-3) / 1e9,
                        "max_err_over_tolerance": float(err.max())}
    peak, _ = measured_peak()
    print(json.dumps({
        "ablation": "pairs", "metric": METRIC, "unit": UNIT, "value": result["pairs"]["value"],
        "ms_per_step": result["pairs"]["ms_per_step"], "steps": args.steps,
        "config": {"workload": describe(cid, w)}, "pairs": result["pairs"], "log_space": result["log_space"],
        "frac_of_measured_hbm": {k: v["algorithmic_GBs"] / peak for k, v in result.items()},
    }), flush=True)


def main():
    args = parse_args()
    if args.ablation == "unfused":
        run_unfused(args)
        return
    if args.ablation == "pairs":
        run_pairs(args)
        return
    if args.fig1:
        run_fig1(args)
        return
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
