#!/usr/bin/env python
"""Benchmark of the MXNorm hot path on B200.

One "step" is one `mxnorm_fwd` pass (Algorithm 2: block absmax -> RMS estimate -> E8M0 scales ->
E4M3 codes -> store, scales in the tiled GEMM layout) over one batch of the Llama-3-8B-like
workload: bf16 [16384, 4096] with outlier channels.  The metric is algorithmic HBM GB/s
(bytes in + codes + scales + r~ per launch / time).  The same JSON line carries the roofline
fraction against the measured copy peak, the other kernels of the path (conventional
RMSNorm+cast baseline, plain cast, NVFP4, backward), the end-to-end figure with host buffers,
and the CPU oracle timed on this machine's host cores.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

N > 1 (under torchrun): rows are independent, so every rank runs the same per-GPU batch with no
collective (weak scaling); value = bytes of all ranks / max-over-ranks device time.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2603_13180_b200 import sharding  # noqa: E402
from paper_2603_13180_b200 import workloads as wl  # noqa: E402

WORKLOAD = "C3"
EPS = 1e-5
SETS = 4            # rotating input/output buffer sets: 4 x 203 MB > 126 MB of L2
FALLBACK_HBM_GBS = 6650.0
REPEATS = 5         # the timed region (K launches) is repeated this often; the median repeat is the headline
# dram__bytes_read.sum + dram__bytes_write.sum per mxnorm_fwd launch at [16384, 4096]: the mean over eight consecutive
# launches that rotate over the buffer sets, captured with ncu in steady state (caches not flushed between launches)
NCU_TRAFFIC_BYTES = 202_970_368
NCU_TRAFFIC_KIND = "ncu, mean of 8 consecutive launches rotating over the buffer sets (steady state)"


def algorithmic_bytes(kind: str, T: int, D: int) -> int:
    if kind in ("mx", "rms", "cast"):
        return T * D * 2 + T * D + T * (D // 32) + (0 if kind == "cast" else 4 * T)
    if kind == "nvfp4":
        return T * D * 2 + T * D // 2 + T * (D // 16) + 4 * T
    if kind == "bwd":
        return 3 * T * D * 2 + 4 * T + 2 * D + 4 * D
    raise ValueError(kind)


def workload_name(T: int, D: int) -> str:
    """The same string in both arms (the GPU path and the CPU oracle run the same workload)."""
    return (f"{WORKLOAD}: mxnorm_fwd bf16 [{T},{D}] per GPU (batch 4 x seq 4096, Llama-3-8B hidden), outlier channels, "
            "MXFP8 E4M3 codes + E8M0 scales (B=32) in the 128x4 tiled GEMM layout, p=2")


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "50", "-i", str(self.index)],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            pass
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            parts = [p.strip() for p in r.split(",")]
            if len(parts) != 6:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[2:]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


GATE_CYCLES = 200_000      # about 0.1 ms of a clock-spin kernel in front of a timed region (see time_launches)


def time_launches(fn, n_sets: int, steps: int, warmup: int, stream, gate: bool = True) -> float:
    """Average device milliseconds per call of fn(set_index) over `steps` back-to-back launches.

    After the synchronize the GPU is idle, and an event recorded then is stamped at once while the first timed launch is
    still on its way from the host (some 10 us, which a region of 20 launches of 30 us would carry as +1.5 %).  With
    `gate` a short clock-spin kernel is enqueued first: the host queues the timed launches behind it, and the start event
    is stamped when the first of them can begin."""
    for i in range(warmup):
        fn(i % n_sets)
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    if gate:
        with torch.cuda.stream(stream):
            torch.cuda._sleep(GATE_CYCLES)
    start.record(stream)
    for i in range(steps):
        fn(i % n_sets)
    end.record(stream)
    torch.cuda.synchronize()
    return start.elapsed_time(end) / steps


def time_repeated(fn, n_sets: int, steps: int, warmup: int, stream, repeats: int = REPEATS):
    """`repeats` timed regions of `steps` launches each (one warm-up phase); returns the per-launch milliseconds of every
    repeat, sorted."""
    out = [time_launches(fn, n_sets, steps, warmup if r == 0 else 0, stream) for r in range(repeats)]
    return sorted(out)


REST_S = 0.5        # idle time before a secondary kernel is timed (see time_median)
OTHERS_MIN_STEPS = 100   # launches per timed region of a secondary kernel, at least


def time_median(fn, n_sets: int, steps: int, warmup: int, stream, repeats: int = 3) -> float:
    """Median of `repeats` timed regions, started from a rested GPU like the headline's regions are: on this pool a
    kernel timed a second or more into an uninterrupted load runs up to 8 % slower than in a burst (power management;
    the SM clock samples stay at their maximum), and the copy bandwidth the fractions refer to is a burst figure too."""
    torch.cuda.synchronize()
    time.sleep(REST_S)
    return statistics.median(time_repeated(fn, n_sets, steps, warmup, stream, repeats))


def spread(ms_sorted):
    return {"median": statistics.median(ms_sorted), "min": ms_sorted[0], "max": ms_sorted[-1], "repeats": len(ms_sorted)}


def time_graph_replay(fn, n_sets: int, steps: int, warmup: int, stream) -> float:
    """Like time_launches, but the `steps` launches are captured once into a CUDA graph and the replay is
    timed: kernels of a few microseconds are otherwise limited by the host's launch rate."""
    for i in range(warmup):
        fn(i % n_sets)
    graph = torch.cuda.CUDAGraph()
    torch.cuda.synchronize()
    with torch.cuda.graph(graph, stream=stream):
        for i in range(steps):
            fn(i % n_sets)
    graph.replay()
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    start.record(stream)
    graph.replay()
    end.record(stream)
    torch.cuda.synchronize()
    return start.elapsed_time(end) / steps


def time_small_configs(mx, args, main_stream):
    """Forward kernels on the small parity configs C1 [2048,768] and C2 [16384,2048] (context: C1 is
    launch- and L2-bound, 4.8 MB in all): direct launches ("ms") and the replay of a CUDA graph of the same
    launches ("ms_graph")."""
    stream = torch.cuda.Stream()        # a side stream: the default stream cannot be captured
    stream.wait_stream(main_stream)
    with torch.cuda.stream(stream):
        out = _time_small_configs(mx, args, stream)
    main_stream.wait_stream(stream)
    return out


def _time_small_configs(mx, args, stream):
    out = {}
    L, sh = mx.lib, stream.cuda_stream
    for name in ("C1", "C2"):
        w = wl.CONFIGS[name]
        T, D = w.T, w.D
        x_cpu = wl.make_inputs(w)["x"]
        nbytes = algorithmic_bytes("mx", T, D)
        sets = max(4, min(64, -(-3 * (126 << 20) // nbytes)))
        xs = [x_cpu.cuda() for _ in range(sets)]
        outs = [mx.alloc_outputs(T, D, 32, mx.SCALES_ROWMAJOR) for _ in range(sets)]

        def fwd(i):
            c, s, r = outs[i]
            L.mxnorm_fwd(xs[i].data_ptr(), None, T, D, 32, 2, 0.0, EPS, c.data_ptr(), s.data_ptr(), r.data_ptr(), 0, 0, sh)

        def rms(i):
            c, s, r = outs[i]
            L.rmsnorm_mxfp8_fwd(xs[i].data_ptr(), None, T, D, 32, EPS, c.data_ptr(), s.data_ptr(), r.data_ptr(), 0, 0, sh)

        def cast(i):
            c, s, r = outs[i]
            L.mx_cast(xs[i].data_ptr(), T, D, 32, c.data_ptr(), s.data_ptr(), 0, 0, sh)

        res = {}
        for kname, fn in (("mxnorm_fwd", fwd), ("rmsnorm_mxfp8_fwd", rms), ("mx_cast", cast)):
            ms = time_launches(fn, sets, args.steps, args.warmup, stream)
            ms_graph = time_graph_replay(fn, sets, args.steps, args.warmup, stream)
            res[kname] = {"ms": ms, "gbs": nbytes / ms / 1e6, "tokens_per_s": T / (ms * 1e-3),
                          "ms_graph": ms_graph, "gbs_graph": nbytes / ms_graph / 1e6}
        res["buffer_sets"] = sets
        out[name] = res
        del xs, outs
    return out


def profile_run(mx, xs, outs, T, D, layout, fwd, rms, cast):
    """Three launches of every kernel of the path on the benchmark's tensors (for a profiler capture)."""
    w5 = wl.CONFIGS["C5"]
    inp5 = wl.make_inputs(w5) if T == w5.T else wl.make_inputs(w5, T=T)
    g = inp5["grad"].cuda()
    gain = inp5["gain"].cuda()
    c, s, r = outs[0]
    o4 = mx.alloc_outputs(T, D, 16, mx.SCALES_ROWMAJOR, nvfp4=True)
    m4 = mx.alloc_outputs(T, D, 32, layout, nvfp4=True)
    dx = torch.empty_like(xs[0])
    dgain = torch.empty(D, dtype=torch.float32, device="cuda")
    ws = torch.empty(mx.mxnorm_bwd_workspace_bytes(T, D), dtype=torch.uint8, device="cuda")
    ct = torch.empty((D, T), dtype=torch.uint8, device="cuda")
    st = torch.empty(mx.scale_bytes(D, T // 32, layout), dtype=torch.uint8, device="cuda")
    for i in range(3):
        fwd(i)
        rms(i)
        cast(i)
        mx.mxnorm_nvfp4_fwd(xs[i], o4[0], o4[1], o4[2], eps=EPS)
        mx.mxnorm_mxfp4_fwd(xs[i], m4[0], m4[1], m4[2], eps=EPS, layout=layout)
        mx.mxnorm_bwd(xs[i], g, gain, r, dx, dgain, ws)
        mx.mx_cast_transposed(xs[i], r, ct, st, eps=EPS, layout=layout)
        mx.rmsnorm_nvfp4_fwd(xs[i], o4[0], o4[1], o4[2], eps=EPS)
        mx.mxnorm_postround_fwd(xs[i], c, s, r, eps=EPS, layout=layout)
        mx.mxnorm_add_fwd(xs[i], xs[(i + 1) % len(xs)], dx, c, s, r, eps=EPS, layout=layout)
    torch.cuda.synchronize()
    print(json.dumps({"profile_run": "3 launches of each kernel", "rows": T, "hidden": D, "timeouts": mx.device_timeouts()}))


def oracle_throughput(x_bits, reps: int = 1):
    """The CPU oracle as it stands, timed on this machine's host cores. Returns (GB/s, seconds, threads)."""
    import oracle
    oracle.build()
    T, D = x_bits.shape
    oracle.mxnorm_ref(x_bits[:256], eps=EPS)   # load the library, warm the pages
    t0 = time.perf_counter()
    for _ in range(reps):
        oracle.mxnorm_ref(x_bits, eps=EPS)
    dt = (time.perf_counter() - t0) / reps
    return algorithmic_bytes("mx", T, D) / dt / 1e9, dt, oracle.num_threads()


def run_reference(args, rank: int):
    if rank != 0:
        return
    w = wl.CONFIGS[WORKLOAD]
    x_bits = wl.bits(wl.make_inputs(w)["x"])
    vals = []
    for i in range(args.warmup + args.steps):
        gbs, dt, threads = oracle_throughput(x_bits)
        if i >= args.warmup:
            vals.append((gbs, dt))
    gbs = statistics.mean(v[0] for v in vals)
    dt = statistics.mean(v[1] for v in vals)
    line = {
        "impl": "reference", "metric": "mxnorm_fwd_hbm_gbs_d4096", "value": gbs, "unit": "GB/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": workload_name(w.T, w.D), "impl_note": "CPU oracle mxnorm_ref (plain C, binary64 statistics, OpenMP over rows)"},
        "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": threads, "kind": "oracle",
                         "sample": f"the full [{w.T},{w.D}] batch per step"},
        "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--skip-others", action="store_true", help="only the headline kernel (for profiler runs)")
    ap.add_argument("--rows", type=int, default=0, help="override the row count (profiler runs on a smaller case)")
    ap.add_argument("--all-configs", action="store_true", help="also time the forward kernels on configs C1 and C2")
    ap.add_argument("--profile", action="store_true",
                    help="launch every kernel of the path three times at full size and exit (a short run for ncu)")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        run_reference(args, rank)
        return
    if args.warmup < 3:
        args.warmup = 3

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback for the MXNorm path)")
    from paper_2603_13180_b200 import binding as mx   # fails loudly when libmxnorm.so is missing

    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    w = wl.CONFIGS[WORKLOAD]
    T, D = (args.rows or w.T), w.D
    inp = wl.make_inputs(w) if T == w.T else wl.make_inputs(w, T=T)
    x_cpu, gain_cpu = inp["x"], inp["gain"]
    layout = mx.SCALES_SWIZZLE_128x4
    stream = torch.cuda.current_stream()
    sh = stream.cuda_stream

    xs = [x_cpu.cuda() for _ in range(SETS)]
    outs = [mx.alloc_outputs(T, D, 32, layout) for _ in range(SETS)]
    L = mx.lib

    def fwd(i):
        c, s, r = outs[i]
        st = L.mxnorm_fwd(xs[i].data_ptr(), None, T, D, 32, 2, 0.0, EPS, c.data_ptr(), s.data_ptr(), r.data_ptr(),
                          0, layout, sh)
        if st != 0:
            raise RuntimeError(mx.status_string(st))

    def rms(i):
        c, s, r = outs[i]
        st = L.rmsnorm_mxfp8_fwd(xs[i].data_ptr(), None, T, D, 32, EPS, c.data_ptr(), s.data_ptr(), r.data_ptr(),
                                 0, layout, sh)
        if st != 0:
            raise RuntimeError(mx.status_string(st))

    def cast(i):
        c, s, r = outs[i]
        st = L.mx_cast(xs[i].data_ptr(), T, D, 32, c.data_ptr(), s.data_ptr(), 0, layout, sh)
        if st != 0:
            raise RuntimeError(mx.status_string(st))

    if args.profile:
        profile_run(mx, xs, outs, T, D, layout, fwd, rms, cast)
        return

    # ---- headline: K steps of mxnorm_fwd, device-timed, clocks sampled alongside ----
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    if dist is not None:
        dist.barrier()
    reps = time_repeated(fwd, SETS, args.steps, args.warmup, stream)      # REPEATS regions of exactly K launches each
    reps = sorted(sharding.max_over_ranks(v, device="cuda") for v in reps)   # max over ranks, repeat by repeat
    ms = statistics.median(reps)
    # keep the GPU under load a little longer so that the 50 ms sampler sees it
    if rank == 0:
        t_end = time.time() + 0.5
        while time.time() < t_end:
            for i in range(50):
                fwd(i % SETS)
            torch.cuda.synchronize()
    clocks = sampler.stop() if rank == 0 else None

    # the same launches with an event record between them: an event breaks the programmatic dependency, so
    # each kernel starts only after the previous one has fully retired (no overlap of launch and tail)
    def fwd_serialised(i):
        fwd(i)
        marker.record(stream)

    marker = torch.cuda.Event()
    ms_serial = time_median(fwd_serialised, SETS, args.steps, args.warmup, stream)

    nbytes = algorithmic_bytes("mx", T, D)
    gbs_one = nbytes / (ms * 1e-3) / 1e9
    peak, peak_kind = measured_peak()
    result = {
        "metric": "mxnorm_fwd_hbm_gbs_d4096", "value": gbs_one * world, "unit": "GB/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": workload_name(T, D),
                   "l2": f"inputs/outputs rotate over {SETS} buffer sets ({SETS * nbytes / 1e6:.0f} MB > 126 MB L2)",
                   "timing": f"{REPEATS} timed regions of {args.steps} launches each after {args.warmup} warm-up launches, every region bracketed by a "
                             "device synchronize and started behind a 0.1 ms clock-spin kernel so that the start event is not stamped "
                             "while the first launch is still on its way from the host; ms_per_step "
                             "is the median region, ms_per_step_spread its minimum and maximum; the other kernels: median of 3 regions of "
                             f"max(steps, {OTHERS_MIN_STEPS}) launches (half as many for the backward), each kernel "
                             f"after {REST_S} s of idle (burst figures, like the measured copy peak; seconds into an uninterrupted load "
                             "the instruction-heavier kernels run up to 8 % slower on this pool)",
                   "launch": "back-to-back launches in one stream, as the library issues them: programmatic stream "
                             "serialisation (each kernel waits for the previous one before it reads or writes any value; launch "
                             "latency and L2 prefetch hints for the first-wave rows overlap the previous kernel's tail); "
                             "event_between_launches_ms_per_step records an event after every launch",
                   "parallelism": f"rows sharded, no collective (x{world})"},
        "ms_per_step_spread": spread(reps),
        "event_between_launches_ms_per_step": ms_serial,
        "tokens_per_s": T * world / (ms * 1e-3),
        "gpu_launches": args.steps,                      # per timed region (ms_per_step is the median region)
        "gpu_launches_all_regions": args.steps * REPEATS,
        "clocks": clocks,
        "roofline": {"bound": "hbm", "achieved": gbs_one, "peak": peak, "unit": "GB/s", "frac": gbs_one / peak,
                     "peak_kind": f"of {peak_kind}", "frac_of_8TBs": gbs_one / 8000.0,
                     "traffic": NCU_TRAFFIC_BYTES if T == w.T else None, "traffic_kind": NCU_TRAFFIC_KIND,
                     "algorithmic_bytes": nbytes,
                     "kernel": "fwd_e4m3_kernel<B=32,NPASS=2,WPR=2,STAT=MX>"},
    }

    if not args.skip_others:
        # ---- the rest of the path, each timed the same way (context for the headline) ----
        others = {}
        # regions of at least OTHERS_MIN_STEPS launches whatever --steps says: a region of 10-20 launches carries the ramp
        # of its first and the tail of its last launch as 1-2 % (the headline keeps exactly --steps launches per region)
        osteps = max(args.steps, OTHERS_MIN_STEPS)
        ms_rms = time_median(rms, SETS, osteps, args.warmup, stream)
        ms_cast = time_median(cast, SETS, osteps, args.warmup, stream)
        ms_fwd_same = time_median(fwd, SETS, osteps, args.warmup, stream)      # the headline kernel timed the same way, for the ratio
        others["rmsnorm_mxfp8_fwd"] = {"ms": ms_rms, "gbs": algorithmic_bytes("rms", T, D) / ms_rms / 1e6}
        others["mx_cast"] = {"ms": ms_cast, "gbs": algorithmic_bytes("cast", T, D) / ms_cast / 1e6}
        others["mxnorm_fwd"] = {"ms": ms_fwd_same, "gbs": nbytes / ms_fwd_same / 1e6}
        result["speedup_vs_rmsnorm_mxfp8_fwd"] = ms_rms / ms_fwd_same
        def time_secondary_kernels():
            # NVFP4
            o4 = [mx.alloc_outputs(T, D, 16, mx.SCALES_ROWMAJOR, nvfp4=True) for _ in range(SETS)]

            def nvfp4(i):
                c, s, r = o4[i]
                st = L.mxnorm_nvfp4_fwd(xs[i].data_ptr(), T, D, 2, 0.0, EPS, 1.0, c.data_ptr(), s.data_ptr(), r.data_ptr(), 0, sh)
                if st != 0:
                    raise RuntimeError(mx.status_string(st))

            def rms_nvfp4(i):
                c, s, r = o4[i]
                st = L.rmsnorm_nvfp4_fwd(xs[i].data_ptr(), T, D, EPS, 1.0, c.data_ptr(), s.data_ptr(), r.data_ptr(), 0, sh)
                if st != 0:
                    raise RuntimeError(mx.status_string(st))

            ms4 = time_median(nvfp4, SETS, osteps, args.warmup, stream)
            ms4r = time_median(rms_nvfp4, SETS, osteps, args.warmup, stream)
            others["mxnorm_nvfp4_fwd"] = {"ms": ms4, "gbs": algorithmic_bytes("nvfp4", T, D) / ms4 / 1e6}
            others["rmsnorm_nvfp4_fwd"] = {"ms": ms4r, "gbs": algorithmic_bytes("nvfp4", T, D) / ms4r / 1e6}
            result["nvfp4_speedup_vs_rmsnorm_nvfp4_fwd"] = ms4r / ms4
            del o4
            # MXFP4 (E2M1 codes, E8M0 scales) and the column-wise cast of rho~*X for the weight-gradient GEMM
            m4 = [mx.alloc_outputs(T, D, 32, layout, nvfp4=True) for _ in range(SETS)]

            def mxfp4(i):
                c, s, r = m4[i]
                st = L.mxnorm_mxfp4_fwd(xs[i].data_ptr(), T, D, 32, 2, 0.0, EPS, c.data_ptr(), s.data_ptr(), r.data_ptr(), layout, sh)
                if st != 0:
                    raise RuntimeError(mx.status_string(st))

            msm4 = time_median(mxfp4, SETS, osteps, args.warmup, stream)
            others["mxnorm_mxfp4_fwd"] = {"ms": msm4, "gbs": (T * D * 2 + T * D // 2 + T * (D // 32) + 4 * T) / msm4 / 1e6}
            del m4
            if T % 32 == 0:
                ct = [torch.empty((D, T), dtype=torch.uint8, device="cuda") for _ in range(SETS)]
                stt = [torch.empty(mx.scale_bytes(D, T // 32, layout), dtype=torch.uint8, device="cuda") for _ in range(SETS)]
                r0 = outs[0][2]

                def transposed(i):
                    st = L.mx_cast_transposed(xs[i].data_ptr(), r0.data_ptr(), T, D, EPS, ct[i].data_ptr(), stt[i].data_ptr(), 0, layout, sh)
                    if st != 0:
                        raise RuntimeError(mx.status_string(st))

                mst = time_median(transposed, SETS, osteps, args.warmup, stream)
                others["mx_cast_transposed"] = {"ms": mst, "gbs": (T * D * 3 + T * D // 32 + 4 * T) / mst / 1e6}

                def transposed_plain(i):   # no normaliser: the column-wise cast of the upstream gradient
                    st = L.mx_cast_transposed(xs[i].data_ptr(), None, T, D, 0.0, ct[i].data_ptr(), stt[i].data_ptr(), 0, layout, sh)
                    if st != 0:
                        raise RuntimeError(mx.status_string(st))

                mstp = time_median(transposed_plain, SETS, osteps, args.warmup, stream)
                others["mx_cast_transposed_no_normaliser"] = {"ms": mstp, "gbs": (T * D * 3 + T * D // 32) / mstp / 1e6}
                del ct, stt
            # the ablation with power-of-two-rounded block maxima, and the residual add fused in front
            def postround(i):
                c, s, r = outs[i]
                st = L.mxnorm_postround_fwd(xs[i].data_ptr(), T, D, 32, EPS, c.data_ptr(), s.data_ptr(), r.data_ptr(), layout, sh)
                if st != 0:
                    raise RuntimeError(mx.status_string(st))

            mspr = time_median(postround, SETS, osteps, args.warmup, stream)
            others["mxnorm_postround_fwd"] = {"ms": mspr, "gbs": algorithmic_bytes("mx", T, D) / mspr / 1e6}
            # the same two kernels with a gain vector (the extension of Algorithm 2; Algorithm 1 as commonly deployed)
            gain_vec = (1.0 + 0.1 * torch.randn(D, generator=torch.Generator().manual_seed(2))).to(torch.bfloat16).cuda()   # made on the host: no torch kernel

            def fwd_gain(i):
                c, s, r = outs[i]
                st = L.mxnorm_fwd(xs[i].data_ptr(), gain_vec.data_ptr(), T, D, 32, 2, 0.0, EPS, c.data_ptr(), s.data_ptr(), r.data_ptr(), 0, layout, sh)
                if st != 0:
                    raise RuntimeError(mx.status_string(st))

            def rms_gain(i):
                c, s, r = outs[i]
                st = L.rmsnorm_mxfp8_fwd(xs[i].data_ptr(), gain_vec.data_ptr(), T, D, 32, EPS, c.data_ptr(), s.data_ptr(), r.data_ptr(), 0, layout, sh)
                if st != 0:
                    raise RuntimeError(mx.status_string(st))

            msg = time_median(fwd_gain, SETS, osteps, args.warmup, stream)
            others["mxnorm_fwd_with_gain"] = {"ms": msg, "gbs": (algorithmic_bytes("mx", T, D) + 2 * D) / msg / 1e6}
            msg = time_median(rms_gain, SETS, osteps, args.warmup, stream)
            others["rmsnorm_mxfp8_fwd_with_gain"] = {"ms": msg, "gbs": (algorithmic_bytes("rms", T, D) + 2 * D) / msg / 1e6}
            hs = [torch.empty_like(xs[0]) for _ in range(SETS)]

            def add_fwd(i):
                c, s, r = outs[i]
                st = L.mxnorm_add_fwd(xs[i].data_ptr(), xs[(i + 1) % SETS].data_ptr(), T, D, 32, 2, 0.0, EPS, hs[i].data_ptr(),
                                      c.data_ptr(), s.data_ptr(), r.data_ptr(), layout, sh)
                if st != 0:
                    raise RuntimeError(mx.status_string(st))

            msadd = time_median(add_fwd, SETS, osteps, args.warmup, stream)
            others["mxnorm_add_fwd"] = {"ms": msadd, "gbs": (algorithmic_bytes("mx", T, D) + 4 * T * D) / msadd / 1e6}
            del hs
            # backward (C5 tensors: seed 1, gradient ~ N(0, 1e-2), gain)
            w5 = wl.CONFIGS["C5"]
            inp5 = wl.make_inputs(w5) if T == w5.T else wl.make_inputs(w5, T=T)
            nb = 3
            xb = [inp5["x"].cuda() for _ in range(nb)]
            gb = [inp5["grad"].cuda() for _ in range(nb)]
            gain5 = inp5["gain"].cuda()
            dxb = [torch.empty_like(xb[0]) for _ in range(nb)]
            rmsb = torch.empty(T, dtype=torch.float32, device="cuda")
            c, s, _ = outs[0]
            mx.mxnorm_fwd(xb[0], None, c, s, rmsb, eps=EPS, layout=layout)
            dgain = torch.empty(D, dtype=torch.float32, device="cuda")
            ws = torch.empty(mx.mxnorm_bwd_workspace_bytes(T, D), dtype=torch.uint8, device="cuda")

            def bwd(i):
                st = L.mxnorm_bwd(xb[i].data_ptr(), gb[i].data_ptr(), gain5.data_ptr(), rmsb.data_ptr(), T, D,
                                  dxb[i].data_ptr(), 0, dgain.data_ptr(), ws.data_ptr(), ws.numel(), sh)
                if st != 0:
                    raise RuntimeError(mx.status_string(st))

            msb = time_median(bwd, nb, max(osteps // 2, 10), args.warmup, stream)
            others["mxnorm_bwd"] = {"ms": msb, "gbs": algorithmic_bytes("bwd", T, D) / msb / 1e6}

            def bwd_dx_only(i):   # the method's own configuration: no gain (folded into the next weight), hence no gain gradient
                st = L.mxnorm_bwd(xb[i].data_ptr(), gb[i].data_ptr(), None, rmsb.data_ptr(), T, D, dxb[i].data_ptr(), 0, None, None, 0, sh)
                if st != 0:
                    raise RuntimeError(mx.status_string(st))

            msbx = time_median(bwd_dx_only, nb, max(osteps // 2, 10), args.warmup, stream)
            others["mxnorm_bwd_dx_only"] = {"ms": msbx, "gbs": (3 * T * D * 2 + 4 * T) / msbx / 1e6}
            del xb, gb, dxb

        sampler2 = ClockSampler(local_rank)    # the secondary kernels run minutes into a sustained load: record the clock they saw
        if rank == 0:
            sampler2.start()
        try:   # context only: a failure here must not cost the headline line
            time_secondary_kernels()
        except Exception as e:   # noqa: BLE001
            result["others_error"] = f"{type(e).__name__}: {e}"[:300]
        if rank == 0:
            result["others_clocks"] = sampler2.stop()
        for v in others.values():
            v["frac_of_peak"] = v["gbs"] / peak
        result["others"] = others

        # ---- end to end through the C ABI with HOST buffers (pinned), copies inside the timed region ----
        xh = x_cpu.pin_memory()
        ch = torch.empty((T, D), dtype=torch.uint8).pin_memory()
        shh = torch.empty((mx.scale_bytes(T, D // 32, layout),), dtype=torch.uint8).pin_memory()
        rh = torch.empty((T,), dtype=torch.float32).pin_memory()
        wsh = torch.empty(mx.mxnorm_fwd_host_workspace_bytes(T, D, 32, layout), dtype=torch.uint8, device="cuda")

        def e2e_step(_):
            mx.mxnorm_fwd_host(xh, ch, shh, rh, wsh, eps=EPS, layout=layout, stream=stream)

        e2e_steps = max(3, min(args.steps, 20))
        ms_e2e = time_launches(e2e_step, 1, e2e_steps, 3, stream, gate=False)   # end to end: the host's latency belongs to it
        ms_e2e = sharding.max_over_ranks(ms_e2e, device="cuda")
        result["e2e"] = {"value": nbytes * world / (ms_e2e * 1e-3) / 1e9, "unit": "GB/s", "ms_per_step": ms_e2e,
                         "steps": e2e_steps, "h2d_bytes_per_step": T * D * 2,
                         "d2h_bytes_per_step": T * D + shh.numel() + 4 * T,
                         "api": "mxnorm_fwd_host (pinned host buffers, chunked copy/compute overlap)"}

        # ---- CPU oracle on this machine's host cores (rank 0, one GPU runs only) ----
        if rank == 0 and world == 1:
            gbs_cpu, dt, threads = oracle_throughput(wl.bits(x_cpu), reps=20)
            result["cpu_baseline"] = {"value": gbs_cpu, "unit": "GB/s", "cores": threads, "kind": "oracle",
                                      "seconds_per_batch": dt,
                                      "sample": f"20 passes of the full [{T},{D}] batch through mxnorm_ref (plain C, OpenMP over rows)"}

    if args.all_configs and not args.skip_others:
        result["configs"] = time_small_configs(mx, args, stream)

    if rank == 0:
        print(json.dumps(result))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
