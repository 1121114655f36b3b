#!/usr/bin/env python
"""Benchmark of the group-wise int8-quantized Winograd convolution on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 2] [--impl reference]

A *step* is one pass of the whole forward path (input transform + group quantization,
int8 tensor-core contraction with per-group dequantization, output transform) over
every layer of one workload configuration, called through the C ABI.  The metric is
direct-convolution-equivalent throughput, 2*N*K*C*H*W*9 operations per layer divided
by the time of the forward call (filter preparation is offline and not timed).

One JSON line is printed by rank 0.  Besides the throughput it carries
  roofline      achieved HBM GB/s of the kernel that takes the most time in a step,
                from CUDA events around the chain prefixes K1, K1+K2, K1+K2+K3
  e2e           the same metric through wfq_conv_forward_host (pinned host buffers,
                host<->device copies inside the timed region)
  cpu_baseline  the CPU oracle timed on this machine's cores on a sample of tiles
  clocks        SM clock and throttle reasons sampled during the timed region

With --gpus N > 1 every rank runs an independent replica of the workload (the path
needs no exchange between GPUs); the value is the aggregate over the ranks.
--impl reference times the CPU oracle instead of the CUDA path.
"""
import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "direct_conv_equivalent_TOPS"
UNIT = "TOPS"
FALLBACK_HBM_GBS = 6650.0
L2_FLUSH_BYTES = 256 << 20

# dram__bytes_read.sum + dram__bytes_write.sum per launch (mean over the layers of a step)
# from the ncu capture summarised in profiles/launches_cfg2_resnet18_stage.txt; cold-cache
# reads, and output that is still dirty in L2 when the kernel ends is not counted.  Only the
# default workload was captured; set an entry to None when its kernel changes.
NCU_TRAFFIC_BYTES = {2: {"input_transform_quantize": 6.07e6, "gemm_dequantize": 13.6e6,
                         "output_transform": 28.6e6}}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--config", type=int, default=2, help="workload configuration 1..5")
    ap.add_argument("--impl", default="wfq", choices=["wfq", "reference"])
    ap.add_argument("--only-layer", type=int, default=None,
                    help="restrict the workload to one layer of the configuration (profiling)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-graph", action="store_true",
                    help="enqueue every step with stream launches instead of replaying a CUDA graph")
    ap.add_argument("--cpu-seconds", type=float, default=16.0,
                    help="CPU time budget of the oracle baseline")
    return ap.parse_args()


def workload_name(cfg):
    return {1: "cfg1: single 64->64 32x32 F(4,3) layer, fp32 input",
            2: "cfg2: ResNet-18-style stage, four 3x3 layers N=32 C=K=64/128/256/512 "
               "at 56/28/14/7, F(6,3), group 64, fp16 input",
            3: "cfg3: ResNet-34-style sweep, N=64, 12 runs F(4,3)/F(6,3) x groups 32/64/128",
            4: "cfg4: diffusion-UNet block, N=2, C=K=320/640/1280 at 64/32/16, F(4,3), group 64",
            5: "cfg5: UNet conv-layer set at 128/64/32 latent, N=1, F(4,3) and F(6,3)"}[cfg]


def select_layers(wl, args):
    layers = wl.config_layers(args.config)
    return layers if args.only_layer is None else [layers[args.only_layer]]


# ---- byte counts the method itself must move (per launch) ----------------------------

def geometry(L):
    n = L.m + 2
    P = n * n
    T = L.N * (-(-L.H // L.m)) * (-(-L.W // L.m))
    G = L.C // L.gs
    return P, T, G


def algorithmic_bytes(L):
    """Bytes each of the three kernels has to read and write once."""
    P, T, G = geometry(L)
    e_in = 2 if L.dtype == "f16" else 4
    k1 = L.N * L.C * L.H * L.W * e_in + P * T * L.C + 4 * P * T * G
    k2 = P * T * L.C + P * L.K * L.C + 4 * P * G * (T + L.K) + 4 * P * T * L.K
    k3 = 4 * P * T * L.K + 4 * L.N * L.K * L.H * L.W
    return {"input_transform_quantize": k1, "gemm_dequantize": k2, "output_transform": k3}


# ---- clocks -----------------------------------------------------------------------------

class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index):
        self.samples, self.reasons = [], set()
        self.max_mhz = None
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

    def _loop(self):
        nv = self.nv
        names = {"hw_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8),
                 "hw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40),
                 "sw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20),
                 "sw_power_cap": getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4)}
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            self._stop.wait(0.01)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        med = None
        if self.samples:
            s = sorted(self.samples)
            med = s[len(s) // 2]
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# ---- CPU oracle legs -------------------------------------------------------------------

def oracle_time_sample(layers, tensors, seconds):
    """Times the oracle's forward pipeline on a sample of tiles of every layer.

    Each layer gets an equal share of `seconds`: as many (randomly chosen) tiles as that
    share allows, or, where the whole layer takes less, the whole layer several times.
    Returns (ops, secs, description, threads): direct-equivalent operations covered and
    the CPU seconds they took (filter preparation excluded, as on the GPU side).
    """
    import numpy as np
    from oracle import oracle as orc
    total_ops, total_s, desc = 0.0, 0.0, []
    per_layer = seconds / max(len(layers), 1)
    for L, (x, w, sB, sG) in zip(layers, tensors):
        P, T, G = geometry(L)
        mats = orc.matrices(L.m, sB, sG)
        filt = orc.prepare_filters(w, L.m, L.gs, mats)
        rng = np.random.default_rng(L.seed + 7)

        def run(n):
            tiles = np.sort(rng.choice(T, n, replace=False))
            t0 = time.perf_counter()
            orc.wfq(x, w, L.m, L.gs, sB=sB, sG=sG, tiles=tiles, filters=filt)
            return time.perf_counter() - t0

        n = min(T, 16)
        dt = run(n)
        while n < T and dt < 0.25 * per_layer:            # grow the sample towards the budget
            n = min(T, max(2 * n, int(n * 0.8 * per_layer / max(dt, 1e-6))))
            dt = run(n)
        reps, spent = 1, dt
        while n == T and spent + dt < per_layer:          # a small layer: whole layer, repeated
            spent += run(n)
            reps += 1
        total_ops += L.direct_ops * (n / T) * reps
        total_s += spent
        desc.append(f"{n}/{T}" + (f"x{reps}" if reps > 1 else ""))
    return total_ops, total_s, "tiles per layer " + ",".join(desc), orc.num_threads()


def run_reference(args):
    """The CPU oracle as the reference arm (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from paper_2412_19867_b200 import workloads as wl
    layers = select_layers(wl, args)
    tensors = [wl.make_tensors(L) for L in layers]
    nsteps = args.steps + args.warmup
    per_step = max(0.5, min(20.0, 90.0 / max(nsteps, 1)))
    ops = secs = 0.0
    sample, cores = "", 0
    for i in range(nsteps):
        o, s, sample, cores = oracle_time_sample(layers, tensors, per_step)
        if i >= args.warmup:
            ops += o
            secs += s
    value = ops / secs / 1e12
    step_ops = sum(L.direct_ops for L in layers)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": step_ops / (value * 1e12) * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": workload_name(args.config),
                       "note": "CPU oracle; each step times a sample of tiles and is scaled "
                               "to the whole workload"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": sample + " per step"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ---- aggregation over replicas ---------------------------------------------------------

def max_over_ranks(value, device=None):
    """The maximum of a per-rank time over all ranks (no-op without a process group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replica_throughput(ops_per_replica, world, ms_per_step):
    """Whole-job throughput in TOPS: every rank runs an independent replica of the
    workload (the path needs no exchange), the job takes as long as its slowest rank."""
    return world * ops_per_replica / (ms_per_step * 1e-3) / 1e12


# ---- the CUDA path ---------------------------------------------------------------------

def run_wfq(args):
    import torch
    import torch.distributed as dist
    from paper_2412_19867_b200 import binding as b
    from paper_2412_19867_b200 import build as wfq_build
    from paper_2412_19867_b200 import workloads as wl

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    if rank == 0:
        wfq_build.build()
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        dist.barrier()
    b.load()
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    stream = torch.cuda.current_stream(dev)

    layers = select_layers(wl, args)
    tensors = [wl.make_tensors(L) for L in layers]
    convs, xs, ys = [], [], []
    for L, (x, w, sB, sG) in zip(layers, tensors):
        conv = b.Conv(L.N, L.C, L.K, L.H, L.W, L.m, L.gs, L.dtype, dev)
        conv.prepare(torch.from_numpy(w).to(dev), list(sB), list(sG))
        convs.append(conv)
        xs.append(torch.from_numpy(x).to(dev))
        ys.append(torch.empty((L.N, L.K, L.H, L.W), dtype=torch.float32, device=dev))
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    step_ops = float(sum(L.direct_ops for L in layers))
    sptr = stream.cuda_stream

    def enqueue(stream_ptr):
        for conv, x, y in zip(convs, xs, ys):
            b.wfq_conv_forward(conv.plan, x.data_ptr(), y.data_ptr(), stream_ptr)

    # One step = the forward calls of all layers.  They are captured once into a CUDA graph
    # and replayed (same kernels, same order, one submission per step); stream launches are
    # the fallback and what --no-graph selects.
    enqueue(sptr)
    torch.cuda.synchronize(dev)
    graph, launch_mode = None, "stream launches"
    if not args.no_graph:
        try:
            side = torch.cuda.Stream(dev)
            side.wait_stream(stream)
            cand = torch.cuda.CUDAGraph()
            with torch.cuda.graph(cand, stream=side):
                enqueue(side.cuda_stream)
            torch.cuda.synchronize(dev)
            graph, launch_mode = cand, "CUDA graph replay"
        except Exception as exc:   # capture is an optimisation of the submission only
            print(f"bench: graph capture failed ({exc!r}); using stream launches", file=sys.stderr)
            torch.cuda.synchronize(dev)

    def step():
        if graph is not None:
            graph.replay()
        else:
            enqueue(sptr)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    for _ in range(max(args.warmup, 3)):
        flush.zero_()
        step()
    barrier()
    for conv in convs:
        conv.check_status()

    # ---- timed region: K steps, L2 flushed before each, one event pair per step --------
    sampler = ClockSampler(local)
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    stops = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    barrier()
    sampler.start()
    wall0 = time.perf_counter()
    for i in range(args.steps):
        flush.zero_()
        starts[i].record(stream)
        step()
        stops[i].record(stream)
    barrier()
    wall = time.perf_counter() - wall0
    clocks = sampler.stop()
    ms_steps = [s.elapsed_time(e) for s, e in zip(starts, stops)]
    total_ms = float(sum(ms_steps))
    total_ms = max_over_ranks(total_ms, dev)
    ms_per_step = total_ms / args.steps
    value = replica_throughput(step_ops, world, ms_per_step)

    # ---- the same steps back to back, no L2 flush (operands may sit in the 126 MB L2) ------
    wsteps = min(args.steps, 100)
    step()
    torch.cuda.synchronize(dev)
    w0, w1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    w0.record(stream)
    for _ in range(wsteps):
        step()
    w1.record(stream)
    torch.cuda.synchronize(dev)
    warm_ms = max_over_ranks(w0.elapsed_time(w1) / wsteps, dev)
    warm = {"ms_per_step": warm_ms, "value": replica_throughput(step_ops, world, warm_ms), "unit": UNIT,
            "steps": wsteps, "l2": "not flushed"}

    # ---- per-kernel durations: differences of chain prefixes ---------------------------
    # An event pair around a single short kernel adds several microseconds of launch
    # latency to it.  So each layer is timed three times per step, as K1, K1+K2 and
    # K1+K2+K3 (L2 flushed before each, one event pair around each prefix); the stage
    # durations are the differences, the first one carries the pair's overhead.
    names = ["input_transform_quantize", "gemm_dequantize", "output_transform"]
    ksteps = min(args.steps, 100)
    kern_ms = [[0.0, 0.0, 0.0] for _ in layers]
    for _ in range(ksteps):
        evs = []
        for conv, x, y in zip(convs, xs, ys):
            per_prefix = []
            for depth in (1, 2, 3):
                flush.zero_()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                b.wfq_input_transform_quantize(conv.plan, x.data_ptr(), sptr)
                if depth >= 2:
                    b.wfq_gemm_dequantize(conv.plan, sptr)
                if depth >= 3:
                    b.wfq_output_transform(conv.plan, y.data_ptr(), sptr)
                e1.record(stream)
                per_prefix.append((e0, e1))
            evs.append(per_prefix)
        torch.cuda.synchronize(dev)
        for li, per_prefix in enumerate(evs):
            t = [a.elapsed_time(z) for a, z in per_prefix]
            kern_ms[li][0] += t[0] / ksteps
            kern_ms[li][1] += (t[1] - t[0]) / ksteps
            kern_ms[li][2] += (t[2] - t[1]) / ksteps
    abytes = [algorithmic_bytes(L) for L in layers]
    tot_ms = [sum(kern_ms[li][k] for li in range(len(layers))) for k in range(3)]
    tot_bytes = [sum(abytes[li][names[k]] for li in range(len(layers))) for k in range(3)]
    dom = max(range(3), key=lambda k: tot_ms[k])
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        with open(peaks_path) as f:
            peak, peak_src = float(json.load(f)["hbm_gbs"]), "measured copy bandwidth"
    else:
        peak, peak_src = FALLBACK_HBM_GBS, "fallback"
    achieved = tot_bytes[dom] / (tot_ms[dom] * 1e-3) / 1e9
    traffic = None
    if args.only_layer is None:
        traffic = NCU_TRAFFIC_BYTES.get(args.config, {}).get(names[dom])
    roofline = {"bound": "hbm", "kernel": names[dom], "achieved": achieved, "peak": peak,
                "unit": "GB/s", "frac": achieved / peak, "traffic": traffic, "peak_source": peak_src,
                "launches_per_step": len(layers),
                "algorithmic_bytes_per_step": tot_bytes[dom],
                "algorithmic_bytes_per_launch": tot_bytes[dom] / len(layers),
                "all_kernels": {names[k]: {"us_per_step": tot_ms[k] * 1e3,
                                           "GBps": tot_bytes[k] / (tot_ms[k] * 1e-3) / 1e9,
                                           "frac": tot_bytes[k] / (tot_ms[k] * 1e-3) / 1e9 / peak}
                                for k in range(3)}}
    # contraction alone: algorithmic int8 operations 2*P*T*C*K per layer against the tensor peak
    def tiles(L):
        return L.N * (-(-L.H // L.m)) * (-(-L.W // L.m))
    gemm_ops = float(sum(2.0 * (L.m + 2) ** 2 * tiles(L) * L.C * L.K for L in layers))
    gemm_tops = gemm_ops / (tot_ms[1] * 1e-3) / 1e12
    gk = roofline["all_kernels"][names[1]]
    gk["int8_TOPS"] = gemm_tops
    gk["frac_of_nominal_int8_4500_TOPS"] = gemm_tops / 4500.0
    if os.path.exists(peaks_path):
        with open(peaks_path) as f:
            bf16 = json.load(f).get("bf16_tflops")
        if bf16:
            gk["frac_of_2x_measured_bf16"] = gemm_tops / (2.0 * float(bf16))
    layer_rows = []
    for li, L in enumerate(layers):
        us = [kern_ms[li][k] * 1e3 for k in range(3)]
        layer_rows.append({"layer": L.name, "us": sum(us), "us_k1_k2_k3": [round(u, 2) for u in us],
                           "eq_TOPS": L.direct_ops / (sum(us) * 1e-6) / 1e12})

    # ---- end to end through the host-buffer entry point ----------------------------------
    e2e = None
    if not args.no_e2e:
        xh = [torch.from_numpy(t[0]).pin_memory() for t in tensors]
        yh = [torch.empty(y.shape, dtype=torch.float32).pin_memory() for y in ys]
        esteps = max(3, min(args.steps, 20))
        for conv, x, y in zip(convs, xh, yh):
            conv.forward_host(x, y)
        barrier()
        t0 = time.perf_counter()
        for _ in range(esteps):
            for conv, x, y in zip(convs, xh, yh):
                conv.forward_host(x, y)          # synchronous: copies + kernels + copy back
        torch.cuda.synchronize(dev)
        dt = time.perf_counter() - t0
        dt = max_over_ranks(dt, dev)
        e2e = {"value": replica_throughput(step_ops, world, dt * 1e3 / esteps), "unit": UNIT,
               "h2d_bytes_per_step": int(sum(x.numel() * x.element_size() for x in xh)),
               "d2h_bytes_per_step": int(sum(y.numel() * 4 for y in yh)), "steps": esteps}

    for conv in convs:
        conv.check_status()
        conv.close()

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        o, s, sample, cores = oracle_time_sample(layers, tensors, args.cpu_seconds)
        cpu = {"value": o / s / 1e12, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": sample + f" ({s:.1f} s of CPU time)"}

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
                "config": {"workload": workload_name(args.config) +
                           ("" if args.only_layer is None else f" (layer {args.only_layer} only)"),
                           "layers": len(layers), "launch": launch_mode,
                           "l2": "flushed before every step (256 MiB memset outside the step's "
                                 "event pair)",
                           "parallelism": "replicas" if world > 1 else "single GPU"},
                "us_per_layer": layer_rows, "wall_s_timed_region": wall,
                "warm": warm, "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e,
                "gpu_launches": 3 * len(layers) * args.steps, "clocks": clocks}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_wfq(args)


if __name__ == "__main__":
    main()
