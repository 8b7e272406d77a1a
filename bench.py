#!/usr/bin/env python
"""Benchmark of the Tune-mode ConvBN hot path on B200.

A step is one pass of the whole path - convbn_tune_fwd, then convbn_tune_bwd_begin (input gradient on the
caller's stream, parameter gradients on the library's side stream) - over every layer of a configuration,
closed by one convbn_tune_bwd_join (``--join-per-layer``: convbn_tune_bwd, which joins in every call;
``--order training``: every forward call first, then every backward call).  With no ``--workload`` all five
configurations run in one process and ONE JSON line is printed: ``value`` is the fwd+bwd TFLOP/s
over the three dense bf16 configurations (1-3: total FLOPs / total time), ``per_config`` holds
every configuration on its own (config 4 in GB/s against the copy bandwidth, config 0 as a
latency), ``backbone`` a whole ResNet-50 (batch 32 and 256 at 224x224, batch 32 at 448x448) replayed in Tune, Eval and Deploy mode
with time per iteration and peak memory.  FLOPs = 3 phases x 2 P C_out (C_in/G) kh kw per layer.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload i]

Under torchrun every rank runs its own replica on its own batch (the path needs no exchange
between samples), times it with CUDA events, and rank 0 prints the line with the max-over-ranks
time; ``--gpus N`` without a launcher starts the N ranks itself.  ``--impl reference`` times the
fp64 CPU oracle instead (rank 0 only).
"""
import argparse
import json
import math
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "Tune ConvBN fwd+bwd TFLOP/s"
UNIT = "TFLOP/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
WORKLOAD_NAMES = {
    0: "config0: single fp32 NCHW block 3x3 16->32 at 16x16, N=2",
    1: "config1: ResNet-50 stage-2 bottleneck chain (1x1 256->64, 3x3 64->64, 1x1 64->256), bf16 NHWC, N=32, 56x56",
    2: "config2: ResNet-50 stem 7x7 s2 and stage-4 layers, bf16 NHWC, N=64",
    3: "config3: detection-backbone 3x3 layers at 800x1333, bf16 NHWC, N=2",
    4: "config4: depthwise 3x3 C=96 at 112x112 and grouped 3x3 G=32 256->256 at 28x28, bf16 NHWC, N=64",
}
DENSE = (1, 2, 3)          # the configurations behind `value`


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def layer_flops(spec, out_hw):
    return 2.0 * spec.n * out_hw[0] * out_hw[1] * spec.c_out * (spec.c_in // spec.groups) * spec.kh * spec.kw


# ---- algorithmic bytes of each main kernel, per launch ------------------------------------------
def kernel_bytes(kind, spec, out_hw):
    es = 2 if spec.dtype == "bf16" else 4
    x = spec.n * spec.c_in * spec.h_in * spec.w_in * es
    z = spec.n * spec.c_out * out_hw[0] * out_hw[1] * es
    wel = spec.c_out * (spec.c_in // spec.groups) * spec.kh * spec.kw
    if kind == "fwd":      # read X and omega', write Z
        return x + wel * es + z
    if kind == "dgrad":    # read dZ and omega', write dX
        return z + wel * es + x
    if kind == "wgrad":    # read dZ and X, write fp32 domega'
        return z + x + wel * 4
    if kind == "bwd":      # fused backward: dZ and X read once, dX and fp32 domega' written
        return z + 2 * x + wel * es + wel * 4
    raise KeyError(kind)


# DRAM bytes (read + write) per launch, from ncu captures of the kernels as they are now; a kernel that
# changed after its capture has no entry (traffic: null).  key: (kernel family, layer) -> (bytes, summary file).
_P1, _P2S, _P2D, _P4 = ("profiles/config1_kernels_ncu_full.md", "profiles/config2_stem_window_kernels_ncu_full.md",
                        "profiles/config2_dense_gemm_ncu_full.md", "profiles/config4a_depthwise_kernels_ncu_full.md")
NCU_TRAFFIC = {("stem_fwd", "c2s"): (66.3e6, _P2S), ("stem_dgrad", "c2s"): (116.6e6, _P2S), ("stem_wgrad", "c2s"): (126.9e6, _P2S),
               ("umma_bwd", "c1a"): (76.4e6, _P1), ("strip_fwd", "c1b"): (13.0e6, _P1), ("strip_dgrad", "c1b"): (13.0e6, _P1),
               ("umma_fwd", "c2a"): (14.99e6, _P2D), ("umma_dgrad", "c2a"): (5.35e6, _P2D), ("umma_wgrad", "c2a"): (16.10e6, _P2D),
               ("umma_fwd", "c2b"): (7.98e6, _P2D),
               ("dw_fwd", "c4a"): (259.0e6, _P4), ("dw_dgrad", "c4a"): (258.7e6, _P4), ("dw_wgrad", "c4a"): (312.0e6, _P4)}

KIND_OF = {"strip_fwd": "fwd", "strip_dgrad": "dgrad", "direct_fwd": "fwd", "direct_dgrad": "dgrad", "direct_wgrad": "wgrad",
           "umma_fwd": "fwd", "umma_dgrad": "dgrad", "umma_wgrad": "wgrad", "umma_bwd": "bwd",
           "dw_fwd": "fwd", "dw_dgrad": "dgrad", "dw_wgrad": "wgrad",
           "grouped_fwd": "fwd", "grouped_dgrad": "dgrad", "grouped_wgrad": "wgrad",
           "stem_fwd": "fwd", "stem_dgrad": "dgrad", "stem_wgrad": "wgrad"}
PHASE_KIND = {"fwd": "fwd", "bwd_data": "dgrad", "bwd_weight": "wgrad", "bwd": "bwd"}


def shape_tag(spec):
    return "n%d_c%d_%dx%d_o%d_k%dx%d_s%d_g%d" % (spec.n, spec.c_in, spec.h_in, spec.w_in, spec.c_out,
                                                 spec.kh, spec.kw, spec.stride, spec.groups)


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU through NVML (read-only) while running."""

    def __init__(self, uuid, period=0.005):
        super().__init__(daemon=True)
        self.period, self.stop_flag = period, threading.Event()
        self.sm, self.reasons, self.sm_max, self.ok = [], set(), None, False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode() if isinstance(uuid, str) else uuid)
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            self.sm_max = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception as e:  # NVML absent: report that instead of clocks
            self.err = repr(e)

    def run(self):
        nv = self.nv if self.ok else None
        names = {}
        if nv:
            for n in ("HwSlowdown", "HwThermalSlowdown", "SwThermalSlowdown", "SwPowerCap",
                      "HwPowerBrakeSlowdown", "SyncBoost", "ApplicationsClocksSetting"):
                v = getattr(nv, "nvmlClocksEventReason" + n, None) or getattr(nv, "nvmlClocksThrottleReason" + n, None)
                if v:
                    names[int(v)] = n
        while nv and not self.stop_flag.is_set():
            try:
                self.sm.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                get = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
                    nv.nvmlDeviceGetCurrentClocksThrottleReasons
                mask = int(get(self.h))
                for bit, n in names.items():
                    if mask & bit:
                        self.reasons.add(n)
            except Exception:
                pass
            self.stop_flag.wait(self.period)

    def finish(self):
        self.stop_flag.set()
        self.join()
        return self.summary()

    def summary(self):
        if not self.ok or not self.sm:
            return {"sm_mhz": None, "sm_max_mhz": self.sm_max, "reasons": ["nvml-unavailable"]}
        s = sorted(self.sm)
        snake = {"HwSlowdown": "hw_slowdown", "HwThermalSlowdown": "hw_thermal_slowdown",
                 "SwThermalSlowdown": "sw_thermal_slowdown", "SwPowerCap": "sw_power_cap",
                 "HwPowerBrakeSlowdown": "hw_power_brake", "SyncBoost": "sync_boost",
                 "ApplicationsClocksSetting": "applications_clocks_setting"}
        return {"sm_mhz": s[len(s) // 2], "sm_max_mhz": self.sm_max, "samples": len(s),
                "reasons": sorted(snake[r] for r in self.reasons)}


def merge_clocks(summaries):
    """One clocks object over several timed regions: median of the medians, union of the reasons."""
    ok = [c for c in summaries if c.get("sm_mhz") is not None]
    if not ok:
        return summaries[0] if summaries else {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvml-unavailable"]}
    med = sorted(c["sm_mhz"] for c in ok)
    return {"sm_mhz": med[len(med) // 2], "sm_max_mhz": ok[0]["sm_max_mhz"],
            "samples": sum(c.get("samples", 0) for c in ok),
            "reasons": sorted(set(r for c in ok for r in c["reasons"]))}


def tensor_peak(peaks, clocks):
    """The measured bf16 peak that applies: the burst figure while the sampled SM clock stays within
    5 % of its maximum with no power cap, else the sustained one."""
    burst, sus = peaks["bf16_tflops"], peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])
    sm, mx = clocks.get("sm_mhz"), clocks.get("sm_max_mhz")
    at_max = sm is not None and mx and sm >= 0.95 * mx and "sw_power_cap" not in clocks.get("reasons", [])
    return (burst, "burst") if at_max or sm is None else (sus, "sustained")


# ---- multi-rank bookkeeping (replicas: every rank runs the whole workload on its own batch) -------
def max_over_ranks(value, device=None):
    """The slowest rank's time: MAX all-reduce over the default process group (identity for one rank)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(flops_per_step, steps, ms_max, world):
    """Aggregate TFLOP/s of `world` replicas that each did `steps` steps within `ms_max` milliseconds."""
    return world * flops_per_step * steps / (ms_max * 1e-3) / 1e12


def spawn_ranks(args):
    """`--gpus N` without a launcher: start N ranks of this script under torch.distributed.run."""
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "INFO")           # the communicator's rank count stays in the log
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(args.gpus),
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd, env=env)


# ---- the CPU oracle, timed (reported baseline and the --impl reference arm) ----------------------
def oracle_step_time(workload, batch, repeats, seed=7):
    """Seconds per Tune fwd+bwd step of the fp64 oracle on `batch` samples of every layer of the
    workload, and the FLOPs of that step.  Inputs are drawn once, outside the timed region."""
    import dataclasses
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    import parity
    from oracle import oracle as O
    from paper_2305_11624_b200 import inputs as I
    jobs, flops = [], 0.0
    for li, sp in enumerate(I.CONFIGS[workload]):
        sp = dataclasses.replace(sp, n=min(batch, sp.n))
        t = parity.make_inputs(sp, seed + li)
        jobs.append((sp, t))
        flops += 3 * layer_flops(sp, O.out_hw(parity.oracle_shape(sp)))
    times = []
    for _ in range(repeats):
        t0 = time.perf_counter()
        for sp, t in jobs:
            parity.oracle_tune(sp, t)
        times.append(time.perf_counter() - t0)
    return times, flops, O.num_threads()


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    batch = args.ref_batch
    workloads = [args.workload] if args.workload is not None else list(DENSE)
    per, flops, cores = 0.0, 0.0, 0
    for wl in workloads:
        times, fl, cores = oracle_step_time(wl, batch, args.warmup + args.steps)
        timed = times[args.warmup:]
        per += sum(timed) / len(timed)
        flops += fl
    val = flops / per / 1e12
    sample = "fp64 oracle, Tune fwd+bwd of every layer of the workload on a batch of %d samples per step" % batch
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": per * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": "; ".join(WORKLOAD_NAMES[w] for w in workloads), "sample": sample},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ---- the CUDA path ------------------------------------------------------------------------------
class Ctx:
    pass


def measured_activation_bytes(ctx, layers, mode):
    """Peak of torch's allocator over forward (every layer) then backward (reverse order) of the layers, minus
    what was allocated before: what a framework holding these layers keeps alive between the two passes plus
    the transients of a call.  Outputs, `saved` state and per-call scratch are allocated inside the region;
    an input whose shape matches the previous layer's output IS that output (a chain)."""
    torch, C, Block = ctx.torch, ctx.C, ctx.Block
    dev = ctx.dev
    blks = [Block(sp, device=dev, modes=(mode,), allocate="params") for sp in layers]
    for i, b in enumerate(blks):
        b.randomize_params(1000 + i)
    es = lambda b: 2 if b.spec.dtype == "bf16" else 4
    new = lambda n, dt: torch.empty(int(n), dtype=dt, device=dev)
    torch.cuda.synchronize()
    torch.cuda.reset_peak_memory_stats(dev)
    base = torch.cuda.memory_allocated(dev)
    x = None
    for b in blks:
        nx = math.prod(b.x_shape)
        if x is None or x.numel() != nx or x.dtype != b.tdtype:
            x = new(nx, b.tdtype).normal_()
        b.x = x
        b.z = new(math.prod(b.z_shape), b.tdtype)
        if mode == "tune":
            b.saved = new(max(16, C.convbn_saved_bytes(b.desc, C.MODE_TUNE)), torch.uint8)
            b.with_scratch(C.PHASE_TUNE_FWD, b.tune_fwd)
        else:
            b.y_saved = new(C.convbn_saved_bytes(b.desc, C.MODE_EVAL), torch.uint8)
            b.with_scratch(C.PHASE_EVAL_FWD, b.eval_fwd)
        x = b.z
        b.z = None                      # the output lives on only as the next layer's input (or the loss's)
    dz = torch.empty_like(x).normal_()
    del x
    for b in reversed(blks):
        if dz.numel() != math.prod(b.z_shape):
            dz = new(math.prod(b.z_shape), b.tdtype).normal_()
        b.dz = dz
        b.dx = new(math.prod(b.x_shape), b.tdtype)
        if mode == "tune":
            b.with_scratch(C.PHASE_TUNE_BWD_DATA, b.tune_bwd_data)
            b.with_scratch(C.PHASE_TUNE_BWD_WEIGHT, b.tune_bwd_weight)
            b.saved = None
        else:
            b.with_scratch(C.PHASE_EVAL_BWD, b.eval_bwd)
            b.y_saved = None
        dz = b.dx
        b.x = b.dz = b.dx = None
    torch.cuda.synchronize()
    C.convbn_check()
    peak = torch.cuda.max_memory_allocated(dev) - base
    del blks, dz
    return int(peak)


def bench_config(ctx, wl):
    """Everything measured on one configuration; returns its per_config entry (rank 0) plus raw sums."""
    args, torch, C, I, Block = ctx.args, ctx.torch, ctx.C, ctx.I, ctx.Block
    dev, rank, world, peaks, peak_src = ctx.dev, ctx.rank, ctx.world, ctx.peaks, ctx.peak_src
    dist = ctx.dist
    layers = I.CONFIGS[wl]
    probe = [Block(sp, device=dev) for sp in layers]
    step_flops = sum(3 * b.flops_per_phase() for b in probe)
    footprint = sum(t.numel() * t.element_size() for b in probe for t in (b.x, b.dz, b.z, b.dx))
    two_pass_bytes = sum(kernel_bytes(k, b.spec, (b.h_out, b.w_out)) for b in probe for k in ("fwd", "dgrad", "wgrad"))
    l2 = int(torch.cuda.get_device_properties(dev).L2_cache_size)
    sets = args.buffer_sets if args.buffer_sets > 0 else max(2, min(16, int(math.ceil(2.0 * l2 / footprint)) + 1))
    blocks = [probe] + [[Block(sp, device=dev) for sp in layers] for _ in range(sets - 1)]
    for si, bs in enumerate(blocks):
        for li, b in enumerate(bs):
            b.randomize(I.config_seed(wl, li) + 7919 * (rank * sets + si))
    stream = torch.cuda.current_stream()
    calls_per_step = 2 * len(layers)             # convbn_tune_fwd and convbn_tune_bwd per layer
    # --dp-allreduce: the layers' parameter gradients are views of one fp32 bucket per buffer set, summed over
    # the ranks at the end of every step (the only exchange data-parallel Tune mode needs); default: replicas
    buckets = None
    if args.dp_allreduce and world > 1:
        from paper_2305_11624_b200.dataparallel import GradientBucket
        buckets = []
        for bs in blocks:
            sizes = GradientBucket.sizes_for([(b.spec.name, b.spec.c_out, b.dw.numel() // b.spec.c_out, b.db is not None)
                                              for b in bs])
            bk = GradientBucket(sizes, device=dev)
            for b in bs:
                b.dw, b.dgamma, b.dbeta = (bk.views[b.spec.name + k] for k in (".dw", ".dgamma", ".dbeta"))
                if b.db is not None:
                    b.db = bk.views[b.spec.name + ".db"]
            buckets.append(bk)

    # Parameter gradients off the critical path: every layer's backward call leaves its weight-gradient pass on the
    # library's side stream and the step joins once at its end (--join-per-layer: every call joins before it returns).
    defer = not args.join_per_layer

    def run_layers(bs, st=None):
        """One step over the layers `bs`.  Deferred mode follows the order of a training step: every forward call,
        each followed by the preparation of its backward weights on the library's prepare stream; then every backward
        call (input gradients on the caller's stream, parameter gradients on the side stream); one join."""
        if not defer:
            for b in bs:
                b.tune_step(st)
            return
        if args.order == "layer":
            for b in bs:
                b.tune_step(st, defer_join=True)
        else:
            for b in bs:
                b.tune_fwd(st)
            for b in bs:
                b.tune_bwd_begin(st)
        C.convbn_tune_bwd_join(st)

    def step(i):
        run_layers(blocks[i % sets], stream)
        if buckets:
            buckets[i % sets].all_reduce_async()
            buckets[i % sets].wait()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(max(args.warmup, sets)):
        step(i)
    C.convbn_check()
    barrier()

    # ---- timed region: K steps, each a replay of the CUDA graph of one step (one graph per buffer set), so
    # the launches of a step cost no host time; --no-graph times eager calls.
    graphs, launch_mode = None, "eager library calls"
    if not args.no_graph and not buckets:        # (the collective is issued eagerly, outside a captured graph)
        try:
            graphs = []
            for si in range(sets):
                gr = torch.cuda.CUDAGraph()
                with torch.cuda.graph(gr):
                    run_layers(blocks[si])
                graphs.append(gr)
            for gr in graphs:
                gr.replay()
            torch.cuda.synchronize()
            launch_mode = "CUDA graph replay (one captured step per buffer set)"
        except Exception as exc:  # capture unsupported: say so and time eager calls
            graphs, launch_mode = None, "eager library calls (graph capture failed: %r)" % (exc,)

    launch_mode += ("; %s; parameter-gradient passes on the library's side stream, one join per step"
                    % ("forward then backward of each layer in turn" if args.order == "layer"
                       else "every forward call, then every backward call") if defer
                    else "; every backward call joins its parameter-gradient pass")

    def timed(n_sets):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for i in range(3):                      # a few untimed replays settle clocks and caches
            graphs[i % n_sets].replay() if graphs else step(i % n_sets)
        barrier()
        e0.record(stream)
        for i in range(args.steps):
            if graphs:
                graphs[i % n_sets].replay()
            else:
                step(i % n_sets)
        e1.record(stream)
        barrier()
        return max_over_ranks(e0.elapsed_time(e1), dev)

    uuid = str(torch.cuda.get_device_properties(dev).uuid)
    sampler = ClockSampler(uuid if uuid.startswith("GPU-") else "GPU-" + uuid)
    sampler.start()
    ms = timed(sets)                            # cold: rotating sets, together larger than twice the L2
    ms_warm = timed(1)                          # warm: the same buffers every step
    # the other orders of the same step, for comparison: every forward call before every backward call (what a
    # training step does: the forward phase then has nothing to overlap with), and one stream joined in every call
    ms_other = {}
    if graphs and defer and args.order == "layer":
        keep_graphs = graphs
        for name, order, dfr in (("training_order", "training", True), ("join_per_layer", "layer", False)):
            args.order, defer, graphs = order, dfr, []
            for si in range(sets):
                gr = torch.cuda.CUDAGraph()
                with torch.cuda.graph(gr):
                    run_layers(blocks[si])
                graphs.append(gr)
            ms_other[name] = timed(sets) / args.steps
        args.order, defer, graphs = "layer", True, keep_graphs
    # ---- second pass, same K steps as eager calls with a CUDA-event pair around every kernel: the
    # per-kernel durations behind the roofline object (events cannot be read back out of a graph)
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    C.convbn_profile_begin()
    barrier()
    f0.record(stream)
    for i in range(args.steps):
        step(i)
    f1.record(stream)
    barrier()
    prof = C.convbn_profile_end()
    eager_ms = max_over_ranks(f0.elapsed_time(f1), dev)
    clocks = sampler.finish()
    C.convbn_check()
    # host time of a library call (descriptor checks, plans, tensor maps, launches), GPU work queued behind
    hsteps = max(1, min(args.steps, 256 // calls_per_step))
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for i in range(hsteps):
        step(i)
    host_us = (time.perf_counter() - t0) / (hsteps * calls_per_step) * 1e6
    torch.cuda.synchronize()

    # ---- rooflines ---------------------------------------------------------------------------------
    hbm = peaks["hbm_gbs"]
    tc, tc_kind = tensor_peak(peaks, clocks)
    tc_burst, tc_sus = peaks["bf16_tflops"], peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])
    ridge = tc_burst * 1e12 / (hbm * 1e9)               # FLOP per byte above which the tensor peak bounds
    tag2layer = {shape_tag(b.spec): b for b in blocks[0]}
    kernels, phase_ms = [], {}
    for name, (count, total_ms) in prof.items():
        fam, _, rest = name.partition("@")
        tag, _, phase = rest.partition("#")
        kernels.append({"kernel": fam, "layer": tag2layer[tag].spec.name if tag in tag2layer else tag,
                        "launches": count, "total_ms": total_ms, "_tag": tag})
        phase_ms[(tag, phase)] = phase_ms.get((tag, phase), 0.0) + total_ms
    kernels.sort(key=lambda k: -k["total_ms"])
    all_ms = sum(k["total_ms"] for k in kernels) or 1.0
    for k in kernels:
        k["share"] = k["total_ms"] / all_ms

    def roofline_of(top):
        b = tag2layer.get(top["_tag"])
        kind = KIND_OF.get(top["kernel"])
        if b is None or not kind:
            return None
        # a pass that takes several launches of this kernel per step (one per residue class of a strided
        # backward pass) is judged as a whole: its algorithmic bytes and FLOPs are those of the pass
        per_step = max(1, round(top["launches"] / args.steps))
        dur = top["total_ms"] / top["launches"] * per_step * 1e-3
        fl = b.flops_per_phase() * (2 if kind == "bwd" else 1)
        by = kernel_bytes(kind, b.spec, (b.h_out, b.w_out))
        dense_bf16 = b.spec.dtype == "bf16" and b.spec.groups == 1
        traffic, traffic_from = NCU_TRAFFIC.get((top["kernel"], top["layer"]), (None, None))
        if dense_bf16 and fl / by > ridge:
            ach = fl / dur / 1e12
            r = {"bound": "tensor", "achieved": ach, "peak": tc, "unit": "TFLOP/s", "frac": ach / tc,
                 "traffic": traffic, "peak_source": "%s bf16 %s peak (clocks %s MHz of %s, reasons %s)"
                 % (peak_src, tc_kind, clocks.get("sm_mhz"), clocks.get("sm_max_mhz"), clocks.get("reasons")),
                 "frac_of_burst": ach / tc_burst, "frac_of_sustained": ach / tc_sus}
        else:
            ach = by / dur / 1e9
            r = {"bound": "hbm", "achieved": ach, "peak": hbm, "unit": "GB/s", "frac": ach / hbm,
                 "traffic": traffic, "peak_source": peak_src + " copy bandwidth"}
        r.update({"kernel": top["kernel"], "layer": top["layer"], "us_per_launch": dur * 1e6 / per_step,
                  "launches_per_step": per_step, "us_per_step": dur * 1e6, "algorithmic_bytes": by,
                  "algorithmic_flops": fl, "share_of_step": top["share"], "total_ms": top["total_ms"],
                  "traffic_from": traffic_from,
                  "timing": "CUDA-event pair around each launch on the launching stream, eager pass"})
        return r

    roofline = roofline_of(kernels[0]) if kernels else None
    # every layer and phase (all kernels of the call, weight re-layouts and epilogues included) against its
    # own roofline: the larger of FLOPs / tensor peak (dense bf16 only) and algorithmic bytes / copy bandwidth
    per_layer = []
    for (tag, phase), tot in sorted(phase_ms.items()):
        b = tag2layer.get(tag)
        kind = PHASE_KIND.get(phase)
        if b is None or kind is None:
            continue
        us = tot / args.steps * 1e3
        fl = b.flops_per_phase() * (2 if kind == "bwd" else 1)
        by = kernel_bytes(kind, b.spec, (b.h_out, b.w_out))
        t_hbm = by / (hbm * 1e9) * 1e6
        t_tc = fl / (tc * 1e12) * 1e6 if (b.spec.dtype == "bf16" and b.spec.groups == 1) else 0.0
        per_layer.append({"layer": b.spec.name, "phase": phase, "us": round(us, 2),
                          "bound": "tensor" if t_tc > t_hbm else "hbm", "roof_us": round(max(t_hbm, t_tc), 2),
                          "frac": round(max(t_hbm, t_tc) / us, 3) if us > 0 else None})
    launches_per_step = sum(k["launches"] for k in kernels) / float(args.steps)
    for k in kernels:
        k.pop("_tag")

    out = {"workload": WORKLOAD_NAMES[wl], "layers": [b.spec.name for b in blocks[0]],
           "ms_per_step": ms / args.steps, "ms_per_step_warm": ms_warm / args.steps,
           "tflops": whole_job_value(step_flops, args.steps, ms, world),
           "gbs_two_pass": world * two_pass_bytes * args.steps / (ms * 1e-3) / 1e9,
           "frac_of_copy_bandwidth": world * two_pass_bytes * args.steps / (ms * 1e-3) / 1e9 / hbm / world,
           "flops_per_step": step_flops, "two_pass_bytes_per_step": two_pass_bytes,
           "l2": "cold: %d rotating buffer sets of %.0f MB (activations) against an L2 of %.0f MB; warm: one set"
                 % (sets, footprint / 1e6, l2 / 1e6),
           "ms_per_step_other_orders": ms_other,
           "launch": launch_mode, "launches_per_step": launches_per_step, "host_us_per_call": round(host_us, 2),
           "eager_ms_per_step": eager_ms / args.steps, "clocks": clocks, "roofline": roofline,
           "kernels": kernels[:10], "per_layer": per_layer,
           "activation_bytes": {b.spec.name: {m: b.saved_bytes(m) for m in ("tune", "eval", "deploy")}
                                for b in blocks[0]}}
    if wl == 0:
        out["latency_us_per_step"] = ms / args.steps * 1e3
    gpu_launches = sum(k["launches"] for k in kernels)

    # ---- end to end through the host-buffer entry point ---------------------------------------
    e2e = None
    if not args.no_e2e:
        e2e = run_e2e(ctx, blocks[0], stream, step_flops)
        out["e2e"] = e2e
    del graphs
    blocks = [blocks[0]]
    torch.cuda.empty_cache()

    # ---- Tune against the Eval- and Deploy-mode paths built from the same kernels (the paper's comparison:
    # Table 2, Fig. 3), eager calls, forward + full backward of every layer per step; and the measured
    # allocator peak of a forward-hold-backward pass, Tune against Eval (Sec. 3.4, Appendix M)
    if not args.no_modes and rank == 0:
        mblocks = [Block(sp, device=dev, modes=("tune", "eval", "deploy")) for sp in layers]
        for li, b in enumerate(mblocks):
            b.randomize(I.config_seed(wl, li) + 17)
            b.deploy_prepare()

        def run_mode(m):
            for b in mblocks:
                if m == "tune":
                    b.tune_step()
                elif m == "eval":
                    b.eval_fwd(); b.eval_bwd()
                else:
                    b.deploy_fwd(); b.deploy_bwd()

        modes = {}
        ksteps = max(3, min(args.steps, 50))
        for m in ("tune", "eval", "deploy"):
            for _ in range(3):
                run_mode(m)
            torch.cuda.synchronize()
            m0, m1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            m0.record(stream)
            for _ in range(ksteps):
                run_mode(m)
            m1.record(stream)
            torch.cuda.synchronize()
            modes[m] = {"ms_per_step": m0.elapsed_time(m1) / ksteps,
                        "saved_bytes": sum(b.saved_bytes(m) for b in mblocks)}
        modes["note"] = "eager calls, %d steps each; saved_bytes = X plus what the mode keeps for backward (analytic)" % ksteps
        C.convbn_check()
        del mblocks
        torch.cuda.empty_cache()
        meas = {m: measured_activation_bytes(ctx, layers, m) for m in ("tune", "eval")}
        meas["note"] = ("torch.cuda.max_memory_allocated minus the bytes allocated before, over forward of every "
                        "layer then backward in reverse order; outputs, saved state and per-call scratch allocated inside")
        out["modes"] = modes
        out["activation_bytes_measured"] = meas
    del blocks, probe
    torch.cuda.empty_cache()

    # ---- CPU baseline (rank 0, single GPU only): the oracle as it stands, one full step of this config ----
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        times, fl, cores = oracle_step_time(wl, layers[0].n, 1)
        out["cpu_baseline"] = {"value": fl / times[0] / 1e12, "unit": UNIT, "cores": cores, "kind": "oracle",
                               "seconds": times[0], "flops": fl,
                               "sample": "one full step (all %d samples of every layer) of the fp64 oracle, %.1f s"
                                         % (layers[0].n, times[0])}
    out["_raw"] = {"ms": ms, "flops": step_flops, "gpu_launches": gpu_launches, "bytes": two_pass_bytes}
    return out


def run_e2e(ctx, blks, stream, step_flops):
    """The same step through convbn_tune_step_host: inputs in pinned host memory, every output
    copied back, copies inside the timed region."""
    args, torch, C, dev, world, dist = ctx.args, ctx.torch, ctx.C, ctx.dev, ctx.world, ctx.dist
    host = []
    h2d = d2h = 0
    for b in blks:
        pin = lambda t: None if t is None else t.detach().cpu().pin_memory()
        out = lambda t: None if t is None else torch.empty(t.shape, dtype=t.dtype).pin_memory()
        ins = [pin(t) for t in (b.x, b.dz, b.w, b.b, b.gamma, b.beta, b.mu_hat, b.var_hat)]
        outs = [out(t) for t in (b.z, b.dx, b.dw, b.db, b.dgamma, b.dbeta)]
        arena = torch.empty(C.convbn_host_step_arena_bytes(b.desc), dtype=torch.uint8, device=dev)
        host.append((b.desc, ins, outs, arena))
        h2d += sum(t.numel() * t.element_size() for t in ins if t is not None)
        d2h += sum(t.numel() * t.element_size() for t in outs if t is not None)

    def step():
        # every layer has its own arena: the next layer's inputs go up while this layer's results come down
        for desc, ins, outs, arena in host:
            C.convbn_tune_step_host_begin(desc, *ins, *outs, arena, stream=stream)
        C.convbn_tune_step_host_join(stream)

    steps = max(1, min(args.steps, args.e2e_steps))
    for _ in range(2):
        step()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(steps):
        step()
    e1.record(stream)
    torch.cuda.synchronize()
    ms = max_over_ranks(e0.elapsed_time(e1), dev)
    return {"value": world * step_flops * steps / (ms * 1e-3) / 1e12, "unit": UNIT,
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": steps,
            "ms_per_step": ms / steps}


BACKBONE_CASES = ((32, 224), (256, 224), (32, 448))


def run_backbones(ctx):
    return [run_backbone(ctx, b, s, iters=10 if b * s * s <= 32 * 224 * 224 else 4) for b, s in BACKBONE_CASES]


def run_backbone(ctx, batch=32, size=224, iters=10):
    """Forward + backward of all 53 ConvBN blocks of a ResNet-50 with their ReLUs and skip connections, in each
    mode: time per iteration and peak bytes above parameters, gradients and inputs (Sec. 3.4, Fig. 3)."""
    torch = ctx.torch
    from paper_2305_11624_b200.backbone import BackboneReplay, resnet50_plan
    stem, plan = resnet50_plan(size)
    out = {"network": "ResNet-50 ConvBN blocks + ReLU + skip connections (max-pool replaced by synthetic tensors)",
           "batch": batch, "image": size, "dtype": "bf16", "iters": iters, "modes": {}}
    for mode in ("tune", "eval", "deploy", "tune_async", "tune_f16", "eval_f16"):
        # tune_async: Tune mode with the parameter-gradient passes joined once per bottleneck instead of per call;
        # tune_f16, eval_f16: IEEE-half storage (the paper's mixed-precision rows)
        rp = BackboneReplay(batch, plan, mode.split("_")[0], stem_hw=stem, device=ctx.dev, async_param_grads=mode == "tune_async",
                            dtype="f16" if mode.endswith("_f16") else "bf16")
        try:
            ms, peak, how = rp.measure(iters=iters, warmup=3)
        except ctx.C.ConvBNError as exc:       # a layer shape that has no half path
            if not mode.endswith("_f16") or exc.status != ctx.C.EUNSUPPORTED:
                raise
            out["modes"][mode] = {"unsupported": str(exc)}
            del rp
            torch.cuda.empty_cache()
            continue
        out["modes"][mode] = {"ms_per_iter": ms, "peak_bytes": peak, "tflops": rp.flops / ms / 1e9, "timing": how}
        out["flops_per_iter"] = rp.flops
        out["conv_bn_blocks"] = len(rp.layers)
        del rp
        torch.cuda.empty_cache()
    m = out["modes"]
    out["tune_vs_eval"] = {"time": m["tune"]["ms_per_iter"] / m["eval"]["ms_per_iter"],
                           "peak_memory": m["tune"]["peak_bytes"] / m["eval"]["peak_bytes"]}
    return out


def run_ours(args):
    import torch
    import torch.distributed as dist
    import __graft_entry__ as G
    from paper_2305_11624_b200 import convbn as C
    from paper_2305_11624_b200 import inputs as I
    from paper_2305_11624_b200.harness import Block

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        G.build()
    if world > 1:
        dist.barrier()
    C.lib()
    ctx = Ctx()
    ctx.args, ctx.torch, ctx.C, ctx.I, ctx.Block, ctx.dist = args, torch, C, I, Block, dist
    ctx.dev, ctx.rank, ctx.world = dev, rank, world
    ctx.peaks, ctx.peak_src = load_peaks()

    workloads = [args.workload] if args.workload is not None else [0, 1, 2, 3, 4]
    per_config = [bench_config(ctx, wl) for wl in workloads]
    headline = [c for wl, c in zip(workloads, per_config) if wl in DENSE] or per_config
    raw = [c.pop("_raw") for c in per_config]
    hraw = [r for wl, r in zip(workloads, raw) if wl in DENSE] or raw
    ms_total = sum(r["ms"] for r in hraw)                       # K steps of every headline configuration
    flops_total = sum(r["flops"] for r in hraw)
    value = whole_job_value(flops_total, args.steps, ms_total, world)
    # the dominant kernel of the headline configurations: the one with the largest total time
    roofs = [c["roofline"] for c in headline if c.get("roofline")]
    roofline = max(roofs, key=lambda r: r["total_ms"]) if roofs else None
    e2e = None
    es = [c["e2e"] for c in headline if c.get("e2e")]
    if es:
        e2e_ms = sum(e["ms_per_step"] for e in es)
        e2e = {"value": world * flops_total / (e2e_ms * 1e-3) / 1e12, "unit": UNIT,
               "h2d_bytes_per_step": sum(e["h2d_bytes_per_step"] for e in es),
               "d2h_bytes_per_step": sum(e["d2h_bytes_per_step"] for e in es),
               "ms_per_step": e2e_ms, "steps": es[0]["steps"],
               "note": "convbn_tune_step_host_begin per layer (its own arena each) and one join per step: pinned host inputs up, every output down, inside the timed region"}
    cpu = None
    cs = [c["cpu_baseline"] for c in headline if c.get("cpu_baseline")]
    if cs:
        secs, fl = sum(c["seconds"] for c in cs), sum(c["flops"] for c in cs)
        cpu = {"value": fl / secs / 1e12, "unit": UNIT, "cores": cs[0]["cores"], "kind": "oracle",
               "sample": "one full step of every headline configuration of the fp64 oracle as it stands, %.1f s" % secs}
    backbone = None
    if rank == 0 and args.workload is None and not args.no_backbone:
        backbone = run_backbones(ctx)
    if world > 1:
        dist.barrier()
    if rank == 0:
        names = [WORKLOAD_NAMES[w] for w in workloads]
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_total / args.steps, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None,
                "dtype": "bf16" if any(w != 0 for w in workloads) else "f32", "data": "synthetic",
                "config": {"workload": "; ".join(names),
                           "value_over": "configs %s (dense bf16): total FLOPs / total time of one step of each"
                                         % ", ".join(str(w) for w in workloads if w in DENSE or len(workloads) == 1),
                           "l2": "inputs larger than L2: per configuration, rotating buffer sets that together exceed "
                                 "twice the L2 (see per_config[].l2); warm numbers beside them",
                           "flops_per_step": flops_total,
                           "parallelism": ("data parallel x%d, gradient all-reduce per step" if args.dp_allreduce and world > 1
                                           else "replicas x%d") % world,
                           "launch": headline[0]["launch"]},
                "clocks": merge_clocks([c["clocks"] for c in per_config]), "e2e": e2e,
                "gpu_launches": sum(r["gpu_launches"] for r in raw),
                "roofline": roofline, "cpu_baseline": cpu, "backbone": backbone, "per_config": per_config}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=None, choices=sorted(WORKLOAD_NAMES),
                    help="one configuration only (default: all five)")
    ap.add_argument("--buffer-sets", type=int, default=0, help="rotating buffer sets (0: enough to exceed twice the L2)")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--ref-batch", type=int, default=2, help="samples per step of the reference arm")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-modes", action="store_true", help="skip the Tune / Eval / Deploy comparison")
    ap.add_argument("--no-graph", action="store_true", help="time eager library calls instead of graph replays")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--order", default="layer", choices=["layer", "training"],
                    help="layer: forward then backward of each layer in turn; training: every forward call, then every "
                         "backward call")
    ap.add_argument("--join-per-layer", action="store_true",
                    help="every backward call joins its parameter-gradient pass before returning (default: one join per step)")
    ap.add_argument("--no-backbone", action="store_true", help="skip the whole-ResNet-50 replay in the three modes")
    ap.add_argument("--dp-allreduce", action="store_true",
                    help="with N > 1 ranks: sum the parameter gradients over the ranks every step (default: replicas)")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args))
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
