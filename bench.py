#!/usr/bin/env python
"""Benchmark of the Tune-mode ConvBN hot path on B200.

A step is one pass of the whole path - convbn_tune_fwd, convbn_tune_bwd_data and
convbn_tune_bwd_weight - over every layer of the workload (default: the ResNet-50 stage-2
bottleneck chain, bf16 NHWC, N=32 at 56x56).  The metric is fwd+bwd TFLOP/s with
FLOPs = 3 phases x 2 P C_out (C_in/G) kh kw per layer.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload 1]

Under torchrun every rank runs its own replica of the workload on its own batch (the path needs
no exchange between samples), times it with CUDA events, and rank 0 prints one JSON line with the
max-over-ranks time.  ``--impl reference`` times the fp64 CPU oracle instead (rank 0 only).
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
    raise KeyError(kind)


# DRAM bytes (read + write) per launch from the ncu capture summarised in
# profiles/config1_gemm_kernels_ncu_full.md; None for kernels changed or not captured since.
NCU_TRAFFIC = {("umma_fwd", "c1a"): 51.71e6, ("umma_dgrad", "c1a"): 13.80e6, ("umma_wgrad", "c1a"): 65.09e6,
               ("strip_fwd", "c1b"): 12.96e6, ("strip_dgrad", "c1b"): 12.96e6, ("umma_wgrad", "c1b"): 25.71e6,
               ("umma_fwd", "c1c"): 13.86e6, ("umma_dgrad", "c1c"): 51.94e6, ("umma_wgrad", "c1c"): 65.54e6,
               ("dw_fwd", "c4a"): 262.4e6, ("dw_dgrad", "c4a"): 261.0e6, ("dw_wgrad", "c4a"): 312.3e6,
               ("grouped_dgrad", "c4b"): 29.1e6, ("grouped_wgrad", "c4b"): 51.8e6,
               ("stem_dgrad", "c2s"): 109.5e6}

KIND_OF = {"strip_fwd": "fwd", "strip_dgrad": "dgrad", "direct_fwd": "fwd", "direct_dgrad": "dgrad", "direct_wgrad": "wgrad",
           "umma_fwd": "fwd", "umma_dgrad": "dgrad", "umma_wgrad": "wgrad",
           "dw_fwd": "fwd", "dw_dgrad": "dgrad", "dw_wgrad": "wgrad",
           "grouped_fwd": "fwd", "grouped_dgrad": "dgrad", "grouped_wgrad": "wgrad",
           "stem_fwd": "fwd", "stem_dgrad": "dgrad", "stem_wgrad": "wgrad"}


def shape_tag(spec):
    return "n%d_c%d_%dx%d_o%d_k%dx%d_s%d_g%d" % (spec.n, spec.c_in, spec.h_in, spec.w_in, spec.c_out,
                                                 spec.kh, spec.kw, spec.stride, spec.groups)


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU through NVML (read-only) while running."""

    def __init__(self, uuid, period=0.01):
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
    times, flops, cores = oracle_step_time(args.workload, batch, args.warmup + args.steps)
    timed = times[args.warmup:]
    per = sum(timed) / len(timed)
    val = flops / per / 1e12
    sample = "fp64 oracle, Tune fwd+bwd of every layer of the workload on a batch of %d samples per step" % batch
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": per * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": WORKLOAD_NAMES[args.workload], "sample": sample},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ---- the CUDA path ------------------------------------------------------------------------------
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

    layers = I.CONFIGS[args.workload]
    sets = max(1, args.buffer_sets)
    blocks = [[Block(sp, device=dev) for sp in layers] for _ in range(sets)]
    for si, bs in enumerate(blocks):
        for li, b in enumerate(bs):
            b.randomize(I.config_seed(args.workload, li) + 7919 * (rank * sets + si))
    step_flops = sum(3 * b.flops_per_phase() for b in blocks[0])
    footprint = sum(t.numel() * t.element_size() for b in blocks[0] for t in (b.x, b.dz, b.z, b.dx))

    stream = torch.cuda.current_stream()

    def step(i):
        for b in blocks[i % sets]:
            b.tune_step(stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        step(i)
    C.convbn_check()
    barrier()
    uuid = str(torch.cuda.get_device_properties(dev).uuid)
    sampler = ClockSampler(uuid if uuid.startswith("GPU-") else "GPU-" + uuid)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    # ---- timed region: K steps, each a replay of the CUDA graph of one step (one graph per buffer
    # set), so the layers' ~15 launches per step cost no host time; --no-graph times eager calls.
    graphs, launch_mode = None, "eager library calls"
    if not args.no_graph:
        try:
            graphs = []
            for si in range(sets):
                gr = torch.cuda.CUDAGraph()
                with torch.cuda.graph(gr):
                    for b in blocks[si]:
                        b.tune_step()
                graphs.append(gr)
            for gr in graphs:
                gr.replay()
            torch.cuda.synchronize()
            launch_mode = "CUDA graph replay (one captured step per buffer set)"
        except Exception as exc:  # capture unsupported: say so and time eager calls
            graphs, launch_mode = None, "eager library calls (graph capture failed: %r)" % (exc,)
    barrier()
    e0.record(stream)
    for i in range(args.steps):
        if graphs:
            graphs[(args.warmup + i) % sets].replay()
        else:
            step(args.warmup + i)
    e1.record(stream)
    barrier()
    ms = max_over_ranks(e0.elapsed_time(e1), dev)
    value = whole_job_value(step_flops, args.steps, ms, world)

    # ---- second pass, same K steps as eager calls with a CUDA-event pair around every kernel: the
    # per-kernel durations behind the roofline object (events cannot be read back out of a graph)
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    C.convbn_profile_begin()
    barrier()
    f0.record(stream)
    for i in range(args.steps):
        step(args.warmup + i)
    f1.record(stream)
    barrier()
    prof = C.convbn_profile_end()
    eager_ms = max_over_ranks(f0.elapsed_time(f1), dev)
    sampler.stop_flag.set()
    sampler.join()
    C.convbn_check()

    # ---- roofline of the dominant kernel -----------------------------------------------------
    peaks, peak_src = load_peaks()
    tag2layer = {shape_tag(b.spec): b for b in blocks[0]}
    kernels = []
    phase_ms = {}                                    # (layer tag, phase) -> milliseconds over the eager pass
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
    roofline = None
    if kernels:
        top = kernels[0]
        b = tag2layer.get(top["_tag"])
        kind = KIND_OF.get(top["kernel"])
        # a pass that takes several launches of this kernel per step (one per residue class of a strided
        # backward pass) is judged as a whole: its algorithmic bytes and FLOPs are those of the pass
        per_step = max(1, round(top["launches"] / args.steps))
        dur = top["total_ms"] / top["launches"] * per_step * 1e-3
        if b is not None and kind:
            fl = b.flops_per_phase()
            by = kernel_bytes(kind, b.spec, (b.h_out, b.w_out))
            hbm, tc = peaks["hbm_gbs"], peaks["bf16_tflops_sustained"]
            dense_bf16 = b.spec.dtype == "bf16" and b.spec.groups == 1
            tensor_bound = dense_bf16 and (fl / by) > (tc * 1e12) / (hbm * 1e9)
            if tensor_bound:
                ach = fl / dur / 1e12
                roofline = {"bound": "tensor", "achieved": ach, "peak": tc, "unit": "TFLOP/s",
                            "frac": ach / tc, "traffic": NCU_TRAFFIC.get((top["kernel"], top["layer"])),
                            "peak_source": peak_src + " bf16 sustained (kernel timed inside a long step)"}
            else:
                ach = by / dur / 1e9
                roofline = {"bound": "hbm", "achieved": ach, "peak": hbm, "unit": "GB/s",
                            "frac": ach / hbm, "traffic": NCU_TRAFFIC.get((top["kernel"], top["layer"])),
                            "peak_source": peak_src + " copy bandwidth"}
            roofline.update({"kernel": top["kernel"], "layer": top["layer"], "us_per_launch": dur * 1e6 / per_step,
                             "launches_per_step": per_step, "us_per_step": dur * 1e6,
                             "algorithmic_bytes": by, "algorithmic_flops": fl, "share_of_step": top["share"]})
    for k in kernels:
        k.pop("_tag")
    # every layer and phase (all kernels of the call, weight re-layouts and epilogues included) against its
    # own roofline: the larger of FLOPs / tensor peak (dense bf16 only) and algorithmic bytes / copy bandwidth
    per_layer = []
    hbm, tc = peaks["hbm_gbs"], peaks["bf16_tflops_sustained"]
    for (tag, phase), tot in sorted(phase_ms.items()):
        b = tag2layer.get(tag)
        kind = {"fwd": "fwd", "bwd_data": "dgrad", "bwd_weight": "wgrad"}.get(phase)
        if b is None or kind is None:
            continue
        us = tot / args.steps * 1e3
        fl, by = b.flops_per_phase(), kernel_bytes(kind, b.spec, (b.h_out, b.w_out))
        t_hbm = by / (hbm * 1e9) * 1e6
        t_tc = fl / (tc * 1e12) * 1e6 if (b.spec.dtype == "bf16" and b.spec.groups == 1) else 0.0
        per_layer.append({"layer": b.spec.name, "phase": phase, "us": round(us, 2),
                          "bound": "tensor" if t_tc > t_hbm else "hbm", "roof_us": round(max(t_hbm, t_tc), 2),
                          "frac": round(max(t_hbm, t_tc) / us, 3) if us > 0 else None})

    # ---- Tune against the Eval- and Deploy-mode paths built from the same kernels (the paper's
    # comparison: Table 2, Fig. 3), eager calls, forward + full backward of every layer per step
    modes = None
    if not args.no_modes and rank == 0:
        mblocks = [Block(sp, device=dev, modes=("tune", "eval", "deploy")) for sp in layers]
        for li, b in enumerate(mblocks):
            b.randomize(I.config_seed(args.workload, li) + 17)
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
        modes["note"] = "eager calls, %d steps each; saved_bytes = X plus what the mode keeps for backward" % ksteps
        C.convbn_check()
        del mblocks

    # ---- end to end through the host-buffer entry point ---------------------------------------
    e2e = None
    if not args.no_e2e:
        e2e = run_e2e(args, torch, C, blocks[0], dev, stream, world, step_flops)

    # ---- CPU baseline (rank 0, single GPU only) ------------------------------------------------
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        full = layers[0].n
        times, fl, cores = oracle_step_time(args.workload, full, 2)  # ~2 x 3 s on 16 cores
        cpu = {"value": fl / min(times) / 1e12, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": "one full step (all %d samples of every layer) of the fp64 oracle, best of 2, %.1f s"
                         % (full, min(times))}

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None,
                "dtype": "bf16" if layers[0].dtype == "bf16" else "f32", "data": "synthetic",
                "config": {"workload": WORKLOAD_NAMES[args.workload],
                           "layers": [b.spec.name for b in blocks[0]],
                           "l2": "step footprint %.0f MB of activations > L2; %d rotating buffer sets"
                                 % (footprint / 1e6, sets),
                           "flops_per_step": step_flops, "parallelism": "replicas x%d" % world,
                           "launch": launch_mode},
                "eager": {"ms_per_step": eager_ms / args.steps,
                          "value": world * step_flops * args.steps / (eager_ms * 1e-3) / 1e12,
                          "note": "same steps as plain library calls with per-kernel CUDA events (source of `kernels` and `roofline`)"},
                "clocks": sampler.summary(), "e2e": e2e,
                "gpu_launches": sum(k["launches"] for k in kernels),
                "roofline": roofline, "cpu_baseline": cpu, "modes": modes, "kernels": kernels[:12], "per_layer": per_layer,
                "activation_bytes": {b.spec.name: {m: b.saved_bytes(m) for m in ("tune", "eval", "deploy")}
                                     for b in blocks[0]}}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_e2e(args, torch, C, blks, dev, stream, world, step_flops):
    """The same step through convbn_tune_step_host: inputs in pinned host memory, every output
    copied back, copies inside the timed region."""
    import torch.distributed as dist
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
        for desc, ins, outs, arena in host:
            C.convbn_tune_step_host(desc, *ins, *outs, arena, stream=stream)

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
    ms = e0.elapsed_time(e1)
    if world > 1:
        t = torch.tensor([ms], device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    return {"value": world * step_flops * steps / (ms * 1e-3) / 1e12, "unit": UNIT,
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": steps,
            "ms_per_step": ms / steps}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=1, choices=sorted(WORKLOAD_NAMES))
    ap.add_argument("--buffer-sets", type=int, default=2)
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--ref-batch", type=int, default=4, help="samples per step of the reference arm")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-modes", action="store_true", help="skip the Tune / Eval / Deploy comparison")
    ap.add_argument("--no-graph", action="store_true", help="time eager library calls instead of graph replays")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
