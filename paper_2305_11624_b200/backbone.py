"""Whole-backbone replay: forward + backward of a ResNet-50-shaped chain of ConvBN blocks in Tune, Eval or Deploy mode.

This is the shape of the paper's efficiency experiment (Sec. 3.4, Fig. 3, App. D: time per iteration and peak
memory of a ResNet-50 under the three modes) with synthetic weights and inputs: the 53 ConvBN blocks of the
network (stem, 16 bottlenecks of three convolutions, four projection shortcuts), ReLU after every block but the
last of a bottleneck, the skip connection and its ReLU at the end of each bottleneck.  Every ConvBN block, every
ReLU and every add runs through `libconvbn.so`; this module only owns buffers and the order of the calls.

What is kept from forward to backward is what a framework would keep: each convolution's input (the previous
ReLU's output), the mode's extra state (Tune: three vectors per block; Eval: the pre-normalisation tensor Y of
every block; Deploy: nothing), and nothing else.  Buffers are allocated with torch inside the pass and dropped
as soon as the backward pass has used them, so `torch.cuda.max_memory_allocated` sees the peak a training
framework would see.

The max-pool between the stem and the first stage is not a ConvBN block and has no counterpart in the library:
the first stage is fed with a synthetic tensor of the pooled shape and the stem's backward pass with a synthetic
gradient (one cheap operator out of ~170 is missing from the timed pass).
"""
import math
from dataclasses import dataclass
from typing import List, Optional, Tuple

import torch

from . import convbn as C
from . import inputs as I
from .harness import Block


@dataclass
class Bottleneck:
    c_in: int
    width: int
    c_out: int
    stride: int          # of the 3x3 convolution (and of the projection shortcut)
    hw: Tuple[int, int]  # input extent


def resnet50_plan(size: int = 224) -> Tuple[Optional[Tuple[int, int]], List[Bottleneck]]:
    """(stem input extent, bottlenecks) of a ResNet-50 for `size` x `size` images."""
    h = size // 4                     # after the stride-2 stem and the stride-2 max-pool
    plan, c_in = [], 64
    for width, blocks, stride in ((64, 3, 1), (128, 4, 2), (256, 6, 2), (512, 3, 2)):
        for b in range(blocks):
            s = stride if b == 0 else 1
            plan.append(Bottleneck(c_in, width, 4 * width, s, (h, h)))
            h //= s
            c_in = 4 * width
    return (size, size), plan


class _Layer:
    """One ConvBN block of the chain: parameters, gradients, the calls of the chosen mode."""

    def __init__(self, name, n, c_in, hw, c_out, k, stride, mode, device, seed, dtype="bf16"):
        spec = I.LayerSpec(name, n, c_in, hw[0], hw[1], c_out, k, k, stride=stride, pad=k // 2, dtype=dtype)
        self.blk = Block(spec, device=device, modes=(mode,), allocate="params")
        self.blk.randomize_params(seed)
        self.mode = mode
        if mode == "deploy":
            b = self.blk
            b.w_fused = torch.empty_like(b.w)
            b.b_fused = torch.empty(spec.c_out, dtype=torch.float32, device=device)
            b.dw_fused = torch.empty_like(b.dw)
            b.db_fused = torch.empty(spec.c_out, dtype=torch.float32, device=device)
            b.deploy_prepare()
        self.out_elems = n * c_out * self.blk.h_out * self.blk.w_out
        self.in_elems = n * c_in * hw[0] * hw[1]

    def forward(self, x):
        b = self.blk
        b.x = x
        b.z = torch.empty(self.out_elems, dtype=b.tdtype, device=b.device)
        if self.mode == "tune":
            b.saved = torch.empty(max(16, C.convbn_saved_bytes(b.desc, C.MODE_TUNE)), dtype=torch.uint8, device=b.device)
            b.with_scratch(C.PHASE_TUNE_FWD, b.tune_fwd)
        elif self.mode == "eval":
            b.y_saved = torch.empty(C.convbn_saved_bytes(b.desc, C.MODE_EVAL), dtype=torch.uint8, device=b.device)
            b.with_scratch(C.PHASE_EVAL_FWD, b.eval_fwd)
        else:
            b.with_scratch(C.PHASE_DEPLOY_FWD, b.deploy_fwd)
        z, b.z = b.z, None
        return z

    def backward(self, dz, held=None):
        """Gradient with respect to the block's input; drops what the block kept for it.  With `held` (a list, Tune
        mode) the parameter-gradient pass stays on the library's side stream: what it still reads (dZ, X, the saved
        vectors, the scratch) is parked in `held` until the caller has joined."""
        b = self.blk
        b.dz = dz
        b.dx = torch.empty(self.in_elems, dtype=b.tdtype, device=b.device)
        if self.mode == "tune" and held is not None:
            b.workspace = torch.empty(max(256, C.convbn_workspace_bytes(b.desc, C.PHASE_TUNE_BWD)), dtype=torch.uint8,
                                      device=b.device)
            b.tune_bwd_begin()
            held.append((b.workspace, b.saved, b.x, b.dz))
            b.workspace = b.saved = None
        elif self.mode == "tune":
            b.with_scratch(C.PHASE_TUNE_BWD, b.tune_bwd)
            b.saved = None
        elif self.mode == "eval":
            b.with_scratch(C.PHASE_EVAL_BWD, b.eval_bwd)
            b.y_saved = None
        else:
            b.with_scratch(C.PHASE_DEPLOY_BWD, b.deploy_bwd)
        dx, b.dx, b.dz, b.x = b.dx, None, None, None
        return dx


class BackboneReplay:
    def __init__(self, batch: int, plan: List[Bottleneck], mode: str, stem_hw: Optional[Tuple[int, int]] = None,
                 device="cuda:0", seed: int = 0, async_param_grads: bool = False, dtype: str = "bf16"):
        assert mode in ("tune", "eval", "deploy") and dtype in ("bf16", "f16")
        self.async_param_grads = async_param_grads
        self.mode, self.batch, self.device = mode, batch, torch.device(device)
        self.dtype = torch.bfloat16 if dtype == "bf16" else torch.float16
        n, k = batch, seed
        self.stem = None
        if stem_hw is not None:
            self.stem = _Layer("stem", n, 3, stem_hw, 64, 7, 2, mode, device, k, dtype)
            k += 1
        self.blocks = []
        for i, bt in enumerate(plan):
            hw2 = bt.hw
            hw3 = (bt.hw[0] // bt.stride, bt.hw[1] // bt.stride) if bt.stride > 1 else bt.hw
            if bt.stride > 1:      # floor convention of a 3x3 stride-2 pad-1 convolution
                hw3 = ((bt.hw[0] - 1) // bt.stride + 1, (bt.hw[1] - 1) // bt.stride + 1)
            c1 = _Layer("b%d.c1" % i, n, bt.c_in, bt.hw, bt.width, 1, 1, mode, device, k, dtype)
            c2 = _Layer("b%d.c2" % i, n, bt.width, hw2, bt.width, 3, bt.stride, mode, device, k + 1, dtype)
            c3 = _Layer("b%d.c3" % i, n, bt.width, hw3, bt.c_out, 1, 1, mode, device, k + 2, dtype)
            ds = None
            if bt.stride > 1 or bt.c_in != bt.c_out:
                ds = _Layer("b%d.ds" % i, n, bt.c_in, bt.hw, bt.c_out, 1, bt.stride, mode, device, k + 3, dtype)
            k += 4
            self.blocks.append((c1, c2, c3, ds))
        self.first = plan[0]
        self.layers = ([self.stem] if self.stem else []) + [l for blk in self.blocks for l in blk if l is not None]
        self.flops = sum(3 * l.blk.flops_per_phase() for l in self.layers)

    # ---- one iteration ---------------------------------------------------------------------------------
    def make_inputs(self, seed: int = 1):
        g = torch.Generator(device=self.device)
        g.manual_seed(seed)
        rn = lambda n: torch.randn(n, generator=g, device=self.device).to(self.dtype)
        bt = self.first
        ins = {"x": rn(self.batch * bt.c_in * bt.hw[0] * bt.hw[1]).abs_()}      # a ReLU output feeds the first stage
        last = self.blocks[-1][2]
        ins["g"] = rn(last.out_elems)
        if self.stem:
            ins["image"] = rn(self.stem.in_elems)
            ins["g_stem"] = rn(self.stem.out_elems)
        return ins

    def forward_backward(self, ins, keep=None):
        """One training iteration.  `keep` (a dict) receives the network output, the input gradient and copies of
        every ReLU output (whose signs are the decisions a comparison has to share)."""
        relu_outs = []
        if self.stem:
            s = self.stem.forward(ins["image"])
            C.convbn_relu(s, s)
        x = ins["x"]
        for c1, c2, c3, ds in self.blocks:
            a = c1.forward(x); C.convbn_relu(a, a)
            b = c2.forward(a); C.convbn_relu(b, b)
            c = c3.forward(b)
            idt = ds.forward(x) if ds is not None else x
            C.convbn_add_relu(c, idt, c)                       # out = relu(c + idt), in place in c's buffer
            relu_outs.append((x, a, b, c))
            if keep is not None:
                keep.setdefault("relu_outputs", []).append((a.clone(), b.clone(), c.clone()))
            x = c
            del idt
        if keep is not None:
            keep["out"] = x.clone()
        g = ins["g"].clone()
        # Tune mode: the parameter gradients of a bottleneck's blocks run beside its input-gradient chain and are
        # joined once per bottleneck, after which what they were reading can be released
        held = [] if self.mode == "tune" and self.async_param_grads else None
        for (c1, c2, c3, ds), (xin, a, b, out) in zip(reversed(self.blocks), reversed(relu_outs)):
            C.convbn_relu_bwd(g, out, g)                       # through the block's final ReLU; g feeds both branches
            gb = c3.backward(g, held); C.convbn_relu_bwd(gb, b, gb)
            ga = c2.backward(gb, held); C.convbn_relu_bwd(ga, a, ga)
            gx = c1.backward(ga, held)
            if ds is not None:
                gs = ds.backward(g, held)
                C.convbn_add(gx, gs, gx)
                del gs
            else:
                C.convbn_add(gx, g, gx)
            if held is not None:
                C.convbn_tune_bwd_join()
                held.clear()
            g = gx
            del gb, ga
        relu_outs.clear()
        if keep is not None:
            keep["dx"] = g.clone()
        if self.stem:
            gs = ins["g_stem"].clone()
            C.convbn_relu_bwd(gs, s, gs)
            gi = self.stem.backward(gs)
            if keep is not None:
                keep["d_image"] = gi.clone()
        return g

    # ---- measurements ------------------------------------------------------------------------------------
    def measure(self, iters: int = 5, warmup: int = 2):
        """(milliseconds per iteration from a CUDA-graph replay, peak bytes of one eager iteration above the
        bytes held before it: parameters, gradients and inputs)."""
        dev = self.device
        ins = self.make_inputs()
        for _ in range(warmup):
            self.forward_backward(ins)
        C.convbn_check()
        torch.cuda.synchronize(dev)
        torch.cuda.reset_peak_memory_stats(dev)
        base = torch.cuda.memory_allocated(dev)
        self.forward_backward(ins)
        torch.cuda.synchronize(dev)
        peak = torch.cuda.max_memory_allocated(dev) - base
        mode = "CUDA graph replay"
        try:
            gr = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gr):
                self.forward_backward(ins)
            run = gr.replay
            run(); torch.cuda.synchronize(dev)
        except Exception as exc:          # capture unsupported: time eager calls and say so
            run, mode = (lambda: self.forward_backward(ins)), "eager calls (graph capture failed: %r)" % (exc,)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(iters):
            run()
        e1.record()
        torch.cuda.synchronize(dev)
        C.convbn_check()
        return e0.elapsed_time(e1) / iters, int(peak), mode
