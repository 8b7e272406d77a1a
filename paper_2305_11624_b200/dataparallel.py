"""Data-parallel training of Tune-mode ConvBN blocks, and the search for Conv -> BN pairs in a model graph.

The path shards by batch: forward and dX need no exchange; the parameter gradients (d omega, db, d gamma,
d beta: Table 2, Tune row) are sums over samples, so one sum all-reduce per bucket of layers finishes them.
The running statistics are frozen in Tune mode (Sec. 3.1), so nothing else crosses ranks - unlike Train mode
there is no statistics exchange.  `GradientBucket` owns ONE contiguous fp32 buffer that the layers' gradient
tensors are views of, so the collective is a single call on memory the kernels wrote directly (no packing
copy); `all_reduce_async` issues it on a side stream after the producing stream's work so that the next
layer's backward kernels overlap it.  torch.distributed does the plumbing (NCCL on GPUs, gloo on CPU).

`find_conv_bn_pairs` is the graph-level helper that replaces the paper's traced-graph pattern match (Sec. 3,
App. N): given the operator graph of a model it returns the (convolution, BatchNorm) pairs that may run as
one Tune-mode block - consecutive, the convolution feeding nothing else, the BatchNorm using tracked
statistics - and works on a plain node list, so it needs no tracing compiler.
"""
from dataclasses import dataclass, field
from typing import Dict, Iterable, List, Optional, Sequence, Tuple

import torch
import torch.distributed as dist


class GradientBucket:
    """Parameter gradients of several layers in one fp32 buffer: `views[name]` are the tensors to hand to
    convbn_tune_bwd / convbn_tune_bwd_weight as dw, db, dgamma, dbeta."""

    def __init__(self, sizes: Dict[str, int], device="cuda"):
        self.device = torch.device(device)
        self.offsets, off = {}, 0
        for name, n in sizes.items():
            self.offsets[name] = (off, int(n))
            off += (int(n) + 63) // 64 * 64                  # 256-byte aligned views (the library wants 16)
        self.flat = torch.zeros(max(off, 64), dtype=torch.float32, device=self.device)
        self.views = {name: self.flat[o:o + n] for name, (o, n) in self.offsets.items()}
        self._stream = torch.cuda.Stream(device=self.device) if self.device.type == "cuda" else None
        self._done = torch.cuda.Event() if self._stream is not None else None
        self._work = None

    @staticmethod
    def sizes_for(layers: Sequence[Tuple[str, int, int, bool]]) -> Dict[str, int]:
        """layers: (name, C_out, weight elements per output channel, has conv bias)."""
        out = {}
        for name, c_out, kdim, bias in layers:
            out[name + ".dw"] = c_out * kdim
            if bias:
                out[name + ".db"] = c_out
            out[name + ".dgamma"] = c_out
            out[name + ".dbeta"] = c_out
        return out

    def all_reduce(self, group=None, average: bool = False):
        """Sum (or mean) over the ranks, in place, synchronous with respect to the current stream."""
        if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
            dist.all_reduce(self.flat, op=dist.ReduceOp.SUM, group=group)
            if average:
                self.flat.div_(dist.get_world_size(group))
        return self.flat

    def all_reduce_async(self, group=None):
        """Issue the all-reduce on the bucket's side stream once the current stream's queued kernels (which write
        the gradients) are done; kernels queued on the current stream afterwards overlap it.  wait() joins."""
        if self._stream is None:
            self._work = None
            return self.all_reduce(group)
        ready = torch.cuda.Event()
        ready.record(torch.cuda.current_stream(self.device))
        self._stream.wait_event(ready)
        with torch.cuda.stream(self._stream):
            if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
                dist.all_reduce(self.flat, op=dist.ReduceOp.SUM, group=group)
            self._done.record(self._stream)
        return self.flat

    def wait(self):
        if self._done is not None:
            torch.cuda.current_stream(self.device).wait_event(self._done)


# ---- Conv -> BN pairs ---------------------------------------------------------------------------------
CONV_OPS = ("conv2d", "linear", "conv_transpose2d")
BN_OPS = ("batch_norm",)


@dataclass
class Node:
    """One operator of a model graph: `inputs` are the names of the nodes whose outputs it reads."""
    name: str
    op: str
    inputs: Tuple[str, ...] = ()
    attrs: dict = field(default_factory=dict)      # batch_norm: {"tracked_stats": bool, "training": bool}


def find_conv_bn_pairs(nodes: Iterable[Node]) -> List[Tuple[str, str]]:
    """(conv name, bn name) for every BatchNorm that reads exactly one convolution-like node (conv2d, linear,
    transposed conv: Sec. 3.2.2) whose output nothing else reads, and that normalises with tracked statistics
    (Eval / Tune semantics: not in training mode, statistics tracked).  Order follows the node list."""
    nodes = list(nodes)
    by_name = {n.name: n for n in nodes}
    consumers: Dict[str, int] = {}
    for n in nodes:
        for i in n.inputs:
            consumers[i] = consumers.get(i, 0) + 1
    pairs = []
    for n in nodes:
        if n.op not in BN_OPS or len(n.inputs) != 1:
            continue
        if n.attrs.get("training", False) or not n.attrs.get("tracked_stats", True):
            continue
        src = by_name.get(n.inputs[0])
        if src is None or src.op not in CONV_OPS or consumers.get(src.name, 0) != 1:
            continue
        pairs.append((src.name, n.name))
    return pairs


def nodes_of_sequential(modules: Sequence[Tuple[str, "torch.nn.Module"]], first_input: str = "input") -> List[Node]:
    """Node list of modules applied one after the other (an nn.Sequential's named children)."""
    import torch.nn as nn
    out, prev = [], first_input
    for name, m in modules:
        if isinstance(m, nn.Conv2d):
            op, attrs = "conv2d", {}
        elif isinstance(m, nn.ConvTranspose2d):
            op, attrs = "conv_transpose2d", {}
        elif isinstance(m, nn.Linear):
            op, attrs = "linear", {}
        elif isinstance(m, (nn.BatchNorm1d, nn.BatchNorm2d)):
            op, attrs = "batch_norm", {"training": m.training, "tracked_stats": m.track_running_stats}
        else:
            op, attrs = type(m).__name__.lower(), {}
        out.append(Node(name, op, (prev,), attrs))
        prev = name
    return out
