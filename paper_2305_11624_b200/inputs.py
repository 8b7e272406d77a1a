"""Seeded synthetic inputs for ConvBN blocks, and the layer shapes of the benchmark configs.

This module holds no arithmetic of the method: it only draws numbers, rounds them to the
storage type and lays them out.  Both the CUDA path and the CPU checker are fed from here, so
that they see the same bit patterns.

Random numbers come from a counter-based generator: element ``i`` of tensor ``tag`` under
``seed`` is a pure function of ``(seed, tag, i)`` (SplitMix64 finaliser over a 64-bit counter),
so a tensor's values do not depend on which other tensors were drawn, nor on chunking.

Value distributions (one recipe for every config; second argument of N is the standard
deviation):
    x ~ N(0,1)          w ~ N(0, sqrt(2/fan_in)), fan_in = (C_in/G) kh kw   (Kaiming normal)
    b ~ N(0,0.01)       mu_hat ~ N(0,0.1)      var_hat ~ U(0.5,2)
    gamma ~ U(0.5,1.5)  beta ~ N(0,0.1)        dz ~ N(0,1)                  eps = 1e-5
Tensors are generated in fp32 in logical NCHW index order, then rounded (RNE) to bf16 where
the layer's storage type is bf16; per-channel vectors always stay fp32.
"""
from dataclasses import dataclass
from typing import Dict, Optional, Tuple

import numpy as np

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)
_TAGS = {"x": 1, "w": 2, "b": 3, "mu_hat": 4, "var_hat": 5, "gamma": 6, "beta": 7, "dz": 8}


def _splitmix64(z: np.ndarray) -> np.ndarray:
    """SplitMix64 output function (Steele, Lea, Flood 2014) applied elementwise to uint64."""
    with np.errstate(over="ignore"):
        z = (z + np.uint64(0x9E3779B97F4A7C15)) & _M64
        z = ((z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)) & _M64
        z = ((z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)) & _M64
        return z ^ (z >> np.uint64(31))


def _bits(seed: int, tag: int, lane: int, start: int, count: int) -> np.ndarray:
    with np.errstate(over="ignore"):
        key = _splitmix64(np.array([(seed * 0x1000193 + tag * 16 + lane) & 0xFFFFFFFFFFFFFFFF],
                                   dtype=np.uint64))[0]
        ctr = np.arange(start, start + count, dtype=np.uint64)
        return _splitmix64(ctr ^ key)


def uniform01(seed: int, tag: int, count: int, lane: int = 0, start: int = 0) -> np.ndarray:
    """count doubles in (0, 1): (top 53 bits + 0.5) / 2^53."""
    b = _bits(seed, tag, lane, start, count)
    return ((b >> np.uint64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def normal(seed: int, tag: int, count: int) -> np.ndarray:
    """count standard normals (Box-Muller on two independent uniform lanes), float32."""
    out = np.empty(count, dtype=np.float32)
    step = 1 << 22
    for s0 in range(0, count, step):
        c = min(step, count - s0)
        u1 = uniform01(seed, tag, c, lane=0, start=s0)
        u2 = uniform01(seed, tag, c, lane=1, start=s0)
        out[s0:s0 + c] = (np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)).astype(np.float32)
    return out


def uniform(seed: int, tag: int, count: int, lo: float, hi: float) -> np.ndarray:
    return (lo + (hi - lo) * uniform01(seed, tag, count)).astype(np.float32)


# ---- bf16 storage -------------------------------------------------------------------------

def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16, returned as uint16 bit patterns (finite inputs)."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rnd = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + rnd) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def round_bf16(a: np.ndarray) -> np.ndarray:
    """fp32 array holding the bf16-representable values nearest to ``a``."""
    return bf16_bits_to_f32(f32_to_bf16_bits(a)).reshape(np.shape(a))


# ---- layer shapes -------------------------------------------------------------------------

@dataclass(frozen=True)
class LayerSpec:
    """One ConvBN layer: sizes, storage type (``"f32"``/``"bf16"``/``"f16"``), memory layout
    (``"nchw"``/``"nhwc"``) and whether the convolution has a bias."""
    name: str
    n: int
    c_in: int
    h_in: int
    w_in: int
    c_out: int
    kh: int
    kw: int
    stride: int = 1
    pad: int = 0
    dil: int = 1
    groups: int = 1
    dtype: str = "bf16"
    layout: str = "nhwc"
    bias: bool = False
    eps: float = 1e-5

    def dims(self) -> Dict[str, int]:
        return dict(n=self.n, c_in=self.c_in, h_in=self.h_in, w_in=self.w_in, c_out=self.c_out,
                    kh=self.kh, kw=self.kw, stride_h=self.stride, stride_w=self.stride,
                    pad_h=self.pad, pad_w=self.pad, dil_h=self.dil, dil_w=self.dil,
                    groups=self.groups)


# The five benchmark configurations, as lists of layers.
CONFIGS: Dict[int, Tuple[LayerSpec, ...]] = {
    # single block, fp32 NCHW, with conv bias
    0: (LayerSpec("c0", 2, 16, 16, 16, 32, 3, 3, pad=1, dtype="f32", layout="nchw", bias=True),),
    # ResNet-50 stage-2 bottleneck chain, N=32 at 56x56
    1: (LayerSpec("c1a", 32, 256, 56, 56, 64, 1, 1),
        LayerSpec("c1b", 32, 64, 56, 56, 64, 3, 3, pad=1),
        LayerSpec("c1c", 32, 64, 56, 56, 256, 1, 1)),
    # ResNet-50 stem and stage-4 layers, N=64
    2: (LayerSpec("c2s", 64, 3, 224, 224, 64, 7, 7, stride=2, pad=3),
        LayerSpec("c2a", 64, 2048, 7, 7, 512, 1, 1),
        LayerSpec("c2b", 64, 512, 7, 7, 512, 3, 3, pad=1),
        LayerSpec("c2c", 64, 512, 7, 7, 2048, 1, 1)),
    # detection-backbone shaped layers, N=2 at 800x1333 (feature strides 4 / 16 / 4->8)
    3: (LayerSpec("c3a", 2, 64, 200, 334, 64, 3, 3, pad=1),
        LayerSpec("c3b", 2, 256, 50, 84, 256, 3, 3, pad=1),
        LayerSpec("c3c", 2, 128, 200, 334, 128, 3, 3, stride=2, pad=1)),
    # depthwise and grouped, N=64
    4: (LayerSpec("c4a", 64, 96, 112, 112, 96, 3, 3, pad=1, groups=96),
        LayerSpec("c4b", 64, 256, 28, 28, 256, 3, 3, pad=1, groups=32)),
}

BASE_SEED = 20230511


def config_seed(config_index: int, layer_index: int = 0) -> int:
    return BASE_SEED + 1000 * layer_index + config_index


def find_layer(name: str) -> Tuple[int, int, LayerSpec]:
    for ci, layers in CONFIGS.items():
        for li, sp in enumerate(layers):
            if sp.name == name:
                return ci, li, sp
    raise KeyError(name)


# ---- one block's tensors ------------------------------------------------------------------

def make_block(spec: LayerSpec, seed: int, out_hw: Tuple[int, int]) -> Dict[str, Optional[np.ndarray]]:
    """Draw every tensor of one ConvBN block.

    Returns fp32 arrays in logical NCHW order whose values are already representable in the
    layer's storage type: ``x [N,C_in,H,W]``, ``w [C_out,C_in/G,kh,kw]``, ``dz [N,C_out,Ho,Wo]``
    and the fp32 vectors ``b`` (None without bias), ``gamma, beta, mu_hat, var_hat``.
    ``out_hw`` is the caller's (H_out, W_out).
    """
    cg = spec.c_in // spec.groups
    x_shape = (spec.n, spec.c_in, spec.h_in, spec.w_in)
    w_shape = (spec.c_out, cg, spec.kh, spec.kw)
    z_shape = (spec.n, spec.c_out, out_hw[0], out_hw[1])
    fan_in = cg * spec.kh * spec.kw
    t: Dict[str, Optional[np.ndarray]] = {}
    t["x"] = normal(seed, _TAGS["x"], int(np.prod(x_shape))).reshape(x_shape)
    t["w"] = (normal(seed, _TAGS["w"], int(np.prod(w_shape))) *
              np.float32(np.sqrt(2.0 / fan_in))).reshape(w_shape)
    t["dz"] = normal(seed, _TAGS["dz"], int(np.prod(z_shape))).reshape(z_shape)
    t["b"] = (normal(seed, _TAGS["b"], spec.c_out) * np.float32(0.01)) if spec.bias else None
    t["mu_hat"] = normal(seed, _TAGS["mu_hat"], spec.c_out) * np.float32(0.1)
    t["var_hat"] = uniform(seed, _TAGS["var_hat"], spec.c_out, 0.5, 2.0)
    t["gamma"] = uniform(seed, _TAGS["gamma"], spec.c_out, 0.5, 1.5)
    t["beta"] = normal(seed, _TAGS["beta"], spec.c_out) * np.float32(0.1)
    if spec.dtype == "f16":
        for k in ("x", "w", "dz"):
            t[k] = t[k].astype(np.float16).astype(np.float32)          # numpy rounds to nearest even
    if spec.dtype == "bf16":
        for k in ("x", "w", "dz"):
            t[k] = round_bf16(t[k])
    return t


# ---- layouts ------------------------------------------------------------------------------

def act_to_layout(a_nchw: np.ndarray, layout: str) -> np.ndarray:
    """Logical [N,C,H,W] -> contiguous memory order of ``layout``."""
    if layout == "nchw":
        return np.ascontiguousarray(a_nchw)
    return np.ascontiguousarray(a_nchw.transpose(0, 2, 3, 1))


def act_from_layout(a: np.ndarray, layout: str, nchw_shape) -> np.ndarray:
    """Memory order of ``layout`` -> logical [N,C,H,W]."""
    n, c, h, w = nchw_shape
    if layout == "nchw":
        return np.asarray(a).reshape(n, c, h, w)
    return np.asarray(a).reshape(n, h, w, c).transpose(0, 3, 1, 2)


def weight_to_layout(w_oihw: np.ndarray, layout: str) -> np.ndarray:
    """Logical [C_out,C_in/G,kh,kw] -> memory order: same for nchw, [C_out,kh,kw,C_in/G] for nhwc."""
    if layout == "nchw":
        return np.ascontiguousarray(w_oihw)
    return np.ascontiguousarray(w_oihw.transpose(0, 2, 3, 1))


def weight_from_layout(w: np.ndarray, layout: str, oihw_shape) -> np.ndarray:
    co, cg, kh, kw = oihw_shape
    if layout == "nchw":
        return np.asarray(w).reshape(co, cg, kh, kw)
    return np.asarray(w).reshape(co, kh, kw, cg).transpose(0, 3, 1, 2)
