"""Seeded synthetic inputs shaped like the paper's workloads.

This module serves both the CPU oracle's tests and the CUDA library's tests and
benchmark.  It holds no coder or dequantiser arithmetic: it only draws quantised
weight symbols, layer by layer, and names the layer parameters (shape, alphabet,
zero-point, step, table size, chunk size) that both sides are then given.

What stands in for what: the paper trains ImageNet ResNets and codes each layer's
integer weights (Section III-A); those weights are not available, so layers keep
the real ResNet-18/50 convolution shapes and draw symbols from a discrete
two-sided geometric ("Laplacian") law centred on the zero-point, p_s ~ theta^|s-zp|,
with theta solved for the zero-point mass or the entropy the paper reports
(odd bin counts from 3 to 31 and more, Section III-C; about 0.85 bit per weight,
Section III-C).
"""
from __future__ import annotations

import ctypes
import math
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB = None
_GOLDEN = 0x9E3779B97F4A7C15
_M64 = (1 << 64) - 1


def build(force: bool = False) -> str:
    """Compile the generator's C helper in-tree and return the .so path."""
    src = os.path.join(_HERE, "synthgen.c")
    out = os.path.join(_HERE, "libsynthgen.so")
    if force or not os.path.exists(out) or os.path.getmtime(out) < os.path.getmtime(src):
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-shared", "-fPIC", "-o", out, src])
    return out


def _lib():
    global _LIB
    if _LIB is None:
        _LIB = ctypes.CDLL(build())
        _LIB.synth_draw_symbols.argtypes = [ctypes.c_uint64, ctypes.c_uint64, ctypes.c_uint64,
                                            ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p]
        _LIB.synth_draw_symbols.restype = None
        _LIB.synth_draw_u32.argtypes = [ctypes.c_uint64, ctypes.c_uint64, ctypes.c_uint64, ctypes.c_void_p]
        _LIB.synth_draw_u32.restype = None
    return _LIB


def splitmix64_at(key: int, i: int) -> int:
    """Draw i of stream `key` (pure Python statement of the generator)."""
    z = (key + (i + 1) * _GOLDEN) & _M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
    return z ^ (z >> 31)


def stream_key(seed: int, index: int) -> int:
    """Key of sub-stream `index` under `seed`: seed * 2^32 + index, mixed once."""
    return splitmix64_at((seed << 32 | (index & 0xFFFFFFFF)) & _M64, 0)


def uniform01(key: int, i: int) -> float:
    return (splitmix64_at(key, i) >> 11) / float(1 << 53)


# ----------------------------------------------------------------------------
# distributions
# ----------------------------------------------------------------------------
def geometric_pmf(A: int, zp: int, theta: float) -> np.ndarray:
    """p_s proportional to theta^|s - zp| on s in [0, A); powers by repeated multiply."""
    w = np.empty(A, dtype=np.float64)
    for s in range(A):
        v = 1.0
        for _ in range(abs(s - zp)):
            v *= theta
        w[s] = v
    return w / w.sum()


def entropy_bits(p) -> float:
    p = np.asarray(p, dtype=np.float64)
    p = p[p > 0]
    p = p / p.sum()
    return float(-(p * np.log2(p)).sum())


def _bisect(fn, target, lo=1e-9, hi=1.0 - 1e-9, iters=80):
    for _ in range(iters):
        mid = 0.5 * (lo + hi)
        if fn(mid) < target:
            lo = mid
        else:
            hi = mid
    th = 0.5 * (lo + hi)
    return round(th * (1 << 24)) / float(1 << 24)      # snap so libm noise cannot move it


def theta_for_pzp(A: int, zp: int, pzp: float) -> float:
    """theta with P(zero-point) = pzp (mass at zp falls as theta grows)."""
    return _bisect(lambda th: -geometric_pmf(A, zp, th)[zp], -pzp)


def theta_for_entropy(A: int, zp: int, h: float) -> float:
    return _bisect(lambda th: entropy_bits(geometric_pmf(A, zp, th)), h)


def integer_cdf(p: np.ndarray) -> np.ndarray:
    """Cumulative thresholds on the 32-bit draw; these integers DEFINE the data."""
    c = np.floor(np.cumsum(p) * float(1 << 32)).astype(np.uint64)
    c[-1] = 1 << 32
    return c


# ----------------------------------------------------------------------------
# layers
# ----------------------------------------------------------------------------
def alphabet_for_bits(b: int) -> tuple[int, int]:
    """b-bit zero-point quantiser: 2^b - 1 bins centred on zp (odd bin count,
    Section II-B); 1 bit cannot hold an odd count > 1, so b = 1 is {0, 1}, zp 0."""
    if b == 1:
        return 2, 0
    return (1 << b) - 1, (1 << (b - 1)) - 1


@dataclass
class LayerSpec:
    name: str
    shape: tuple
    bitwidth: int
    alphabet: int
    zero_point: int
    theta: float
    scale: float
    table_log: int
    chunk_symbols: int
    out_dtype: str          # "u8" | "f32" | "bf16"
    key: int
    n: int = field(init=False)

    def __post_init__(self):
        self.n = int(np.prod(self.shape))

    def pmf(self) -> np.ndarray:
        return geometric_pmf(self.alphabet, self.zero_point, self.theta)


def draw_symbols(spec: LayerSpec, threads: int | None = None) -> np.ndarray:
    """The layer's n symbols (flattened in memory order), uint8."""
    out = np.empty(spec.n, dtype=np.uint8)
    cdf = integer_cdf(spec.pmf())
    lib = _lib()
    block = 1 << 22
    starts = list(range(0, spec.n, block))

    def work(s0):
        cnt = min(block, spec.n - s0)
        lib.synth_draw_symbols(spec.key, s0, cnt, cdf.ctypes.data, spec.alphabet,
                               out.ctypes.data + s0)

    if len(starts) <= 1:
        for s0 in starts:
            work(s0)
    else:
        with ThreadPoolExecutor(threads or min(32, os.cpu_count() or 1)) as ex:
            list(ex.map(work, starts))
    return out


def draw_symbols_numpy(spec: LayerSpec) -> np.ndarray:
    """Same stream, stated with numpy (used to check the C helper on small layers)."""
    i = np.arange(1, spec.n + 1, dtype=np.uint64)
    with np.errstate(over="ignore"):
        z = np.uint64(spec.key) + i * np.uint64(_GOLDEN)
        z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
        z = z ^ (z >> np.uint64(31))
    u = z >> np.uint64(32)
    cdf = integer_cdf(spec.pmf())
    return np.minimum(np.searchsorted(cdf, u, side="right"), spec.alphabet - 1).astype(np.uint8)


def resnet18_conv_shapes():
    """The 20 convolutions of torchvision-style ResNet-18 (OIHW)."""
    shapes = [("conv1", (64, 3, 7, 7))]
    shapes += [(f"layer1.{b}.conv{c}", (64, 64, 3, 3)) for b in range(2) for c in (1, 2)]
    cin = 64
    for li, w in ((2, 128), (3, 256), (4, 512)):
        shapes.append((f"layer{li}.0.conv1", (w, cin, 3, 3)))
        shapes.append((f"layer{li}.0.conv2", (w, w, 3, 3)))
        shapes.append((f"layer{li}.0.downsample", (w, cin, 1, 1)))
        shapes.append((f"layer{li}.1.conv1", (w, w, 3, 3)))
        shapes.append((f"layer{li}.1.conv2", (w, w, 3, 3)))
        cin = w
    return shapes


def resnet50_conv_shapes():
    """The 53 convolutions of ResNet-50's feature extractor (OIHW)."""
    shapes = [("conv1", (64, 3, 7, 7))]
    cin = 64
    for li, (w, blocks) in enumerate(((64, 3), (128, 4), (256, 6), (512, 3)), start=1):
        for b in range(blocks):
            shapes.append((f"layer{li}.{b}.conv1", (w, cin, 1, 1)))
            shapes.append((f"layer{li}.{b}.conv2", (w, w, 3, 3)))
            shapes.append((f"layer{li}.{b}.conv3", (4 * w, w, 1, 1)))
            if b == 0:
                shapes.append((f"layer{li}.{b}.downsample", (4 * w, cin, 1, 1)))
            cin = 4 * w
    return shapes


# ----------------------------------------------------------------------------
# the five benchmark workloads
# ----------------------------------------------------------------------------
def workload_conv3x3(seed: int = 0) -> list[LayerSpec]:
    A, zp = alphabet_for_bits(4)
    return [LayerSpec("conv3x3_64_64", (64, 64, 3, 3), 4, A, zp, theta_for_pzp(A, zp, 0.6), 0.02,
                      12, 4096, "f32", stream_key(seed, 0))]


def workload_resnet18(seed: int = 1, table_log: int = 8, chunk: int = 16384) -> list[LayerSpec]:
    """The workload's description names no table size: the paper's own 256-state coder
    (Section III-A) is the default."""
    pk = stream_key(seed, 0xFFFF0001)
    out = []
    for li, (name, shape) in enumerate(resnet18_conv_shapes()):
        b = (2, 3, 4, 6)[int(uniform01(pk, 2 * li) * 4)]
        A, zp = alphabet_for_bits(b)
        h = min(0.8 + 0.7 * uniform01(pk, 2 * li + 1), 0.98 * math.log2(A))
        out.append(LayerSpec(name, shape, b, A, zp, theta_for_entropy(A, zp, h), 0.1 / (1 << b),
                             table_log, chunk, "bf16", stream_key(seed, li)))
    return out


def workload_resnet50(seed: int = 2, table_log: int = 8, chunk: int = 16384) -> list[LayerSpec]:
    """The workload's description names no table size: the paper's own 256-state coder
    (Section III-A) is the default (its 8-bit layers, 255 bins, code about 0.02 bit per weight
    better with 2^12 states)."""
    pk = stream_key(seed, 0xFFFF0002)
    out = []
    for li, (name, shape) in enumerate(resnet50_conv_shapes()):
        b = 1 + int(uniform01(pk, 2 * li) * 8)
        A, zp = alphabet_for_bits(b)
        pzp = 0.85 + 0.10 * uniform01(pk, 2 * li + 1)
        out.append(LayerSpec(name, shape, b, A, zp, theta_for_pzp(A, zp, pzp), 0.1 / (1 << b),
                             table_log, chunk, "bf16", stream_key(seed, li)))
    return out


def workload_sweep(seed: int = 3, table_log: int = 12, chunk: int = 16384,
                   n: int = 1 << 28) -> list[LayerSpec]:
    A, zp = 255, 127
    return [LayerSpec("sweep_u8", (n,), 8, A, zp, theta_for_entropy(A, zp, 2.5), 1.0,
                      table_log, chunk, "u8", stream_key(seed, 0))]


def workload_large(seed: int = 4, n_mats: int = 8, dim: int = 8192, chunk: int = 32768,
                   table_log: int = 8) -> list[LayerSpec]:
    """8 dense matrices, 7 bins.  The workload's description fixes no table size, so the paper's
    own 256-state coder (Section III-A) is the default; 2^12 states is the other measured case."""
    A, zp = alphabet_for_bits(3)
    th = theta_for_pzp(A, zp, 0.7)
    return [LayerSpec(f"dense{m}", (dim, dim), 3, A, zp, th, 0.05, table_log, chunk, "bf16",
                      stream_key(seed, m)) for m in range(n_mats)]


WORKLOADS = {
    "conv3x3": workload_conv3x3,
    "resnet18": workload_resnet18,
    "resnet50": workload_resnet50,
    "sweep": workload_sweep,
    "large": workload_large,
}
