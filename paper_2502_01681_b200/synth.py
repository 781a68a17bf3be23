"""Seeded synthetic inputs: And-Inverter Graphs and random tensors.

This module only *draws inputs*.  It holds none of the layer's arithmetic (no
attention, no projection, no neighbourhood / bucket / permutation building), so
both the CUDA library and the CPU checker can be fed from it without sharing any
of the method's code.

Graphs come from the small C generator in ``csrc/synth_aig.c`` (compiled with gcc
on first use); tensors come from numpy's PCG64 generator seeded per row block, so
any row block can be drawn independently and in parallel.

The five workloads mirror the circuit shapes of the paper's dataset tables
(in-degree 0/1/2 node kinds, under two edges per node, a few per cent primary
inputs, depth from tens to thousands of levels); they stand in for ITC99 / EPFL /
OpenABC-D circuits, which are not redistributable here.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "csrc", "synth_aig.c")
_LIB = os.path.join(_HERE, "_dg4synth.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the graph generator with gcc (no CUDA involved)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"])
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i32p = ctypes.POINTER(ctypes.c_int32)
        lib.dg4_synth_window_aig.restype = ctypes.c_int64
        lib.dg4_synth_window_aig.argtypes = [ctypes.c_uint64, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                                             ctypes.c_double, ctypes.c_double, ctypes.c_double, i32p, i32p, i32p]
        lib.dg4_synth_layered_aig.restype = ctypes.c_int64
        lib.dg4_synth_layered_aig.argtypes = [ctypes.c_uint64, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                                              ctypes.c_double, i32p, i32p, i32p]
        _lib = lib
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))


@dataclass
class AIG:
    """Destination-sorted CSR of direct fan-ins plus the logic level of each node."""
    n_pi: int
    row_ptr: np.ndarray   # int32 [n+1]
    col_idx: np.ndarray   # int32 [e], sources ascending inside a row
    level: np.ndarray     # int32 [n]

    @property
    def n(self) -> int:
        return int(self.row_ptr.shape[0] - 1)

    @property
    def e(self) -> int:
        return int(self.col_idx.shape[0])

    def prefix(self, n: int) -> "AIG":
        """The first ``n`` nodes.  Ids are topological, so a prefix is closed under fan-in."""
        e = int(self.row_ptr[n])
        return AIG(min(self.n_pi, n), self.row_ptr[:n + 1].copy(), self.col_idx[:e].copy(), self.level[:n].copy())


def window_aig(seed: int, n_pi: int, n_gates: int, *, window: int = 0, win_exp=(4.0, 16.0),
               not_ratio: float = 0.3) -> AIG:
    """Gates in id (= topological) order; fan-ins uniform from the previous ``window`` nodes, or from a
    per-node window floor(2^U), U ~ Uniform[win_exp) when ``window`` is 0."""
    n = n_pi + n_gates
    row_ptr = np.zeros(n + 1, np.int32)
    col_idx = np.zeros(max(2 * n_gates, 1), np.int32)
    level = np.zeros(n, np.int32)
    e = _load().dg4_synth_window_aig(seed, n_pi, n_gates, window, float(win_exp[0]), float(win_exp[1]),
                                     not_ratio, _p(row_ptr), _p(col_idx), _p(level))
    if e < 0:
        raise ValueError("bad generator arguments")
    return AIG(n_pi, row_ptr, col_idx[:e].copy(), level)


def layered_aig(seed: int, n_pi: int, n_levels: int, gates_per_level: int, *, not_ratio: float = 0.3) -> AIG:
    """Level-major ids; first fan-in from the previous level, second from the previous 1-3 levels."""
    n = n_pi + n_levels * gates_per_level
    row_ptr = np.zeros(n + 1, np.int32)
    col_idx = np.zeros(max(2 * n_levels * gates_per_level, 1), np.int32)
    level = np.zeros(n, np.int32)
    e = _load().dg4_synth_layered_aig(seed, n_pi, n_levels, gates_per_level, not_ratio,
                                      _p(row_ptr), _p(col_idx), _p(level))
    if e < 0:
        raise ValueError("bad generator arguments")
    return AIG(n_pi, row_ptr, col_idx[:e].copy(), level)


# ---------------------------------------------------------------------------------------------
# tensors
# ---------------------------------------------------------------------------------------------

def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to the nearest bfloat16 (ties to even); returns the 16-bit patterns."""
    u = np.ascontiguousarray(x, np.float32).view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + r) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _normal_blocks(seed, stream, shape, std, out, convert, threads):
    rows = shape[0]
    inner = int(np.prod(shape[1:])) if len(shape) > 1 else 1
    out2 = out.reshape(rows, inner)
    blk = 65536
    nblk = (rows + blk - 1) // blk

    def fill(b):
        lo, hi = b * blk, min(rows, (b + 1) * blk)
        g = np.random.Generator(np.random.PCG64(np.random.SeedSequence([int(seed), int(stream), int(b)])))
        if convert is None:
            g.standard_normal((hi - lo, inner), dtype=np.float32, out=out2[lo:hi])
            if std != 1.0:
                out2[lo:hi] *= np.float32(std)
        else:
            t = g.standard_normal((hi - lo, inner), dtype=np.float32)
            if std != 1.0:
                t *= np.float32(std)
            out2[lo:hi] = convert(t)

    if nblk <= 1:
        for b in range(nblk):
            fill(b)
    else:
        with ThreadPoolExecutor(max_workers=threads or min(32, os.cpu_count() or 1)) as ex:
            list(ex.map(fill, range(nblk)))
    return out


def normal_f32(seed: int, stream: int, shape, std: float = 1.0, threads: int | None = None) -> np.ndarray:
    """N(0, std^2) float32 tensor.  Rows are drawn in blocks of 65536, block b from a PCG64 stream
    seeded with (seed, stream, b), so the result does not depend on the number of threads."""
    shape = tuple(int(s) for s in shape)
    return _normal_blocks(seed, stream, shape, std, np.empty(shape, np.float32), None, threads)


def normal_bf16_bits(seed: int, stream: int, shape, std: float = 1.0, threads: int | None = None,
                     out: np.ndarray | None = None) -> np.ndarray:
    """The same draw as :func:`normal_f32`, rounded once to bfloat16; returns uint16 bit patterns
    (optionally into a caller-provided buffer, e.g. pinned memory)."""
    shape = tuple(int(s) for s in shape)
    if out is None:
        out = np.empty(shape, np.uint16)
    return _normal_blocks(seed, stream, shape, std, out, f32_to_bf16_bits, threads)


# ---------------------------------------------------------------------------------------------
# the five workloads
# ---------------------------------------------------------------------------------------------

@dataclass
class Workload:
    """One benchmark configuration: how to draw the circuit and the tensors, and how the layer is run."""
    name: str
    seed: int
    kind: str                 # "window" | "layered"
    n_pi: int
    n_gates: int
    hops: int
    heads: int
    dtype: str                # "f32" | "bf16"
    layers: int
    modes: tuple              # subset of ("parallel", "levelised")
    with_projection: bool     # False: Q, K, V are drawn directly (attention only)
    window: int = 0
    win_exp: tuple = (4.0, 16.0)
    n_levels: int = 0
    gates_per_level: int = 0
    d: int = 128
    not_ratio: float = 0.3
    residual: bool = True
    extra: dict = field(default_factory=dict)

    @property
    def n(self) -> int:
        return self.n_pi + self.n_gates

    @property
    def d_head(self) -> int:
        return self.d // self.heads

    @property
    def scale(self) -> float:
        return 1.0 / float(np.sqrt(self.d_head))

    def graph(self) -> AIG:
        if self.kind == "window":
            return window_aig(self.seed, self.n_pi, self.n_gates, window=self.window, win_exp=self.win_exp,
                              not_ratio=self.not_ratio)
        return layered_aig(self.seed, self.n_pi, self.n_levels, self.gates_per_level, not_ratio=self.not_ratio)

    # tensor streams: 10 X; 1100+layer W_qkv; 1200+layer W_o; 20/21/22 Q/K/V
    def x_f32(self, n: int | None = None) -> np.ndarray:
        return normal_f32(self.seed, 10, (n or self.n, self.d), 1.0)

    def x_bf16_bits(self, n: int | None = None, out=None) -> np.ndarray:
        return normal_bf16_bits(self.seed, 10, (n or self.n, self.d), 1.0, out=out)

    def w_qkv_f32(self, layer: int) -> np.ndarray:
        return normal_f32(self.seed, 1100 + layer, (3 * self.d, self.d), 0.02)

    def w_o_f32(self, layer: int) -> np.ndarray:
        return normal_f32(self.seed, 1200 + layer, (self.d, self.d), 0.02)

    def qkv_f32(self, n: int | None = None):
        s = 1.0 / float(np.sqrt(self.d_head))
        return tuple(normal_f32(self.seed, 20 + i, (n or self.n, self.d), s) for i in range(3))

    def qkv_bf16_bits(self, n: int | None = None):
        s = 1.0 / float(np.sqrt(self.d_head))
        return tuple(normal_bf16_bits(self.seed, 20 + i, (n or self.n, self.d), s) for i in range(3))


def workload(cfg: int, shrink: int = 1) -> Workload:
    """The benchmark configurations 1..5; ``shrink`` divides the node counts (same generator, same
    shape parameters) so a CPU checker can cover every configuration in seconds."""
    s = max(1, int(shrink))
    if cfg == 1:
        return Workload("cfg1-tiny", 0, "window", 64, 2000 // s, hops=1, heads=4, dtype="f32", layers=1,
                        modes=("parallel",), with_projection=False, window=256)
    if cfg == 2:
        return Workload("cfg2-medium", 1, "window", max(2, 1000 // s), 100_000 // s, hops=1, heads=8, dtype="bf16",
                        layers=3, modes=("parallel",), with_projection=True, window=4096)
    if cfg == 3:
        return Workload("cfg3-large", 2, "window", max(2, 10_000 // s), 1_000_000 // s, hops=2, heads=8,
                        dtype="bf16", layers=1, modes=("parallel",), with_projection=False, win_exp=(4.0, 16.0))
    if cfg == 4:
        gpl = max(2, 2000 // s)
        nl = 500 if s == 1 else max(4, 500 // max(1, s // 4))
        return Workload("cfg4-levelised", 3, "layered", max(2, 10_000 // s), nl * gpl, hops=1, heads=8,
                        dtype="bf16", layers=3, modes=("levelised",), with_projection=True,
                        n_levels=nl, gates_per_level=gpl)
    if cfg == 5:
        return Workload("cfg5-scale", 4, "window", max(2, 50_000 // s), 10_000_000 // s, hops=2, heads=8,
                        dtype="bf16", layers=3, modes=("parallel", "levelised"), with_projection=True,
                        win_exp=(4.0, 20.0))
    raise ValueError("cfg must be 1..5")
