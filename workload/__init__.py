"""Seeded synthetic inputs for the W4A4 linear path (host side, numpy in / numpy out).

This package only *draws inputs*: heavy-tailed VGGT-shaped activations, random weights and biases,
stand-in smoothing factors and sign vectors.  It contains none of the method's arithmetic and is
the one piece of code that both the CPU oracle's tests and the CUDA path's tests/bench may use.

bf16 tensors are carried as ``numpy.uint16`` bit patterns (numpy has no bf16 dtype).

The activations stand in for VGGT aggregator activations on the paper's datasets, which are not
available here; only the shapes (1374 tokens per frame = 37x37 patches + 1 camera + 4 register
tokens, d = 1024, MLP width 4096) and the structure the paper describes (a few outlier channels,
five much larger special-token rows at the start of every frame; Sec. 3.2, Observation 1) are kept.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gen.c")
_LIB = os.path.join(_HERE, "libqvggt_workload.so")

TOKENS_PER_FRAME = 1374  # 37*37 patch tokens + 1 camera token + 4 register tokens
SPECIAL_ROWS = 5
SPECIAL_GAIN = 100.0
OUTLIER_GAIN = 50.0

DIST_NORMAL, DIST_GELU, DIST_STUDENT_T3 = 0, 1, 2

# (name, K = d_in, N = d_out, activation distribution) of one aggregator block's linears
BLOCK_LINEARS = (
    ("qkv", 1024, 3072, DIST_NORMAL),
    ("proj", 1024, 1024, DIST_NORMAL),
    ("fc1", 1024, 4096, DIST_NORMAL),
    ("fc2", 4096, 1024, DIST_GELU),
)


def build(force: bool = False) -> str:
    """Compile gen.c into a shared library next to it (gcc, OpenMP)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _L():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        u64, i64, i32, dbl, vp = ctypes.c_uint64, ctypes.c_int64, ctypes.c_int, ctypes.c_double, ctypes.c_void_p
        lib.wl_activations_bf16.argtypes = [u64, u64, i64, i64, i32, i32, vp, i32, i32, dbl, vp, i64]
        lib.wl_activations_bf16.restype = None
        lib.wl_normal_bf16.argtypes = [u64, u64, i64, i64, i32, dbl, dbl, vp, i64]
        lib.wl_normal_bf16.restype = None
        lib.wl_loguniform_f32.argtypes = [u64, u64, i32, dbl, dbl, vp]
        lib.wl_loguniform_f32.restype = None
        lib.wl_signs_i8.argtypes = [u64, u64, i32, vp]
        lib.wl_signs_i8.restype = None
        _lib = lib
    return _lib


def outlier_gains(seed: int, stream: int, K: int, n_outlier: int, gain: float = OUTLIER_GAIN) -> np.ndarray:
    """fp32 [K] vector: `gain` on `n_outlier` channels drawn from (seed, stream), 1 elsewhere."""
    rng = np.random.Generator(np.random.Philox(key=[seed & (2**64 - 1), stream & (2**64 - 1)]))
    g = np.ones(K, dtype=np.float32)
    if n_outlier > 0:
        g[rng.choice(K, size=n_outlier, replace=False)] = gain
    return g


def activations(seed: int, stream: int, row0: int, nrows: int, K: int, dist: int = DIST_NORMAL,
                ch_gain: np.ndarray | None = None, frame_rows: int = TOKENS_PER_FRAME,
                special_rows: int = SPECIAL_ROWS, special_gain: float = SPECIAL_GAIN,
                out: np.ndarray | None = None) -> np.ndarray:
    """bf16 bits [nrows, K] of rows row0.. of the virtual activation matrix of (seed, stream)."""
    if out is None:
        out = np.empty((nrows, K), dtype=np.uint16)
    assert out.dtype == np.uint16 and out.shape == (nrows, K) and out.strides[1] == 2
    gp = None
    if ch_gain is not None:
        ch_gain = np.ascontiguousarray(ch_gain, dtype=np.float32)
        assert ch_gain.shape == (K,)
        gp = ch_gain.ctypes.data
    _L().wl_activations_bf16(seed, stream, row0, nrows, K, dist, gp, frame_rows, special_rows,
                             float(special_gain), out.ctypes.data, out.strides[0] // 2)
    return out


def normal_bf16(seed: int, stream: int, nrows: int, ncols: int, std: float, mean: float = 0.0,
                row0: int = 0) -> np.ndarray:
    out = np.empty((nrows, ncols), dtype=np.uint16)
    _L().wl_normal_bf16(seed, stream, row0, nrows, ncols, float(mean), float(std), out.ctypes.data, ncols)
    return out


def loguniform_f32(seed: int, stream: int, n: int, lo: float, hi: float) -> np.ndarray:
    out = np.empty(n, dtype=np.float32)
    _L().wl_loguniform_f32(seed, stream, n, float(lo), float(hi), out.ctypes.data)
    return out


def signs_i8(seed: int, stream: int, n: int) -> np.ndarray:
    out = np.empty(n, dtype=np.int8)
    _L().wl_signs_i8(seed, stream, n, out.ctypes.data)
    return out


def bf16_to_f32(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float32 (a format conversion, not method arithmetic)."""
    return (bits.astype(np.uint32) << 16).view(np.float32)


# ---------------------------------------------------------------------------------------------
# Layer recipes.  Streams: 4*layer + {0: activations, 1: weights, 2: bias, 3: calibration
# activations}; outlier channels come from (seed, 1000 + layer).
# ---------------------------------------------------------------------------------------------
@dataclass(frozen=True)
class LinearSpec:
    name: str
    K: int
    N: int
    dist: int
    seed: int
    layer: int          # layer index within the seed's stack (decides the streams)
    n_outlier: int = 8  # outlier channels (x50)

    def ch_gain(self) -> np.ndarray:
        return outlier_gains(self.seed, 1000 + self.layer, self.K, self.n_outlier)

    def x_rows(self, row0: int, nrows: int, out: np.ndarray | None = None) -> np.ndarray:
        return activations(self.seed, 4 * self.layer + 0, row0, nrows, self.K, self.dist, self.ch_gain(), out=out)

    def x_calib(self, nrows: int = TOKENS_PER_FRAME) -> np.ndarray:
        """One frame of calibration activations: same distribution, separate stream."""
        return activations(self.seed, 4 * self.layer + 3, 0, nrows, self.K, self.dist, self.ch_gain())

    def weight(self) -> np.ndarray:
        return normal_bf16(self.seed, 4 * self.layer + 1, self.N, self.K, 0.02)

    def bias(self) -> np.ndarray:
        return normal_bf16(self.seed, 4 * self.layer + 2, 1, self.N, 0.01).reshape(self.N)


def block_specs(seed: int, block: int = 0) -> list[LinearSpec]:
    """The four linears (qkv, proj, fc1, fc2) of aggregator block `block`."""
    return [LinearSpec(n, K, N, d, seed, 4 * block + i) for i, (n, K, N, d) in enumerate(BLOCK_LINEARS)]


def sweep_activations(seed: int, K: int, row0: int, nrows: int, out: np.ndarray | None = None) -> np.ndarray:
    """Bandwidth-sweep input: Student-t(3) entries, 1 % of the channels x50, no special rows."""
    g = outlier_gains(seed, 2000 + K, K, max(1, round(0.01 * K)))
    return activations(seed, 77, row0, nrows, K, DIST_STUDENT_T3, g, frame_rows=0, out=out)
