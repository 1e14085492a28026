"""CPU ORACLE -- TEST INFRASTRUCTURE ONLY (numpy wrapper around qvggt_oracle.c).

A slow, plain restatement of the paper's W4A4 linear layer (Dual-Smoothed Fine-Grained
Quantization, Sec. 3.2).  Only the tests, the smoke check and the benchmark's CPU-baseline leg may
import this package; the CUDA path never does, and this package imports nothing from it.

bf16 tensors are ``numpy.uint16`` bit patterns.  Parity status is listed in the C file's header
(unpinned: fp32 stage order convention, group-wise variant for G < K, end-to-end layer error).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import time

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "qvggt_oracle.c")
_LIB = os.path.join(_HERE, "libqvggt_oracle.so")


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _L():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i64, i32, dbl, vp = ctypes.c_int64, ctypes.c_int, ctypes.c_double, ctypes.c_void_p
        sig = {
            "orc_fwht_f32": [vp, i32],
            "orc_fwht_f64": [vp, i32],
            "orc_multipliers": [vp, vp, i32, vp, vp],
            "orc_rotate_smooth_quantize": [vp, i64, i64, i32, vp, i32, vp, vp],
            "orc_rotate_smooth_quantize_bits": [vp, i64, i64, i32, vp, i32, i32, vp, vp],
            "orc_rotate_smooth_quantize_static": [vp, i64, i64, i32, vp, ctypes.c_float, i32, vp],
            "orc_layernorm": [vp, i64, i64, i32, vp, vp, ctypes.c_float, vp],
            "orc_rotate_smooth_quantize_wide": [vp, i64, i64, i32, vp, i32, vp, vp, vp, vp],
            "orc_gelu": [vp, i64, i64, i32, vp],
            "orc_pack_int4": [vp, i64, i32, vp],
            "orc_unpack_int4": [vp, i64, i32, vp],
            "orc_gemm_i32": [vp, vp, i64, i32, i32, i32, vp],
            "orc_epilogue": [vp, vp, vp, vp, i64, i32, i32, vp, i64],
            "orc_smooth_factors": [vp, i64, vp, i32, i32, dbl, dbl, dbl, vp],
            "orc_rotate_f64": [vp, i64, i64, i32, vp, vp],
            "orc_linear_f64": [vp, vp, vp, i64, i32, i32, vp],
        }
        for name, args in sig.items():
            fn = getattr(lib, name)
            fn.argtypes = args
            fn.restype = None
        lib.orc_gelu_f64.argtypes = [dbl]
        lib.orc_gelu_f64.restype = dbl
        _lib = lib
    return _lib


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def threads() -> int:
    """Threads the OpenMP loops use (all cores visible to the process unless OMP_NUM_THREADS is set)."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        return int(env)
    return len(os.sched_getaffinity(0))


def _fwht(u: np.ndarray, dtype, fn) -> np.ndarray:
    u = np.array(u, dtype=dtype, order="C")  # always a fresh copy; transformed in place, row by row
    K = u.shape[-1]
    for r in u.reshape(-1, K):
        fn(r.ctypes.data, K)
    return u


def fwht_f32(u: np.ndarray) -> np.ndarray:
    """Un-normalized Sylvester-Hadamard transform of every row (fp32 butterflies, ascending stride)."""
    return _fwht(u, np.float32, _L().orc_fwht_f32)


def fwht_f64(u: np.ndarray) -> np.ndarray:
    return _fwht(u, np.float64, _L().orc_fwht_f64)


def multipliers(c: np.ndarray, v: np.ndarray | None = None):
    c = _c(c, np.float32)
    K = c.shape[0]
    amul = np.empty(K, np.float32)
    wmul = np.empty(K, np.float32)
    vp = None
    if v is not None:
        v = _c(v, np.int8)
        vp = v.ctypes.data
    _L().orc_multipliers(c.ctypes.data, vp, K, amul.ctypes.data, wmul.ctypes.data)
    return amul, wmul


def rotate_smooth_quantize(X: np.ndarray, mul: np.ndarray, group: int = 0, bits: int = 4):
    """X bf16 bits [M, K] -> (codes int8 [M, K], scales fp32 [M] or [M, K/group]).
    bits: N of Eq. "quantization" (4 = the W4A4 setting, 8 = the paper's W8A8 setting)."""
    assert X.dtype == np.uint16 and X.ndim == 2 and X.strides[1] == 2 and 2 <= bits <= 8
    M, K = X.shape
    mul = _c(mul, np.float32)
    G = K // group if group else 1
    codes = np.empty((M, K), np.int8)
    scales = np.empty((M, G), np.float32)
    if bits == 4:
        _L().orc_rotate_smooth_quantize(X.ctypes.data, X.strides[0] // 2, M, K, mul.ctypes.data, group,
                                        codes.ctypes.data, scales.ctypes.data)
    else:
        _L().orc_rotate_smooth_quantize_bits(X.ctypes.data, X.strides[0] // 2, M, K, mul.ctypes.data, group, bits,
                                             codes.ctypes.data, scales.ctypes.data)
    return codes, (scales if group else scales.reshape(M))


def rotate_smooth_quantize_wide(X: np.ndarray, mul: np.ndarray, bits: int = 4):
    """The quantizer behind a rotation evaluated in fp64 and rounded to fp32 once (reference of the tolerance contract
    for rotations that do not follow the fp32 butterfly order).
    -> dict(codes int8 [M, K], scales fp32 [M], y fp32 [M, K] rotated and smoothed rows, abs_sum fp64 [M] = sum |x|)."""
    assert X.dtype == np.uint16 and X.ndim == 2 and X.strides[1] == 2 and 2 <= bits <= 8
    M, K = X.shape
    mul = _c(mul, np.float32)
    codes, scales = np.empty((M, K), np.int8), np.empty(M, np.float32)
    y, abs_sum = np.empty((M, K), np.float32), np.empty(M, np.float64)
    _L().orc_rotate_smooth_quantize_wide(X.ctypes.data, X.strides[0] // 2, M, K, mul.ctypes.data, bits, codes.ctypes.data,
                                         scales.ctypes.data, y.ctypes.data, abs_sum.ctypes.data)
    return dict(codes=codes, scales=scales, y=y, abs_sum=abs_sum)


def gelu_f64(x: float) -> float:
    """x * Phi(x) in fp64 (Phi through erfc)."""
    return _L().orc_gelu_f64(float(x))


def gelu(X: np.ndarray) -> np.ndarray:
    """bf16 bits [M, K] -> bf16 bits [M, K]: gelu evaluated in fp64, rounded to bf16 once."""
    assert X.dtype == np.uint16 and X.ndim == 2 and X.strides[1] == 2
    M, K = X.shape
    out = np.empty((M, K), np.uint16)
    _L().orc_gelu(X.ctypes.data, X.strides[0] // 2, M, K, out.ctypes.data)
    return out


def layernorm(X: np.ndarray, gamma: np.ndarray, beta: np.ndarray, eps: float = 1e-5) -> np.ndarray:
    """LayerNorm over the K channels of every token row, fp32 with pairwise-summed statistics -> bf16 bits [M, K]."""
    assert X.dtype == np.uint16 and X.ndim == 2 and X.strides[1] == 2
    M, K = X.shape
    assert K & (K - 1) == 0
    gamma, beta = _c(gamma, np.float32), _c(beta, np.float32)
    out = np.empty((M, K), np.uint16)
    _L().orc_layernorm(X.ctypes.data, X.strides[0] // 2, M, K, gamma.ctypes.data, beta.ctypes.data, np.float32(eps), out.ctypes.data)
    return out


def rotate_smooth_quantize_static(X: np.ndarray, mul: np.ndarray, delta: float, bits: int = 4) -> np.ndarray:
    """Static tensor-wise quantizer (Tab. "granularity"): X bf16 bits [M, K], one given step size -> codes int8 [M, K]
    (clamped to [-2^(bits-1), 2^(bits-1) - 1])."""
    assert X.dtype == np.uint16 and X.ndim == 2 and X.strides[1] == 2 and 2 <= bits <= 8 and delta > 0
    M, K = X.shape
    mul = _c(mul, np.float32)
    codes = np.empty((M, K), np.int8)
    _L().orc_rotate_smooth_quantize_static(X.ctypes.data, X.strides[0] // 2, M, K, mul.ctypes.data, np.float32(delta), bits,
                                           codes.ctypes.data)
    return codes


def pack_int4(codes: np.ndarray) -> np.ndarray:
    codes = _c(codes, np.int8)
    rows, K = codes.shape
    out = np.empty((rows, K // 2), np.uint8)
    _L().orc_pack_int4(codes.ctypes.data, rows, K, out.ctypes.data)
    return out


def unpack_int4(packed: np.ndarray) -> np.ndarray:
    packed = _c(packed, np.uint8)
    rows, Kh = packed.shape
    out = np.empty((rows, Kh * 2), np.int8)
    _L().orc_unpack_int4(packed.ctypes.data, rows, Kh * 2, out.ctypes.data)
    return out


def gemm_i32(xq: np.ndarray, wq: np.ndarray, group: int = 0) -> np.ndarray:
    """acc int32 [M, N] (group = 0) or [G, M, N]."""
    xq = _c(xq, np.int8)
    wq = _c(wq, np.int8)
    M, K = xq.shape
    N = wq.shape[0]
    assert wq.shape[1] == K
    G = K // group if group else 1
    acc = np.empty((G, M, N), np.int32)
    _L().orc_gemm_i32(xq.ctypes.data, wq.ctypes.data, M, N, K, group, acc.ctypes.data)
    return acc if group else acc.reshape(M, N)


def epilogue(acc: np.ndarray, a_scale: np.ndarray, w_scale: np.ndarray, bias: np.ndarray | None) -> np.ndarray:
    """-> Y bf16 bits [M, N]."""
    acc = _c(acc, np.int32)
    if acc.ndim == 2:
        G, (M, N) = 1, acc.shape
    else:
        G, M, N = acc.shape
    a_scale = _c(a_scale, np.float32)
    w_scale = _c(w_scale, np.float32)
    assert a_scale.size == M * G and w_scale.size == N
    bp = None
    if bias is not None:
        bias = _c(bias, np.uint16)
        bp = bias.ctypes.data
    Y = np.empty((M, N), np.uint16)
    _L().orc_epilogue(acc.ctypes.data, a_scale.ctypes.data, w_scale.ctypes.data, bp, M, N, G, Y.ctypes.data, N)
    return Y


def smooth_factors(Xcal: np.ndarray, W: np.ndarray, alpha: float = 0.5, lo: float = 1e-2, hi: float = 1e2):
    Xcal = _c(Xcal, np.uint16)
    W = _c(W, np.uint16)
    Mc, K = Xcal.shape
    N = W.shape[0]
    c = np.empty(K, np.float32)
    _L().orc_smooth_factors(Xcal.ctypes.data, Mc, W.ctypes.data, N, K, alpha, lo, hi, c.ctypes.data)
    return c


def rotate_f64(X: np.ndarray, mul: np.ndarray) -> np.ndarray:
    assert X.dtype == np.uint16 and X.ndim == 2 and X.strides[1] == 2
    M, K = X.shape
    mul = _c(mul, np.float64)
    out = np.empty((M, K), np.float64)
    _L().orc_rotate_f64(X.ctypes.data, X.strides[0] // 2, M, K, mul.ctypes.data, out.ctypes.data)
    return out


def linear_f64(X: np.ndarray, W: np.ndarray, bias: np.ndarray | None) -> np.ndarray:
    X = _c(X, np.uint16)
    W = _c(W, np.uint16)
    M, K = X.shape
    N = W.shape[0]
    bp = None
    if bias is not None:
        bias = _c(bias, np.uint16)
        bp = bias.ctypes.data
    Y = np.empty((M, N), np.float64)
    _L().orc_linear_f64(X.ctypes.data, W.ctypes.data, bp, M, N, K, Y.ctypes.data)
    return Y


def bf16_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.asarray(bits).astype(np.uint32) << 16).view(np.float32)


def prepare_weights(W: np.ndarray, c: np.ndarray, v: np.ndarray | None = None, bits: int = 4, tensorwise: bool = False):
    """Offline weight path: fold H and diag(c) into W, quantize per output channel (N = bits), or -- tensorwise, the other arm of
    Tab. "granularity" -- with one step size for the whole tensor: Delta = max|W~| / qmax = the largest per-row step size, then
    Eq. "quantization" with that Delta for every row (its clamp cannot act: Delta covers the largest element).

    -> dict(wq codes int8 [N, K], wq_packed uint8 [N, K/2] (bits = 4 only), w_scale fp32 [N], amul fp32 [K], wmul fp32 [K])
    """
    amul, wmul = multipliers(c, v)
    wq, w_scale = rotate_smooth_quantize(W, wmul, 0, bits)
    if tensorwise:
        delta = np.float32(w_scale.max())
        wq = rotate_smooth_quantize_static(W, wmul, float(delta), bits)
        w_scale = np.full(W.shape[0], delta, np.float32)
    return dict(wq=wq, wq_packed=pack_int4(wq) if bits == 4 else None, w_scale=w_scale, amul=amul, wmul=wmul, bits=bits)


def w4a4_linear(X: np.ndarray, prepared: dict, bias: np.ndarray | None, group: int = 0, timings: dict | None = None):
    """Online path for activations X (bf16 bits [M, K]) -> dict(xq, a_scale, acc, y)."""
    t0 = time.perf_counter()
    xq, a_scale = rotate_smooth_quantize(X, prepared["amul"], group, prepared.get("bits", 4))
    t1 = time.perf_counter()
    acc = gemm_i32(xq, prepared["wq"], group)
    t2 = time.perf_counter()
    y = epilogue(acc, a_scale, prepared["w_scale"], bias)
    t3 = time.perf_counter()
    if timings is not None:
        timings["rotate_smooth_quantize_s"] = timings.get("rotate_smooth_quantize_s", 0.0) + (t1 - t0)
        timings["gemm_s"] = timings.get("gemm_s", 0.0) + (t2 - t1)
        timings["epilogue_s"] = timings.get("epilogue_s", 0.0) + (t3 - t2)
    return dict(xq=xq, a_scale=a_scale, acc=acc, y=y)
