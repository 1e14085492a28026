"""Thin Python binding of libqvggt (ctypes): argument marshalling only.

Every step of the path runs in the CUDA kernels behind the C ABI declared in include/qvggt.h;
PyTorch is used for device memory and streams.  There is no CPU fallback: if the shared library
is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os

import torch

from . import buildlib as _build

OK = 0
_STATUS_NAMES = {0: "QVGGT_OK", -1: "QVGGT_ERR_NULL", -2: "QVGGT_ERR_SHAPE", -3: "QVGGT_ERR_ALIGN",
                 -4: "QVGGT_ERR_UNSUPPORTED", -5: "QVGGT_ERR_CUDA", -6: "QVGGT_ERR_DEVICE_TIMEOUT",
                 -7: "QVGGT_ERR_NOMEM"}

EXPORTS = ("qvggt_prepare_weights", "qvggt_rotate_smooth_quantize", "qvggt_w4a4_linear", "qvggt_free_weights",
           "qvggt_weights_view", "qvggt_device_status", "qvggt_calibrate_smooth", "qvggt_status_string",
           "qvggt_quantize_weights_static", "qvggt_rotate_smooth_quantize_c8", "qvggt_w4a4_linear_c8",
           "qvggt_weights_view_c8", "qvggt_rotate_smooth_quantize_static_c8",
           "qvggt_layernorm_rotate_smooth_quantize_c8", "qvggt_layernorm", "qvggt_debug_starved_linear_c8",
           "qvggt_rotate_smooth_quantize_tc", "qvggt_rotate_smooth_quantize_tc_c8", "qvggt_gelu",
           "qvggt_gelu_rotate_smooth_quantize_c8", "qvggt_w4a4_linear_c8_packed_weights",
           "qvggt_rotate_smooth_quantize_c8_grouped", "qvggt_w4a4_linear_c8_grouped",
           "qvggt_rotate_smooth_quantize_c8_expand", "qvggt_w4a4_linear_c8_expanded")
PREP_C8 = 1   # QVGGT_PREP_C8: keep an int8 [N, K] copy of the weight codes for the *_c8 entry points
PREP_W8A8 = 2  # QVGGT_PREP_W8A8: 8-bit codes (one per byte only)
PREP_C8_ONLY = 4  # QVGGT_PREP_C8_ONLY: 4-bit codes one per byte only (no packed copy)
PREP_W_TENSORWISE = 8  # QVGGT_PREP_W_TENSORWISE: one weight step size for the whole tensor


class QvggtError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().qvggt_status_string(status).decode()
        super().__init__(f"{where}: {_STATUS_NAMES.get(status, status)} ({msg})")


_lib = None


def lib() -> ctypes.CDLL:
    """Loads libqvggt.so (built in-tree by `build.build()`); raises if it is not there."""
    global _lib
    if _lib is None:
        path = _build.LIB
        if not os.path.exists(path):
            raise RuntimeError(f"{path} is missing: run __graft_entry__.build() (nvcc, sm_100a) first; "
                               "there is no fallback path")
        L = ctypes.CDLL(path)
        vp, i32, i64, f32 = ctypes.c_void_p, ctypes.c_int, ctypes.c_longlong, ctypes.c_float
        L.qvggt_prepare_weights.argtypes = [vp, vp, vp, vp, i32, i32, i32, vp, ctypes.POINTER(vp)]
        L.qvggt_rotate_smooth_quantize.argtypes = [vp, vp, i64, i32, i32, vp, vp, vp]
        L.qvggt_w4a4_linear.argtypes = [vp, vp, vp, i32, i32, vp, i64, vp, vp]
        L.qvggt_rotate_smooth_quantize_c8.argtypes = [vp, vp, i64, i32, vp, vp, vp]
        L.qvggt_w4a4_linear_c8.argtypes = [vp, vp, vp, i32, vp, i64, vp, vp]
        L.qvggt_rotate_smooth_quantize_static_c8.argtypes = [vp, vp, i64, i32, vp, vp, vp, vp]
        L.qvggt_layernorm_rotate_smooth_quantize_c8.argtypes = [vp, vp, i64, i32, vp, vp, f32, vp, vp, vp]
        L.qvggt_layernorm.argtypes = [vp, i64, i32, i32, vp, vp, f32, vp, vp]
        L.qvggt_rotate_smooth_quantize_tc.argtypes = [vp, vp, i64, i32, vp, vp, vp, vp]
        L.qvggt_rotate_smooth_quantize_tc_c8.argtypes = [vp, vp, i64, i32, vp, vp, vp, vp]
        L.qvggt_w4a4_linear_c8_packed_weights.argtypes = [vp, vp, vp, i32, vp, i64, vp, vp, vp]
        L.qvggt_rotate_smooth_quantize_c8_grouped.argtypes = [vp, vp, i64, i32, vp, vp, vp]
        L.qvggt_rotate_smooth_quantize_c8_expand.argtypes = [vp, vp, i64, i32, vp, vp, vp, vp]
        L.qvggt_w4a4_linear_c8_expanded.argtypes = [vp, vp, vp, i32, vp, i64, vp, vp, vp]
        L.qvggt_w4a4_linear_c8_grouped.argtypes = [vp, vp, vp, i32, vp, i64, vp, vp]
        L.qvggt_gelu.argtypes = [vp, i64, i32, i32, vp, vp]
        L.qvggt_gelu_rotate_smooth_quantize_c8.argtypes = [vp, vp, i64, i32, vp, vp, vp]
        L.qvggt_debug_starved_linear_c8.argtypes = [vp, vp, vp, i32, vp, i64, i64, vp]
        L.qvggt_weights_view_c8.argtypes = [vp, ctypes.POINTER(vp), ctypes.POINTER(i32)]
        L.qvggt_free_weights.argtypes = [vp]
        L.qvggt_free_weights.restype = None
        L.qvggt_weights_view.argtypes = [vp] + [ctypes.POINTER(vp)] * 4 + [ctypes.POINTER(i32)] * 2
        L.qvggt_device_status.argtypes = [vp, vp, ctypes.POINTER(i32)]
        L.qvggt_calibrate_smooth.argtypes = [vp, i32, vp, i32, i32, f32, f32, f32, vp, vp, vp]
        L.qvggt_quantize_weights_static.argtypes = [vp, vp, vp, i32, i32, vp, vp, vp, vp]
        L.qvggt_status_string.argtypes = [i32]
        L.qvggt_status_string.restype = ctypes.c_char_p
        for name in EXPORTS:
            if name not in ("qvggt_free_weights", "qvggt_status_string"):
                getattr(L, name).restype = i32
        _lib = L
    return _lib


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t: torch.Tensor | None) -> int | None:
    if t is None:
        return None
    assert t.is_cuda, "device tensor expected"
    return t.data_ptr()


def _check(status: int, where: str) -> None:
    if status != OK:
        raise QvggtError(status, where)


class Weights:
    """Owner of a qvggt_weights_t handle (prepared int4 weights of one linear layer)."""

    def __init__(self, handle: int, N: int, K: int):
        self._h = handle
        self.N, self.K = N, K

    @property
    def handle(self) -> int:
        if not self._h:
            raise RuntimeError("weights handle already freed")
        return self._h

    def view(self) -> dict:
        """Copies of the handle's device arrays as torch tensors: wq [N,K/2] u8, w_scale [N], amul [K], bias [N] or None."""
        ptrs = [ctypes.c_void_p() for _ in range(4)]
        n, k = ctypes.c_int(), ctypes.c_int()
        _check(lib().qvggt_weights_view(self.handle, *[ctypes.byref(p) for p in ptrs], ctypes.byref(n), ctypes.byref(k)),
               "qvggt_weights_view")
        N, K = n.value, k.value

        def wrap(p, nbytes, dtype, shape):
            if not p.value:
                return None
            return _from_device_ptr(p.value, nbytes, dtype, shape)

        return dict(wq=wrap(ptrs[0], N * K // 2, torch.uint8, (N, K // 2)),
                    w_scale=wrap(ptrs[1], 4 * N, torch.float32, (N,)),
                    amul=wrap(ptrs[2], 4 * K, torch.float32, (K,)),
                    bias=wrap(ptrs[3], 2 * N, torch.bfloat16, (N,)))

    def view_c8(self) -> torch.Tensor | None:
        """Copy of the int8 [N, K] codes (None if prepared without c8=True)."""
        p, bits = ctypes.c_void_p(), ctypes.c_int()
        _check(lib().qvggt_weights_view_c8(self.handle, ctypes.byref(p), ctypes.byref(bits)), "qvggt_weights_view_c8")
        self.bits = bits.value
        if not p.value:
            return None
        return _from_device_ptr(p.value, self.N * self.K, torch.uint8, (self.N, self.K)).view(torch.int8)

    def device_status(self) -> int:
        code = ctypes.c_int(0)
        st = lib().qvggt_device_status(self.handle, _stream(), ctypes.byref(code))
        if st not in (OK, -6):
            raise QvggtError(st, "qvggt_device_status")
        return code.value

    def free(self) -> None:
        if self._h:
            lib().qvggt_free_weights(self._h)
            self._h = 0

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


class _DeviceArray:
    """Minimal __cuda_array_interface__ carrier so torch can wrap a raw device pointer."""

    def __init__(self, ptr: int, shape, typestr: str):
        self.__cuda_array_interface__ = {"shape": tuple(shape), "typestr": typestr, "data": (ptr, False), "version": 2}


def _from_device_ptr(ptr: int, nbytes: int, dtype: torch.dtype, shape) -> torch.Tensor:
    """Copy of the device array at `ptr` as a fresh torch tensor (so it outlives the handle)."""
    typestr = {torch.uint8: "|u1", torch.float32: "<f4", torch.bfloat16: "<i2"}[dtype]
    t = torch.as_tensor(_DeviceArray(ptr, shape, typestr), device="cuda")
    assert t.numel() * t.element_size() == nbytes
    t = t.clone()
    return t.view(torch.bfloat16) if dtype == torch.bfloat16 else t


def prepare_weights(W: torch.Tensor, bias: torch.Tensor | None, smooth_c: torch.Tensor,
                    sign_v: torch.Tensor | None = None, c8: bool | str = False, bits: int = 4, w_tensorwise: bool = False) -> Weights:
    """W [N,K] bf16, bias [N] bf16 or None, smooth_c [K] fp32, sign_v [K] int8 (+1/-1) or None.
    c8: True = also keep the codes one per byte, as the *_c8 entry points need them; "only" = keep only that copy.
    bits: 4 (W4A4) or 8 (W8A8: one code per byte only; use the *_c8 entry points).
    w_tensorwise: one weight step size for the whole tensor instead of one per output channel (needs c8="only" or bits=8)."""
    assert bits in (4, 8) and c8 in (False, True, "only")
    assert W.dim() == 2 and W.element_size() == 2 and W.is_contiguous()
    N, K = W.shape
    assert smooth_c.dtype == torch.float32 and smooth_c.numel() == K and smooth_c.is_contiguous()
    if bias is not None:
        assert bias.element_size() == 2 and bias.numel() == N and bias.is_contiguous()
    if sign_v is not None:
        assert sign_v.dtype == torch.int8 and sign_v.numel() == K and sign_v.is_contiguous()
    h = ctypes.c_void_p()
    _check(lib().qvggt_prepare_weights(_ptr(W), _ptr(bias), _ptr(smooth_c), _ptr(sign_v), N, K,
                                       (PREP_W8A8 if bits == 8 else (PREP_C8_ONLY if c8 == "only" else (PREP_C8 if c8 else 0))) | (PREP_W_TENSORWISE if w_tensorwise else 0),
                                       _stream(),
                                       ctypes.byref(h)), "qvggt_prepare_weights")
    return Weights(h.value, N, K)


def rotate_smooth_quantize(w: Weights, X: torch.Tensor, group: int = 0, Xq: torch.Tensor | None = None,
                           a_scale: torch.Tensor | None = None):
    """X [M,K] bf16 (row stride may exceed K) -> (Xq [M,K/2] uint8, a_scale fp32 [M] or [M,K/128])."""
    assert X.dim() == 2 and X.element_size() == 2 and X.stride(1) == 1 and X.shape[1] == w.K
    M = X.shape[0]
    if Xq is None:
        Xq = torch.empty((M, w.K // 2), dtype=torch.uint8, device=X.device)
    if a_scale is None:
        a_scale = torch.empty((M, w.K // 128) if group else (M,), dtype=torch.float32, device=X.device)
    ldx = X.stride(0) if M > 1 else w.K
    _check(lib().qvggt_rotate_smooth_quantize(w.handle, _ptr(X), ldx, M, group, _ptr(Xq), _ptr(a_scale), _stream()),
           "qvggt_rotate_smooth_quantize")
    return Xq, a_scale


def w4a4_linear(w: Weights, Xq: torch.Tensor, a_scale: torch.Tensor, group: int = 0, Y: torch.Tensor | None = None,
                acc_debug: torch.Tensor | None = None) -> torch.Tensor:
    """-> Y [M,N] bf16.  acc_debug: optional int32 [M,N] (group 0) or [K/128,M,N] receiving the integer sums."""
    M = Xq.shape[0]
    assert Xq.dtype == torch.uint8 and Xq.is_contiguous() and Xq.shape[1] == w.K // 2
    assert a_scale.dtype == torch.float32 and a_scale.is_contiguous()
    if Y is None:
        Y = torch.empty((M, w.N), dtype=torch.bfloat16, device=Xq.device)
    assert Y.element_size() == 2 and Y.stride(1) == 1 and Y.shape == (M, w.N)
    ldy = Y.stride(0) if M > 1 else w.N
    if acc_debug is not None:
        assert acc_debug.dtype == torch.int32 and acc_debug.is_contiguous()
    _check(lib().qvggt_w4a4_linear(w.handle, _ptr(Xq), _ptr(a_scale), M, group, _ptr(Y), ldy, _ptr(acc_debug), _stream()),
           "qvggt_w4a4_linear")
    return Y


def rotate_smooth_quantize_c8(w: Weights, X: torch.Tensor, Xq8: torch.Tensor | None = None,
                              a_scale: torch.Tensor | None = None):
    """X [M,K] bf16 (row stride may exceed K) -> (Xq8 [M,K] int8, one code per byte; a_scale fp32 [M])."""
    assert X.dim() == 2 and X.element_size() == 2 and X.stride(1) == 1 and X.shape[1] == w.K
    M = X.shape[0]
    if Xq8 is None:
        Xq8 = torch.empty((M, w.K), dtype=torch.int8, device=X.device)
    if a_scale is None:
        a_scale = torch.empty((M,), dtype=torch.float32, device=X.device)
    assert Xq8.dtype == torch.int8 and Xq8.is_contiguous() and a_scale.dtype == torch.float32
    ldx = X.stride(0) if M > 1 else w.K
    _check(lib().qvggt_rotate_smooth_quantize_c8(w.handle, _ptr(X), ldx, M, _ptr(Xq8), _ptr(a_scale), _stream()),
           "qvggt_rotate_smooth_quantize_c8")
    return Xq8, a_scale


def rotate_smooth_quantize_tc(w: Weights, X: torch.Tensor, c8: bool = False, Xq: torch.Tensor | None = None,
                              a_scale: torch.Tensor | None = None, y_debug: torch.Tensor | None = None):
    """Tensor-core Hadamard mode (tolerance contract, see include/qvggt.h): X [M,K] bf16 ->
    (Xq [M,K/2] uint8, or [M,K] int8 with c8=True; a_scale fp32 [M]).  y_debug: optional fp32 [M,K] receiving the rotated rows."""
    assert X.dim() == 2 and X.element_size() == 2 and X.stride(1) == 1 and X.shape[1] == w.K
    M = X.shape[0]
    if Xq is None:
        Xq = torch.empty((M, w.K) if c8 else (M, w.K // 2), dtype=torch.int8 if c8 else torch.uint8, device=X.device)
    if a_scale is None:
        a_scale = torch.empty((M,), dtype=torch.float32, device=X.device)
    assert Xq.is_contiguous() and a_scale.dtype == torch.float32
    if y_debug is not None:
        assert y_debug.dtype == torch.float32 and y_debug.is_contiguous() and y_debug.shape == (M, w.K)
    ldx = X.stride(0) if M > 1 else w.K
    fn = lib().qvggt_rotate_smooth_quantize_tc_c8 if c8 else lib().qvggt_rotate_smooth_quantize_tc
    _check(fn(w.handle, _ptr(X), ldx, M, _ptr(Xq), _ptr(a_scale), _ptr(y_debug), _stream()), "qvggt_rotate_smooth_quantize_tc")
    return Xq, a_scale


def rotate_smooth_quantize_static_c8(w: Weights, X: torch.Tensor, delta: torch.Tensor, Xq8: torch.Tensor | None = None,
                                     a_scale: torch.Tensor | None = None):
    """Static tensor-wise quantizer: delta = one fp32 step size on the device -> (Xq8 [M,K] int8, a_scale [M] = delta)."""
    assert X.dim() == 2 and X.element_size() == 2 and X.stride(1) == 1 and X.shape[1] == w.K
    assert delta.dtype == torch.float32 and delta.numel() == 1 and delta.is_cuda
    M = X.shape[0]
    if Xq8 is None:
        Xq8 = torch.empty((M, w.K), dtype=torch.int8, device=X.device)
    if a_scale is None:
        a_scale = torch.empty((M,), dtype=torch.float32, device=X.device)
    ldx = X.stride(0) if M > 1 else w.K
    _check(lib().qvggt_rotate_smooth_quantize_static_c8(w.handle, _ptr(X), ldx, M, _ptr(delta), _ptr(Xq8), _ptr(a_scale),
                                                        _stream()), "qvggt_rotate_smooth_quantize_static_c8")
    return Xq8, a_scale


def layernorm_rotate_smooth_quantize_c8(w: Weights, X: torch.Tensor, gamma: torch.Tensor, beta: torch.Tensor, eps: float = 1e-5,
                                        Xq8: torch.Tensor | None = None, a_scale: torch.Tensor | None = None):
    """LayerNorm (gamma, beta fp32 [K]) fused in front of rotate_smooth_quantize_c8 -> (Xq8 [M,K] int8, a_scale [M])."""
    assert X.dim() == 2 and X.element_size() == 2 and X.stride(1) == 1 and X.shape[1] == w.K
    assert gamma.dtype == torch.float32 and beta.dtype == torch.float32 and gamma.numel() == w.K and beta.numel() == w.K
    M = X.shape[0]
    if Xq8 is None:
        Xq8 = torch.empty((M, w.K), dtype=torch.int8, device=X.device)
    if a_scale is None:
        a_scale = torch.empty((M,), dtype=torch.float32, device=X.device)
    ldx = X.stride(0) if M > 1 else w.K
    _check(lib().qvggt_layernorm_rotate_smooth_quantize_c8(w.handle, _ptr(X), ldx, M, _ptr(gamma), _ptr(beta), eps, _ptr(Xq8),
                                                           _ptr(a_scale), _stream()), "qvggt_layernorm_rotate_smooth_quantize_c8")
    return Xq8, a_scale


def layernorm(X: torch.Tensor, gamma: torch.Tensor, beta: torch.Tensor, eps: float = 1e-5, Y: torch.Tensor | None = None):
    """The same LayerNorm alone: X [M,K] bf16 -> Y [M,K] bf16 (K = 1024 or 4096)."""
    assert X.dim() == 2 and X.element_size() == 2 and X.stride(1) == 1
    M, K = X.shape
    assert gamma.dtype == torch.float32 and beta.dtype == torch.float32 and gamma.numel() == K and beta.numel() == K
    if Y is None:
        Y = torch.empty((M, K), dtype=torch.bfloat16, device=X.device)
    assert Y.is_contiguous() and Y.element_size() == 2
    ldx = X.stride(0) if M > 1 else K
    _check(lib().qvggt_layernorm(_ptr(X), ldx, M, K, _ptr(gamma), _ptr(beta), eps, _ptr(Y), _stream()), "qvggt_layernorm")
    return Y


def rotate_smooth_quantize_c8_grouped(w: Weights, X: torch.Tensor, Xq8: torch.Tensor | None = None, a_scale: torch.Tensor | None = None):
    """One scale per token per 128 rotated channels, codes one per byte -> (Xq8 [M,K] int8, a_scale fp32 [M, K/128])."""
    assert X.dim() == 2 and X.element_size() == 2 and X.stride(1) == 1 and X.shape[1] == w.K
    M = X.shape[0]
    if Xq8 is None:
        Xq8 = torch.empty((M, w.K), dtype=torch.int8, device=X.device)
    if a_scale is None:
        a_scale = torch.empty((M, w.K // 128), dtype=torch.float32, device=X.device)
    _check(lib().qvggt_rotate_smooth_quantize_c8_grouped(w.handle, _ptr(X), X.stride(0) if M > 1 else w.K, M, _ptr(Xq8), _ptr(a_scale),
                                                         _stream()), "qvggt_rotate_smooth_quantize_c8_grouped")
    return Xq8, a_scale


def w4a4_linear_c8_grouped(w: Weights, Xq8: torch.Tensor, a_scale: torch.Tensor, Y: torch.Tensor | None = None,
                           acc_debug: torch.Tensor | None = None) -> torch.Tensor:
    """-> Y [M,N] bf16 from one-code-per-byte codes with group-128 scales; acc_debug: optional int32 [K/128, M, N]."""
    M = Xq8.shape[0]
    assert Xq8.dtype == torch.int8 and Xq8.is_contiguous() and Xq8.shape[1] == w.K
    assert a_scale.dtype == torch.float32 and a_scale.is_contiguous() and a_scale.shape == (M, w.K // 128)
    if Y is None:
        Y = torch.empty((M, w.N), dtype=torch.bfloat16, device=Xq8.device)
    ldy = Y.stride(0) if M > 1 else w.N
    _check(lib().qvggt_w4a4_linear_c8_grouped(w.handle, _ptr(Xq8), _ptr(a_scale), M, _ptr(Y), ldy, _ptr(acc_debug), _stream()),
           "qvggt_w4a4_linear_c8_grouped")
    return Y


def gelu(X: torch.Tensor, Y: torch.Tensor | None = None) -> torch.Tensor:
    """GELU x Phi(x) alone: X [M,K] bf16 -> Y [M,K] bf16 (K = 1024 or 4096)."""
    assert X.dim() == 2 and X.element_size() == 2 and X.stride(1) == 1
    M, K = X.shape
    if Y is None:
        Y = torch.empty((M, K), dtype=torch.bfloat16, device=X.device)
    assert Y.is_contiguous() and Y.element_size() == 2
    _check(lib().qvggt_gelu(_ptr(X), X.stride(0) if M > 1 else K, M, K, _ptr(Y), _stream()), "qvggt_gelu")
    return Y


def gelu_rotate_smooth_quantize_c8(w: Weights, X: torch.Tensor, Xq8: torch.Tensor | None = None, a_scale: torch.Tensor | None = None):
    """GELU fused in front of rotate_smooth_quantize_c8 -> (Xq8 [M,K] int8, a_scale [M])."""
    assert X.dim() == 2 and X.element_size() == 2 and X.stride(1) == 1 and X.shape[1] == w.K
    M = X.shape[0]
    if Xq8 is None:
        Xq8 = torch.empty((M, w.K), dtype=torch.int8, device=X.device)
    if a_scale is None:
        a_scale = torch.empty((M,), dtype=torch.float32, device=X.device)
    _check(lib().qvggt_gelu_rotate_smooth_quantize_c8(w.handle, _ptr(X), X.stride(0) if M > 1 else w.K, M, _ptr(Xq8), _ptr(a_scale),
                                                      _stream()), "qvggt_gelu_rotate_smooth_quantize_c8")
    return Xq8, a_scale


def w4a4_linear_c8(w: Weights, Xq8: torch.Tensor, a_scale: torch.Tensor, Y: torch.Tensor | None = None,
                   acc_debug: torch.Tensor | None = None) -> torch.Tensor:
    """-> Y [M,N] bf16 from codes held one per byte.  acc_debug: optional int32 [M,N] receiving the integer sums."""
    M = Xq8.shape[0]
    assert Xq8.dtype == torch.int8 and Xq8.is_contiguous() and Xq8.shape[1] == w.K
    assert a_scale.dtype == torch.float32 and a_scale.is_contiguous()
    if Y is None:
        Y = torch.empty((M, w.N), dtype=torch.bfloat16, device=Xq8.device)
    assert Y.element_size() == 2 and Y.stride(1) == 1 and Y.shape == (M, w.N)
    ldy = Y.stride(0) if M > 1 else w.N
    if acc_debug is not None:
        assert acc_debug.dtype == torch.int32 and acc_debug.is_contiguous()
    _check(lib().qvggt_w4a4_linear_c8(w.handle, _ptr(Xq8), _ptr(a_scale), M, _ptr(Y), ldy, _ptr(acc_debug), _stream()),
           "qvggt_w4a4_linear_c8")
    return Y


def w4a4_linear_c8_packed_weights(w: Weights, Xq8: torch.Tensor, a_scale: torch.Tensor, w_scratch: torch.Tensor,
                                  Y: torch.Tensor | None = None, acc_debug: torch.Tensor | None = None) -> torch.Tensor:
    """The one-code-per-byte GEMM on a handle that keeps only packed weight codes; w_scratch: int8, at least N*K elements."""
    M = Xq8.shape[0]
    assert Xq8.dtype == torch.int8 and Xq8.is_contiguous() and Xq8.shape[1] == w.K
    assert w_scratch.dtype == torch.int8 and w_scratch.is_contiguous() and w_scratch.numel() >= w.N * w.K
    if Y is None:
        Y = torch.empty((M, w.N), dtype=torch.bfloat16, device=Xq8.device)
    ldy = Y.stride(0) if M > 1 else w.N
    _check(lib().qvggt_w4a4_linear_c8_packed_weights(w.handle, _ptr(Xq8), _ptr(a_scale), M, _ptr(Y), ldy, _ptr(w_scratch), _ptr(acc_debug),
                                                     _stream()), "qvggt_w4a4_linear_c8_packed_weights")
    return Y


def rotate_smooth_quantize_c8_expand(w: Weights, X: torch.Tensor, w_scratch: torch.Tensor, Xq8: torch.Tensor | None = None,
                                     a_scale: torch.Tensor | None = None):
    """rotate_smooth_quantize_c8 whose launch also expands the handle's packed weight codes into w_scratch (int8, at
    least N*K elements) -> (Xq8 [M,K] int8, a_scale [M])."""
    assert X.dim() == 2 and X.element_size() == 2 and X.stride(1) == 1 and X.shape[1] == w.K
    assert w_scratch.dtype == torch.int8 and w_scratch.is_contiguous() and w_scratch.numel() >= w.N * w.K
    M = X.shape[0]
    if Xq8 is None:
        Xq8 = torch.empty((M, w.K), dtype=torch.int8, device=X.device)
    if a_scale is None:
        a_scale = torch.empty((M,), dtype=torch.float32, device=X.device)
    _check(lib().qvggt_rotate_smooth_quantize_c8_expand(w.handle, _ptr(X), X.stride(0) if M > 1 else w.K, M, _ptr(Xq8), _ptr(a_scale),
                                                        _ptr(w_scratch), _stream()), "qvggt_rotate_smooth_quantize_c8_expand")
    return Xq8, a_scale


def w4a4_linear_c8_expanded(w: Weights, Xq8: torch.Tensor, a_scale: torch.Tensor, w_scratch: torch.Tensor,
                            Y: torch.Tensor | None = None, acc_debug: torch.Tensor | None = None) -> torch.Tensor:
    """The one-code-per-byte GEMM reading this handle's weight codes from w_scratch, where rotate_smooth_quantize_c8_expand
    put them."""
    M = Xq8.shape[0]
    assert Xq8.dtype == torch.int8 and Xq8.is_contiguous() and Xq8.shape[1] == w.K
    assert w_scratch.dtype == torch.int8 and w_scratch.is_contiguous() and w_scratch.numel() >= w.N * w.K
    if Y is None:
        Y = torch.empty((M, w.N), dtype=torch.bfloat16, device=Xq8.device)
    ldy = Y.stride(0) if M > 1 else w.N
    _check(lib().qvggt_w4a4_linear_c8_expanded(w.handle, _ptr(Xq8), _ptr(a_scale), M, _ptr(Y), ldy, _ptr(w_scratch), _ptr(acc_debug),
                                               _stream()), "qvggt_w4a4_linear_c8_expanded")
    return Y


def debug_starved_linear_c8(w: Weights, Xq8: torch.Tensor, a_scale: torch.Tensor, Y: torch.Tensor, wait_limit_cycles: int) -> int:
    """Test hook: the GEMM launch with its loads switched off and short wait limits; returns the C status of the launch
    (the expired wait shows in w.device_status())."""
    M = Xq8.shape[0]
    return lib().qvggt_debug_starved_linear_c8(w.handle, _ptr(Xq8), _ptr(a_scale), M, _ptr(Y), Y.stride(0) if M > 1 else w.N,
                                               wait_limit_cycles, _stream())


def calibrate_smooth(X_calib: torch.Tensor, W: torch.Tensor, alpha: float = 0.5, lo: float = 1e-2,
                     hi: float = 1e2) -> torch.Tensor:
    """Smoothing factors c [K] fp32 from calibration activations [Mc,K] bf16 and weights [N,K] bf16."""
    assert X_calib.is_contiguous() and W.is_contiguous() and X_calib.element_size() == 2 and W.element_size() == 2
    Mc, K = X_calib.shape
    N = W.shape[0]
    scratch = torch.empty(2 * K, dtype=torch.float32, device=W.device)
    c = torch.empty(K, dtype=torch.float32, device=W.device)
    _check(lib().qvggt_calibrate_smooth(_ptr(X_calib), Mc, _ptr(W), N, K, alpha, lo, hi, _ptr(scratch), _ptr(c), _stream()),
           "qvggt_calibrate_smooth")
    return c


def quantize_weights_static(W: torch.Tensor, smooth_c: torch.Tensor, sign_v: torch.Tensor | None, Wq: torch.Tensor,
                            w_scale: torch.Tensor, amul: torch.Tensor) -> None:
    """Weight quantization into caller-provided buffers without any device allocation.

    For callers that cannot allocate (all device memory already owned by their own arena, or no
    implicit device synchronisation allowed): the temporary multipliers live in a fixed array
    inside the library, so K <= 4096 and concurrent calls on different streams must be serialised.
    W [N,K] bf16, smooth_c [K] fp32, sign_v [K] int8 or None -> Wq [N,K/2] uint8, w_scale [N], amul [K].
    """
    N, K = W.shape
    assert W.element_size() == 2 and W.is_contiguous() and smooth_c.dtype == torch.float32
    assert Wq.dtype == torch.uint8 and Wq.shape == (N, K // 2) and Wq.is_contiguous()
    assert w_scale.dtype == torch.float32 and w_scale.numel() == N and amul.dtype == torch.float32 and amul.numel() == K
    _check(lib().qvggt_quantize_weights_static(_ptr(W), _ptr(smooth_c), _ptr(sign_v), N, K, _ptr(Wq), _ptr(w_scale),
                                               _ptr(amul), _stream()), "qvggt_quantize_weights_static")
