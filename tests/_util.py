"""Helpers shared by the GPU parity tests (marshalling between numpy bf16 bit patterns and torch)."""
import numpy as np
import torch


def dev_bf16(bits: np.ndarray) -> torch.Tensor:
    """numpy uint16 bf16 bit patterns -> CUDA bfloat16 tensor with the same bytes."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def host_bits(t: torch.Tensor) -> np.ndarray:
    """CUDA bfloat16 tensor -> numpy uint16 bit patterns."""
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def bf16_value(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32)


def unpack_codes(packed: np.ndarray) -> np.ndarray:
    """Canonical layout: byte i = code 2i (bits 0-3) | code 2i+1 (bits 4-7), two's complement."""
    lo = (packed & 0xF).astype(np.int8)
    hi = (packed >> 4).astype(np.int8)
    lo = np.where(lo >= 8, lo - 16, lo).astype(np.int8)
    hi = np.where(hi >= 8, hi - 16, hi).astype(np.int8)
    out = np.empty(packed.shape[:-1] + (packed.shape[-1] * 2,), np.int8)
    out[..., 0::2] = lo
    out[..., 1::2] = hi
    return out


def assert_bf16_within_one_ulp(got_bits: np.ndarray, want_bits: np.ndarray, what: str = "Y") -> float:
    """Tolerance for bf16 outputs: equal or adjacent bf16 values, or |diff| <= 2^-7 |want|.

    Returns the fraction of elements that are not bit-equal (expected 0: the kernel uses the same
    separate multiply, multiply, add as the oracle)."""
    same = got_bits == want_bits
    if same.all():
        return 0.0
    # only the elements that differ go through the tolerance (whole-output comparisons hold ~10^9 elements)
    n = got_bits.size
    got_bits, want_bits = got_bits[~same], want_bits[~same]
    g = bf16_value(got_bits).astype(np.float64)
    w = bf16_value(want_bits).astype(np.float64)
    assert np.all(np.isfinite(g)), f"{what}: non-finite output"
    rel_ok = np.abs(g - w) <= 2.0 ** -7 * np.abs(w)
    # adjacent representable values: the ordered-integer views differ by one
    def key(b):
        b = b.astype(np.int32)
        return np.where(b & 0x8000, -(b & 0x7FFF), b & 0x7FFF)
    adj = np.abs(key(got_bits) - key(want_bits)) <= 1
    bad = ~(rel_ok | adj)
    assert not bad.any(), f"{what}: {bad.sum()} elements beyond 1 bf16 ulp"
    return float(got_bits.size) / n
