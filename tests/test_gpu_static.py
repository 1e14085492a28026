"""GPU parity of the static tensor-wise activation quantizer (the other arm of the paper's granularity ablation,
Tab. "granularity") against the oracle: codes bit-exact including both ends of the clamp, every row's scale equal
to the given step size, and the GEMM + epilogue that follow within one bf16 ulp (bit-equal in practice)."""
import numpy as np
import pytest
import torch

import oracle
import workload
from _util import assert_bf16_within_one_ulp, dev_bf16, host_bits

pytestmark = pytest.mark.gpu

q = None


@pytest.fixture(scope="module", autouse=True)
def _lib():
    global q
    import paper_2509_21302_b200 as pkg
    pkg.build()
    q = pkg
    yield
    torch.cuda.synchronize()


@pytest.mark.parametrize("bits", [4, 8])
@pytest.mark.parametrize("K,delta", [(1024, 2.0 ** -4), (1024, 0.037), (4096, 0.25), (4096, 0.0913)])
def test_static_quantizer_parity(K, delta, bits):
    N, M = 256, 301
    spec = workload.LinearSpec("s", K, N, workload.DIST_GELU if K == 4096 else workload.DIST_NORMAL, 31, 2)
    W, b = spec.weight(), spec.bias()
    c = oracle.smooth_factors(spec.x_calib(256), W)
    v = workload.signs_i8(31, 7, K)
    prep = oracle.prepare_weights(W, c, v, bits=bits)
    h = q.prepare_weights(dev_bf16(W), dev_bf16(b), torch.from_numpy(c).cuda(), torch.from_numpy(v).cuda(), c8=True, bits=bits)
    X = spec.x_rows(0, M)                         # the first five rows are x100 special tokens: they saturate
    X[7] = 0                                      # a zero row
    X[8] = 0
    X[8, 3] = 0x7F7F                              # the largest finite bf16: far beyond the clamp
    X[9] = 0
    X[9, 5] = 0xFF7F
    d32 = np.float32(delta)
    codes = oracle.rotate_smooth_quantize_static(X, prep["amul"], float(d32), bits)
    Xq8, a_scale = q.rotate_smooth_quantize_static_c8(h, dev_bf16(X), torch.tensor([d32], device="cuda"))
    lo, hi = -(2 ** (bits - 1)), 2 ** (bits - 1) - 1
    assert codes.min() == lo and codes.max() == hi                 # both ends of the clamp occur
    assert np.array_equal(Xq8.cpu().numpy(), codes)
    assert np.array_equal(a_scale.cpu().numpy(), np.full(M, d32, np.float32))
    acc = torch.zeros((M, N), dtype=torch.int32, device="cuda")
    Y = q.w4a4_linear_c8(h, Xq8, a_scale, acc_debug=acc)
    want_acc = oracle.gemm_i32(codes, prep["wq"])
    assert np.array_equal(acc.cpu().numpy(), want_acc)
    want = oracle.epilogue(want_acc, np.full(M, d32, np.float32), prep["w_scale"], b)
    assert assert_bf16_within_one_ulp(host_bits(Y), want) == 0.0
    assert h.device_status() == 0


@pytest.mark.parametrize("bits", [4, 8])
@pytest.mark.parametrize("which", [2, 3])
def test_static_quantizer_full_size_every_row(which, bits):
    """fc1 and fc2 inputs at 8 frames (M = 10992) with a step size taken from the dynamic scales' median: every row."""
    spec = workload.block_specs(0, 0)[which]
    M = 8 * workload.TOKENS_PER_FRAME
    W = spec.weight()
    c = oracle.smooth_factors(spec.x_calib(256), W)
    prep = oracle.prepare_weights(W, c, None, bits=bits)
    h = q.prepare_weights(dev_bf16(W), None, torch.from_numpy(c).cuda(), None, c8=True, bits=bits)
    X = spec.x_rows(0, M)
    Xd = dev_bf16(X)
    _, dyn = q.rotate_smooth_quantize_c8(h, Xd)
    delta = dyn.median().reshape(1).contiguous()
    Xq8, a_scale = q.rotate_smooth_quantize_static_c8(h, Xd, delta)
    codes = oracle.rotate_smooth_quantize_static(X, prep["amul"], float(delta.item()), bits)
    assert np.abs(codes.astype(np.int32)).max() >= (7 if bits == 4 else 127)      # the clamp is active on the rows above the median
    assert np.array_equal(Xq8.cpu().numpy(), codes)
    assert torch.all(a_scale == delta)
    h.free()


@pytest.mark.parametrize("bits", [4, 8])
@pytest.mark.parametrize("K,N", [(1024, 384), (4096, 128), (1024, 4096)])
def test_tensorwise_weight_quantizer_matches_the_oracle_through_the_layer(K, N, bits):
    """QVGGT_PREP_W_TENSORWISE (the weight side of Tab. "granularity"): one step size for the whole weight tensor.  Codes and the
    step bit-exact against the oracle, and the layer built on them reproduces the oracle's sums and outputs."""
    import workload
    M = 300
    spec = workload.LinearSpec("tw", K, N, workload.DIST_NORMAL, 51, 0)
    W, b, X = spec.weight(), spec.bias(), spec.x_rows(0, M)
    c = oracle.smooth_factors(spec.x_calib(128), W)
    prep = oracle.prepare_weights(W, c, None, bits, tensorwise=True)
    h = q.prepare_weights(dev_bf16(W), dev_bf16(b), torch.from_numpy(c).cuda(), None, c8=("only" if bits == 4 else True), bits=bits, w_tensorwise=True)
    assert np.array_equal(h.view_c8().cpu().numpy(), prep["wq"])
    assert np.array_equal(h.view()["w_scale"].cpu().numpy(), prep["w_scale"])
    ref = oracle.w4a4_linear(X, prep, b, 0)
    Xq8, a = q.rotate_smooth_quantize_c8(h, dev_bf16(X))
    acc = torch.zeros((M, N), dtype=torch.int32, device="cuda")
    Y = q.w4a4_linear_c8(h, Xq8, a, acc_debug=acc)
    assert np.array_equal(acc.cpu().numpy(), ref["acc"]) and np.array_equal(host_bits(Y), ref["y"])
    assert h.device_status() == 0
    h.free()
    # the flag needs a handle without packed copy
    import ctypes
    out = ctypes.c_void_p()
    Wd, cd = dev_bf16(W), torch.from_numpy(c).cuda()
    st = q.lib().qvggt_prepare_weights(Wd.data_ptr(), None, cd.data_ptr(), None, N, K, 8, torch.cuda.current_stream().cuda_stream, ctypes.byref(out))
    assert st == -4 and out.value is None
