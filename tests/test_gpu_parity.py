"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle on the same seeded inputs.

Bar: int4 codes and int32 sums bit-exact; scales and bf16 outputs within one bf16 ulp
(relative error <= 2^-7) -- in practice bit-equal, which the tests also report.
"""
import numpy as np
import pytest
import torch

import oracle
import workload
from _util import assert_bf16_within_one_ulp, dev_bf16, host_bits, unpack_codes

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


def make_layer(spec, use_signs=False, calib_rows=256):
    """Host inputs of one linear layer + oracle-prepared weights + GPU handle."""
    W, b = spec.weight(), spec.bias()
    c = oracle.smooth_factors(spec.x_calib(calib_rows), W)
    v = workload.signs_i8(spec.seed, 900 + spec.layer, spec.K) if use_signs else None
    prep = oracle.prepare_weights(W, c, v)
    h = q.prepare_weights(dev_bf16(W), dev_bf16(b), torch.from_numpy(c).cuda(),
                          torch.from_numpy(v).cuda() if v is not None else None)
    return dict(W=W, b=b, c=c, v=v, prep=prep, h=h)


def check_scales(got, want, what):
    got, want = np.asarray(got), np.asarray(want)
    assert np.all(np.abs(got.astype(np.float64) - want) <= 2.0 ** -7 * np.abs(want)), what
    return float((got != want).mean())


# ------------------------------------------------------------------------------ offline weight path
@pytest.mark.parametrize("K,N,signs", [(1024, 128, False), (1024, 1024, True), (4096, 256, True), (4096, 1024, False)])
def test_prepare_weights_parity(K, N, signs):
    spec = workload.LinearSpec("w", K, N, workload.DIST_GELU if K == 4096 else workload.DIST_NORMAL, 7, 3)
    L = make_layer(spec, signs)
    view = L["h"].view()
    assert np.array_equal(view["amul"].cpu().numpy(), L["prep"]["amul"])
    assert np.array_equal(view["wq"].cpu().numpy(), L["prep"]["wq_packed"])
    assert check_scales(view["w_scale"].cpu().numpy(), L["prep"]["w_scale"], "w_scale") == 0.0
    assert np.array_equal(host_bits(view["bias"]), L["b"])
    assert L["h"].device_status() == 0


# ------------------------------------------------------------------------------ rotate-smooth-quantize
@pytest.mark.parametrize("K", [1024, 4096])
@pytest.mark.parametrize("group", [0, 128])
@pytest.mark.parametrize("M", [1, 5, 127, 129, 1374])
def test_rotate_smooth_quantize_parity(K, group, M):
    spec = workload.LinearSpec("a", K, 128, workload.DIST_GELU if K == 4096 else workload.DIST_NORMAL, 1, 1)
    L = make_layer(spec, use_signs=True)
    X = spec.x_rows(0, M)
    codes, scales = oracle.rotate_smooth_quantize(X, L["prep"]["amul"], group)
    Xq, a_scale = q.rotate_smooth_quantize(L["h"], dev_bf16(X), group)
    assert np.array_equal(unpack_codes(Xq.cpu().numpy()), codes)
    assert np.array_equal(Xq.cpu().numpy(), oracle.pack_int4(codes))
    assert check_scales(a_scale.cpu().numpy(), scales, "a_scale") == 0.0


@pytest.mark.parametrize("K", [1024, 4096])
def test_rotate_smooth_quantize_edge_rows(K):
    spec = workload.LinearSpec("e", K, 128, workload.DIST_NORMAL, 2, 0)
    L = make_layer(spec)
    X = spec.x_rows(0, 8)
    X[0] = 0                                    # all-zero row -> codes 0, floor scale
    X[1] = 0
    X[1, K // 3] = 0x4580                       # single spike
    X[2] = 0
    X[2, 0] = 0x7F7F                            # one element at the largest finite bf16
    X[3] = 0
    X[3, 0] = 0xFF7F                            # and its negative
    X[4, :] = 0x3F80                            # all ones: the transform concentrates everything in channel 0
    X[5, ::2] = 0x3F80
    X[5, 1::2] = 0xBF80                         # alternating signs
    for group in (0, 128):
        codes, scales = oracle.rotate_smooth_quantize(X, L["prep"]["amul"], group)
        Xq, a_scale = q.rotate_smooth_quantize(L["h"], dev_bf16(X), group)
        assert np.array_equal(unpack_codes(Xq.cpu().numpy()), codes), group
        assert np.array_equal(a_scale.cpu().numpy(), scales), group
    assert not codes[0].any()


def test_rotate_smooth_quantize_near_ties():
    """Rows whose rotated values sit on or next to .5 boundaries of y * (7/amax): both sides must
    take the same half-to-even decision from the exact product."""
    K = 1024
    c = np.full(K, 2.0 ** -5, np.float32)        # amul = K^-1/2 / c = 1 exactly
    W = workload.normal_bf16(3, 1, 128, K, 0.02)
    h = q.prepare_weights(dev_bf16(W), None, torch.from_numpy(c).cuda(), None)
    amul, _ = oracle.multipliers(c)
    assert np.all(amul == 1.0)
    rng = np.random.default_rng(5)
    y = rng.integers(-13, 14, size=(16, K)).astype(np.float64) * 0.5    # multiples of 0.5 in [-6.5, 6.5]
    y[:, 0] = 7.0                                                       # amax = 7 -> 7/amax = 1
    x = (y @ _sylvester(K)) / K                                         # x H_K = y before rounding x to bf16
    X = np.ascontiguousarray((x.astype(np.float32).view(np.uint32) >> 16).astype(np.uint16))
    codes, scales = oracle.rotate_smooth_quantize(X, amul, 0)
    Xq, a_scale = q.rotate_smooth_quantize(h, dev_bf16(X), 0)
    assert np.array_equal(unpack_codes(Xq.cpu().numpy()), codes)
    assert np.array_equal(a_scale.cpu().numpy(), scales)


def _sylvester(K):
    i = np.arange(K, dtype=np.int64)
    x = i[:, None] & i[None, :]
    pc = np.zeros_like(x)
    while np.any(x):
        pc += x & 1
        x >>= 1
    return (1 - 2 * (pc & 1)).astype(np.float64)


def test_strided_input_and_empty_batch():
    spec = workload.LinearSpec("s", 1024, 128, workload.DIST_NORMAL, 4, 0)
    L = make_layer(spec)
    X = spec.x_rows(0, 37)
    wide = torch.zeros((37, 1024 + 64), dtype=torch.bfloat16, device="cuda")
    wide[:, :1024] = dev_bf16(X)
    Xq, a_scale = q.rotate_smooth_quantize(L["h"], wide[:, :1024], 0)
    codes, scales = oracle.rotate_smooth_quantize(X, L["prep"]["amul"], 0)
    assert np.array_equal(unpack_codes(Xq.cpu().numpy()), codes)
    assert np.array_equal(a_scale.cpu().numpy(), scales)
    Ywide = torch.zeros((37, 128 + 8), dtype=torch.bfloat16, device="cuda")
    q.w4a4_linear(L["h"], Xq, a_scale, 0, Y=Ywide[:, :128])
    want = oracle.epilogue(oracle.gemm_i32(codes, L["prep"]["wq"]), scales, L["prep"]["w_scale"], L["b"])
    assert_bf16_within_one_ulp(host_bits(Ywide[:, :128]), want)
    assert not Ywide[:, 128:].any()                                   # nothing written past N
    # M = 0 is a no-op
    e = torch.empty((0, 1024), dtype=torch.bfloat16, device="cuda")
    Xq0, s0 = q.rotate_smooth_quantize(L["h"], e, 0)
    assert q.w4a4_linear(L["h"], Xq0, s0, 0).shape == (0, 128)
    assert L["h"].device_status() == 0


# ------------------------------------------------------------------------------ GEMM + epilogue
@pytest.mark.parametrize("K,N,M", [(1024, 128, 1), (1024, 256, 127), (1024, 1024, 129), (4096, 256, 300),
                                   (1024, 384, 257), (4096, 1024, 1374)])
def test_w4a4_linear_parity(K, N, M):
    spec = workload.LinearSpec("g", K, N, workload.DIST_GELU if K == 4096 else workload.DIST_NORMAL, 9, 2)
    L = make_layer(spec, use_signs=(N == 256))
    X = spec.x_rows(0, M)
    ref = oracle.w4a4_linear(X, L["prep"], L["b"], 0)
    Xq, a_scale = q.rotate_smooth_quantize(L["h"], dev_bf16(X), 0)
    acc = torch.full((M, N), -123456, dtype=torch.int32, device="cuda")
    Y = q.w4a4_linear(L["h"], Xq, a_scale, 0, acc_debug=acc)
    assert L["h"].device_status() == 0
    assert np.array_equal(acc.cpu().numpy(), ref["acc"])               # int32 sums bit-exact
    frac = assert_bf16_within_one_ulp(host_bits(Y), ref["y"])
    assert frac == 0.0, f"{frac:.3e} of the outputs differ in the last bit (allowed, but unexpected)"


@pytest.mark.parametrize("K,N,M", [(1024, 128, 1), (1024, 384, 257), (4096, 256, 300), (1024, 1024, 1374)])
def test_w4a4_linear_group128_parity(K, N, M):
    """One activation scale per token per 128 rotated channels: per-group integer sums bit-exact,
    outputs against the oracle's ascending-group fp32 accumulation."""
    spec = workload.LinearSpec("gg", K, N, workload.DIST_GELU if K == 4096 else workload.DIST_NORMAL, 11, 1)
    L = make_layer(spec, use_signs=(N == 256))
    X = spec.x_rows(0, M)
    ref = oracle.w4a4_linear(X, L["prep"], L["b"], 128)
    Xq, a_scale = q.rotate_smooth_quantize(L["h"], dev_bf16(X), 128)
    assert np.array_equal(a_scale.cpu().numpy(), ref["a_scale"])
    acc = torch.full((K // 128, M, N), -123456, dtype=torch.int32, device="cuda")
    Y = q.w4a4_linear(L["h"], Xq, a_scale, 128, acc_debug=acc)
    assert L["h"].device_status() == 0
    assert np.array_equal(acc.cpu().numpy(), ref["acc"])               # per-group int32 sums bit-exact
    frac = assert_bf16_within_one_ulp(host_bits(Y), ref["y"])
    assert frac == 0.0, f"{frac:.3e} of the outputs differ in the last bit (allowed, but unexpected)"


def test_w4a4_linear_extreme_codes():
    """Codes of magnitude 7 everywhere: the sums reach +-49 K, the largest possible; plus a zero token."""
    K, N, M = 4096, 128, 130
    W = np.zeros((N, K), np.uint16)
    W[np.arange(N), np.arange(N)] = 0x3F80       # row n = e_n: its rotation is row n of H_K, so every code is +-7
    h = q.prepare_weights(dev_bf16(W), None, torch.ones(K, device="cuda"), None)
    wq = unpack_codes(h.view()["wq"].cpu().numpy())
    assert np.all(np.abs(wq) == 7)
    xq = np.ascontiguousarray(np.tile(wq, (2, 1))[:M])                  # token m carries the pattern of channel m % N
    xq[1] = -xq[1]
    xq[2] = 0
    a_np = np.full(M, 0.5, np.float32)
    acc = torch.zeros((M, N), dtype=torch.int32, device="cuda")
    Y = q.w4a4_linear(h, torch.from_numpy(oracle.pack_int4(xq)).cuda(), torch.from_numpy(a_np).cuda(), 0, acc_debug=acc)
    want_acc = oracle.gemm_i32(xq, wq)
    assert want_acc[0, 0] == 49 * K and want_acc[1, 1] == -49 * K and not want_acc[2].any()
    assert np.array_equal(acc.cpu().numpy(), want_acc)
    want = oracle.epilogue(want_acc, a_np, h.view()["w_scale"].cpu().numpy(), None)
    assert assert_bf16_within_one_ulp(host_bits(Y), want) == 0.0
    assert h.device_status() == 0


# ------------------------------------------------------------------------------ calibration helper
@pytest.mark.parametrize("K,N,rows", [(1024, 256, 300), (4096, 256, 300), (1024, 3072, 10992), (4096, 1024, 10992), (1024, 128, 1)])
def test_calibrate_smooth_matches_oracle(K, N, rows):
    """Column maxima of the rotated calibration rows and weight rows and Eq. "smooth_factor" on them: a few hundred rows, one
    row, and the block's own sizes (every thread block then walks through many rows)."""
    spec = workload.LinearSpec("c", K, N, workload.DIST_NORMAL, 6, 0)
    Xc, W = spec.x_calib(rows), spec.weight()
    want = oracle.smooth_factors(Xc, W)
    got = q.calibrate_smooth(dev_bf16(Xc), dev_bf16(W)).cpu().numpy()
    assert np.allclose(got, want, rtol=2e-5, atol=0)


# ------------------------------------------------------------------------------ the single-frame proj layer (the smallest benchmark configuration)
def test_config1_single_frame_proj():
    spec = workload.LinearSpec("proj", 1024, 1024, workload.DIST_NORMAL, 0, 1)
    L = make_layer(spec, calib_rows=workload.TOKENS_PER_FRAME)
    M = workload.TOKENS_PER_FRAME
    X = spec.x_rows(0, M)
    ref = oracle.w4a4_linear(X, L["prep"], L["b"], 0)
    Xq, a_scale = q.rotate_smooth_quantize(L["h"], dev_bf16(X), 0)
    acc = torch.zeros((M, 1024), dtype=torch.int32, device="cuda")
    Y = q.w4a4_linear(L["h"], Xq, a_scale, 0, acc_debug=acc)
    assert np.array_equal(unpack_codes(Xq.cpu().numpy()), ref["xq"])
    assert np.array_equal(a_scale.cpu().numpy(), ref["a_scale"])
    assert np.array_equal(acc.cpu().numpy(), ref["acc"])
    assert assert_bf16_within_one_ulp(host_bits(Y), ref["y"]) == 0.0
    full = oracle.linear_f64(X, L["W"], L["b"])
    y = oracle.bf16_to_f32(host_bits(Y)).astype(np.float64)
    rel = np.linalg.norm(y - full) / np.linalg.norm(full)
    print(f"config 1: relative error vs the unquantized fp64 layer = {rel:.4f} (information only)")
    assert rel < 0.3
