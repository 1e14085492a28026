"""GPU parity of the W8A8 setting (Eq. "quantization" with N = 8, the paper's other configuration) through the same
one-code-per-byte entry points: 8-bit codes and int32 sums bit-exact against the oracle, scales and bf16 outputs
within one bf16 ulp (bit-equal in practice)."""
import numpy as np
import pytest
import torch

import oracle
import workload
from _util import assert_bf16_within_one_ulp, dev_bf16, host_bits

pytestmark = pytest.mark.gpu

q = None
F = workload.TOKENS_PER_FRAME


@pytest.fixture(scope="module", autouse=True)
def _lib():
    global q
    import paper_2509_21302_b200 as pkg
    pkg.build()
    q = pkg
    yield
    torch.cuda.synchronize()


def make_layer(spec, use_signs=False):
    W, b = spec.weight(), spec.bias()
    c = oracle.smooth_factors(spec.x_calib(256), W)
    v = workload.signs_i8(spec.seed, 900 + spec.layer, spec.K) if use_signs else None
    prep = oracle.prepare_weights(W, c, v, bits=8)
    h = q.prepare_weights(dev_bf16(W), dev_bf16(b), torch.from_numpy(c).cuda(),
                          torch.from_numpy(v).cuda() if v is not None else None, bits=8)
    return dict(W=W, b=b, prep=prep, h=h)


@pytest.mark.parametrize("K,N,signs", [(1024, 128, False), (1024, 1024, True), (4096, 256, True)])
def test_w8_prepare_weights_parity(K, N, signs):
    spec = workload.LinearSpec("w", K, N, workload.DIST_GELU if K == 4096 else workload.DIST_NORMAL, 7, 3)
    L = make_layer(spec, signs)
    wq8 = L["h"].view_c8().cpu().numpy()
    assert L["h"].bits == 8
    assert np.array_equal(wq8, L["prep"]["wq"])
    assert np.abs(wq8).max() == 127 and wq8.min() >= -127
    view = L["h"].view()
    assert view["wq"] is None                                        # no packed copy of 8-bit codes
    assert np.array_equal(view["w_scale"].cpu().numpy(), L["prep"]["w_scale"])
    assert L["h"].device_status() == 0


@pytest.mark.parametrize("K", [1024, 4096])
@pytest.mark.parametrize("M", [1, 5, 129, 1374])
def test_a8_rotate_smooth_quantize_parity(K, M):
    spec = workload.LinearSpec("a", K, 128, workload.DIST_GELU if K == 4096 else workload.DIST_NORMAL, 1, 1)
    L = make_layer(spec, use_signs=True)
    X = spec.x_rows(0, M)
    X[0, :] = 0 if M > 1 else X[0]                                    # a zero row among the others
    codes, scales = oracle.rotate_smooth_quantize(X, L["prep"]["amul"], 0, 8)
    Xq8, a_scale = q.rotate_smooth_quantize_c8(L["h"], dev_bf16(X))
    assert np.array_equal(Xq8.cpu().numpy(), codes)
    assert np.array_equal(a_scale.cpu().numpy(), scales)


@pytest.mark.parametrize("K,N,M", [(1024, 128, 1), (1024, 256, 127), (1024, 1024, 129), (4096, 256, 300),
                                   (1024, 384, 257), (4096, 1024, 1374)])
def test_w8a8_linear_parity(K, N, M):
    spec = workload.LinearSpec("g", K, N, workload.DIST_GELU if K == 4096 else workload.DIST_NORMAL, 9, 2)
    L = make_layer(spec, use_signs=(N == 256))
    X = spec.x_rows(0, M)
    ref = oracle.w4a4_linear(X, L["prep"], L["b"], 0)                 # the oracle path takes N = 8 from the prepared weights
    Xq8, a_scale = q.rotate_smooth_quantize_c8(L["h"], dev_bf16(X))
    acc = torch.full((M, N), -123456, dtype=torch.int32, device="cuda")
    Y = q.w4a4_linear_c8(L["h"], Xq8, a_scale, acc_debug=acc)
    Y2 = q.w4a4_linear_c8(L["h"], Xq8, a_scale)
    assert L["h"].device_status() == 0
    assert np.array_equal(Xq8.cpu().numpy(), ref["xq"]) and np.abs(ref["xq"]).max() == 127
    assert np.array_equal(acc.cpu().numpy(), ref["acc"])
    assert assert_bf16_within_one_ulp(host_bits(Y), ref["y"]) == 0.0
    assert np.array_equal(host_bits(Y2), host_bits(Y))
    # 8 bits are closer to the unquantized layer than 4 bits (information, with a loose bar)
    full = oracle.linear_f64(X, L["W"], L["b"])
    y = oracle.bf16_to_f32(host_bits(Y)).astype(np.float64)
    if M >= 127:
        assert np.linalg.norm(y - full) / np.linalg.norm(full) < 0.05


def test_w8a8_extreme_codes_and_refusals():
    """Codes of magnitude 127 everywhere: the sums reach +-127^2 K = 66 064 384 at K = 4096 (beyond 2^24: the
    int32 -> fp32 conversion of the epilogue rounds, identically on both sides)."""
    K, N, M = 4096, 128, 130
    W = np.zeros((N, K), np.uint16)
    W[np.arange(N), np.arange(N)] = 0x3F80       # row n = e_n: its rotation is row n of H_K, so every code is +-127
    h = q.prepare_weights(dev_bf16(W), None, torch.ones(K, device="cuda"), None, bits=8)
    wq = h.view_c8().cpu().numpy()
    assert np.all(np.abs(wq) == 127)
    xq = np.ascontiguousarray(np.tile(wq, (2, 1))[:M])
    xq[1] = -xq[1]
    xq[2] = 0
    a_np = np.full(M, 0.5, np.float32)
    acc = torch.zeros((M, N), dtype=torch.int32, device="cuda")
    Y = q.w4a4_linear_c8(h, torch.from_numpy(xq).cuda(), torch.from_numpy(a_np).cuda(), acc_debug=acc)
    want_acc = oracle.gemm_i32(xq, wq)
    assert want_acc[0, 0] == 127 * 127 * K and want_acc[1, 1] == -127 * 127 * K and not want_acc[2].any()
    assert np.array_equal(acc.cpu().numpy(), want_acc)
    want = oracle.epilogue(want_acc, a_np, h.view()["w_scale"].cpu().numpy(), None)
    assert assert_bf16_within_one_ulp(host_bits(Y), want) == 0.0
    assert h.device_status() == 0
    # the packed entry points refuse an 8-bit handle
    X = torch.zeros((4, K), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(q.QvggtError) as err:
        q.rotate_smooth_quantize(h, X, 0)
    assert err.value.status == -4
    with pytest.raises(q.QvggtError) as err:
        q.w4a4_linear(h, torch.zeros((4, K // 2), dtype=torch.uint8, device="cuda"), torch.ones(4, device="cuda"), 0)
    assert err.value.status == -4


@pytest.mark.parametrize("which", [0, 1, 2, 3])
def test_w8a8_config2_full_size_every_row(which):
    """The four linears of the block at 8 frames (M = 10992), the launch configuration the benchmark times, with 8-bit
    codes: every row of codes, scales and outputs against the oracle; for qkv and fc2 the int32 sums as well (8-bit sums
    reach 127^2 K: the largest accumulators the kernel sees)."""
    spec = workload.block_specs(0, 0)[which]
    M = 8 * F
    W, b = spec.weight(), spec.bias()
    c = oracle.smooth_factors(spec.x_calib(256), W)
    prep = oracle.prepare_weights(W, c, None, bits=8)
    h = q.prepare_weights(dev_bf16(W), dev_bf16(b), torch.from_numpy(c).cuda(), None, bits=8)
    X = spec.x_rows(0, M)
    Xq8, a_scale = q.rotate_smooth_quantize_c8(h, dev_bf16(X))
    codes, scales = oracle.rotate_smooth_quantize(X, prep["amul"], 0, 8)
    assert np.array_equal(Xq8.cpu().numpy(), codes)
    assert np.array_equal(a_scale.cpu().numpy(), scales)
    dump = which in (0, 3)
    acc = torch.full((M, spec.N), -12345, dtype=torch.int32, device="cuda") if dump else None
    Y = q.w4a4_linear_c8(h, Xq8, a_scale, acc_debug=acc)
    want_acc = oracle.gemm_i32(codes, prep["wq"])
    if dump:
        assert np.array_equal(acc.cpu().numpy(), want_acc)
        Yp = q.w4a4_linear_c8(h, Xq8, a_scale)                      # production instantiation
        assert torch.equal(Yp.view(torch.int16), Y.view(torch.int16))
    want = oracle.epilogue(want_acc, scales, prep["w_scale"], b)
    assert assert_bf16_within_one_ulp(host_bits(Y), want, spec.name) == 0.0
    assert h.device_status() == 0
    h.free()
