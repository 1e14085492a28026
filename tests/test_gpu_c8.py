"""GPU parity of the 8-bit-container entry points (one int4 code per byte between the kernels) against the CPU
oracle: the codes, scales, int32 sums and bf16 outputs must be those of the packed path, i.e. of the oracle --
int4 codes and int32 sums bit-exact, scales and outputs within one bf16 ulp (bit-equal in practice).
"""
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


def make_layer(spec, use_signs=False, calib_rows=256):
    W, b = spec.weight(), spec.bias()
    c = oracle.smooth_factors(spec.x_calib(calib_rows), W)
    v = workload.signs_i8(spec.seed, 900 + spec.layer, spec.K) if use_signs else None
    prep = oracle.prepare_weights(W, c, v)
    h = q.prepare_weights(dev_bf16(W), dev_bf16(b), torch.from_numpy(c).cuda(),
                          torch.from_numpy(v).cuda() if v is not None else None, c8=True)
    return dict(W=W, b=b, prep=prep, h=h)


@pytest.mark.parametrize("K,N,signs", [(1024, 128, False), (1024, 1024, True), (4096, 256, True), (4096, 1024, False)])
def test_prepare_weights_c8_parity(K, N, signs):
    spec = workload.LinearSpec("w", K, N, workload.DIST_GELU if K == 4096 else workload.DIST_NORMAL, 7, 3)
    L = make_layer(spec, signs)
    assert np.array_equal(L["h"].view_c8().cpu().numpy(), L["prep"]["wq"])          # one code per byte
    assert np.array_equal(L["h"].view()["wq"].cpu().numpy(), L["prep"]["wq_packed"])  # the packed copy is still there
    assert np.array_equal(L["h"].view()["w_scale"].cpu().numpy(), L["prep"]["w_scale"])
    assert L["h"].device_status() == 0


@pytest.mark.parametrize("K", [1024, 4096])
@pytest.mark.parametrize("M", [1, 5, 127, 129, 1374])
def test_rotate_smooth_quantize_c8_parity(K, M):
    spec = workload.LinearSpec("a", K, 128, workload.DIST_GELU if K == 4096 else workload.DIST_NORMAL, 1, 1)
    L = make_layer(spec, use_signs=True)
    X = spec.x_rows(0, M)
    codes, scales = oracle.rotate_smooth_quantize(X, L["prep"]["amul"], 0)
    Xq8, a_scale = q.rotate_smooth_quantize_c8(L["h"], dev_bf16(X))
    assert np.array_equal(Xq8.cpu().numpy(), codes)
    assert np.array_equal(a_scale.cpu().numpy(), scales)


@pytest.mark.parametrize("K", [1024, 4096])
def test_rotate_smooth_quantize_c8_edge_rows(K):
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
    codes, scales = oracle.rotate_smooth_quantize(X, L["prep"]["amul"], 0)
    Xq8, a_scale = q.rotate_smooth_quantize_c8(L["h"], dev_bf16(X))
    assert np.array_equal(Xq8.cpu().numpy(), codes)
    assert np.array_equal(a_scale.cpu().numpy(), scales)
    assert not codes[0].any() and codes.min() >= -7 and codes.max() <= 7


def test_c8_strided_input_empty_batch_and_missing_copy():
    spec = workload.LinearSpec("s", 1024, 128, workload.DIST_NORMAL, 4, 0)
    L = make_layer(spec)
    X = spec.x_rows(0, 37)
    wide = torch.zeros((37, 1024 + 64), dtype=torch.bfloat16, device="cuda")
    wide[:, :1024] = dev_bf16(X)
    Xq8, a_scale = q.rotate_smooth_quantize_c8(L["h"], wide[:, :1024])
    codes, scales = oracle.rotate_smooth_quantize(X, L["prep"]["amul"], 0)
    assert np.array_equal(Xq8.cpu().numpy(), codes)
    Ywide = torch.zeros((37, 128 + 8), dtype=torch.bfloat16, device="cuda")
    q.w4a4_linear_c8(L["h"], Xq8, a_scale, Y=Ywide[:, :128])
    want = oracle.epilogue(oracle.gemm_i32(codes, L["prep"]["wq"]), scales, L["prep"]["w_scale"], L["b"])
    assert assert_bf16_within_one_ulp(host_bits(Ywide[:, :128]), want) == 0.0
    assert not Ywide[:, 128:].any()                                   # nothing written past N
    e = torch.empty((0, 1024), dtype=torch.bfloat16, device="cuda")
    Xq0, s0 = q.rotate_smooth_quantize_c8(L["h"], e)
    assert q.w4a4_linear_c8(L["h"], Xq0, s0).shape == (0, 128)
    assert L["h"].device_status() == 0
    # a handle prepared without the one-code-per-byte copy refuses the c8 GEMM
    plain = q.prepare_weights(dev_bf16(L["W"]), None, torch.ones(1024, device="cuda"), None)
    assert plain.view_c8() is None
    with pytest.raises(q.QvggtError) as err:
        q.w4a4_linear_c8(plain, Xq8, a_scale)
    assert err.value.status == -4


@pytest.mark.parametrize("K,N,M", [(1024, 128, 1), (1024, 256, 127), (1024, 1024, 129), (4096, 256, 300),
                                   (1024, 384, 257), (4096, 1024, 1374), (1024, 3072, 2500)])
def test_w4a4_linear_c8_parity(K, N, M):
    spec = workload.LinearSpec("g", K, N, workload.DIST_GELU if K == 4096 else workload.DIST_NORMAL, 9, 2)
    L = make_layer(spec, use_signs=(N == 256))
    X = spec.x_rows(0, M)
    ref = oracle.w4a4_linear(X, L["prep"], L["b"], 0)
    Xq8, a_scale = q.rotate_smooth_quantize_c8(L["h"], dev_bf16(X))
    acc = torch.full((M, N), -123456, dtype=torch.int32, device="cuda")
    Y = q.w4a4_linear_c8(L["h"], Xq8, a_scale, acc_debug=acc)
    Y2 = q.w4a4_linear_c8(L["h"], Xq8, a_scale)                         # the production instantiation (no dump)
    assert L["h"].device_status() == 0
    assert np.array_equal(Xq8.cpu().numpy(), ref["xq"])
    assert np.array_equal(acc.cpu().numpy(), ref["acc"])               # int32 sums bit-exact
    assert assert_bf16_within_one_ulp(host_bits(Y), ref["y"]) == 0.0
    assert np.array_equal(host_bits(Y2), host_bits(Y))


def test_w4a4_linear_c8_extreme_codes():
    """Codes of magnitude 7 everywhere: the sums reach +-49 K, the largest possible; plus a zero token."""
    K, N, M = 4096, 128, 130
    W = np.zeros((N, K), np.uint16)
    W[np.arange(N), np.arange(N)] = 0x3F80       # row n = e_n: its rotation is row n of H_K, so every code is +-7
    h = q.prepare_weights(dev_bf16(W), None, torch.ones(K, device="cuda"), None, c8=True)
    wq = h.view_c8().cpu().numpy()
    assert np.all(np.abs(wq) == 7)
    xq = np.ascontiguousarray(np.tile(wq, (2, 1))[:M])                  # token m carries the pattern of channel m % N
    xq[1] = -xq[1]
    xq[2] = 0
    a_np = np.full(M, 0.5, np.float32)
    acc = torch.zeros((M, N), dtype=torch.int32, device="cuda")
    Y = q.w4a4_linear_c8(h, torch.from_numpy(xq).cuda(), torch.from_numpy(a_np).cuda(), acc_debug=acc)
    want_acc = oracle.gemm_i32(xq, wq)
    assert want_acc[0, 0] == 49 * K and want_acc[1, 1] == -49 * K and not want_acc[2].any()
    assert np.array_equal(acc.cpu().numpy(), want_acc)
    want = oracle.epilogue(want_acc, a_np, h.view()["w_scale"].cpu().numpy(), None)
    assert assert_bf16_within_one_ulp(host_bits(Y), want) == 0.0
    assert h.device_status() == 0


def test_c8_config1_single_frame_proj():
    spec = workload.LinearSpec("proj", 1024, 1024, workload.DIST_NORMAL, 0, 1)
    L = make_layer(spec, calib_rows=workload.TOKENS_PER_FRAME)
    M = workload.TOKENS_PER_FRAME
    X = spec.x_rows(0, M)
    ref = oracle.w4a4_linear(X, L["prep"], L["b"], 0)
    Xq8, a_scale = q.rotate_smooth_quantize_c8(L["h"], dev_bf16(X))
    acc = torch.zeros((M, 1024), dtype=torch.int32, device="cuda")
    Y = q.w4a4_linear_c8(L["h"], Xq8, a_scale, acc_debug=acc)
    assert np.array_equal(Xq8.cpu().numpy(), ref["xq"])
    assert np.array_equal(a_scale.cpu().numpy(), ref["a_scale"])
    assert np.array_equal(acc.cpu().numpy(), ref["acc"])
    assert assert_bf16_within_one_ulp(host_bits(Y), ref["y"]) == 0.0


def test_c8_chained_launches_are_deterministic():
    """The quantize kernel and the GEMM chained 60 times on one stream (consecutive kernels overlap through
    programmatic dependent launch: each one's blocks may become resident while its predecessor drains): every
    repetition must reproduce the oracle-checked first result bit for bit."""
    spec = workload.LinearSpec("d", 1024, 1024, workload.DIST_NORMAL, 13, 1)
    L = make_layer(spec)
    M = 4 * workload.TOKENS_PER_FRAME
    X = spec.x_rows(0, M)
    rows = np.arange(0, M, 97)
    Xd = dev_bf16(X)
    Xq8, a_scale = q.rotate_smooth_quantize_c8(L["h"], Xd)
    Y0 = q.w4a4_linear_c8(L["h"], Xq8, a_scale).clone()
    codes, scales = oracle.rotate_smooth_quantize(np.ascontiguousarray(X[rows]), L["prep"]["amul"], 0)
    want = oracle.epilogue(oracle.gemm_i32(codes, L["prep"]["wq"]), scales, L["prep"]["w_scale"], L["b"])
    assert assert_bf16_within_one_ulp(host_bits(Y0[torch.from_numpy(rows).cuda()]), want) == 0.0
    q0, a0 = Xq8.clone(), a_scale.clone()
    Y = torch.empty_like(Y0)
    for i in range(60):
        q.rotate_smooth_quantize_c8(L["h"], Xd, Xq8, a_scale)
        q.w4a4_linear_c8(L["h"], Xq8, a_scale, Y)
        if i % 6 == 5:
            assert torch.equal(Y.view(torch.int16), Y0.view(torch.int16)) and torch.equal(Xq8, q0) and torch.equal(a_scale, a0), i
    assert L["h"].device_status() == 0


def test_c8_entry_points_validate_their_arguments():
    """Bad arguments are refused on the host with the documented status, before anything is launched."""
    import ctypes
    from paper_2509_21302_b200 import binding as B
    L = B.lib()
    K, N, M = 1024, 128, 16
    h = q.prepare_weights(dev_bf16(workload.normal_bf16(1, 1, N, K, 0.02)), None, torch.ones(K, device="cuda"), None, c8=True)
    X = torch.zeros((M, K), dtype=torch.bfloat16, device="cuda")
    Xq8 = torch.zeros((M, K + 16), dtype=torch.int8, device="cuda")
    a = torch.zeros(M, dtype=torch.float32, device="cuda")
    Y = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    g = torch.ones(K + 4, dtype=torch.float32, device="cuda")
    st = torch.cuda.current_stream().cuda_stream
    hp, xp, qp, ap, yp, gp = h.handle, X.data_ptr(), Xq8.data_ptr(), a.data_ptr(), Y.data_ptr(), g.data_ptr()
    NULL, SHAPE, ALIGN, UNSUP = -1, -2, -3, -4
    assert L.qvggt_rotate_smooth_quantize_c8(None, xp, K, M, qp, ap, st) == NULL
    assert L.qvggt_rotate_smooth_quantize_c8(hp, xp, K, -1, qp, ap, st) == SHAPE
    assert L.qvggt_rotate_smooth_quantize_c8(hp, xp, K - 8, M, qp, ap, st) == SHAPE          # row stride below K
    assert L.qvggt_rotate_smooth_quantize_c8(hp, xp, K + 4, M, qp, ap, st) == ALIGN          # row stride not a multiple of 8
    assert L.qvggt_rotate_smooth_quantize_c8(hp, xp, K, M, qp + 4, ap, st) == ALIGN
    assert L.qvggt_rotate_smooth_quantize_c8(hp, xp, K, M, None, ap, st) == NULL
    assert L.qvggt_rotate_smooth_quantize_c8(hp, xp, K, 0, None, None, st) == 0              # M = 0 is a no-op
    assert L.qvggt_w4a4_linear_c8(hp, qp, ap, M, yp, N - 8, None, st) == SHAPE
    assert L.qvggt_w4a4_linear_c8(hp, qp, ap, M, yp + 2, N, None, st) == ALIGN
    assert L.qvggt_w4a4_linear_c8(hp, None, ap, M, yp, N, None, st) == NULL
    assert L.qvggt_rotate_smooth_quantize_static_c8(hp, xp, K, M, None, qp, ap, st) == NULL  # no step size
    assert L.qvggt_layernorm_rotate_smooth_quantize_c8(hp, xp, K, M, gp, None, 1e-5, qp, ap, st) == NULL
    assert L.qvggt_layernorm_rotate_smooth_quantize_c8(hp, xp, K, M, gp + 4, gp, 1e-5, qp, ap, st) == ALIGN
    assert L.qvggt_layernorm(xp, K, M, 2048, gp, gp, 1e-5, yp, st) == SHAPE                   # K must be 1024 or 4096
    out = ctypes.c_void_p()
    assert L.qvggt_prepare_weights(xp, None, gp, None, N, K, 16, st, ctypes.byref(out)) == UNSUP  # unknown flag
    assert out.value is None
    # the pair that folds the weight expansion into the quantize launch
    scratch = torch.zeros(N * K + 32, dtype=torch.int8, device="cuda")
    sp = scratch.data_ptr()
    assert L.qvggt_rotate_smooth_quantize_c8_expand(None, xp, K, M, qp, ap, sp, st) == NULL
    assert L.qvggt_rotate_smooth_quantize_c8_expand(hp, xp, K, M, qp, ap, None, st) == NULL      # no scratch
    assert L.qvggt_rotate_smooth_quantize_c8_expand(hp, xp, K, M, qp, ap, sp + 8, st) == ALIGN
    assert L.qvggt_rotate_smooth_quantize_c8_expand(hp, xp, K - 8, M, qp, ap, sp, st) == SHAPE
    assert L.qvggt_rotate_smooth_quantize_c8_expand(hp, None, K, M, qp, ap, sp, st) == NULL
    assert L.qvggt_rotate_smooth_quantize_c8_expand(hp, xp, K, -1, qp, ap, sp, st) == SHAPE
    assert L.qvggt_w4a4_linear_c8_expanded(hp, qp, ap, M, yp, N, None, None, st) == NULL         # no scratch
    assert L.qvggt_w4a4_linear_c8_expanded(hp, qp, ap, M, yp, N, sp + 8, None, st) == ALIGN
    assert L.qvggt_w4a4_linear_c8_expanded(hp, qp, ap, M, yp, N - 8, sp, None, st) == SHAPE
    assert L.qvggt_w4a4_linear_c8_expanded(hp, qp, ap, 0, None, N, None, None, st) == 0          # M = 0 is a no-op
    h8 = q.prepare_weights(dev_bf16(workload.normal_bf16(1, 1, N, K, 0.02)), None, torch.ones(K, device="cuda"), None, bits=8)
    assert L.qvggt_rotate_smooth_quantize_c8_expand(h8.handle, xp, K, M, qp, ap, sp, st) == UNSUP    # 8-bit handles hold no packed codes
    assert L.qvggt_w4a4_linear_c8_expanded(h8.handle, qp, ap, M, yp, N, sp, None, st) == UNSUP
    h8.free()
    torch.cuda.synchronize()
    assert h.device_status() == 0


def test_c8_only_handle_keeps_one_byte_per_weight():
    """QVGGT_PREP_C8_ONLY: the handle holds the codes one per byte and no packed copy (1 byte per weight instead of 1.5);
    the one-code-per-byte entry points work as before, the packed ones refuse the handle."""
    K, N, M = 1024, 256, 140
    spec = workload.LinearSpec("only", K, N, workload.DIST_NORMAL, 21, 0)
    W, b, X = spec.weight(), spec.bias(), spec.x_rows(0, M)
    c = oracle.smooth_factors(spec.x_calib(128), W)
    torch.cuda.synchronize()
    used0 = torch.cuda.memory_allocated()
    free0 = torch.cuda.mem_get_info()[0]
    h = q.prepare_weights(dev_bf16(W), dev_bf16(b), torch.from_numpy(c).cuda(), None, c8="only")
    torch.cuda.synchronize()
    v = h.view()
    assert v["wq"] is None and v["w_scale"].shape == (N,)
    ref = oracle.w4a4_linear(X, oracle.prepare_weights(W, c), b, 0)
    assert np.array_equal(h.view_c8().cpu().numpy(), oracle.prepare_weights(W, c)["wq"])
    Xq8, a_scale = q.rotate_smooth_quantize_c8(h, dev_bf16(X))
    Y = q.w4a4_linear_c8(h, Xq8, a_scale)
    assert np.array_equal(Xq8.cpu().numpy(), ref["xq"]) and np.array_equal(host_bits(Y), ref["y"])
    Xq = torch.zeros((M, K // 2), dtype=torch.uint8, device="cuda")
    st = q.lib().qvggt_w4a4_linear(h.handle, Xq.data_ptr(), a_scale.data_ptr(), M, 0, Y.data_ptr(), N, None,
                                   torch.cuda.current_stream().cuda_stream)
    assert st == -4                                               # QVGGT_ERR_UNSUPPORTED: no packed weights in this handle
    assert h.device_status() == 0
    h.free()


@pytest.mark.parametrize("K,N,M", [(1024, 384, 700), (4096, 128, 300), (1024, 1024, 1374)])
def test_packed_weights_handle_on_the_one_code_per_byte_gemm(K, N, M):
    """A handle prepared without flags keeps only the packed weight codes (0.5 bytes per weight); the one-code-per-byte GEMM
    takes it through a caller-supplied scratch that holds the unpacked codes of one layer.  Same sums, same outputs."""
    spec = workload.LinearSpec("pw", K, N, workload.DIST_NORMAL, 23, 0)
    W, b, X = spec.weight(), spec.bias(), spec.x_rows(0, M)
    c = oracle.smooth_factors(spec.x_calib(128), W)
    ref = oracle.w4a4_linear(X, oracle.prepare_weights(W, c), b, 0)
    torch.cuda.synchronize()
    free0 = torch.cuda.mem_get_info()[0]
    h = q.prepare_weights(dev_bf16(W), dev_bf16(b), torch.from_numpy(c).cuda(), None)          # flags = 0
    torch.cuda.synchronize()
    taken = free0 - torch.cuda.mem_get_info()[0]
    assert taken <= N * K // 2 + (4 << 20), "the handle should hold about half a byte per weight (plus allocation granules)"
    assert h.view_c8() is None and h.view()["wq"].shape == (N, K // 2)
    scratch = torch.full((N * K + 64,), 0x55, dtype=torch.int8, device="cuda")
    Xq8, a = q.rotate_smooth_quantize_c8(h, dev_bf16(X))
    assert np.array_equal(Xq8.cpu().numpy(), ref["xq"])
    acc = torch.zeros((M, N), dtype=torch.int32, device="cuda")
    Y = q.w4a4_linear_c8_packed_weights(h, Xq8, a, scratch, acc_debug=acc)
    assert np.array_equal(scratch[:N * K].view(N, K).cpu().numpy(), ref_wq := oracle.prepare_weights(W, c)["wq"])   # the unpacked codes
    assert np.array_equal(acc.cpu().numpy(), ref["acc"])
    assert np.array_equal(host_bits(Y), ref["y"])
    Y2 = q.w4a4_linear_c8_packed_weights(h, Xq8, a, scratch)                                      # production instantiation, scratch reused
    assert torch.equal(Y2.view(torch.int16), Y.view(torch.int16))
    assert torch.all(scratch[N * K:] == 0x55)
    assert h.device_status() == 0
    h.free()
    only = q.prepare_weights(dev_bf16(W), None, torch.from_numpy(c).cuda(), None, c8="only")
    st = q.lib().qvggt_w4a4_linear_c8_packed_weights(only.handle, Xq8.data_ptr(), a.data_ptr(), M, Y.data_ptr(), N, scratch.data_ptr(), None,
                                                     torch.cuda.current_stream().cuda_stream)
    assert st == -4
    only.free()


@pytest.mark.parametrize("K,N,M", [(1024, 128, 1), (1024, 384, 700), (4096, 128, 300), (1024, 4096, 10992), (4096, 1024, 5000), (1024, 1024, 0),
                                   (1024, 4096, 3), (4096, 3072, 1), (4096, 1024, 43968)])
def test_weight_expansion_folded_into_the_quantize_launch(K, N, M):
    """The quantize launch that also expands the handle's packed weight codes: codes and scales as without the expansion
    (the rows are dealt to fewer blocks, the arithmetic per row is the same), the scratch holds the oracle's weight codes
    and nothing beyond them, and the GEMM reading it gives the oracle's sums and outputs."""
    spec = workload.LinearSpec("ex", K, N, workload.DIST_NORMAL, 31, 0)
    W, b = spec.weight(), spec.bias()
    c = oracle.smooth_factors(spec.x_calib(128), W)
    prep = oracle.prepare_weights(W, c)
    h = q.prepare_weights(dev_bf16(W), dev_bf16(b), torch.from_numpy(c).cuda(), None)          # packed codes only
    scratch = torch.full((N * K + 64,), 0x55, dtype=torch.int8, device="cuda")
    X = spec.x_rows(0, M) if M else np.zeros((0, K), dtype=np.uint16)
    Xd = dev_bf16(X) if M else torch.empty((0, K), dtype=torch.bfloat16, device="cuda")
    Xq8, a = q.rotate_smooth_quantize_c8_expand(h, Xd, scratch)
    assert np.array_equal(scratch[:N * K].view(N, K).cpu().numpy(), prep["wq"])
    assert torch.all(scratch[N * K:] == 0x55)
    if M:
        rows = np.arange(M) if M <= 1500 else np.unique(np.concatenate([np.arange(0, M, 97), np.arange(M - 300, M), np.arange(300)]))
        codes, scales = oracle.rotate_smooth_quantize(np.ascontiguousarray(X[rows]), prep["amul"], 0)
        ridx = torch.from_numpy(rows).cuda()
        assert np.array_equal(Xq8[ridx].cpu().numpy(), codes) and np.array_equal(a[ridx].cpu().numpy(), scales)
        Xq_plain, a_plain = q.rotate_smooth_quantize_c8(h, Xd)                                  # every row against the plain launch
        assert torch.equal(Xq8, Xq_plain) and torch.equal(a, a_plain)
        acc = torch.zeros((M, N), dtype=torch.int32, device="cuda")
        Y = q.w4a4_linear_c8_expanded(h, Xq8, a, scratch, acc_debug=acc)
        acc_ref = oracle.gemm_i32(codes, prep["wq"], 0)
        assert np.array_equal(acc[ridx].cpu().numpy(), acc_ref)
        assert np.array_equal(host_bits(Y[ridx]), oracle.epilogue(acc_ref, scales, prep["w_scale"], b))
        Y2 = q.w4a4_linear_c8_expanded(h, Xq8, a, scratch)
        assert torch.equal(Y2.view(torch.int16), Y.view(torch.int16))
    else:
        assert q.w4a4_linear_c8_expanded(h, Xq8, a, scratch).shape == (0, N)
    assert h.device_status() == 0
    h.free()
    only = q.prepare_weights(dev_bf16(W), None, torch.from_numpy(c).cuda(), None, c8="only")
    st = q.lib().qvggt_rotate_smooth_quantize_c8_expand(only.handle, Xd.data_ptr(), K, M, Xq8.data_ptr(), a.data_ptr(), scratch.data_ptr(),
                                                        torch.cuda.current_stream().cuda_stream)
    assert st == -4                                               # QVGGT_ERR_UNSUPPORTED: no packed codes to expand
    only.free()


@pytest.mark.parametrize("K,N,M", [(1024, 128, 1), (1024, 384, 257), (4096, 256, 300), (4096, 128, 1374)])
def test_c8_grouped_matches_the_oracle_and_the_packed_grouped_path(K, N, M):
    """Group-128 activation scales on codes held one per byte: codes, scales, per-group integer sums bit-exact against the
    oracle, outputs bit-equal, and identical to the packed group-wise entry points."""
    spec = workload.LinearSpec("g8", K, N, workload.DIST_NORMAL, 29, 0)
    W, b, X = spec.weight(), spec.bias(), spec.x_rows(0, M)
    c = oracle.smooth_factors(spec.x_calib(128), W)
    prep = oracle.prepare_weights(W, c)
    ref = oracle.w4a4_linear(X, prep, b, 128)
    h = q.prepare_weights(dev_bf16(W), dev_bf16(b), torch.from_numpy(c).cuda(), None, c8=True)
    Xq8, a = q.rotate_smooth_quantize_c8_grouped(h, dev_bf16(X))
    assert np.array_equal(Xq8.cpu().numpy(), ref["xq"]) and np.array_equal(a.cpu().numpy(), ref["a_scale"])
    acc = torch.full((K // 128, M, N), -7, dtype=torch.int32, device="cuda")
    Y = q.w4a4_linear_c8_grouped(h, Xq8, a, acc_debug=acc)
    assert np.array_equal(acc.cpu().numpy(), ref["acc"])
    assert np.array_equal(host_bits(Y), ref["y"])
    Y2 = q.w4a4_linear_c8_grouped(h, Xq8, a)
    assert torch.equal(Y2.view(torch.int16), Y.view(torch.int16))
    Xq, a4 = q.rotate_smooth_quantize(h, dev_bf16(X), 128)
    assert torch.equal(a4, a) and torch.equal(q.w4a4_linear(h, Xq, a4, 128).view(torch.int16), Y.view(torch.int16))
    assert h.device_status() == 0
    h.free()
