"""The tensor-core Hadamard mode of the activation path against its tolerance contract.

This mode transforms 7 of the index bits as a product with H_128 on the tensor core, so its fp32 additions do not
follow the oracle's butterfly order and it cannot be bit-exact against oracle.rotate_smooth_quantize.  It is held,
element by element, to the contract stated in include/qvggt.h against the rotation WITHOUT intermediate rounding
(oracle.rotate_f64 / oracle.rotate_smooth_quantize_wide):
  rotated values within (tau S + 2^-24 |u*|) |mul| of the exact ones, tau = 2 log2(K) 2^-24, S = sum |x| of the row;
  scales within the largest such bound of the row (in scale units);
  codes = the nearest integer to the exact position on the code axis, except next to a half-integer boundary (within
  the bound, in code units), where the other neighbour is allowed -- off by one, never more.
The integer GEMM that follows is unchanged, so given these codes it must reproduce the oracle's sums bit for bit.
"""
import numpy as np
import pytest
import torch

import oracle
import workload
from _util import dev_bf16, host_bits, unpack_codes

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


def check_contract(X, mul, codes, scales, y, qmax=7):
    """X bf16 bits [m, K]; codes int8 [m, K], scales fp32 [m], y fp32 [m, K] from the GPU.  Returns statistics."""
    K = X.shape[1]
    bits = 4 if qmax == 7 else 8
    mul64 = mul.astype(np.float64)
    ystar = oracle.rotate_f64(X, mul64)                                       # (x H_K) mul, fp64
    ref = oracle.rotate_smooth_quantize_wide(X, mul, bits)
    S = ref["abs_sum"]
    tau = 2.0 * np.log2(K) * 2.0 ** -24
    bound = tau * S[:, None] * np.abs(mul64)[None, :] + 2.0 ** -24 * np.abs(ystar)
    err = np.abs(y.astype(np.float64) - ystar)
    assert np.all(err <= bound * (1 + 1e-9) + 1e-300), f"rotated values beyond the bound: worst ratio {np.max(err / np.maximum(bound, 1e-300)):.3f}"
    amax = np.maximum(np.abs(ystar).max(axis=1), 1e-8)
    bmax = bound.max(axis=1)
    assert np.all(np.abs(scales.astype(np.float64) - amax / qmax) <= bmax / qmax + 2.0 ** -22 * amax / qmax), "scales beyond the bound"
    pos = ystar * (qmax / amax)[:, None]
    want = np.rint(pos)
    diff = codes.astype(np.int32) - want.astype(np.int32)
    assert np.abs(diff).max() <= 1, "a code is off by more than one"
    off = diff != 0
    eps = qmax * (bound + bmax[:, None]) / amax[:, None] + 2.0 ** -20
    to_boundary = np.abs(pos - (np.floor(pos) + 0.5))
    assert np.all(to_boundary[off] <= eps[off]), "a code differs away from a rounding boundary"
    return dict(ratio=float(np.max(err / np.maximum(bound, 1e-300))), off=int(off.sum()), n=int(off.size),
                vs_wide=int((codes != ref["codes"]).sum()))


def make_handle(K, seed, bits=4):
    spec = workload.LinearSpec("tc", K, 128, workload.DIST_NORMAL, seed, 0)
    W = spec.weight()
    c = workload.loguniform_f32(seed, 5, K, 0.1, 10.0)
    v = workload.signs_i8(seed, 6, K)
    prep = oracle.prepare_weights(W, c, v, bits)
    h = q.prepare_weights(dev_bf16(W), None, torch.from_numpy(c).cuda(), torch.from_numpy(v).cuda(), c8=True, bits=bits)
    return spec, prep, h


@pytest.mark.parametrize("K", [1024, 4096])
@pytest.mark.parametrize("M", [1, 5, 31, 32, 33, 257, 1374])
def test_tc_mode_meets_its_contract_small(K, M):
    spec, prep, h = make_handle(K, 11)
    X = spec.x_rows(0, M)
    if M >= 5:
        X[3] = 0                                                   # a zero token: codes 0, floor scale
    Xd = dev_bf16(X)
    for c8 in (False, True):
        ydbg = torch.full((M, K), float("nan"), device="cuda")
        Xq, a = q.rotate_smooth_quantize_tc(h, Xd, c8=c8, y_debug=ydbg)
        codes = Xq.cpu().numpy() if c8 else unpack_codes(Xq.cpu().numpy())
        st = check_contract(X, prep["amul"], codes, a.cpu().numpy(), ydbg.cpu().numpy())
        assert st["ratio"] < 1.0
        # the production instantiation (no dump) returns the same codes and scales
        Xq2, a2 = q.rotate_smooth_quantize_tc(h, Xd, c8=c8)
        assert torch.equal(Xq2, Xq) and torch.equal(a2, a)
    if M >= 5:
        assert not codes[3].any() and a.cpu().numpy()[3] == np.float32(1e-8) / np.float32(7)
    assert h.device_status() == 0
    h.free()


@pytest.mark.parametrize("K", [1024, 4096])
def test_tc_mode_8bit_codes_and_strided_rows(K):
    spec, prep, h = make_handle(K, 12, bits=8)
    M = 300
    X = spec.x_rows(0, M)
    wide = torch.zeros((M, K + 64), dtype=torch.bfloat16, device="cuda")
    wide[:, :K] = dev_bf16(X)
    ydbg = torch.zeros((M, K), device="cuda")
    Xq8, a = q.rotate_smooth_quantize_tc(h, wide[:, :K], c8=True, y_debug=ydbg)
    st = check_contract(X, prep["amul"], Xq8.cpu().numpy(), a.cpu().numpy(), ydbg.cpu().numpy(), qmax=127)
    assert st["ratio"] < 1.0 and np.abs(Xq8.cpu().numpy()).max() == 127
    assert h.device_status() == 0
    h.free()


@pytest.mark.parametrize("K,frames", [(1024, 8), (4096, 8), (1024, 100), (4096, 100)])
def test_tc_mode_meets_its_contract_at_full_size_every_row(K, frames):
    """Config 3's inputs (Student-t entries, outlier channels) at the benchmark's sizes, every row, in chunks."""
    M = frames * F
    spec, prep, h = make_handle(K, 13)
    X = workload.sweep_activations(3, K, 0, M)
    ydbg = torch.empty((M, K), device="cuda")
    Xq8, a = q.rotate_smooth_quantize_tc(h, dev_bf16(X), c8=True, y_debug=ydbg)
    Xq, a_p = q.rotate_smooth_quantize_tc(h, dev_bf16(X), c8=False)
    assert torch.equal(a_p, a)
    codes_p = Xq.cpu().numpy()
    codes, scales = Xq8.cpu().numpy(), a.cpu().numpy()
    assert np.array_equal(codes_p, oracle.pack_int4(codes)), "the two storage formats of the mode disagree"
    chunk = 16384 * 1024 // K
    worst, off, vs_wide = 0.0, 0, 0
    for r0 in range(0, M, chunk):
        r1 = min(M, r0 + chunk)
        st = check_contract(X[r0:r1], prep["amul"], codes[r0:r1], scales[r0:r1], ydbg[r0:r1].cpu().numpy())
        worst, off, vs_wide = max(worst, st["ratio"]), off + st["off"], vs_wide + st["vs_wide"]
    print(f"\\ntensor-core Hadamard K={K} M={M}: worst |error| / bound = {worst:.4f}; codes not at the nearest integer of the exact "
          f"position: {off} of {M * K} ({off / (M * K):.2e}); codes differing from the fp64-rotation quantizer: {vs_wide}")
    assert worst < 1.0
    assert h.device_status() == 0
    h.free()


def test_tc_codes_through_the_gemm_are_exact():
    """The GEMM is unchanged: on the codes and scales this mode produced it reproduces the oracle's sums and outputs."""
    K, N, M = 1024, 256, 700
    spec = workload.LinearSpec("tcg", K, N, workload.DIST_NORMAL, 14, 0)
    W, b, X = spec.weight(), spec.bias(), spec.x_rows(0, M)
    c = oracle.smooth_factors(spec.x_calib(128), W)
    prep = oracle.prepare_weights(W, c)
    h = q.prepare_weights(dev_bf16(W), dev_bf16(b), torch.from_numpy(c).cuda(), None, c8=True)
    Xq8, a = q.rotate_smooth_quantize_tc(h, dev_bf16(X), c8=True)
    acc = torch.zeros((M, N), dtype=torch.int32, device="cuda")
    Y = q.w4a4_linear_c8(h, Xq8, a, acc_debug=acc)
    want_acc = oracle.gemm_i32(Xq8.cpu().numpy(), prep["wq"])
    assert np.array_equal(acc.cpu().numpy(), want_acc)
    assert np.array_equal(host_bits(Y), oracle.epilogue(want_acc, a.cpu().numpy(), prep["w_scale"], b))
    Xq, a2 = q.rotate_smooth_quantize_tc(h, dev_bf16(X), c8=False)
    Y2 = q.w4a4_linear(h, Xq, a2)
    assert torch.equal(Y2.view(torch.int16), Y.view(torch.int16))
    assert h.device_status() == 0
    h.free()


def test_tc_entry_points_validate_their_arguments():
    spec, prep, h = make_handle(1024, 15)
    L = q.lib()
    X = torch.zeros((8, 1024), dtype=torch.bfloat16, device="cuda")
    Xq = torch.zeros((8, 1024), dtype=torch.int8, device="cuda")
    a = torch.zeros(8, device="cuda")
    st = torch.cuda.current_stream().cuda_stream
    for fn in (L.qvggt_rotate_smooth_quantize_tc, L.qvggt_rotate_smooth_quantize_tc_c8):
        assert fn(None, X.data_ptr(), 1024, 8, Xq.data_ptr(), a.data_ptr(), None, st) == -1
        assert fn(h.handle, X.data_ptr(), 1000, 8, Xq.data_ptr(), a.data_ptr(), None, st) == -2
        assert fn(h.handle, X.data_ptr(), 1028, 8, Xq.data_ptr(), a.data_ptr(), None, st) == -3
        assert fn(h.handle, X.data_ptr(), 1024, 8, Xq.data_ptr(), a.data_ptr(), a.data_ptr() + 4, st) == -3
        assert fn(h.handle, X.data_ptr(), 1024, 0, None, None, None, st) == 0
    h.free()
    h8 = make_handle(1024, 15, bits=8)[2]
    assert L.qvggt_rotate_smooth_quantize_tc(h8.handle, X.data_ptr(), 1024, 8, Xq.data_ptr(), a.data_ptr(), None, st) == -4
    h8.free()
