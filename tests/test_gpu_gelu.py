"""GELU in front of the activation path (the fc2 half of the upstream fusion).

Contract (the GPU's GELU is an approximation of its own design, so it is not bit-exact against the fp64 oracle):
  qvggt_gelu alone: every output equals the oracle's bf16 value (fp64 x Phi(x), rounded once) or one of its two bf16
  neighbours; results whose exact magnitude is below 2^-120 may be flushed to zero;
  qvggt_gelu_rotate_smooth_quantize_c8: bit for bit the result of qvggt_gelu followed by
  qvggt_rotate_smooth_quantize_c8, and therefore the oracle's quantizer applied to the GPU's own bf16 GELU output.
"""
import numpy as np
import pytest
import torch

import oracle
import workload
from _util import bf16_value, dev_bf16, host_bits

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


def ordered(bits):
    b = bits.astype(np.int32)
    return np.where(b & 0x8000, -(b & 0x7FFF), b & 0x7FFF)


def assert_gelu_within_one_ulp(got, want):
    w = bf16_value(want).astype(np.float64)
    tiny = np.abs(w) < 2.0 ** -120
    d = np.abs(ordered(got) - ordered(want))
    assert d[~tiny].max(initial=0) <= 1, f"{(d[~tiny] > 1).sum()} outputs beyond one bf16 ulp"
    assert np.all(np.abs(bf16_value(got[tiny]).astype(np.float64)) <= 2.0 ** -119), "a result in the flush zone is not tiny"
    return float((d[~tiny] == 0).mean())


@pytest.mark.parametrize("K", [1024, 4096])
def test_gelu_every_finite_bf16_input(K):
    """All 65280 finite bf16 values (both signs, subnormals, the far tails), laid out as rows of K."""
    bits = np.arange(65536, dtype=np.uint32)
    bits = bits[((bits >> 7) & 0xFF) != 0xFF].astype(np.uint16)
    n = (len(bits) + K - 1) // K * K
    X = np.zeros(n, np.uint16)
    X[:len(bits)] = bits
    X = X.reshape(-1, K)
    got = host_bits(q.gelu(dev_bf16(X)))
    exact = assert_gelu_within_one_ulp(got, oracle.gelu(X))
    assert exact > 0.99                                        # almost everywhere it IS the correctly rounded value


@pytest.mark.parametrize("K,M", [(4096, 1374), (1024, 257), (4096, 5), (1024, 1)])
def test_gelu_on_mlp_shaped_activations_and_strided_rows(K, M):
    spec = workload.LinearSpec("g", K, 128, workload.DIST_NORMAL, 41, 0)
    X = spec.x_rows(0, M)                                      # pre-activations: N(0,1) with outlier channels and special rows
    wide = torch.zeros((M, K + 32), dtype=torch.bfloat16, device="cuda")
    wide[:, :K] = dev_bf16(X)
    got = host_bits(q.gelu(wide[:, :K]))
    assert_gelu_within_one_ulp(got, oracle.gelu(X))
    assert np.array_equal(got, host_bits(q.gelu(dev_bf16(X))))


@pytest.mark.parametrize("bits", [4, 8])
@pytest.mark.parametrize("K,M", [(4096, 1374), (4096, 129), (1024, 300), (4096, 1)])
def test_fused_gelu_quantize_equals_the_two_kernels_and_the_oracle_on_their_input(K, M, bits):
    spec = workload.LinearSpec("gq", K, 128, workload.DIST_NORMAL, 42, 0)
    W = spec.weight()
    c = workload.loguniform_f32(42, 5, K, 0.1, 10.0)
    v = workload.signs_i8(42, 6, K)
    prep = oracle.prepare_weights(W, c, v, bits)
    h = q.prepare_weights(dev_bf16(W), None, torch.from_numpy(c).cuda(), torch.from_numpy(v).cuda(), c8=True, bits=bits)
    X = spec.x_rows(0, M)
    Xd = dev_bf16(X)
    act = q.gelu(Xd)                                            # the unfused arm: the activated tensor goes through memory
    Xq_two, a_two = q.rotate_smooth_quantize_c8(h, act)
    Xq, a = q.gelu_rotate_smooth_quantize_c8(h, Xd)
    assert torch.equal(Xq, Xq_two) and torch.equal(a, a_two), "fused and unfused results differ"
    # the quantizer itself stays bit-exact: the oracle on the GPU's own bf16 activations
    codes, scales = oracle.rotate_smooth_quantize(host_bits(act), prep["amul"], 0, bits)
    assert np.array_equal(Xq.cpu().numpy(), codes) and np.array_equal(a.cpu().numpy(), scales)
    assert h.device_status() == 0
    h.free()


def test_fused_gelu_through_fc2_matches_the_oracle_layer_on_the_activated_input():
    """fc1 output -> GELU -> fc2 (K = 4096) with the fused kernel; the oracle runs the whole fc2 layer on the GPU's bf16
    activations: integer sums bit-exact, outputs bit-equal."""
    M = 700
    spec = workload.block_specs(7, 0)[3]
    W, b = spec.weight(), spec.bias()
    pre = workload.LinearSpec("pre", spec.K, 128, workload.DIST_NORMAL, 43, 0).x_rows(0, M)
    c = oracle.smooth_factors(oracle.gelu(pre[:256]), W)
    prep = oracle.prepare_weights(W, c)
    h = q.prepare_weights(dev_bf16(W), dev_bf16(b), torch.from_numpy(c).cuda(), None, c8="only")
    Xd = dev_bf16(pre)
    Xq, a = q.gelu_rotate_smooth_quantize_c8(h, Xd)
    acc = torch.zeros((M, spec.N), dtype=torch.int32, device="cuda")
    Y = q.w4a4_linear_c8(h, Xq, a, acc_debug=acc)
    ref = oracle.w4a4_linear(host_bits(q.gelu(Xd)), prep, b, 0)
    assert np.array_equal(Xq.cpu().numpy(), ref["xq"]) and np.array_equal(acc.cpu().numpy(), ref["acc"])
    assert np.array_equal(host_bits(Y), ref["y"])
    assert h.device_status() == 0
    h.free()


@pytest.mark.parametrize("which,frames", [(3, 8), (1, 8), (3, 32)])
def test_fused_gelu_full_size_every_row(which, frames):
    """The fc2 input of the block (K = 4096; K = 1024 as well) at 8 and 32 frames through the GELU kernel and the fused
    GELU -> rotate -> smooth -> quantize kernel: every row of the activation within one bf16 ulp of the oracle's GELU,
    and every row of codes and scales equal to the oracle's quantizer on the GPU's own bf16 GELU output.  (Many rows per
    thread block: the blocks walk through their rows with a two-deep staging ring.)"""
    spec = workload.block_specs(0, 0)[which]
    M = frames * workload.TOKENS_PER_FRAME
    W = spec.weight()
    pre = workload.LinearSpec("pre", spec.K, 128, workload.DIST_NORMAL, 47, 0).x_rows(0, M)
    c = oracle.smooth_factors(oracle.gelu(pre[:256]), W)
    prep = oracle.prepare_weights(W, c)
    h = q.prepare_weights(dev_bf16(W), None, torch.from_numpy(c).cuda(), None, c8="only")
    Xd = dev_bf16(pre)
    act = host_bits(q.gelu(Xd))
    assert_gelu_within_one_ulp(act, oracle.gelu(pre))
    Xq, a = q.gelu_rotate_smooth_quantize_c8(h, Xd)
    codes, scales = oracle.rotate_smooth_quantize(act, prep["amul"], 0)
    assert np.array_equal(Xq.cpu().numpy(), codes) and np.array_equal(a.cpu().numpy(), scales)
    assert h.device_status() == 0
    h.free()


def test_gelu_entry_points_validate_their_arguments():
    L = q.lib()
    X = torch.zeros((8, 1024), dtype=torch.bfloat16, device="cuda")
    st = torch.cuda.current_stream().cuda_stream
    assert L.qvggt_gelu(X.data_ptr(), 1024, 8, 2048, X.data_ptr(), st) == -2
    assert L.qvggt_gelu(None, 1024, 8, 1024, X.data_ptr(), st) == -1
    assert L.qvggt_gelu(X.data_ptr(), 1020, 8, 1024, X.data_ptr(), st) == -2
    assert L.qvggt_gelu(X.data_ptr() + 2, 1024, 8, 1024, X.data_ptr(), st) == -3
    assert L.qvggt_gelu(X.data_ptr(), 1024, 0, 1024, None, st) == 0
    assert L.qvggt_gelu_rotate_smooth_quantize_c8(None, X.data_ptr(), 1024, 8, X.data_ptr(), X.data_ptr(), st) == -1
