"""GPU parity of the upstream fusion (LayerNorm -> rotate -> smooth -> quantize in one pass) against the oracle: the
LayerNorm alone bit-exact in bf16, and the fused kernel's codes and scales equal to the oracle's LayerNorm followed by
its quantizer -- hence to the two GPU kernels run one after the other."""
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


def ln_params(K, seed):
    rng = np.random.default_rng(seed)
    return rng.uniform(0.5, 2.0, K).astype(np.float32), rng.normal(0, 0.3, K).astype(np.float32)


@pytest.mark.parametrize("K", [1024, 4096])
@pytest.mark.parametrize("M", [1, 7, 129, 1374, 10992])
def test_layernorm_alone_bit_exact(K, M):
    spec = workload.LinearSpec("ln", K, 128, workload.DIST_NORMAL, 41, 0)
    X = spec.x_rows(0, M)
    if M > 4:
        X[2] = 0x4049                                   # a constant row: output = bf16(beta)
        X[3] = 0                                        # a zero row
    gamma, beta = ln_params(K, K + M)
    want = oracle.layernorm(X, gamma, beta, 1e-5)
    got = q.layernorm(dev_bf16(X), torch.from_numpy(gamma).cuda(), torch.from_numpy(beta).cuda(), 1e-5)
    assert np.array_equal(host_bits(got), want)


@pytest.mark.parametrize("bits", [4, 8])
@pytest.mark.parametrize("K,M", [(1024, 5), (1024, 1374), (4096, 300)])
def test_fused_layernorm_quantize_parity(K, M, bits):
    N = 256
    spec = workload.LinearSpec("lnq", K, N, workload.DIST_NORMAL, 43, 1)
    W, b = spec.weight(), spec.bias()
    c = oracle.smooth_factors(spec.x_calib(256), W)
    v = workload.signs_i8(43, 9, K)
    prep = oracle.prepare_weights(W, c, v, bits=bits)
    h = q.prepare_weights(dev_bf16(W), dev_bf16(b), torch.from_numpy(c).cuda(), torch.from_numpy(v).cuda(), c8=True, bits=bits)
    X = spec.x_rows(0, M)
    gamma, beta = ln_params(K, 5 * K + M)
    g_d, b_d = torch.from_numpy(gamma).cuda(), torch.from_numpy(beta).cuda()
    ln = oracle.layernorm(X, gamma, beta, 1e-5)
    codes, scales = oracle.rotate_smooth_quantize(ln, prep["amul"], 0, bits)
    Xq8, a_scale = q.layernorm_rotate_smooth_quantize_c8(h, dev_bf16(X), g_d, b_d, 1e-5)
    assert np.array_equal(Xq8.cpu().numpy(), codes)
    assert np.array_equal(a_scale.cpu().numpy(), scales)
    # the two kernels one after the other give the same
    Xq8b, a_b = q.rotate_smooth_quantize_c8(h, q.layernorm(dev_bf16(X), g_d, b_d, 1e-5))
    assert torch.equal(Xq8b, Xq8) and torch.equal(a_b, a_scale)
    # and the GEMM that follows
    Y = q.w4a4_linear_c8(h, Xq8, a_scale)
    want = oracle.epilogue(oracle.gemm_i32(codes, prep["wq"]), scales, prep["w_scale"], b)
    assert assert_bf16_within_one_ulp(host_bits(Y), want) == 0.0
    assert h.device_status() == 0


@pytest.mark.parametrize("which", [0, 3])
def test_fused_layernorm_full_size_every_row(which):
    """qkv input (K = 1024) and an fc2-shaped input (K = 4096) at 8 frames (M = 10992), strided input rows: every row of
    codes and scales against the oracle's LayerNorm followed by its quantizer."""
    spec = workload.block_specs(0, 0)[which]
    M, K = 8 * workload.TOKENS_PER_FRAME, spec.K
    W = spec.weight()
    c = oracle.smooth_factors(spec.x_calib(256), W)
    prep = oracle.prepare_weights(W, c, None)
    h = q.prepare_weights(dev_bf16(W), None, torch.from_numpy(c).cuda(), None, c8=True)
    X = spec.x_rows(0, M)
    gamma, beta = ln_params(K, 99)
    wide = torch.zeros((M, K + 64), dtype=torch.bfloat16, device="cuda")
    wide[:, :K] = dev_bf16(X)
    Xq8, a_scale = q.layernorm_rotate_smooth_quantize_c8(h, wide[:, :K], torch.from_numpy(gamma).cuda(), torch.from_numpy(beta).cuda())
    codes, scales = oracle.rotate_smooth_quantize(oracle.layernorm(X, gamma, beta, 1e-5), prep["amul"], 0)
    assert np.array_equal(Xq8.cpu().numpy(), codes)
    assert np.array_equal(a_scale.cpu().numpy(), scales)
    assert h.device_status() == 0
    h.free()
