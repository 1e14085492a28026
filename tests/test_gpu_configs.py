"""GPU parity at the full sizes of the benchmark configurations, on sampled token rows.

Every step of the path is independent per token row, so the oracle can check any subset of rows of
a full-size run exactly: the kernels process all M rows in the launch configuration the benchmark
times, and the oracle recomputes the sampled rows one by one.  Bar as everywhere: int4 codes and
int32 sums bit-exact, scales and bf16 outputs within one bf16 ulp (bit-equal in practice).
"""
import numpy as np
import pytest
import torch

import oracle
import workload
from _util import assert_bf16_within_one_ulp, dev_bf16, host_bits, unpack_codes

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


def sample_rows(M, seed, n_random=40):
    """Special-token rows of the first and last frame, tile edges, the ragged tail, and random rows."""
    fixed = [0, 1, 4, 5, 127, 128, 255, 256, 257, M - F, M - F + 4, M - 130, M - 3, M - 2, M - 1]
    rng = np.random.default_rng(seed)
    rows = set(int(r) for r in fixed if 0 <= r < M) | set(int(r) for r in rng.integers(0, M, n_random))
    return np.array(sorted(rows), dtype=np.int64)


def run_layer_sampled(spec, M, group=0, check_gemm=True, X=None, fmt="packed"):
    """Full-size rotate-smooth-quantize (+ GEMM) on the GPU; oracle on sampled rows. Returns rows checked.
    fmt: "packed" (two codes per byte) or "c8" (one code per byte, per-token scales only)."""
    W, b = spec.weight(), spec.bias()
    c = oracle.smooth_factors(spec.x_calib(256), W)
    prep = oracle.prepare_weights(W, c, None)
    h = q.prepare_weights(dev_bf16(W), dev_bf16(b), torch.from_numpy(c).cuda(), None, c8=(fmt == "c8"))
    if X is None:
        X = spec.x_rows(0, M)
    rows = sample_rows(M, spec.layer + 17 * spec.seed)
    Xd = dev_bf16(X)
    if fmt == "c8":
        assert group == 0
        Xq, a_scale = q.rotate_smooth_quantize_c8(h, Xd)
    else:
        Xq, a_scale = q.rotate_smooth_quantize(h, Xd, group)
    codes, scales = oracle.rotate_smooth_quantize(np.ascontiguousarray(X[rows]), prep["amul"], group)
    ridx = torch.from_numpy(rows).cuda()
    got = Xq[ridx].cpu().numpy()
    assert np.array_equal(got if fmt == "c8" else unpack_codes(got), codes), spec.name
    assert np.array_equal(a_scale[ridx].cpu().numpy(), scales), spec.name
    if check_gemm:
        Y = q.w4a4_linear_c8(h, Xq, a_scale) if fmt == "c8" else q.w4a4_linear(h, Xq, a_scale, group)
        acc = oracle.gemm_i32(codes, prep["wq"], group)
        want = oracle.epilogue(acc, scales, prep["w_scale"], b)
        frac = assert_bf16_within_one_ulp(host_bits(Y[ridx]), want, spec.name)
        assert frac == 0.0, f"{spec.name}: {frac:.3e} of the sampled outputs differ in the last bit"
        assert torch.isfinite(Y.float()).all()
    assert h.device_status() == 0
    del Xd
    return len(rows)


# ------------------------------------------------------------------------------ config 2: one block, 8 frames
@pytest.mark.parametrize("fmt", ["packed", "c8"])
@pytest.mark.parametrize("which", [0, 1, 2, 3])
def test_config2_block_linears_8_frames(which, fmt):
    spec = workload.block_specs(0, 0)[which]
    assert run_layer_sampled(spec, 8 * F, fmt=fmt) > 40


# ------------------------------------------------------------------------------ config 3: quantize kernel sweep
@pytest.mark.parametrize("fmt", ["packed", "c8"])
@pytest.mark.parametrize("K,frames", [(1024, 1), (1024, 100), (4096, 1), (4096, 100)])
def test_config3_quantize_sweep(K, frames, fmt):
    M = frames * F
    X = workload.sweep_activations(3, K, 0, M)            # Student-t(3) entries, 1 % outlier channels x50
    spec = workload.LinearSpec("sweep", K, 128, workload.DIST_NORMAL, 3, 0)
    assert run_layer_sampled(spec, M, check_gemm=False, X=X, fmt=fmt) > 20


# ------------------------------------------------------------------------------ config 4: 48-block stack, 32 frames
@pytest.mark.parametrize("fmt", ["packed", "c8"])
@pytest.mark.parametrize("block", [0, 23, 47])
def test_config4_stack_blocks_32_frames(block, fmt):
    """Three of the 48 blocks (first, middle, last) with their own seeded weights, smoothing factors
    and activations; all four linears at M = 43968."""
    for spec in workload.block_specs(1, block):
        run_layer_sampled(spec, 32 * F, fmt=fmt)


# ------------------------------------------------------------------------------ config 5: 100 frames, fc1 / fc2, both granularities
@pytest.mark.parametrize("which,group,fmt", [(2, 0, "packed"), (3, 0, "packed"), (2, 128, "packed"), (3, 128, "packed"),
                                             (2, 0, "c8"), (3, 0, "c8")])
def test_config5_large_scene(which, group, fmt):
    spec = workload.block_specs(4, 0)[which]
    assert run_layer_sampled(spec, 100 * F, group=group, fmt=fmt) > 40
