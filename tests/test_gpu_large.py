"""GPU parity where element and byte offsets leave the 32-bit range: one linear with M = 2 200 003 token rows.

With K = N = 1024 the activation matrix holds 2.25e9 elements (4.5 GB of bf16), its codes 2.25 GB one per byte, the
output 4.5 GB: element offsets pass 2^31 and byte offsets 2^32 at row 2 097 152, inside the matrix.  Every step of the
path is independent per token row, so windows of rows are checked against the oracle exactly: the first rows, the
rows on both sides of that boundary, a few windows in between and the ragged tail (M is odd).  A kernel that computed
a row offset in 32 bits would read or write a wrong row there.
"""
import numpy as np
import pytest
import torch

import oracle
import workload
from _util import dev_bf16, host_bits

pytestmark = pytest.mark.gpu

M_LARGE = 2_200_003
K = N = 1024
BOUNDARY = (1 << 31) // K            # first row whose element offset does not fit a signed 32-bit integer


@pytest.fixture(scope="module")
def q():
    import paper_2509_21302_b200 as pkg
    pkg.build()
    yield pkg
    torch.cuda.synchronize()


def windows():
    w = [(0, 64), (BOUNDARY - 96, 192), (BOUNDARY // 2 - 32, 64), (BOUNDARY + 40_000, 64), (M_LARGE - 259, 259)]
    rows = np.concatenate([np.arange(a, a + n) for a, n in w])
    assert rows.max() == M_LARGE - 1 and rows.min() == 0
    return w, rows


def test_row_offsets_beyond_32_bits(q):
    spec = workload.LinearSpec("large", K, N, workload.DIST_NORMAL, 41, 0)
    W, b = spec.weight(), spec.bias()
    c = oracle.smooth_factors(spec.x_calib(128), W)
    prep = oracle.prepare_weights(W, c)
    h = q.prepare_weights(dev_bf16(W), dev_bf16(b), torch.from_numpy(c).cuda(), None, c8=True)
    # the seeded activation rows, generated and uploaded in chunks (the generator addresses any window of rows)
    X = torch.empty((M_LARGE, K), dtype=torch.bfloat16, device="cuda")
    chunk = 1 << 17
    buf = np.empty((chunk, K), dtype=np.uint16)
    for r0 in range(0, M_LARGE, chunk):
        n = min(chunk, M_LARGE - r0)
        spec.x_rows(r0, n, out=buf[:n])
        X[r0:r0 + n].view(torch.int16).copy_(torch.from_numpy(buf[:n].view(np.int16)))
    wins, rows = windows()
    Xs = np.concatenate([spec.x_rows(a, n) for a, n in wins])
    ridx = torch.from_numpy(rows).cuda()
    assert np.array_equal(host_bits(X[ridx]), Xs)                       # the upload itself
    codes, scales = oracle.rotate_smooth_quantize(Xs, prep["amul"], 0)
    acc = oracle.gemm_i32(codes, prep["wq"], 0)
    want_y = oracle.epilogue(acc, scales, prep["w_scale"], b)

    # one code per byte: exact kernel, tensor-core mode (its own contract: checked for agreement off the rounding ties), GEMM
    Xq8, a8 = q.rotate_smooth_quantize_c8(h, X)
    assert np.array_equal(Xq8[ridx].cpu().numpy(), codes) and np.array_equal(a8[ridx].cpu().numpy(), scales)
    Y = q.w4a4_linear_c8(h, Xq8, a8)
    assert np.array_equal(host_bits(Y[ridx]), want_y)
    Xq_tc, a_tc = q.rotate_smooth_quantize_tc(h, X, True)
    got_tc = Xq_tc[ridx].cpu().numpy().astype(np.int32)
    assert np.abs(got_tc - codes).max() <= 1 and (got_tc != codes).mean() < 1e-3
    assert np.allclose(a_tc[ridx].cpu().numpy(), scales, rtol=1e-5, atol=0)
    del Xq_tc, a_tc, Y
    torch.cuda.empty_cache()

    # two codes per byte: quantize kernel and the packed-operand GEMM
    Xq4, a4 = q.rotate_smooth_quantize(h, X, 0)
    assert np.array_equal(Xq4[ridx].cpu().numpy(), oracle.pack_int4(codes)) and np.array_equal(a4[ridx].cpu().numpy(), scales)
    del X
    torch.cuda.empty_cache()
    Y4 = q.w4a4_linear(h, Xq4, a4, 0)
    assert np.array_equal(host_bits(Y4[ridx]), want_y)
    # rows the windows do not cover: the two GEMM kernels agree on every output of the 2.2 M rows
    Y8 = q.w4a4_linear_c8(h, Xq8, a8)
    assert torch.equal(Y8.view(torch.int16), Y4.view(torch.int16))
    assert torch.isfinite(Y8[::4099].float()).all()
    assert h.device_status() == 0
    h.free()
