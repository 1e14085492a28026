"""Repeated launches on random shapes: every GEMM kernel must return the same bits every time.

The persistent kernels hand tiles, stages and accumulators between their warps through barriers; a missing
dependency would show as an output that changes from launch to launch (or differs between the kernels, which
compute the same function).  Per shape and scale granularity: the quantize kernels against the oracle on sampled
rows, then twelve GEMM launches back to back (one code per byte, packed weights expanded by the quantize launch,
packed operands) whose outputs must all be bit-equal to the first, and the first equal to the oracle on the
sampled rows.
"""
import numpy as np
import pytest
import torch

import oracle
import workload
from _util import dev_bf16, host_bits

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def q():
    import paper_2509_21302_b200 as pkg
    pkg.build()
    yield pkg
    torch.cuda.synchronize()


@pytest.mark.parametrize("seed", [3, 4])
def test_repeated_launches_agree_bit_for_bit(q, seed):
    rng = np.random.default_rng(seed)
    for it in range(12):
        K = int(rng.choice([1024, 4096]))
        N = 128 * int(rng.integers(1, 33))
        M = int(rng.choice([rng.integers(1, 600), rng.integers(600, 12000), rng.integers(12000, 30000)]))
        spec = workload.LinearSpec("rep", K, N, workload.DIST_NORMAL, 700 + 16 * seed + it, it % 7)
        W, b, X = spec.weight(), spec.bias(), spec.x_rows(0, M)
        c = oracle.smooth_factors(spec.x_calib(64), W)
        prep = oracle.prepare_weights(W, c)
        h = q.prepare_weights(dev_bf16(W), dev_bf16(b), torch.from_numpy(c).cuda(), None, c8=True)
        Xd = dev_bf16(X)
        rows = np.unique(np.concatenate([np.arange(min(M, 40)), np.arange(max(0, M - 300), M), rng.integers(0, M, 60)]))
        ridx = torch.from_numpy(rows).cuda()
        Xs = np.ascontiguousarray(X[rows])
        for group in (0, 128):
            what = f"K={K} N={N} M={M} group={group}"
            codes, scales = oracle.rotate_smooth_quantize(Xs, prep["amul"], group)
            want = oracle.epilogue(oracle.gemm_i32(codes, prep["wq"], group), scales, prep["w_scale"], b)
            scratch = torch.empty(N * K, dtype=torch.int8, device="cuda")
            if group:
                Xq8, a8 = q.rotate_smooth_quantize_c8_grouped(h, Xd)
            else:
                Xq8, a8 = q.rotate_smooth_quantize_c8_expand(h, Xd, scratch)
            Xq4, a4 = q.rotate_smooth_quantize(h, Xd, group)
            assert np.array_equal(Xq8[ridx].cpu().numpy(), codes) and np.array_equal(a8[ridx].cpu().numpy(), scales), what
            assert torch.equal(a8, a4), what
            outs = []
            for rep in range(6):
                if group:
                    outs.append(q.w4a4_linear_c8_grouped(h, Xq8, a8))
                else:
                    outs.append(q.w4a4_linear_c8(h, Xq8, a8) if rep % 2 else q.w4a4_linear_c8_expanded(h, Xq8, a8, scratch))
                outs.append(q.w4a4_linear(h, Xq4, a4, group))
            torch.cuda.synchronize()
            assert np.array_equal(host_bits(outs[0][ridx]), want), what
            for o in outs[1:]:
                assert torch.equal(o.view(torch.int16), outs[0].view(torch.int16)), what
            del outs
        assert h.device_status() == 0
        h.free()
        del Xd
        torch.cuda.empty_cache()


def test_two_streams_share_a_handle(q):
    """The same handle used from two CUDA streams at once (different inputs and outputs, launches interleaved from the
    host): the results are those of the same calls made one after the other.  The handle is read-only during launches
    (its status word apart), tensor maps travel with each launch, and the host-side caches are per device and atomic."""
    spec = workload.block_specs(0, 0)[2]                         # fc1: K = 1024, N = 4096
    W, b = spec.weight(), spec.bias()
    c = oracle.smooth_factors(spec.x_calib(256), W)
    h = q.prepare_weights(dev_bf16(W), dev_bf16(b), torch.from_numpy(c).cuda(), None, c8=True)
    M = [5000, 3 * workload.TOKENS_PER_FRAME]
    X = [dev_bf16(spec.x_rows(0, M[0])), dev_bf16(spec.x_rows(20000, M[1]))]
    want = []
    for x in X:                                                  # one after the other on the current stream
        xq, a = q.rotate_smooth_quantize_c8(h, x)
        xq4, a4 = q.rotate_smooth_quantize(h, x, 0)
        want.append((q.w4a4_linear_c8(h, xq, a), q.w4a4_linear(h, xq4, a4, 0), xq, a))
    torch.cuda.synchronize()
    assert torch.equal(want[0][0].view(torch.int16), want[0][1].view(torch.int16))
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    got = [[], []]
    for rep in range(8):
        for i in (0, 1):
            with torch.cuda.stream(streams[i]):
                xq, a = q.rotate_smooth_quantize_c8(h, X[i])
                y8 = q.w4a4_linear_c8(h, xq, a)
                xq4, a4 = q.rotate_smooth_quantize(h, X[i], 0)
                y4 = q.w4a4_linear(h, xq4, a4, 0)
                got[i].append((y8, y4, xq, a))
    torch.cuda.synchronize()
    for i in (0, 1):
        for y8, y4, xq, a in got[i]:
            assert torch.equal(xq, want[i][2]) and torch.equal(a, want[i][3])
            assert torch.equal(y8.view(torch.int16), want[i][0].view(torch.int16))
            assert torch.equal(y4.view(torch.int16), want[i][0].view(torch.int16))
    assert h.device_status() == 0
    h.free()
