"""Cross-consistency of the activation-side kernels on random sizes, on every row.

Several entry points compute the same codes by different routes (two storage formats, fused or separate prologues, two
scale granularities, the tensor-core mode within its contract).  Comparing them with each other on the GPU covers
every row of sizes the oracle only samples: up to 70 000 rows per case, row counts drawn at random so that the ragged
ends of every kernel's blocking are hit.  The oracle checks a sample of rows of every case.
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


def unpack_gpu(p):
    lo, hi = (p & 0xF).to(torch.int8), (p >> 4).to(torch.int8)
    lo, hi = torch.where(lo >= 8, lo - 16, lo), torch.where(hi >= 8, hi - 16, hi)
    return torch.stack((lo, hi), dim=-1).reshape(p.shape[0], -1)


@pytest.mark.parametrize("seed", [1, 2])
def test_routes_to_the_same_codes_agree_on_every_row(q, seed):
    rng = np.random.default_rng(seed)
    for it in range(10):
        K = int(rng.choice([1024, 4096]))
        M = int(rng.choice([rng.integers(1, 700), rng.integers(700, 15000), rng.integers(15000, 70000)]))
        dist = workload.DIST_GELU if (K == 4096 and it % 2) else workload.DIST_NORMAL
        spec = workload.LinearSpec("x", K, 128, dist, 1000 + 32 * seed + it, it % 5)
        W, X = spec.weight(), spec.x_rows(0, M)
        c = oracle.smooth_factors(spec.x_calib(64), W)
        prep = oracle.prepare_weights(W, c)
        h = q.prepare_weights(dev_bf16(W), None, torch.from_numpy(c).cuda(), None, c8=True)
        Xd = dev_bf16(X)
        rows = np.unique(np.concatenate([np.arange(min(M, 20)), np.arange(max(0, M - 150), M), rng.integers(0, M, 40)]))
        ridx, Xs = torch.from_numpy(rows).cuda(), np.ascontiguousarray(X[rows])
        what = f"K={K} M={M}"
        # exact kernel: one code per byte against the oracle, two codes per byte against one per byte
        xq8, a8 = q.rotate_smooth_quantize_c8(h, Xd)
        xq4, a4 = q.rotate_smooth_quantize(h, Xd, 0)
        codes, scales = oracle.rotate_smooth_quantize(Xs, prep["amul"], 0)
        assert np.array_equal(xq8[ridx].cpu().numpy(), codes) and np.array_equal(a8[ridx].cpu().numpy(), scales), what
        assert torch.equal(unpack_gpu(xq4), xq8) and torch.equal(a4, a8), what
        # one scale per 128 channels
        g8, ga8 = q.rotate_smooth_quantize_c8_grouped(h, Xd)
        g4, ga4 = q.rotate_smooth_quantize(h, Xd, 128)
        gc, gs = oracle.rotate_smooth_quantize(Xs, prep["amul"], 128)
        assert np.array_equal(g8[ridx].cpu().numpy(), gc) and np.array_equal(ga8[ridx].cpu().numpy(), gs), what
        assert torch.equal(unpack_gpu(g4), g8) and torch.equal(ga4, ga8), what
        del g8, g4
        # tensor-core mode: its two formats agree exactly; against the exact codes off by at most one, rarely
        t8, ta8 = q.rotate_smooth_quantize_tc(h, Xd, True)
        t4, ta4 = q.rotate_smooth_quantize_tc(h, Xd, False)
        d = (t8.to(torch.int16) - xq8.to(torch.int16)).abs()
        assert int(d.max()) <= 1 and float((d != 0).float().mean()) < 1e-3, what
        assert torch.equal(unpack_gpu(t4), t8) and torch.equal(ta4, ta8) and torch.allclose(ta8, a8, rtol=2e-6, atol=0), what
        del t8, t4, d
        # fused prologues against the two kernels they replace
        f8, fa = q.gelu_rotate_smooth_quantize_c8(h, Xd)
        u8, ua = q.rotate_smooth_quantize_c8(h, q.gelu(Xd))
        assert torch.equal(f8, u8) and torch.equal(fa, ua), what
        gamma, beta = rng.uniform(0.5, 2.0, K).astype(np.float32), rng.normal(0, 0.3, K).astype(np.float32)
        gd, bd = torch.from_numpy(gamma).cuda(), torch.from_numpy(beta).cuda()
        ln = q.layernorm(Xd, gd, bd)
        l8, la = q.layernorm_rotate_smooth_quantize_c8(h, Xd, gd, bd)
        v8, va = q.rotate_smooth_quantize_c8(h, ln)
        assert torch.equal(l8, v8) and torch.equal(la, va), what
        assert np.array_equal(host_bits(ln[ridx]), oracle.layernorm(Xs, gamma, beta, 1e-5)), what
        assert h.device_status() == 0
        h.free()
        del Xd, xq8, xq4, f8, u8, l8, v8, ln
        torch.cuda.empty_cache()
