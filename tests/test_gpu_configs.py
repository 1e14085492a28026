"""GPU parity at the full sizes of the five benchmark configurations, in the launch configuration the benchmark times.

Every step of the path is independent per token row, so the oracle can check any subset of rows of a full-size run
exactly.  Per configuration one layer (at least) is compared on EVERY row -- codes, scales, integer sums where
dumped, outputs -- and the remaining layers on the first and last row of every 256-row tile of the GEMM's token
dimension (every tile of the persistent schedule, hence every turn of its stage and accumulator rings, is looked
at), plus the special-token rows.  Bar as everywhere: int4 codes and int32 sums bit-exact, scales and bf16 outputs
within one bf16 ulp (the tests also demand zero mismatching bits: the kernels use the oracle's operation order).
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


def edge_rows(M, tile=256):
    """First and last row of every `tile`-row tile, the rows next to the middle of a tile (where the two CTAs of a
    pair meet), the special-token rows of the first and last frame, and the ragged tail."""
    starts = np.arange(0, M, tile)
    rows = set(starts.tolist()) | set(np.minimum(starts + tile - 1, M - 1).tolist())
    rows |= set(np.minimum(starts + tile // 2 - 1, M - 1).tolist()) | set(np.minimum(starts + tile // 2, M - 1).tolist())
    rows |= {r for r in (0, 1, 4, 5, M - F, M - F + 4, M - 130, M - 3, M - 2, M - 1) if 0 <= r < M}
    return np.array(sorted(rows), dtype=np.int64)


def run_layer(spec, M, rows="all", group=0, fmt="packed", X=None, check_gemm=True, check_acc=False):
    """Full-size rotate-smooth-quantize (+ GEMM) on the GPU over all M rows; the oracle on `rows` ("all", or
    "edges" = edge_rows).  fmt: "packed" (two codes per byte) or "c8" (one code per byte, per-token scales only).
    check_acc: also dump the integer sums (the kernel's DUMP instantiation), compare them exactly, and demand that
    the production instantiation writes the same outputs bit for bit.  Returns the number of rows compared."""
    W, b = spec.weight(), spec.bias()
    c = oracle.smooth_factors(spec.x_calib(256), W)
    prep = oracle.prepare_weights(W, c, None)
    h = q.prepare_weights(dev_bf16(W), dev_bf16(b), torch.from_numpy(c).cuda(), None, c8=("only" if fmt == "c8" else False))
    if X is None:
        X = spec.x_rows(0, M)
    Xd = dev_bf16(X)
    if fmt == "c8":
        Xq, a_scale = q.rotate_smooth_quantize_c8_grouped(h, Xd) if group else q.rotate_smooth_quantize_c8(h, Xd)
    else:
        Xq, a_scale = q.rotate_smooth_quantize(h, Xd, group)
    del Xd
    if isinstance(rows, str) and rows == "all":
        ridx, Xs = None, X
    else:
        rows = edge_rows(M, 128 if group else 256) if isinstance(rows, str) else rows
        ridx, Xs = torch.from_numpy(rows).cuda(), np.ascontiguousarray(X[rows])

    def pick(t):
        return t if ridx is None else t[ridx]

    codes, scales = oracle.rotate_smooth_quantize(Xs, prep["amul"], group)
    want_codes = torch.from_numpy(codes if fmt == "c8" else oracle.pack_int4(codes)).cuda()
    assert torch.equal(pick(Xq).view(want_codes.dtype), want_codes), f"{spec.name}: codes differ from the oracle"
    assert torch.equal(pick(a_scale), torch.from_numpy(scales).cuda()), f"{spec.name}: scales differ from the oracle"
    del want_codes
    if check_gemm:
        if fmt == "c8":
            lin = (lambda acc: q.w4a4_linear_c8_grouped(h, Xq, a_scale, acc_debug=acc)) if group else \
                  (lambda acc: q.w4a4_linear_c8(h, Xq, a_scale, acc_debug=acc))
        else:
            lin = lambda acc: q.w4a4_linear(h, Xq, a_scale, group, acc_debug=acc)
        Y = lin(None)
        acc = oracle.gemm_i32(codes, prep["wq"], group)
        want = oracle.epilogue(acc, scales, prep["w_scale"], b)
        got = host_bits(pick(Y))
        frac = assert_bf16_within_one_ulp(got, want, spec.name)
        assert frac == 0.0, f"{spec.name}: {frac:.3e} of the compared outputs differ in the last bit"
        assert torch.isfinite(Y.float()).all()
        if check_acc:
            G = spec.K // 128 if group else 1
            dbg = torch.full((G, M, spec.N) if group else (M, spec.N), -12345, dtype=torch.int32, device="cuda")
            Yd = lin(dbg)
            got_acc = dbg if ridx is None else (dbg[:, ridx] if group else dbg[ridx])
            assert torch.equal(got_acc, torch.from_numpy(acc).cuda()), f"{spec.name}: integer sums differ from the oracle"
            assert torch.equal(Yd.view(torch.int16), Y.view(torch.int16)), f"{spec.name}: dump and production kernels disagree"
            del dbg, Yd
    assert h.device_status() == 0
    h.free()
    return M if ridx is None else len(rows)


# ------------------------------------------------------------------------------ config 1: one linear, one frame, seed 0
@pytest.mark.parametrize("fmt", ["packed", "c8"])
def test_config1_single_linear_one_frame_every_row(fmt):
    spec = workload.block_specs(0, 0)[1]                  # K = N = 1024
    assert (spec.K, spec.N) == (1024, 1024)
    assert run_layer(spec, F, fmt=fmt, check_acc=True) == F


# ------------------------------------------------------------------------------ config 2: one block, 8 frames: every row
@pytest.mark.parametrize("fmt", ["packed", "c8"])
@pytest.mark.parametrize("which", [0, 1, 2, 3])
def test_config2_block_linears_8_frames_every_row(which, fmt):
    spec = workload.block_specs(0, 0)[which]
    # the integer sums of every row as well for one K = 1024 and the K = 4096 layer of each kernel
    assert run_layer(spec, 8 * F, fmt=fmt, check_acc=which in (0, 3)) == 8 * F


@pytest.mark.parametrize("fmt", ["packed", "c8"])
@pytest.mark.parametrize("which", [1, 3])
def test_config2_group128_every_row_with_integer_sums(which, fmt):
    spec = workload.block_specs(0, 0)[which]
    assert run_layer(spec, 8 * F, group=128, fmt=fmt, check_acc=(which == 1)) == 8 * F


# ------------------------------------------------------------------------------ config 3: quantize kernel sweep, every row
@pytest.mark.parametrize("fmt", ["packed", "c8"])
@pytest.mark.parametrize("K,frames", [(1024, 1), (1024, 100), (4096, 1), (4096, 100)])
def test_config3_quantize_sweep_every_row(K, frames, fmt):
    M = frames * F
    X = workload.sweep_activations(3, K, 0, M)            # Student-t(3) entries, 1 % outlier channels x50
    spec = workload.LinearSpec("sweep", K, 128, workload.DIST_NORMAL, 3, 0)
    assert run_layer(spec, M, check_gemm=False, X=X, fmt=fmt) == M


# ------------------------------------------------------------------------------ config 4: 48-block stack, 32 frames
@pytest.mark.parametrize("fmt", ["packed", "c8"])
@pytest.mark.parametrize("block", [0, 23, 47])
def test_config4_stack_blocks_32_frames(block, fmt):
    """Three of the 48 blocks (first, middle, last) with their own seeded weights, smoothing factors and
    activations; all four linears at M = 43968.  One layer of each block on every row (a different one per block, so
    that qkv, fc1 and fc2 are all covered whole at this size), the others on every tile's edge rows."""
    whole = {0: 0, 23: 2, 47: 3}[block]
    for i, spec in enumerate(workload.block_specs(1, block)):
        n = run_layer(spec, 32 * F, rows="all" if i == whole else "edges", fmt=fmt)
        assert n == 32 * F if i == whole else n > 2 * (32 * F // 256)


# ------------------------------------------------------------------------------ config 5: 100 frames, fc1 / fc2, both granularities
@pytest.mark.parametrize("which,group,fmt,rows,acc", [
    (2, 0, "c8", "all", True),         # fc1 whole, with the integer sums: 537 token tiles x 16 channel tiles
    (3, 0, "c8", "edges", False),
    (2, 0, "packed", "edges", False),
    (3, 0, "packed", "all", False),    # fc2 whole through the packed-operand kernel
    (2, 128, "packed", "edges", False),
    (3, 128, "packed", "edges", False),
    (2, 128, "c8", "all", False),      # group-wise scales on the TMA-fed GEMM, every row
    (3, 128, "c8", "edges", False),
])
def test_config5_large_scene(which, group, fmt, rows, acc):
    spec = workload.block_specs(4, 0)[which]
    n = run_layer(spec, 100 * F, rows=rows, group=group, fmt=fmt, check_acc=acc)
    assert n == 100 * F if rows == "all" else n > 2 * (100 * F // 256)
