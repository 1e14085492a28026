"""Pins for the CPU oracle: what the paper and the mathematics fix, checked without the CUDA path.

Each test names the passage it leans on.  Where a check recomputes something, it does so by a
different route than the oracle (dense +-1 matrices from the closed form, numpy int64/fp64 matmul,
pure-Python loops), never by retyping the oracle's own loop.
"""
import os

import numpy as np
import pytest

import oracle
import workload

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def f32_to_bf16_bits(a):
    """Exact only for values already representable in bf16 (asserted)."""
    a = np.asarray(a, np.float32)
    u = a.view(np.uint32)
    assert np.all((u & 0xFFFF) == 0), "test input is not bf16-representable"
    return (u >> 16).astype(np.uint16)


def sylvester(K):
    """Closed form of the Kronecker recursion: H[i][j] = (-1)^popcount(i & j)."""
    i = np.arange(K, dtype=np.int64)
    x = i[:, None] & i[None, :]
    pc = np.zeros_like(x)
    while np.any(x):
        pc += x & 1
        x >>= 1
    return (1 - 2 * (pc & 1)).astype(np.int64)


def load_table(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append([float(t) for t in line.split()])
    return np.array(rows)


def ordered_bf16(bits):
    """bf16 bit patterns -> integers ordered like the values (adjacent values differ by one)."""
    b = np.asarray(bits).astype(np.int32)
    return np.where(b & 0x8000, -(b & 0x7FFF), b & 0x7FFF)


# ------------------------------------------------------------------ Hadamard (Sec. 3.2, Pre-Global-Rotation)
def test_h8_matches_handwritten_kronecker_recursion():
    H8 = load_table("sylvester_h8.txt")
    assert H8.shape == (8, 8)
    got = oracle.fwht_f32(np.eye(8, dtype=np.float32))  # row j = e_j H
    assert np.array_equal(got, H8.astype(np.float32))
    assert np.array_equal(sylvester(8), H8.astype(np.int64))  # the closed form used below agrees too


@pytest.mark.parametrize("K", [2, 4, 16, 64, 1024, 4096])
def test_fwht_of_unit_vectors_is_closed_form_column(K):
    H = sylvester(K) if K <= 1024 else None
    for j in sorted({j for j in (0, 1, 2, 3, K // 2, K - 1, (K // 3) | 1) if j < K}):
        e = np.zeros(K, np.float32)
        e[j] = 1.0
        got = oracle.fwht_f32(e)
        if H is not None:
            want = H[j]
        else:
            i = np.arange(K)
            want = 1 - 2 * (np.array([bin(v).count("1") for v in (i & j)]) & 1)
        assert np.array_equal(got, want.astype(np.float32)), (K, j)


@pytest.mark.parametrize("K", [2, 8, 64])
def test_h_ht_equals_k_identity(K):
    H = oracle.fwht_f64(np.eye(K))
    assert np.array_equal(H @ H.T, K * np.eye(K))
    assert np.array_equal(H, H.T)


@pytest.mark.parametrize("K", [16, 1024, 4096])
def test_fwht_twice_is_k_times_identity_on_small_integers(K):
    rng = np.random.default_rng(K)
    x = rng.integers(-8, 9, size=(3, K)).astype(np.float32)
    assert np.array_equal(oracle.fwht_f32(oracle.fwht_f32(x)), K * x)


@pytest.mark.parametrize("K", [64, 1024, 4096])
def test_fwht_equals_dense_product_on_integer_inputs(K):
    """Integer inputs keep every fp32 partial sum exact, so any butterfly order must match x @ H."""
    rng = np.random.default_rng(7 + K)
    x = rng.integers(-100, 101, size=(4, K)).astype(np.int64)
    want = x @ sylvester(K)
    got = oracle.fwht_f32(x.astype(np.float32))
    assert np.array_equal(got.astype(np.int64), want)
    got64 = oracle.fwht_f64(x.astype(np.float64))
    assert np.array_equal(got64.astype(np.int64), want)


@pytest.mark.parametrize("K", [1024, 4096])
def test_fwht_f32_stays_within_rounding_bound_of_f64(K):
    spec = workload.LinearSpec("t", K, 8, workload.DIST_NORMAL, 11, 0)
    x = workload.bf16_to_f32(spec.x_rows(0, 6)).astype(np.float64)
    u64 = oracle.fwht_f64(x)
    u32 = oracle.fwht_f32(x.astype(np.float32)).astype(np.float64)
    bound = np.log2(K) * 2.0 ** -24 * np.abs(x).sum(axis=1, keepdims=True) * 1.01
    assert np.all(np.abs(u32 - u64) <= bound)
    assert np.any(u32 != u64)  # the fp32 path really rounds (so the bound is not vacuous)


def test_rotation_invariance_fp64():
    """X W^T = (X H)(W H)^T for the random Hadamard H = K^-1/2 H_K diag(v), H^T H = I."""
    K, M, N = 1024, 9, 7
    spec = workload.LinearSpec("t", K, N, workload.DIST_NORMAL, 3, 0)
    X, W = spec.x_rows(0, M), spec.weight()
    v = workload.signs_i8(3, 9, K).astype(np.float64)
    assert set(np.unique(v)) == {-1.0, 1.0}
    mul = v / np.sqrt(K)
    lhs = oracle.rotate_f64(X, mul) @ oracle.rotate_f64(W, mul).T
    rhs = workload.bf16_to_f32(X).astype(np.float64) @ workload.bf16_to_f32(W).astype(np.float64).T
    assert np.max(np.abs(lhs - rhs)) <= 1e-12 * np.max(np.abs(rhs))


@pytest.mark.parametrize("K", [1024, 4096])
def test_smoothing_invariance_fp64_with_oracle_multipliers(K):
    """X W^T = (X H diag(c)^-1)(diag(c) H^T W^T) using the multipliers the oracle really applies."""
    M, N = 6, 5
    spec = workload.LinearSpec("t", K, N, workload.DIST_NORMAL, 5, 0)
    X, W = spec.x_rows(0, M), spec.weight()
    c = workload.loguniform_f32(5, 50, K, 1e-2, 1e2)
    v = workload.signs_i8(5, 51, K)
    amul, wmul = oracle.multipliers(c, v)
    assert amul.dtype == np.float32 and np.all(np.sign(amul) == v) and np.all(np.sign(wmul) == v)
    nrm = np.float32(2.0 ** -(np.log2(K) / 2))
    assert np.array_equal(amul, (v * nrm).astype(np.float32) / c)  # one IEEE division
    assert np.array_equal(wmul, (v * nrm).astype(np.float32) * c)
    lhs = oracle.rotate_f64(X, amul.astype(np.float64)) @ oracle.rotate_f64(W, wmul.astype(np.float64)).T
    rhs = workload.bf16_to_f32(X).astype(np.float64) @ workload.bf16_to_f32(W).astype(np.float64).T
    # amul*wmul = (1/K)(1 + O(2^-23)) per channel, so the identity holds to fp32 rounding of c
    assert np.max(np.abs(lhs - rhs)) <= 4e-7 * np.sum(np.abs(workload.bf16_to_f32(X[:, None, :]).astype(np.float64)
                                                            * workload.bf16_to_f32(W[None]).astype(np.float64)), axis=2).max()


def test_default_signs_are_plus_one():
    c = workload.loguniform_f32(1, 2, 1024, 0.1, 10)
    a0, w0 = oracle.multipliers(c, None)
    a1, w1 = oracle.multipliers(c, np.ones(1024, np.int8))
    assert np.array_equal(a0, a1) and np.array_equal(w0, w1) and np.all(a0 > 0)


# ------------------------------------------------------------------ quantizer (Eq. "quantization", N = 4)
def _rotated_y(X, mul):
    u = oracle.fwht_f32(workload.bf16_to_f32(X))
    return u * mul.astype(np.float32)[None, :]


@pytest.mark.parametrize("K,group", [(1024, 0), (4096, 0), (1024, 128), (4096, 128)])
def test_quantizer_error_bound_and_range(K, group):
    spec = workload.LinearSpec("t", K, 8, workload.DIST_NORMAL, 21, 0)
    X = spec.x_rows(0, 12)  # includes the five x100 special rows
    c = workload.loguniform_f32(21, 5, K, 0.05, 20)
    amul, _ = oracle.multipliers(c, workload.signs_i8(21, 6, K))
    codes, scales = oracle.rotate_smooth_quantize(X, amul, group)
    y = _rotated_y(X, amul).astype(np.float64)
    G = K // group if group else 1
    yg = y.reshape(12, G, -1)
    qg = codes.reshape(12, G, -1).astype(np.float64)
    sg = scales.reshape(12, G, 1).astype(np.float64)
    assert np.all(np.abs(yg - sg * qg) <= sg / 2 * (1 + 2.0 ** -22))      # |x - Delta q| <= Delta / 2
    amax = np.abs(yg).max(axis=2, keepdims=True)
    assert np.array_equal(sg.astype(np.float32), (amax.astype(np.float32) / np.float32(7)))  # Delta = max|x| / 7
    assert codes.min() >= -7 and codes.max() <= 7                           # -8 is never produced
    hit = np.abs(yg) == amax
    assert np.all(np.abs(qg[hit]) == 7)                                     # the absmax element maps to +-7
    assert np.all(np.sign(qg[hit]) == np.sign(yg[hit]))


@pytest.mark.parametrize("bits", [8, 6, 4])
def test_nbit_quantizer_error_bound_range_and_independent_rounding(bits):
    """Eq. "quantization" for general N (N = 8 is the W8A8 setting): Delta = max|x| / (2^(N-1) - 1), error at most
    Delta / 2, the absolute maximum maps to +-(2^(N-1) - 1), the most negative code never appears; away from ties
    the codes equal an independent float64 evaluation of round(y / Delta)."""
    K, qmax = 1024, 2 ** (bits - 1) - 1
    spec = workload.LinearSpec("t", K, 8, workload.DIST_NORMAL, 23, 0)
    X = spec.x_rows(0, 12)
    c = workload.loguniform_f32(23, 5, K, 0.05, 20)
    amul, _ = oracle.multipliers(c, workload.signs_i8(23, 6, K))
    codes, scales = oracle.rotate_smooth_quantize(X, amul, 0, bits)
    y = _rotated_y(X, amul).astype(np.float64)
    q, s_ = codes.astype(np.float64), scales.astype(np.float64)[:, None]
    assert np.all(np.abs(y - s_ * q) <= s_ / 2 * (1 + 2.0 ** -20))
    amax = np.abs(y).max(axis=1, keepdims=True)
    assert np.array_equal(scales, (amax[:, 0].astype(np.float32) / np.float32(qmax)))
    assert codes.min() >= -qmax and codes.max() <= qmax
    hit = np.abs(y) == amax
    assert np.all(np.abs(q[hit]) == qmax) and np.all(np.sign(q[hit]) == np.sign(y[hit]))
    t = y * qmax / amax                                    # float64, a different evaluation order
    clear = np.abs(t - np.floor(t) - 0.5) > 1e-4           # not within 1e-4 of a rounding boundary
    assert clear.mean() > 0.99
    assert np.array_equal(q[clear], np.rint(t)[clear])
    if bits == 4:                                          # the general routine at N = 4 is the W4A4 routine
        c4, s4 = oracle.rotate_smooth_quantize(X, amul, 0)
        assert np.array_equal(c4, codes) and np.array_equal(s4, scales)


def test_8bit_round_half_to_even_and_extremes():
    """N = 8 on exactly representable values: a unit vector rotates to all ones, so y equals the multiplier vector;
    with amax = 127 the factor 127/amax is 1 and y itself is rounded: ties go to the even integer, +-127 stay,
    nothing reaches -128."""
    K = 16
    y = np.array([127.0, -127.0, 0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 126.5, -126.5, 63.5, 64.5, 0.0, 1.0, -100.5, 99.5], np.float32)
    want = np.array([127, -127, 0, 2, 2, 0, -2, -2, 126, -126, 64, 64, 0, 1, -100, 100], np.int8)
    X = np.zeros((1, K), np.uint16)
    X[0, 0] = 0x3F80                                              # 1.0: its transform is the all-ones row of H_16
    assert np.array_equal(oracle.fwht_f32(workload.bf16_to_f32(X))[0], np.ones(K, np.float32))
    codes, scales = oracle.rotate_smooth_quantize(X, y, 0, 8)
    assert scales[0] == np.float32(1.0)
    assert np.array_equal(codes[0], want)


@pytest.mark.parametrize("bits", [4, 8])
def test_static_quantizer_power_of_two_step_against_float64(bits):
    """Static tensor-wise quantizer (Tab. "granularity"): with Delta a power of two, y / Delta is exact in any
    precision, so the codes must equal clamp(rint(y / Delta)) computed independently in float64; both ends of the
    clamp are reached (outlier channels and special-token rows)."""
    K = 1024
    spec = workload.LinearSpec("t", K, 8, workload.DIST_NORMAL, 29, 0)
    X = spec.x_rows(0, 12)
    amul, _ = oracle.multipliers(workload.loguniform_f32(29, 5, K, 0.05, 20), workload.signs_i8(29, 6, K))
    y = _rotated_y(X, amul).astype(np.float64)
    delta = 2.0 ** np.floor(np.log2(np.median(np.abs(y)) / 2))
    codes = oracle.rotate_smooth_quantize_static(X, amul, float(delta), bits)
    lo, hi = -(2 ** (bits - 1)), 2 ** (bits - 1) - 1
    want = np.clip(np.rint(y / delta), lo, hi)
    assert np.array_equal(codes.astype(np.float64), want)
    assert codes.min() == lo and codes.max() == hi                 # the clamp is exercised on both sides
    inside = (want > lo) & (want < hi)
    assert np.all(np.abs(y - delta * want)[inside] <= delta / 2)     # |x - Delta q| <= Delta / 2 where nothing was clamped


def test_static_quantizer_ties_and_saturation_by_hand():
    """Delta = 1 on hand-picked values (a unit vector rotates to all ones, so y equals the multiplier vector)."""
    K = 16
    y = np.array([0.5, 1.5, 2.5, -0.5, 7.49, 7.5, 7.51, 8.5, 100.0, -8.5, -9.0, -100.0, 1e30, -1e30, 6.5, -7.5], np.float32)
    want = np.array([0, 2, 2, 0, 7, 7, 7, 7, 7, -8, -8, -8, 7, -8, 6, -8], np.int8)
    X = np.zeros((1, K), np.uint16)
    X[0, 0] = 0x3F80
    assert np.array_equal(oracle.rotate_smooth_quantize_static(X, y, 1.0, 4)[0], want)
    # a step that is not a power of two: the factor is fl(1/3); 4.5 * fl(1/3) = 1.5000000447 rounds up to 2
    y3 = np.array([3.0, 4.5, -4.5, 1.5, 21.0, 22.5, -24.0, -25.5] * 2, np.float32)
    want3 = np.array([1, 2, -2, 1, 7, 7, -8, -8] * 2, np.int8)
    assert float(np.float32(1.0) / np.float32(3.0)) > 1.0 / 3.0    # fl(1/3) lies above 1/3
    assert np.array_equal(oracle.rotate_smooth_quantize_static(X, y3, 3.0, 4)[0], want3)


@pytest.mark.parametrize("K", [1024, 4096])
def test_layernorm_against_float64_and_special_rows(K):
    """LayerNorm of the upstream-fusion row: within fp32 rounding of a float64 LayerNorm (numpy, a different
    summation) on heavy-tailed rows, so a wrong statistic, a dropped eps, gamma or beta would show; exact on rows
    whose arithmetic is exact (constant row -> beta; a +-a row with gamma = a power of two)."""
    spec = workload.LinearSpec("t", K, 8, workload.DIST_NORMAL, 37, 0)
    X = spec.x_rows(0, 9)
    rng = np.random.default_rng(K)
    gamma = rng.uniform(0.5, 2.0, K).astype(np.float32)
    beta = rng.normal(0, 0.3, K).astype(np.float32)
    eps = 1e-5
    got = workload.bf16_to_f32(oracle.layernorm(X, gamma, beta, eps)).astype(np.float64)
    x = workload.bf16_to_f32(X).astype(np.float64)
    mu = x.mean(axis=1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=1, keepdims=True)
    want = (x - mu) / np.sqrt(var + eps) * gamma + beta
    assert np.all(np.abs(got - want) <= 2.0 ** -8 * np.abs(want) + 1e-5 * (np.abs(x - mu) / np.sqrt(var + eps) + 1))
    # constant row: d = 0 exactly, so the output is bf16(beta) whatever gamma is
    Xc = np.full((1, K), 0x4049, np.uint16)
    assert np.array_equal(oracle.layernorm(Xc, gamma, beta, eps), f32_round_to_bf16_bits(beta)[None, :])
    # +-2 alternating: mean 0, var 4, rstd = fl(1/sqrt(4 + eps)); output = bf16(fl(fl(+-2 * rstd) * 4) + 0)
    Xa = np.tile(np.array([0x4000, 0xC000], np.uint16), K // 2)[None, :]
    rstd = np.float32(1.0) / np.sqrt(np.float32(4.0) + np.float32(eps), dtype=np.float32)
    val = np.float32(np.float32(2.0) * rstd) * np.float32(4.0)
    out = oracle.layernorm(Xa, np.full(K, 4.0, np.float32), np.zeros(K, np.float32), eps)
    assert np.array_equal(out[0, 0::2], np.full(K // 2, f32_round_to_bf16_bits(np.array([val]))[0]))
    assert np.array_equal(out[0, 1::2], np.full(K // 2, f32_round_to_bf16_bits(np.array([-val]))[0]))


def test_layernorm_pairwise_order_is_the_stated_tree():
    """The statistic is summed pairwise (halves, recursively), not left to right: a row on which the two orders
    give different fp32 sums must follow the tree."""
    K = 1024
    x = np.zeros(K, np.float32)
    x[0] = 2.0 ** 24                 # left to right, every later 1.0 is absorbed by 2^24; pairwise keeps them
    x[1:] = 1.0
    X = (x.view(np.uint32) >> 16).astype(np.uint16)[None, :]

    def pairwise(a):
        a = a.astype(np.float32)
        while a.size > 1:
            a = (a[0::2] + a[1::2]).astype(np.float32)
        return a[0]

    seq = np.float32(0)
    for v in x:
        seq = np.float32(seq + v)
    assert pairwise(x) != seq
    mean = np.float32(pairwise(x) * np.float32(1.0 / K))
    d = (x - mean).astype(np.float32)
    var = np.float32(pairwise((d * d).astype(np.float32)) * np.float32(1.0 / K))
    rstd = np.float32(1.0) / np.sqrt(np.float32(var + np.float32(1e-5)), dtype=np.float32)
    want = f32_round_to_bf16_bits((d * rstd).astype(np.float32))
    got = oracle.layernorm(X, np.ones(K, np.float32), np.zeros(K, np.float32), 1e-5)[0]
    assert np.array_equal(got, want)


def f32_round_to_bf16_bits(a):
    """Round-to-nearest-even fp32 -> bf16 bits, written out independently of the oracle."""
    u = np.asarray(a, np.float32).view(np.uint32).astype(np.uint64)
    return (((u + 0x7FFF + ((u >> 16) & 1)) >> 16) & 0xFFFF).astype(np.uint16)


def test_round_half_to_even_on_handbuilt_ties():
    tab = load_table("round_ties.txt")
    y, want = tab[:, 0], tab[:, 1].astype(np.int8)
    K = len(y)
    assert K == 16
    x = (sylvester(K) @ y) / K                     # x H_K = y exactly (all partial sums are dyadic and small)
    X = f32_to_bf16_bits(x.astype(np.float32))[None, :]
    assert np.array_equal(oracle.fwht_f32(workload.bf16_to_f32(X))[0], y.astype(np.float32))
    codes, scales = oracle.rotate_smooth_quantize(X, np.ones(K, np.float32), 0)
    assert scales[0] == np.float32(1.0)
    assert np.array_equal(codes[0], want)


def test_zero_row_gives_zero_codes_and_floor_scale():
    X = np.zeros((2, 1024), np.uint16)
    X[1, 5] = 0x3F80
    codes, scales = oracle.rotate_smooth_quantize(X, np.full(1024, 2.0 ** -5, np.float32), 0)
    assert not codes[0].any() and scales[0] == np.float32(1e-8) / np.float32(7)
    # a single 1.0 spreads to +-2^-5 everywhere: every code is +-7 and follows the Sylvester column
    assert np.array_equal(codes[1], 7 * sylvester(1024)[5])
    assert scales[1] == np.float32(2.0 ** -5) / np.float32(7)


def test_group_equal_to_k_reduces_to_per_token():
    K = 1024
    spec = workload.LinearSpec("t", K, 8, workload.DIST_NORMAL, 2, 0)
    X = spec.x_rows(0, 7)
    amul, _ = oracle.multipliers(workload.loguniform_f32(2, 5, K, 0.1, 10))
    c0, s0 = oracle.rotate_smooth_quantize(X, amul, 0)
    c1, s1 = oracle.rotate_smooth_quantize(X, amul, K)
    assert np.array_equal(c0, c1) and np.array_equal(s0, s1.reshape(-1))
    acc0 = oracle.gemm_i32(c0, c0[:5], 0)
    acc1 = oracle.gemm_i32(c0, c0[:5], K)
    assert np.array_equal(acc0, acc1[0])


def test_pack_layout_low_nibble_is_even_index():
    codes = np.array([[1, -1, 7, -8, 0, 3, -7, 5]], np.int8)
    packed = oracle.pack_int4(codes)
    assert packed.tolist() == [[0xF1, 0x87, 0x30, 0x59]]
    assert np.array_equal(oracle.unpack_int4(packed), codes)
    rng = np.random.default_rng(0)
    r = rng.integers(-8, 8, size=(5, 64)).astype(np.int8)
    assert np.array_equal(oracle.unpack_int4(oracle.pack_int4(r)), r)


# ------------------------------------------------------------------ integer GEMM (Sec. 3.2, granularity)
def test_gemm_bruteforce_tiny():
    rng = np.random.default_rng(1)
    M, N, K = 3, 4, 8
    a = rng.integers(-8, 8, size=(M, K)).astype(np.int8)
    b = rng.integers(-8, 8, size=(N, K)).astype(np.int8)
    want = [[sum(int(a[m, k]) * int(b[n, k]) for k in range(K)) for n in range(N)] for m in range(M)]
    assert oracle.gemm_i32(a, b).tolist() == want
    assert oracle.gemm_i32(a, b).shape == (M, N)  # [tokens, out channels], not transposed


@pytest.mark.parametrize("K,group", [(1024, 0), (4096, 0), (1024, 128), (4096, 128)])
def test_gemm_matches_int64_matmul_and_bound(K, group):
    rng = np.random.default_rng(K + group)
    M, N = 11, 13
    a = rng.integers(-7, 8, size=(M, K)).astype(np.int8)
    b = rng.integers(-7, 8, size=(N, K)).astype(np.int8)
    a[0], b[0] = 7, -7                                    # extreme row: acc = -49 K
    acc = oracle.gemm_i32(a, b, group)
    if group:
        G = K // group
        want = np.einsum("mgk,ngk->gmn", a.reshape(M, G, -1).astype(np.int64), b.reshape(N, G, -1).astype(np.int64))
        assert acc.shape == (G, M, N) and np.array_equal(acc, want)
        assert np.array_equal(acc.sum(axis=0), a.astype(np.int64) @ b.astype(np.int64).T)
    else:
        assert np.array_equal(acc, a.astype(np.int64) @ b.astype(np.int64).T)
        assert acc[0, 0] == -49 * K
    assert np.abs(acc).max() <= 49 * K


# ------------------------------------------------------------------ epilogue
def bf16_neighbors_ok(got_bits, want_f64):
    """got is the bf16 nearest to want_f64, or one of its two neighbours."""
    got = oracle.bf16_to_f32(got_bits).astype(np.float64)
    ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(want_f64), 1e-300))) - 7)
    return np.abs(got - want_f64) <= ulp * 1.0000001


def test_epilogue_against_fp64_recomputation():
    rng = np.random.default_rng(4)
    M, N = 17, 19
    acc = rng.integers(-200000, 200001, size=(M, N)).astype(np.int32)
    a_s = rng.uniform(0.01, 3.0, M).astype(np.float32)
    w_s = rng.uniform(1e-4, 1e-2, N).astype(np.float32)
    bias = workload.normal_bf16(4, 1, 1, N, 0.01).reshape(N)
    Y = oracle.epilogue(acc, a_s, w_s, bias)
    want = acc.astype(np.float64) * a_s[:, None].astype(np.float64) * w_s[None, :].astype(np.float64) \
        + oracle.bf16_to_f32(bias).astype(np.float64)[None, :]
    assert np.all(bf16_neighbors_ok(Y, want))
    Y0 = oracle.epilogue(acc, a_s, w_s, None)
    assert np.all(bf16_neighbors_ok(Y0, want - oracle.bf16_to_f32(bias).astype(np.float64)[None, :]))


def test_epilogue_exact_special_cases():
    N = 8
    bias = workload.normal_bf16(9, 1, 1, N, 0.01).reshape(N)
    zero = np.zeros((2, N), np.int32)
    one = np.ones(2, np.float32)
    assert np.array_equal(oracle.epilogue(zero, one, np.ones(N, np.float32), bias), np.tile(bias, (2, 1)))  # acc = 0 -> bias
    acc = np.arange(-8, 8, dtype=np.int32).reshape(2, N) * 3
    Y = oracle.epilogue(acc, 2 * one, np.full(N, 0.5, np.float32), None)       # scales cancel -> small integers, exact
    assert np.array_equal(oracle.bf16_to_f32(Y), acc.astype(np.float32))
    # per-token scale goes with the row, per-channel scale with the column
    a_s = np.array([1.0, 4.0], np.float32)
    w_s = np.array([1, 2, 1, 1, 1, 1, 1, 8], np.float32)
    Y = oracle.bf16_to_f32(oracle.epilogue(np.ones((2, N), np.int32), a_s, w_s, None))
    assert np.array_equal(Y, a_s[:, None] * w_s[None, :])


def test_epilogue_groupwise_against_fp64():
    rng = np.random.default_rng(6)
    G, M, N = 8, 5, 6
    acc = rng.integers(-6000, 6001, size=(G, M, N)).astype(np.int32)
    a_s = rng.uniform(0.01, 3.0, (M, G)).astype(np.float32)
    w_s = rng.uniform(1e-4, 1e-2, N).astype(np.float32)
    bias = workload.normal_bf16(6, 1, 1, N, 0.01).reshape(N)
    Y = oracle.bf16_to_f32(oracle.epilogue(acc, a_s, w_s, bias)).astype(np.float64)
    terms = acc.astype(np.float64) * a_s.T[:, :, None].astype(np.float64)
    want = terms.sum(axis=0) * w_s[None, :] + oracle.bf16_to_f32(bias)[None, :]
    slack = 2.0 ** -7 * np.abs(want) + G * 2.0 ** -23 * np.abs(terms).sum(axis=0) * w_s[None, :]
    assert np.all(np.abs(Y - want) <= slack)


# ------------------------------------------------------------------ smoothing factors (Eq. "smooth_factor")
def test_smooth_factors_against_dense_closed_form():
    K, Mc, N = 64, 10, 12
    X = workload.activations(8, 0, 0, Mc, K, workload.DIST_NORMAL, workload.outlier_gains(8, 1, K, 2), frame_rows=0)
    W = workload.normal_bf16(8, 2, N, K, 0.02)
    H = sylvester(K).astype(np.float64) / np.sqrt(K)
    ax = np.abs(workload.bf16_to_f32(X).astype(np.float64) @ H).max(axis=0)
    aw = np.abs(workload.bf16_to_f32(W).astype(np.float64) @ H).max(axis=0)
    for alpha in (0.3, 0.5, 0.7):
        want = np.clip(ax ** alpha / aw ** (1 - alpha), 1e-2, 1e2)
        got = oracle.smooth_factors(X, W, alpha)
        assert np.allclose(got, want, rtol=1e-6, atol=0)
    # clipping and the 0/0 convention
    Xz = np.zeros((3, K), np.uint16)
    Wz = np.zeros((3, K), np.uint16)
    assert np.array_equal(oracle.smooth_factors(Xz, Wz), np.ones(K, np.float32))
    assert np.array_equal(oracle.smooth_factors(Xz, W), np.full(K, 1e-2, np.float32))
    assert np.array_equal(oracle.smooth_factors(X, Wz), np.full(K, 1e2, np.float32))


# ------------------------------------------------------------------ whole layer
def test_linear_f64_is_x_wt_plus_b():
    spec = workload.LinearSpec("t", 64, 5, workload.DIST_NORMAL, 1, 0)
    X, W, b = spec.x_rows(0, 4), spec.weight(), spec.bias()
    want = workload.bf16_to_f32(X).astype(np.float64) @ workload.bf16_to_f32(W).astype(np.float64).T \
        + workload.bf16_to_f32(b).astype(np.float64)
    assert np.allclose(oracle.linear_f64(X, W, b), want, rtol=1e-13, atol=1e-15)


@pytest.mark.parametrize("group", [0, 128])
def test_quantized_layer_approximates_the_fp_layer(group):
    """Information-level sanity (parity unpinned by the paper): the W4A4 output tracks X W^T + b."""
    spec = workload.LinearSpec("proj", 1024, 256, workload.DIST_NORMAL, 0, 1)
    X, W, b = spec.x_rows(0, 64), spec.weight(), spec.bias()
    c = oracle.smooth_factors(spec.x_calib(256), W)
    prep = oracle.prepare_weights(W, c, None)
    out = oracle.w4a4_linear(X, prep, b, group)
    ref = oracle.linear_f64(X, W, b)
    y = oracle.bf16_to_f32(out["y"]).astype(np.float64)
    rel = np.linalg.norm(y - ref) / np.linalg.norm(ref)
    assert rel < 0.25, rel
    # dequantized integer sums reproduce the same numbers (scales factor out of the sum)
    if not group:
        deq = out["acc"].astype(np.float64) * out["a_scale"][:, None] * prep["w_scale"][None, :] \
            + oracle.bf16_to_f32(b)[None, :]
        assert np.all(bf16_neighbors_ok(out["y"], deq))


# ------------------------------------------------------------------ wide rotation (reference of the tolerance contract)
@pytest.mark.parametrize("K", [1024, 4096])
def test_wide_rotation_quantizer_equals_fp32_one_where_fp32_is_exact(K):
    """On small-integer inputs every butterfly of the fp32 transform is exact, so rounding order cannot matter: the
    quantizer behind the fp64 rotation must return the codes and scales of the fp32 one, bit for bit (Sec. 3.2,
    Pre-Global-Rotation: the Kronecker recursion defines ONE transform, whatever the evaluation order)."""
    rng = np.random.default_rng(K)
    x = rng.integers(-3, 4, size=(9, K)).astype(np.float32)
    x[3] = 0
    X = f32_to_bf16_bits(x)
    mul = (rng.choice([-1.0, 1.0], K) * 2.0 ** rng.integers(-7, -3, K)).astype(np.float32)
    for bits in (4, 8):
        codes, scales = oracle.rotate_smooth_quantize(X, mul, 0, bits)
        wide = oracle.rotate_smooth_quantize_wide(X, mul, bits)
        assert np.array_equal(wide["codes"], codes) and np.array_equal(wide["scales"], scales)
        assert np.array_equal(wide["abs_sum"], np.abs(x.astype(np.float64)).sum(axis=1))
        # its rotated rows are the dense +-1 product (exact in integers) times the multiplier
        dense = (x.astype(np.int64) @ sylvester(K) if K <= 1024 else oracle.fwht_f64(x.astype(np.float64))).astype(np.float64)
        assert np.array_equal(wide["y"].astype(np.float64), dense * mul.astype(np.float64))


@pytest.mark.parametrize("K", [1024, 4096])
def test_wide_rotation_quantizer_on_heavy_tailed_rows(K):
    """On real-valued rows the two quantizers may differ, but only as far as the fp32 transform's rounding allows:
    rotated values within log2(K) 2^-24 sum|x| |mul| of each other, quantizer error bound |y - Delta q| <= Delta / 2
    (Eq. "quantization") for the wide one as well, codes apart by at most one and only next to a rounding boundary."""
    X = workload.sweep_activations(5, K, 0, 64)
    mul = oracle.multipliers(workload.loguniform_f32(5, 1, K, 0.1, 10.0), workload.signs_i8(5, 2, K))[0]
    wide = oracle.rotate_smooth_quantize_wide(X, mul)
    codes, scales = oracle.rotate_smooth_quantize(X, mul, 0)
    y64 = oracle.rotate_f64(X, mul.astype(np.float64))
    tol = (np.log2(K) * 2.0 ** -24 * wide["abs_sum"])[:, None] * np.abs(mul)[None, :].astype(np.float64)
    assert np.all(np.abs(wide["y"].astype(np.float64) - y64) <= 2.0 ** -23 * np.abs(y64) + 1e-300)   # two roundings in all
    delta = wide["scales"].astype(np.float64)[:, None]
    assert np.all(np.abs(wide["y"].astype(np.float64) - delta * wide["codes"]) <= delta / 2 * (1 + 2.0 ** -20))
    assert np.all(np.abs(wide["codes"]).max(axis=1) == 7) and wide["codes"].min() >= -7
    assert np.all(np.abs(wide["scales"] - scales) <= (tol.max(axis=1) / 7 + 2.0 ** -22 * scales))
    diff = wide["codes"].astype(np.int32) - codes
    assert np.abs(diff).max() <= 1
    pos = y64 * (7.0 / np.abs(y64).max(axis=1))[:, None]                  # position on the code axis, fp64
    to_boundary = np.abs(pos - (np.floor(pos) + 0.5))
    slack = 7.0 / np.abs(y64).max(axis=1)[:, None] * 2 * tol + 2.0 ** -20
    assert np.all(to_boundary[diff != 0] <= slack[diff != 0])
    assert (diff != 0).mean() < 1e-3


# ------------------------------------------------------------------ GELU (the producer of fc2's input)
def test_gelu_matches_tabulated_normal_distribution():
    tab = load_table("normal_cdf.txt")
    for x, phi in tab:
        want = x * phi
        got = oracle.gelu_f64(x)
        assert abs(got - want) <= 2e-14 * abs(want) + 1e-300, (x, got, want)     # the table carries 15 digits


def test_gelu_identities_and_library_cdf():
    from scipy.special import ndtr
    x = np.concatenate([np.linspace(-12.0, 8.0, 4001), [0.0, -0.0, 1e-30, -1e-30, 37.0, -37.0]])
    g = np.array([oracle.gelu_f64(v) for v in x])
    assert np.allclose(g, x * ndtr(x), rtol=1e-13, atol=0.0)
    gm = np.array([oracle.gelu_f64(-v) for v in x])
    assert np.allclose(g - gm, x, rtol=1e-15, atol=1e-300)                       # Phi(x) + Phi(-x) = 1
    assert np.all(g[x > 0] > 0) and np.all(g[x < 0] <= 0) and g[list(x).index(0.0)] == 0.0
    grid = x[:4001]
    assert np.all(np.diff(g[:4001][(grid > -0.75) & (grid < 8.0)]) > 0)          # increasing right of its minimum (x ~ -0.7518)
    assert abs(min(g) - (-0.16997120747990369)) < 2e-5                           # the minimum of x Phi(x)


def test_gelu_bf16_is_the_nearest_bf16_of_the_fp64_value():
    rng = np.random.default_rng(3)
    xb = f32_to_bf16_bits((rng.standard_normal((37, 128)) * 3).astype(np.float32).view(np.uint32).__and__(0xFFFF0000).view(np.float32))
    out = oracle.gelu(xb)
    x = oracle.bf16_to_f32(xb).astype(np.float64)
    want = x * __import__("scipy.special", fromlist=["ndtr"]).ndtr(x)
    got = oracle.bf16_to_f32(out).astype(np.float64)
    ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(want), 1e-300))) - 7)
    assert np.all(np.abs(got - want) <= ulp / 2 * (1 + 1e-9))                    # correctly rounded: within half a bf16 ulp
    # rows with a stride, zeros keep their sign
    z = np.array([[0x0000, 0x8000, 0x3F80, 0xBF80]], np.uint16)
    assert [int(v) & 0x7FFF for v in oracle.gelu(z)[0][:2]] == [0, 0]
    wide = np.zeros((4, 256), np.uint16)
    wide[:, :128] = xb[:4]
    assert np.array_equal(oracle.gelu(wide[:, :128]), out[:4])


# ------------------------------------------------------------------ tensor-wise weight quantizer (Tab. "granularity")
@pytest.mark.parametrize("bits", [4, 8])
def test_tensorwise_weight_quantizer_bound_extreme_and_reduction_to_channelwise(bits):
    K, N = 1024, 24
    qmax = 2 ** (bits - 1) - 1
    W = workload.normal_bf16(9, 1, N, K, 0.02)
    c = workload.loguniform_f32(9, 2, K, 0.2, 5.0)
    tw = oracle.prepare_weights(W, c, None, bits, tensorwise=True)
    cw = oracle.prepare_weights(W, c, None, bits)
    delta = tw["w_scale"][0]
    assert np.all(tw["w_scale"] == delta) and delta == cw["w_scale"].max()          # one step for the tensor: the largest row's
    y = oracle.rotate_f64(W, tw["wmul"].astype(np.float64))
    assert abs(delta * qmax - np.abs(y).max()) <= 2.0 ** -20 * np.abs(y).max()       # Delta = max|W~| / qmax
    assert np.all(np.abs(y - np.float64(delta) * tw["wq"]) <= delta / 2 * (1 + 2.0 ** -12))   # Eq. "quantization": |y - Delta q| <= Delta / 2
    assert np.abs(tw["wq"]).max() == qmax and tw["wq"].min() >= -qmax                # the largest element reaches +-qmax, nothing clips
    row = int(np.argmax(cw["w_scale"]))
    assert np.array_equal(tw["wq"][row], cw["wq"][row])                              # on the row that sets Delta the two quantizers coincide
    # rows that are sign flips and copies of one row have equal maxima: tensor-wise == channel-wise everywhere
    W2 = np.stack([W[0], W[0] ^ np.uint16(0x8000), W[0]])
    a, b = oracle.prepare_weights(W2, c, None, bits, tensorwise=True), oracle.prepare_weights(W2, c, None, bits)
    assert np.array_equal(a["wq"], b["wq"]) and np.array_equal(a["w_scale"], b["w_scale"])
