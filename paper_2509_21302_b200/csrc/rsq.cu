// Rotate -> smooth -> 4-bit quantize (Sec. 3.2: pre-global rotation, post-local smooth, Eq. "quantization").
//
// One row of K bf16 values is transformed by the un-normalised Sylvester-Hadamard matrix with fp32
// radix-2 butterflies in ascending-stride order (strides 1, 2, 4, ..., K/2), multiplied by a
// per-rotated-channel factor, and quantized to signed 4-bit codes with one scale per row or per
// 128 rotated channels.  The logical stage order and the rounding of every operation are fixed
// (explicit round-to-nearest intrinsics, no FMA contraction), so codes and scales are reproducible
// bit for bit; only the mapping of elements to lanes, registers and shared memory is free.
//
// The same kernel serves the activations (multiplier amul) and the weight rows (multiplier wmul).
#include "qvggt_internal.cuh"
#include "sm100_ptx.cuh"
#include "tensor_map.cuh"
#include "unpack_w4.cuh"

namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ int padded(int i) { return i + (i >> 5); }

// Five butterfly stages over the 32 values a thread holds; register bit b is stride 2^b.
__device__ __forceinline__ void butterfly32(float (&r)[32])
{
#pragma unroll
    for (int h = 1; h < 32; h <<= 1) {
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            if (!(i & h)) {
                float a = r[i], b = r[i + h];
                r[i] = __fadd_rn(a, b);
                r[i + h] = __fsub_rn(a, b);
            }
        }
    }
}

template <int K>
struct RowGeom {
    static constexpr int T = K / 32;             // threads per row
    static constexpr int ROWS = kThreads / T;    // rows per CTA pass
    static constexpr int PADDED = K + K / 32;    // floats of shared memory per row
};

__device__ __forceinline__ void row_sync(int T, int slot)
{
    if (T == 32) {
        __syncwarp();
    } else {
        asm volatile("bar.sync %0, %1;" ::"r"(slot + 1), "r"(T) : "memory");
    }
}

// Loads row `x` (bf16, K values), leaves the transformed row in shared memory `s` (padded fp32),
// element i at s[padded(i)], already multiplied by mul[i] if mul != nullptr.
template <int K>
__device__ __forceinline__ void rotate_row_to_smem(const uint16_t *x, const float *mul, float *s, int t, int slot)
{
    constexpr int T = RowGeom<K>::T;
    float r[32];
    // strides 1..16: thread t holds elements 32t .. 32t+31
    {
        const uint4 *src = reinterpret_cast<const uint4 *>(x + t * 32);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            uint4 w = __ldg(src + q);
            uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                r[q * 8 + 2 * e] = __uint_as_float(ww[e] << 16);
                r[q * 8 + 2 * e + 1] = __uint_as_float(ww[e] & 0xFFFF0000u);
            }
        }
    }
    butterfly32(r);
#pragma unroll
    for (int j = 0; j < 32; ++j) s[padded(t * 32 + j)] = r[j];
    row_sync(T, slot);
    // strides 32..512: thread holds elements base + 32 j
    const int base = (t >> 5) * 1024 + (t & 31);
#pragma unroll
    for (int j = 0; j < 32; ++j) r[j] = s[padded(base + 32 * j)];
    butterfly32(r);
    if (K == 1024) {
        if (mul) {
#pragma unroll
            for (int j = 0; j < 32; ++j) r[j] = __fmul_rn(r[j], __ldg(mul + base + 32 * j));
        }
#pragma unroll
        for (int j = 0; j < 32; ++j) s[padded(base + 32 * j)] = r[j];
        row_sync(T, slot);
    } else {
#pragma unroll
        for (int j = 0; j < 32; ++j) s[padded(base + 32 * j)] = r[j];
        row_sync(T, slot);
        // strides 1024, 2048: thread holds elements 8t + e + 1024 q  (register 4e + q)
#pragma unroll
        for (int e = 0; e < 8; ++e)
#pragma unroll
            for (int q = 0; q < 4; ++q) r[4 * e + q] = s[padded(8 * t + e + 1024 * q)];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            float a0 = r[4 * e], a1 = r[4 * e + 1], a2 = r[4 * e + 2], a3 = r[4 * e + 3];
            float b0 = __fadd_rn(a0, a1), b1 = __fsub_rn(a0, a1);   // stride 1024
            float b2 = __fadd_rn(a2, a3), b3 = __fsub_rn(a2, a3);
            r[4 * e] = __fadd_rn(b0, b2);                            // stride 2048
            r[4 * e + 2] = __fsub_rn(b0, b2);
            r[4 * e + 1] = __fadd_rn(b1, b3);
            r[4 * e + 3] = __fsub_rn(b1, b3);
        }
        if (mul) {
#pragma unroll
            for (int e = 0; e < 8; ++e)
#pragma unroll
                for (int q = 0; q < 4; ++q) r[4 * e + q] = __fmul_rn(r[4 * e + q], __ldg(mul + 8 * t + e + 1024 * q));
        }
#pragma unroll
        for (int e = 0; e < 8; ++e)
#pragma unroll
            for (int q = 0; q < 4; ++q) s[padded(8 * t + e + 1024 * q)] = r[4 * e + q];
        row_sync(T, slot);
    }
}

// (a0, a1) <- (a0 + b0, a1 + b1), (b0, b1) <- (a0 - b0, a1 - b1): two butterflies per instruction pair
__device__ __forceinline__ void bfly2(float &a0, float &a1, float &b0, float &b1)
{
    const uint64_t A = ptx::f32x2_pack(a0, a1), B = ptx::f32x2_pack(b0, b1);
    ptx::f32x2_unpack(ptx::f32x2_add(A, B), a0, a1);
    ptx::f32x2_unpack(ptx::f32x2_sub(A, B), b0, b1);
}

// ------------------------------------------------------------------------------------------------
// K = T * T (T = 32: one warp per row; T = 64: two warps per row), T values per thread, a single
// transpose.  The bf16 row is staged in shared memory with 16-byte asynchronous copies (coalesced
// in global memory, double-buffered), so that thread t can start from the T contiguous elements
// T t .. T t + T - 1:
//   strides 1 .. T/2      in registers (element T t + j, bits of j)
//   T x T transpose through shared memory (16-byte chunk c of row r kept at chunk c XOR (r mod 8))
//   strides T .. T*T/2    in registers (thread t' holds elements T t + t', bits of t)
// The codes of thread t' then belong to elements T t + t': eight neighbouring lanes exchange
// nibbles with three shuffle steps so that every lane ends up with whole 32-bit output words.
__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gmem_src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(ptx::smem_addr(smem_dst)), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

template <int LOGT>
struct SqGeom {
    static constexpr int T = 1 << LOGT;              // threads per row = values per thread
    static constexpr int K = T * T;
    static constexpr int CTA_THREADS = 128;
    static constexpr int ROWS = CTA_THREADS / T;     // rows in flight per CTA
    static constexpr int CH = T / 8;                 // 16-byte pieces of bf16 per thread
    static constexpr int STAGE_BYTES = 2 * K;        // one bf16 row
    static constexpr int ROW_SMEM = 2 * STAGE_BYTES + 4 * K + 256;  // two stages, fp32 transpose tile, 2 x 32 reduction words
    static constexpr int SMEM = ROWS * ROW_SMEM;
};

// Resident CTAs per SM the kernel is built for: 4 (K = 1024) or 3 (K = 4096); with the fused LayerNorm at K = 4096 the
// CTA's shared-memory copy of gamma and beta (32 KB) leaves room for 2.
constexpr int sq_ctas_per_sm(int logt, int ln) { return logt == 5 ? 4 : ((ln == 1 || ln == 2) ? 2 : 3); }

template <int T>
__device__ __forceinline__ void group_sync(int slot)
{
    if (T == 32) __syncwarp();
    else asm volatile("bar.sync %0, %1;" ::"r"(slot + 1), "r"(T) : "memory");
}

// In-register stages over n values: the first joins neighbours (scalar: packing it costs more register
// moves than it saves), the others pair (k, k + 1).
template <int N, bool FIRST = true>
__device__ __forceinline__ void stages_in_registers(float (&v)[N])
{
    if (FIRST) {
#pragma unroll
        for (int k = 0; k < N; k += 2) {
            const float a = v[k], b = v[k + 1];
            v[k] = __fadd_rn(a, b);
            v[k + 1] = __fsub_rn(a, b);
        }
    }
#pragma unroll
    for (int h = 2; h < N; h <<= 1)
#pragma unroll
        for (int k = 0; k < N; k += 2)
            if (!(k & h)) bfly2(v[k], v[k + 1], v[k + h], v[k + 1 + h]);
}

// Pairwise sum of N registers: adjacent pairs, recursively (the tree of the LayerNorm statistics).
template <int N>
__device__ __forceinline__ float tree_sum(const float (&a)[N])
{
    if constexpr (N == 1) {
        return a[0];
    } else {
        float b[N / 2];
#pragma unroll
        for (int i = 0; i < N / 2; ++i) b[i] = __fadd_rn(a[2 * i], a[2 * i + 1]);
        return tree_sum<N / 2>(b);
    }
}

// GELU x Phi(x) (the activation between the two linears of the MLP: the producer of fc2's input), evaluated so that the
// negative tail keeps its RELATIVE accuracy.  With t = |x|, z = t / sqrt(2):
//   Q(t) = 1 - Phi(t) = exp(-z^2) E(z) / 2,   E(z) = exp(z^2) erfc(z)  (smooth, from 1 down to ~1 / (z sqrt(pi))),
//   E(z) ~ s P(s),  s = 1 / (1 + 0.55 z),  P a degree-4 polynomial (own weighted least-squares fit on z in [0, 9.6]: relative
//   error below 6e-5), then gelu(x) = x - x Q for x >= 0 and x Q for x < 0.
// About 16 instructions, two of them special-function (reciprocal, exp2); relative error ~1e-4 wherever the result is a
// normal number above 2^-120, i.e. at most one bf16 ulp after rounding; below that (x < -12.9) the exponential
// flushes to zero.  The fused multiply-adds are written explicitly (the file is compiled without contraction).
__device__ __forceinline__ float gelu_f32(float x)
{
    const float z = __fmul_rn(fabsf(x), 0.70710678f);
    float s;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(s) : "f"(__fmaf_rn(0.55f, z, 1.0f)));
    float p = -0.17450283f;
    p = __fmaf_rn(p, s, 0.33387650f);
    p = __fmaf_rn(p, s, 0.21415194f);
    p = __fmaf_rn(p, s, 0.31633197f);
    p = __fmaf_rn(p, s, 0.31008677f);
    float e;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(__fmul_rn(__fmul_rn(z, z), -1.44269504f)));
    const float q = __fmul_rn(__fmul_rn(0.5f, e), __fmul_rn(s, p));
    return x >= 0.0f ? __fmaf_rn(-x, q, x) : __fmul_rn(x, q);
}

// Parameters of the LayerNorm that may run in front of the rotation (gamma == nullptr: none).
struct LnArgs {
    const float *gamma, *beta;   // fp32 [K]
    float eps;
    uint16_t *out;               // LN == 2 / 4 only: bf16 [M, K], the normalized / activated rows (nothing else is computed)
};

// C8: one code per byte (int8, natural element order, row pitch K) instead of two per byte.
// QMAX: largest code magnitude, 2^(N-1) - 1 of Eq. "quantization": 7 (N = 4) or, with C8 only, 127 (N = 8).
// STATIC (C8 only): one given step size *static_delta for the whole tensor (the static tensor-wise arm of the
// granularity ablation) instead of one per row from the row's absolute maximum; the clamp of Eq. "quantization"
// to [-QMAX - 1, QMAX] is then active, and every row's scale is written as that step size.
// LN (the operation fused in front of the rotation): 3 = GELU on every element, rounded to bf16 as a separate activation
// kernel would store it; 4 = only that, written out.  1 = every row goes through LayerNorm first (fp32, statistics summed pairwise: in-thread tree over the thread's
// T contiguous elements, then the xor-shuffle tree over the row's threads -- together the halves-recursion over the
// row), its output rounded to bf16 as a separate normalization kernel would store it; 2 = only that, written out.
template <int LOGT, int GROUP, bool C8 = false, int QMAX = 7, bool STATIC = false, int LN = 0>
__global__ void __launch_bounds__(SqGeom<LOGT>::CTA_THREADS, sq_ctas_per_sm(LOGT, LN))
rsq_sq_kernel(const uint16_t *__restrict__ X, long long ldx, int M, const float *__restrict__ mul,
              unsigned char *__restrict__ Xq, float *__restrict__ scales, const float *__restrict__ static_delta,
              const LnArgs ln, const QvggtExpand ex)
{
    static_assert(!STATIC || (C8 && GROUP == 0), "the static step size is built for one code per byte");
    static_assert(LN == 0 || (C8 && GROUP == 0 && !STATIC), "the fused LayerNorm is built for the dynamic one-code-per-byte path");
    using G = SqGeom<LOGT>;
    constexpr int T = G::T, K = G::K, CH = G::CH;
    constexpr int NG = (GROUP == 128) ? K / 128 : 1;           // scale groups per row
    constexpr int GREGS = (GROUP == 128) ? 128 / T : T;        // consecutive registers of one thread in the same group
    extern __shared__ __align__(16) unsigned char dsm[];
    const int slot = threadIdx.x / T, t = threadIdx.x % T, lane = threadIdx.x & 31;
    unsigned char *stage = dsm + slot * G::ROW_SMEM;
    float *Tm = reinterpret_cast<float *>(stage + 2 * G::STAGE_BYTES);
    float *red = Tm + K;                                       // cross-warp maxima (T = 64 only)

    // staging copy: 16-byte piece cg = t + T j belongs to thread cg / CH, piece cg % CH of its T values
    uint32_t cp_dst[CH];
#pragma unroll
    for (int j = 0; j < CH; ++j) {
        const int cg = t + T * j, to = cg / CH, c = cg % CH;
        const int sw = (T == 32) ? ((to >> 1) & 3) : (to & 7);
        cp_dst[j] = to * (2 * T) + ((c ^ sw) << 4);
    }
    const int my_sw = (T == 32) ? ((t >> 1) & 3) : (t & 7);
    // nibble exchange between the 8 lanes that share (t / 8): per step d the lane keeps half of its nibbles
    uint32_t nb_send[3], nb_keep[3], nb_rot[3];
#pragma unroll
    for (int i = 0; i < 3; ++i) {
        const uint32_t m0 = (i == 0) ? 0x0F0F0F0Fu : (i == 1) ? 0x00FF00FFu : 0x0000FFFFu;   // nibble index bit clear
        const bool up = (lane >> i) & 1;
        nb_send[i] = up ? m0 : ~m0;
        nb_keep[i] = up ? ~m0 : m0;
        nb_rot[i] = up ? (4u << i) : 32u - (4u << i);
    }

    const long long stride = (long long)gridDim.x * G::ROWS;
    long long row = (long long)blockIdx.x * G::ROWS + slot;
    // the blocks may have become resident before the previous kernel in the stream finished (programmatic
    // dependent launch): no global memory is touched before that kernel is done
    ptx::grid_launch_dependents();
    ptx::grid_dependency_wait();
    if (row < M) {
        const unsigned char *src = reinterpret_cast<const unsigned char *>(X + row * ldx);
#pragma unroll
        for (int j = 0; j < CH; ++j) cp_async16(stage + cp_dst[j], src + 16 * (t + T * j));
    }
    cp_async_commit();
    // Handles that keep the weights at half a byte per code: while the first row's copies are in flight, every block
    // expands its share of the layer's packed weight codes into the scratch that the GEMM behind this launch reads.
    if constexpr (C8 && GROUP == 0 && !STATIC && QMAX == 7) {
        for (long long i = (long long)blockIdx.x * G::CTA_THREADS + threadIdx.x; i < ex.n16; i += (long long)gridDim.x * G::CTA_THREADS)
            qvggt_unpack_w4_item(ex.packed, ex.out, i);
    }
    const float delta = STATIC ? __ldg(static_delta) : 0.0f;
    // LayerNorm parameters: one copy per CTA in shared memory behind the row slots, as 16-byte pieces ordered
    // [piece][thread], so that thread t reads its T contiguous gammas with conflict-free 16-byte loads (read straight
    // from global memory, thread t's T contiguous values are 4 T bytes away from its neighbour's: 32 sectors per load)
    constexpr bool LN_SMEM = (LN == 1 || LN == 2);
    float4 *g_sm = reinterpret_cast<float4 *>(dsm + G::SMEM), *b_sm = g_sm + K / 4;
    if constexpr (LN_SMEM) {
        for (int i = threadIdx.x; i < K / 4; i += G::CTA_THREADS) {
            const int dst = (i % (T / 4)) * T + i / (T / 4);
            g_sm[dst] = __ldg(reinterpret_cast<const float4 *>(ln.gamma) + i);
            b_sm[dst] = __ldg(reinterpret_cast<const float4 *>(ln.beta) + i);
        }
        __syncthreads();
    }
    float m[T];                                                // multipliers of elements T k + t (loaded behind the first row's copies)
#pragma unroll
    for (int k = 0; k < T; ++k) m[k] = (LN == 2 || LN == 4) ? 0.0f : __ldg(mul + T * k + t);   // the prologue alone uses none
    int buf = 0;
    for (; row < M; row += stride, buf ^= 1) {
        const long long next = row + stride;
        if (next < M) {
            const unsigned char *src = reinterpret_cast<const unsigned char *>(X + next * ldx);
#pragma unroll
            for (int j = 0; j < CH; ++j) cp_async16(stage + (buf ^ 1) * G::STAGE_BYTES + cp_dst[j], src + 16 * (t + T * j));
        }
        cp_async_commit();
        cp_async_wait<1>();                 // this row's copies (mine) have landed; the barrier covers the others'
        group_sync<T>(slot);
        float v[T];
        {
            const unsigned char *mine = stage + buf * G::STAGE_BYTES + t * (2 * T);
#pragma unroll
            for (int c = 0; c < CH; ++c) {
                const uint4 w4 = *reinterpret_cast<const uint4 *>(mine + ((c ^ my_sw) << 4));
                const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (LN) {                               // plain conversion: the normalization comes first
                        v[8 * c + 2 * j] = __uint_as_float(w[j] << 16);
                        v[8 * c + 2 * j + 1] = __uint_as_float(w[j] & 0xFFFF0000u);
                        continue;
                    }
                    // a 32-bit word holds elements 2i (low half) and 2i + 1 of the row: the first stage joins exactly
                    // these two, and the mixed-precision add takes the bf16 half as it is (its conversion is exact,
                    // so this is fl(float(lo) + float(hi)) and fl(float(lo) - float(hi)), one rounding each)
                    const float hi = __uint_as_float(w[j] & 0xFFFF0000u);
                    const unsigned short lo = static_cast<unsigned short>(w[j]);
                    asm("add.rn.f32.bf16 %0, %1, %2;" : "=f"(v[8 * c + 2 * j]) : "h"(lo), "f"(hi));
                    asm("sub.rn.f32.bf16 %0, %1, %2;" : "=f"(v[8 * c + 2 * j + 1]) : "h"(lo), "f"(hi));
                }
            }
        }
        if constexpr (LN == 3 || LN == 4) {
            uint32_t packed[T / 2];
#pragma unroll
            for (int k = 0; k < T; k += 2) {
                const uint32_t p01 = ptx::pack_bf16x2(gelu_f32(v[k]), gelu_f32(v[k + 1]));   // what an activation kernel would store
                v[k] = __uint_as_float(p01 << 16);
                v[k + 1] = __uint_as_float(p01 & 0xFFFF0000u);
                packed[k / 2] = p01;
            }
            if constexpr (LN == 4) {
                uint4 *dst = reinterpret_cast<uint4 *>(ln.out + row * K + T * t);
#pragma unroll
                for (int k = 0; k < T / 8; ++k) dst[k] = make_uint4(packed[4 * k], packed[4 * k + 1], packed[4 * k + 2], packed[4 * k + 3]);
                // every thread of the row has read its share of this stage before any of them starts the copy that will
                // overwrite it (the next iteration's prefetch goes into this buffer; the other paths meet further down)
                group_sync<T>(slot);
                continue;
            }
            stages_in_registers<T, true>(v);    // strides 1 .. T/2
        } else if constexpr (LN != 0) {
            // row sum over the tree: registers, lanes, and (T = 64) the two warps of the row
            auto row_sum = [&](float part, int word) {
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) part = __fadd_rn(part, __shfl_xor_sync(0xFFFFFFFFu, part, o));
                if (T == 64) {
                    if (lane == 0) red[word + (t >> 5)] = part;
                    group_sync<T>(slot);
                    part = __fadd_rn(red[word], red[word + 1]);
                }
                return part;
            };
            constexpr float inv_k = 1.0f / K;                      // a power of two: the divisions are exact
            const float mean = __fmul_rn(row_sum(tree_sum<T>(v), 8), inv_k);
            // two elements per instruction where no multiply feeds an add (the bias add stays scalar: a packed multiply
            // in front of a packed add was seen contracted into one fused operation)
            const uint64_t mean2 = ptx::f32x2_pack(mean, mean);
            uint64_t d2[T / 2];
            float sq[T];
#pragma unroll
            for (int k = 0; k < T; k += 2) {
                d2[k / 2] = ptx::f32x2_sub(ptx::f32x2_pack(v[k], v[k + 1]), mean2);
                ptx::f32x2_unpack(ptx::f32x2_mul(d2[k / 2], d2[k / 2]), sq[k], sq[k + 1]);
            }
            const float var = __fmul_rn(row_sum(tree_sum<T>(sq), 10), inv_k);
            const float rstd = __fdiv_rn(1.0f, __fsqrt_rn(__fadd_rn(var, ln.eps)));
            const uint64_t rstd2 = ptx::f32x2_pack(rstd, rstd);
            uint32_t packed[T / 2];
#pragma unroll
            for (int k = 0; k < T; k += 4) {
                const float4 g = g_sm[(k / 4) * T + t], b = b_sm[(k / 4) * T + t];
                float n0, n1, n2, n3;
                ptx::f32x2_unpack(ptx::f32x2_mul(ptx::f32x2_mul(d2[k / 2], rstd2), ptx::f32x2_pack(g.x, g.y)), n0, n1);
                ptx::f32x2_unpack(ptx::f32x2_mul(ptx::f32x2_mul(d2[k / 2 + 1], rstd2), ptx::f32x2_pack(g.z, g.w)), n2, n3);
                // bf16 pair, round to nearest even: what a separate normalization kernel would have stored
                const uint32_t p01 = ptx::pack_bf16x2(__fadd_rn(n0, b.x), __fadd_rn(n1, b.y));
                const uint32_t p23 = ptx::pack_bf16x2(__fadd_rn(n2, b.z), __fadd_rn(n3, b.w));
                v[k] = __uint_as_float(p01 << 16);
                v[k + 1] = __uint_as_float(p01 & 0xFFFF0000u);
                v[k + 2] = __uint_as_float(p23 << 16);
                v[k + 3] = __uint_as_float(p23 & 0xFFFF0000u);
                if (LN == 2) {
                    packed[k / 2] = p01;
                    packed[k / 2 + 1] = p23;
                }
            }
            if constexpr (LN == 2) {
                uint4 *dst = reinterpret_cast<uint4 *>(ln.out + row * K + T * t);
#pragma unroll
                for (int k = 0; k < T / 8; ++k) dst[k] = make_uint4(packed[4 * k], packed[4 * k + 1], packed[4 * k + 2], packed[4 * k + 3]);
                continue;                       // (the row sums above already made the row's threads meet after their reads of the stage)
            }
            stages_in_registers<T, true>(v);    // strides 1 .. T/2
        } else {
            stages_in_registers<T, false>(v);   // strides 2 .. T/2 (stride 1 was taken with the conversion)
        }
#pragma unroll
        for (int j = 0; j < T; ++j) Tm[j * T + ((((t >> 2) ^ (j & 7)) << 2) | (t & 3))] = v[j];
        group_sync<T>(slot);
#pragma unroll
        for (int g = 0; g < T / 4; ++g) {
            const float4 f = *reinterpret_cast<const float4 *>(Tm + t * T + ((g ^ (t & 7)) << 2));
            v[4 * g] = f.x; v[4 * g + 1] = f.y; v[4 * g + 2] = f.z; v[4 * g + 3] = f.w;
        }
        stages_in_registers<T>(v);          // strides T .. K/2: v[k] is element T k + t
#pragma unroll
        for (int k = 0; k < T; k += 2) {
            const uint64_t y = ptx::f32x2_mul(ptx::f32x2_pack(v[k], v[k + 1]), ptx::f32x2_pack(m[k], m[k + 1]));
            ptx::f32x2_unpack(y, v[k], v[k + 1]);
        }
        // absolute maxima: one per row, or one per 128 consecutive elements (GREGS registers of every thread).  Non-negative
        // floats order like their bit patterns, so the warp-wide maximum is one integer reduction (redux.sync) per value.
        float am[NG];          // GROUP == 0: the row's maximum; GROUP == 128: overwritten below by qmax / maximum of every group
#pragma unroll
        for (int g = 0; g < (STATIC ? 0 : NG); ++g) {
            float a = fmaxf(fabsf(v[g * GREGS]), fabsf(v[g * GREGS + 1]));
#pragma unroll
            for (int k = 2; k < GREGS; k += 2)     // max(|a|, |x|, |y|) in one instruction
                asm("max.abs.f32 %0, %1, %2, %3;" : "=f"(a) : "f"(a), "f"(v[g * GREGS + k]), "f"(v[g * GREGS + k + 1]));
            am[g] = __uint_as_float(__reduce_max_sync(0xFFFFFFFFu, __float_as_uint(a)));
        }
        if constexpr (GROUP == 128) {
            // One lane per group finishes it: floor, the two divisions (scale = max / qmax is stored from here, 128 bytes
            // per row in one piece; qmax / max goes back to every thread), instead of NG divisions in every thread.
            float mine;                                        // the maximum of group `lane mod NG`
            if constexpr (T == 64) {
                static_assert(NG == 32, "one group per lane");
                if (lane == 0) {
#pragma unroll
                    for (int g = 0; g < NG; g += 4)
                        *reinterpret_cast<float4 *>(red + (t >> 5) * NG + g) = make_float4(am[g], am[g + 1], am[g + 2], am[g + 3]);
                }
                group_sync<T>(slot);
                mine = fmaxf(red[lane], red[NG + lane]);       // both warps of the row compute all 32 (no second exchange)
            } else {
                static_assert(NG == 8, "eight groups per row");
                mine = am[0];
#pragma unroll
                for (int g = 1; g < NG; ++g) mine = ((lane & (NG - 1)) == g) ? am[g] : mine;
            }
            mine = fmaxf(mine, 1e-8f);
            const float inv_mine = __fdiv_rn(static_cast<float>(QMAX), mine);
            if (t < NG) scales[row * NG + t] = __fdiv_rn(mine, static_cast<float>(QMAX));
#pragma unroll
            for (int g = 0; g < NG; ++g) am[g] = __shfl_sync(0xFFFFFFFFu, inv_mine, g);
        } else if (T == 64 && !STATIC) {
            if (lane == 0) red[t >> 5] = am[0];
            group_sync<T>(slot);
            am[0] = fmaxf(red[0], red[1]);
        }
        if constexpr (GROUP == 0 && !STATIC) {
            // One division sequence yields both quotients: thread 1 of the row divides the other way round and stores the
            // scale max / qmax; every other lane gets qmax / max, which thread 1 then takes from lane 0.
            const float amax = fmaxf(am[0], 1e-8f);
            const bool scale_lane = (t == 1);
            const float r = __fdiv_rn(scale_lane ? amax : static_cast<float>(QMAX), scale_lane ? static_cast<float>(QMAX) : amax);
            if (scale_lane) scales[row] = r;
            am[0] = __shfl_sync(0xFFFFFFFFu, r, 0);            // am[0] = qmax / maximum from here on
        }
        if constexpr (C8) {
            static_assert(QMAX == 7 || QMAX == 127, "4-bit or 8-bit codes");
            float inv;
            if (STATIC) {
                inv = __fdiv_rn(1.0f, delta);
            } else {
                inv = am[0];                                    // qmax / maximum (GROUP == 128: replaced per group below)
            }
            uint64_t inv2 = ptx::f32x2_pack(inv, inv), inv2b = inv2;
            const uint64_t magic2 = ptx::f32x2_pack(12582912.0f, 12582912.0f);
            // byte exchange between the 4 lanes that share (t / 4): a 4 x 4 byte transpose in two steps
            const uint32_t sel0 = (lane & 1) ? 0x3715u : 0x6240u, sel1 = (lane & 2) ? 0x3276u : 0x5410u;
#pragma unroll
            for (int kk = 0; kk < T / 4; ++kk) {
                if constexpr (GROUP == 128) {
                    // registers 4 kk .. 4 kk + 3 lie in one scale group (T = 32: GREGS = 4) or in two (T = 64: GREGS = 2)
                    const int g0 = (4 * kk) / GREGS, g1 = (4 * kk + 2) / GREGS;   // compile-time after unrolling
                    inv2 = ptx::f32x2_pack(am[g0], am[g0]);                        // am[] holds qmax / maximum here
                    inv2b = ptx::f32x2_pack(am[g1], am[g1]);
                }
                // exact product + 1.5*2^23, rounded once (half-to-even): the low mantissa byte is the int8 code
                float f0, f1, f2, f3;
                ptx::f32x2_unpack(ptx::f32x2_fma(ptx::f32x2_pack(v[4 * kk], v[4 * kk + 1]), inv2, magic2), f0, f1);
                ptx::f32x2_unpack(ptx::f32x2_fma(ptx::f32x2_pack(v[4 * kk + 2], v[4 * kk + 3]), inv2b, magic2), f2, f3);
                if (STATIC) {
                    // The clamp of Eq. "quantization", taken on the sum with the magic number: inside +-2^22 that sum is
                    // 1.5 * 2^23 + q exactly; beyond, the fused operation still returns the correctly rounded (huge) sum,
                    // which the clamp saturates all the same.  The low mantissa byte stays the two's-complement code.
                    constexpr float lo = 12582912.0f - (QMAX + 1), hi = 12582912.0f + QMAX;
                    f0 = fminf(fmaxf(f0, lo), hi); f1 = fminf(fmaxf(f1, lo), hi);
                    f2 = fminf(fmaxf(f2, lo), hi); f3 = fminf(fmaxf(f3, lo), hi);
                }
                // byte n = code of element T (4 kk + n) + t
                uint32_t x = __byte_perm(__byte_perm(__float_as_uint(f0), __float_as_uint(f1), 0x0040),
                                         __byte_perm(__float_as_uint(f2), __float_as_uint(f3), 0x0040), 0x5410);
                x = __byte_perm(x, __shfl_xor_sync(0xFFFFFFFFu, x, 1), sel0);
                x = __byte_perm(x, __shfl_xor_sync(0xFFFFFFFFu, x, 2), sel1);
                // now byte n = code of element T (4 kk + e) + 4 (t / 4) + n, e = t mod 4: one whole output word
                *reinterpret_cast<uint32_t *>(Xq + row * K + T * (4 * kk + (t & 3)) + 4 * (t >> 2)) = x;
            }
        } else {
        static_assert(C8 || QMAX == 7, "two codes per byte hold 4-bit codes only");
        uint32_t word[T / 8];
#pragma unroll
        for (int g = 0; g < NG; ++g) {
            const float inv = am[g];                            // qmax / maximum of the row or of the group
            const uint64_t inv2 = ptx::f32x2_pack(inv, inv), magic2 = ptx::f32x2_pack(12582912.0f, 12582912.0f);
#pragma unroll
            for (int k = g * GREGS; k < (g + 1) * GREGS; k += 2) {
                // exact product + 1.5*2^23, rounded once (half-to-even): low mantissa bits = two's-complement code
                float f0, f1;
                ptx::f32x2_unpack(ptx::f32x2_fma(ptx::f32x2_pack(v[k], v[k + 1]), inv2, magic2), f0, f1);
                uint32_t w = (k & 7) ? word[k >> 3] : 0u;
                w = __funnelshift_r(w, __float_as_uint(f0), 4);        // shift the low nibble in from the top
                word[k >> 3] = __funnelshift_r(w, __float_as_uint(f1), 4);
            }
        }
        // word[kk] holds the codes of elements T (8 kk + n) + t in nibble n; after the exchange it holds the
        // codes of elements T (8 kk + e) + 8 (t / 8) + n, e = t mod 8: one whole output word
#pragma unroll
        for (int kk = 0; kk < T / 8; ++kk) {
            uint32_t x = word[kk];
#pragma unroll
            for (int i = 0; i < 3; ++i) {
                const uint32_t send = __funnelshift_l(x & nb_send[i], x & nb_send[i], nb_rot[i]);
                x = (x & nb_keep[i]) | __shfl_xor_sync(0xFFFFFFFFu, send, 1 << i);
            }
            *reinterpret_cast<uint32_t *>(Xq + row * (K / 2) + 4 * ((T / 8) * (8 * kk + (t & 7)) + (t >> 3))) = x;
        }
        }
        if (STATIC && t == 0) scales[row] = delta;
    }
}

// Column-wise absolute maximum of the normalised rotated rows (calibration statistics for Eq. "smooth_factor").
template <int K>
__global__ void __launch_bounds__(kThreads)
colmax_kernel(const uint16_t *__restrict__ X, int M, float *__restrict__ colmax)
{
    using G = RowGeom<K>;
    __shared__ float smem[G::ROWS * G::PADDED];
    const int slot = threadIdx.x / G::T;
    const int t = threadIdx.x % G::T;
    float *s = smem + slot * G::PADDED;
    const float nrm = (K == 1024) ? 0.03125f : 0.015625f;
    float best[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) best[j] = 0.0f;
    for (long long m0 = (long long)blockIdx.x * G::ROWS; m0 < M; m0 += (long long)gridDim.x * G::ROWS) {
        const long long m = m0 + slot;
        if (m < M) {
            rotate_row_to_smem<K>(X + m * (long long)K, nullptr, s, t, slot);
#pragma unroll
            for (int j = 0; j < 32; ++j) best[j] = fmaxf(best[j], fabsf(s[padded(t * 32 + j)]));
        }
        if (G::T == 32) __syncwarp(); else __syncthreads();
    }
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        // non-negative floats order like their bit patterns
        atomicMax(reinterpret_cast<int *>(colmax) + t * 32 + j, __float_as_int(__fmul_rn(best[j], nrm)));
    }
}

__global__ void multipliers_kernel(const float *__restrict__ c, const signed char *__restrict__ v, int K,
                                   float *__restrict__ amul, float *__restrict__ wmul)
{
    int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= K) return;
    const float nrm = (K == 1024) ? 0.03125f : 0.015625f;   // K^{-1/2}, exact
    const float sgn = (v != nullptr && v[k] < 0) ? -nrm : nrm;
    if (amul) amul[k] = __fdiv_rn(sgn, c[k]);
    if (wmul) wmul[k] = __fmul_rn(sgn, c[k]);
}

// out[0] = max_i in[i] (one block; the values are non-negative scales)
__global__ void __launch_bounds__(1024) max_reduce_kernel(const float *__restrict__ in, int n, float *__restrict__ out)
{
    __shared__ float part[32];
    float m = 0.0f;
    for (int i = threadIdx.x; i < n; i += blockDim.x) m = fmaxf(m, in[i]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = m;
    __syncthreads();
    if (threadIdx.x < 32) {
        m = part[threadIdx.x];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
        if (threadIdx.x == 0) out[0] = m;
    }
}

__global__ void smooth_finalize_kernel(const float *__restrict__ ax, const float *__restrict__ aw, int K, float alpha,
                                       float lo, float hi, float *__restrict__ c)
{
    int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= K) return;
    float x = ax[k], w = aw[k], r;
    if (x == 0.0f && w == 0.0f) r = 1.0f;
    else r = powf(x, alpha) / powf(w, 1.0f - alpha);
    if (!(r >= lo)) r = lo;
    if (r > hi) r = hi;
    c[k] = r;
}

int rsq_grid(int M, int rows_per_cta, int ctas_per_sm = 6)
{
    int sms = qvggt_sm_count();
    if (sms < 1) sms = 148;
    long long need = ((long long)M + rows_per_cta - 1) / rows_per_cta;
    long long cap = (long long)sms * ctas_per_sm;
    return (int)(need < cap ? need : cap);
}

}  // namespace

cudaError_t qvggt_launch_multipliers(const float *c, const signed char *v, int K, float *amul, float *wmul,
                                     cudaStream_t st)
{
    multipliers_kernel<<<(K + 255) / 256, 256, 0, st>>>(c, v, K, amul, wmul);
    return cudaGetLastError();
}

namespace {

// Launch with programmatic stream serialization allowed: the blocks may become resident while the previous
// kernel of the stream drains (they wait in grid_dependency_wait() before touching global memory).
template <int LOGT, int GROUP, bool C8, int QMAX = 7, bool STATIC = false, int LN = 0>
cudaError_t launch_sq(const uint16_t *x, long long ldx, int M, const float *mul, unsigned char *out, float *scales,
                      cudaStream_t st, const float *static_delta = nullptr, LnArgs ln = LnArgs{nullptr, nullptr, 0.0f, nullptr},
                      QvggtExpand ex = QvggtExpand{nullptr, nullptr, 0})
{
    using G = SqGeom<LOGT>;
    constexpr int SMEM = G::SMEM + ((LN == 1 || LN == 2) ? 2 * G::K * 4 : 0);   // + the CTA's copy of gamma and beta
    static QvggtPerDevice configured;     // per device and instantiation
    const int dev = qvggt_current_device();
    if (dev < 0) return cudaErrorInvalidDevice;
    if (!configured.v[dev].load(std::memory_order_acquire)) {
        cudaError_t e = cudaFuncSetAttribute(rsq_sq_kernel<LOGT, GROUP, C8, QMAX, STATIC, LN>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
        if (e != cudaSuccess) return e;
        configured.v[dev].store(1, std::memory_order_release);
    }
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    int grid = rsq_grid(M, G::ROWS, sq_ctas_per_sm(LOGT, LN));
    if (ex.n16 > 0) {
        // enough blocks for the expansion even when there are few rows (blocks without rows only expand)
        const long long want = (ex.n16 + G::CTA_THREADS - 1) / G::CTA_THREADS;
        const int cap = rsq_grid(1 << 30, G::ROWS, sq_ctas_per_sm(LOGT, LN));
        const int need = (int)(want < cap ? want : cap);
        if (grid < need) grid = need;
    }
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(G::CTA_THREADS);
    cfg.dynamicSmemBytes = SMEM;
    cfg.stream = st;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, rsq_sq_kernel<LOGT, GROUP, C8, QMAX, STATIC, LN>, x, ldx, M, mul, out, scales, static_delta, ln, ex);
}

}  // namespace

cudaError_t qvggt_launch_rsq_c8(const void *X, long long ldx, int M, int K, const float *mul, int bits, signed char *Xq8,
                                float *scales, cudaStream_t st, int group, const void *w_packed, void *w_expanded, long long w_codes)
{
    if (M == 0) return cudaSuccess;
    const uint16_t *x = static_cast<const uint16_t *>(X);
    unsigned char *out = reinterpret_cast<unsigned char *>(Xq8);
    if (w_packed) {
        // the same launch also expands w_codes packed weight codes (4-bit, token-wise activations only)
        if (group != 0 || bits != 4) return cudaErrorNotSupported;
        const QvggtExpand ex{static_cast<const uint4 *>(w_packed), static_cast<uint4 *>(w_expanded), w_codes / 32};
        const LnArgs none{nullptr, nullptr, 0.0f, nullptr};
        return K == 1024 ? launch_sq<5, 0, true>(x, ldx, M, mul, out, scales, st, nullptr, none, ex)
                         : launch_sq<6, 0, true>(x, ldx, M, mul, out, scales, st, nullptr, none, ex);
    }
    if (group == 128) {
        if (bits != 4) return cudaErrorNotSupported;
        return K == 1024 ? launch_sq<5, 128, true>(x, ldx, M, mul, out, scales, st) : launch_sq<6, 128, true>(x, ldx, M, mul, out, scales, st);
    }
    if (bits == 8)
        return K == 1024 ? launch_sq<5, 0, true, 127>(x, ldx, M, mul, out, scales, st) : launch_sq<6, 0, true, 127>(x, ldx, M, mul, out, scales, st);
    return K == 1024 ? launch_sq<5, 0, true>(x, ldx, M, mul, out, scales, st) : launch_sq<6, 0, true>(x, ldx, M, mul, out, scales, st);
}

cudaError_t qvggt_launch_rsq_static_c8(const void *X, long long ldx, int M, int K, const float *mul, int bits, const float *delta,
                                       signed char *Xq8, float *scales, cudaStream_t st)
{
    if (M == 0) return cudaSuccess;
    const uint16_t *x = static_cast<const uint16_t *>(X);
    unsigned char *out = reinterpret_cast<unsigned char *>(Xq8);
    if (bits == 8)
        return K == 1024 ? launch_sq<5, 0, true, 127, true>(x, ldx, M, mul, out, scales, st, delta)
                         : launch_sq<6, 0, true, 127, true>(x, ldx, M, mul, out, scales, st, delta);
    return K == 1024 ? launch_sq<5, 0, true, 7, true>(x, ldx, M, mul, out, scales, st, delta)
                     : launch_sq<6, 0, true, 7, true>(x, ldx, M, mul, out, scales, st, delta);
}

cudaError_t qvggt_launch_ln_rsq_c8(const void *X, long long ldx, int M, int K, const float *mul, int bits, const float *gamma,
                                   const float *beta, float eps, signed char *Xq8, float *scales, void *ln_out, cudaStream_t st)
{
    if (M == 0) return cudaSuccess;
    const uint16_t *x = static_cast<const uint16_t *>(X);
    unsigned char *out = reinterpret_cast<unsigned char *>(Xq8);
    const LnArgs ln = {gamma, beta, eps, static_cast<uint16_t *>(ln_out)};
    if (ln_out)       // the normalization alone
        return K == 1024 ? launch_sq<5, 0, true, 7, false, 2>(x, ldx, M, mul, out, scales, st, nullptr, ln)
                         : launch_sq<6, 0, true, 7, false, 2>(x, ldx, M, mul, out, scales, st, nullptr, ln);
    if (bits == 8)
        return K == 1024 ? launch_sq<5, 0, true, 127, false, 1>(x, ldx, M, mul, out, scales, st, nullptr, ln)
                         : launch_sq<6, 0, true, 127, false, 1>(x, ldx, M, mul, out, scales, st, nullptr, ln);
    return K == 1024 ? launch_sq<5, 0, true, 7, false, 1>(x, ldx, M, mul, out, scales, st, nullptr, ln)
                     : launch_sq<6, 0, true, 7, false, 1>(x, ldx, M, mul, out, scales, st, nullptr, ln);
}

cudaError_t qvggt_launch_gelu_rsq_c8(const void *X, long long ldx, int M, int K, const float *mul, int bits, signed char *Xq8,
                                     float *scales, void *gelu_out, cudaStream_t st)
{
    if (M == 0) return cudaSuccess;
    const uint16_t *x = static_cast<const uint16_t *>(X);
    unsigned char *out = reinterpret_cast<unsigned char *>(Xq8);
    const LnArgs ln = {nullptr, nullptr, 0.0f, static_cast<uint16_t *>(gelu_out)};
    if (gelu_out)     // the activation alone
        return K == 1024 ? launch_sq<5, 0, true, 7, false, 4>(x, ldx, M, mul, out, scales, st, nullptr, ln)
                         : launch_sq<6, 0, true, 7, false, 4>(x, ldx, M, mul, out, scales, st, nullptr, ln);
    if (bits == 8)
        return K == 1024 ? launch_sq<5, 0, true, 127, false, 3>(x, ldx, M, mul, out, scales, st, nullptr, ln)
                         : launch_sq<6, 0, true, 127, false, 3>(x, ldx, M, mul, out, scales, st, nullptr, ln);
    return K == 1024 ? launch_sq<5, 0, true, 7, false, 3>(x, ldx, M, mul, out, scales, st, nullptr, ln)
                     : launch_sq<6, 0, true, 7, false, 3>(x, ldx, M, mul, out, scales, st, nullptr, ln);
}

cudaError_t qvggt_launch_rsq(const void *X, long long ldx, int M, int K, const float *mul, int group,
                             unsigned char *Xq, float *scales, cudaStream_t st)
{
    if (M == 0) return cudaSuccess;
    const uint16_t *x = static_cast<const uint16_t *>(X);
    if (K == 1024)
        return group == 128 ? launch_sq<5, 128, false>(x, ldx, M, mul, Xq, scales, st) : launch_sq<5, 0, false>(x, ldx, M, mul, Xq, scales, st);
    return group == 128 ? launch_sq<6, 128, false>(x, ldx, M, mul, Xq, scales, st) : launch_sq<6, 0, false>(x, ldx, M, mul, Xq, scales, st);
}

cudaError_t qvggt_launch_max_reduce(const float *in, int n, float *out, cudaStream_t st)
{
    max_reduce_kernel<<<1, 1024, 0, st>>>(in, n, out);
    return cudaGetLastError();
}

cudaError_t qvggt_launch_colmax(const void *X, int M, int K, float *colmax, cudaStream_t st)
{
    if (M == 0) return cudaSuccess;
    const uint16_t *x = static_cast<const uint16_t *>(X);
    if (K == 1024) colmax_kernel<1024><<<rsq_grid(M, RowGeom<1024>::ROWS), kThreads, 0, st>>>(x, M, colmax);
    else colmax_kernel<4096><<<rsq_grid(M, RowGeom<4096>::ROWS), kThreads, 0, st>>>(x, M, colmax);
    return cudaGetLastError();
}

cudaError_t qvggt_launch_smooth_finalize(const float *ax, const float *aw, int K, float alpha, float lo, float hi,
                                         float *c, cudaStream_t st)
{
    smooth_finalize_kernel<<<(K + 255) / 256, 256, 0, st>>>(ax, aw, K, alpha, lo, hi, c);
    return cudaGetLastError();
}
