// Rotate -> smooth -> quantize with the bulk of the Hadamard transform on the tensor core (Sec. 3.2, Pre-Global-Rotation:
// H_{2^n} = H_2 (x) H_{2^(n-1)}, so the transform factors over any split of the index bits).
//
// Element index k of a row of K = 1024 is split as k = 8 j + c (j: bits 3..9, c: bits 0..2); for K = 4096 as
// k = 1024 a + 8 j + c (a: bits 10..11).  The 7 bits of j are transformed by ONE product with the 128 x 128 matrix
// H_128[j'][j] = (-1)^popcount(j' & j) on the tensor core:
//     D[j'][n] = sum_j H_128[j'][j] * x_n[j],          n = (token, a, c): one column per (token, a, c)
// with bf16 operands (the inputs are bf16, +-1 is exact, so every product is exact) and fp32 accumulation in tensor
// memory.  The remaining 3 (K = 1024) or 5 (K = 4096) bits are fp32 butterflies in registers: TMEM lane j' of a
// thread holds, in consecutive columns, exactly the 8 (32) values of one token that those butterflies join.  Then
// multiplier, per-token absolute maximum, Eq. "quantization" as in the exact kernel (rsq.cu).
//
// The accumulation order inside the tensor core is not the ascending-stride butterfly order of the exact kernel, so
// this kernel does NOT reproduce that kernel's codes bit for bit: it is held to a tolerance against the rotation
// without intermediate rounding (see qvggt_rotate_smooth_quantize_tc in include/qvggt.h).  The exact kernel stays the
// default.
//
// No data is reshuffled for the tensor core: a token row lands in shared memory as it is in global memory (TMA, no
// swizzle), and is read as an MN-major B operand whose 16-byte units are the 8 consecutive elements (c = 0..7) of one j.
// Persistent, one CTA per SM:
//   warps 0..15 epilogue (TMEM lane quarter w % 4, column group w / 4 of 64 columns): TMEM -> registers, butterflies,
//               multiplier, absolute maximum (warp reduction + exchange through shared memory: a token spans all 128
//               lanes), quantize, pack, coalesced global stores (thread j' owns 8 consecutive codes of a token)
//   warp 16     one thread issues the 8 tcgen05.mma (K = 16 each) of a tile and the commits
//   warp 17     one thread issues the TMA loads (4 boxes of 16 KB per 64 KB stage)
// The epilogue is latency-bound, not issue-bound (two barriers and a division sit on every tile's critical path), hence
// the 16 warps: four per scheduler, each with 64 live values.
#include <cuda.h>

#include "qvggt_internal.cuh"
#include "sm100_ptx.cuh"
#include "tensor_map.cuh"

namespace {

constexpr int EPI_WARPS = 16;
constexpr int MMA_WARP = EPI_WARPS, TMA_WARP = EPI_WARPS + 1;
constexpr int THREADS = (EPI_WARPS + 2) * 32;
constexpr int NCOL = 256;                         // columns of one tile = (token, a, c) triples
constexpr int STAGE = NCOL / 8 * 2048;            // 32 pieces of 1024 bf16: 64 KB
constexpr int ACC_BUFS = 2;
constexpr int H_BYTES = 128 * 128 * 2;            // the bf16 matrix H_128
constexpr int OFF_H = 0;
constexpr int OFF_STAGE = OFF_H + H_BYTES;

// Shared-memory layout behind H_128: K = 1024 has three 64 KB stages and keeps a thread's 8 multipliers in registers;
// K = 4096 has two stages (the loads still run up to four tiles ahead of the epilogue: two stages plus two
// accumulators) and a 16 KB copy of the multipliers, [register r][lane j], that every epilogue thread reads per token.
template <int PIECES>
struct Lay {
    static constexpr int STAGES = (PIECES == 1) ? 3 : 2;
    static constexpr int OFF_MUL = OFF_STAGE + STAGES * STAGE;
    static constexpr int OFF_BAR = OFF_MUL + ((PIECES == 1) ? 0 : 32 * 128 * 4);       // full[STAGES] empty[STAGES] tfull[2] tempty[2]
    static constexpr int NBARS = 2 * STAGES + 2 * ACC_BUFS;
    static constexpr int OFF_TMEM = OFF_BAR + NBARS * 8;
    static constexpr int OFF_ABORT = OFF_TMEM + 4;
    static constexpr int OFF_EXCH = (OFF_ABORT + 4 + 15) & ~15;     // [2 tile parities][4 column groups][8 tokens][4 lane quarters] partial maxima
    static constexpr int SMEM_BYTES = OFF_EXCH + 2 * 4 * 8 * 4 * 4;
    static constexpr int DYN_SMEM = SMEM_BYTES + 128;               // slack to align the base to 128 bytes
    static_assert(DYN_SMEM <= 232448, "exceeds the 227 KB of shared memory a CTA may use");
};

// H_128 as the K-major A operand, no swizzle: core matrix (8 rows m) x (8 elements k) = 128 contiguous bytes;
// core matrices that are neighbours along k are 128 bytes apart, 8-row groups 2048 bytes.
constexpr uint32_t A_K_STRIDE = 128, A_MN_STRIDE = 2048;
// A stage as the MN-major B operand: a 16-byte unit = elements 8 j .. 8 j + 7 of one piece (8 columns n); the
// units of j, j + 1, ... follow each other (a core matrix = 8 consecutive j = 128 contiguous bytes); within a
// 256-element box the next 8 j are 128 bytes on and the next piece (the next 8 columns) 512 bytes.
constexpr uint32_t B_K_STRIDE = 128, B_MN_STRIDE = 512;
constexpr int BOX_ELEMS = 256, BOX_BYTES = NCOL / 8 * BOX_ELEMS * 2;      // 16 KB: 32 pieces x 256 elements

__device__ __forceinline__ void bfly(float &a, float &b)
{
    const float s = __fadd_rn(a, b), d = __fsub_rn(a, b);
    a = s;
    b = d;
}

// (a0, a1) <- (a0 + b0, a1 + b1), (b0, b1) <- (a0 - b0, a1 - b1)
__device__ __forceinline__ void bfly2(float &a0, float &a1, float &b0, float &b1)
{
    const uint64_t A = ptx::f32x2_pack(a0, a1), B = ptx::f32x2_pack(b0, b1);
    ptx::f32x2_unpack(ptx::f32x2_add(A, B), a0, a1);
    ptx::f32x2_unpack(ptx::f32x2_sub(A, B), b0, b1);
}

// Butterflies over the register index bits of n values (n = 8: strides 1, 2, 4; n = 32: strides 1 .. 16).
template <int N>
__device__ __forceinline__ void stages_over_registers(float *v)
{
#pragma unroll
    for (int i = 0; i < N; i += 2) bfly(v[i], v[i + 1]);
#pragma unroll
    for (int h = 2; h < N; h <<= 1)
#pragma unroll
        for (int i = 0; i < N; i += 2)
            if (!(i & h)) bfly2(v[i], v[i + 1], v[i + h], v[i + h + 1]);
}

// LOGK: 10 or 12.  C8: one code per byte instead of two.  QMAX: 7, or 127 with C8.  DUMP: also write the rotated,
// smoothed rows (fp32 [M, K]) to y_debug.
template <int LOGK, bool C8, int QMAX, bool DUMP>
__global__ void __launch_bounds__(THREADS, 1)
rsq_tc_kernel(const __grid_constant__ CUtensorMap map_x, int M, const float *__restrict__ mul, unsigned char *__restrict__ Xq,
              float *__restrict__ scales, float *__restrict__ y_debug, int *status)
{
    static_assert(LOGK == 10 || LOGK == 12, "K = 1024 or 4096");
    static_assert(C8 || QMAX == 7, "two codes per byte hold 4-bit codes only");
    constexpr int K = 1 << LOGK;
    constexpr int PIECES = K / 1024;                 // 1024-element pieces per token (the index bits above bit 9)
    constexpr int VPT = 8 * PIECES;                  // values of one token in one thread: 8 or 32
    constexpr int TOK_TILE = NCOL / VPT;             // tokens per tile: 32 or 8
    constexpr int TOK_G = 64 / VPT;                  // tokens per column group of 64 columns: 8 or 2
    using L = Lay<PIECES>;
    constexpr int STAGES = L::STAGES;
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
    const uint32_t sbase = ptx::smem_addr(smem);
    const uint32_t bar_full = sbase + L::OFF_BAR;
    const uint32_t bar_empty = bar_full + STAGES * 8;
    const uint32_t bar_tfull = bar_empty + STAGES * 8;
    const uint32_t bar_tempty = bar_tfull + ACC_BUFS * 8;
    uint32_t *s_tmem = reinterpret_cast<uint32_t *>(smem + L::OFF_TMEM);
    volatile int *s_abort = reinterpret_cast<volatile int *>(smem + L::OFF_ABORT);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tiles = (M + TOK_TILE - 1) / TOK_TILE;
    const int my_tiles = (tiles > (int)blockIdx.x) ? (tiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;

    // H_128 in shared memory, 16 bytes (row m, 8 consecutive k) at a time
    for (int u = threadIdx.x; u < 128 * 16; u += THREADS) {
        const int m = u >> 4, kc = u & 15;
        uint32_t w[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const uint32_t lo = (__popc(m & (8 * kc + 2 * e)) & 1) ? 0xBF80u : 0x3F80u;
            const uint32_t hi = (__popc(m & (8 * kc + 2 * e + 1)) & 1) ? 0xBF80u : 0x3F80u;
            w[e] = lo | (hi << 16);
        }
        *reinterpret_cast<uint4 *>(smem + OFF_H + (m >> 3) * A_MN_STRIDE + kc * A_K_STRIDE + (m & 7) * 16) = make_uint4(w[0], w[1], w[2], w[3]);
    }
    if (PIECES > 1) {
        // multiplier of element 1024 a + 8 j + c -> slot [8 a + c][j]
        float *m_s = reinterpret_cast<float *>(smem + L::OFF_MUL);
        for (int e = threadIdx.x; e < K; e += THREADS) m_s[(((e >> 10) << 3) | (e & 7)) * 128 + ((e >> 3) & 127)] = __ldg(mul + e);
    }
    ptx::fence_proxy_async_smem();            // generic-proxy writes -> visible to the tensor core's reads
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(bar_full + 8 * s, 1);         // the producer's arrive.expect_tx
            ptx::mbar_init(bar_empty + 8 * s, 1);        // tcgen05.commit
        }
        for (int b = 0; b < ACC_BUFS; ++b) {
            ptx::mbar_init(bar_tfull + 8 * b, 1);        // tcgen05.commit
            ptx::mbar_init(bar_tempty + 8 * b, EPI_WARPS);
        }
        *s_abort = 0;
        ptx::fence_mbar_init();
    }
    if (warp == MMA_WARP) { ptx::tmem_alloc(ptx::smem_addr(s_tmem), ACC_BUFS * NCOL); ptx::tmem_relinquish(); }
    if (warp == TMA_WARP && lane == 0) ptx::prefetch_tensormap(&map_x);
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *s_tmem;
    // the set-up above touched no global memory: it may overlap the tail of the previous kernel in the stream
    ptx::grid_launch_dependents();
    ptx::grid_dependency_wait();

    if (warp < EPI_WARPS) {
        // ------------------------------------------------------------ epilogue
        const int quarter = warp & 3, cg = warp >> 2;
        const int j = quarter * 32 + lane;                       // TMEM lane = transformed index bits 3..9
        float *exch = reinterpret_cast<float *>(smem + L::OFF_EXCH) + cg * 32;    // [parity][group][token][quarter]
        const float *m_s = reinterpret_cast<const float *>(smem + L::OFF_MUL) + j;
        // multipliers of this thread's elements: register 8 a + c <-> element 1024 a + 8 j + c.  K = 1024 keeps them in
        // registers; K = 4096 re-reads them per token from shared memory: 32 more live registers would spill.
        float m[8];
        if (PIECES == 1) {
            const float4 lo = __ldg(reinterpret_cast<const float4 *>(mul + 8 * j));
            const float4 hi = __ldg(reinterpret_cast<const float4 *>(mul + 8 * j + 4));
            m[0] = lo.x; m[1] = lo.y; m[2] = lo.z; m[3] = lo.w; m[4] = hi.x; m[5] = hi.y; m[6] = hi.z; m[7] = hi.w;
        }
        bool alive = true;
        // The loop is NOT left when a wait expires: the four warps of a column group meet at a hardware barrier in
        // every tile, so a warp whose wait gave up keeps taking part (its remaining waits return at once, the abort
        // flag being set; what it computes is discarded by the caller, who finds the expiry in *status).
        for (int t = 0; t < my_tiles; ++t) {
            const int tile = blockIdx.x + t * gridDim.x;
            const int b = t & 1;
            const long long row0 = (long long)tile * TOK_TILE + cg * TOK_G;         // first token of this warp's column group
            {   // lane 0 polls, the warp follows
                int ok = 1;
                if (lane == 0) ok = (alive && ptx::mbar_wait(bar_tfull + 8 * b, (t >> 1) & 1, s_abort, status, QVGGT_DEV_TIMEOUT_ACCUM, 32)) ? 1 : 0;
                alive = __shfl_sync(0xFFFFFFFFu, ok, 0) != 0;
            }
            ptx::tc_fence_after_sync();
            // the warp's 32 lanes x 64 columns of the accumulator -> registers; tensor memory is handed back at once
            uint32_t raw[2][32];
#pragma unroll
            for (int c = 0; c < 2; ++c)
                ptx::tmem_ld_32x32(tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + b * NCOL + cg * 64 + c * 32, raw[c]);
            ptx::tmem_ld_wait();
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(bar_tempty + 8 * b);
            float *v = reinterpret_cast<float *>(&raw[0][0]);   // v[VPT * i + r]: token i of the group, register r
            // remaining index bits in registers, multiplier, per-token maximum of this warp's 32 lanes
            uint32_t mine = 0;                                   // lane i keeps the warp's maximum of token i
#pragma unroll
            for (int i = 0; i < TOK_G; ++i) {
                float *y = v + VPT * i;
                stages_over_registers<VPT>(y);
#pragma unroll
                for (int a = 0; a < PIECES; ++a) {
                    if (PIECES > 1) {
#pragma unroll
                        for (int r = 0; r < 8; ++r) m[r] = m_s[(8 * a + r) * 128];
                    }
#pragma unroll
                    for (int r = 0; r < 8; r += 2) {
                        const uint64_t p = ptx::f32x2_mul(ptx::f32x2_pack(y[8 * a + r], y[8 * a + r + 1]), ptx::f32x2_pack(m[r], m[r + 1]));
                        ptx::f32x2_unpack(p, y[8 * a + r], y[8 * a + r + 1]);
                    }
                }
                float am = fmaxf(fabsf(y[0]), fabsf(y[1]));
#pragma unroll
                for (int r = 2; r < VPT; r += 2) asm("max.abs.f32 %0, %1, %2, %3;" : "=f"(am) : "f"(am), "f"(y[r]), "f"(y[r + 1]));
                // non-negative floats order like their bit patterns: one integer warp reduction
                const uint32_t wm = __reduce_max_sync(0xFFFFFFFFu, __float_as_uint(am));
                if (lane == i) mine = wm;
                if (DUMP && y_debug && alive && row0 + i < M) {
#pragma unroll
                    for (int a = 0; a < PIECES; ++a) {
                        float4 *d = reinterpret_cast<float4 *>(y_debug + (row0 + i) * K + 1024 * a + 8 * j);
                        d[0] = make_float4(y[8 * a], y[8 * a + 1], y[8 * a + 2], y[8 * a + 3]);
                        d[1] = make_float4(y[8 * a + 4], y[8 * a + 5], y[8 * a + 6], y[8 * a + 7]);
                    }
                }
            }
            // the four warps of the column group exchange their maxima (buffers alternate with the tile parity: a warp may
            // already write the next tile's maxima while a slower one still reads this tile's)
            float *ex = exch + b * 128;
            if (lane < TOK_G) ex[lane * 4 + quarter] = __uint_as_float(mine);
            asm volatile("bar.sync %0, %1;" ::"r"(1 + cg), "r"(128) : "memory");
            // lanes 0 .. TOK_G-1 compute qmax / max of their token, lanes TOK_G .. 2 TOK_G-1 the scale max / qmax of the same tokens:
            // one division sequence for both quotients
            float inv_mine = 0.0f;
            if (lane < 2 * TOK_G) {
                const int tok = lane & (TOK_G - 1);
                const bool scale_lane = lane >= TOK_G;
                const float4 q4 = *reinterpret_cast<const float4 *>(ex + tok * 4);
                const float amax = fmaxf(fmaxf(fmaxf(q4.x, q4.y), fmaxf(q4.z, q4.w)), 1e-8f);
                inv_mine = __fdiv_rn(scale_lane ? amax : static_cast<float>(QMAX), scale_lane ? static_cast<float>(QMAX) : amax);
                if (scale_lane && alive && quarter == 0 && row0 + tok < M) scales[row0 + tok] = inv_mine;
            }
            const uint64_t magic2 = ptx::f32x2_pack(12582912.0f, 12582912.0f);
#pragma unroll
            for (int i = 0; i < TOK_G; ++i) {
                const float *y = v + VPT * i;
                const float inv = __shfl_sync(0xFFFFFFFFu, inv_mine, i);
                const uint64_t inv2 = ptx::f32x2_pack(inv, inv);
                const bool row_ok = alive && row0 + i < M;   // nothing is stored after an expired wait
#pragma unroll
                for (int a = 0; a < PIECES; ++a) {
                    // exact product + 1.5 * 2^23, rounded once (half-to-even): the low mantissa bits are the code
                    float f[8];
#pragma unroll
                    for (int r = 0; r < 8; r += 2)
                        ptx::f32x2_unpack(ptx::f32x2_fma(ptx::f32x2_pack(y[8 * a + r], y[8 * a + r + 1]), inv2, magic2), f[r], f[r + 1]);
                    if (C8) {
                        const uint32_t w0 = __byte_perm(__byte_perm(__float_as_uint(f[0]), __float_as_uint(f[1]), 0x0040),
                                                        __byte_perm(__float_as_uint(f[2]), __float_as_uint(f[3]), 0x0040), 0x5410);
                        const uint32_t w1 = __byte_perm(__byte_perm(__float_as_uint(f[4]), __float_as_uint(f[5]), 0x0040),
                                                        __byte_perm(__float_as_uint(f[6]), __float_as_uint(f[7]), 0x0040), 0x5410);
                        if (row_ok) *reinterpret_cast<uint2 *>(Xq + (row0 + i) * K + 1024 * a + 8 * j) = make_uint2(w0, w1);
                    } else {
                        uint32_t w = 0;
#pragma unroll
                        for (int r = 0; r < 8; ++r) w = __funnelshift_r(w, __float_as_uint(f[r]), 4);   // nibble r = code of element r
                        if (row_ok) *reinterpret_cast<uint32_t *>(Xq + (row0 + i) * (K / 2) + 512 * a + 4 * j) = w;
                    }
                }
            }
        }
    } else if (warp == MMA_WARP) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = ptx::idesc_bf16_f32(128, NCOL, true);
            bool alive = true;
            int s = 0;
            uint32_t ph = 0;
            for (int t = 0; t < my_tiles && alive; ++t) {
                const int b = t & 1;
                if (t >= ACC_BUFS) {
                    alive = ptx::mbar_wait(bar_tempty + 8 * b, ((t >> 1) - 1) & 1, s_abort, status, QVGGT_DEV_TIMEOUT_TMEM_FREE);
                    if (!alive) break;
                }
                alive = ptx::mbar_wait(bar_full + 8 * s, ph, s_abort, status, QVGGT_DEV_TIMEOUT_FULL);
                if (!alive) break;
                ptx::tc_fence_after_sync();
                const uint32_t stage = sbase + OFF_STAGE + s * STAGE;
#pragma unroll
                for (int i = 0; i < 8; ++i) {          // K-slice i: j = 16 i .. 16 i + 15
                    const uint64_t a_desc = ptx::smem_desc_noswizzle(sbase + OFF_H + i * 2 * A_K_STRIDE, A_K_STRIDE, A_MN_STRIDE);
                    const uint64_t b_desc = ptx::smem_desc_noswizzle(stage + (i >> 1) * BOX_BYTES + (i & 1) * 2 * B_K_STRIDE, B_K_STRIDE, B_MN_STRIDE);
                    ptx::mma_bf16_ss(tmem_base + b * NCOL, a_desc, b_desc, idesc, i != 0);
                }
                ptx::mma_commit(bar_empty + 8 * s);
                ptx::mma_commit(bar_tfull + 8 * b);
                if (++s == STAGES) { s = 0; ph ^= 1; }
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            bool alive = true;
            int s = 0;
            uint32_t ph = 0;
            for (int t = 0; t < my_tiles && alive; ++t) {
                const int tile = blockIdx.x + t * gridDim.x;
                if (t >= STAGES) {
                    alive = ptx::mbar_wait(bar_empty + 8 * s, ph ^ 1, s_abort, status, QVGGT_DEV_TIMEOUT_EMPTY, 20);
                    if (!alive) break;
                }
                const uint32_t dst = sbase + OFF_STAGE + s * STAGE;
                ptx::mbar_arrive_expect_tx(bar_full + 8 * s, STAGE);
#pragma unroll
                for (int qd = 0; qd < 4; ++qd) {       // elements 256 qd .. 256 qd + 255 of every piece of the tile's tokens
                    if (PIECES == 1) ptx::tma_load_2d(&map_x, bar_full + 8 * s, dst + qd * BOX_BYTES, qd * BOX_ELEMS, tile * TOK_TILE);
                    else ptx::tma_load_3d(&map_x, bar_full + 8 * s, dst + qd * BOX_BYTES, qd * BOX_ELEMS, 0, tile * TOK_TILE);
                }
                if (++s == STAGES) { s = 0; ph ^= 1; }
            }
        }
        __syncwarp();
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == MMA_WARP) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, ACC_BUFS * NCOL);
    }
}

template <int LOGK, bool C8, int QMAX, bool DUMP>
cudaError_t launch(const uint16_t *x, long long ldx, int M, const float *mul, unsigned char *out, float *scales, float *y_debug,
                   int *status, cudaStream_t st)
{
    constexpr int K = 1 << LOGK, PIECES = K / 1024, TOK_TILE = NCOL / (8 * PIECES);
    static QvggtPerDevice configured;
    const int dev = qvggt_current_device();
    if (dev < 0) return cudaErrorInvalidDevice;
    if (!configured.v[dev].load(std::memory_order_acquire)) {
        cudaError_t e = cudaFuncSetAttribute(rsq_tc_kernel<LOGK, C8, QMAX, DUMP>, cudaFuncAttributeMaxDynamicSharedMemorySize, Lay<PIECES>::DYN_SMEM);
        if (e != cudaSuccess) return e;
        configured.v[dev].store(1, std::memory_order_release);
    }
    CUtensorMap map_x;
    const bool ok = (PIECES == 1)
        ? qvggt_make_map(&map_x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, x, K, M, (uint64_t)ldx * 2, BOX_ELEMS, TOK_TILE, CU_TENSOR_MAP_SWIZZLE_NONE)
        : qvggt_make_map3(&map_x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, x, 1024, PIECES, M, 2048, (uint64_t)ldx * 2, BOX_ELEMS, PIECES, TOK_TILE);
    if (!ok) return cudaErrorInvalidValue;
    const int tiles = (M + TOK_TILE - 1) / TOK_TILE, sms = qvggt_sm_count();
    if (sms < 1) return cudaErrorInvalidDevice;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(tiles < sms ? tiles : sms);
    cfg.blockDim = dim3(THREADS);
    cfg.dynamicSmemBytes = Lay<PIECES>::DYN_SMEM;
    cfg.stream = st;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, rsq_tc_kernel<LOGK, C8, QMAX, DUMP>, map_x, M, mul, out, scales, y_debug, status);
}

template <bool C8, int QMAX>
cudaError_t dispatch(const uint16_t *x, long long ldx, int M, int K, const float *mul, unsigned char *out, float *scales,
                     float *y_debug, int *status, cudaStream_t st)
{
    if (K == 1024)
        return y_debug ? launch<10, C8, QMAX, true>(x, ldx, M, mul, out, scales, y_debug, status, st)
                       : launch<10, C8, QMAX, false>(x, ldx, M, mul, out, scales, y_debug, status, st);
    return y_debug ? launch<12, C8, QMAX, true>(x, ldx, M, mul, out, scales, y_debug, status, st)
                   : launch<12, C8, QMAX, false>(x, ldx, M, mul, out, scales, y_debug, status, st);
}

}  // namespace

cudaError_t qvggt_launch_rsq_tc(const void *X, long long ldx, int M, int K, const float *mul, int bits, bool c8, void *Xq,
                                float *scales, float *y_debug, int *status, cudaStream_t st)
{
    if (M == 0) return cudaSuccess;
    const uint16_t *x = static_cast<const uint16_t *>(X);
    unsigned char *out = static_cast<unsigned char *>(Xq);
    if (!c8) return dispatch<false, 7>(x, ldx, M, K, mul, out, scales, y_debug, status, st);
    if (bits == 8) return dispatch<true, 127>(x, ldx, M, K, mul, out, scales, y_debug, status, st);
    return dispatch<true, 7>(x, ldx, M, K, mul, out, scales, y_debug, status, st);
}
