// W4A4 GEMM + rescale + bias + bf16 for sm_100a (Sec. 3.2: integer sum over the inner dimension,
// per-token and per-out-channel scales applied outside the sum).
//
// tcgen05 has no 4-bit integer kind, so the codes are fed to kind::i8.  Converter warps read the
// packed codes straight from global memory (L2), expand every nibble into the HIGH half of a byte
// (value 16*q, no sign extension needed) and write the int8 operand tiles into shared memory in
// the 128-byte-swizzled K-major layout the tensor core reads.  The raw accumulator is therefore
// 256 * sum(q_x q_w) (at most 2^26 in magnitude), shifted back exactly in the epilogue.  Even and
// odd codes of a 32-code slice land in separate 16-byte chunks; the same permutation of K is
// applied to both operands, so the dot product is unchanged.
#include <cuda_bf16.h>

#include "qvggt_internal.cuh"
#include "sm100_ptx.cuh"

namespace {

constexpr int BM = 128;           // tokens per CTA tile (TMEM lanes)
constexpr int BK = 128;           // codes along K per pipeline stage = one 128-byte swizzled row of int8
constexpr int STAGES = 4;
constexpr int CONV_WARPS = 8;
constexpr int CONV_THREADS = CONV_WARPS * 32;
constexpr int MMA_WARP = CONV_WARPS;
constexpr int THREADS = CONV_THREADS + 32;

template <int BN>
struct Tile {
    static constexpr int A_BYTES = BM * 128;
    static constexpr int B_BYTES = BN * 128;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int CHUNKS = (BM + BN) * 4 / CONV_THREADS;   // 16-byte packed pieces per thread per stage
    static constexpr int OFF_WSCALE = STAGES * STAGE_BYTES;
    static constexpr int OFF_BIAS = OFF_WSCALE + BN * 4;
    static constexpr int OFF_BAR = OFF_BIAS + BN * 4;             // full[STAGES], empty[STAGES], accum
    static constexpr int OFF_TMEM = OFF_BAR + (2 * STAGES + 1) * 8;
    static constexpr int OFF_ABORT = OFF_TMEM + 4;
    static constexpr int BYTES = OFF_ABORT + 4;
    static constexpr int DYN_SMEM = BYTES + 1024;                 // slack to align the base to 1024 bytes
};

__device__ __forceinline__ float bf16_bits_to_f32(uint16_t b) { return __uint_as_float(static_cast<uint32_t>(b) << 16); }

template <int BN>
__global__ void __launch_bounds__(THREADS, 1)
gemm_w4a4_kernel(const unsigned char *__restrict__ Xq, const unsigned char *__restrict__ Wq,
                 const float *__restrict__ a_scale, const float *__restrict__ w_scale,
                 const uint16_t *__restrict__ bias, uint16_t *__restrict__ Y, long long ldy,
                 int *__restrict__ acc_debug, int M, int N, int K, int *status)
{
    using T = Tile<BN>;
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = ptx::smem_addr(smem);
    float *s_wscale = reinterpret_cast<float *>(smem + T::OFF_WSCALE);
    float *s_bias = reinterpret_cast<float *>(smem + T::OFF_BIAS);
    const uint32_t bar_full = sbase + T::OFF_BAR;
    const uint32_t bar_empty = bar_full + STAGES * 8;
    const uint32_t bar_accum = bar_empty + STAGES * 8;
    uint32_t *s_tmem = reinterpret_cast<uint32_t *>(smem + T::OFF_TMEM);
    volatile int *s_abort = reinterpret_cast<volatile int *>(smem + T::OFF_ABORT);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m0 = blockIdx.x * BM, n0 = blockIdx.y * BN;
    const int KB = K / BK;
    const int row_bytes = K / 2;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(bar_full + 8 * s, CONV_THREADS);
            ptx::mbar_init(bar_empty + 8 * s, 1);
        }
        ptx::mbar_init(bar_accum, 1);
        *s_abort = 0;
        ptx::fence_mbar_init();
    }
    if (warp == MMA_WARP) {
        ptx::tmem_alloc(ptx::smem_addr(s_tmem), BN);
        ptx::tmem_relinquish();
    }
    for (int i = threadIdx.x; i < BN; i += THREADS) {
        s_wscale[i] = w_scale[n0 + i];
        s_bias[i] = bias ? bf16_bits_to_f32(bias[n0 + i]) : 0.0f;
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *s_tmem;

    if (warp < CONV_WARPS) {
        // ------------------------------------------------------------ converters
        const unsigned char *gptr[T::CHUNKS];
        uint32_t soff[T::CHUNKS];
#pragma unroll
        for (int i = 0; i < T::CHUNKS; ++i) {
            const int c = threadIdx.x + CONV_THREADS * i;
            const int row = c >> 2, piece = c & 3;
            if (row < BM) {
                const int gm = m0 + row;
                gptr[i] = (gm < M) ? Xq + (long long)gm * row_bytes + piece * 16 : nullptr;
                soff[i] = row * 128;
            } else {
                const int r = row - BM;
                gptr[i] = Wq + (long long)(n0 + r) * row_bytes + piece * 16;
                soff[i] = T::A_BYTES + r * 128;
            }
            // even codes -> 16-byte chunk 2*piece, odd codes -> chunk 2*piece+1, both XOR (row mod 8)
            soff[i] += ((2 * piece) ^ (row & 7)) << 4;
        }
        uint4 cur[T::CHUNKS], nxt[T::CHUNKS];
#pragma unroll
        for (int i = 0; i < T::CHUNKS; ++i) cur[i] = gptr[i] ? __ldg(reinterpret_cast<const uint4 *>(gptr[i])) : make_uint4(0, 0, 0, 0);

        bool alive = true;
        for (int kb = 0; kb < KB && alive; ++kb) {
            if (kb + 1 < KB) {
#pragma unroll
                for (int i = 0; i < T::CHUNKS; ++i)
                    nxt[i] = gptr[i] ? __ldg(reinterpret_cast<const uint4 *>(gptr[i] + (kb + 1) * (BK / 2))) : make_uint4(0, 0, 0, 0);
            }
            const int s = kb % STAGES;
            if (kb >= STAGES) alive = ptx::mbar_wait(bar_empty + 8 * s, ((kb / STAGES) - 1) & 1, s_abort, status, QVGGT_DEV_TIMEOUT_EMPTY);
            if (!alive) break;
            unsigned char *stage = smem + s * T::STAGE_BYTES;
#pragma unroll
            for (int i = 0; i < T::CHUNKS; ++i) {
                const uint4 w = cur[i];
                uint4 lo, hi;
                lo.x = (w.x << 4) & 0xF0F0F0F0u; hi.x = w.x & 0xF0F0F0F0u;
                lo.y = (w.y << 4) & 0xF0F0F0F0u; hi.y = w.y & 0xF0F0F0F0u;
                lo.z = (w.z << 4) & 0xF0F0F0F0u; hi.z = w.z & 0xF0F0F0F0u;
                lo.w = (w.w << 4) & 0xF0F0F0F0u; hi.w = w.w & 0xF0F0F0F0u;
                *reinterpret_cast<uint4 *>(stage + soff[i]) = lo;
                *reinterpret_cast<uint4 *>(stage + (soff[i] ^ 16)) = hi;
            }
            ptx::fence_proxy_async_smem();
            ptx::mbar_arrive(bar_full + 8 * s);
#pragma unroll
            for (int i = 0; i < T::CHUNKS; ++i) cur[i] = nxt[i];
        }

        // ------------------------------------------------------------ epilogue (same warps)
        if (alive) alive = ptx::mbar_wait(bar_accum, 0, s_abort, status, QVGGT_DEV_TIMEOUT_ACCUM);
        ptx::tc_fence_after_sync();
        if (alive) {
            const int lane_base = 32 * (warp & 3);
            const int col_base = (warp >> 2) * (BN / 2);
            const int gm = m0 + lane_base + lane;
            const bool row_ok = gm < M;
            const float as = row_ok ? a_scale[gm] : 0.0f;
            for (int c = col_base; c < col_base + BN / 2; c += 32) {
                uint32_t raw[32];
                ptx::tmem_ld_32x32(tmem_base + (static_cast<uint32_t>(lane_base) << 16) + c, raw);
                ptx::tmem_ld_wait();
                if (row_ok) {
                    uint32_t out[16];
#pragma unroll
                    for (int j = 0; j < 32; j += 2) {
                        const int a0 = static_cast<int>(raw[j]) >> 8, a1 = static_cast<int>(raw[j + 1]) >> 8;
                        raw[j] = a0; raw[j + 1] = a1;
                        float z0 = __fmul_rn(static_cast<float>(a0), __fmul_rn(as, s_wscale[c + j]));
                        float z1 = __fmul_rn(static_cast<float>(a1), __fmul_rn(as, s_wscale[c + j + 1]));
                        z0 = __fadd_rn(z0, s_bias[c + j]);
                        z1 = __fadd_rn(z1, s_bias[c + j + 1]);
                        __nv_bfloat162 p = __floats2bfloat162_rn(z0, z1);
                        out[j >> 1] = *reinterpret_cast<uint32_t *>(&p);
                    }
                    uint4 *dst = reinterpret_cast<uint4 *>(Y + (long long)gm * ldy + n0 + c);
#pragma unroll
                    for (int q = 0; q < 4; ++q) dst[q] = make_uint4(out[4 * q], out[4 * q + 1], out[4 * q + 2], out[4 * q + 3]);
                    if (acc_debug) {
                        uint4 *dbg = reinterpret_cast<uint4 *>(acc_debug + (long long)gm * N + n0 + c);
#pragma unroll
                        for (int q = 0; q < 8; ++q) dbg[q] = make_uint4(raw[4 * q], raw[4 * q + 1], raw[4 * q + 2], raw[4 * q + 3]);
                    }
                }
            }
        }
    } else {
        // ------------------------------------------------------------ MMA issuer (one thread)
        if (lane == 0) {
            constexpr uint32_t idesc = ptx::idesc_i8(BM, BN);
            bool alive = true;
            for (int kb = 0; kb < KB; ++kb) {
                const int s = kb % STAGES;
                alive = ptx::mbar_wait(bar_full + 8 * s, (kb / STAGES) & 1, s_abort, status, QVGGT_DEV_TIMEOUT_FULL);
                if (!alive) break;
                ptx::tc_fence_after_sync();
                const uint32_t a_addr = sbase + s * T::STAGE_BYTES;
                const uint32_t b_addr = a_addr + T::A_BYTES;
                const uint64_t a_desc = ptx::smem_desc_k_sw128(a_addr);
                const uint64_t b_desc = ptx::smem_desc_k_sw128(b_addr);
#pragma unroll
                for (int p = 0; p < BK / 32; ++p) {
                    // advance 32 bytes (one K = 32 slice) inside the swizzled row: +2 in 16-byte units
                    ptx::mma_i8_ss(tmem_base, a_desc + 2 * p, b_desc + 2 * p, idesc, (kb | p) != 0);
                }
                ptx::mma_commit(bar_empty + 8 * s);
            }
            ptx::mma_commit(bar_accum);
        }
        __syncwarp();
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == MMA_WARP) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, BN);
    }
}

template <int BN>
cudaError_t launch(const qvggt_weights *w, const unsigned char *Xq, const float *a_scale, int M, void *Y, long long ldy,
                   int *acc_debug, cudaStream_t st)
{
    using T = Tile<BN>;
    static bool configured = false;   // per process; the attribute is per function and device-independent on one GPU type
    cudaError_t e;
    if (!configured) {
        e = cudaFuncSetAttribute(gemm_w4a4_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, T::DYN_SMEM);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    dim3 grid((M + BM - 1) / BM, w->N / BN);
    gemm_w4a4_kernel<BN><<<grid, THREADS, T::DYN_SMEM, st>>>(Xq, w->Wq, a_scale, w->w_scale, w->bias,
                                                             static_cast<uint16_t *>(Y), ldy, acc_debug, M, w->N, w->K, w->status);
    return cudaGetLastError();
}

}  // namespace

cudaError_t qvggt_launch_gemm(const qvggt_weights *w, const unsigned char *Xq, const float *a_scale, int M, int group,
                              void *Y, long long ldy, int *acc_debug, cudaStream_t st)
{
    if (M == 0) return cudaSuccess;
    if (group != 0) return cudaErrorNotSupported;
    if (w->N % 256 == 0) return launch<256>(w, Xq, a_scale, M, Y, ldy, acc_debug, st);
    return launch<128>(w, Xq, a_scale, M, Y, ldy, acc_debug, st);
}
