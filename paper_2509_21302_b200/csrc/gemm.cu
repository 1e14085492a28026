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

#ifdef QVGGT_PROFILE
__device__ long long g_prof[32];
extern "C" int qvggt_debug_read_prof(long long *host_out)
{
    return (int)cudaMemcpyFromSymbol(host_out, g_prof, sizeof(long long) * 32);
}
#define PROF_DECL(n) long long n = 0
#define PROF_T0(t) long long t = clock64()
#define PROF_ADD(acc, t) do { long long _n = clock64(); acc += _n - t; t = _n; } while (0)
#define PROF_STORE(i, v) do { g_prof[i] = (v); } while (0)
#else
#define PROF_DECL(n)
#define PROF_T0(t)
#define PROF_ADD(acc, t)
#define PROF_STORE(i, v)
#endif

namespace {

constexpr int BM = 128;            // tokens per CTA tile (TMEM lanes)
constexpr int BK = 128;            // codes along K per pipeline stage = one 128-byte swizzled row of int8
constexpr int STAGES = 4;          // shared-memory operand ring; also the converter's register ring
constexpr int PREFETCH = 3;        // K-blocks of packed codes in flight (in registers) per converter thread
constexpr int CONV_WARPS = 8;
constexpr int CONV_THREADS = CONV_WARPS * 32;
constexpr int MMA_WARP = CONV_WARPS;
constexpr int EPI_WARP0 = CONV_WARPS + 1;
constexpr int EPI_WARPS = 4;       // warp (EPI_WARP0 + i) owns TMEM lanes 32 * ((EPI_WARP0 + i) % 4) ..
constexpr int EPI_THREADS = EPI_WARPS * 32;
constexpr int THREADS = (CONV_WARPS + 1 + EPI_WARPS) * 32;
constexpr int ACC_BUFS = 2;        // TMEM accumulators: the epilogue of tile i overlaps the MMAs of tile i+1

template <int BN>
struct Tile {
    static constexpr int A_BYTES = BM * 128;
    static constexpr int B_BYTES = BN * 128;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int CHUNKS = (BM + BN) * 4 / CONV_THREADS;   // 16-byte packed pieces per thread per stage
    static constexpr int OFF_WSCALE = STAGES * STAGE_BYTES;
    static constexpr int OFF_BIAS = OFF_WSCALE + BN * 4;
    static constexpr int OFF_BAR = OFF_BIAS + BN * 4;             // full[STAGES], empty[STAGES], tfull[2], tempty[2]
    static constexpr int NBARS = 2 * STAGES + 2 * ACC_BUFS;
    static constexpr int OFF_TMEM = OFF_BAR + NBARS * 8;
    static constexpr int OFF_ABORT = OFF_TMEM + 4;
    static constexpr int BYTES = OFF_ABORT + 4;
    static constexpr int DYN_SMEM = BYTES + 1024;                 // slack to align the base to 1024 bytes
    static constexpr int TMEM_COLS = ACC_BUFS * BN;               // 512 (BN = 256) or 256 (BN = 128): powers of two
};

__device__ __forceinline__ float bf16_bits_to_f32(uint16_t b) { return __uint_as_float(static_cast<uint32_t>(b) << 16); }

// Persistent, warp-specialised: CTA b works on tiles b, b + gridDim.x, ... (n fastest, so CTAs that run
// together share the token rows of A and all of W stays in L2).
//   warps 0-7   converters: packed codes global -> registers (PREFETCH K-blocks ahead) -> int8 operand tiles in smem
//   warp  8     one thread issues tcgen05.mma and the commits that release stages / publish accumulators
//   warps 9-12  epilogue: TMEM -> registers -> scale, bias, bf16 -> global
template <int BN>
__global__ void __launch_bounds__(THREADS, 1)
gemm_w4a4_kernel(const unsigned char *__restrict__ Xq, const unsigned char *__restrict__ Wq,
                 const float *__restrict__ a_scale, const float *__restrict__ w_scale,
                 const uint16_t *__restrict__ bias, uint16_t *__restrict__ Y, long long ldy,
                 int *__restrict__ acc_debug, int M, int N, int K, int *status)
{
    using T = Tile<BN>;
    static_assert(STAGES == 4 && PREFETCH == 3, "the converter loop is unrolled for a 4-slot ring");
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = ptx::smem_addr(smem);
    float *s_wscale = reinterpret_cast<float *>(smem + T::OFF_WSCALE);
    float *s_bias = reinterpret_cast<float *>(smem + T::OFF_BIAS);
    const uint32_t bar_full = sbase + T::OFF_BAR;
    const uint32_t bar_empty = bar_full + STAGES * 8;
    const uint32_t bar_tfull = bar_empty + STAGES * 8;
    const uint32_t bar_tempty = bar_tfull + ACC_BUFS * 8;
    uint32_t *s_tmem = reinterpret_cast<uint32_t *>(smem + T::OFF_TMEM);
    volatile int *s_abort = reinterpret_cast<volatile int *>(smem + T::OFF_ABORT);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int KB = K / BK;                      // 8 or 32: a multiple of STAGES
    const int row_bytes = K / 2;
    const int n_tiles = N / BN;
    const int total_tiles = ((M + BM - 1) / BM) * n_tiles;
    const int my_tiles = (total_tiles > (int)blockIdx.x) ? (total_tiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(bar_full + 8 * s, CONV_WARPS);     // one arrival per converter warp
            ptx::mbar_init(bar_empty + 8 * s, 1);
        }
        for (int b = 0; b < ACC_BUFS; ++b) {
            ptx::mbar_init(bar_tfull + 8 * b, 1);
            ptx::mbar_init(bar_tempty + 8 * b, EPI_WARPS);
        }
        *s_abort = 0;
        ptx::fence_mbar_init();
    }
    if (warp == MMA_WARP) {
        ptx::tmem_alloc(ptx::smem_addr(s_tmem), T::TMEM_COLS);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *s_tmem;

    if (warp < CONV_WARPS) {
        // ------------------------------------------------------------ converters
        int row_of[T::CHUNKS];          // row inside the A region (< BM) or BM + row inside the B region
        uint32_t soff[T::CHUNKS];
#pragma unroll
        for (int i = 0; i < T::CHUNKS; ++i) {
            const int c = threadIdx.x + CONV_THREADS * i;
            const int row = c >> 2, piece = c & 3;
            row_of[i] = row;
            // even codes -> 16-byte chunk 2*piece, odd codes -> chunk 2*piece+1, both XOR (row mod 8)
            soff[i] = (row < BM ? row * 128 : T::A_BYTES + (row - BM) * 128) + (((2 * piece) ^ (row & 7)) << 4);
        }
        const int piece_off = (threadIdx.x & 3) * 16;

        // load cursor: walks (tile, kb) PREFETCH blocks ahead of the conversion
        const unsigned char *lptr[T::CHUNKS];
        int l_tile = 0, l_kb = 0;
        auto set_tile_ptrs = [&](int t_local) {
            const int tile = blockIdx.x + t_local * gridDim.x;
            const int m0 = (tile / n_tiles) * BM, n0 = (tile % n_tiles) * BN;
#pragma unroll
            for (int i = 0; i < T::CHUNKS; ++i) {
                if (row_of[i] < BM) {
                    const int gm = m0 + row_of[i];
                    lptr[i] = (gm < M) ? Xq + (long long)gm * row_bytes + piece_off : nullptr;
                } else {
                    lptr[i] = Wq + (long long)(n0 + row_of[i] - BM) * row_bytes + piece_off;
                }
            }
        };
        auto issue_load = [&](uint4 (&dst)[T::CHUNKS]) {
            if (l_tile < my_tiles) {
#pragma unroll
                for (int i = 0; i < T::CHUNKS; ++i) {
#ifdef QVGGT_PROBE_NO_LOADS
                    dst[i] = make_uint4(l_kb, i, l_tile, 0);
#else
                    dst[i] = lptr[i] ? __ldg(reinterpret_cast<const uint4 *>(lptr[i] + l_kb * (BK / 2))) : make_uint4(0, 0, 0, 0);
#endif
                }
                if (++l_kb == KB) {
                    l_kb = 0;
                    if (++l_tile < my_tiles) set_tile_ptrs(l_tile);
                }
            }
        };
        auto convert = [&](const uint4 (&src)[T::CHUNKS], unsigned char *stage) {
#pragma unroll
            for (int i = 0; i < T::CHUNKS; ++i) {
                const uint4 w = src[i];
                uint4 lo, hi;
                lo.x = (w.x << 4) & 0xF0F0F0F0u; hi.x = w.x & 0xF0F0F0F0u;
                lo.y = (w.y << 4) & 0xF0F0F0F0u; hi.y = w.y & 0xF0F0F0F0u;
                lo.z = (w.z << 4) & 0xF0F0F0F0u; hi.z = w.z & 0xF0F0F0F0u;
                lo.w = (w.w << 4) & 0xF0F0F0F0u; hi.w = w.w & 0xF0F0F0F0u;
                *reinterpret_cast<uint4 *>(stage + soff[i]) = lo;
                *reinterpret_cast<uint4 *>(stage + (soff[i] ^ 16)) = hi;
            }
        };

        uint4 buf[STAGES][T::CHUNKS];
        if (my_tiles > 0) set_tile_ptrs(0);
        issue_load(buf[0]);
        issue_load(buf[1]);
        issue_load(buf[2]);
        const int rounds = my_tiles * (KB / STAGES);
        bool alive = true;
        PROF_DECL(p_load); PROF_DECL(p_wait); PROF_DECL(p_conv); PROF_DECL(p_fence); PROF_DECL(p_arrive);
        PROF_T0(pt);
        for (int r = 0; r < rounds && alive; ++r) {
#pragma unroll
            for (int u = 0; u < STAGES; ++u) {
                issue_load(buf[(u + PREFETCH) & (STAGES - 1)]);
                PROF_ADD(p_load, pt);
                if (r > 0) alive = alive && ptx::mbar_wait_warp(bar_empty + 8 * u, (r - 1) & 1, s_abort, status, QVGGT_DEV_TIMEOUT_EMPTY, lane);
                PROF_ADD(p_wait, pt);
                if (alive) {
                    convert(buf[u], smem + u * T::STAGE_BYTES);
                    PROF_ADD(p_conv, pt);
                    ptx::fence_proxy_async_smem();      // my generic-proxy writes -> visible to the tensor core's async proxy
                    PROF_ADD(p_fence, pt);
                }
                __syncwarp();                            // orders the whole warp's writes before the single arrival
                if (alive && lane == 0) ptx::mbar_arrive(bar_full + 8 * u);
                PROF_ADD(p_arrive, pt);
            }
        }
#ifdef QVGGT_PROFILE
        if (blockIdx.x == 0 && threadIdx.x == 0) {
            PROF_STORE(0, p_load); PROF_STORE(1, p_wait); PROF_STORE(2, p_conv); PROF_STORE(3, p_fence); PROF_STORE(4, p_arrive);
            PROF_STORE(5, (long long)rounds * STAGES);
        }
#endif
    } else if (warp == MMA_WARP) {
        // ------------------------------------------------------------ MMA issuer (one thread)
        if (lane == 0) {
            constexpr uint32_t idesc = ptx::idesc_i8(BM, BN);
            bool alive = true;
            int g = 0;                                   // K-blocks consumed so far (all tiles)
            PROF_DECL(p_tempty); PROF_DECL(p_full); PROF_DECL(p_issue);
            PROF_T0(pt);
            for (int t = 0; t < my_tiles && alive; ++t) {
                const int b = t & 1;
                if (t >= ACC_BUFS) {
                    alive = ptx::mbar_wait(bar_tempty + 8 * b, ((t >> 1) - 1) & 1, s_abort, status, QVGGT_DEV_TIMEOUT_TMEM_FREE);
                    if (!alive) break;
                    ptx::tc_fence_after_sync();
                }
                PROF_ADD(p_tempty, pt);
                const uint32_t d_tmem = tmem_base + b * BN;
                for (int kb = 0; kb < KB; ++kb, ++g) {
                    const int s = g & (STAGES - 1);
                    alive = ptx::mbar_wait(bar_full + 8 * s, (g / STAGES) & 1, s_abort, status, QVGGT_DEV_TIMEOUT_FULL);
                    if (!alive) break;
                    ptx::tc_fence_after_sync();
                    PROF_ADD(p_full, pt);
                    const uint32_t a_addr = sbase + s * T::STAGE_BYTES;
                    const uint64_t a_desc = ptx::smem_desc_k_sw128(a_addr);
                    const uint64_t b_desc = ptx::smem_desc_k_sw128(a_addr + T::A_BYTES);
#pragma unroll
                    for (int p = 0; p < BK / 32; ++p) {
                        // advance 32 bytes (one K = 32 slice) inside the swizzled row: +2 in 16-byte units
                        ptx::mma_i8_ss(d_tmem, a_desc + 2 * p, b_desc + 2 * p, idesc, (kb | p) != 0);
                    }
                    ptx::mma_commit(bar_empty + 8 * s);
                    PROF_ADD(p_issue, pt);
                }
                if (alive) ptx::mma_commit(bar_tfull + 8 * b);
            }
#ifdef QVGGT_PROFILE
            if (blockIdx.x == 0) { PROF_STORE(8, p_tempty); PROF_STORE(9, p_full); PROF_STORE(10, p_issue); }
#endif
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ epilogue
        const int et = threadIdx.x - EPI_WARP0 * 32;       // 0..127
        const int lane_base = 32 * (warp & 3);
        bool alive = true;
        PROF_DECL(p_twait); PROF_DECL(p_work);
        PROF_T0(pt);
        for (int t = 0; t < my_tiles; ++t) {
            const int tile = blockIdx.x + t * gridDim.x;
            const int m0 = (tile / n_tiles) * BM, n0 = (tile % n_tiles) * BN;
            const int b = t & 1;
            // per-channel scale and bias of this tile's columns (previous tile's readers are past this barrier)
            asm volatile("bar.sync 1, %0;" ::"n"(EPI_THREADS) : "memory");
            for (int i = et; i < BN; i += EPI_THREADS) {
                s_wscale[i] = w_scale[n0 + i];
                s_bias[i] = bias ? bf16_bits_to_f32(bias[n0 + i]) : 0.0f;
            }
            asm volatile("bar.sync 1, %0;" ::"n"(EPI_THREADS) : "memory");
            const int gm = m0 + lane_base + lane;
            const bool row_ok = gm < M;
            const float as = row_ok ? a_scale[gm] : 0.0f;
            PROF_ADD(p_work, pt);
            if (alive) alive = ptx::mbar_wait_warp(bar_tfull + 8 * b, (t >> 1) & 1, s_abort, status, QVGGT_DEV_TIMEOUT_ACCUM, lane, 32);
            ptx::tc_fence_after_sync();
            PROF_ADD(p_twait, pt);
            if (alive) {
#pragma unroll 1
                for (int c = 0; c < BN; c += 32) {
                    uint32_t raw[32];
                    ptx::tmem_ld_32x32(tmem_base + (static_cast<uint32_t>(lane_base) << 16) + b * BN + c, raw);
                    ptx::tmem_ld_wait();
#ifdef QVGGT_PROBE_NO_EPILOGUE_MATH
                    if (row_ok && raw[0] == 0x7fffffffu) {
#else
                    if (row_ok) {
#endif
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
                ptx::tc_fence_before_sync();
            }
            __syncwarp();
            if (alive && lane == 0) ptx::mbar_arrive(bar_tempty + 8 * b);
            PROF_ADD(p_work, pt);
        }
#ifdef QVGGT_PROFILE
        if (blockIdx.x == 0 && et == 0) { PROF_STORE(16, p_twait); PROF_STORE(17, p_work); PROF_STORE(18, my_tiles); }
#endif
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == MMA_WARP) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, T::TMEM_COLS);
    }
}

int sm_count()
{
    static int sms = 0;
    if (!sms) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    }
    return sms;
}

template <int BN>
cudaError_t launch(const qvggt_weights *w, const unsigned char *Xq, const float *a_scale, int M, void *Y, long long ldy,
                   int *acc_debug, cudaStream_t st)
{
    using T = Tile<BN>;
    static bool configured = false;   // per process; one GPU type per process
    cudaError_t e;
    if (!configured) {
        e = cudaFuncSetAttribute(gemm_w4a4_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, T::DYN_SMEM);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    const int total_tiles = ((M + BM - 1) / BM) * (w->N / BN);
    const int grid = total_tiles < sm_count() ? total_tiles : sm_count();
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
