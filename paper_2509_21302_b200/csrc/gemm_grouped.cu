// W4A4 GEMM with one activation scale per token per 128 consecutive rotated channels (an extension of
// the paper's token-wise granularity; the weights keep one scale per output channel).  Because the
// scale changes along the inner dimension, the integer sum of every 128-wide K-group is rescaled on
// its own before it joins the fp32 running sum:
//   Y[m][n] = bf16( (sum_g float(acc_g[m][n]) * a_scale[m][g]) * w_scale[n] + bias[n] ),  g ascending.
//
// Same building blocks as the token-wise kernel (TMA-staged packed codes, converter warps, int8
// tcgen05.mma with the codes in the high nibble, bounded waits), with these differences:
//   - one CTA per tile of 128 tokens x 128 channels (tcgen05.mma.cta_group::1, M = 128, N = 128);
//   - every K-block of 128 codes is one scale group: it accumulates into its own TMEM buffer (two
//     buffers of 128 columns, ping-pong), which the epilogue warps drain while the next group runs;
//   - the fp32 running sums live in a third region of tensor memory (128 columns): an epilogue thread reads 16 of
//     its row's sums, adds the rescaled group sums and writes them back, so it never holds more than 32 values
//     (64 sums in registers next to the accumulator chunk did not fit the 96 registers a thread of this 18-warp CTA
//     may use: they spilled to local memory and the kernel ran 10 x slower).
#include <cuda.h>
#include <cuda_bf16.h>

#include "gemm_common.cuh"
#include "qvggt_internal.cuh"
#include "sm100_ptx.cuh"
#include "tensor_map.cuh"

namespace {

using gemmc::STG_BYTES;

constexpr int BM = 128, BN = 128, BK = 128;
constexpr int EPI_WARPS = 8;       // warp w: TMEM lanes 32*(w%4).., columns 64*(w/4)..
constexpr int CONV_WARPS = 8;
constexpr int CONV_WARP0 = EPI_WARPS;
constexpr int MMA_WARP = EPI_WARPS + CONV_WARPS;
constexpr int TMA_WARP = MMA_WARP + 1;
constexpr int THREADS = (TMA_WARP + 1) * 32;
constexpr int ACC_BUFS = 2;

struct C {
    static constexpr int ROWS = BM + BN;                  // packed / operand rows per stage: tokens, then channels
    static constexpr int PK_STAGE = ROWS * (BK / 2);
    static constexpr int UP_STAGE = ROWS * BK;
    static constexpr int PS = 4, US = 4;
    static constexpr int GROUPS = 4;                      // converter groups, as in the token-wise kernel
    static constexpr int GROUP_WARPS = CONV_WARPS / GROUPS;
    static constexpr int GROUP_THREADS = GROUP_WARPS * 32;
    static constexpr int CHUNKS = ROWS * 4 / GROUP_THREADS;
    static constexpr int OFF_UP = 0;
    static constexpr int OFF_STG = OFF_UP + US * UP_STAGE;
    static constexpr int OFF_CH = OFF_STG + EPI_WARPS * STG_BYTES;      // [2][BN] channel scales, [2][BN] bias, fp32
    static constexpr int OFF_PK = OFF_CH + 2 * 2 * BN * 4;
    static constexpr int OFF_BAR = OFF_PK + PS * PK_STAGE;              // pfull[PS] pempty[PS] ufull[US] uempty[US] tfull[2] tempty[2]
    static constexpr int NBARS = 2 * PS + 2 * US + 2 * ACC_BUFS;
    static constexpr int OFF_TMEM = OFF_BAR + NBARS * 8;
    static constexpr int OFF_ABORT = OFF_TMEM + 4;
    static constexpr int OFF_FLAGS = OFF_ABORT + 4;
    static constexpr int SMEM_BYTES = OFF_FLAGS + 8 * (2 + CONV_WARPS);
    static constexpr int DYN_SMEM = SMEM_BYTES + 1024;
    static constexpr int SUM_COL = ACC_BUFS * BN;                       // first tensor-memory column of the running sums
    static constexpr int TMEM_COLS = 512;                               // 2 accumulators + sums = 384, rounded up to a power of two
    static_assert(DYN_SMEM <= 232448, "exceeds the 227 KB of shared memory a CTA may use");
};
constexpr int PS = C::PS, US = C::US, PK_STAGE = C::PK_STAGE, UP_STAGE = C::UP_STAGE;
constexpr int OFF_UP = C::OFF_UP, OFF_STG = C::OFF_STG, OFF_CH = C::OFF_CH, OFF_PK = C::OFF_PK, OFF_BAR = C::OFF_BAR;
constexpr int OFF_TMEM = C::OFF_TMEM, OFF_ABORT = C::OFF_ABORT, OFF_FLAGS = C::OFF_FLAGS, DYN_SMEM = C::DYN_SMEM, TMEM_COLS = C::TMEM_COLS;

__global__ void __launch_bounds__(THREADS, 1)
gemm_w4a4_grouped_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                         const __grid_constant__ CUtensorMap map_y, const float *__restrict__ a_scale,
                         const float *__restrict__ w_scale, const uint16_t *__restrict__ bias, int *__restrict__ acc_debug,
                         int M, int N, int K, int *status)
{
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = ptx::smem_addr(smem);
    const uint32_t bar_pfull = sbase + OFF_BAR;
    const uint32_t bar_pempty = bar_pfull + PS * 8;
    const uint32_t bar_ufull = bar_pempty + PS * 8;
    const uint32_t bar_uempty = bar_ufull + US * 8;
    const uint32_t bar_tfull = bar_uempty + US * 8;
    const uint32_t bar_tempty = bar_tfull + ACC_BUFS * 8;
    uint32_t *s_tmem = reinterpret_cast<uint32_t *>(smem + OFF_TMEM);
    volatile int *s_abort = reinterpret_cast<volatile int *>(smem + OFF_ABORT);
    volatile int *s_flags = reinterpret_cast<volatile int *>(smem + OFF_FLAGS);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int worker = blockIdx.x, workers = gridDim.x;
    const int KB = K / BK;                                    // = number of scale groups
    const int n_tiles = N / BN;
    const int total_tiles = ((M + BM - 1) / BM) * n_tiles;
    const int my_tiles = (total_tiles > worker) ? (total_tiles - 1 - worker) / workers + 1 : 0;

    if (threadIdx.x == 0) {
        gemmc::init_barriers(bar_pfull, PS, 1);                      // the producer's arrive.expect_tx
        gemmc::init_barriers(bar_pempty, PS, C::GROUP_WARPS);
        gemmc::init_barriers(bar_ufull, US, C::GROUP_WARPS);
        gemmc::init_barriers(bar_uempty, US, 1);                     // tcgen05.commit
        gemmc::init_barriers(bar_tfull, ACC_BUFS, 1);                // tcgen05.commit
        gemmc::init_barriers(bar_tempty, ACC_BUFS, EPI_WARPS);
        *s_abort = 0;
        ptx::fence_mbar_init();
    }
    if (warp == MMA_WARP) {
        ptx::tmem_alloc(ptx::smem_addr(s_tmem), TMEM_COLS);
        ptx::tmem_relinquish();
    }
    if (warp == TMA_WARP && lane == 0) {
        ptx::prefetch_tensormap(&map_x);
        ptx::prefetch_tensormap(&map_w);
        ptx::prefetch_tensormap(&map_y);
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *s_tmem;

    if (warp < EPI_WARPS) {
        // ------------------------------------------------------------ epilogue
        const int quarter = warp & 3, chalf = warp >> 2;   // TMEM lane quarter, column half (64 columns)
        unsigned char *stg = smem + OFF_STG + warp * STG_BYTES;
        const uint32_t stg_addr = sbase + OFF_STG + warp * STG_BYTES;
        float *s_ws = reinterpret_cast<float *>(smem + OFF_CH);    // [2][BN]
        float *s_bs = s_ws + 2 * BN;                                // [2][BN]
        bool alive = true;
        int it = 0;                                                 // K-blocks seen so far (all tiles)
        for (int t = 0; t < my_tiles; ++t) {
            const int tile = worker + t * workers;
            const int m0 = (tile / n_tiles) * BM + quarter * 32;
            const int nt0 = (tile % n_tiles) * BN;
            const int n0 = nt0 + chalf * 64;
            const int tb = t & 1;
            const int gm = m0 + lane;
            const bool row_ok = gm < M;
            if (threadIdx.x < BN) {
                // buffer tb was last read two tiles ago; every epilogue warp has passed the barrier of the tile in between since
                gemmc::load_channel_params(s_ws + tb * BN, s_bs + tb * BN, w_scale, bias, nt0, N, threadIdx.x);
            }
            // once per tile the epilogue warps meet: publishes s_ws / s_bs of this tile and orders their reuse two tiles on
            asm volatile("bar.sync %0, %1;" ::"r"(1), "r"(EPI_WARPS * 32) : "memory");
            // the group's activation scale is fetched one K-block ahead: it comes from L2, several hundred cycles away
            float as_next = row_ok ? __ldg(a_scale + (long long)gm * KB) : 0.0f;
#pragma unroll 1
            for (int kb = 0; kb < KB; ++kb, ++it) {
                const int b = it & 1;
                const bool first = kb == 0, last = kb == KB - 1;
                // a_scale / 256: exact, cancels the factor 256 carried by the raw accumulator
                const float as = __fmul_rn(as_next, 0.00390625f);
                if (!last && row_ok) as_next = __ldg(a_scale + (long long)gm * KB + kb + 1);
                {   // every warp polls for itself (lane 0; the warp follows): no warp waits for a slower one between K-blocks
                    int ok = 1;
                    if (lane == 0) ok = (alive && ptx::mbar_wait(bar_tfull + 8 * b, (it >> 1) & 1, s_abort, status, QVGGT_DEV_TIMEOUT_ACCUM, 20)) ? 1 : 0;
                    alive = __shfl_sync(0xFFFFFFFFu, ok, 0) != 0;
                }
                ptx::tc_fence_after_sync();
                if (!alive) continue;
                const uint32_t lane_base = static_cast<uint32_t>(quarter * 32) << 16;
                const float *wsb = s_ws + tb * BN + chalf * 64;
                const float *bsb = s_bs + tb * BN + chalf * 64;
                uint32_t out[16];                     // two 16-column chunks make one 32-column staging tile
                // the loads of chunk c + 1 are in flight while chunk c is rescaled (tcgen05.wait::ld waits for every load
                // issued so far, so the next chunk's loads go out right behind the wait)
                uint32_t raw[2][16], sum[2][16];
                const uint32_t acc_addr = tmem_base + lane_base + b * BN + chalf * 64, sum_addr = tmem_base + lane_base + C::SUM_COL + chalf * 64;
                ptx::tmem_ld_32x16(acc_addr, raw[0]);
                if (!first) ptx::tmem_ld_32x16(sum_addr, sum[0]);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    ptx::tmem_ld_wait();
                    if (c < 3) {
                        ptx::tmem_ld_32x16(acc_addr + (c + 1) * 16, raw[(c + 1) & 1]);
                        if (!first) ptx::tmem_ld_32x16(sum_addr + (c + 1) * 16, sum[(c + 1) & 1]);
                    } else {
                        // last read of this accumulator: hand it back to the MMA thread
                        ptx::tc_fence_before_sync();
                        __syncwarp();
                        if (lane == 0) ptx::mbar_arrive(bar_tempty + 8 * b);
                    }
                    uint32_t (&r)[16] = raw[c & 1];
                    uint32_t (&sm)[16] = sum[c & 1];
                    // s = fl(s + fl(float(acc_g) * a_scale[m][g])), g ascending: separate multiply and add
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const float p = __fmul_rn(static_cast<float>(static_cast<int>(r[j])), as);
                        sm[j] = __float_as_uint(__fadd_rn(first ? 0.0f : __uint_as_float(sm[j]), p));
                    }
                    if (acc_debug && row_ok) {
                        uint4 *dbg = reinterpret_cast<uint4 *>(acc_debug + ((long long)kb * M + gm) * N + n0 + c * 16);
#pragma unroll
                        for (int q4 = 0; q4 < 4; ++q4)
                            dbg[q4] = make_uint4(static_cast<int>(r[4 * q4]) >> 8, static_cast<int>(r[4 * q4 + 1]) >> 8,
                                                 static_cast<int>(r[4 * q4 + 2]) >> 8, static_cast<int>(r[4 * q4 + 3]) >> 8);
                    }
                    if (!last) {
                        ptx::tmem_st_32x16(sum_addr + c * 16, sm);
                    } else {
                        // bf16( fl(fl(s * w_scale) + bias) )
#pragma unroll
                        for (int j = 0; j < 16; j += 2) {
                            const float z0 = __fadd_rn(__fmul_rn(__uint_as_float(sm[j]), wsb[16 * c + j]), bsb[16 * c + j]);
                            const float z1 = __fadd_rn(__fmul_rn(__uint_as_float(sm[j + 1]), wsb[16 * c + j + 1]), bsb[16 * c + j + 1]);
                            out[8 * (c & 1) + (j >> 1)] = ptx::pack_bf16x2(z0, z1);
                        }
                        if (c & 1) {
                            gemmc::stage_row_32(stg, out, lane);
                            gemmc::store_staged_32x32(&map_y, stg_addr, n0 + (c >> 1) * 32, m0, m0 < M, lane);
                        }
                    }
                }
                if (!last) ptx::tmem_st_wait();       // the sums are back in tensor memory before the next group reads them
            }
        }
        if (lane == 0) ptx::tma_store_wait_all();
    } else if (warp < MMA_WARP) {
        // ------------------------------------------------------------ converters (see the token-wise kernel)
        gemmc::convert_packed_stages<C, false>(smem, warp - CONV_WARP0, lane, my_tiles * KB, bar_pfull, bar_pempty, bar_uempty,
                                               bar_ufull, s_abort, status, s_flags + 2, s_flags + 1 + 2 * CONV_WARPS,
                                               QVGGT_DEV_TIMEOUT_PACKED, QVGGT_DEV_TIMEOUT_EMPTY);
    } else if (warp == MMA_WARP) {
        // ------------------------------------------------------------ MMA issuer: one accumulator per K-block
        if (lane == 0) {
            constexpr uint32_t idesc = ptx::idesc_i8(BM, BN);
            bool alive = true;
            const int total_kb = my_tiles * KB;
            for (int it = 0; it < total_kb && alive; ++it) {
                const int b = it & 1, us = it % US;
                if (it >= ACC_BUFS) {
                    alive = ptx::mbar_wait(bar_tempty + 8 * b, ((it >> 1) - 1) & 1, s_abort, status, QVGGT_DEV_TIMEOUT_TMEM_FREE);
                    if (!alive) break;
                }
                alive = ptx::mbar_wait(bar_ufull + 8 * us, (it / US) & 1, s_abort, status, QVGGT_DEV_TIMEOUT_FULL);
                if (!alive) break;
                ptx::tc_fence_after_sync();
                const uint32_t a_addr = sbase + OFF_UP + us * UP_STAGE;
                gemmc::mma_kblock_i8<false>(tmem_base + b * BN, a_addr, a_addr + BM * BK, idesc, true);
                ptx::mma_commit(bar_uempty + 8 * us);
                ptx::mma_commit(bar_tfull + 8 * b);
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            bool alive = true;
            int it = 0;
            for (int t = 0; t < my_tiles && alive; ++t) {
                const int tile = worker + t * workers;
                const int m0 = (tile / n_tiles) * BM, n0 = (tile % n_tiles) * BN;
                for (int kb = 0; kb < KB; ++kb, ++it) {
                    const int ps = it % PS;
                    if (it >= PS) {
                        alive = ptx::mbar_wait(bar_pempty + 8 * ps, ((it / PS) - 1) & 1, s_abort, status, QVGGT_DEV_TIMEOUT_PACKED_FREE, 20);
                        if (!alive) break;
                    }
                    const uint32_t dst = sbase + OFF_PK + ps * PK_STAGE;
                    ptx::mbar_arrive_expect_tx(bar_pfull + 8 * ps, PK_STAGE);
                    ptx::tma_load_2d(&map_x, bar_pfull + 8 * ps, dst, kb * (BK / 2), m0);
                    ptx::tma_load_2d(&map_w, bar_pfull + 8 * ps, dst + BM * (BK / 2), kb * (BK / 2), n0);
                }
            }
        }
        __syncwarp();
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == MMA_WARP) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

}  // namespace

cudaError_t qvggt_launch_gemm_grouped(const qvggt_weights *w, const unsigned char *Xq, const float *a_scale, int M, void *Y,
                                      long long ldy, int *acc_debug, cudaStream_t st)
{
    static QvggtPerDevice cache;
    int sms = 0;
    cudaError_t e = qvggt_configure_kernel(gemm_w4a4_grouped_kernel, THREADS, DYN_SMEM, 1, cache, &sms);
    if (e != cudaSuccess) return e;
    const int K = w->K, N = w->N;
    CUtensorMap map_x, map_w, map_y;
    if (!qvggt_make_map(&map_x, CU_TENSOR_MAP_DATA_TYPE_UINT8, Xq, K / 2, M, K / 2, BK / 2, BM, CU_TENSOR_MAP_SWIZZLE_NONE) ||
        !qvggt_make_map(&map_w, CU_TENSOR_MAP_DATA_TYPE_UINT8, w->Wq, K / 2, N, K / 2, BK / 2, BN, CU_TENSOR_MAP_SWIZZLE_NONE) ||
        !qvggt_make_map(&map_y, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, Y, N, M, (uint64_t)ldy * 2, 32, 32, CU_TENSOR_MAP_SWIZZLE_64B))
        return cudaErrorInvalidValue;
    const int total_tiles = ((M + BM - 1) / BM) * (N / BN);
    const int grid = total_tiles < sms ? total_tiles : sms;
    gemm_w4a4_grouped_kernel<<<grid, THREADS, DYN_SMEM, st>>>(map_x, map_w, map_y, a_scale, w->w_scale, w->bias, acc_debug, M, N,
                                                              K, w->status);
    return cudaGetLastError();
}
