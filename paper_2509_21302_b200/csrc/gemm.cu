// W4A4 GEMM + rescale + bias + bf16 for sm_100a (Sec. 3.2: integer sum over the inner dimension,
// per-token and per-out-channel scales applied outside the sum).
//
// tcgen05 has no 4-bit integer kind, so the codes are fed to kind::i8.  TMA stages tiles of packed
// codes in shared memory; converter warps expand every nibble into the HIGH half of a byte (value
// 16*q, so no sign extension is needed) and write the int8 operand tiles in the 128-byte-swizzled
// K-major layout the tensor core reads.  The raw accumulator is therefore 256 * sum(q_x q_w) (at
// most 2^26 in magnitude), undone exactly in the epilogue.  Even and odd codes of a 32-code slice
// land in separate 16-byte chunks; the same permutation of K is applied to both operands, so the
// dot product is unchanged.
//
// Persistent and warp-specialised.  A "worker" is a pair of CTAs on neighbouring SMs (tile 256 x 256, each
// CTA stages 128 token rows and 128 weight rows, one thread of the leader CTA issues tcgen05.mma.cta_group::2
// for both; a single-CTA configuration measured 10-35 % slower on every VGGT shape: the pair halves the
// weight traffic).
//   warps 0-7    epilogue: TMEM -> registers -> scale, bias, bf16 -> swizzled staging -> TMA store
//   warps 8-15   converters: packed stage -> registers -> int8 operand stage
//   warp  16     one thread issues tcgen05.mma and the commits that release stages / publish accumulators
//   warp  17     one thread issues the TMA loads of packed tiles
// Every wait is bounded; on expiry the kernel records a code in *status and all roles fall through
// to the common exit, where tensor memory is released.
#include <cuda.h>
#include <cuda_bf16.h>

#include "gemm_common.cuh"
#include "qvggt_internal.cuh"
#include "sm100_ptx.cuh"
#include "tensor_map.cuh"

namespace {

using gemmc::STG_BYTES;

constexpr int BM = 128;            // token rows per CTA (TMEM lanes)
constexpr int BN = 256;            // output channels per tile
constexpr int BK = 128;            // codes along K per pipeline stage = one 128-byte swizzled row of int8
constexpr int EPI_WARPS = 8;       // warp w reads TMEM lanes 32*(w%4).., columns 128*(w/4)..
constexpr int CONV_WARPS = 8;
constexpr int CONV_WARP0 = EPI_WARPS;
constexpr int MMA_WARP = EPI_WARPS + CONV_WARPS;
constexpr int TMA_WARP = MMA_WARP + 1;
constexpr int THREADS = (TMA_WARP + 1) * 32;
constexpr int ACC_BUFS = 2;        // TMEM accumulators: the epilogue of tile i overlaps the MMAs of tile i+1

constexpr int CG = 2;               // CTAs per worker

struct C {
    static constexpr int B_ROWS = BN / CG;                 // weight rows staged by one CTA
    static constexpr int ROWS = BM + B_ROWS;
    static constexpr int PK_STAGE = ROWS * (BK / 2);       // packed codes
    static constexpr int UP_STAGE = ROWS * BK;             // int8 operands
    static constexpr int PS = 4;                           // packed stages (cover the L2 latency)
    static constexpr int US = 4;                           // operand stages (decouple converters and MMA)
    // Converter warps form GROUPS independent groups; group g converts K-blocks g, g + GROUPS, ...  so the
    // fixed costs of a stage (draining the stores, the proxy fence, barrier round trips) overlap.
    static constexpr int GROUPS = 4;
    static constexpr int GROUP_WARPS = CONV_WARPS / GROUPS;
    static constexpr int GROUP_THREADS = GROUP_WARPS * 32;
    static constexpr int CHUNKS = ROWS * 4 / GROUP_THREADS;   // 16-byte packed pieces per thread per stage
    static constexpr int OFF_UP = 0;                       // operand stages first: they need 1024-byte alignment
    static constexpr int OFF_STG = OFF_UP + US * UP_STAGE;
    static constexpr int OFF_CH = OFF_STG + EPI_WARPS * STG_BYTES;   // per-channel scale and bias of two tiles, fp32
    static constexpr int OFF_PK = OFF_CH + 2 * ACC_BUFS * BN * 4;
    static constexpr int OFF_BAR = OFF_PK + PS * PK_STAGE; // pfull[PS] pempty[PS] ufull[US] uempty[US] tfull[2] tempty[2]
    static constexpr int NBARS = 2 * PS + 2 * US + 2 * ACC_BUFS;
    static constexpr int OFF_TMEM = OFF_BAR + NBARS * 8;
    static constexpr int OFF_ABORT = OFF_TMEM + 4;
    static constexpr int OFF_FLAGS = OFF_ABORT + 4;        // outcome words of the group waits: epilogue, converter groups
    static constexpr int BYTES = OFF_FLAGS + 8 * (2 + CONV_WARPS);
    static constexpr int DYN_SMEM = BYTES + 1024;          // slack to align the base to 1024 bytes
    static constexpr int TMEM_COLS = ACC_BUFS * BN;        // 512
    static_assert(DYN_SMEM <= 232448, "exceeds the 227 KB of shared memory a CTA may use");
    static_assert(UP_STAGE % 1024 == 0 && (BM * BK) % 1024 == 0, "operand tiles must stay 1024-byte aligned");
};

// DUMP: also write the int32 sums to acc_debug (a separate instantiation keeps that code, and the registers it
// pins, out of the production kernel)
template <bool DUMP>
__global__ void __launch_bounds__(THREADS, 1)
gemm_w4a4_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                 const __grid_constant__ CUtensorMap map_y, const float *__restrict__ a_scale,
                 const float *__restrict__ w_scale, const uint16_t *__restrict__ bias, int *__restrict__ acc_debug,
                 int M, int N, int K, int *status)
{
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = ptx::smem_addr(smem);
    const uint32_t bar_pfull = sbase + C::OFF_BAR;
    const uint32_t bar_pempty = bar_pfull + C::PS * 8;
    const uint32_t bar_ufull = bar_pempty + C::PS * 8;
    const uint32_t bar_uempty = bar_ufull + C::US * 8;
    const uint32_t bar_tfull = bar_uempty + C::US * 8;
    const uint32_t bar_tempty = bar_tfull + ACC_BUFS * 8;
    uint32_t *s_tmem = reinterpret_cast<uint32_t *>(smem + C::OFF_TMEM);
    volatile int *s_abort = reinterpret_cast<volatile int *>(smem + C::OFF_ABORT);
    volatile int *s_flags = reinterpret_cast<volatile int *>(smem + C::OFF_FLAGS);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank();                       // 0 = leader of the pair
    const int worker = blockIdx.x / CG, workers = gridDim.x / CG;
    const int KB = K / BK;
    const int n_tiles = (N + BN - 1) / BN;
    const int total_tiles = ((M + BM * CG - 1) / (BM * CG)) * n_tiles;
    const int my_tiles = (total_tiles > worker) ? (total_tiles - 1 - worker) / workers + 1 : 0;

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::PS; ++s) {
            ptx::mbar_init(bar_pfull + 8 * s, 1);                    // the producer's arrive.expect_tx
            ptx::mbar_init(bar_pempty + 8 * s, C::GROUP_WARPS);
        }
        for (int s = 0; s < C::US; ++s) {
            ptx::mbar_init(bar_ufull + 8 * s, C::GROUP_WARPS * CG); // one converter group of every CTA of the worker
            ptx::mbar_init(bar_uempty + 8 * s, 1);                   // tcgen05.commit
        }
        for (int b = 0; b < ACC_BUFS; ++b) {
            ptx::mbar_init(bar_tfull + 8 * b, 1);                    // tcgen05.commit
            ptx::mbar_init(bar_tempty + 8 * b, EPI_WARPS * CG);
        }
        *s_abort = 0;
        ptx::fence_mbar_init();
    }
    if (warp == MMA_WARP) { ptx::tmem_alloc_pair(ptx::smem_addr(s_tmem), C::TMEM_COLS); ptx::tmem_relinquish_pair(); }
    if (warp == TMA_WARP && lane == 0) {
        ptx::prefetch_tensormap(&map_x);
        ptx::prefetch_tensormap(&map_w);
        ptx::prefetch_tensormap(&map_y);
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync();                     // the peer's barriers exist before anything arrives on them remotely
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *s_tmem;

    if (warp < EPI_WARPS) {
        // ------------------------------------------------------------ epilogue
        const int quarter = warp & 3, chalf = warp >> 2;   // TMEM lane quarter, column half
        unsigned char *stg = smem + C::OFF_STG + warp * STG_BYTES;
        const uint32_t stg_addr = sbase + C::OFF_STG + warp * STG_BYTES;
        float *s_ws = reinterpret_cast<float *>(smem + C::OFF_CH);          // [2][BN] per-channel scale of the tile
        float *s_bs = s_ws + ACC_BUFS * BN;                                   // [2][BN] bias as fp32
        const uint32_t leader_tempty = ptx::map_to_cta(bar_tempty, 0);
        bool alive = true;
        for (int t = 0; t < my_tiles; ++t) {
            const int tile = worker + t * workers;
            const int m0 = (tile / n_tiles) * (BM * CG) + (int)rank * BM + quarter * 32;
            const int nt0 = (tile % n_tiles) * BN;             // first channel of the tile
            const int n0 = nt0 + chalf * 128;                  // first channel of this warp's half
            const int b = t & 1;
            const int gm = m0 + lane;
            const bool row_ok = gm < M;
            const bool cols_ok = n0 < N;                       // N is a multiple of 128: a half tile is all in or all out
            // per-channel scale and bias of the tile -> shared memory; buffer b was last read two tiles ago,
            // and every epilogue warp has passed the group barrier of the tile in between since then
            gemmc::load_channel_params(s_ws + b * BN, s_bs + b * BN, w_scale, bias, nt0, N, threadIdx.x);   // 256 threads, one channel each
            // a_scale / 256: exact (power of two), cancels the factor 256 carried by the raw accumulator
            const float as = row_ok ? __fmul_rn(__ldg(a_scale + gm), 0.00390625f) : 0.0f;
            const uint64_t as2 = ptx::f32x2_pack(as, as);
            // the epilogue warps meet (named barrier 1: publishes s_ws / s_bs), then every warp polls the accumulator barrier itself
            asm volatile("bar.sync %0, %1;" ::"r"(1), "r"(EPI_WARPS * 32) : "memory");
            {
                int ok = 1;
                if (lane == 0) ok = (alive && ptx::mbar_wait(bar_tfull + 8 * b, (t >> 1) & 1, s_abort, status, QVGGT_DEV_TIMEOUT_ACCUM, 32)) ? 1 : 0;
                alive = __shfl_sync(0xFFFFFFFFu, ok, 0) != 0;
            }
            ptx::tc_fence_after_sync();
            if (alive) {
                const float *wsb = s_ws + b * BN + chalf * 128;
                const float *bsb = s_bs + b * BN + chalf * 128;
#pragma unroll 1
                for (int c = 0; c < 4; ++c) {
                    const int col = c * 32;                               // within this warp's 128 columns
                    uint32_t raw[32];
                    ptx::tmem_ld_32x32(tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + b * BN + chalf * 128 + col, raw);
                    ptx::tmem_ld_wait();
                    if (c == 3) {
                        // last read of this accumulator: hand it back to the MMA thread before the math
                        ptx::tc_fence_before_sync();
                        __syncwarp();
                        if (lane == 0) ptx::mbar_arrive_cluster(leader_tempty + 8 * b);
                    }
                    if (cols_ok) {
                        uint32_t out[16];
                        gemmc::scale_bias_bf16_x32(raw, as2, wsb + col, bsb + col, out);
                        gemmc::stage_row_32(stg, out, lane);
                        // the raw sums carry a factor 256 (codes in the high half-byte)
                        if (DUMP && acc_debug && row_ok) gemmc::dump_acc_x32<8>(acc_debug + (long long)gm * N + n0 + col, raw);
                        gemmc::store_staged_32x32(&map_y, stg_addr, n0 + col, m0, m0 < M, lane);
                    }
                }
            }
        }
        if (lane == 0) ptx::tma_store_wait_all();
    } else if (warp < MMA_WARP) {
        // ------------------------------------------------------------ converters
        gemmc::convert_packed_stages<C, true>(smem, warp - CONV_WARP0, lane, my_tiles * KB, bar_pfull, bar_pempty, bar_uempty,
                                              ptx::map_to_cta(bar_ufull, 0), s_abort, status, s_flags + 2,
                                              s_flags + 1 + 2 * CONV_WARPS, QVGGT_DEV_TIMEOUT_PACKED, QVGGT_DEV_TIMEOUT_EMPTY);
    } else if (warp == MMA_WARP) {
        // ------------------------------------------------------------ MMA issuer (one thread of the leader CTA)
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = ptx::idesc_i8(BM * CG, BN);
            bool alive = true;
            int us = 0;
            uint32_t uph = 0;
            for (int t = 0; t < my_tiles && alive; ++t) {
                const int b = t & 1;
                if (t >= ACC_BUFS) {
                    alive = ptx::mbar_wait_cluster(bar_tempty + 8 * b, ((t >> 1) - 1) & 1, s_abort, status, QVGGT_DEV_TIMEOUT_TMEM_FREE);
                    if (!alive) break;
                    ptx::tc_fence_after_sync();
                }
                const uint32_t d_tmem = tmem_base + b * BN;
                for (int kb = 0; kb < KB; ++kb) {
                    alive = ptx::mbar_wait_cluster(bar_ufull + 8 * us, uph, s_abort, status, QVGGT_DEV_TIMEOUT_FULL);
                    if (!alive) break;
                    ptx::tc_fence_after_sync();
                    const uint32_t a_addr = sbase + C::OFF_UP + us * C::UP_STAGE;
                    gemmc::mma_kblock_i8<true>(d_tmem, a_addr, a_addr + BM * BK, idesc, kb == 0);
                    ptx::mma_commit_pair(bar_uempty + 8 * us, 3);
                    if (++us == C::US) { us = 0; uph ^= 1; }
                }
                if (alive) ptx::mma_commit_pair(bar_tfull + 8 * b, 3);
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ TMA producer (one thread)
        if (lane == 0) {
            bool alive = true;
            int ps = 0;
            uint32_t pph = 0;
            int it = 0;
            for (int t = 0; t < my_tiles && alive; ++t) {
                const int tile = worker + t * workers;
                const int m0 = (tile / n_tiles) * (BM * CG) + (int)rank * BM;
                const int n0 = (tile % n_tiles) * BN + (int)rank * C::B_ROWS;
                for (int kb = 0; kb < KB; ++kb, ++it) {
                    if (it >= C::PS) {
                        alive = ptx::mbar_wait(bar_pempty + 8 * ps, pph ^ 1, s_abort, status, QVGGT_DEV_TIMEOUT_PACKED_FREE, 20);
                        if (!alive) break;
                    }
                    const uint32_t dst = sbase + C::OFF_PK + ps * C::PK_STAGE;
                    ptx::mbar_arrive_expect_tx(bar_pfull + 8 * ps, C::PK_STAGE);
                    ptx::tma_load_2d(&map_x, bar_pfull + 8 * ps, dst, kb * (BK / 2), m0);
                    ptx::tma_load_2d(&map_w, bar_pfull + 8 * ps, dst + BM * (BK / 2), kb * (BK / 2), n0);
                    if (++ps == C::PS) { ps = 0; pph ^= 1; }
                }
            }
        }
        __syncwarp();
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync();                     // no remote arrival or multicast commit may target a CTA that has exited
    if (warp == MMA_WARP) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc_pair(tmem_base, C::TMEM_COLS);
    }
}

template <bool DUMP>
cudaError_t launch(const qvggt_weights *w, const unsigned char *Xq, const float *a_scale, int M, void *Y, long long ldy,
                   int *acc_debug, cudaStream_t st)
{
    static QvggtPerDevice cache;
    int max_workers = 0;
    cudaError_t e = qvggt_configure_kernel(gemm_w4a4_kernel<DUMP>, THREADS, C::DYN_SMEM, CG, cache, &max_workers);
    if (e != cudaSuccess) return e;
    const int K = w->K, N = w->N;
    CUtensorMap map_x, map_w, map_y;
    if (!qvggt_make_map(&map_x, CU_TENSOR_MAP_DATA_TYPE_UINT8, Xq, K / 2, M, K / 2, BK / 2, BM, CU_TENSOR_MAP_SWIZZLE_NONE) ||
        !qvggt_make_map(&map_w, CU_TENSOR_MAP_DATA_TYPE_UINT8, w->Wq, K / 2, N, K / 2, BK / 2, C::B_ROWS, CU_TENSOR_MAP_SWIZZLE_NONE) ||
        !qvggt_make_map(&map_y, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, Y, N, M, (uint64_t)ldy * 2, 32, 32, CU_TENSOR_MAP_SWIZZLE_64B))
        return cudaErrorInvalidValue;
    const int total_tiles = ((M + BM * CG - 1) / (BM * CG)) * ((N + BN - 1) / BN);
    const int workers = total_tiles < max_workers ? total_tiles : max_workers;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(workers * CG);
    cfg.blockDim = dim3(THREADS);
    cfg.dynamicSmemBytes = C::DYN_SMEM;
    cfg.stream = st;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = CG; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, gemm_w4a4_kernel<DUMP>, map_x, map_w, map_y, a_scale, (const float *)w->w_scale,
                              (const uint16_t *)w->bias, acc_debug, M, N, K, w->status);
}

}  // namespace

cudaError_t qvggt_launch_gemm(const qvggt_weights *w, const unsigned char *Xq, const float *a_scale, int M, int group,
                              void *Y, long long ldy, int *acc_debug, cudaStream_t st)
{
    if (M == 0) return cudaSuccess;
    if (group == 128) return qvggt_launch_gemm_grouped(w, Xq, a_scale, M, Y, ldy, acc_debug, st);
    if (group != 0) return cudaErrorNotSupported;
    return acc_debug ? launch<true>(w, Xq, a_scale, M, Y, ldy, acc_debug, st) : launch<false>(w, Xq, a_scale, M, Y, ldy, acc_debug, st);
}
