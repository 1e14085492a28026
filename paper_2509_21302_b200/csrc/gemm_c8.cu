// W4A4 GEMM on codes held in 8-bit containers (Sec. 3.2: integer sum over the inner dimension, per-token and
// per-out-channel scales applied outside the sum), for sm_100a.
//
// tcgen05 has no 4-bit integer kind: whatever the storage format, the tensor core multiplies int8.  Here the
// producers already emit one code per byte (the quantize kernel for the activations, the offline weight
// preparation for the weights), so the tiles go from global memory straight into the 128-byte-swizzled operand
// stages by TMA and nothing in this kernel touches an operand byte with an ordinary instruction.  Per K-block
// a CTA's shared memory sees one TMA write and one tensor-core read of its 32 KB of operands, the minimum.
//
// Persistent and warp-specialised; a worker is a pair of CTAs on neighbouring SMs (tile 256 tokens x 256
// channels, each CTA stages 128 token rows and 128 weight rows; one thread of the leader CTA issues
// tcgen05.mma.cta_group::2.kind::i8 for both; accumulators int32 in tensor memory, two buffers of 256 columns).
//   warps 0..7   epilogue: TMEM -> registers -> scale, bias, bf16 -> swizzled staging -> TMA store
//   warp  8      one thread issues tcgen05.mma and the commits that release stages / publish accumulators
//   warp  9      one thread per CTA issues the TMA loads of its half of every operand stage; both CTAs signal
//                the leader's "full" barrier (cta_group::2 form of the load)
// The tiles are dealt round-robin to the workers.  (Cutting the tiles of a short last round into halves of 128
// channels was built and measured: an N = 128 MMA takes ~0.75 of an N = 256 one, a half tile ~0.9 of a whole
// one, and the extra bookkeeping cost the main path 5 %: not kept.)
// Every wait is bounded; on expiry the kernel records a code in *status and all roles fall through to the
// common exit, where tensor memory is released.
#include <cuda.h>
#include <cuda_bf16.h>

#include "gemm_common.cuh"
#include "qvggt_internal.cuh"
#include "sm100_ptx.cuh"
#include "tensor_map.cuh"
#include "unpack_w4.cuh"

namespace {

using gemmc::Ring;
using gemmc::STG_BYTES;

constexpr int BM = 128;            // token rows per CTA (TMEM lanes)
constexpr int BN = 256;            // output channels per whole tile
constexpr int BK = 128;            // codes along K per stage = one 128-byte swizzled row
constexpr int ACC_BUFS = 2;        // TMEM accumulators: the epilogue of tile i overlaps the MMAs of tile i+1
constexpr int EPI_WARPS = 8;       // warp w: TMEM lane quarter w % 4, column part w / 4
constexpr int MMA_WARP = EPI_WARPS;
constexpr int TMA_WARP = EPI_WARPS + 1;
constexpr int THREADS = (EPI_WARPS + 2) * 32;
constexpr int B_ROWS = BN / 2;                         // weight rows staged by one CTA for a whole tile
constexpr int STAGE = (BM + B_ROWS) * BK;              // 32 KB
constexpr int STAGES = 6;
constexpr int OFF_STG = STAGES * STAGE;                // operand stages first: they need 1024-byte alignment
constexpr int OFF_CH = OFF_STG + EPI_WARPS * STG_BYTES;          // per-channel scale and bias of two tiles, fp32
constexpr int OFF_BAR = OFF_CH + 2 * ACC_BUFS * BN * 4;          // full[STAGES] empty[STAGES] tfull[2] tempty[2]
constexpr int NBARS = 2 * STAGES + 2 * ACC_BUFS;
constexpr int OFF_TMEM = OFF_BAR + NBARS * 8;
constexpr int OFF_ABORT = OFF_TMEM + 4;
constexpr int OFF_FLAGS = OFF_ABORT + 4;
constexpr int SMEM_BYTES = OFF_FLAGS + 8;
constexpr int DYN_SMEM = SMEM_BYTES + 1024;            // slack to align the base to 1024 bytes
constexpr int TMEM_COLS = ACC_BUFS * BN;               // 512
static_assert(DYN_SMEM <= 232448, "exceeds the 227 KB of shared memory a CTA may use");
static_assert(2 * STAGE < (1 << 20), "transaction count of a stage must fit the barrier");

// DUMP: also write the int32 sums to acc_debug (its own instantiation keeps that code out of the production kernel).
// wait_limit: bound of every device-side wait, in cycles.  skip_loads: the TMA producers issue nothing, so that the
// first wait for operands runs out (used only to exercise the timeout path; no asynchronous operation is in flight).
template <bool DUMP>
__global__ void __launch_bounds__(THREADS, 1)
gemm_c8_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
               const __grid_constant__ CUtensorMap map_y,
               const float *__restrict__ a_scale, const float *__restrict__ w_scale, const uint16_t *__restrict__ bias,
               int *__restrict__ acc_debug, int M, int N, int K, int *status, long long wait_limit, int skip_loads)
{
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = ptx::smem_addr(smem);
    const uint32_t bar_full = sbase + OFF_BAR;
    const uint32_t bar_empty = bar_full + STAGES * 8;
    const uint32_t bar_tfull = bar_empty + STAGES * 8;
    const uint32_t bar_tempty = bar_tfull + ACC_BUFS * 8;
    uint32_t *s_tmem = reinterpret_cast<uint32_t *>(smem + OFF_TMEM);
    volatile int *s_abort = reinterpret_cast<volatile int *>(smem + OFF_ABORT);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank();                       // 0 = leader of the pair
    const int worker = blockIdx.x / 2, workers = gridDim.x / 2;
    const int KB = K / BK;
    const int n_tiles = (N + BN - 1) / BN;
    const int total_tiles = ((M + 2 * BM - 1) / (2 * BM)) * n_tiles;
    const int my_tiles = (total_tiles > worker) ? (total_tiles - 1 - worker) / workers + 1 : 0;

    if (threadIdx.x == 0) {
        gemmc::init_barriers(bar_full, STAGES, 1);                     // the leader's arrive.expect_tx (bytes of both CTAs)
        gemmc::init_barriers(bar_empty, STAGES, 1);                    // tcgen05.commit
        gemmc::init_barriers(bar_tfull, ACC_BUFS, 1);                  // tcgen05.commit
        gemmc::init_barriers(bar_tempty, ACC_BUFS, EPI_WARPS * 2);     // the epilogue warps of both CTAs
        *s_abort = 0;
        ptx::fence_mbar_init();
    }
    if (warp == MMA_WARP) { ptx::tmem_alloc_pair(ptx::smem_addr(s_tmem), TMEM_COLS); ptx::tmem_relinquish_pair(); }
    if (warp == TMA_WARP && lane == 0) {
        ptx::prefetch_tensormap(&map_x);
        ptx::prefetch_tensormap(&map_w);
        ptx::prefetch_tensormap(&map_y);
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync();                     // the leader's barriers exist before the peer's loads signal them
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *s_tmem;
    // everything above touched only kernel parameters and on-chip state: it may overlap the tail of the previous
    // kernel in the stream; the operands (and the output buffer) may not be touched before that kernel is done
    ptx::grid_launch_dependents();
    ptx::grid_dependency_wait();

    if (warp < EPI_WARPS) {
        // ------------------------------------------------------------ epilogue
        const int quarter = warp & 3, cpart = warp >> 2;   // TMEM lane quarter, column part
        unsigned char *stg = smem + OFF_STG + warp * STG_BYTES;
        const uint32_t stg_addr = sbase + OFF_STG + warp * STG_BYTES;
        float *s_ws = reinterpret_cast<float *>(smem + OFF_CH);             // [2][BN] per-channel scale of the tile
        float *s_bs = s_ws + ACC_BUFS * BN;                                  // [2][BN] bias as fp32
        const uint32_t leader_tempty = ptx::map_to_cta(bar_tempty, 0);
        bool alive = true;
        constexpr int CW = BN / 2, NCH = CW / 32;              // columns and 32-column chunks of one warp's part
        for (int t = 0; t < my_tiles; ++t) {
            const int tile = worker + t * workers;
            const int m0 = (tile / n_tiles) * (2 * BM) + (int)rank * BM + quarter * 32;
            const int nt0 = (tile % n_tiles) * BN;             // first channel of the tile
            const int n0 = nt0 + cpart * CW;                   // first channel of this warp's part
            const int b = t & 1;
            const int gm = m0 + lane;
            const bool row_ok = gm < M;
            const bool cols_ok = n0 < N;                       // N is a multiple of 128: a part is all in or all out
            // per-channel scale and bias of the tile -> shared memory; buffer b was last read two tiles ago,
            // and every epilogue warp has passed the group barrier of the tile in between since then
            gemmc::load_channel_params(s_ws + b * BN, s_bs + b * BN, w_scale, bias, nt0, N, threadIdx.x);
            const float as = row_ok ? __ldg(a_scale + gm) : 0.0f;
            const uint64_t as2 = ptx::f32x2_pack(as, as);
            // the epilogue warps meet (named barrier 1: publishes s_ws / s_bs), then every warp polls the accumulator barrier itself
            asm volatile("bar.sync %0, %1;" ::"r"(1), "r"(EPI_WARPS * 32) : "memory");
            {
                int ok = 1;
                if (lane == 0) ok = (alive && ptx::mbar_wait(bar_tfull + 8 * b, (t >> 1) & 1, s_abort, status, QVGGT_DEV_TIMEOUT_ACCUM, 32, wait_limit)) ? 1 : 0;
                alive = __shfl_sync(0xFFFFFFFFu, ok, 0) != 0;
            }
            ptx::tc_fence_after_sync();
            if (alive) {
                const float *wsb = s_ws + b * BN + cpart * CW;
                const float *bsb = s_bs + b * BN + cpart * CW;
                // the warp's whole share of the accumulator goes to registers first, so that tensor memory is
                // handed back to the MMA thread a few hundred cycles after the tile completed, not after the
                // conversions and stores of the first chunks
                uint32_t raw[NCH][32];
#pragma unroll
                for (int c = 0; c < NCH; ++c)
                    ptx::tmem_ld_32x32(tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + b * BN + cpart * CW + c * 32, raw[c]);
                ptx::tmem_ld_wait();
                ptx::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive_cluster(leader_tempty + 8 * b);
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
                    const int col = c * 32;                               // within this warp's columns
                    if (cols_ok) {
                        uint32_t out[16];
                        gemmc::scale_bias_bf16_x32(raw[c], as2, wsb + col, bsb + col, out);
                        gemmc::stage_row_32(stg, out, lane);
                        if (DUMP && acc_debug && row_ok) gemmc::dump_acc_x32<0>(acc_debug + (long long)gm * N + n0 + col, raw[c]);
                        gemmc::store_staged_32x32(&map_y, stg_addr, n0 + col, m0, m0 < M, lane);
                    }
                }
            }
        }
        // the staging tiles must outlive the stores' reads; the writes themselves are complete when the grid is
        if (lane == 0) ptx::tma_store_wait_read<0>();
    } else if (warp == MMA_WARP) {
        // ------------------------------------------------------------ MMA issuer (one thread of the leader CTA)
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = ptx::idesc_i8(2 * BM, BN);
            bool alive = true;
            Ring r;
            for (int t = 0; t < my_tiles && alive; ++t) {
                const int b = t & 1;
                if (t >= ACC_BUFS) {
                    alive = ptx::mbar_wait_cluster(bar_tempty + 8 * b, ((t >> 1) - 1) & 1, s_abort, status, QVGGT_DEV_TIMEOUT_TMEM_FREE, wait_limit);
                    if (!alive) break;
                    ptx::tc_fence_after_sync();
                }
                const uint32_t d_tmem = tmem_base + b * BN;
                for (int kb = 0; kb < KB; ++kb) {
                    alive = ptx::mbar_wait_cluster(bar_full + 8 * r.s, r.ph, s_abort, status, QVGGT_DEV_TIMEOUT_FULL, wait_limit);
                    if (!alive) break;
                    ptx::tc_fence_after_sync();
                    const uint32_t a_addr = sbase + r.s * STAGE;
                    gemmc::mma_kblock_i8<true>(d_tmem, a_addr, a_addr + BM * BK, idesc, kb == 0);
                    ptx::mma_commit_pair(bar_empty + 8 * r.s, 3);      // frees the stage in both CTAs
                    r.advance(STAGES);
                }
                if (alive) ptx::mma_commit_pair(bar_tfull + 8 * b, 3);
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ TMA producer (one thread per CTA)
        if (lane == 0 && !skip_loads) {
            const uint32_t leader_full = ptx::map_to_cta(bar_full, 0);
            bool alive = true;
            Ring r;
            int it = 0;
            for (int t = 0; t < my_tiles && alive; ++t) {
                const int tile = worker + t * workers;
                const int m0 = (tile / n_tiles) * (2 * BM) + (int)rank * BM;
                const int n0 = (tile % n_tiles) * BN + (int)rank * B_ROWS;
                for (int kb = 0; kb < KB; ++kb, ++it) {
                    if (it >= STAGES) {
                        alive = ptx::mbar_wait(bar_empty + 8 * r.s, r.ph ^ 1, s_abort, status, QVGGT_DEV_TIMEOUT_EMPTY, 20, wait_limit);
                        if (!alive) break;
                    }
                    const uint32_t dst = sbase + r.s * STAGE;
                    // the leader's barrier expects the bytes of both CTAs; the peer's completions may arrive first
                    // (the count goes negative for a while), the phase cannot end before the leader has arrived
                    if (rank == 0) ptx::mbar_arrive_expect_tx(bar_full + 8 * r.s, 2 * STAGE);
                    ptx::tma_load_2d_pair(&map_x, leader_full + 8 * r.s, dst, kb * BK, m0);
                    ptx::tma_load_2d_pair(&map_w, leader_full + 8 * r.s, dst + BM * BK, kb * BK, n0);
                    r.advance(STAGES);
                }
            }
        }
        __syncwarp();
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync();        // no remote arrival or multicast commit may target a CTA that has exited
    if (warp == MMA_WARP) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc_pair(tmem_base, TMEM_COLS);
    }
}

// ------------------------------------------------------------------------------------------------
// The same TMA-fed CTA-pair design for one activation scale per token per 128 rotated channels (an extension of the
// paper's token-wise granularity; the weights keep one scale per output channel).  A K-block of 128 codes is one scale
// group, so every K-block accumulates into its own tensor-memory buffer (two of 128 columns, ping-pong) and the
// epilogue warps rescale it while the next one runs:
//   s = fl(s + fl(float(acc_g) * a_scale[m][g])), g ascending;  Y = bf16(fl(fl(s * w_scale[n]) + bias[n])).
// Tile 256 tokens x 128 channels per pair; an epilogue thread keeps the 64 running sums of its row in registers (10
// warps per CTA leave 168 registers per thread).  Per K-block the pair does 376 cycles of MMA work (four N = 128
// instructions) against 3 instructions per output element in the epilogue: the epilogue sets the pace.
namespace grp {

constexpr int GN = 128;                                // channels per tile
constexpr int GEPI = 16;                               // epilogue warps: lane quarter w % 4, 32-column part w / 4 (four per scheduler: the
                                                       // epilogue is latency-bound, cf. 1400 against 2400 cycles per K-block with eight)
constexpr int G_MMA_WARP = GEPI, G_TMA_WARP = GEPI + 1;
constexpr int GTHREADS = (GEPI + 2) * 32;
constexpr int GB_ROWS = GN / 2;                        // weight rows staged by one CTA
constexpr int GSTAGE = (BM + GB_ROWS) * BK;            // 24 KB
constexpr int GACC = 4;                                // accumulators of 128 columns (a ring of four instead of two: 5-8 % faster)
constexpr int GSTAGES = 7;
constexpr int OFF_STG = GSTAGES * GSTAGE;
constexpr int OFF_CH = OFF_STG + GEPI * STG_BYTES;          // [2][GN] channel scales, [2][GN] bias, fp32
constexpr int OFF_BAR = OFF_CH + 2 * 2 * GN * 4;                 // full[GSTAGES] empty[GSTAGES] tfull[2] tempty[2]
constexpr int NBARS = 2 * GSTAGES + 2 * GACC;
constexpr int OFF_TMEM = OFF_BAR + NBARS * 8;
constexpr int OFF_ABORT = OFF_TMEM + 4;
constexpr int OFF_FLAGS = OFF_ABORT + 4;
constexpr int DYN_SMEM = OFF_FLAGS + 8 + 1024;
constexpr int TMEM_COLS = GACC * GN;                              // 512
static_assert(DYN_SMEM <= 232448, "exceeds the 227 KB of shared memory a CTA may use");
static_assert(GSTAGE % 1024 == 0, "operand tiles must stay 1024-byte aligned");

template <bool DUMP>
__global__ void __launch_bounds__(GTHREADS, 1)
gemm_c8_grouped_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                       const __grid_constant__ CUtensorMap map_y, const float *__restrict__ a_scale,
                       const float *__restrict__ w_scale, const uint16_t *__restrict__ bias, int *__restrict__ acc_debug,
                       int M, int N, int K, int *status)
{
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = ptx::smem_addr(smem);
    const uint32_t bar_full = sbase + OFF_BAR;
    const uint32_t bar_empty = bar_full + GSTAGES * 8;
    const uint32_t bar_tfull = bar_empty + GSTAGES * 8;
    const uint32_t bar_tempty = bar_tfull + GACC * 8;
    uint32_t *s_tmem = reinterpret_cast<uint32_t *>(smem + OFF_TMEM);
    volatile int *s_abort = reinterpret_cast<volatile int *>(smem + OFF_ABORT);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank();
    const int worker = blockIdx.x / 2, workers = gridDim.x / 2;
    const int KB = K / BK;                                   // = number of scale groups
    const int n_tiles = N / GN;
    const int total_tiles = ((M + 2 * BM - 1) / (2 * BM)) * n_tiles;
    const int my_tiles = (total_tiles > worker) ? (total_tiles - 1 - worker) / workers + 1 : 0;

    if (threadIdx.x == 0) {
        gemmc::init_barriers(bar_full, GSTAGES, 1);
        gemmc::init_barriers(bar_empty, GSTAGES, 1);
        gemmc::init_barriers(bar_tfull, GACC, 1);
        gemmc::init_barriers(bar_tempty, GACC, GEPI * 2);
        *s_abort = 0;
        ptx::fence_mbar_init();
    }
    if (warp == G_MMA_WARP) { ptx::tmem_alloc_pair(ptx::smem_addr(s_tmem), TMEM_COLS); ptx::tmem_relinquish_pair(); }
    if (warp == G_TMA_WARP && lane == 0) {
        ptx::prefetch_tensormap(&map_x);
        ptx::prefetch_tensormap(&map_w);
        ptx::prefetch_tensormap(&map_y);
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *s_tmem;
    ptx::grid_launch_dependents();
    ptx::grid_dependency_wait();

    if (warp < GEPI) {
        // ------------------------------------------------------------ epilogue
        const int quarter = warp & 3, cpart = warp >> 2;   // TMEM lane quarter, 32-column part
        unsigned char *stg = smem + OFF_STG + warp * STG_BYTES;
        const uint32_t stg_addr = sbase + OFF_STG + warp * STG_BYTES;
        float *s_ws = reinterpret_cast<float *>(smem + OFF_CH);    // [2][GN]
        float *s_bs = s_ws + 2 * GN;                                // [2][GN]
        const uint32_t leader_tempty = ptx::map_to_cta(bar_tempty, 0);
        const uint32_t lane_base = static_cast<uint32_t>(quarter * 32) << 16;
        bool alive = true;
        int it = 0;                                                 // K-blocks seen so far (all tiles)
        for (int t = 0; t < my_tiles; ++t) {
            const int tile = worker + t * workers;
            const int m0 = (tile / n_tiles) * (2 * BM) + (int)rank * BM + quarter * 32;
            const int nt0 = (tile % n_tiles) * GN;
            const int n0 = nt0 + cpart * 32;
            const int tb = t & 1;
            const int gm = m0 + lane;
            const bool row_ok = gm < M;
            // buffer tb was last read two tiles ago; every epilogue warp has passed a group barrier since
            if (threadIdx.x < GN) gemmc::load_channel_params(s_ws + tb * GN, s_bs + tb * GN, w_scale, bias, nt0, N, threadIdx.x);
            float sum[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) sum[j] = 0.0f;
            // the group's scale is fetched one K-block ahead (it comes from L2)
            float as_next = row_ok ? __ldg(a_scale + (long long)gm * KB) : 0.0f;
#pragma unroll 1
            for (int kb = 0; kb < KB; ++kb, ++it) {
                const int b = it % GACC;
                const float as = as_next;
                if (kb + 1 < KB && row_ok) as_next = __ldg(a_scale + (long long)gm * KB + kb + 1);
                {   // every warp polls for itself (lane 0; the warp follows): no warp waits for a slower one between K-blocks
                    int ok = 1;
                    if (lane == 0) ok = (alive && ptx::mbar_wait(bar_tfull + 8 * b, (it / GACC) & 1, s_abort, status, QVGGT_DEV_TIMEOUT_ACCUM, 20)) ? 1 : 0;
                    alive = __shfl_sync(0xFFFFFFFFu, ok, 0) != 0;
                }
                ptx::tc_fence_after_sync();
                if (!alive) continue;
                uint32_t raw[32];
                ptx::tmem_ld_32x32(tmem_base + lane_base + b * GN + cpart * 32, raw);
                ptx::tmem_ld_wait();
                ptx::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive_cluster(leader_tempty + 8 * b);
                // two elements per multiply (one issue slot for two IEEE multiplications); the additions stay scalar: a packed
                // multiply feeding a packed add was seen contracted into one fused operation, one rounding instead of two
                const uint64_t as2 = ptx::f32x2_pack(as, as);
#pragma unroll
                for (int j = 0; j < 32; j += 2) {
                    float p0, p1;
                    ptx::f32x2_unpack(ptx::f32x2_mul(ptx::f32x2_pack(static_cast<float>(static_cast<int>(raw[j])), static_cast<float>(static_cast<int>(raw[j + 1]))), as2), p0, p1);
                    sum[j] = __fadd_rn(sum[j], p0);
                    sum[j + 1] = __fadd_rn(sum[j + 1], p1);
                }
                if (DUMP && acc_debug && row_ok) gemmc::dump_acc_x32<0>(acc_debug + ((long long)kb * M + gm) * N + n0, raw);
            }
            // once per tile the epilogue warps meet: publishes s_ws / s_bs of this tile and orders their reuse two tiles on
            asm volatile("bar.sync %0, %1;" ::"r"(1), "r"(GEPI * 32) : "memory");
            if (alive) {
                const float *wsb = s_ws + tb * GN + cpart * 32;
                const float *bsb = s_bs + tb * GN + cpart * 32;
                uint32_t out[16];
#pragma unroll
                for (int j = 0; j < 32; j += 2) {
                    const float z0 = __fadd_rn(__fmul_rn(sum[j], wsb[j]), bsb[j]);
                    const float z1 = __fadd_rn(__fmul_rn(sum[j + 1], wsb[j + 1]), bsb[j + 1]);
                    out[j >> 1] = ptx::pack_bf16x2(z0, z1);
                }
                gemmc::stage_row_32(stg, out, lane);
                gemmc::store_staged_32x32(&map_y, stg_addr, n0, m0, m0 < M, lane);
            }
        }
        if (lane == 0) ptx::tma_store_wait_read<0>();
    } else if (warp == G_MMA_WARP) {
        // ------------------------------------------------------------ MMA issuer: one accumulator per K-block
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = ptx::idesc_i8(2 * BM, GN);
            bool alive = true;
            Ring r;
            const int total_kb = my_tiles * KB;
            for (int it = 0; it < total_kb && alive; ++it) {
                const int b = it % GACC;
                if (it >= GACC) {
                    alive = ptx::mbar_wait_cluster(bar_tempty + 8 * b, ((it / GACC) - 1) & 1, s_abort, status, QVGGT_DEV_TIMEOUT_TMEM_FREE);
                    if (!alive) break;
                    ptx::tc_fence_after_sync();
                }
                alive = ptx::mbar_wait_cluster(bar_full + 8 * r.s, r.ph, s_abort, status, QVGGT_DEV_TIMEOUT_FULL);
                if (!alive) break;
                ptx::tc_fence_after_sync();
                const uint32_t a_addr = sbase + r.s * GSTAGE;
                gemmc::mma_kblock_i8<true>(tmem_base + b * GN, a_addr, a_addr + BM * BK, idesc, true);
                ptx::mma_commit_pair(bar_empty + 8 * r.s, 3);
                ptx::mma_commit_pair(bar_tfull + 8 * b, 3);
                r.advance(GSTAGES);
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ TMA producer (one thread per CTA)
        if (lane == 0) {
            const uint32_t leader_full = ptx::map_to_cta(bar_full, 0);
            bool alive = true;
            Ring r;
            int it = 0;
            for (int t = 0; t < my_tiles && alive; ++t) {
                const int tile = worker + t * workers;
                const int m0 = (tile / n_tiles) * (2 * BM) + (int)rank * BM;
                const int n0 = (tile % n_tiles) * GN + (int)rank * GB_ROWS;
                for (int kb = 0; kb < KB; ++kb, ++it) {
                    if (it >= GSTAGES) {
                        alive = ptx::mbar_wait(bar_empty + 8 * r.s, r.ph ^ 1, s_abort, status, QVGGT_DEV_TIMEOUT_EMPTY, 20);
                        if (!alive) break;
                    }
                    const uint32_t dst = sbase + r.s * GSTAGE;
                    if (rank == 0) ptx::mbar_arrive_expect_tx(bar_full + 8 * r.s, 2 * GSTAGE);
                    ptx::tma_load_2d_pair(&map_x, leader_full + 8 * r.s, dst, kb * BK, m0);
                    ptx::tma_load_2d_pair(&map_w, leader_full + 8 * r.s, dst + BM * BK, kb * BK, n0);
                    r.advance(GSTAGES);
                }
            }
        }
        __syncwarp();
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync();
    if (warp == G_MMA_WARP) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc_pair(tmem_base, TMEM_COLS);
    }
}

template <bool DUMP>
cudaError_t launch(const qvggt_weights *w, const signed char *Xq8, const float *a_scale, int M, void *Y, long long ldy,
                   int *acc_debug, cudaStream_t st)
{
    static QvggtPerDevice cache;
    int max_workers = 0;
    cudaError_t e = qvggt_configure_kernel(gemm_c8_grouped_kernel<DUMP>, GTHREADS, DYN_SMEM, 2, cache, &max_workers);
    if (e != cudaSuccess) return e;
    const int K = w->K, N = w->N;
    CUtensorMap map_x, map_w, map_y;
    if (!qvggt_make_map(&map_x, CU_TENSOR_MAP_DATA_TYPE_UINT8, Xq8, K, M, K, BK, BM, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !qvggt_make_map(&map_w, CU_TENSOR_MAP_DATA_TYPE_UINT8, w->Wq8, K, N, K, BK, GB_ROWS, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !qvggt_make_map(&map_y, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, Y, N, M, (uint64_t)ldy * 2, 32, 32, CU_TENSOR_MAP_SWIZZLE_64B))
        return cudaErrorInvalidValue;
    const int total_tiles = ((M + 2 * BM - 1) / (2 * BM)) * (N / GN);
    const int workers = total_tiles < max_workers ? total_tiles : max_workers;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(workers * 2);
    cfg.blockDim = dim3(GTHREADS);
    cfg.dynamicSmemBytes = DYN_SMEM;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, gemm_c8_grouped_kernel<DUMP>, map_x, map_w, map_y, a_scale, (const float *)w->w_scale,
                              (const uint16_t *)w->bias, acc_debug, M, N, K, w->status);
}

}  // namespace grp

// Packed weight codes [N, K/2] (byte i = code 2i in bits 0-3, code 2i+1 in bits 4-7, two's complement) -> one code per
// byte [N, K], 16 packed bytes per thread.  Used when the handle keeps only the packed codes: the unpacked copy is a
// per-launch scratch of a few megabytes that the GEMM behind it reads back from L2.
__global__ void __launch_bounds__(256) unpack_w4_kernel(const uint4 *__restrict__ packed, uint4 *__restrict__ out, long long n16)
{
    ptx::grid_launch_dependents();
    ptx::grid_dependency_wait();           // the scratch may still be read by the previous GEMM of the stream
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n16) return;
    qvggt_unpack_w4_item(packed, out, i);
}

template <bool DUMP>
cudaError_t launch(const qvggt_weights *w, const signed char *wq8, const signed char *Xq8, const float *a_scale, int M, void *Y, long long ldy,
                   int *acc_debug, cudaStream_t st, long long wait_limit, int skip_loads)
{
    static QvggtPerDevice cache;
    int max_workers = 0;
    cudaError_t e = qvggt_configure_kernel(gemm_c8_kernel<DUMP>, THREADS, DYN_SMEM, 2, cache, &max_workers);
    if (e != cudaSuccess) return e;
    const int K = w->K, N = w->N;
    CUtensorMap map_x, map_w, map_y;
    if (!qvggt_make_map(&map_x, CU_TENSOR_MAP_DATA_TYPE_UINT8, Xq8, K, M, K, BK, BM, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !qvggt_make_map(&map_w, CU_TENSOR_MAP_DATA_TYPE_UINT8, wq8, K, N, K, BK, B_ROWS, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !qvggt_make_map(&map_y, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, Y, N, M, (uint64_t)ldy * 2, 32, 32, CU_TENSOR_MAP_SWIZZLE_64B))
        return cudaErrorInvalidValue;
    const int total_tiles = ((M + 2 * BM - 1) / (2 * BM)) * ((N + BN - 1) / BN);
    const int workers = total_tiles < max_workers ? total_tiles : max_workers;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;      // see grid_dependency_wait()
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(workers * 2);
    cfg.blockDim = dim3(THREADS);
    cfg.dynamicSmemBytes = DYN_SMEM;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, gemm_c8_kernel<DUMP>, map_x, map_w, map_y, a_scale, (const float *)w->w_scale,
                              (const uint16_t *)w->bias, acc_debug, M, N, K, w->status, wait_limit, skip_loads);
}

}  // namespace

cudaError_t qvggt_launch_gemm_c8(const qvggt_weights *w, const signed char *Xq8, const float *a_scale, int M, void *Y,
                                 long long ldy, int *acc_debug, cudaStream_t st)
{
    if (M == 0) return cudaSuccess;
    if (!w->Wq8) return cudaErrorNotSupported;      // the handle was prepared without the 8-bit-container copy
    return acc_debug ? launch<true>(w, w->Wq8, Xq8, a_scale, M, Y, ldy, acc_debug, st, ptx::kWaitLimitCycles, 0)
                     : launch<false>(w, w->Wq8, Xq8, a_scale, M, Y, ldy, acc_debug, st, ptx::kWaitLimitCycles, 0);
}

cudaError_t qvggt_launch_unpack_w4(const qvggt_weights *w, signed char *w_scratch, cudaStream_t st)
{
    if (!w->Wq) return cudaErrorNotSupported;       // the handle holds no packed codes
    const long long n16 = (long long)w->N * w->K / 32;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((n16 + 255) / 256));
    cfg.blockDim = dim3(256);
    cfg.stream = st;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, unpack_w4_kernel, reinterpret_cast<const uint4 *>(w->Wq), reinterpret_cast<uint4 *>(w_scratch), n16);
}

cudaError_t qvggt_launch_gemm_c8_packed_weights(const qvggt_weights *w, const signed char *Xq8, const float *a_scale, int M, void *Y,
                                                long long ldy, signed char *w_scratch, int *acc_debug, cudaStream_t st)
{
    if (M == 0) return cudaSuccess;
    cudaError_t e = qvggt_launch_unpack_w4(w, w_scratch, st);
    if (e != cudaSuccess) return e;
    return acc_debug ? launch<true>(w, w_scratch, Xq8, a_scale, M, Y, ldy, acc_debug, st, ptx::kWaitLimitCycles, 0)
                     : launch<false>(w, w_scratch, Xq8, a_scale, M, Y, ldy, acc_debug, st, ptx::kWaitLimitCycles, 0);
}

cudaError_t qvggt_launch_gemm_c8_expanded(const qvggt_weights *w, const signed char *Xq8, const float *a_scale, int M, void *Y,
                                          long long ldy, const signed char *w_expanded, int *acc_debug, cudaStream_t st)
{
    if (M == 0) return cudaSuccess;
    return acc_debug ? launch<true>(w, w_expanded, Xq8, a_scale, M, Y, ldy, acc_debug, st, ptx::kWaitLimitCycles, 0)
                     : launch<false>(w, w_expanded, Xq8, a_scale, M, Y, ldy, acc_debug, st, ptx::kWaitLimitCycles, 0);
}

cudaError_t qvggt_launch_gemm_c8_starved(const qvggt_weights *w, const signed char *Xq8, const float *a_scale, int M, void *Y,
                                         long long ldy, long long wait_limit_cycles, cudaStream_t st)
{
    if (M == 0) return cudaSuccess;
    if (!w->Wq8) return cudaErrorNotSupported;
    return launch<false>(w, w->Wq8, Xq8, a_scale, M, Y, ldy, nullptr, st, wait_limit_cycles, 1);
}

cudaError_t qvggt_launch_gemm_c8_grouped(const qvggt_weights *w, const signed char *Xq8, const float *a_scale, int M, void *Y,
                                         long long ldy, int *acc_debug, cudaStream_t st)
{
    if (M == 0) return cudaSuccess;
    if (!w->Wq8 || w->bits != 4) return cudaErrorNotSupported;
    return acc_debug ? grp::launch<true>(w, Xq8, a_scale, M, Y, ldy, acc_debug, st) : grp::launch<false>(w, Xq8, a_scale, M, Y, ldy, acc_debug, st);
}
