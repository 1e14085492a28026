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
//   warps 0..E-1  epilogue: TMEM -> registers -> scale, bias, bf16 -> swizzled staging -> TMA store
//   warp  E       one thread issues tcgen05.mma and the commits that release stages / publish accumulators
//   warp  E+1     one thread per CTA issues the TMA loads of its half of every operand stage; both CTAs signal
//                 the leader's "full" barrier (cta_group::2 form of the load)
// Every wait is bounded; on expiry the kernel records a code in *status and all roles fall through to the
// common exit, where tensor memory is released.
#include <cuda.h>
#include <cuda_bf16.h>

#include "qvggt_internal.cuh"
#include "sm100_ptx.cuh"
#include "tensor_map.cuh"

namespace {

constexpr int BM = 128;            // token rows per CTA (TMEM lanes)
constexpr int BN = 256;            // output channels per tile
constexpr int BK = 128;            // codes along K per stage = one 128-byte swizzled row
constexpr int ACC_BUFS = 2;        // TMEM accumulators: the epilogue of tile i overlaps the MMAs of tile i+1
constexpr int STG_BYTES = 32 * 64; // per epilogue warp: 32 rows x 32 bf16, 64-byte swizzled

template <int EPI_WARPS>
struct Cfg {
    static constexpr int MMA_WARP = EPI_WARPS;
    static constexpr int TMA_WARP = EPI_WARPS + 1;
    static constexpr int THREADS = (EPI_WARPS + 2) * 32;
    static constexpr int COL_PARTS = EPI_WARPS / 4;            // warp w: TMEM lane quarter w % 4, column part w / 4
    static constexpr int CW = BN / COL_PARTS;                  // columns per epilogue warp
    static constexpr int B_ROWS = BN / 2;                      // weight rows staged by one CTA
    static constexpr int STAGE = (BM + B_ROWS) * BK;           // 32 KB
    static constexpr int STAGES = (EPI_WARPS == 16) ? 5 : 6;
    static constexpr int OFF_STG = STAGES * STAGE;             // operand stages first: they need 1024-byte alignment
    static constexpr int OFF_CH = OFF_STG + EPI_WARPS * STG_BYTES;   // per-channel scale and bias of two tiles, fp32
    static constexpr int OFF_BAR = OFF_CH + 2 * ACC_BUFS * BN * 4;   // full[STAGES] empty[STAGES] tfull[2] tempty[2]
    static constexpr int NBARS = 2 * STAGES + 2 * ACC_BUFS;
    static constexpr int OFF_TMEM = OFF_BAR + NBARS * 8;
    static constexpr int OFF_ABORT = OFF_TMEM + 4;
    static constexpr int OFF_FLAGS = OFF_ABORT + 4;
    static constexpr int BYTES = OFF_FLAGS + 8;
    static constexpr int DYN_SMEM = BYTES + 1024;              // slack to align the base to 1024 bytes
    static constexpr int TMEM_COLS = ACC_BUFS * BN;            // 512
    static_assert(DYN_SMEM <= 232448, "exceeds the 227 KB of shared memory a CTA may use");
    static_assert(2 * STAGE < (1 << 20), "transaction count of a stage must fit the barrier");
};

template <int EPI_WARPS, bool DUMP>
__global__ void __launch_bounds__(Cfg<EPI_WARPS>::THREADS, 1)
gemm_c8_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
               const __grid_constant__ CUtensorMap map_y, const float *__restrict__ a_scale,
               const float *__restrict__ w_scale, const uint16_t *__restrict__ bias, int *__restrict__ acc_debug,
               int M, int N, int K, int *status)
{
    using C = Cfg<EPI_WARPS>;
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = ptx::smem_addr(smem);
    const uint32_t bar_full = sbase + C::OFF_BAR;
    const uint32_t bar_empty = bar_full + C::STAGES * 8;
    const uint32_t bar_tfull = bar_empty + C::STAGES * 8;
    const uint32_t bar_tempty = bar_tfull + ACC_BUFS * 8;
    uint32_t *s_tmem = reinterpret_cast<uint32_t *>(smem + C::OFF_TMEM);
    volatile int *s_abort = reinterpret_cast<volatile int *>(smem + C::OFF_ABORT);
    volatile int *s_flags = reinterpret_cast<volatile int *>(smem + C::OFF_FLAGS);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank();                       // 0 = leader of the pair
    const int worker = blockIdx.x / 2, workers = gridDim.x / 2;
    const int KB = K / BK;
    const int n_tiles = (N + BN - 1) / BN;
    const int total_tiles = ((M + 2 * BM - 1) / (2 * BM)) * n_tiles;
    const int my_tiles = (total_tiles > worker) ? (total_tiles - 1 - worker) / workers + 1 : 0;

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::STAGES; ++s) {
            ptx::mbar_init(bar_full + 8 * s, 1);                       // the leader's arrive.expect_tx (bytes of both CTAs)
            ptx::mbar_init(bar_empty + 8 * s, 1);                      // tcgen05.commit
        }
        for (int b = 0; b < ACC_BUFS; ++b) {
            ptx::mbar_init(bar_tfull + 8 * b, 1);                      // tcgen05.commit
            ptx::mbar_init(bar_tempty + 8 * b, EPI_WARPS * 2);         // the epilogue warps of both CTAs
        }
        *s_abort = 0;
        ptx::fence_mbar_init();
    }
    if (warp == C::MMA_WARP) { ptx::tmem_alloc_pair(ptx::smem_addr(s_tmem), C::TMEM_COLS); ptx::tmem_relinquish_pair(); }
    if (warp == C::TMA_WARP && lane == 0) {
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
        unsigned char *stg = smem + C::OFF_STG + warp * STG_BYTES;
        const uint32_t stg_addr = sbase + C::OFF_STG + warp * STG_BYTES;
        float *s_ws = reinterpret_cast<float *>(smem + C::OFF_CH);          // [2][BN] per-channel scale of the tile
        float *s_bs = s_ws + ACC_BUFS * BN;                                   // [2][BN] bias as fp32
        const uint32_t leader_tempty = ptx::map_to_cta(bar_tempty, 0);
        bool alive = true;
        uint32_t toggle = 0;
        for (int t = 0; t < my_tiles; ++t) {
            const int tile = worker + t * workers;
            const int m0 = (tile / n_tiles) * (2 * BM) + (int)rank * BM + quarter * 32;
            const int nt0 = (tile % n_tiles) * BN;             // first channel of the tile
            const int n0 = nt0 + cpart * C::CW;                // first channel of this warp's part
            const int b = t & 1;
            const int gm = m0 + lane;
            const bool row_ok = gm < M;
            const bool cols_ok = n0 < N;                       // N is a multiple of 128 (and of CW): a part is all in or all out
            // per-channel scale and bias of the tile -> shared memory; buffer b was last read two tiles ago,
            // and every epilogue warp has passed the group barrier of the tile in between since then
            if (threadIdx.x < BN) {
                const int e = threadIdx.x;
                const bool ch_ok = nt0 + e < N;
                s_ws[b * BN + e] = ch_ok ? __ldg(w_scale + nt0 + e) : 0.0f;
                s_bs[b * BN + e] = (ch_ok && bias) ? __uint_as_float(static_cast<uint32_t>(__ldg(bias + nt0 + e)) << 16) : 0.0f;
            }
            const float as = row_ok ? __ldg(a_scale + gm) : 0.0f;
            const uint64_t as2 = ptx::f32x2_pack(as, as);
            // one thread polls for all epilogue warps (named barrier 1); the barrier also publishes s_ws / s_bs
            alive = ptx::mbar_wait_group(bar_tfull + 8 * b, (t >> 1) & 1, s_abort, status, QVGGT_DEV_TIMEOUT_ACCUM,
                                         threadIdx.x == 0, 1, EPI_WARPS * 32, s_flags, toggle, 64) && alive;
            ptx::tc_fence_after_sync();
            if (alive) {
                const float *wsb = s_ws + b * BN + cpart * C::CW;
                const float *bsb = s_bs + b * BN + cpart * C::CW;
                constexpr int NCH = C::CW / 32;
                // the warp's whole share of the accumulator goes to registers first, so that tensor memory is
                // handed back to the MMA thread a few hundred cycles after the tile completed, not after the
                // conversions and stores of the first chunks
                uint32_t raw[NCH][32];
#pragma unroll
                for (int c = 0; c < NCH; ++c)
                    ptx::tmem_ld_32x32(tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + b * BN + cpart * C::CW + c * 32, raw[c]);
                ptx::tmem_ld_wait();
                ptx::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive_cluster(leader_tempty + 8 * b);
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
                    const int col = c * 32;                               // within this warp's columns
                    if (cols_ok) {
                        uint32_t out[16];
#pragma unroll
                        for (int j = 0; j < 32; j += 4) {
                            const ulonglong2 w2 = *reinterpret_cast<const ulonglong2 *>(wsb + col + j);
                            const ulonglong2 b2 = *reinterpret_cast<const ulonglong2 *>(bsb + col + j);
                            uint64_t z01 = ptx::f32x2_pack(static_cast<float>(static_cast<int>(raw[c][j])), static_cast<float>(static_cast<int>(raw[c][j + 1])));
                            uint64_t z23 = ptx::f32x2_pack(static_cast<float>(static_cast<int>(raw[c][j + 2])), static_cast<float>(static_cast<int>(raw[c][j + 3])));
                            // fl(fl(float(acc) * fl(a_scale * w_scale)) + bias), every operation rounded to nearest.
                            // The additions are scalar intrinsics: a packed multiply feeding a packed add was
                            // observed to be contracted into one fused operation (single rounding).
                            z01 = ptx::f32x2_mul(z01, ptx::f32x2_mul(as2, w2.x));
                            z23 = ptx::f32x2_mul(z23, ptx::f32x2_mul(as2, w2.y));
                            float y0, y1, y2, y3, c0, c1, c2, c3;
                            ptx::f32x2_unpack(z01, y0, y1);
                            ptx::f32x2_unpack(z23, y2, y3);
                            ptx::f32x2_unpack(b2.x, c0, c1);
                            ptx::f32x2_unpack(b2.y, c2, c3);
                            out[j >> 1] = ptx::pack_bf16x2(__fadd_rn(y0, c0), __fadd_rn(y1, c1));
                            out[(j >> 1) + 1] = ptx::pack_bf16x2(__fadd_rn(y2, c2), __fadd_rn(y3, c3));
                        }
                        // the previous TMA store has finished reading the staging buffer
                        if (lane == 0) ptx::tma_store_wait_read<0>();
                        __syncwarp();
                        // row `lane` of the staging tile (64-byte rows, 64-byte swizzle): 16-byte chunk q XOR ((lane / 2) mod 4)
#pragma unroll
                        for (int q = 0; q < 4; ++q)
                            *reinterpret_cast<uint4 *>(stg + lane * 64 + ((q ^ ((lane >> 1) & 3)) << 4)) =
                                make_uint4(out[4 * q], out[4 * q + 1], out[4 * q + 2], out[4 * q + 3]);
                        if (DUMP && acc_debug && row_ok) {
                            uint4 *dbg = reinterpret_cast<uint4 *>(acc_debug + (long long)gm * N + n0 + col);
#pragma unroll
                            for (int q = 0; q < 8; ++q) dbg[q] = make_uint4(raw[c][4 * q], raw[c][4 * q + 1], raw[c][4 * q + 2], raw[c][4 * q + 3]);
                        }
                        ptx::fence_proxy_async_smem();          // staging writes -> visible to the TMA engine
                        __syncwarp();
                        if (lane == 0 && m0 < M) {
                            ptx::tma_store_2d(&map_y, stg_addr, n0 + col, m0);   // rows >= M are clipped by the tensor map
                            ptx::tma_store_commit();
                        }
                    }
                }
            }
        }
        if (lane == 0) ptx::tma_store_wait_all();
    } else if (warp == C::MMA_WARP) {
        // ------------------------------------------------------------ MMA issuer (one thread of the leader CTA)
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = ptx::idesc_i8(2 * BM, BN);
            bool alive = true;
            int s = 0;
            uint32_t ph = 0;
            for (int t = 0; t < my_tiles && alive; ++t) {
                const int b = t & 1;
                if (t >= ACC_BUFS) {
                    alive = ptx::mbar_wait_cluster(bar_tempty + 8 * b, ((t >> 1) - 1) & 1, s_abort, status, QVGGT_DEV_TIMEOUT_TMEM_FREE);
                    if (!alive) break;
                    ptx::tc_fence_after_sync();
                }
                const uint32_t d_tmem = tmem_base + b * BN;
                for (int kb = 0; kb < KB; ++kb) {
                    alive = ptx::mbar_wait_cluster(bar_full + 8 * s, ph, s_abort, status, QVGGT_DEV_TIMEOUT_FULL);
                    if (!alive) break;
                    ptx::tc_fence_after_sync();
                    const uint32_t a_addr = sbase + s * C::STAGE;
                    const uint64_t a_desc = ptx::smem_desc_k_sw128(a_addr);
                    const uint64_t b_desc = ptx::smem_desc_k_sw128(a_addr + BM * BK);
#pragma unroll
                    for (int p = 0; p < BK / 32; ++p)   // advance 32 bytes (one K = 32 slice) inside the swizzled row: +2 in 16-byte units
                        ptx::mma_i8_ss_pair(d_tmem, a_desc + 2 * p, b_desc + 2 * p, idesc, (kb | p) != 0);
                    ptx::mma_commit_pair(bar_empty + 8 * s, 3);      // frees the stage in both CTAs
                    if (++s == C::STAGES) { s = 0; ph ^= 1; }
                }
                if (alive) ptx::mma_commit_pair(bar_tfull + 8 * b, 3);
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ TMA producer (one thread per CTA)
        if (lane == 0) {
            const uint32_t leader_full = ptx::map_to_cta(bar_full, 0);
            bool alive = true;
            int s = 0;
            uint32_t ph = 0;
            int it = 0;
            for (int t = 0; t < my_tiles && alive; ++t) {
                const int tile = worker + t * workers;
                const int m0 = (tile / n_tiles) * (2 * BM) + (int)rank * BM;
                const int n0 = (tile % n_tiles) * BN + (int)rank * C::B_ROWS;
                for (int kb = 0; kb < KB; ++kb, ++it) {
                    if (it >= C::STAGES) {
                        alive = ptx::mbar_wait(bar_empty + 8 * s, ph ^ 1, s_abort, status, QVGGT_DEV_TIMEOUT_EMPTY, 20);
                        if (!alive) break;
                    }
                    const uint32_t dst = sbase + s * C::STAGE;
                    // the leader's barrier expects the bytes of both CTAs; the peer's completions may arrive first
                    // (the count goes negative for a while), the phase cannot end before the leader has arrived
                    if (rank == 0) ptx::mbar_arrive_expect_tx(bar_full + 8 * s, 2 * C::STAGE);
                    ptx::tma_load_2d_pair(&map_x, leader_full + 8 * s, dst, kb * BK, m0);
                    ptx::tma_load_2d_pair(&map_w, leader_full + 8 * s, dst + BM * BK, kb * BK, n0);
                    if (++s == C::STAGES) { s = 0; ph ^= 1; }
                }
            }
        }
        __syncwarp();
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync();        // no remote arrival or multicast commit may target a CTA that has exited
    if (warp == C::MMA_WARP) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc_pair(tmem_base, C::TMEM_COLS);
    }
}

template <int EPI_WARPS, bool DUMP>
cudaError_t launch(const qvggt_weights *w, const signed char *Xq8, const float *a_scale, int M, void *Y, long long ldy,
                   int *acc_debug, cudaStream_t st)
{
    using C = Cfg<EPI_WARPS>;
    static int max_workers = 0;       // per process; one GPU type per process
    cudaError_t e;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;      // see grid_dependency_wait()
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    if (!max_workers) {
        e = cudaFuncSetAttribute(gemm_c8_kernel<EPI_WARPS, DUMP>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::DYN_SMEM);
        if (e != cudaSuccess) return e;
        cudaLaunchConfig_t probe = {};
        probe.gridDim = dim3(2 * qvggt_sm_count());
        probe.blockDim = dim3(C::THREADS);
        probe.dynamicSmemBytes = C::DYN_SMEM;
        probe.attrs = attr;
        probe.numAttrs = 1;
        int clusters = 0;
        e = cudaOccupancyMaxActiveClusters(&clusters, gemm_c8_kernel<EPI_WARPS, DUMP>, &probe);
        if (e != cudaSuccess) return e;
        if (clusters < 1) return cudaErrorLaunchOutOfResources;
        max_workers = clusters;
    }
    const int K = w->K, N = w->N;
    CUtensorMap map_x, map_w, map_y;
    if (!qvggt_make_map(&map_x, CU_TENSOR_MAP_DATA_TYPE_UINT8, Xq8, K, M, K, BK, BM, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !qvggt_make_map(&map_w, CU_TENSOR_MAP_DATA_TYPE_UINT8, w->Wq8, K, N, K, BK, C::B_ROWS, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !qvggt_make_map(&map_y, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, Y, N, M, (uint64_t)ldy * 2, 32, 32, CU_TENSOR_MAP_SWIZZLE_64B))
        return cudaErrorInvalidValue;
    const int total_tiles = ((M + 2 * BM - 1) / (2 * BM)) * ((N + BN - 1) / BN);
    const int workers = total_tiles < max_workers ? total_tiles : max_workers;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(workers * 2);
    cfg.blockDim = dim3(C::THREADS);
    cfg.dynamicSmemBytes = C::DYN_SMEM;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, gemm_c8_kernel<EPI_WARPS, DUMP>, map_x, map_w, map_y, a_scale, (const float *)w->w_scale,
                              (const uint16_t *)w->bias, acc_debug, M, N, K, w->status);
}

#ifndef QVGGT_C8_EPI_WARPS
#define QVGGT_C8_EPI_WARPS 8
#endif

}  // namespace

cudaError_t qvggt_launch_gemm_c8(const qvggt_weights *w, const signed char *Xq8, const float *a_scale, int M, void *Y,
                                 long long ldy, int *acc_debug, cudaStream_t st)
{
    if (M == 0) return cudaSuccess;
    if (!w->Wq8) return cudaErrorNotSupported;      // the handle was prepared without the 8-bit-container copy
    return acc_debug ? launch<QVGGT_C8_EPI_WARPS, true>(w, Xq8, a_scale, M, Y, ldy, acc_debug, st)
                     : launch<QVGGT_C8_EPI_WARPS, false>(w, Xq8, a_scale, M, Y, ldy, acc_debug, st);
}
