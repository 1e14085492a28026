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
// Persistent and warp-specialised.  A "worker" is one CTA (CG = 1: tile 128 tokens x 256 channels)
// or a pair of CTAs on neighbouring SMs (CG = 2: tile 256 x 256, each CTA stages 128 token rows and
// 128 weight rows, one thread of the leader CTA issues tcgen05.mma.cta_group::2 for both).
//   warps 0-7    epilogue: TMEM -> registers -> scale, bias, bf16 -> swizzled staging -> TMA store
//   warps 8-15   converters: packed stage -> registers -> int8 operand stage
//   warp  16     one thread issues tcgen05.mma and the commits that release stages / publish accumulators
//   warp  17     one thread issues the TMA loads of packed tiles
// Every wait is bounded; on expiry the kernel records a code in *status and all roles fall through
// to the common exit, where tensor memory is released.
#include <cuda.h>
#include <cuda_bf16.h>

#include "qvggt_internal.cuh"
#include "sm100_ptx.cuh"
#include "tensor_map.cuh"

namespace {

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
constexpr int STG_BYTES = 32 * 64;    // per epilogue warp: 32 rows x 32 bf16, 64-byte swizzled

template <int CG>
struct Cfg {
    static constexpr int B_ROWS = BN / CG;                 // weight rows staged by one CTA
    static constexpr int ROWS = BM + B_ROWS;
    static constexpr int PK_STAGE = ROWS * (BK / 2);       // packed codes
    static constexpr int UP_STAGE = ROWS * BK;             // int8 operands
    static constexpr int PS = 4;                           // packed stages (cover the L2 latency)
    static constexpr int US = (CG == 1) ? 2 : 4;           // operand stages (decouple converters and MMA)
    // Converter warps form GROUPS independent groups; group g converts K-blocks g, g + GROUPS, ...  so the
    // fixed costs of a stage (draining the stores, the proxy fence, barrier round trips) overlap.
    static constexpr int GROUPS = (CG == 1) ? 2 : 4;
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
template <int CG, bool DUMP>
__global__ void __launch_bounds__(THREADS, 1)
gemm_w4a4_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                 const __grid_constant__ CUtensorMap map_y, const float *__restrict__ a_scale,
                 const float *__restrict__ w_scale, const uint16_t *__restrict__ bias, int *__restrict__ acc_debug,
                 int M, int N, int K, int *status)
{
    using C = Cfg<CG>;
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
    const uint32_t rank = (CG == 2) ? ptx::cluster_ctarank() : 0u;     // 0 = leader of the pair
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
    if (warp == MMA_WARP) {
        if (CG == 2) { ptx::tmem_alloc_pair(ptx::smem_addr(s_tmem), C::TMEM_COLS); ptx::tmem_relinquish_pair(); }
        else         { ptx::tmem_alloc(ptx::smem_addr(s_tmem), C::TMEM_COLS);      ptx::tmem_relinquish(); }
    }
    if (warp == TMA_WARP && lane == 0) {
        ptx::prefetch_tensormap(&map_x);
        ptx::prefetch_tensormap(&map_w);
        ptx::prefetch_tensormap(&map_y);
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (CG == 2) ptx::cluster_sync();        // the peer's barriers exist before anything arrives on them remotely
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *s_tmem;

    if (warp < EPI_WARPS) {
        // ------------------------------------------------------------ epilogue
        const int quarter = warp & 3, chalf = warp >> 2;   // TMEM lane quarter, column half
        unsigned char *stg = smem + C::OFF_STG + warp * STG_BYTES;
        const uint32_t stg_addr = sbase + C::OFF_STG + warp * STG_BYTES;
        float *s_ws = reinterpret_cast<float *>(smem + C::OFF_CH);          // [2][BN] per-channel scale of the tile
        float *s_bs = s_ws + ACC_BUFS * BN;                                   // [2][BN] bias as fp32
        const uint32_t leader_tempty = (CG == 2) ? ptx::map_to_cta(bar_tempty, 0) : bar_tempty;
        bool alive = true;
        uint32_t toggle = 0;
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
            {
                const int e = threadIdx.x;                     // 0..255: one channel each
                const bool ch_ok = nt0 + e < N;
                s_ws[b * BN + e] = ch_ok ? __ldg(w_scale + nt0 + e) : 0.0f;
                s_bs[b * BN + e] = (ch_ok && bias) ? __uint_as_float(static_cast<uint32_t>(__ldg(bias + nt0 + e)) << 16) : 0.0f;
            }
            // a_scale / 256: exact (power of two), cancels the factor 256 carried by the raw accumulator
            const float as = row_ok ? __fmul_rn(__ldg(a_scale + gm), 0.00390625f) : 0.0f;
            const uint64_t as2 = ptx::f32x2_pack(as, as);
            // one thread polls for all epilogue warps (named barrier 1); the barrier also publishes s_ws / s_bs
            alive = ptx::mbar_wait_group(bar_tfull + 8 * b, (t >> 1) & 1, s_abort, status, QVGGT_DEV_TIMEOUT_ACCUM,
                                         threadIdx.x == 0, 1, EPI_WARPS * 32, s_flags, toggle, 64) && alive;
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
                        if (lane == 0) {
                            if (CG == 2) ptx::mbar_arrive_cluster(leader_tempty + 8 * b);
                            else ptx::mbar_arrive(bar_tempty + 8 * b);
                        }
                    }
                    if (cols_ok) {
                        uint32_t out[16];
#pragma unroll
                        for (int j = 0; j < 32; j += 4) {
                            const ulonglong2 w2 = *reinterpret_cast<const ulonglong2 *>(wsb + col + j);
                            const ulonglong2 b2 = *reinterpret_cast<const ulonglong2 *>(bsb + col + j);
                            uint64_t z01 = ptx::f32x2_pack(static_cast<float>(static_cast<int>(raw[j])), static_cast<float>(static_cast<int>(raw[j + 1])));
                            uint64_t z23 = ptx::f32x2_pack(static_cast<float>(static_cast<int>(raw[j + 2])), static_cast<float>(static_cast<int>(raw[j + 3])));
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
                            for (int q = 0; q < 8; ++q)
                                dbg[q] = make_uint4(static_cast<int>(raw[4 * q]) >> 8, static_cast<int>(raw[4 * q + 1]) >> 8,
                                                    static_cast<int>(raw[4 * q + 2]) >> 8, static_cast<int>(raw[4 * q + 3]) >> 8);
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
    } else if (warp < MMA_WARP) {
        // ------------------------------------------------------------ converters
        const int cw = warp - CONV_WARP0;
        const int group = cw / C::GROUP_WARPS;
        const int gt = (cw % C::GROUP_WARPS) * 32 + lane;                // thread within the group
        const int row = gt >> 2, piece = gt & 3;                         // piece i of this thread: row + (GROUP_THREADS/4) i
        constexpr int SRC_STEP = C::GROUP_THREADS * 16;                  // bytes between a thread's consecutive packed pieces
        constexpr int DST_STEP = (C::GROUP_THREADS / 4) * 128;
        const uint32_t src_off = gt * 16;
        const uint32_t dst_off = row * 128 + (((2 * piece) ^ (row & 7)) << 4);   // even codes
        const uint32_t dst_hi_off = dst_off ^ 16;                                // odd codes: the neighbouring 16-byte chunk
        const uint32_t leader_ufull = (CG == 2) ? ptx::map_to_cta(bar_ufull, 0) : bar_ufull;
        const int total_kb = my_tiles * KB;
        bool alive = true;
        uint32_t toggle = 0;
        for (int it = group; it < total_kb && alive; it += C::GROUPS) {
            const int ps = it % C::PS, us = it % C::US;
            alive = ptx::mbar_wait_group(bar_pfull + 8 * ps, (it / C::PS) & 1, s_abort, status, QVGGT_DEV_TIMEOUT_PACKED, gt == 0,
                                         2 + group, C::GROUP_THREADS, s_flags + 2 + 2 * group, toggle, 20);
            if (!alive) break;
            // the whole share of the stage goes to registers first, so the packed stage is handed back
            // to the TMA producer before the (longer) conversion starts
            const unsigned char *src = smem + C::OFF_PK + ps * C::PK_STAGE + src_off;
            uint4 pk[C::CHUNKS];
#pragma unroll
            for (int i = 0; i < C::CHUNKS; ++i) pk[i] = *reinterpret_cast<const uint4 *>(src + SRC_STEP * i);
            // consume one value of every load: the loads have completed before the stage is released
            uint32_t seen = 0;
#pragma unroll
            for (int i = 0; i < C::CHUNKS; ++i) seen |= pk[i].x;
            // a real (if never taken) use of every loaded value: the loads must have returned before
            // this branch resolves, hence before the arrival below lets the TMA overwrite the stage
            if (seen == 0x9E3779B9u) s_flags[1 + 2 * CONV_WARPS] = 1;
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(bar_pempty + 8 * ps);
            if (it >= C::US) {
                alive = ptx::mbar_wait_group(bar_uempty + 8 * us, ((it / C::US) - 1) & 1, s_abort, status, QVGGT_DEV_TIMEOUT_EMPTY,
                                             gt == 0, 2 + group, C::GROUP_THREADS, s_flags + 2 + 2 * group, toggle, 20);
                if (!alive) break;
            }
            unsigned char *dst = smem + C::OFF_UP + us * C::UP_STAGE;
#pragma unroll
            for (int i = 0; i < C::CHUNKS; ++i) {
                const uint4 w = pk[i];
                uint4 lo, hi;
                lo.x = (w.x << 4) & 0xF0F0F0F0u; hi.x = w.x & 0xF0F0F0F0u;
                lo.y = (w.y << 4) & 0xF0F0F0F0u; hi.y = w.y & 0xF0F0F0F0u;
                lo.z = (w.z << 4) & 0xF0F0F0F0u; hi.z = w.z & 0xF0F0F0F0u;
                lo.w = (w.w << 4) & 0xF0F0F0F0u; hi.w = w.w & 0xF0F0F0F0u;
                *reinterpret_cast<uint4 *>(dst + dst_off + DST_STEP * i) = lo;
                *reinterpret_cast<uint4 *>(dst + dst_hi_off + DST_STEP * i) = hi;
            }
            ptx::fence_proxy_async_smem();      // my generic-proxy writes -> visible to the tensor core's async proxy
            __syncwarp();                        // orders the whole warp's reads and writes before the two arrivals
            if (lane == 0) {
                if (CG == 2) ptx::mbar_arrive_cluster(leader_ufull + 8 * us);
                else ptx::mbar_arrive(bar_ufull + 8 * us);
            }
        }
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
                    const uint64_t a_desc = ptx::smem_desc_k_sw128(a_addr);
                    const uint64_t b_desc = ptx::smem_desc_k_sw128(a_addr + BM * BK);
#pragma unroll
                    for (int p = 0; p < BK / 32; ++p) {
                        // advance 32 bytes (one K = 32 slice) inside the swizzled row: +2 in 16-byte units
                        if (CG == 2) ptx::mma_i8_ss_pair(d_tmem, a_desc + 2 * p, b_desc + 2 * p, idesc, (kb | p) != 0);
                        else ptx::mma_i8_ss(d_tmem, a_desc + 2 * p, b_desc + 2 * p, idesc, (kb | p) != 0);
                    }
                    if (CG == 2) ptx::mma_commit_pair(bar_uempty + 8 * us, 3);
                    else ptx::mma_commit(bar_uempty + 8 * us);
                    if (++us == C::US) { us = 0; uph ^= 1; }
                }
                if (alive) {
                    if (CG == 2) ptx::mma_commit_pair(bar_tfull + 8 * b, 3);
                    else ptx::mma_commit(bar_tfull + 8 * b);
                }
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
    if (CG == 2) ptx::cluster_sync();        // no remote arrival or multicast commit may target a CTA that has exited
    if (warp == MMA_WARP) {
        ptx::tc_fence_after_sync();
        if (CG == 2) ptx::tmem_dealloc_pair(tmem_base, C::TMEM_COLS);
        else ptx::tmem_dealloc(tmem_base, C::TMEM_COLS);
    }
}

template <int CG, bool DUMP>
cudaError_t launch(const qvggt_weights *w, const unsigned char *Xq, const float *a_scale, int M, void *Y, long long ldy,
                   int *acc_debug, cudaStream_t st)
{
    using C = Cfg<CG>;
    static int max_workers = 0;       // per process; one GPU type per process
    cudaError_t e;
    if (!max_workers) {
        e = cudaFuncSetAttribute(gemm_w4a4_kernel<CG, DUMP>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::DYN_SMEM);
        if (e != cudaSuccess) return e;
        if (CG == 1) {
            max_workers = qvggt_sm_count();
        } else {
            cudaLaunchConfig_t probe = {};
            probe.gridDim = dim3(2 * qvggt_sm_count());
            probe.blockDim = dim3(THREADS);
            probe.dynamicSmemBytes = C::DYN_SMEM;
            cudaLaunchAttribute a;
            a.id = cudaLaunchAttributeClusterDimension;
            a.val.clusterDim.x = CG; a.val.clusterDim.y = 1; a.val.clusterDim.z = 1;
            probe.attrs = &a;
            probe.numAttrs = 1;
            int clusters = 0;
            e = cudaOccupancyMaxActiveClusters(&clusters, gemm_w4a4_kernel<CG, DUMP>, &probe);
            if (e != cudaSuccess) return e;
            if (clusters < 1) return cudaErrorLaunchOutOfResources;
            max_workers = clusters;
        }
    }
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
    return cudaLaunchKernelEx(&cfg, gemm_w4a4_kernel<CG, DUMP>, map_x, map_w, map_y, a_scale, (const float *)w->w_scale,
                              (const uint16_t *)w->bias, acc_debug, M, N, K, w->status);
}

}  // namespace

cudaError_t qvggt_launch_gemm(const qvggt_weights *w, const unsigned char *Xq, const float *a_scale, int M, int group,
                              void *Y, long long ldy, int *acc_debug, cudaStream_t st)
{
    if (M == 0) return cudaSuccess;
    if (group == 128) return qvggt_launch_gemm_grouped(w, Xq, a_scale, M, Y, ldy, acc_debug, st);
    if (group != 0) return cudaErrorNotSupported;
    // the single-CTA configuration (CG = 1) measured 10-35 % slower on every VGGT shape: the pair halves the weight traffic
    return acc_debug ? launch<2, true>(w, Xq, a_scale, M, Y, ldy, acc_debug, st) : launch<2, false>(w, Xq, a_scale, M, Y, ldy, acc_debug, st);
}
