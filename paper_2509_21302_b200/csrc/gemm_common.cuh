// Pieces shared by the integer GEMM kernels (gemm.cu, gemm_c8.cu, gemm_grouped.cu): the per-K-block MMA issue,
// the rescale + bias + bf16 arithmetic of the epilogue (Sec. 3.2: both scales stay outside the integer sum), the
// staging tile behind every TMA store, and the host-side per-device configuration of a kernel.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "sm100_ptx.cuh"
#include "tensor_map.cuh"

namespace gemmc {

constexpr int STG_BYTES = 32 * 64;   // staging tile of one epilogue warp: 32 rows x 32 bf16, 64-byte swizzled

// A position in a ring of pipeline stages together with the parity of the phase it is in.
struct Ring {
    int s = 0;
    uint32_t ph = 0;
    __device__ __forceinline__ void advance(int stages)
    {
        if (++s == stages) { s = 0; ph ^= 1; }
    }
};

__device__ __forceinline__ void init_barriers(uint32_t first, int n, uint32_t count)
{
    for (int i = 0; i < n; ++i) ptx::mbar_init(first + 8 * i, count);
}

// One K-block (128 int8 codes along K = one 128-byte swizzled row per operand row) as four tcgen05.mma of K = 32:
// the start address advances 32 bytes (+2 in 16-byte units) inside the swizzled row.  `fresh` = this K-block
// starts a new accumulation (the first MMA overwrites the accumulator).
template <bool PAIR>
__device__ __forceinline__ void mma_kblock_i8(uint32_t d_tmem, uint32_t a_addr, uint32_t b_addr, uint32_t idesc, bool fresh)
{
    const uint64_t a_desc = ptx::smem_desc_k_sw128(a_addr);
    const uint64_t b_desc = ptx::smem_desc_k_sw128(b_addr);
#pragma unroll
    for (int p = 0; p < 4; ++p) {
        if (PAIR) ptx::mma_i8_ss_pair(d_tmem, a_desc + 2 * p, b_desc + 2 * p, idesc, !(fresh && p == 0));
        else ptx::mma_i8_ss(d_tmem, a_desc + 2 * p, b_desc + 2 * p, idesc, !(fresh && p == 0));
    }
}

// Per-channel scale and bias (bf16 -> fp32) of channel nt0 + e -> slot e of the tile's shared-memory copies.
__device__ __forceinline__ void load_channel_params(float *s_ws, float *s_bs, const float *__restrict__ w_scale,
                                                    const uint16_t *__restrict__ bias, int nt0, int N, int e)
{
    const bool ch_ok = nt0 + e < N;
    s_ws[e] = ch_ok ? __ldg(w_scale + nt0 + e) : 0.0f;
    s_bs[e] = (ch_ok && bias) ? __uint_as_float(static_cast<uint32_t>(__ldg(bias + nt0 + e)) << 16) : 0.0f;
}

// 32 consecutive channels of one token row: fl(fl(float(acc) * fl(a_scale * w_scale)) + bias), every operation
// rounded to nearest, then bf16 (round to nearest even), two per word.  `as2` holds a_scale in both halves; ws / bs
// point at the 32 channel scales / biases (fp32, 16-byte aligned, shared memory).
// The additions are scalar intrinsics: a packed multiply feeding a packed add was observed to be contracted
// into one fused operation (single rounding).
__device__ __forceinline__ void scale_bias_bf16_x32(const uint32_t (&raw)[32], uint64_t as2, const float *ws, const float *bs,
                                                    uint32_t (&out)[16])
{
#pragma unroll
    for (int j = 0; j < 32; j += 4) {
        const ulonglong2 w2 = *reinterpret_cast<const ulonglong2 *>(ws + j);
        const ulonglong2 b2 = *reinterpret_cast<const ulonglong2 *>(bs + j);
        uint64_t z01 = ptx::f32x2_pack(static_cast<float>(static_cast<int>(raw[j])), static_cast<float>(static_cast<int>(raw[j + 1])));
        uint64_t z23 = ptx::f32x2_pack(static_cast<float>(static_cast<int>(raw[j + 2])), static_cast<float>(static_cast<int>(raw[j + 3])));
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
}

// Whole warp: waits until the previous TMA store has read the warp's staging tile, writes row `lane` (64-byte rows,
// 16-byte chunk q kept at q XOR ((lane / 2) mod 4): the 64-byte swizzle the output tensor map expects).
__device__ __forceinline__ void stage_row_32(unsigned char *stg, const uint32_t (&out)[16], int lane)
{
    if (lane == 0) ptx::tma_store_wait_read<0>();
    __syncwarp();
#pragma unroll
    for (int q = 0; q < 4; ++q)
        *reinterpret_cast<uint4 *>(stg + lane * 64 + ((q ^ ((lane >> 1) & 3)) << 4)) =
            make_uint4(out[4 * q], out[4 * q + 1], out[4 * q + 2], out[4 * q + 3]);
}

// Whole warp: makes the staging tile visible to the TMA engine and stores it at (x = first channel, y = first
// row); rows beyond the tensor are clipped by the tensor map.  `issue` is false when the whole tile lies beyond.
__device__ __forceinline__ void store_staged_32x32(const void *map_y, uint32_t stg_addr, int x, int y, bool issue, int lane)
{
    ptx::fence_proxy_async_smem();
    __syncwarp();
    if (lane == 0 && issue) {
        ptx::tma_store_2d(map_y, stg_addr, x, y);
        ptx::tma_store_commit();
    }
}

// Converter role of the kernels whose operands arrive packed (two 4-bit codes per byte).  The converter warps of a
// CTA form C::GROUPS independent groups; group g takes K-blocks g, g + GROUPS, ... so that the fixed costs of a
// stage (draining the stores, the proxy fence, barrier round trips) overlap.  Per K-block: wait for the TMA-loaded
// packed stage, pull the group's whole share into registers and hand the stage back at once, wait for a free
// operand stage, write every nibble into the HIGH half of an int8 byte (value 16 q: no sign extension needed; even
// and odd codes of a 32-code slice land in neighbouring 16-byte chunks of the 128-byte-swizzled K-major row, the
// same permutation of K for both operands), fence for the tensor core's proxy and arrive on `ufull_arrive` (the
// leader CTA's barrier for a CTA pair, given as a shared::cluster address).
// C supplies PS, US, GROUPS, GROUP_WARPS, GROUP_THREADS, CHUNKS, OFF_PK, PK_STAGE, OFF_UP, UP_STAGE.
// `cw` = index of the warp among the converter warps; s_flags: 2 words per group + 1 sink word at s_sink.
template <class C, bool PAIR>
__device__ __forceinline__ void convert_packed_stages(unsigned char *smem, int cw, int lane, int total_kb, uint32_t bar_pfull,
                                                      uint32_t bar_pempty, uint32_t bar_uempty, uint32_t ufull_arrive,
                                                      volatile int *s_abort, int *status, volatile int *s_flags,
                                                      volatile int *s_sink, int code_packed, int code_empty)
{
    const int group = cw / C::GROUP_WARPS;
    const int gt = (cw % C::GROUP_WARPS) * 32 + lane;                // thread within the group
    const int row = gt >> 2, piece = gt & 3;                         // piece i of this thread: row + (GROUP_THREADS/4) i
    constexpr int SRC_STEP = C::GROUP_THREADS * 16;                  // bytes between a thread's consecutive packed pieces
    constexpr int DST_STEP = (C::GROUP_THREADS / 4) * 128;
    const uint32_t src_off = gt * 16;
    const uint32_t dst_off = row * 128 + (((2 * piece) ^ (row & 7)) << 4);   // even codes
    const uint32_t dst_hi_off = dst_off ^ 16;                                // odd codes: the neighbouring 16-byte chunk
    bool alive = true;
    uint32_t toggle = 0;
    for (int it = group; it < total_kb && alive; it += C::GROUPS) {
        const int ps = it % C::PS, us = it % C::US;
        alive = ptx::mbar_wait_group(bar_pfull + 8 * ps, (it / C::PS) & 1, s_abort, status, code_packed, gt == 0,
                                     2 + group, C::GROUP_THREADS, s_flags + 2 * group, toggle, 20);
        if (!alive) break;
        const unsigned char *src = smem + C::OFF_PK + ps * C::PK_STAGE + src_off;
        uint4 pk[C::CHUNKS];
#pragma unroll
        for (int i = 0; i < C::CHUNKS; ++i) pk[i] = *reinterpret_cast<const uint4 *>(src + SRC_STEP * i);
        // a real (if never taken) use of every loaded value: the loads must have returned before this branch
        // resolves, hence before the arrival below lets the TMA overwrite the stage (an empty inline-asm "use"
        // is dropped by the assembler)
        uint32_t seen = 0;
#pragma unroll
        for (int i = 0; i < C::CHUNKS; ++i) seen |= pk[i].x;
        if (seen == 0x9E3779B9u) *s_sink = 1;
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(bar_pempty + 8 * ps);
        if (it >= C::US) {
            alive = ptx::mbar_wait_group(bar_uempty + 8 * us, ((it / C::US) - 1) & 1, s_abort, status, code_empty,
                                         gt == 0, 2 + group, C::GROUP_THREADS, s_flags + 2 * group, toggle, 20);
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
        __syncwarp();                        // orders the whole warp's reads and writes before the arrival
        if (lane == 0) {
            if (PAIR) ptx::mbar_arrive_cluster(ufull_arrive + 8 * us);
            else ptx::mbar_arrive(ufull_arrive + 8 * us);
        }
    }
}

// 32 raw int32 sums of one row -> global memory (debug dump), optionally shifted right (the packed kernels carry
// the codes in the high half-byte, so their raw sums are 256 x the integer sums).
template <int SHIFT>
__device__ __forceinline__ void dump_acc_x32(int *dst, const uint32_t (&raw)[32])
{
    uint4 *d = reinterpret_cast<uint4 *>(dst);
#pragma unroll
    for (int q = 0; q < 8; ++q)
        d[q] = make_uint4(static_cast<int>(raw[4 * q]) >> SHIFT, static_cast<int>(raw[4 * q + 1]) >> SHIFT,
                          static_cast<int>(raw[4 * q + 2]) >> SHIFT, static_cast<int>(raw[4 * q + 3]) >> SHIFT);
}

}  // namespace gemmc

// Host side, once per device and kernel: opts the kernel in to `smem` bytes of dynamic shared memory and finds how
// many clusters of `cluster` CTAs (1 = plain CTAs) can be resident at once.  The result is cached in `cache`.
template <class Kernel>
cudaError_t qvggt_configure_kernel(Kernel kernel, int threads, int smem, int cluster, QvggtPerDevice &cache, int *workers)
{
    const int dev = qvggt_current_device();
    if (dev < 0) return cudaErrorInvalidDevice;
    int n = cache.v[dev].load(std::memory_order_acquire);
    if (!n) {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        const int sms = qvggt_sm_count();
        if (sms < 1) return cudaErrorInvalidDevice;
        if (cluster == 1) {
            n = sms;
        } else {
            cudaLaunchAttribute a;
            a.id = cudaLaunchAttributeClusterDimension;
            a.val.clusterDim.x = cluster; a.val.clusterDim.y = 1; a.val.clusterDim.z = 1;
            cudaLaunchConfig_t probe = {};
            probe.gridDim = dim3(cluster * sms);
            probe.blockDim = dim3(threads);
            probe.dynamicSmemBytes = smem;
            probe.attrs = &a;
            probe.numAttrs = 1;
            e = cudaOccupancyMaxActiveClusters(&n, kernel, &probe);
            if (e != cudaSuccess) return e;
            if (n < 1) return cudaErrorLaunchOutOfResources;
        }
        cache.v[dev].store(n, std::memory_order_release);
    }
    *workers = n;
    return cudaSuccess;
}
