// Packed 4-bit weight codes -> one code per byte (Eq. "quantization" with N = 4 stores 4-bit codes; the tensor core
// multiplies them as int8).  Shared by the stand-alone expansion kernel and by the quantize kernel.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

// Expansion job carried by a quantize launch: its blocks share the items between them before they turn to their rows.
// n16 == 0: nothing to expand.
struct QvggtExpand {
    const uint4 *packed;     // [N, K / 2] packed codes, viewed as 16-byte items
    uint4 *out;              // [N, K] one code per byte
    long long n16;           // number of 16-byte items of `packed` = N * K / 32
};

// Item i: 16 packed bytes (byte b = code 2b in bits 0-3, code 2b+1 in bits 4-7, two's complement) -> 32 code bytes.
__device__ __forceinline__ void qvggt_unpack_w4_item(const uint4 *__restrict__ packed, uint4 *__restrict__ out, long long i)
{
    const uint4 p = __ldg(packed + i);
    const uint32_t w[4] = {p.x, p.y, p.z, p.w};
    uint32_t o[8];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            uint32_t x = (w[e] >> (16 * h)) & 0xFFFFu;          // four nibbles
            x = (x | (x << 8)) & 0x00FF00FFu;
            x = (x | (x << 4)) & 0x0F0F0F0Fu;                    // one nibble per byte, natural order
            o[2 * e + h] = x | ((x & 0x08080808u) * 0x1Eu);     // sign extension: bit 3 -> bits 4..7 of its byte
        }
    }
    out[2 * i] = make_uint4(o[0], o[1], o[2], o[3]);
    out[2 * i + 1] = make_uint4(o[4], o[5], o[6], o[7]);
}
