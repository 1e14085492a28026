// Host helpers shared by the GEMM translation units: TMA tensor maps and the SM count.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

// 2-D row-major tensor: `inner` elements per row, `rows` rows, `pitch_bytes` between rows; the box is
// box_inner x box_rows elements.  Out-of-range parts of a box read as zero and are not written.
// Returns false if the driver entry point is missing or the encoding is refused.
bool qvggt_make_map(CUtensorMap *map, CUtensorMapDataType type, const void *base, uint64_t inner, uint64_t rows,
                    uint64_t pitch_bytes, uint32_t box_inner, uint32_t box_rows, CUtensorMapSwizzle swizzle);

// 3-D tensor: `d0` contiguous elements, then `d1` pieces `pitch1_bytes` apart, then `d2` pieces `pitch2_bytes` apart;
// the box is b0 x b1 x b2 elements, no swizzle.
bool qvggt_make_map3(CUtensorMap *map, CUtensorMapDataType type, const void *base, uint64_t d0, uint64_t d1, uint64_t d2,
                     uint64_t pitch1_bytes, uint64_t pitch2_bytes, uint32_t b0, uint32_t b1, uint32_t b2);

// Per-device host-side caches.  Function attributes (the opt-in to large dynamic shared memory), occupancy
// results and SM counts belong to a device, and one process may drive several: every cache is an array indexed
// by the device ordinal.  Zero means "not set yet"; concurrent first calls both compute the same value.
constexpr int kQvggtMaxDevices = 64;
struct QvggtPerDevice {
    std::atomic<int> v[kQvggtMaxDevices];
};
int qvggt_current_device();   // ordinal of the current device, or -1 (no device, or beyond kQvggtMaxDevices)
int qvggt_sm_count();         // SMs of the current device (cached per device); 0 on failure
