// Host helpers shared by the GEMM translation units: TMA tensor maps and the SM count.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

// 2-D row-major tensor: `inner` elements per row, `rows` rows, `pitch_bytes` between rows; the box is
// box_inner x box_rows elements.  Out-of-range parts of a box read as zero and are not written.
// Returns false if the driver entry point is missing or the encoding is refused.
bool qvggt_make_map(CUtensorMap *map, CUtensorMapDataType type, const void *base, uint64_t inner, uint64_t rows,
                    uint64_t pitch_bytes, uint32_t box_inner, uint32_t box_rows, CUtensorMapSwizzle swizzle);

int qvggt_sm_count();   // SMs of the current device (cached: one GPU type per process)
