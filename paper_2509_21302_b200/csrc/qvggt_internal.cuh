// Internal declarations shared by the translation units of libqvggt (device code for sm_100a).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/qvggt.h"

struct qvggt_weights {
    int N, K;
    int device;
    int bits;            // 4 (W4A4) or 8 (W8A8: codes one per byte only)
    unsigned char *Wq;   // [N, K/2] packed int4 (nullptr when bits == 8 or prepared with QVGGT_PREP_C8_ONLY)
    signed char *Wq8;    // [N, K] one code per byte, or nullptr (prepared without QVGGT_PREP_C8)
    float *w_scale;      // [N]
    float *amul;         // [K]
    uint16_t *bias;      // [N] bf16 bits, or nullptr
    int *status;         // device status word (0 = ok)
};

// Device status codes written by kernels whose bounded waits expire.
enum : int {
    QVGGT_DEV_OK = 0,
    QVGGT_DEV_TIMEOUT_FULL = 1,    // MMA thread gave up waiting for a converted operand stage
    QVGGT_DEV_TIMEOUT_EMPTY = 2,   // converter gave up waiting for a stage to be released
    QVGGT_DEV_TIMEOUT_ACCUM = 3,   // epilogue gave up waiting for the accumulator
    QVGGT_DEV_TIMEOUT_TMEM_FREE = 4, // MMA thread gave up waiting for the epilogue to drain TMEM
    QVGGT_DEV_TIMEOUT_PACKED = 5,    // converter gave up waiting for a TMA-loaded stage of packed codes
    QVGGT_DEV_TIMEOUT_PACKED_FREE = 6 // TMA producer gave up waiting for a packed stage to be released
};

// rsq.cu
cudaError_t qvggt_launch_multipliers(const float *c, const signed char *v, int K, float *amul, float *wmul,
                                     cudaStream_t st);
cudaError_t qvggt_launch_rsq(const void *X, long long ldx, int M, int K, const float *mul, int group,
                             unsigned char *Xq, float *scales, cudaStream_t st);
cudaError_t qvggt_launch_rsq_c8(const void *X, long long ldx, int M, int K, const float *mul, int bits, signed char *Xq8,
                                float *scales, cudaStream_t st, int group = 0, const void *w_packed = nullptr,
                                void *w_expanded = nullptr, long long w_codes = 0);
cudaError_t qvggt_launch_rsq_static_c8(const void *X, long long ldx, int M, int K, const float *mul, int bits, const float *delta,
                                       signed char *Xq8, float *scales, cudaStream_t st);
cudaError_t qvggt_launch_ln_rsq_c8(const void *X, long long ldx, int M, int K, const float *mul, int bits, const float *gamma,
                                   const float *beta, float eps, signed char *Xq8, float *scales, void *ln_out, cudaStream_t st);
cudaError_t qvggt_launch_gelu_rsq_c8(const void *X, long long ldx, int M, int K, const float *mul, int bits, signed char *Xq8,
                                     float *scales, void *gelu_out, cudaStream_t st);
cudaError_t qvggt_launch_max_reduce(const float *in, int n, float *out, cudaStream_t st);
cudaError_t qvggt_launch_colmax(const void *X, int M, int K, float *colmax, cudaStream_t st);
cudaError_t qvggt_launch_smooth_finalize(const float *ax, const float *aw, int K, float alpha, float lo, float hi,
                                         float *c, cudaStream_t st);

// rsq_tc.cu (tensor-core Hadamard mode; per-token scales; c8: one code per byte; y_debug fp32 [M, K] or nullptr)
cudaError_t qvggt_launch_rsq_tc(const void *X, long long ldx, int M, int K, const float *mul, int bits, bool c8, void *Xq,
                                float *scales, float *y_debug, int *status, cudaStream_t st);

// gemm.cu
cudaError_t qvggt_launch_gemm(const qvggt_weights *w, const unsigned char *Xq, const float *a_scale, int M,
                              int group, void *Y, long long ldy, int *acc_debug, cudaStream_t st);

// gemm_grouped.cu (group = 128: one activation scale per token per 128 rotated channels)
cudaError_t qvggt_launch_gemm_grouped(const qvggt_weights *w, const unsigned char *Xq, const float *a_scale, int M, void *Y,
                                      long long ldy, int *acc_debug, cudaStream_t st);


// gemm_c8.cu (codes in 8-bit containers: TMA feeds the tensor core directly)
cudaError_t qvggt_launch_gemm_c8(const qvggt_weights *w, const signed char *Xq8, const float *a_scale, int M, void *Y,
                                 long long ldy, int *acc_debug, cudaStream_t st);
// The same launch with the TMA producers switched off and a short wait limit: the first wait for operands runs
// out and the kernel leaves through its timeout path (exercised by the tests; nothing asynchronous is in flight).
cudaError_t qvggt_launch_gemm_c8_starved(const qvggt_weights *w, const signed char *Xq8, const float *a_scale, int M, void *Y,
                                         long long ldy, long long wait_limit_cycles, cudaStream_t st);
// The same GEMM for a handle that keeps only the packed weight codes: they are unpacked into w_scratch (int8 [N, K]) by a
// small kernel in front of the GEMM.
cudaError_t qvggt_launch_gemm_c8_packed_weights(const qvggt_weights *w, const signed char *Xq8, const float *a_scale, int M, void *Y,
                                                long long ldy, signed char *w_scratch, int *acc_debug, cudaStream_t st);
// The expansion alone.
cudaError_t qvggt_launch_unpack_w4(const qvggt_weights *w, signed char *w_scratch, cudaStream_t st);
// The same GEMM on weight codes that an earlier launch of the stream already expanded into w_expanded (int8 [N, K]).
cudaError_t qvggt_launch_gemm_c8_expanded(const qvggt_weights *w, const signed char *Xq8, const float *a_scale, int M, void *Y,
                                          long long ldy, const signed char *w_expanded, int *acc_debug, cudaStream_t st);
// One activation scale per token per 128 rotated channels on one-code-per-byte operands (a_scale [M, K/128]).
cudaError_t qvggt_launch_gemm_c8_grouped(const qvggt_weights *w, const signed char *Xq8, const float *a_scale, int M, void *Y,
                                         long long ldy, int *acc_debug, cudaStream_t st);
