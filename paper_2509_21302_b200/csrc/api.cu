// C-ABI entry points of libqvggt: argument validation, handle management, kernel launches.
#include <new>

#include "qvggt_internal.cuh"

namespace {

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

bool valid_k(int K) { return K == 1024 || K == 4096; }

int device_is_sm100()
{
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return 0;
    return major == 10;
}

void release(qvggt_weights *w)
{
    if (!w) return;
    cudaFree(w->Wq);
    cudaFree(w->Wq8);
    cudaFree(w->w_scale);
    cudaFree(w->amul);
    cudaFree(w->bias);
    cudaFree(w->status);
    delete w;
}

}  // namespace

extern "C" {

int qvggt_prepare_weights(const void *W_bf16, const void *bias_bf16, const float *smooth_c, const signed char *sign_v,
                          int N, int K, int flags, void *cuda_stream, qvggt_weights_t **out)
{
    if (flags & ~(QVGGT_PREP_C8 | QVGGT_PREP_W8A8 | QVGGT_PREP_C8_ONLY | QVGGT_PREP_W_TENSORWISE)) return QVGGT_ERR_UNSUPPORTED;
    const bool tensorwise = (flags & QVGGT_PREP_W_TENSORWISE) != 0;
    // the tensor-wise weight quantizer is built on the one-code-per-byte kernels: it needs a handle without packed copy
    if (tensorwise && !(flags & (QVGGT_PREP_W8A8 | QVGGT_PREP_C8_ONLY))) return QVGGT_ERR_UNSUPPORTED;
    const bool w8 = (flags & QVGGT_PREP_W8A8) != 0;       // 8-bit codes exist one per byte only
    const bool c8 = w8 || (flags & (QVGGT_PREP_C8 | QVGGT_PREP_C8_ONLY)) != 0;
    const bool packed = !w8 && !(flags & QVGGT_PREP_C8_ONLY);
    if (!out) return QVGGT_ERR_NULL;
    *out = nullptr;
    if (!W_bf16 || !smooth_c) return QVGGT_ERR_NULL;
    if (!valid_k(K) || N <= 0 || N % 128 != 0) return QVGGT_ERR_SHAPE;
    if (!aligned16(W_bf16)) return QVGGT_ERR_ALIGN;
    if (!device_is_sm100()) return QVGGT_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);

    qvggt_weights *w = new (std::nothrow) qvggt_weights();
    if (!w) return QVGGT_ERR_NOMEM;
    w->N = N;
    w->K = K;
    w->bits = w8 ? 8 : 4;
    w->Wq = nullptr; w->Wq8 = nullptr; w->w_scale = nullptr; w->amul = nullptr; w->bias = nullptr; w->status = nullptr;
    cudaGetDevice(&w->device);
    float *wmul = nullptr;                                   // [K] multipliers, followed by one float for the tensor-wise step size
    bool ok = (!packed || cudaMalloc(&w->Wq, (size_t)N * K / 2) == cudaSuccess) &&
              cudaMalloc(&w->w_scale, sizeof(float) * N) == cudaSuccess &&
              cudaMalloc(&w->amul, sizeof(float) * K) == cudaSuccess &&
              cudaMalloc(&w->status, sizeof(int)) == cudaSuccess &&
              cudaMallocAsync(&wmul, sizeof(float) * (K + 4), st) == cudaSuccess &&
              (!bias_bf16 || cudaMalloc(&w->bias, sizeof(uint16_t) * N) == cudaSuccess) &&
              (!c8 || cudaMalloc(&w->Wq8, (size_t)N * K) == cudaSuccess);
    if (!ok) {
        cudaGetLastError();
        if (wmul) cudaFreeAsync(wmul, st);
        release(w);
        return QVGGT_ERR_NOMEM;
    }
    cudaError_t e = cudaMemsetAsync(w->status, 0, sizeof(int), st);
    if (e == cudaSuccess && bias_bf16)
        e = cudaMemcpyAsync(w->bias, bias_bf16, sizeof(uint16_t) * N, cudaMemcpyDeviceToDevice, st);
    if (e == cudaSuccess) e = qvggt_launch_multipliers(smooth_c, sign_v, K, w->amul, wmul, st);
    if (e == cudaSuccess && w->Wq) e = qvggt_launch_rsq(W_bf16, K, N, K, wmul, 0, w->Wq, w->w_scale, st);
    if (e == cudaSuccess && w->Wq8) e = qvggt_launch_rsq_c8(W_bf16, K, N, K, wmul, w->bits, w->Wq8, w->w_scale, st);
    if (e == cudaSuccess && tensorwise) {
        // one step size for the whole tensor (Tab. "granularity"): the largest of the per-row step sizes just computed,
        // i.e. max|W~| / qmax (the division is monotone), then the static quantizer, which also writes that step as every row's scale
        e = qvggt_launch_max_reduce(w->w_scale, N, wmul + K, st);
        if (e == cudaSuccess) e = qvggt_launch_rsq_static_c8(W_bf16, K, N, K, wmul, w->bits, wmul + K, w->Wq8, w->w_scale, st);
    }
    // wmul is scratch: stream-ordered release so that the call stays asynchronous
    if (cudaFreeAsync(wmul, st) != cudaSuccess) cudaGetLastError();
    if (e != cudaSuccess) {
        cudaStreamSynchronize(st);
        release(w);
        return QVGGT_ERR_CUDA;
    }
    *out = w;
    return QVGGT_OK;
}

int qvggt_rotate_smooth_quantize(const qvggt_weights_t *w, const void *X_bf16, long long ldx, int M, int group,
                                 unsigned char *Xq, float *a_scale, void *cuda_stream)
{
    if (!w) return QVGGT_ERR_NULL;
    if (M < 0) return QVGGT_ERR_SHAPE;
    if ((group != 0 && group != 128) || w->bits != 4) return QVGGT_ERR_UNSUPPORTED;
    if (M == 0) return QVGGT_OK;
    if (!X_bf16 || !Xq || !a_scale) return QVGGT_ERR_NULL;
    if (ldx < w->K) return QVGGT_ERR_SHAPE;
    if (ldx % 8 != 0 || !aligned16(X_bf16) || !aligned16(Xq) || (reinterpret_cast<uintptr_t>(a_scale) & 3u)) return QVGGT_ERR_ALIGN;
    cudaError_t e = qvggt_launch_rsq(X_bf16, ldx, M, w->K, w->amul, group, Xq, a_scale, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? QVGGT_OK : QVGGT_ERR_CUDA;
}

int qvggt_w4a4_linear(const qvggt_weights_t *w, const unsigned char *Xq, const float *a_scale, int M, int group,
                      void *Y_bf16, long long ldy, int *acc_debug, void *cuda_stream)
{
    if (!w) return QVGGT_ERR_NULL;
    if (M < 0) return QVGGT_ERR_SHAPE;
    if ((group != 0 && group != 128) || w->bits != 4 || !w->Wq) return QVGGT_ERR_UNSUPPORTED;
    if (M == 0) return QVGGT_OK;
    if (!Xq || !a_scale || !Y_bf16) return QVGGT_ERR_NULL;
    if (ldy < w->N) return QVGGT_ERR_SHAPE;
    if (ldy % 8 != 0 || !aligned16(Xq) || !aligned16(Y_bf16) || (acc_debug && !aligned16(acc_debug)) ||
        (reinterpret_cast<uintptr_t>(a_scale) & 3u))
        return QVGGT_ERR_ALIGN;
    cudaError_t e = qvggt_launch_gemm(w, Xq, a_scale, M, group, Y_bf16, ldy, acc_debug, static_cast<cudaStream_t>(cuda_stream));
    if (e == cudaErrorNotSupported) return QVGGT_ERR_UNSUPPORTED;
    return e == cudaSuccess ? QVGGT_OK : QVGGT_ERR_CUDA;
}

int qvggt_rotate_smooth_quantize_c8(const qvggt_weights_t *w, const void *X_bf16, long long ldx, int M, signed char *Xq8,
                                    float *a_scale, void *cuda_stream)
{
    if (!w) return QVGGT_ERR_NULL;
    if (M < 0) return QVGGT_ERR_SHAPE;
    if (M == 0) return QVGGT_OK;
    if (!X_bf16 || !Xq8 || !a_scale) return QVGGT_ERR_NULL;
    if (ldx < w->K) return QVGGT_ERR_SHAPE;
    if (ldx % 8 != 0 || !aligned16(X_bf16) || !aligned16(Xq8) || (reinterpret_cast<uintptr_t>(a_scale) & 3u)) return QVGGT_ERR_ALIGN;
    cudaError_t e = qvggt_launch_rsq_c8(X_bf16, ldx, M, w->K, w->amul, w->bits, Xq8, a_scale, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? QVGGT_OK : QVGGT_ERR_CUDA;
}

int qvggt_rotate_smooth_quantize_c8_expand(const qvggt_weights_t *w, const void *X_bf16, long long ldx, int M, signed char *Xq8,
                                           float *a_scale, signed char *w_scratch, void *cuda_stream)
{
    if (!w) return QVGGT_ERR_NULL;
    if (M < 0) return QVGGT_ERR_SHAPE;
    if (!w->Wq || w->bits != 4) return QVGGT_ERR_UNSUPPORTED;
    if (!w_scratch) return QVGGT_ERR_NULL;
    if (!aligned16(w_scratch)) return QVGGT_ERR_ALIGN;
    if (M == 0) {
        // no rows to quantize: the scratch is still filled, by the stand-alone expansion
        cudaError_t e0 = qvggt_launch_unpack_w4(w, w_scratch, static_cast<cudaStream_t>(cuda_stream));
        return e0 == cudaSuccess ? QVGGT_OK : QVGGT_ERR_CUDA;
    }
    if (!X_bf16 || !Xq8 || !a_scale) return QVGGT_ERR_NULL;
    if (ldx < w->K) return QVGGT_ERR_SHAPE;
    if (ldx % 8 != 0 || !aligned16(X_bf16) || !aligned16(Xq8) || (reinterpret_cast<uintptr_t>(a_scale) & 3u)) return QVGGT_ERR_ALIGN;
    cudaError_t e = qvggt_launch_rsq_c8(X_bf16, ldx, M, w->K, w->amul, w->bits, Xq8, a_scale, static_cast<cudaStream_t>(cuda_stream), 0,
                                        w->Wq, w_scratch, (long long)w->N * w->K);
    return e == cudaSuccess ? QVGGT_OK : QVGGT_ERR_CUDA;
}

int qvggt_rotate_smooth_quantize_c8_grouped(const qvggt_weights_t *w, const void *X_bf16, long long ldx, int M, signed char *Xq8,
                                            float *a_scale, void *cuda_stream)
{
    if (!w) return QVGGT_ERR_NULL;
    if (M < 0) return QVGGT_ERR_SHAPE;
    if (w->bits != 4) return QVGGT_ERR_UNSUPPORTED;
    if (M == 0) return QVGGT_OK;
    if (!X_bf16 || !Xq8 || !a_scale) return QVGGT_ERR_NULL;
    if (ldx < w->K) return QVGGT_ERR_SHAPE;
    if (ldx % 8 != 0 || !aligned16(X_bf16) || !aligned16(Xq8) || (reinterpret_cast<uintptr_t>(a_scale) & 3u)) return QVGGT_ERR_ALIGN;
    cudaError_t e = qvggt_launch_rsq_c8(X_bf16, ldx, M, w->K, w->amul, 4, Xq8, a_scale, static_cast<cudaStream_t>(cuda_stream), 128);
    return e == cudaSuccess ? QVGGT_OK : QVGGT_ERR_CUDA;
}

int qvggt_w4a4_linear_c8_grouped(const qvggt_weights_t *w, const signed char *Xq8, const float *a_scale, int M, void *Y_bf16,
                                 long long ldy, int *acc_debug, void *cuda_stream)
{
    if (!w) return QVGGT_ERR_NULL;
    if (M < 0) return QVGGT_ERR_SHAPE;
    if (!w->Wq8 || w->bits != 4) return QVGGT_ERR_UNSUPPORTED;
    if (M == 0) return QVGGT_OK;
    if (!Xq8 || !a_scale || !Y_bf16) return QVGGT_ERR_NULL;
    if (ldy < w->N) return QVGGT_ERR_SHAPE;
    if (ldy % 8 != 0 || !aligned16(Xq8) || !aligned16(Y_bf16) || (acc_debug && !aligned16(acc_debug)) ||
        (reinterpret_cast<uintptr_t>(a_scale) & 3u))
        return QVGGT_ERR_ALIGN;
    cudaError_t e = qvggt_launch_gemm_c8_grouped(w, Xq8, a_scale, M, Y_bf16, ldy, acc_debug, static_cast<cudaStream_t>(cuda_stream));
    if (e == cudaErrorNotSupported) return QVGGT_ERR_UNSUPPORTED;
    return e == cudaSuccess ? QVGGT_OK : QVGGT_ERR_CUDA;
}

int qvggt_rotate_smooth_quantize_tc(const qvggt_weights_t *w, const void *X_bf16, long long ldx, int M, unsigned char *Xq,
                                    float *a_scale, float *y_debug, void *cuda_stream)
{
    if (!w) return QVGGT_ERR_NULL;
    if (M < 0) return QVGGT_ERR_SHAPE;
    if (w->bits != 4) return QVGGT_ERR_UNSUPPORTED;
    if (M == 0) return QVGGT_OK;
    if (!X_bf16 || !Xq || !a_scale) return QVGGT_ERR_NULL;
    if (ldx < w->K) return QVGGT_ERR_SHAPE;
    if (ldx % 8 != 0 || !aligned16(X_bf16) || !aligned16(Xq) || (reinterpret_cast<uintptr_t>(a_scale) & 3u) || (y_debug && !aligned16(y_debug)))
        return QVGGT_ERR_ALIGN;
    cudaError_t e = qvggt_launch_rsq_tc(X_bf16, ldx, M, w->K, w->amul, 4, false, Xq, a_scale, y_debug, w->status,
                                        static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? QVGGT_OK : QVGGT_ERR_CUDA;
}

int qvggt_rotate_smooth_quantize_tc_c8(const qvggt_weights_t *w, const void *X_bf16, long long ldx, int M, signed char *Xq8,
                                       float *a_scale, float *y_debug, void *cuda_stream)
{
    if (!w) return QVGGT_ERR_NULL;
    if (M < 0) return QVGGT_ERR_SHAPE;
    if (M == 0) return QVGGT_OK;
    if (!X_bf16 || !Xq8 || !a_scale) return QVGGT_ERR_NULL;
    if (ldx < w->K) return QVGGT_ERR_SHAPE;
    if (ldx % 8 != 0 || !aligned16(X_bf16) || !aligned16(Xq8) || (reinterpret_cast<uintptr_t>(a_scale) & 3u) || (y_debug && !aligned16(y_debug)))
        return QVGGT_ERR_ALIGN;
    cudaError_t e = qvggt_launch_rsq_tc(X_bf16, ldx, M, w->K, w->amul, w->bits, true, Xq8, a_scale, y_debug, w->status,
                                        static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? QVGGT_OK : QVGGT_ERR_CUDA;
}

int qvggt_rotate_smooth_quantize_static_c8(const qvggt_weights_t *w, const void *X_bf16, long long ldx, int M,
                                           const float *delta, signed char *Xq8, float *a_scale, void *cuda_stream)
{
    if (!w) return QVGGT_ERR_NULL;
    if (M < 0) return QVGGT_ERR_SHAPE;
    if (M == 0) return QVGGT_OK;
    if (!X_bf16 || !Xq8 || !a_scale || !delta) return QVGGT_ERR_NULL;
    if (ldx < w->K) return QVGGT_ERR_SHAPE;
    if (ldx % 8 != 0 || !aligned16(X_bf16) || !aligned16(Xq8) || (reinterpret_cast<uintptr_t>(a_scale) & 3u) ||
        (reinterpret_cast<uintptr_t>(delta) & 3u))
        return QVGGT_ERR_ALIGN;
    cudaError_t e = qvggt_launch_rsq_static_c8(X_bf16, ldx, M, w->K, w->amul, w->bits, delta, Xq8, a_scale,
                                               static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? QVGGT_OK : QVGGT_ERR_CUDA;
}

int qvggt_layernorm_rotate_smooth_quantize_c8(const qvggt_weights_t *w, const void *X_bf16, long long ldx, int M,
                                              const float *gamma, const float *beta, float eps, signed char *Xq8,
                                              float *a_scale, void *cuda_stream)
{
    if (!w) return QVGGT_ERR_NULL;
    if (M < 0) return QVGGT_ERR_SHAPE;
    if (M == 0) return QVGGT_OK;
    if (!X_bf16 || !Xq8 || !a_scale || !gamma || !beta) return QVGGT_ERR_NULL;
    if (ldx < w->K) return QVGGT_ERR_SHAPE;
    if (ldx % 8 != 0 || !aligned16(X_bf16) || !aligned16(Xq8) || !aligned16(gamma) || !aligned16(beta) ||
        (reinterpret_cast<uintptr_t>(a_scale) & 3u))
        return QVGGT_ERR_ALIGN;
    cudaError_t e = qvggt_launch_ln_rsq_c8(X_bf16, ldx, M, w->K, w->amul, w->bits, gamma, beta, eps, Xq8, a_scale, nullptr,
                                           static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? QVGGT_OK : QVGGT_ERR_CUDA;
}

int qvggt_layernorm(const void *X_bf16, long long ldx, int M, int K, const float *gamma, const float *beta, float eps,
                    void *Y_bf16, void *cuda_stream)
{
    if (M < 0 || !valid_k(K)) return QVGGT_ERR_SHAPE;
    if (M == 0) return QVGGT_OK;
    if (!X_bf16 || !Y_bf16 || !gamma || !beta) return QVGGT_ERR_NULL;
    if (ldx < K) return QVGGT_ERR_SHAPE;
    if (ldx % 8 != 0 || !aligned16(X_bf16) || !aligned16(Y_bf16) || !aligned16(gamma) || !aligned16(beta)) return QVGGT_ERR_ALIGN;
    if (!device_is_sm100()) return QVGGT_ERR_UNSUPPORTED;
    cudaError_t e = qvggt_launch_ln_rsq_c8(X_bf16, ldx, M, K, nullptr, 4, gamma, beta, eps, nullptr, nullptr, Y_bf16,
                                           static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? QVGGT_OK : QVGGT_ERR_CUDA;
}

int qvggt_gelu_rotate_smooth_quantize_c8(const qvggt_weights_t *w, const void *X_bf16, long long ldx, int M, signed char *Xq8,
                                         float *a_scale, void *cuda_stream)
{
    if (!w) return QVGGT_ERR_NULL;
    if (M < 0) return QVGGT_ERR_SHAPE;
    if (M == 0) return QVGGT_OK;
    if (!X_bf16 || !Xq8 || !a_scale) return QVGGT_ERR_NULL;
    if (ldx < w->K) return QVGGT_ERR_SHAPE;
    if (ldx % 8 != 0 || !aligned16(X_bf16) || !aligned16(Xq8) || (reinterpret_cast<uintptr_t>(a_scale) & 3u)) return QVGGT_ERR_ALIGN;
    cudaError_t e = qvggt_launch_gelu_rsq_c8(X_bf16, ldx, M, w->K, w->amul, w->bits, Xq8, a_scale, nullptr, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? QVGGT_OK : QVGGT_ERR_CUDA;
}

int qvggt_gelu(const void *X_bf16, long long ldx, int M, int K, void *Y_bf16, void *cuda_stream)
{
    if (M < 0 || !valid_k(K)) return QVGGT_ERR_SHAPE;
    if (M == 0) return QVGGT_OK;
    if (!X_bf16 || !Y_bf16) return QVGGT_ERR_NULL;
    if (ldx < K) return QVGGT_ERR_SHAPE;
    if (ldx % 8 != 0 || !aligned16(X_bf16) || !aligned16(Y_bf16)) return QVGGT_ERR_ALIGN;
    if (!device_is_sm100()) return QVGGT_ERR_UNSUPPORTED;
    cudaError_t e = qvggt_launch_gelu_rsq_c8(X_bf16, ldx, M, K, nullptr, 4, nullptr, nullptr, Y_bf16, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? QVGGT_OK : QVGGT_ERR_CUDA;
}

int qvggt_w4a4_linear_c8(const qvggt_weights_t *w, const signed char *Xq8, const float *a_scale, int M, void *Y_bf16,
                         long long ldy, int *acc_debug, void *cuda_stream)
{
    if (!w) return QVGGT_ERR_NULL;
    if (M < 0) return QVGGT_ERR_SHAPE;
    if (!w->Wq8) return QVGGT_ERR_UNSUPPORTED;
    if (M == 0) return QVGGT_OK;
    if (!Xq8 || !a_scale || !Y_bf16) return QVGGT_ERR_NULL;
    if (ldy < w->N) return QVGGT_ERR_SHAPE;
    if (ldy % 8 != 0 || !aligned16(Xq8) || !aligned16(Y_bf16) || (acc_debug && !aligned16(acc_debug)) ||
        (reinterpret_cast<uintptr_t>(a_scale) & 3u))
        return QVGGT_ERR_ALIGN;
    cudaError_t e = qvggt_launch_gemm_c8(w, Xq8, a_scale, M, Y_bf16, ldy, acc_debug, static_cast<cudaStream_t>(cuda_stream));
    if (e == cudaErrorNotSupported) return QVGGT_ERR_UNSUPPORTED;
    return e == cudaSuccess ? QVGGT_OK : QVGGT_ERR_CUDA;
}

int qvggt_w4a4_linear_c8_packed_weights(const qvggt_weights_t *w, const signed char *Xq8, const float *a_scale, int M, void *Y_bf16,
                                        long long ldy, signed char *w_scratch, int *acc_debug, void *cuda_stream)
{
    if (!w) return QVGGT_ERR_NULL;
    if (M < 0) return QVGGT_ERR_SHAPE;
    if (!w->Wq) return QVGGT_ERR_UNSUPPORTED;
    if (M == 0) return QVGGT_OK;
    if (!Xq8 || !a_scale || !Y_bf16 || !w_scratch) return QVGGT_ERR_NULL;
    if (ldy < w->N) return QVGGT_ERR_SHAPE;
    if (ldy % 8 != 0 || !aligned16(Xq8) || !aligned16(Y_bf16) || !aligned16(w_scratch) || (acc_debug && !aligned16(acc_debug)) ||
        (reinterpret_cast<uintptr_t>(a_scale) & 3u))
        return QVGGT_ERR_ALIGN;
    cudaError_t e = qvggt_launch_gemm_c8_packed_weights(w, Xq8, a_scale, M, Y_bf16, ldy, w_scratch, acc_debug, static_cast<cudaStream_t>(cuda_stream));
    if (e == cudaErrorNotSupported) return QVGGT_ERR_UNSUPPORTED;
    return e == cudaSuccess ? QVGGT_OK : QVGGT_ERR_CUDA;
}

int qvggt_w4a4_linear_c8_expanded(const qvggt_weights_t *w, const signed char *Xq8, const float *a_scale, int M, void *Y_bf16,
                                  long long ldy, const signed char *w_scratch, int *acc_debug, void *cuda_stream)
{
    if (!w) return QVGGT_ERR_NULL;
    if (M < 0) return QVGGT_ERR_SHAPE;
    if (w->bits != 4) return QVGGT_ERR_UNSUPPORTED;
    if (M == 0) return QVGGT_OK;
    if (!Xq8 || !a_scale || !Y_bf16 || !w_scratch) return QVGGT_ERR_NULL;
    if (ldy < w->N) return QVGGT_ERR_SHAPE;
    if (ldy % 8 != 0 || !aligned16(Xq8) || !aligned16(Y_bf16) || !aligned16(w_scratch) || (acc_debug && !aligned16(acc_debug)) ||
        (reinterpret_cast<uintptr_t>(a_scale) & 3u))
        return QVGGT_ERR_ALIGN;
    cudaError_t e = qvggt_launch_gemm_c8_expanded(w, Xq8, a_scale, M, Y_bf16, ldy, w_scratch, acc_debug, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? QVGGT_OK : QVGGT_ERR_CUDA;
}

int qvggt_debug_starved_linear_c8(const qvggt_weights_t *w, const signed char *Xq8, const float *a_scale, int M, void *Y_bf16,
                                  long long ldy, long long wait_limit_cycles, void *cuda_stream)
{
    if (!w) return QVGGT_ERR_NULL;
    if (!w->Wq8) return QVGGT_ERR_UNSUPPORTED;
    if (M < 1 || ldy < w->N || wait_limit_cycles < 1000 || wait_limit_cycles > 2000000000LL) return QVGGT_ERR_SHAPE;
    if (!Xq8 || !a_scale || !Y_bf16) return QVGGT_ERR_NULL;
    if (ldy % 8 != 0 || !aligned16(Xq8) || !aligned16(Y_bf16) || (reinterpret_cast<uintptr_t>(a_scale) & 3u)) return QVGGT_ERR_ALIGN;
    cudaError_t e = qvggt_launch_gemm_c8_starved(w, Xq8, a_scale, M, Y_bf16, ldy, wait_limit_cycles, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? QVGGT_OK : QVGGT_ERR_CUDA;
}

void qvggt_free_weights(qvggt_weights_t *w)
{
    if (!w) return;
    int cur = 0;
    cudaGetDevice(&cur);
    const int owner = w->device;
    if (cur != owner) cudaSetDevice(owner);
    cudaDeviceSynchronize();
    release(w);
    if (cur != owner) cudaSetDevice(cur);
}

int qvggt_weights_view(const qvggt_weights_t *w, const unsigned char **Wq, const float **w_scale, const float **amul,
                       const void **bias_bf16, int *N, int *K)
{
    if (!w) return QVGGT_ERR_NULL;
    if (Wq) *Wq = w->Wq;
    if (w_scale) *w_scale = w->w_scale;
    if (amul) *amul = w->amul;
    if (bias_bf16) *bias_bf16 = w->bias;
    if (N) *N = w->N;
    if (K) *K = w->K;
    return QVGGT_OK;
}

int qvggt_weights_view_c8(const qvggt_weights_t *w, const signed char **Wq8, int *bits)
{
    if (!w || !Wq8) return QVGGT_ERR_NULL;
    *Wq8 = w->Wq8;
    if (bits) *bits = w->bits;
    return QVGGT_OK;
}

int qvggt_device_status(const qvggt_weights_t *w, void *cuda_stream, int *code)
{
    if (!w || !code) return QVGGT_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (cudaStreamSynchronize(st) != cudaSuccess) return QVGGT_ERR_CUDA;
    if (cudaMemcpy(code, w->status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return QVGGT_ERR_CUDA;
    return *code == 0 ? QVGGT_OK : QVGGT_ERR_DEVICE_TIMEOUT;
}

int qvggt_calibrate_smooth(const void *X_calib_bf16, int Mc, const void *W_bf16, int N, int K, float alpha, float lo,
                           float hi, float *colmax_scratch, float *smooth_c, void *cuda_stream)
{
    if (!X_calib_bf16 || !W_bf16 || !colmax_scratch || !smooth_c) return QVGGT_ERR_NULL;
    if (!valid_k(K) || Mc <= 0 || N <= 0) return QVGGT_ERR_SHAPE;
    if (!aligned16(X_calib_bf16) || !aligned16(W_bf16)) return QVGGT_ERR_ALIGN;
    if (!device_is_sm100()) return QVGGT_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e = cudaMemsetAsync(colmax_scratch, 0, sizeof(float) * 2 * K, st);
    if (e == cudaSuccess) e = qvggt_launch_colmax(X_calib_bf16, Mc, K, colmax_scratch, st);
    if (e == cudaSuccess) e = qvggt_launch_colmax(W_bf16, N, K, colmax_scratch + K, st);
    if (e == cudaSuccess) e = qvggt_launch_smooth_finalize(colmax_scratch, colmax_scratch + K, K, alpha, lo, hi, smooth_c, st);
    return e == cudaSuccess ? QVGGT_OK : QVGGT_ERR_CUDA;
}

const char *qvggt_status_string(int status)
{
    switch (status) {
        case QVGGT_OK: return "ok";
        case QVGGT_ERR_NULL: return "a required pointer is NULL";
        case QVGGT_ERR_SHAPE: return "unsupported shape (K must be 1024 or 4096, N a multiple of 128, M >= 0, ld >= row length)";
        case QVGGT_ERR_ALIGN: return "pointer or leading dimension violates the 16-byte alignment rule";
        case QVGGT_ERR_UNSUPPORTED: return "unsupported option or device (group must be 0 or 128; device must be sm_100)";
        case QVGGT_ERR_CUDA: return "a CUDA runtime call failed";
        case QVGGT_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait expired";
        case QVGGT_ERR_NOMEM: return "out of memory";
        default: return "unknown status";
    }
}

}  // extern "C"
