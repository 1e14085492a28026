// Weight quantization for callers that must not allocate device memory.
//
// qvggt_prepare_weights allocates: the handle's arrays, plus a temporary [K] fp32 vector holding
// the weight-side multipliers wmul[k] = (v[k] K^-1/2) * c[k].  Some callers cannot afford that --
// a serving process that has handed every byte of device memory to its own arena at start-up (a
// late cudaMalloc then fails or fragments), or a latency-critical section where the implicit
// device-wide synchronisation of cudaMalloc/cudaFree is not acceptable.  For them this file offers
// one entry point that writes into caller-provided outputs and keeps the temporary vector in a
// fixed array that lives in the library image, so no allocator (CUDA's or PyTorch's) is called.
//
// The array is file-scope device memory: every GPU that loads the library holds its 16 KB until
// the process exits.  In host code its name is only a stand-in for the symbol; the device address
// is looked up per device with cudaGetSymbolAddress and cached.
#include <mutex>

#include "qvggt_internal.cuh"

namespace {

constexpr int kStaticMaxK = 4096;   // largest inner dimension the fixed scratch can serve

static __device__ __align__(256) float g_wmul_scratch[kStaticMaxK];

constexpr int kMaxDevices = 64;
float *g_scratch_addr[kMaxDevices];   // device address of g_wmul_scratch on each device, 0 = not looked up yet
std::mutex g_scratch_mutex;

// Resolves (once per device, with that device current) the device address of the scratch array.
cudaError_t scratch_for_current_device(float **out)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_addr[dev]) {
        void *p = nullptr;
        e = cudaGetSymbolAddress(&p, g_wmul_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_addr[dev] = static_cast<float *>(p);
    }
    *out = g_scratch_addr[dev];
    return cudaSuccess;
}

}  // namespace

extern "C" int qvggt_quantize_weights_static(const void *W_bf16, const float *smooth_c, const signed char *sign_v,
                                             int N, int K, unsigned char *Wq, float *w_scale, float *amul,
                                             void *cuda_stream)
{
    if (!W_bf16 || !smooth_c || !Wq || !w_scale || !amul) return QVGGT_ERR_NULL;
    if (K > kStaticMaxK) return QVGGT_ERR_SHAPE;                 // beyond the fixed scratch: refuse, never overrun
    if ((K != 1024 && K != 4096) || N <= 0) return QVGGT_ERR_SHAPE;
    if ((reinterpret_cast<uintptr_t>(W_bf16) & 15u) || (reinterpret_cast<uintptr_t>(Wq) & 15u) ||
        (reinterpret_cast<uintptr_t>(w_scale) & 3u) || (reinterpret_cast<uintptr_t>(amul) & 3u))
        return QVGGT_ERR_ALIGN;
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
        return QVGGT_ERR_CUDA;
    if (major != 10) return QVGGT_ERR_UNSUPPORTED;               // the kernels exist for sm_100 only
    float *wmul = nullptr;
    if (scratch_for_current_device(&wmul) != cudaSuccess) return QVGGT_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    // wmul[0..K) is fully rewritten before it is read, so nothing left by an earlier call matters.
    cudaError_t e = qvggt_launch_multipliers(smooth_c, sign_v, K, amul, wmul, st);
    if (e == cudaSuccess) e = qvggt_launch_rsq(W_bf16, K, N, K, wmul, 0, Wq, w_scale, st);
    return e == cudaSuccess ? QVGGT_OK : QVGGT_ERR_CUDA;
}
