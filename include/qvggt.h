/*
 * qvggt -- W4A4 linear layer of Dual-Smoothed Fine-Grained Quantization (QuantVGGT, Sec. 3.2)
 * for NVIDIA B200 (sm_100a).  C ABI: plain pointers and sizes, no C++ or framework types.
 *
 * The layer computes an approximation of  Y = X W^T + b  (X: [M tokens, K], W: [N, K]) as
 *
 *   Y[m][n] = a_scale[m] * w_scale[n] * sum_k Xq[m][k] * Wq[n][k] + b[n]
 *
 * where, with the random Hadamard rotation H = K^{-1/2} H_K diag(v) ("Pre-Global-Rotation") and
 * the per-rotated-channel smoothing factors c ("Post-Local-Smooth", Eq. "smooth_factor"),
 *
 *   Xq, a_scale = quant4_per_token  ( X H diag(c)^{-1} )      (online,  qvggt_rotate_smooth_quantize)
 *   Wq, w_scale = quant4_per_channel( W H diag(c)      )      (offline, qvggt_prepare_weights)
 *
 * and quant4 is the symmetric quantizer of Eq. "quantization" with N = 4 bits:
 * Delta = max|x| / 7, q = clamp(round(x / Delta), -8, 7), round = half-to-even.  Because only the
 * inner dimension is summed, both scales stay outside the integer sum ("Fine-Grained Quantization
 * Granularity"), which runs on the int8 tensor cores with int32 accumulation.
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer unless stated otherwise; matrices are row-major; the caller
 *     owns every buffer except the opaque weights handle.
 *   - bf16 buffers are passed as void*; packed int4 buffers as unsigned char*: byte i of a row holds
 *     code 2i in bits 0-3 and code 2i+1 in bits 4-7, two's complement.
 *   - K must be 1024 or 4096 (the rotation is a power-of-two Hadamard; other sizes: QVGGT_ERR_SHAPE).
 *     N must be a multiple of 128.  M >= 0 (M == 0 is a no-op).
 *   - `group` selects the activation-scale granularity: 0 = one scale per token (the paper's
 *     setting); 128 = one scale per token per 128 consecutive rotated channels (an extension; the
 *     integer partial sums are rescaled per group in the epilogue).
 *   - All work is enqueued on `cuda_stream` (a cudaStream_t passed as void*, NULL = default
 *     stream); no call synchronises the device except where stated.
 *     The quantize and *_c8 GEMM kernels are launched with programmatic stream serialization allowed:
 *     their blocks may become resident while the previous kernel of the stream drains, but they touch
 *     no global memory before that kernel has completed, so stream order is what the caller sees.
 *   - Return value: QVGGT_OK or a negative qvggt_status_t.  Arguments are validated on the host
 *     before anything is launched; nothing throws or exits.
 *   - Device-side waits are bounded.  If one expires the kernel records a code in the handle's
 *     status word and returns; read it with qvggt_device_status().
 *   - One process may drive several devices: a handle is bound to the device that was current when it was
 *     prepared, every other call uses the current device, and the library's caches (kernel attributes,
 *     occupancy, SM count) are kept per device.
 *   - A handle is read-only during launches (its status word apart), so one handle may be used from several
 *     streams and host threads at once as long as the calls' output buffers and scratch are distinct; preparing and
 *     freeing a handle must not overlap calls that use it.
 */
#ifndef QVGGT_H
#define QVGGT_H

#ifdef __cplusplus
extern "C" {
#endif

typedef struct qvggt_weights qvggt_weights_t; /* opaque; owns Wq, w_scale, amul, bias, status word on the device */

typedef enum {
    QVGGT_OK = 0,
    QVGGT_ERR_NULL = -1,           /* a required pointer is NULL */
    QVGGT_ERR_SHAPE = -2,          /* K not in {1024, 4096}, N not a multiple of 128, M < 0, bad leading dimension */
    QVGGT_ERR_ALIGN = -3,          /* a pointer or leading dimension breaks the 16-byte alignment rule */
    QVGGT_ERR_UNSUPPORTED = -4,    /* group not in {0, 128}; device is not sm_100 */
    QVGGT_ERR_CUDA = -5,           /* a CUDA runtime call failed (launch, allocation, copy) */
    QVGGT_ERR_DEVICE_TIMEOUT = -6, /* a bounded device-side wait expired (see qvggt_device_status) */
    QVGGT_ERR_NOMEM = -7           /* device allocation failed */
} qvggt_status_t;

/*
 * Offline weight path (Sec. 3.2: fold the rotation and the smoothing factors into W, then
 * out-channel-wise symmetric int4).  Per weight row n:
 *   u = FWHT_K(W[n][:])   un-normalised Sylvester transform, fp32 radix-2 butterflies, strides 1,2,4,..
 *   y[k] = u[k] * wmul[k],  wmul[k] = (v[k] K^{-1/2}) * c[k]
 *   w_scale[n] = max_k|y| / 7,  Wq[n][k] = round(y[k] * (7 / max_k|y|))
 * Also stores amul[k] = (v[k] K^{-1/2}) / c[k] for the activation path and a copy of the bias.
 *   W_bf16    [N, K] bf16, 16-byte aligned
 *   bias_bf16 [N] bf16 or NULL (no bias)
 *   smooth_c  [K] fp32, finite and > 0
 *   sign_v    [K] int8 of +1/-1, or NULL (all +1)
 *   flags     0, QVGGT_PREP_C8 to keep an extra int8 [N, K] copy of the codes for the *_c8 entry points (1.5 bytes
 *             per weight in all), QVGGT_PREP_C8_ONLY to keep only that copy (1 byte per weight), or
 *             QVGGT_PREP_W8A8 for 8-bit codes (see the *_c8 entry points)
 *   out       receives a new handle (device memory is allocated here, on the current device);
 *             release it with qvggt_free_weights.  The handle is bound to that device.
 * Work is enqueued on the stream; the inputs may be released once the stream has passed this call.
 */
int qvggt_prepare_weights(const void *W_bf16, const void *bias_bf16, const float *smooth_c,
                          const signed char *sign_v, int N, int K, int flags, void *cuda_stream,
                          qvggt_weights_t **out);

/*
 * Online activation path (Sec. 3.2: X H diag(c)^{-1}, then dynamic token-wise symmetric int4).
 * Per token row m:  u = FWHT_K(X[m][:]);  y[k] = u[k] * amul[k];  per scale group:
 *   a_scale = max|y| / 7 (max floored at 1e-8),  Xq = round(y * (7 / max|y|)).
 *   w        handle from qvggt_prepare_weights (supplies K and amul)
 *   X_bf16   [M, K] bf16 with row stride ldx elements (ldx >= K, ldx % 8 == 0), 16-byte aligned
 *   group    0 or 128
 *   Xq       [M, K/2] packed int4, 16-byte aligned
 *   a_scale  fp32 [M] (group 0) or [M, K/128] (group 128)
 */
int qvggt_rotate_smooth_quantize(const qvggt_weights_t *w, const void *X_bf16, long long ldx, int M,
                                 int group, unsigned char *Xq, float *a_scale, void *cuda_stream);

/*
 * Integer GEMM + rescale + bias + bf16 (Sec. 3.2, granularity paragraph: scales factor out of the sum).
 *   group 0:    Y[m][n] = bf16( float(acc[m][n]) * (a_scale[m] * w_scale[n]) + bias[n] ),
 *               acc[m][n] = sum_k Xq[m][k] Wq[n][k]   (int32, exact)
 *   group 128:  Y[m][n] = bf16( (sum_g float(acc_g[m][n]) * a_scale[m][g]) * w_scale[n] + bias[n] ),
 *               g ascending over the K/128 groups
 *   Xq, a_scale as written by qvggt_rotate_smooth_quantize with the same `group`
 *   Y_bf16      [M, N] bf16 with row stride ldy elements (ldy >= N, ldy % 8 == 0), 16-byte aligned
 *   acc_debug   NULL, or int32 [M, N] (group 0) / [K/128, M, N] (group 128): the raw integer sums
 */
int qvggt_w4a4_linear(const qvggt_weights_t *w, const unsigned char *Xq, const float *a_scale, int M,
                      int group, void *Y_bf16, long long ldy, int *acc_debug, void *cuda_stream);

/*
 * The same two steps on codes held one per byte ("8-bit containers").  tcgen05 has no 4-bit integer
 * kind, so the tensor core multiplies int8 whatever the storage format; when the producers write one
 * code per byte, the tiles go from global memory straight into the tensor core's operand stages and
 * the GEMM spends nothing on unpacking.  Codes, scales, integer sums and outputs are those of the
 * packed entry points, bit for bit; only the layout of Xq differs.  The handle must have been
 * prepared with QVGGT_PREP_C8 in `flags` (which adds an int8 [N, K] copy of Wq to the handle: 1 byte
 * per weight on top of the packed 0.5) or with QVGGT_PREP_C8_ONLY (that copy alone), otherwise
 * QVGGT_ERR_UNSUPPORTED.  Per-token scales here; the *_c8_grouped pair below takes group-wise scales.
 *   Xq8      int8 [M, K], one code per byte in [-7, 7], natural element order, 16-byte aligned
 *   a_scale  fp32 [M]
 *   Y_bf16, ldy, acc_debug (int32 [M, N]) as for qvggt_w4a4_linear with group 0
 *
 * W8A8 (the paper's other setting, Eq. "quantization" with N = 8: Delta = max|x| / 127, codes in [-127, 127]) uses the
 * same two calls: a handle prepared with QVGGT_PREP_W8A8 holds 8-bit weight codes (one per byte only: there is no
 * packed copy, and the packed entry points refuse it with QVGGT_ERR_UNSUPPORTED), qvggt_rotate_smooth_quantize_c8
 * then quantizes the activations to 8 bits, and qvggt_w4a4_linear_c8 multiplies them: the integer sums stay below
 * 2^31 (127^2 * 4096), the epilogue is the same.
 */
#define QVGGT_PREP_C8 1
#define QVGGT_PREP_W8A8 2
#define QVGGT_PREP_C8_ONLY 4 /* 4-bit codes one per byte only, no packed copy (1 byte per weight; the packed entry points refuse the handle) */
#define QVGGT_PREP_W_TENSORWISE 8 /* weights with ONE step size for the whole tensor (the tensor-wise arm of Tab. "granularity") instead of one
                                     per output channel: Delta = max|W~| / qmax, w_scale[n] = Delta for every n; needs QVGGT_PREP_C8_ONLY or
                                     QVGGT_PREP_W8A8 (otherwise QVGGT_ERR_UNSUPPORTED) */
int qvggt_rotate_smooth_quantize_c8(const qvggt_weights_t *w, const void *X_bf16, long long ldx, int M,
                                    signed char *Xq8, float *a_scale, void *cuda_stream);
int qvggt_w4a4_linear_c8(const qvggt_weights_t *w, const signed char *Xq8, const float *a_scale, int M,
                         void *Y_bf16, long long ldy, int *acc_debug, void *cuda_stream);

/*
 * Group-wise activation scales (group = 128, see qvggt_rotate_smooth_quantize / qvggt_w4a4_linear) on codes held one per byte:
 * the same codes, scales, integer partial sums and outputs as the packed entry points with group = 128, bit for bit, on the
 * TMA-fed GEMM (about twice as fast as the packed group-wise GEMM).  4-bit codes only; the handle needs QVGGT_PREP_C8[_ONLY].
 *   Xq8      int8 [M, K];  a_scale fp32 [M, K/128];  acc_debug NULL or int32 [K/128, M, N]
 */
int qvggt_rotate_smooth_quantize_c8_grouped(const qvggt_weights_t *w, const void *X_bf16, long long ldx, int M,
                                            signed char *Xq8, float *a_scale, void *cuda_stream);
int qvggt_w4a4_linear_c8_grouped(const qvggt_weights_t *w, const signed char *Xq8, const float *a_scale, int M,
                                 void *Y_bf16, long long ldy, int *acc_debug, void *cuda_stream);

/*
 * The one-code-per-byte GEMM for a handle that keeps ONLY the packed weight codes (flags = 0 at preparation: 0.5 bytes
 * per weight, the paper's memory footprint, Tab. "efficiency").  A small kernel in front of the GEMM unpacks the
 * layer's codes into w_scratch, from where the GEMM's TMA loads read them back (a few megabytes: they stay in L2), so
 * the weights exist unpacked only transiently and only one layer at a time.  Activations as written by
 * qvggt_rotate_smooth_quantize_c8 / _tc_c8 (which need nothing but the handle's multipliers).  Results are those of
 * qvggt_w4a4_linear_c8 bit for bit.
 *   w_scratch  int8 [N, K] device scratch supplied by the caller, 16-byte aligned, overwritten; one scratch may serve
 *              every layer as long as the calls that share it are ordered on one stream
 */
int qvggt_w4a4_linear_c8_packed_weights(const qvggt_weights_t *w, const signed char *Xq8, const float *a_scale, int M,
                                        void *Y_bf16, long long ldy, signed char *w_scratch, int *acc_debug,
                                        void *cuda_stream);

/*
 * The same pair of steps for a packed-codes-only handle with the expansion folded into the quantize launch, so that a
 * layer costs two launches as with a QVGGT_PREP_C8 handle (Tab. "efficiency": the memory footprint of 4-bit weights
 * without giving up the latency).  qvggt_rotate_smooth_quantize_c8_expand is qvggt_rotate_smooth_quantize_c8 (same
 * codes and scales bit for bit, per-token scales, 4-bit handles) whose thread blocks, while their first rows are in
 * flight from memory, also expand the handle's packed weight codes into w_scratch between them;
 * qvggt_w4a4_linear_c8_expanded is qvggt_w4a4_linear_c8 reading the weight codes from w_scratch.  The caller keeps the
 * pair together: w_scratch must hold THIS handle's codes, written by an _expand call (or by
 * qvggt_w4a4_linear_c8_packed_weights) ordered before the GEMM on the same stream, with no other write to it in between.
 * M = 0: _expand still fills w_scratch; _expanded does nothing.
 *   w_scratch  int8 [N, K] device scratch supplied by the caller, 16-byte aligned
 * QVGGT_ERR_UNSUPPORTED: the handle holds no packed codes (QVGGT_PREP_C8_ONLY) or is not 4-bit.
 */
int qvggt_rotate_smooth_quantize_c8_expand(const qvggt_weights_t *w, const void *X_bf16, long long ldx, int M,
                                           signed char *Xq8, float *a_scale, signed char *w_scratch, void *cuda_stream);
int qvggt_w4a4_linear_c8_expanded(const qvggt_weights_t *w, const signed char *Xq8, const float *a_scale, int M,
                                  void *Y_bf16, long long ldy, const signed char *w_scratch, int *acc_debug,
                                  void *cuda_stream);

/*
 * The activation path with the bulk of the rotation on the tensor core (Sec. 3.2, Pre-Global-Rotation: the Kronecker
 * recursion H_{2^n} = H_2 (x) H_{2^(n-1)} lets the transform factor over any split of the index bits).  Index bits
 * 3..9 are transformed by one product with the +-1 matrix H_128 (bf16 operands: every product exact, fp32
 * accumulation inside the tensor core), the other 3 (K = 1024) or 5 (K = 4096) bits by fp32 butterflies, then
 * multiplier, per-token absolute maximum and Eq. "quantization" as in qvggt_rotate_smooth_quantize[_c8].
 * Same arguments, same layouts, per-token scales only, about 2.5 x fewer instructions per row than the exact kernel.
 * NOT bit-exact against the exact entry points: an fp32 transform depends on the order of its additions, and the
 * tensor core's is its own.  Contract, against the rotation evaluated without intermediate rounding
 * (u* = x H_K exactly, y* = u* amul, S = sum_k |x_k| of the row, tau = 2 log2(K) 2^-24):
 *   rotated values   |y[k] - y*[k]| <= (tau S + 2^-24 |u*[k]|) |amul[k]|
 *   scale            within max_k of that bound, divided by qmax, of max|y*| / qmax
 *   codes            the nearest integer to qmax y*[k] / max|y*|, except within that bound (in code units) of a
 *                    half-integer, where the other neighbour may be returned (off by one, never more)
 * (the exact entry points' own fp32 transform is only guaranteed log2(K) 2^-24 S).  The GEMM entry points take the
 * codes of either mode.
 *   y_debug  NULL, or fp32 [M, K] (16-byte aligned): receives the rotated, smoothed rows y
 */
int qvggt_rotate_smooth_quantize_tc(const qvggt_weights_t *w, const void *X_bf16, long long ldx, int M,
                                    unsigned char *Xq, float *a_scale, float *y_debug, void *cuda_stream);
int qvggt_rotate_smooth_quantize_tc_c8(const qvggt_weights_t *w, const void *X_bf16, long long ldx, int M,
                                       signed char *Xq8, float *a_scale, float *y_debug, void *cuda_stream);

/*
 * Static tensor-wise activation quantizer: the other arm of the paper's granularity ablation (Tab. "granularity",
 * dynamic token-wise against static tensor-wise).  One step size for the whole tensor, fixed offline, instead of
 * one per token from the token's absolute maximum:  Xq8 = clamp(round(y * fl(1 / delta)), -2^(N-1), 2^(N-1) - 1)
 * (Eq. "quantization" with its clamp active; N = the handle's code width), a_scale[m] = delta for every m, so that
 * qvggt_w4a4_linear_c8 follows unchanged.
 *   delta    DEVICE pointer to one fp32 step size (> 0, finite); read by the kernel, not by the host
 */
int qvggt_rotate_smooth_quantize_static_c8(const qvggt_weights_t *w, const void *X_bf16, long long ldx, int M,
                                           const float *delta, signed char *Xq8, float *a_scale, void *cuda_stream);

/*
 * Upstream fusion (Sec. 3.2 places the quantized linears of a block behind its normalization layers): LayerNorm over
 * the K channels of every token, then the activation path of qvggt_rotate_smooth_quantize_c8, in one pass over X --
 * the normalized activations never go to memory.  The result is, bit for bit, that of qvggt_layernorm followed by
 * qvggt_rotate_smooth_quantize_c8.  LayerNorm in fp32, one rounding per operation, statistics summed pairwise
 * (the sum of n terms is fl(sum of the first half + sum of the second half), recursively):
 *   mean = sum(x) / K;  d = x - mean;  var = sum(d * d) / K;  rstd = 1 / sqrt(var + eps)
 *   ln[k] = bf16( (d[k] * rstd) * gamma[k] + beta[k] )
 *   gamma, beta  fp32 [K], 16-byte aligned;  other arguments as for qvggt_rotate_smooth_quantize_c8
 */
int qvggt_layernorm_rotate_smooth_quantize_c8(const qvggt_weights_t *w, const void *X_bf16, long long ldx, int M,
                                              const float *gamma, const float *beta, float eps, signed char *Xq8,
                                              float *a_scale, void *cuda_stream);

/* The same LayerNorm alone (the unfused arm): Y_bf16 [M, K] contiguous bf16.  K must be 1024 or 4096. */
int qvggt_layernorm(const void *X_bf16, long long ldx, int M, int K, const float *gamma, const float *beta, float eps,
                    void *Y_bf16, void *cuda_stream);

/*
 * Test hook for the bounded device-side waits (the paper has no counterpart).  Launches the GEMM of
 * qvggt_w4a4_linear_c8 with its TMA producers switched off and every wait limited to wait_limit_cycles
 * (1000 .. 2e9) SM cycles: no operand ever arrives, the first wait runs out, the kernel records the code of that
 * wait in the handle's status word, releases its tensor memory and returns -- nothing faults, traps or spins
 * without bound, and no asynchronous operation is in flight when it leaves.  Y_bf16 is not written.  Afterwards
 * qvggt_device_status() on this handle reports QVGGT_ERR_DEVICE_TIMEOUT (the status word is sticky: use a fresh
 * handle for real work).  Arguments as for qvggt_w4a4_linear_c8 (M >= 1).
 */
int qvggt_debug_starved_linear_c8(const qvggt_weights_t *w, const signed char *Xq8, const float *a_scale, int M,
                                  void *Y_bf16, long long ldy, long long wait_limit_cycles, void *cuda_stream);

/*
 * The other half of the upstream fusion: fc2's input is the MLP's activation function applied to fc1's output.  The
 * paper does not name the function; the transformer blocks VGGT is built from use the exact GELU x Phi(x) (Phi the
 * standard normal distribution function), which is what is computed here, in fp32, to within one bf16 ulp of the
 * exactly rounded value (results of magnitude below 2^-120, i.e. x < -12.9, may be flushed to zero).
 * qvggt_gelu_rotate_smooth_quantize_c8 applies it to every element on its way into the activation path of
 * qvggt_rotate_smooth_quantize_c8 -- the activated tensor (the largest activation of the block) never goes to memory --
 * and returns, bit for bit, the result of qvggt_gelu followed by qvggt_rotate_smooth_quantize_c8.
 * Arguments as for qvggt_rotate_smooth_quantize_c8 / qvggt_layernorm (Y_bf16 [M, K] contiguous; K = 1024 or 4096).
 */
int qvggt_gelu_rotate_smooth_quantize_c8(const qvggt_weights_t *w, const void *X_bf16, long long ldx, int M,
                                         signed char *Xq8, float *a_scale, void *cuda_stream);
int qvggt_gelu(const void *X_bf16, long long ldx, int M, int K, void *Y_bf16, void *cuda_stream);

/* Frees the handle and its device memory (synchronises the device first).  NULL is allowed. */
void qvggt_free_weights(qvggt_weights_t *w);

/*
 * Device pointers into the handle, for inspection (any output pointer may be NULL to skip it):
 * Wq [N, K/2] packed int4, w_scale fp32 [N], amul fp32 [K], bias bf16 [N] (NULL if none).
 * The memory stays owned by the handle.
 */
int qvggt_weights_view(const qvggt_weights_t *w, const unsigned char **Wq, const float **w_scale,
                       const float **amul, const void **bias_bf16, int *N, int *K);

/* Device pointer to the int8 [N, K] copy of the codes (NULL if the handle was prepared without QVGGT_PREP_C8 or
 * QVGGT_PREP_W8A8) and, if `bits` is not NULL, the handle's code width (4 or 8). */
int qvggt_weights_view_c8(const qvggt_weights_t *w, const signed char **Wq8, int *bits);

/*
 * Synchronises `cuda_stream`, then reads the handle's device status word into *code (HOST pointer):
 * 0 = no device-side wait has expired since the handle was created; otherwise a positive code
 * naming the wait that gave up.  Returns QVGGT_ERR_DEVICE_TIMEOUT if *code != 0.
 */
int qvggt_device_status(const qvggt_weights_t *w, void *cuda_stream, int *code);

/*
 * Calibration helper (Eq. "smooth_factor"): c[k] = clip( ax[k]^alpha / aw[k]^(1-alpha), lo, hi ) with
 * ax[k] = max_m |(X_calib H)[m][k]|, aw[k] = max_n |(W H)[n][k]| in the rotated space (fp32
 * butterflies; 0/0 -> 1).
 *   X_calib_bf16 [Mc, K] bf16, contiguous;  W_bf16 [N, K] bf16, contiguous;  smooth_c fp32 [K] output
 *   colmax_scratch  fp32 [2*K] device scratch supplied by the caller (overwritten)
 */
int qvggt_calibrate_smooth(const void *X_calib_bf16, int Mc, const void *W_bf16, int N, int K, float alpha,
                           float lo, float hi, float *colmax_scratch, float *smooth_c, void *cuda_stream);

/*
 * Allocation-free variant of the weight quantization in qvggt_prepare_weights.  (The paper has no
 * counterpart; this exists for deployment.)  For callers that cannot allocate device memory at this point:
 * a process whose whole device memory already belongs to its own arena, or a section that cannot
 * take the device-wide synchronisation cudaMalloc/cudaFree may imply.  It calls no cudaMalloc,
 * cudaFree or any other allocating routine.  Same arithmetic and results as qvggt_prepare_weights:
 *   Wq      [N, K/2] packed int4 (output, caller-allocated, 16-byte aligned)
 *   w_scale fp32 [N] (output)        amul  fp32 [K] (output, for the activation path)
 *   W_bf16 [N, K] bf16 16-byte aligned; smooth_c fp32 [K]; sign_v int8 [K] or NULL; any N >= 1.
 * The temporary weight-side multipliers live in a fixed 16 KB device array inside the library
 * (held by every GPU that loads it, until the process exits), which limits K to at most 4096:
 * a larger K is refused with QVGGT_ERR_SHAPE.  The array is shared by all calls and keeps the
 * previous call's contents; each call rewrites the part it reads, but two calls whose kernels
 * overlap on the GPU (different streams) race on it -- serialise them.  The first call on each
 * device looks up the array's device address (with that device current); make that first call
 * before any stream capture begins.
 */
int qvggt_quantize_weights_static(const void *W_bf16, const float *smooth_c, const signed char *sign_v, int N,
                                  int K, unsigned char *Wq, float *w_scale, float *amul, void *cuda_stream);

/* Static, NUL-terminated description of a status code. */
const char *qvggt_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* QVGGT_H */
