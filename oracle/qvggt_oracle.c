/*
 * CPU ORACLE -- TEST INFRASTRUCTURE ONLY.
 *
 * Plain, slow, scalar restatement of the W4A4 linear layer of Dual-Smoothed Fine-Grained
 * Quantization (Sec. 3.2 of the QuantVGGT paper), written step by step from the paper's
 * formulas.  It shares no code with the CUDA path and must never be called from it; only the
 * tests, the smoke check and the CPU-baseline leg of the benchmark use it.
 *
 * Build: gcc -O2 -ffp-contract=off -fopenmp (no fast-math; OpenMP only across independent rows).
 * "fl(.)" below is one IEEE-754 binary32 round-to-nearest-even operation; no FMA is ever formed.
 *
 * Pins (see tests/test_oracle_pins.py): Sylvester closed form (-1)^popcount(i&j), H H^T = K I,
 * brute-force dense +-1 products on integer inputs, fp64 rotation/smoothing invariance,
 * |y - scale*q| <= scale/2, hand-built rounding ties, brute-force integer GEMMs, fp64 epilogue.
 * Unpinned by the paper (this build's conventions): the fp32 butterfly stage order, the
 * group-wise (per 128 channels) variant for G < K, the summation tree of the LayerNorm statistics, and the
 * end-to-end layer error vs. the unquantized layer ("parity unpinned": information only).
 * Further pins: the wide-rotation quantizer (rotation in fp64) coincides with the fp32 one wherever fp32 is exact
 * and stays inside the rounding bound elsewhere; GELU against tabulated values of the normal distribution, the
 * identity gelu(x) - gelu(-x) = x and a library normal CDF.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static inline float orc_bf16_to_f32(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* binary32 -> bf16 bits, round to nearest even; NaN stays NaN. */
static inline uint16_t orc_f32_to_bf16(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)((u >> 16) | 0x0040u);
    u += 0x7FFFu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

/*
 * Un-normalized Sylvester-Hadamard transform of one row, in place (pre-global rotation; the
 * Kronecker recursion H_{2^n} = H_2 (x) H_{2^{n-1}} of Sec. 3.2 unrolled into radix-2 stages).
 * Stage order is ascending stride h = 1, 2, 4, ..., K/2; each butterfly is
 * (a, b) -> (fl(a+b), fl(a-b)).  The result equals u * H_K with H_K[i][j] = (-1)^popcount(i&j),
 * H_K H_K^T = K I.
 */
void orc_fwht_f32(float *u, int K)
{
    for (int h = 1; h < K; h <<= 1)
        for (int i = 0; i < K; ++i)
            if (!(i & h)) {
                float a = u[i], b = u[i + h];
                u[i] = a + b;
                u[i + h] = a - b;
            }
}

void orc_fwht_f64(double *u, int K)
{
    for (int h = 1; h < K; h <<= 1)
        for (int i = 0; i < K; ++i)
            if (!(i & h)) {
                double a = u[i], b = u[i + h];
                u[i] = a + b;
                u[i + h] = a - b;
            }
}

/*
 * LayerNorm in front of the rotation (Sec. 3.2 places the quantized linear behind a normalization layer; the
 * upstream-fusion row fuses the two).  The paper does not say how the statistics are summed, so this build fixes it:
 * plain pairwise summation (the sum of n terms is fl(sum of the first half + sum of the second half), recursively),
 * everything in fp32, one rounding per operation:
 *   mean = pairwise(x) / K;  d_k = fl(x_k - mean);  var = pairwise(fl(d_k * d_k)) / K      (K a power of two: exact divisions)
 *   rstd = fl(1 / fl(sqrt(fl(var + eps))))
 *   out_k = bf16( fl( fl(fl(d_k * rstd) * gamma_k) + beta_k ) )                               (round to nearest even)
 *   X bf16 bits [M, K] (row stride ldx), gamma / beta fp32 [K], out bf16 bits [M, K] contiguous
 */
static float orc_pairwise(const float *a, int n)
{
    if (n == 1) return a[0];
    float lo = orc_pairwise(a, n / 2), hi = orc_pairwise(a + n / 2, n / 2);
    return lo + hi;
}

void orc_layernorm(const uint16_t *X, int64_t ldx, int64_t M, int K, const float *gamma, const float *beta, float eps,
                   uint16_t *out)
{
    const float invK = 1.0f / (float)K;
#pragma omp parallel
    {
        float *x = (float *)malloc(sizeof(float) * (size_t)K);
        float *d = (float *)malloc(sizeof(float) * (size_t)K);
#pragma omp for schedule(static)
        for (int64_t m = 0; m < M; ++m) {
            for (int k = 0; k < K; ++k) x[k] = orc_bf16_to_f32(X[m * ldx + k]);
            float mean = orc_pairwise(x, K) * invK;
            for (int k = 0; k < K; ++k) {
                d[k] = x[k] - mean;
                x[k] = d[k] * d[k];
            }
            float var = orc_pairwise(x, K) * invK;
            float t = var + eps;
            t = sqrtf(t);
            float rstd = 1.0f / t;
            for (int k = 0; k < K; ++k) {
                float n = d[k] * rstd;
                n = n * gamma[k];
                n = n + beta[k];
                out[m * K + k] = orc_f32_to_bf16(n);
            }
        }
        free(x);
        free(d);
    }
}

/* K^{-1/2}: an exact power of two when log2 K is even (K = 1024, 4096). */
static float orc_norm(int K)
{
    return (float)(1.0 / sqrt((double)K));
}

/*
 * Per-rotated-channel multipliers.  With the random Hadamard H = K^{-1/2} H_K diag(v) and the
 * smoothing identity  X W^T = (X H diag(c)^-1)(diag(c) H^T W^T)  (Eq. "smooth_factor"):
 *   amul[k] = fl( (v_k K^{-1/2}) / c_k )   applied to rotated activations,
 *   wmul[k] = fl( (v_k K^{-1/2}) * c_k )   applied to rotated weight rows.
 * v may be NULL (all +1).
 */
void orc_multipliers(const float *c, const int8_t *v, int K, float *amul, float *wmul)
{
    float nrm = orc_norm(K);
    for (int k = 0; k < K; ++k) {
        float s = (v && v[k] < 0) ? -nrm : nrm;
        amul[k] = s / c[k];
        wmul[k] = s * c[k];
    }
}

/*
 * Rotate -> smooth -> symmetric N-bit quantize, row by row (Eq. "quantization":
 * Delta = max|y| / (2^(N-1) - 1), q = clamp(round(y / Delta), -2^(N-1), 2^(N-1) - 1)); N = 4 is the
 * W4A4 setting, N = 8 the paper's W8A8 setting.
 *   X      bf16 bits [M, K], row stride ldx elements
 *   mul    fp32 [K] (amul for activations, wmul for weight rows)
 *   group  scale granularity along K: 0 = one scale per row (the paper's token-wise /
 *          out-channel-wise setting); g > 0 = one scale per g consecutive rotated channels
 *   bits   N (2..8)
 *   codes  int8 [M, K], values in [-2^(N-1), 2^(N-1) - 1] (in fact never the most negative code)
 *   scales fp32 [M, K/group]
 * Reading of the unspecified points: round() is round-half-to-even; y/Delta is evaluated as the
 * exact product y * fl(qmax/amax) rounded once to an integer; an all-zero group gets amax = 1e-8.
 */
void orc_rotate_smooth_quantize_bits(const uint16_t *X, int64_t ldx, int64_t M, int K, const float *mul,
                                     int group, int bits, int8_t *codes, float *scales)
{
    int G = group > 0 ? K / group : 1;
    int glen = group > 0 ? group : K;
    const float qmax = (float)((1 << (bits - 1)) - 1);
    const double lo = -(double)(1 << (bits - 1)), hi = (double)qmax;
#pragma omp parallel
    {
        float *u = (float *)malloc(sizeof(float) * (size_t)K);
#pragma omp for schedule(static)
        for (int64_t m = 0; m < M; ++m) {
            const uint16_t *x = X + m * ldx;
            for (int k = 0; k < K; ++k) u[k] = orc_bf16_to_f32(x[k]);
            orc_fwht_f32(u, K);
            for (int k = 0; k < K; ++k) u[k] = u[k] * mul[k];
            for (int g = 0; g < G; ++g) {
                const float *y = u + g * glen;
                float amax = 0.0f;
                for (int k = 0; k < glen; ++k) {
                    float a = fabsf(y[k]);
                    if (a > amax) amax = a;
                }
                if (amax < 1e-8f) amax = 1e-8f;
                float scale = amax / qmax;
                float inv = qmax / amax;
                scales[m * G + g] = scale;
                int8_t *q = codes + m * K + g * glen;
                for (int k = 0; k < glen; ++k) {
                    double r = nearbyint((double)y[k] * (double)inv); /* exact product, one rounding */
                    if (r < lo) r = lo;
                    if (r > hi) r = hi;
                    q[k] = (int8_t)r;
                }
            }
        }
        free(u);
    }
}

/*
 * Static tensor-wise activation quantizer (the other arm of the paper's granularity ablation, Tab. "granularity":
 * one step size Delta for the whole tensor, fixed offline, instead of one per token computed from the data).
 * Eq. "quantization" with a given Delta: q = clamp(round(y / Delta), -2^(N-1), 2^(N-1) - 1), where the clamp now
 * matters.  Same readings as above: round-half-to-even; y / Delta is the exact product y * fl(1 / Delta) rounded once.
 *   delta  the step size (> 0);  codes int8 [M, K]
 */
void orc_rotate_smooth_quantize_static(const uint16_t *X, int64_t ldx, int64_t M, int K, const float *mul, float delta,
                                       int bits, int8_t *codes)
{
    const double lo = -(double)(1 << (bits - 1)), hi = (double)((1 << (bits - 1)) - 1);
    const float inv = 1.0f / delta;
#pragma omp parallel
    {
        float *u = (float *)malloc(sizeof(float) * (size_t)K);
#pragma omp for schedule(static)
        for (int64_t m = 0; m < M; ++m) {
            const uint16_t *x = X + m * ldx;
            for (int k = 0; k < K; ++k) u[k] = orc_bf16_to_f32(x[k]);
            orc_fwht_f32(u, K);
            for (int k = 0; k < K; ++k) {
                float y = u[k] * mul[k];
                double r = nearbyint((double)y * (double)inv); /* exact product, one rounding */
                if (r < lo) r = lo;
                if (r > hi) r = hi;
                codes[m * K + k] = (int8_t)r;
            }
        }
        free(u);
    }
}

/*
 * The same quantizer behind a rotation WITHOUT intermediate rounding: u = x H_K evaluated in fp64 (for bf16 inputs
 * every partial sum of the transform is exact in fp64 unless the row spans more than ~40 binades) and rounded to
 * fp32 once; the multiplier, the absolute maximum and Eq. "quantization" follow unchanged.  This is the reference of
 * the tolerance contract for rotations that do not reproduce the fp32 butterfly order (a tensor-core Hadamard):
 * such a rotation cannot match orc_rotate_smooth_quantize_bits bit for bit, because that one rounds after each of
 * its log2 K stages in one particular order; it is measured by its distance from the exact rotation instead.
 *   y_out   fp32 [M, K] or NULL: the rotated, smoothed row fl(fl32(u) * mul) the codes were taken from
 *   abs_sum fp64 [M] or NULL: sum_k |x_k|, the quantity the rounding bound of any fp32 rotation scales with
 * Per-row scales only (group = 0).
 */
void orc_rotate_smooth_quantize_wide(const uint16_t *X, int64_t ldx, int64_t M, int K, const float *mul, int bits,
                                     int8_t *codes, float *scales, float *y_out, double *abs_sum)
{
    const float qmax = (float)((1 << (bits - 1)) - 1);
    const double lo = -(double)(1 << (bits - 1)), hi = (double)qmax;
#pragma omp parallel
    {
        double *u = (double *)malloc(sizeof(double) * (size_t)K);
        float *y = (float *)malloc(sizeof(float) * (size_t)K);
#pragma omp for schedule(static)
        for (int64_t m = 0; m < M; ++m) {
            const uint16_t *x = X + m * ldx;
            double s = 0.0;
            for (int k = 0; k < K; ++k) {
                u[k] = (double)orc_bf16_to_f32(x[k]);
                s += fabs(u[k]);
            }
            if (abs_sum) abs_sum[m] = s;
            orc_fwht_f64(u, K);
            float amax = 0.0f;
            for (int k = 0; k < K; ++k) {
                float r = (float)u[k];          /* the one rounding of the rotation */
                y[k] = r * mul[k];
                float a = fabsf(y[k]);
                if (a > amax) amax = a;
            }
            if (amax < 1e-8f) amax = 1e-8f;
            scales[m] = amax / qmax;
            float inv = qmax / amax;
            for (int k = 0; k < K; ++k) {
                double r = nearbyint((double)y[k] * (double)inv);
                if (r < lo) r = lo;
                if (r > hi) r = hi;
                codes[m * K + k] = (int8_t)r;
                if (y_out) y_out[m * K + k] = y[k];
            }
        }
        free(u);
        free(y);
    }
}

/*
 * GELU, the activation between the two linears of the transformer MLP (the producer of fc2's input; the paper
 * does not name it, the ViT blocks VGGT is built from use the exact form):
 *   gelu(x) = x * Phi(x),  Phi(x) = erfc(-x / sqrt(2)) / 2  the standard normal distribution function.
 * Written with erfc so that the negative tail keeps its relative accuracy (1 + erf cancels there).
 */
double orc_gelu_f64(double x)
{
    return x * 0.5 * erfc(-x * 0.70710678118654752440);
}

/* fp64 -> bf16 bits, round to nearest, ties to even, straight from the fp64 value (no fp32 step in between). */
static uint16_t orc_f64_to_bf16(double v)
{
    uint16_t c = orc_f32_to_bf16((float)v);
    /* the fp32 step may have rounded across a bf16 midpoint: look at the neighbours and keep the nearest */
    uint16_t best = c;
    double bd = fabs((double)orc_bf16_to_f32(c) - v);
    for (int d = -1; d <= 1; d += 2) {
        uint16_t n = (uint16_t)(c + d);
        if (((n ^ c) & 0x8000u) || (n & 0x7F80u) == 0x7F80u) continue;   /* stay on this side of zero, finite */
        double nd = fabs((double)orc_bf16_to_f32(n) - v);
        if (nd < bd || (nd == bd && !(n & 1u))) {
            best = n;
            bd = nd;
        }
    }
    return best;
}

/* X bf16 bits [M, K] (row stride ldx) -> out bf16 bits [M, K] contiguous: bf16(gelu(x)) evaluated in fp64. */
void orc_gelu(const uint16_t *X, int64_t ldx, int64_t M, int K, uint16_t *out)
{
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m)
        for (int k = 0; k < K; ++k)
            out[m * K + k] = orc_f64_to_bf16(orc_gelu_f64((double)orc_bf16_to_f32(X[m * ldx + k])));
}

/* The W4A4 setting (N = 4: Delta = max|y| / 7, codes in [-8, 7]). */
void orc_rotate_smooth_quantize(const uint16_t *X, int64_t ldx, int64_t M, int K, const float *mul,
                                int group, int8_t *codes, float *scales)
{
    orc_rotate_smooth_quantize_bits(X, ldx, M, K, mul, group, 4, codes, scales);
}

/* Canonical packed layout: byte i of a row = code 2i in bits 0-3, code 2i+1 in bits 4-7 (two's complement). */
void orc_pack_int4(const int8_t *codes, int64_t rows, int K, uint8_t *packed)
{
    for (int64_t r = 0; r < rows; ++r)
        for (int i = 0; i < K / 2; ++i) {
            uint8_t lo = (uint8_t)codes[r * K + 2 * i] & 0xF;
            uint8_t hi = (uint8_t)codes[r * K + 2 * i + 1] & 0xF;
            packed[r * (K / 2) + i] = (uint8_t)(lo | (hi << 4));
        }
}

void orc_unpack_int4(const uint8_t *packed, int64_t rows, int K, int8_t *codes)
{
    for (int64_t r = 0; r < rows; ++r)
        for (int i = 0; i < K / 2; ++i) {
            uint8_t b = packed[r * (K / 2) + i];
            int lo = b & 0xF, hi = b >> 4;
            codes[r * K + 2 * i] = (int8_t)(lo >= 8 ? lo - 16 : lo);
            codes[r * K + 2 * i + 1] = (int8_t)(hi >= 8 ? hi - 16 : hi);
        }
}

/*
 * Integer GEMM: only the inner dimension is summed, so the per-token and per-out-channel scales
 * stay outside the sum (Sec. 3.2, "Fine-Grained Quantization Granularity").
 *   acc[g][m][n] = sum_{k in group g} xq[m][k] * wq[n][k]   (int32, exact)
 * group = 0: one sum over all K (G = 1).
 */
void orc_gemm_i32(const int8_t *xq, const int8_t *wq, int64_t M, int N, int K, int group, int32_t *acc)
{
    int G = group > 0 ? K / group : 1;
    int glen = group > 0 ? group : K;
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m)
        for (int g = 0; g < G; ++g)
            for (int n = 0; n < N; ++n) {
                const int8_t *a = xq + m * K + g * glen;
                const int8_t *b = wq + (int64_t)n * K + g * glen;
                int32_t s = 0;
                for (int k = 0; k < glen; ++k) s += (int32_t)a[k] * (int32_t)b[k];
                acc[((int64_t)g * M + m) * N + n] = s;
            }
}

/*
 * Rescale + bias + bf16.
 *   G == 1:  t = fl(a_scale[m] * w_scale[n]);  z = fl(float(acc) * t);  z = fl(z + bias[n])
 *   G  > 1:  s = 0; for g ascending: s = fl(s + fl(float(acc_g) * a_scale[m][g]));
 *            z = fl(fl(s * w_scale[n]) + bias[n])
 * bias is bf16 bits or NULL (= 0).  Y is bf16 bits, row stride ldy.
 */
void orc_epilogue(const int32_t *acc, const float *a_scale, const float *w_scale, const uint16_t *bias,
                  int64_t M, int N, int G, uint16_t *Y, int64_t ldy)
{
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m)
        for (int n = 0; n < N; ++n) {
            float z;
            if (G == 1) {
                float t = a_scale[m] * w_scale[n];
                z = (float)acc[m * N + n] * t;
            } else {
                float s = 0.0f;
                for (int g = 0; g < G; ++g) {
                    float p = (float)acc[((int64_t)g * M + m) * N + n] * a_scale[m * G + g];
                    s = s + p;
                }
                z = s * w_scale[n];
            }
            if (bias) z = z + orc_bf16_to_f32(bias[n]);
            Y[m * ldy + n] = orc_f32_to_bf16(z);
        }
}

/*
 * Post-local smoothing factors (Eq. "smooth_factor", alpha = 0.5 in the paper):
 *   c_k = clip( max_m |(X H)_{m,k}|^alpha / max_n |(W H)_{n,k}|^(1-alpha), lo, hi ),
 * both maxima taken in the rotated space with the normalized Hadamard, in fp64 from the bf16
 * inputs; the signs v do not change absolute values.  0/0 -> 1.  Result rounded to fp32.
 */
void orc_smooth_factors(const uint16_t *Xcal, int64_t Mc, const uint16_t *W, int N, int K, double alpha,
                        double lo, double hi, float *c)
{
    double *ax = (double *)calloc((size_t)K, sizeof(double));
    double *aw = (double *)calloc((size_t)K, sizeof(double));
    double *u = (double *)malloc(sizeof(double) * (size_t)K);
    double nrm = 1.0 / sqrt((double)K);
    for (int64_t m = 0; m < Mc; ++m) {
        for (int k = 0; k < K; ++k) u[k] = (double)orc_bf16_to_f32(Xcal[m * K + k]);
        orc_fwht_f64(u, K);
        for (int k = 0; k < K; ++k) {
            double a = fabs(u[k]) * nrm;
            if (a > ax[k]) ax[k] = a;
        }
    }
    for (int n = 0; n < N; ++n) {
        for (int k = 0; k < K; ++k) u[k] = (double)orc_bf16_to_f32(W[(int64_t)n * K + k]);
        orc_fwht_f64(u, K);
        for (int k = 0; k < K; ++k) {
            double a = fabs(u[k]) * nrm;
            if (a > aw[k]) aw[k] = a;
        }
    }
    for (int k = 0; k < K; ++k) {
        double v;
        if (ax[k] == 0.0 && aw[k] == 0.0) v = 1.0;
        else v = pow(ax[k], alpha) / pow(aw[k], 1.0 - alpha);
        if (!(v >= lo)) v = lo;
        if (v > hi) v = hi;
        c[k] = (float)v;
    }
    free(ax);
    free(aw);
    free(u);
}

/* fp64 rotated-and-scaled rows: out[m][k] = (x_m H_K)[k] * mul[k]  (for the invariance pins). */
void orc_rotate_f64(const uint16_t *X, int64_t ldx, int64_t M, int K, const double *mul, double *out)
{
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        double *u = out + m * K;
        for (int k = 0; k < K; ++k) u[k] = (double)orc_bf16_to_f32(X[m * ldx + k]);
        orc_fwht_f64(u, K);
        for (int k = 0; k < K; ++k) u[k] *= mul[k];
    }
}

/* The unquantized layer Y = X W^T + b in fp64 from the bf16 inputs (information-only reference). */
void orc_linear_f64(const uint16_t *X, const uint16_t *W, const uint16_t *bias, int64_t M, int N, int K,
                    double *Y)
{
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m)
        for (int n = 0; n < N; ++n) {
            double s = 0.0;
            for (int k = 0; k < K; ++k)
                s += (double)orc_bf16_to_f32(X[m * K + k]) * (double)orc_bf16_to_f32(W[(int64_t)n * K + k]);
            if (bias) s += (double)orc_bf16_to_f32(bias[n]);
            Y[m * N + n] = s;
        }
}
