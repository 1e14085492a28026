/*
 * Seeded synthetic workload generator for the W4A4 linear path.
 *
 * This file only draws random inputs (activations, weights, biases).  It holds none of the
 * quantization method's arithmetic: no Hadamard transform, no smoothing, no quantizer, no GEMM.
 * Both the CPU oracle's tests and the CUDA path's tests/bench consume the bytes produced here.
 *
 * Every value is a pure function of (seed, stream, row, column), so any row of any layer can be
 * regenerated alone (needed to spot-check full-size runs on sampled rows).
 *
 * The synthetic activations stand in for the VGGT token activations the paper describes: a few
 * outlier channels, and five data-independent special tokens (camera + 4 register) at the start of
 * every frame whose rows are far larger than the patch-token rows (Sec. 3.2, Observation 1).
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

static inline uint64_t wl_mix(uint64_t z)
{
    z += 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

/* Counter-based draw: one 64-bit word per (seed, stream, row, col, draw index). */
static inline uint64_t wl_bits(uint64_t seed, uint64_t stream, uint64_t row, uint64_t col, uint64_t draw)
{
    uint64_t h = wl_mix(seed ^ 0x51ED270B7A3C1D45ull);
    h = wl_mix(h ^ (stream * 0xD6E8FEB86659FD93ull));
    h = wl_mix(h ^ (row * 0xA0761D6478BD642Full));
    h = wl_mix(h ^ (col * 0xE7037ED1A0B428DBull));
    return wl_mix(h ^ draw);
}

static inline double wl_u01(uint64_t bits)
{
    /* uniform on the open interval (0, 1) */
    return ((double)(bits >> 11) + 0.5) * (1.0 / 9007199254740992.0);
}

/* Two independent standard normals (Box-Muller, fp64). */
static inline void wl_normal2(uint64_t seed, uint64_t stream, uint64_t row, uint64_t col, uint64_t draw,
                              double *z0, double *z1)
{
    double u1 = wl_u01(wl_bits(seed, stream, row, col, 2 * draw));
    double u2 = wl_u01(wl_bits(seed, stream, row, col, 2 * draw + 1));
    double r = sqrt(-2.0 * log(u1));
    double t = 6.283185307179586476925286766559 * u2;
    *z0 = r * cos(t);
    *z1 = r * sin(t);
}

/* fp32 -> bf16 bits, round to nearest even (inputs here are always finite). */
static inline uint16_t wl_bf16(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    u += 0x7FFFu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

enum { WL_DIST_NORMAL = 0, WL_DIST_GELU = 1, WL_DIST_STUDENT_T3 = 2 };

/*
 * Activation rows [row0, row0+nrows) of a virtual [*, K] matrix, written as bf16 bits.
 *   dist            WL_DIST_NORMAL      N(0,1)
 *                   WL_DIST_GELU        GELU(1.5 * N(0,1))  (non-negative-skewed, like an MLP hidden state)
 *                   WL_DIST_STUDENT_T3  Z / sqrt(chi2_3 / 3)
 *   ch_gain[K]      per-channel multiplier (outlier channels carry e.g. 50, the rest 1), or NULL
 *   frame_rows      rows per frame (1374), 0 = no special-token structure
 *   special_rows    the first `special_rows` rows of each frame are multiplied by special_gain
 *   out, ld         output, row stride in elements
 */
void wl_activations_bf16(uint64_t seed, uint64_t stream, int64_t row0, int64_t nrows, int K, int dist,
                         const float *ch_gain, int frame_rows, int special_rows, double special_gain,
                         uint16_t *out, int64_t ld)
{
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < nrows; ++r) {
        uint64_t row = (uint64_t)(row0 + r);
        double rg = 1.0;
        if (frame_rows > 0 && (int64_t)(row % (uint64_t)frame_rows) < special_rows) rg = special_gain;
        uint16_t *o = out + r * ld;
        for (int c = 0; c < K; c += 2) {
            double a, b;
            if (dist == WL_DIST_STUDENT_T3) {
                double z0, z1, z2, z3, z4, z5, z6, z7;
                wl_normal2(seed, stream, row, (uint64_t)c, 0, &z0, &z1);
                wl_normal2(seed, stream, row, (uint64_t)c, 1, &z2, &z3);
                wl_normal2(seed, stream, row, (uint64_t)c, 2, &z4, &z5);
                wl_normal2(seed, stream, row, (uint64_t)c, 3, &z6, &z7);
                a = z0 / sqrt((z1 * z1 + z2 * z2 + z3 * z3) / 3.0);
                b = z4 / sqrt((z5 * z5 + z6 * z6 + z7 * z7) / 3.0);
            } else {
                wl_normal2(seed, stream, row, (uint64_t)c, 0, &a, &b);
                if (dist == WL_DIST_GELU) {
                    a *= 1.5;
                    b *= 1.5;
                    a = 0.5 * a * (1.0 + erf(a * 0.70710678118654752440));
                    b = 0.5 * b * (1.0 + erf(b * 0.70710678118654752440));
                }
            }
            double ga = rg, gb = rg;
            if (ch_gain) {
                ga *= (double)ch_gain[c];
                gb *= (double)ch_gain[c + 1];
            }
            o[c] = wl_bf16((float)(a * ga));
            if (c + 1 < K) o[c + 1] = wl_bf16((float)(b * gb));
        }
    }
}

/* Plain N(mean, std) matrix rows as bf16 bits (weights, biases). */
void wl_normal_bf16(uint64_t seed, uint64_t stream, int64_t row0, int64_t nrows, int ncols, double mean,
                    double std, uint16_t *out, int64_t ld)
{
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < nrows; ++r) {
        uint64_t row = (uint64_t)(row0 + r);
        uint16_t *o = out + r * ld;
        for (int c = 0; c < ncols; c += 2) {
            double a, b;
            wl_normal2(seed, stream, row, (uint64_t)c, 0, &a, &b);
            o[c] = wl_bf16((float)(mean + std * a));
            if (c + 1 < ncols) o[c + 1] = wl_bf16((float)(mean + std * b));
        }
    }
}

/* Log-uniform positive fp32 vector on [lo, hi] (stand-in for a learned per-channel factor). */
void wl_loguniform_f32(uint64_t seed, uint64_t stream, int n, double lo, double hi, float *out)
{
    double llo = log(lo), lhi = log(hi);
    for (int i = 0; i < n; ++i) {
        double u = wl_u01(wl_bits(seed, stream, 0, (uint64_t)i, 0));
        out[i] = (float)exp(llo + (lhi - llo) * u);
    }
}

/* Random +-1 vector. */
void wl_signs_i8(uint64_t seed, uint64_t stream, int n, int8_t *out)
{
    for (int i = 0; i < n; ++i) out[i] = (wl_bits(seed, stream, 0, (uint64_t)i, 0) & 1u) ? 1 : -1;
}
