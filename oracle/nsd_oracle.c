/*
 * CPU oracle for non-subtractive dithered (NSD) quantization -- TEST INFRASTRUCTURE.
 *
 * This file is the slow, plain reference that the CUDA kernels are checked against.
 * It shares no code with the CUDA path and must never be linked into the product.
 *
 * What it follows (dithered backprop paper):
 *   - Section 3.1, Eq. (nsd):  x~ = Delta * floor((x + nu)/Delta + 1/2),
 *     nu uniform on the open interval (-Delta/2, Delta/2).
 *   - Algorithm 1:  sigma = std(delta_z);  Delta = s * sigma;  quantize.
 *
 * Readings fixed where the paper is silent:
 *   - std is the population standard deviation about the mean (divide by N).
 *   - floor((x+nu)/Delta + 1/2) == floor(x/Delta + u) with u = nu/Delta + 1/2 in (0,1).
 *     u is taken from a counter-based generator so that any implementation can
 *     reproduce the draw of element i without state: the SplitMix64 stream
 *     (Steele, Lea, Flood 2014) started at `seed`; its c-th output serves elements
 *     2c (low 32 bits) and 2c+1 (high 32 bits). The top 23 bits k of those 32 give
 *     u = (2k+1) * 2^-24: strictly inside (0,1), symmetric about 1/2, exact in fp32.
 *   - The decision floor(.) is taken in fp32: t = fma(x, 1/Delta, u) with a single
 *     rounding, 1/Delta by IEEE single division. Codes saturate to [-127, 127].
 *   - Delta <= 0 (sigma = 0) or non-finite Delta: every code is 0.
 */
#include <math.h>
#include <stdint.h>
#include <stddef.h>

uint64_t oracle_splitmix64_at(uint64_t seed, uint64_t c)
{
    /* output number c (0-based) of the SplitMix64 sequence whose state starts at seed */
    uint64_t z = seed + (c + 1u) * 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

float oracle_dither_u(uint64_t seed, uint64_t i)
{
    uint64_t r = oracle_splitmix64_at(seed, i >> 1);
    uint32_t h = (i & 1u) ? (uint32_t)(r >> 32) : (uint32_t)r;
    uint32_t k = h >> 9;                       /* 23 bits */
    return (float)(2u * k + 1u) * 0x1p-24f;    /* exact: odd integer < 2^24 */
}

/* Algorithm 1, line "sigma <- std(delta_z)": two-pass population std in fp64. */
void oracle_mean_std(const float *x, int64_t n, double *mean, double *std)
{
    double s = 0.0;
    for (int64_t i = 0; i < n; ++i) s += (double)x[i];
    double mu = (n > 0) ? s / (double)n : 0.0;
    double v = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        double d = (double)x[i] - mu;
        v += d * d;
    }
    *mean = mu;
    *std = (n > 0) ? sqrt(v / (double)n) : 0.0;
}

/* Eq. (nsd) for every element, integer code q_i (x~_i = q_i * Delta).
 * index_base is the flat index of x[0] inside the tensor the dither is keyed on.
 * Returns the number of non-zero codes; *nsat counts codes clipped to +-127. */
int64_t oracle_nsd_codes(const float *x, int64_t n, uint64_t seed, float Delta,
                         uint64_t index_base, int8_t *codes, int64_t *nsat)
{
    int64_t nnz = 0, sat = 0;
    if (!(Delta > 0.0f) || isinf(Delta)) {
        for (int64_t i = 0; i < n; ++i) codes[i] = 0;
        if (nsat) *nsat = 0;
        return 0;
    }
    const float inv = 1.0f / Delta;            /* IEEE single division */
    for (int64_t i = 0; i < n; ++i) {
        float u = oracle_dither_u(seed, index_base + (uint64_t)i);
        float t = fmaf(x[i], inv, u);          /* one rounding */
        float f = floorf(t);
        int q;
        if (isnan(t)) q = 0;                   /* Eq. (nsd) is undefined for NaN: no code */
        else if (f > 127.0f) { q = 127; ++sat; }
        else if (f < -127.0f) { q = -127; ++sat; }
        else q = (int)f;
        codes[i] = (int8_t)q;
        nnz += (q != 0);
    }
    if (nsat) *nsat = sat;
    return nnz;
}

/* Eq. (nsd) evaluated literally in fp64, nu = (u - 1/2) * Delta; used only to show that
 * the fp32 decision above is the same quantizer up to ties at the rounding boundary. */
int64_t oracle_nsd_codes_literal_f64(const float *x, int64_t n, uint64_t seed, float Delta,
                                     uint64_t index_base, int32_t *codes)
{
    int64_t nnz = 0;
    double D = (double)Delta;
    for (int64_t i = 0; i < n; ++i) {
        double u = (double)oracle_dither_u(seed, index_base + (uint64_t)i);
        double nu = (u - 0.5) * D;
        double q = floor(((double)x[i] + nu) / D + 0.5);
        codes[i] = (int32_t)q;
        nnz += (q != 0.0);
    }
    return nnz;
}
