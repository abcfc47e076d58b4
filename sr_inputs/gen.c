/*
 * Seeded synthetic inputs for the dictionary-regression path.
 *
 * This file holds no arithmetic of the method itself: it only fills host arrays
 * (LR image, dictionary atoms, coefficient planes) that the CPU oracle and the
 * CUDA library both consume bit for bit.
 *
 * Random numbers are counter based: value(seed, tensor, index) is a pure
 * function, so any element can be produced alone and in parallel.
 *
 *   mix(seed, tensor, index): 64-bit finaliser (two multiply/xor-shift rounds)
 *   uniform  = top 53 bits of mix * 2^-53                         in [0,1)
 *   normal   = Box-Muller in fp64 on the pair (2p, 2p+1), p = index/2;
 *              even index takes the cosine branch, odd the sine branch
 *
 * Tensor ids: 1 = LR image, 2 = dictionary parameters, 3 + frame = coefficients.
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define SRG_TENSOR_LR 1u
#define SRG_TENSOR_DICT 2u
#define SRG_TENSOR_COEF 3u

static inline uint64_t srg_mix(uint64_t seed, uint64_t tensor, uint64_t index)
{
    uint64_t z = seed + 0x9E3779B97F4A7C15ull * (index + 1ull) + 0xD1B54A32D192ED03ull * tensor;
    z ^= z >> 30;
    z *= 0xBF58476D1CE4E5B9ull;
    z ^= z >> 27;
    z *= 0x94D049BB133111EBull;
    z ^= z >> 31;
    return z;
}

static inline double srg_uniform(uint64_t seed, uint64_t tensor, uint64_t index)
{
    return (double)(srg_mix(seed, tensor, index) >> 11) * (1.0 / 9007199254740992.0);
}

static inline double srg_normal(uint64_t seed, uint64_t tensor, uint64_t index)
{
    const uint64_t p = index >> 1;
    const double u1 = 1.0 - srg_uniform(seed, tensor, 2 * p);      /* (0,1] */
    const double u2 = srg_uniform(seed, tensor, 2 * p + 1);
    const double rad = sqrt(-2.0 * log(u1));
    const double ang = 6.283185307179586476925286766559 * u2;
    return (index & 1) ? rad * sin(ang) : rad * cos(ang);
}

/* fp32 -> IEEE binary16 bits, round to nearest even, overflow to infinity. */
static inline uint16_t srg_f32_to_f16(float f)
{
    uint32_t x;
    memcpy(&x, &f, 4);
    const uint32_t sign = (x >> 16) & 0x8000u;
    const uint32_t ax = x & 0x7FFFFFFFu;
    if (ax >= 0x7F800000u) /* inf / nan */
        return (uint16_t)(sign | 0x7C00u | ((ax > 0x7F800000u) ? 0x200u : 0u));
    if (ax >= 0x477FF000u) /* rounds to >= 65520 -> inf */
        return (uint16_t)(sign | 0x7C00u);
    if (ax < 0x33000001u) /* below half the smallest subnormal (or exactly half: ties to even = 0) */
        return (uint16_t)sign;
    int32_t e = (int32_t)(ax >> 23) - 127;
    uint32_t m = (ax & 0x7FFFFFu) | 0x800000u; /* 24-bit significand */
    int shift;
    uint32_t base;
    if (e >= -14) { /* normal half */
        shift = 13;
        base = (uint32_t)(e + 15) << 10;
        m &= 0x7FFFFFu;
    } else { /* subnormal half: value = m * 2^(e-23); unit = 2^-24 */
        shift = 13 + (-14 - e);
        base = 0;
    }
    uint32_t q = m >> shift;
    const uint32_t rem = m & ((1u << shift) - 1u);
    const uint32_t half = 1u << (shift - 1);
    if (rem > half || (rem == half && (q & 1u)))
        q++;
    return (uint16_t)(sign | (base + q)); /* a carry out of the mantissa bumps the exponent correctly */
}

/* LR image: count fp32 values, uniform in [0,1). */
void srg_fill_lr(uint64_t seed, float *dst, int64_t count)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < count; ++i)
        dst[i] = (float)srg_uniform(seed, SRG_TENSOR_LR, (uint64_t)i);
}

/*
 * Coefficients of one frame: count = D*H*W values, mean + sigma * N(0,1),
 * rounded to fp32 and then (as_f16 != 0) to binary16 with round-to-nearest-even.
 * dst is float* or uint16_t*.
 */
void srg_fill_coef(uint64_t seed, int32_t frame, void *dst, int64_t count, double mean, double sigma,
                   int32_t as_f16)
{
    const uint64_t tensor = SRG_TENSOR_COEF + (uint64_t)frame;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < count; ++i) {
        const float v = (float)(mean + sigma * srg_normal(seed, tensor, (uint64_t)i));
        if (as_f16)
            ((uint16_t *)dst)[i] = srg_f32_to_f16(v);
        else
            ((float *)dst)[i] = v;
    }
}

/* Convert count fp32 values to binary16 bit patterns (RNE). */
void srg_round_f16(const float *src, uint16_t *dst, int64_t count)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < count; ++i)
        dst[i] = srg_f32_to_f16(src[i]);
}

/* un-normalised anisotropic Gaussian, peak 1 at the centre tap */
static double srg_gauss(double u, double v, double sx, double sy, double th)
{
    const double c = cos(th), s = sin(th);
    const double ur = c * u + s * v;
    const double vr = -s * u + c * v;
    return exp(-0.5 * (ur * ur / (sx * sx) + vr * vr / (sy * sy)));
}

/*
 * Dictionary of D atoms of k x k taps (row-major, tap j = a*k + b), fp32.
 * Atoms 0 .. D/2-1 (rounded up) are anisotropic rotated Gaussians, the rest are
 * differences of Gaussians (wide minus narrow, widths in ratio 1.6, same
 * rotation); every atom is divided by the sum of its own taps.
 * Per atom three uniforms: sigma_x, sigma_y in [0.3, 2.0], theta in [0, pi).
 */
void srg_make_dictionary(uint64_t seed, float *dict, int32_t D, int32_t k)
{
    const int p = (k - 1) / 2;
    const int n_gauss = (D + 1) / 2;
    for (int l = 0; l < D; ++l) {
        const double sx = 0.3 + 1.7 * srg_uniform(seed, SRG_TENSOR_DICT, 3ull * l + 0);
        const double sy = 0.3 + 1.7 * srg_uniform(seed, SRG_TENSOR_DICT, 3ull * l + 1);
        const double th = 3.14159265358979323846 * srg_uniform(seed, SRG_TENSOR_DICT, 3ull * l + 2);
        double taps[81];
        double sum = 0.0;
        for (int a = 0; a < k; ++a)
            for (int b = 0; b < k; ++b) {
                const double v = (double)(a - p), u = (double)(b - p);
                double e = srg_gauss(u, v, sx, sy, th);
                if (l >= n_gauss)
                    e = srg_gauss(u, v, 1.6 * sx, 1.6 * sy, th) - e;
                taps[a * k + b] = e;
                sum += e;
            }
        for (int j = 0; j < k * k; ++j)
            dict[(int64_t)l * k * k + j] = (float)(taps[j] / sum);
    }
}

int32_t srg_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
