/*
 * CPU oracle (fp64) for the pixel-adaptive dictionary regression path.
 *
 * TEST INFRASTRUCTURE ONLY.  Only the tests, the smoke check and the benchmark's
 * cpu_baseline / reference legs may call this library; the CUDA library never does
 * and the two share no code.  Every function below is the plain definition,
 * pixel by pixel, with no tiling, separable passes, fusion or reordering, so it
 * can be compared with the paper by eye.  Inputs arrive with the same bit
 * patterns the GPU consumes (fp32 / binary16) and are widened exactly to fp64.
 *
 * Notation (paper, Section II-A): LR image x (h x w per channel), scale r,
 * HR size H = r*h, W = r*w; dictionary D in R^{L x k^2} ("dict", L is called D
 * in the argument lists); coefficients Phi in R^{HW r^2 x L}, stored planar
 * [n][L][H][W]; B_i the k x k patch of the up-sampled image U centred at HR
 * pixel i; F_i = Phi_i D (Eq. 2, right half; Eq. 3 image form) and
 * y_i = F_i B_i^T (Eq. 2, left half), pairing taps with the same index
 * (Section III-B describes the filtering as an element-wise product of the two
 * operands summed over the k^2 channels: no flip).
 *
 * Parity pins (tests/test_oracle_pins.py): closed-form bicubic weights, a library
 * bicubic resize, a library cross-correlation on the replicate-padded image, a
 * hand-worked 4x4 example, delta-atom / constant-image / linearity / s = D /
 * prefix / permutation identities, and a brute-force sort for the selection;
 * for the bilinear variant of stage 1a a library bilinear resize, closed-form
 * weights, exact reproduction of affine images away from the border and the
 * delta-atom identity.  No function here is parity-unpinned.
 */
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>

#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

enum { REF_F32 = 0, REF_F16 = 1 };
enum { REF_CLAMP01 = 1u, REF_IDX_GLOBAL = 2u, REF_COEF_COMPACT = 4u, REF_UPSAMPLE_BILINEAR = 8u };
enum { REF_OK = 0, REF_ERR_NULL = 1, REF_ERR_SHAPE = 2, REF_ERR_UNSUPPORTED = 3 };

struct Dims {
    int n, c, h, w, r, k, L;
    int H() const { return h * r; }
    int W() const { return w * r; }
    int p() const { return (k - 1) / 2; }
};

int check_dims(const Dims& d)
{
    if (d.n < 1 || d.c < 1 || d.h < 1 || d.w < 1 || d.L < 1) return REF_ERR_SHAPE;
    if (d.r < 1 || d.r > 8) return REF_ERR_UNSUPPORTED;
    if (d.k < 1 || d.k > 9 || (d.k % 2) == 0) return REF_ERR_UNSUPPORTED;
    if (d.L > 256) return REF_ERR_UNSUPPORTED;
    return REF_OK;
}

/* binary16 bit pattern -> double, exact */
double half_to_double(uint16_t b)
{
    const int sign = b >> 15;
    const int e = (b >> 10) & 0x1F;
    const int m = b & 0x3FF;
    double v;
    if (e == 0)
        v = std::ldexp((double)m, -24);
    else if (e == 31)
        v = m ? NAN : INFINITY;
    else
        v = std::ldexp((double)(m | 0x400), e - 25);
    return sign ? -v : v;
}

/* coefficient element `i` of a buffer in the given storage type, widened exactly */
double coef_at(const void* coef, int dtype, int64_t i)
{
    if (dtype == REF_F16) return half_to_double(((const uint16_t*)coef)[i]);
    return (double)((const float*)coef)[i];
}

/* magnitude bits (sign cleared) as an unsigned integer: the selection key */
uint32_t coef_mag_bits(const void* coef, int dtype, int64_t i)
{
    if (dtype == REF_F16) return (uint32_t)(((const uint16_t*)coef)[i] & 0x7FFFu);
    uint32_t u;
    std::memcpy(&u, (const float*)coef + i, 4);
    return u & 0x7FFFFFFFu;
}

int clampi(int v, int lo, int hi) { return v < lo ? lo : (v > hi ? hi : v); }

/*
 * Keys cubic-convolution weights with A = -0.75 for fractional offset t in [0,1):
 * taps sit at distances t+1, t, 1-t, 2-t from the sample point.
 */
void cubic_weights(double t, double wgt[4])
{
    const double A = -0.75;
    auto inner = [&](double z) { return ((A + 2.0) * z - (A + 3.0)) * z * z + 1.0; };          /* |z| <= 1 */
    auto outer = [&](double z) { return ((A * z - 5.0 * A) * z + 8.0 * A) * z - 4.0 * A; };    /* 1 < |z| < 2 */
    wgt[0] = outer(t + 1.0);
    wgt[1] = inner(t);
    wgt[2] = inner(1.0 - t);
    wgt[3] = outer(2.0 - t);
}

/*
 * Stage 1a: one up-sampled value U[Y][X] of one LR plane (h x w).
 * Half-pixel centres: src = (X + 1/2)/r - 1/2 (not clamped); taps ix-1..ix+2
 * with each index clamped to the image (edge replicate).
 */
double bicubic_at(const float* plane, int h, int w, int r, int Y, int X)
{
    const double sy = (Y + 0.5) / r - 0.5;
    const double sx = (X + 0.5) / r - 0.5;
    const int iy = (int)std::floor(sy);
    const int ix = (int)std::floor(sx);
    double wy[4], wx[4];
    cubic_weights(sy - iy, wy);
    cubic_weights(sx - ix, wx);
    double acc = 0.0;
    for (int a = 0; a < 4; ++a) {
        const int yy = clampi(iy - 1 + a, 0, h - 1);
        double row = 0.0;
        for (int b = 0; b < 4; ++b) {
            const int xx = clampi(ix - 1 + b, 0, w - 1);
            row += wx[b] * (double)plane[(int64_t)yy * w + xx];
        }
        acc += wy[a] * row;
    }
    return acc;
}

/* Per-pixel top-s: keys = (magnitude bits, then lower atom index first); result in rank order. */
void select_pixel(const void* coef, int dtype, int64_t base, int64_t plane_stride, int L, int s, uint8_t* out_idx)
{
    std::vector<std::pair<uint32_t, int>> keys((size_t)L);
    for (int l = 0; l < L; ++l) keys[(size_t)l] = {coef_mag_bits(coef, dtype, base + l * plane_stride), l};
    std::stable_sort(keys.begin(), keys.end(),
                     [](const std::pair<uint32_t, int>& a, const std::pair<uint32_t, int>& b) { return a.first > b.first; });
    for (int q = 0; q < s; ++q) out_idx[q] = (uint8_t)keys[(size_t)q].second;
}

/*
 * Stages 3 + 4 at one HR pixel given the atoms to use:
 *   F[j]  = sum_q  weight_q * dict[atom_q][j]                (Eq. 2, F_i = Phi_i D)
 *   y_c   = sum_j  F[j] * B_c[j],  B_c[a*k+b] = U_c[clamp(Y+a-p)][clamp(X+b-p)]   (Eq. 2, y_i = F_i B_i^T)
 * `patch(c, yy, xx)` returns U_c at an (already clamped) HR position.
 */
template <class PatchFn>
void regress_pixel(const Dims& d, const float* dict, int natoms, const int* atoms, const double* weights, int Y, int X,
                   unsigned flags, PatchFn patch, double* y /* [c] */)
{
    const int k = d.k, p = d.p(), kk = k * k;
    double F[81];
    for (int j = 0; j < kk; ++j) F[j] = 0.0;
    for (int q = 0; q < natoms; ++q)
        for (int j = 0; j < kk; ++j) F[j] += weights[q] * (double)dict[(int64_t)atoms[q] * kk + j];
    for (int ch = 0; ch < d.c; ++ch) {
        double acc = 0.0;
        for (int a = 0; a < k; ++a)
            for (int b = 0; b < k; ++b) {
                const int yy = clampi(Y + a - p, 0, d.H() - 1);
                const int xx = clampi(X + b - p, 0, d.W() - 1);
                acc += F[a * k + b] * patch(ch, yy, xx);
            }
        if (flags & REF_CLAMP01) acc = acc < 0.0 ? 0.0 : (acc > 1.0 ? 1.0 : acc);
        y[ch] = acc;
    }
}

/* Atom list and weights of one pixel for every mode of the selected regression. */
void gather_selected(const Dims& d, const void* coef_or_sel, int dtype, const uint8_t* idx, const float* gamma, int s,
                     unsigned flags, int frame, int64_t pix /* Y*W+X */, int* atoms, double* weights)
{
    const int64_t HW = (int64_t)d.H() * d.W();
    if (flags & REF_IDX_GLOBAL) {
        /* the paper's structured selection: one atom subset S (and channel re-weights gamma) for all pixels */
        for (int q = 0; q < s; ++q) {
            atoms[q] = idx[q];
            const int64_t plane = (flags & REF_COEF_COMPACT) ? q : (int64_t)idx[q];
            const int64_t nplanes = (flags & REF_COEF_COMPACT) ? s : d.L;
            const double phi = coef_at(coef_or_sel, dtype, ((int64_t)frame * nplanes + plane) * HW + pix);
            weights[q] = (gamma ? (double)gamma[q] : 1.0) * phi;
        }
        return;
    }
    uint8_t local[256];
    const uint8_t* my = nullptr;
    if (idx) {
        for (int q = 0; q < s; ++q) local[q] = idx[((int64_t)frame * s + q) * HW + pix];
        my = local;
    } else { /* fused select + regress: choose the atoms here */
        select_pixel(coef_or_sel, dtype, (int64_t)frame * d.L * HW + pix, HW, d.L, s, local);
        my = local;
    }
    for (int q = 0; q < s; ++q) {
        atoms[q] = my[q];
        const int64_t plane = (flags & REF_COEF_COMPACT) ? q : (int64_t)my[q];
        const int64_t nplanes = (flags & REF_COEF_COMPACT) ? s : d.L;
        weights[q] = coef_at(coef_or_sel, dtype, ((int64_t)frame * nplanes + plane) * HW + pix);
    }
}

/*
 * Stage 1a with the interpolation the paper's text names (Section II-A: bilinear): the value at the same
 * half-pixel sample point src = (X + 1/2)/r - 1/2, interpolated linearly between the two nearest LR samples
 * per axis, indices clamped to the image.
 */
double bilinear_at(const float* plane, int h, int w, int r, int Y, int X)
{
    const double sy = (Y + 0.5) / r - 0.5;
    const double sx = (X + 0.5) / r - 0.5;
    const int iy = (int)std::floor(sy);
    const int ix = (int)std::floor(sx);
    const double ty = sy - iy, tx = sx - ix;
    const int y0 = clampi(iy, 0, h - 1), y1 = clampi(iy + 1, 0, h - 1);
    const int x0 = clampi(ix, 0, w - 1), x1 = clampi(ix + 1, 0, w - 1);
    const double top = (1.0 - tx) * (double)plane[(int64_t)y0 * w + x0] + tx * (double)plane[(int64_t)y0 * w + x1];
    const double bot = (1.0 - tx) * (double)plane[(int64_t)y1 * w + x0] + tx * (double)plane[(int64_t)y1 * w + x1];
    return (1.0 - ty) * top + ty * bot;
}

double upsample_at(const float* plane, int h, int w, int r, int Y, int X, unsigned flags)
{
    return (flags & REF_UPSAMPLE_BILINEAR) ? bilinear_at(plane, h, w, r, Y, X) : bicubic_at(plane, h, w, r, Y, X);
}

void set_threads(int threads)
{
#ifdef _OPENMP
    if (threads > 0) omp_set_num_threads(threads);
#else
    (void)threads;
#endif
}

/* U for the whole batch, [n][c][H][W] */
void upsample_all(const float* lr, const Dims& d, std::vector<double>& U, unsigned flags)
{
    const int H = d.H(), W = d.W();
    U.resize((size_t)d.n * d.c * H * W);
    const int64_t planes = (int64_t)d.n * d.c;
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t pl = 0; pl < planes; ++pl)
        for (int Y = 0; Y < H; ++Y) {
            const float* src = lr + pl * (int64_t)d.h * d.w;
            double* dst = U.data() + (pl * H + Y) * (int64_t)W;
            for (int X = 0; X < W; ++X) dst[X] = upsample_at(src, d.h, d.w, d.r, Y, X, flags);
        }
}

} // namespace

extern "C" {

/* Stage 1a alone: hr[n][c][H][W] (fp64) from lr[n][c][h][w] (fp32). */
int sr_ref_bicubic_upsample(const float* lr, double* hr, int n, int c, int h, int w, int r, int threads)
{
    Dims d{n, c, h, w, r, 1, 1};
    if (!lr || !hr) return REF_ERR_NULL;
    if (int e = check_dims(d)) return e;
    set_threads(threads);
    std::vector<double> U;
    upsample_all(lr, d, U, 0u);
    std::memcpy(hr, U.data(), U.size() * sizeof(double));
    return REF_OK;
}

/* Stage 1a alone, bilinear form: hr[n][c][H][W] (fp64) from lr[n][c][h][w] (fp32). */
int sr_ref_bilinear_upsample(const float* lr, double* hr, int n, int c, int h, int w, int r, int threads)
{
    Dims d{n, c, h, w, r, 1, 1};
    if (!lr || !hr) return REF_ERR_NULL;
    if (int e = check_dims(d)) return e;
    set_threads(threads);
    std::vector<double> U;
    upsample_all(lr, d, U, REF_UPSAMPLE_BILINEAR);
    std::memcpy(hr, U.data(), U.size() * sizeof(double));
    return REF_OK;
}

/* Stages 1-4 with every atom: out[n][c][H][W] fp64. */
int sr_ref_dict_regress_dense(const float* lr, const void* coef, int coef_dtype, const float* dict, double* out, int n,
                              int c, int h, int w, int r, int k, int L, unsigned flags, int threads)
{
    Dims d{n, c, h, w, r, k, L};
    if (!lr || !coef || !dict || !out) return REF_ERR_NULL;
    if (int e = check_dims(d)) return e;
    set_threads(threads);
    const int H = d.H(), W = d.W();
    const int64_t HW = (int64_t)H * W;
    std::vector<double> U;
    upsample_all(lr, d, U, flags);
    std::vector<int> atoms((size_t)L);
    for (int l = 0; l < L; ++l) atoms[(size_t)l] = l;
    for (int f = 0; f < n; ++f) {
#pragma omp parallel for schedule(static)
        for (int Y = 0; Y < H; ++Y) {
            std::vector<double> wts((size_t)L), y((size_t)c);
            for (int X = 0; X < W; ++X) {
                const int64_t pix = (int64_t)Y * W + X;
                for (int l = 0; l < L; ++l) wts[(size_t)l] = coef_at(coef, coef_dtype, ((int64_t)f * L + l) * HW + pix);
                auto patch = [&](int ch, int yy, int xx) { return U[(((int64_t)f * c + ch) * H + yy) * W + xx]; };
                regress_pixel(d, dict, L, atoms.data(), wts.data(), Y, X, flags, patch, y.data());
                for (int ch = 0; ch < c; ++ch) out[((int64_t)f * c + ch) * HW + pix] = y[(size_t)ch];
            }
        }
    }
    return REF_OK;
}

/*
 * Per-pixel top-s by coefficient magnitude, ties to the lower atom index.
 * idx[n][s][H][W] in rank order (plane 0 = largest magnitude); sel (nullable)
 * [n][s][H][W] fp64 = the coefficient of each selected atom.
 */
int sr_ref_dict_select(const void* coef, int coef_dtype, uint8_t* idx, double* sel, int n, int H, int W, int L, int s,
                       int threads)
{
    if (!coef || !idx) return REF_ERR_NULL;
    if (n < 1 || H < 1 || W < 1 || L < 1 || L > 256 || s < 1 || s > L) return REF_ERR_SHAPE;
    set_threads(threads);
    const int64_t HW = (int64_t)H * W;
    for (int f = 0; f < n; ++f) {
#pragma omp parallel for schedule(static)
        for (int64_t pix = 0; pix < HW; ++pix) {
            uint8_t local[256];
            select_pixel(coef, coef_dtype, (int64_t)f * L * HW + pix, HW, L, s, local);
            for (int q = 0; q < s; ++q) {
                idx[((int64_t)f * s + q) * HW + pix] = local[q];
                if (sel) sel[((int64_t)f * s + q) * HW + pix] = coef_at(coef, coef_dtype, ((int64_t)f * L + local[q]) * HW + pix);
            }
        }
    }
    return REF_OK;
}

/*
 * Stages 1-4 with s atoms per pixel.
 *   default           idx[n][s][H][W] per pixel (NULL: select here), coefficients read from the full tensor
 *   REF_COEF_COMPACT  coef_or_sel is [n][s][H][W], plane q holds the coefficient of idx plane q
 *   REF_IDX_GLOBAL    idx[s] and gamma[s] (nullable = 1) are one subset for every pixel (the paper's
 *                     structured selection with re-weighted coefficients Phi' = gamma * Phi[S])
 * Kept coefficients are used as they are (no renormalisation); the sum runs in rank order.
 */
int sr_ref_dict_regress_selected(const float* lr, const void* coef_or_sel, int coef_dtype, const uint8_t* idx,
                                 const float* gamma, const float* dict, double* out, int n, int c, int h, int w, int r,
                                 int k, int L, int s, unsigned flags, int threads)
{
    Dims d{n, c, h, w, r, k, L};
    if (!lr || !coef_or_sel || !dict || !out) return REF_ERR_NULL;
    if ((flags & (REF_IDX_GLOBAL | REF_COEF_COMPACT)) && !idx) return REF_ERR_NULL;
    if (int e = check_dims(d)) return e;
    if (s < 1 || s > L) return REF_ERR_SHAPE;
    if (flags & REF_IDX_GLOBAL)
        for (int q = 0; q < s; ++q)
            if (idx[q] >= L) return REF_ERR_SHAPE;
    set_threads(threads);
    const int H = d.H(), W = d.W();
    const int64_t HW = (int64_t)H * W;
    std::vector<double> U;
    upsample_all(lr, d, U, flags);
    for (int f = 0; f < n; ++f) {
#pragma omp parallel for schedule(static)
        for (int Y = 0; Y < H; ++Y) {
            std::vector<double> wts((size_t)s), y((size_t)c);
            std::vector<int> atoms((size_t)s);
            for (int X = 0; X < W; ++X) {
                const int64_t pix = (int64_t)Y * W + X;
                gather_selected(d, coef_or_sel, coef_dtype, idx, gamma, s, flags, f, pix, atoms.data(), wts.data());
                auto patch = [&](int ch, int yy, int xx) { return U[(((int64_t)f * c + ch) * H + yy) * W + xx]; };
                regress_pixel(d, dict, s, atoms.data(), wts.data(), Y, X, flags, patch, y.data());
                for (int ch = 0; ch < c; ++ch) out[((int64_t)f * c + ch) * HW + pix] = y[(size_t)ch];
            }
        }
    }
    return REF_OK;
}

/*
 * The same definitions evaluated only at sampled HR pixels, for frames too
 * large to run in full.  samples[i] is a flat index into [n][H][W]; out is
 * [nsamples][c].  U is evaluated where the patch touches it instead of being
 * stored.  mode 0 = dense, 1 = selected (arguments as above).
 */
int sr_ref_regress_at(int mode, const float* lr, const void* coef_or_sel, int coef_dtype, const uint8_t* idx,
                      const float* gamma, const float* dict, const int64_t* samples, int64_t nsamples, double* out,
                      int n, int c, int h, int w, int r, int k, int L, int s, unsigned flags, int threads)
{
    Dims d{n, c, h, w, r, k, L};
    if (!lr || !coef_or_sel || !dict || !out || !samples) return REF_ERR_NULL;
    if (int e = check_dims(d)) return e;
    if (mode == 0) s = L;
    if (s < 1 || s > L) return REF_ERR_SHAPE;
    if (mode == 1 && (flags & (REF_IDX_GLOBAL | REF_COEF_COMPACT)) && !idx) return REF_ERR_NULL;
    set_threads(threads);
    const int H = d.H(), W = d.W();
    const int64_t HW = (int64_t)H * W;
#pragma omp parallel for schedule(dynamic, 64)
    for (int64_t i = 0; i < nsamples; ++i) {
        const int64_t flat = samples[i];
        const int f = (int)(flat / HW);
        const int64_t pix = flat % HW;
        const int Y = (int)(pix / W), X = (int)(pix % W);
        std::vector<double> wts((size_t)s);
        std::vector<int> atoms((size_t)s);
        if (mode == 0) {
            for (int l = 0; l < L; ++l) {
                atoms[(size_t)l] = l;
                wts[(size_t)l] = coef_at(coef_or_sel, coef_dtype, ((int64_t)f * L + l) * HW + pix);
            }
        } else {
            gather_selected(d, coef_or_sel, coef_dtype, idx, gamma, s, flags, f, pix, atoms.data(), wts.data());
        }
        auto patch = [&](int ch, int yy, int xx) {
            return upsample_at(lr + ((int64_t)f * c + ch) * d.h * d.w, d.h, d.w, d.r, yy, xx, flags);
        };
        regress_pixel(d, dict, s, atoms.data(), wts.data(), Y, X, flags, patch, out + i * c);
    }
    return REF_OK;
}

/* Top-s at sampled pixels only: idx_out[nsamples][s] in rank order. */
int sr_ref_dict_select_at(const void* coef, int coef_dtype, const int64_t* samples, int64_t nsamples, uint8_t* idx_out,
                          int n, int H, int W, int L, int s, int threads)
{
    if (!coef || !samples || !idx_out) return REF_ERR_NULL;
    if (n < 1 || H < 1 || W < 1 || L < 1 || L > 256 || s < 1 || s > L) return REF_ERR_SHAPE;
    set_threads(threads);
    const int64_t HW = (int64_t)H * W;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < nsamples; ++i) {
        const int64_t f = samples[i] / HW, pix = samples[i] % HW;
        select_pixel(coef, coef_dtype, f * L * HW + pix, HW, L, s, idx_out + i * s);
    }
    return REF_OK;
}

int sr_ref_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

} // extern "C"
