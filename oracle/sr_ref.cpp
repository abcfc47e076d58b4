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
 * delta-atom identity.  The selection search of Section III-A (Gram statistics,
 * LASSO by coordinate descent, Algorithm 1, least-squares re-fit) is pinned in
 * tests/test_oracle_pins_selection.py: the Gram matrix against per-atom
 * responses built from the pinned dense regression, the LASSO against a library
 * solver and its optimality conditions, the re-fit against a library least-squares
 * solve, and the search against its stopping rules on hand-built problems.
 * The producer of Phi (last convolution + pixel-shuffle of the coefficient network) is pinned in
 * tests/test_oracle_pins_producer.py against a library convolution and sub-pixel shuffle and against the pinned
 * dense regression fed with its output.
 * No function here is parity-unpinned.
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
enum { REF_CLAMP01 = 1u, REF_IDX_GLOBAL = 2u, REF_COEF_COMPACT = 4u, REF_UPSAMPLE_BILINEAR = 8u, REF_OUT_U8 = 32u, REF_LUMA_ONLY = 64u };
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
    /*
     * Luma-only regression (an I/O variant of this library, the usual practice of SR models that work on the Y channel;
     * not in the paper): the filter is applied to the luma Y = 0.299 R + 0.587 G + 0.114 B (BT.601) of the up-sampled
     * image, the two chroma differences keep their up-sampled values.  In RGB that is
     *     out_c = U_c + (F . B_Y - U_Y)       at the pixel, for c = R, G, B  (needs c = 3).
     */
    double luma_shift = 0.0;
    if (flags & REF_LUMA_ONLY) {
        const double wy[3] = {0.299, 0.587, 0.114};
        double acc = 0.0;
        for (int a = 0; a < k; ++a)
            for (int b = 0; b < k; ++b) {
                const int yy = clampi(Y + a - p, 0, d.H() - 1);
                const int xx = clampi(X + b - p, 0, d.W() - 1);
                acc += F[a * k + b] * (wy[0] * patch(0, yy, xx) + wy[1] * patch(1, yy, xx) + wy[2] * patch(2, yy, xx));
            }
        luma_shift = acc - (wy[0] * patch(0, Y, X) + wy[1] * patch(1, Y, X) + wy[2] * patch(2, Y, X));
    }
    for (int ch = 0; ch < d.c; ++ch) {
        double acc = 0.0;
        if (flags & REF_LUMA_ONLY) {
            acc = patch(ch, Y, X) + luma_shift;
        } else {
            for (int a = 0; a < k; ++a)
                for (int b = 0; b < k; ++b) {
                    const int yy = clampi(Y + a - p, 0, d.H() - 1);
                    const int xx = clampi(X + b - p, 0, d.W() - 1);
                    acc += F[a * k + b] * patch(ch, yy, xx);
                }
        }
        if (flags & REF_CLAMP01) acc = acc < 0.0 ? 0.0 : (acc > 1.0 ? 1.0 : acc);
        if (flags & REF_OUT_U8) {
            /* 8-bit image output (an I/O variant of this library, not in the paper): the code of the value clamped to
             * [0,1] on the 255-step grid, nearest code, ties to the even one */
            const double v = acc < 0.0 ? 0.0 : (acc > 1.0 ? 1.0 : acc);
            acc = std::nearbyint(255.0 * v);
        }
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


/* ---- dictionary selection search (Section III-A) ------------------------------------------------------------------
 *
 * The paper keeps alpha * L of the L atoms: a selecting vector beta enters the filter as F_{W,beta} = Phi diag(beta) D
 * (Eq. 5 / Eq. 6; the printed sums over i = 0..L are read as the sum over atoms), so the model output at HR pixel i,
 * channel c is y[i,c] = sum_l beta_l z_l[i,c] with the per-atom response
 *       z_l[i,c] = Phi_l[i] * (dict_l . B_{i,c}),
 * and the loss against the ground-truth image h is (1/N) || h - Z beta ||^2, N = number of rows (sampled pixels times
 * channels; the paper's N is its batch size: a constant factor on lambda).  Everything the search needs from the
 * images is the Gram matrix G = Z^T Z, b = Z^T h and h^T h.
 */
void selection_rows(const Dims& d, const float* lr, const void* coef, int dtype, const float* dict, unsigned flags,
                    int frame, int Y, int X, double* z /* [c][L] */)
{
    const int k = d.k, p = d.p(), kk = k * k;
    const int64_t HW = (int64_t)d.H() * d.W();
    for (int ch = 0; ch < d.c; ++ch) {
        const float* plane = lr + ((int64_t)frame * d.c + ch) * d.h * d.w;
        double B[81];
        for (int a = 0; a < k; ++a)
            for (int b = 0; b < k; ++b) {
                const int yy = clampi(Y + a - p, 0, d.H() - 1), xx = clampi(X + b - p, 0, d.W() - 1);
                B[a * k + b] = (flags & REF_UPSAMPLE_BILINEAR) ? bilinear_at(plane, d.h, d.w, d.r, yy, xx)
                                                                : bicubic_at(plane, d.h, d.w, d.r, yy, xx);
            }
        for (int l = 0; l < d.L; ++l) {
            double resp = 0.0;
            for (int j = 0; j < kk; ++j) resp += (double)dict[(int64_t)l * kk + j] * B[j];
            const double phi = coef_at(coef, dtype, ((int64_t)frame * d.L + l) * HW + (int64_t)Y * d.W() + X);
            z[ch * d.L + l] = phi * resp;
        }
    }
}

/* loss (1/N) (h^T h - 2 b^T beta + beta^T G beta) over the active atoms, summed in index order */
double selection_loss(const double* G, const double* b, double hh, int L, const uint8_t* active, const double* beta, double nrows)
{
    double quad = 0.0, lin = 0.0;
    for (int l = 0; l < L; ++l) {
        if (!active[l]) continue;
        double row = 0.0;
        for (int m = 0; m < L; ++m)
            if (active[m]) row += G[(int64_t)l * L + m] * beta[m];
        quad += beta[l] * row;
        lin += b[l] * beta[l];
    }
    return (hh - 2.0 * lin + quad) / nrows;
}

/*
 * Eq. 7: beta = argmin (1/N) || h - Z beta ||^2 + lambda |beta|_1 over the active atoms, by cyclic coordinate descent
 * on the Gram matrix.  r = b - G beta is kept up to date; one coordinate step is
 *       rho = r_l + G_ll beta_l,   beta_l <- soft(rho, lambda N / 2) / G_ll,   r <- r - (beta_l_new - beta_l_old) G[:, l].
 * Sweeps repeat until no coefficient moved by more than tol (or max_sweeps).  Returns the number of sweeps.
 */
int lasso_cd(const double* G, const double* b, int L, const uint8_t* active, double nrows, double lambda, double* beta,
             double tol, int max_sweeps)
{
    std::vector<double> r(L, 0.0);
    for (int l = 0; l < L; ++l) {
        if (!active[l]) { beta[l] = 0.0; continue; }
        double acc = 0.0;
        for (int m = 0; m < L; ++m)
            if (active[m]) acc += G[(int64_t)l * L + m] * beta[m];
        r[l] = b[l] - acc;
    }
    const double thr = 0.5 * lambda * nrows;
    int sweep = 0;
    for (; sweep < max_sweeps; ++sweep) {
        double moved = 0.0;
        for (int l = 0; l < L; ++l) {
            if (!active[l]) continue;
            const double gll = G[(int64_t)l * L + l];
            if (!(gll > 0.0)) continue;
            const double rho = r[l] + gll * beta[l];
            double nb = 0.0;
            if (rho > thr) nb = (rho - thr) / gll;
            else if (rho < -thr) nb = (rho + thr) / gll;
            const double delta = nb - beta[l];
            if (delta != 0.0) {
                for (int m = 0; m < L; ++m)
                    if (active[m]) r[m] -= delta * G[(int64_t)m * L + l];
                beta[l] = nb;
                if (std::fabs(delta) > moved) moved = std::fabs(delta);
            }
        }
        if (moved <= tol) { ++sweep; break; }
    }
    return sweep;
}

int count_nonzero(const double* beta, int L, const uint8_t* active)
{
    int n = 0;
    for (int l = 0; l < L; ++l) n += (active[l] && beta[l] != 0.0) ? 1 : 0;
    return n;
}

/* Eq. 9: gamma = argmin || h - sum_{l in S} gamma_l z_l ||^2, i.e. G_SS gamma = b_S, by Cholesky (G_SS = R^T R).
 * Returns false when G_SS is not positive definite. */
bool refit_gamma(const double* G, const double* b, int L, const std::vector<int>& S, std::vector<double>& gamma)
{
    const int s = (int)S.size();
    std::vector<double> A((size_t)s * s), y(s);
    for (int i = 0; i < s; ++i) {
        for (int j = 0; j < s; ++j) A[(size_t)i * s + j] = G[(int64_t)S[i] * L + S[j]];
        y[i] = b[S[i]];
    }
    for (int j = 0; j < s; ++j) {                 /* lower-triangular factor in place, column by column */
        double dj = A[(size_t)j * s + j];
        for (int q = 0; q < j; ++q) dj -= A[(size_t)j * s + q] * A[(size_t)j * s + q];
        if (!(dj > 0.0)) return false;
        dj = std::sqrt(dj);
        A[(size_t)j * s + j] = dj;
        for (int i = j + 1; i < s; ++i) {
            double v = A[(size_t)i * s + j];
            for (int q = 0; q < j; ++q) v -= A[(size_t)i * s + q] * A[(size_t)j * s + q];
            A[(size_t)i * s + j] = v / dj;
        }
    }
    for (int i = 0; i < s; ++i) {                 /* forward, then backward substitution */
        double v = y[i];
        for (int q = 0; q < i; ++q) v -= A[(size_t)i * s + q] * y[q];
        y[i] = v / A[(size_t)i * s + i];
    }
    for (int i = s - 1; i >= 0; --i) {
        double v = y[i];
        for (int q = i + 1; q < s; ++q) v -= A[(size_t)q * s + i] * y[q];
        y[i] = v / A[(size_t)i * s + i];
    }
    gamma.assign(y.begin(), y.end());
    return true;
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
    if ((flags & REF_LUMA_ONLY) && c != 3) return REF_ERR_UNSUPPORTED;
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
    if ((flags & REF_LUMA_ONLY) && c != 3) return REF_ERR_UNSUPPORTED;
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
    if ((flags & REF_LUMA_ONLY) && c != 3) return REF_ERR_UNSUPPORTED;
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

/*
 * Gram statistics of the selection problem over sampled HR pixels (flat [n][H][W] indices; samples == NULL: every
 * pixel), all channels of each: G [L][L] = Z^T Z, b [L] = Z^T h, *hh = h^T h, with the target image h [n][c][H][W].
 */
int sr_ref_selection_gram(const float* lr, const void* coef, int coef_dtype, const float* dict, const float* target,
                          const int64_t* samples, int64_t nsamples, double* G, double* b, double* hh, int n, int c, int h,
                          int w, int r, int k, int L, unsigned flags, int threads)
{
    if (!lr || !coef || !dict || !target || !G || !b || !hh) return REF_ERR_NULL;
    const Dims d{n, c, h, w, r, k, L};
    if (int e = check_dims(d)) return e;
    if (c > 16) return REF_ERR_UNSUPPORTED;
    const int64_t HW = (int64_t)d.H() * d.W();
    const int64_t count = samples ? nsamples : (int64_t)n * HW;
#ifdef _OPENMP
    const int nt = threads > 0 ? threads : omp_get_max_threads();
#else
    const int nt = 1;
#endif
    std::vector<std::vector<double>> part(nt, std::vector<double>((size_t)L * L + L + 1, 0.0));
    int bad = 0;
#pragma omp parallel num_threads(nt)
    {
#ifdef _OPENMP
        std::vector<double>& acc = part[omp_get_thread_num()];
#else
        std::vector<double>& acc = part[0];
#endif
        std::vector<double> z((size_t)c * L);
#pragma omp for schedule(static)
        for (int64_t si = 0; si < count; ++si) {
            const int64_t flat = samples ? samples[si] : si;
            if (flat < 0 || flat >= (int64_t)n * HW) { bad = 1; continue; }
            const int frame = (int)(flat / HW);
            const int64_t pix = flat % HW;
            const int Y = (int)(pix / d.W()), X = (int)(pix % d.W());
            selection_rows(d, lr, coef, coef_dtype, dict, flags, frame, Y, X, z.data());
            for (int ch = 0; ch < c; ++ch) {
                const double hv = (double)target[((int64_t)frame * c + ch) * HW + pix];
                const double* zr = z.data() + (size_t)ch * L;
                for (int l = 0; l < L; ++l) {
                    for (int m = 0; m < L; ++m) acc[(size_t)l * L + m] += zr[l] * zr[m];
                    acc[(size_t)L * L + l] += zr[l] * hv;
                }
                acc[(size_t)L * L + L] += hv * hv;
            }
        }
    }
    if (bad) return REF_ERR_SHAPE;
    for (int64_t i = 0; i < (int64_t)L * L; ++i) { double v = 0.0; for (int t = 0; t < nt; ++t) v += part[t][i]; G[i] = v; }
    for (int l = 0; l < L; ++l) { double v = 0.0; for (int t = 0; t < nt; ++t) v += part[t][(size_t)L * L + l]; b[l] = v; }
    { double v = 0.0; for (int t = 0; t < nt; ++t) v += part[t][(size_t)L * L + L]; *hh = v; }
    return REF_OK;
}

/* Eq. 7 for one lambda; beta holds the start on entry and the solution on return; *sweeps the sweeps used. */
int sr_ref_lasso_cd(const double* G, const double* b, int L, const uint8_t* active, double nrows, double lambda,
                    double* beta, double tol, int max_sweeps, int* sweeps)
{
    if (!G || !b || !active || !beta) return REF_ERR_NULL;
    if (L < 1 || L > 256 || !(nrows > 0.0) || !(lambda >= 0.0)) return REF_ERR_SHAPE;
    const int n = lasso_cd(G, b, L, active, nrows, lambda, beta, tol, max_sweeps);
    if (sweeps) *sweeps = n;
    return REF_OK;
}

/*
 * Algorithm 1 on the Gram statistics.  Step t lowers the kept fraction to alpha_{t+1} = max(alpha, alpha_t -
 * delta_alpha) and looks for a lambda whose LASSO solution keeps alpha_{t+1} L atoms within eps L:
 *   - lambda starts from the previous step's value and is doubled until || beta ||_0 <= alpha_{t+1} L;
 *   - then lambda is bisected between the last two values of the doubling.  (The printed listing brackets
 *     [lambda, 2 lambda] after its last doubling and moves the left end when too few atoms survive, which cannot
 *     approach the target; it is read as the bracket of the last doubling step, as the text says, with the ends
 *     moved the way a bisection needs: too few atoms -> lower the right end, too many -> raise the left end.)
 *     If no lambda lands inside the band within max_bisect halvings, the feasible solution with the most atoms is kept;
 *   - the weights of the coefficient layer are re-fitted on the kept atoms by least squares (Eq. 9): gamma solves
 *     G_SS gamma = b_S; the re-fit layer replaces the old one, i.e. G <- diag(gamma) G_SS diag(gamma), b <- gamma b_S,
 *     and beta restarts from 1 on the kept atoms.
 * Output: the kept atoms in ascending order, the product of their re-weights over all steps, and per step
 * trace[t][0..5] = alpha_{t+1}, lambda used, atoms kept, loss after the beta step, loss after the re-fit, LASSO solves.
 */
int sr_ref_selection_search(const double* G_in, const double* b_in, double hh, int L, double nrows, double alpha,
                            double delta_alpha, double eps, double lambda0, double tol, int max_sweeps, int max_bisect,
                            uint8_t* idx_out, double* gamma_out, int* count_out, double* trace, int max_steps, int* steps_out)
{
    if (!G_in || !b_in || !idx_out || !gamma_out || !count_out) return REF_ERR_NULL;
    if (L < 1 || L > 256 || !(nrows > 0.0) || !(alpha > 0.0) || !(alpha <= 1.0) || !(delta_alpha > 0.0) || !(lambda0 > 0.0) || !(eps >= 0.0))
        return REF_ERR_SHAPE;
    std::vector<double> G(G_in, G_in + (size_t)L * L), b(b_in, b_in + L), beta(L, 1.0), gtot(L, 1.0), best(L), cand(L);
    std::vector<uint8_t> active(L, 1);
    double alpha_t = 1.0, lambda = lambda0;
    int step = 0;
    while (alpha_t > alpha + 1e-12 && step < max_steps) {        /* until alpha_t <= alpha (up to rounding of the schedule) */
        const double alpha_next = std::max(alpha, 1.0 - (double)(step + 1) * delta_alpha);   /* alpha_t - delta_alpha, without the rounding of repeated subtraction */
        const double target = alpha_next * L, band = eps * L;
        int solves = 0;
        int nnz = count_nonzero(beta.data(), L, active.data());
        double lam_used = lambda, lam_hi = lambda;
        bool have = false;                                   /* `best` holds a feasible solution (nnz <= target) */
        int best_nnz = -1;
        double best_lam = lambda;
        /* doubling */
        while ((double)nnz > target) {
            cand = beta;
            lasso_cd(G.data(), b.data(), L, active.data(), nrows, lambda, cand.data(), tol, max_sweeps);
            ++solves;
            nnz = count_nonzero(cand.data(), L, active.data());
            beta = cand;
            lam_hi = lambda;
            lambda = 2.0 * lambda;
        }
        best = beta; best_nnz = nnz; best_lam = lam_hi; have = true;
        /* bisection inside the last doubling step */
        double left = 0.5 * lam_hi, right = lam_hi;
        int it = 0;
        while (std::fabs(target - (double)nnz) > band && it < max_bisect) {
            const double mid = 0.5 * (left + right);
            cand = best;
            lasso_cd(G.data(), b.data(), L, active.data(), nrows, mid, cand.data(), tol, max_sweeps);
            ++solves;
            ++it;
            nnz = count_nonzero(cand.data(), L, active.data());
            if ((double)nnz <= target && nnz > best_nnz) { best = cand; best_nnz = nnz; best_lam = mid; }
            if ((double)nnz < target) right = mid;
            else if ((double)nnz > target) left = mid;
            if (std::fabs(target - (double)nnz) <= band && (double)nnz <= target) { best = cand; best_nnz = nnz; best_lam = mid; }
        }
        (void)have;
        beta = best;
        lam_used = best_lam;
        lambda = best_lam;
        const double loss_beta = selection_loss(G.data(), b.data(), hh, L, active.data(), beta.data(), nrows);
        /* W-step: re-fit on the support */
        std::vector<int> S;
        for (int l = 0; l < L; ++l)
            if (active[l] && beta[l] != 0.0) S.push_back(l);
        if (S.empty()) return REF_ERR_UNSUPPORTED;
        std::vector<double> gamma;
        if (!refit_gamma(G.data(), b.data(), L, S, gamma)) return REF_ERR_UNSUPPORTED;
        std::fill(active.begin(), active.end(), (uint8_t)0);
        for (size_t i = 0; i < S.size(); ++i) active[S[i]] = 1;
        for (size_t i = 0; i < S.size(); ++i) {
            for (size_t j = 0; j < S.size(); ++j) G[(size_t)S[i] * L + S[j]] = gamma[i] * G[(size_t)S[i] * L + S[j]] * gamma[j];
            b[S[i]] = gamma[i] * b[S[i]];
            gtot[S[i]] = gtot[S[i]] * gamma[i];
        }
        for (int l = 0; l < L; ++l) beta[l] = active[l] ? 1.0 : 0.0;
        const double loss_gamma = selection_loss(G.data(), b.data(), hh, L, active.data(), beta.data(), nrows);
        if (trace) {
            double* tr = trace + (size_t)step * 6;
            tr[0] = alpha_next; tr[1] = lam_used; tr[2] = (double)S.size(); tr[3] = loss_beta; tr[4] = loss_gamma; tr[5] = (double)solves;
        }
        alpha_t = alpha_next;
        ++step;
    }
    int cnt = 0;
    for (int l = 0; l < L; ++l)
        if (active[l]) { idx_out[cnt] = (uint8_t)l; gamma_out[cnt] = gtot[l]; ++cnt; }
    *count_out = cnt;
    if (steps_out) *steps_out = step;
    return REF_OK;
}

/*
 * The producer of Phi (Section II-A, stage 2: LaparNet is a stack of fusion blocks, pixel-shuffle layers and
 * convolutions; only its last two layers are restated here, with seeded weights, for the call that fuses them with the
 * regression).
 * The LR feature map feat[n][h][w][cin] (binary16, channels last) goes through one convolution with kc x kc taps,
 * zero padding kc/2, weights wconv[L r^2][cin][kc][kc] and bias[L r^2] (fp32), and a pixel-shuffle by r:
 *     Phi_l(Y, X) = conv[l r^2 + (Y mod r) r + (X mod r)](Y div r, X div r)
 * (the channel order of the common sub-pixel layer).  No activation follows: Phi are the raw outputs.
 */
static double producer_coef_at(const uint16_t* feat, const float* wconv, const float* bias, int cin, int kc, const Dims& d,
                               int frame, int l, int Y, int X)
{
    const int r = d.r, pc = kc / 2;
    const int o = l * r * r + (Y % r) * r + (X % r);
    const int y0 = Y / r, x0 = X / r;
    double acc = bias ? (double)bias[o] : 0.0;
    for (int ci = 0; ci < cin; ++ci)
        for (int dy = 0; dy < kc; ++dy)
            for (int dx = 0; dx < kc; ++dx) {
                const int yy = y0 + dy - pc, xx = x0 + dx - pc;
                if (yy < 0 || yy >= d.h || xx < 0 || xx >= d.w) continue;            /* zero padding */
                const double v = half_to_double(feat[(((int64_t)frame * d.h + yy) * d.w + xx) * cin + ci]);
                acc += v * (double)wconv[(((int64_t)o * cin + ci) * kc + dy) * kc + dx];
            }
    return acc;
}

/* Phi[n][L][H][W] (fp64) from the feature map: the tensor the regression calls would otherwise read from memory. */
int sr_ref_producer_coef(const void* feat, const float* wconv, const float* bias, double* phi, int n, int h, int w, int r,
                         int L, int cin, int kc, int threads)
{
    Dims d{n, 1, h, w, r, 1, L};
    if (!feat || !wconv || !phi) return REF_ERR_NULL;
    if (int e = check_dims(d)) return e;
    if (cin < 1 || kc < 1 || (kc % 2) == 0) return REF_ERR_UNSUPPORTED;
    set_threads(threads);
    const int H = d.H(), W = d.W();
    for (int f = 0; f < n; ++f)
        for (int l = 0; l < L; ++l) {
#pragma omp parallel for schedule(static)
            for (int Y = 0; Y < H; ++Y)
                for (int X = 0; X < W; ++X)
                    phi[(((int64_t)f * L + l) * H + Y) * W + X] =
                        producer_coef_at((const uint16_t*)feat, wconv, bias, cin, kc, d, f, l, Y, X);
        }
    return REF_OK;
}

/*
 * Stages 1-4 with Phi taken from the producer instead of memory: out[n][c][H][W] fp64.  With idx == NULL every atom is
 * used (Eq. 2); with idx[s] (and gamma[s], or NULL for ones) the global subset of Section III-A, Eq. 6 / Eq. 9.
 * Phi is not rounded to any storage type on the way: the fused path never stores it.
 */
int sr_ref_producer_regress(const float* lr, const void* feat, const float* wconv, const float* bias, const float* dict,
                            const uint8_t* idx, const float* gamma, int s, double* out, int n, int c, int h, int w, int r,
                            int k, int L, int cin, int kc, unsigned flags, int threads)
{
    Dims d{n, c, h, w, r, k, L};
    if (!lr || !feat || !wconv || !dict || !out) return REF_ERR_NULL;
    if (int e = check_dims(d)) return e;
    if (cin < 1 || kc < 1 || (kc % 2) == 0) return REF_ERR_UNSUPPORTED;
    if ((flags & REF_LUMA_ONLY) && c != 3) return REF_ERR_UNSUPPORTED;
    if (idx && (s < 1 || s > L)) return REF_ERR_SHAPE;
    set_threads(threads);
    const int H = d.H(), W = d.W();
    std::vector<double> U;
    upsample_all(lr, d, U, flags);
    const int natoms = idx ? s : L;
    std::vector<int> atoms((size_t)natoms);
    for (int q = 0; q < natoms; ++q) atoms[(size_t)q] = idx ? (int)idx[q] : q;
    for (int q = 0; q < natoms; ++q)
        if (atoms[(size_t)q] >= L) return REF_ERR_SHAPE;
    for (int f = 0; f < n; ++f) {
#pragma omp parallel for schedule(static)
        for (int Y = 0; Y < H; ++Y) {
            std::vector<double> wts((size_t)natoms), y((size_t)c), xwin((size_t)cin * kc * kc);
            for (int X = 0; X < W; ++X) {
                /* the feature values under the kernel at this pixel's LR position, widened once ([ci][dy][dx], zeros
                 * outside the map); then Phi_l as in producer_coef_at, one dot product per atom */
                const int pc = kc / 2, y0 = Y / r, x0 = X / r;
                for (int ci = 0; ci < cin; ++ci)
                    for (int dy = 0; dy < kc; ++dy)
                        for (int dx = 0; dx < kc; ++dx) {
                            const int yy = y0 + dy - pc, xx = x0 + dx - pc;
                            const bool inside = yy >= 0 && yy < h && xx >= 0 && xx < w;
                            xwin[((size_t)ci * kc + dy) * kc + dx] =
                                inside ? half_to_double(((const uint16_t*)feat)[(((int64_t)f * h + yy) * w + xx) * cin + ci]) : 0.0;
                        }
                for (int q = 0; q < natoms; ++q) {
                    const int o = atoms[(size_t)q] * r * r + (Y % r) * r + (X % r);
                    const float* wrow = wconv + (int64_t)o * cin * kc * kc;
                    double phi = bias ? (double)bias[o] : 0.0;
                    for (int i = 0; i < cin * kc * kc; ++i) phi += xwin[(size_t)i] * (double)wrow[i];
                    wts[(size_t)q] = ((idx && gamma) ? (double)gamma[q] : 1.0) * phi;
                }
                auto patch = [&](int ch, int yy, int xx) { return U[(((int64_t)f * c + ch) * H + yy) * W + xx]; };
                regress_pixel(d, dict, natoms, atoms.data(), wts.data(), Y, X, flags, patch, y.data());
                for (int ch = 0; ch < c; ++ch) out[(((int64_t)f * c + ch) * H + Y) * W + X] = y[(size_t)ch];
            }
        }
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
