// Dictionary selection search on the device (Section III-A: Eq. 5-9, Algorithm 1).
//
// The search decides which alpha L of the L atoms a model keeps, and the per-atom re-weights gamma of its coefficient
// layer; its result is what the global-subset mode of sr_dict_regress_selected consumes. Two kernels:
//
//  selection_gram_kernel   Gram statistics over sampled HR pixels (all pixels when no sample list is given): with
//        z_l[i,c] = Phi_l[i] (dict_l . B_{i,c}) the response of atom l alone at pixel i, channel c (Eq. 6 with
//        F_{W,beta} = Phi diag(beta) D), G = Z^T Z, b = Z^T h, hh = h^T h for the target image h. A CTA takes 32
//        pixels at a time: patches B from the LR image (bicubic or bilinear taps, HR-clamped), responses, Z tile in
//        shared memory, then a register-tiled fp32 rank update of its private G (thread = a TB x TB block). After
//        every 32 pixels the fp32 block is added into the CTA's own slot of fp64 scratch memory, so fp32 only ever
//        sums 32 c terms; a second kernel adds the slots in a fixed order (no atomics: results are reproducible).
//        The arithmetic here is fp32 multiply-add on sampled pixels (the paper samples its LASSO features too): an
//        offline tool, bound by the FMA pipe.
//  selection_search_kernel   Algorithm 1 on G, b, hh in fp64 by ONE warp: LASSO by cyclic coordinate descent
//        (Eq. 7), lambda doubling and bisection to || beta ||_0 ~ alpha_t L, least-squares re-fit of gamma on the
//        support (Eq. 9, Cholesky), gamma folded into G and b, next alpha_t. A lane owns the vector elements lane,
//        lane + 32, ...; every element-wise update and every sum runs in the same order as a sequential program, with
//        separate multiplies and adds (no contraction), so the result does not depend on the parallelisation.
#include "sr_common.cuh"
#include "sr_selection.cuh"

namespace sr {

namespace {

constexpr int kGramThreads = 256;
constexpr int kGramPixels = 32;       // pixels per chunk
constexpr int kMaxSearchL = 128;

struct GramParams {
    const float* lr;
    const void* coef;
    int coef_f16;
    const float* dict;
    const float* target;
    const int64_t* samples;
    int64_t count;            // sampled pixels (or n H W)
    Problem pb;
    double* slots;            // [ctas][Dp * Dp + Dp + 8]
    int Dp;
};

__device__ __forceinline__ float coef_value(const void* coef, int f16, int64_t i)
{
    return f16 ? __half2float(__ldg(reinterpret_cast<const __half*>(coef) + i)) : __ldg(reinterpret_cast<const float*>(coef) + i);
}

template <int TB>
__global__ void __launch_bounds__(kGramThreads) selection_gram_kernel(const GramParams p)
{
    extern __shared__ __align__(16) float gsm[];
    const Problem& pb = p.pb;
    const int C = pb.c, D = pb.D, kk = pb.k * pb.k, P = (pb.k - 1) / 2;
    const int Dp = 16 * TB, rows = kGramPixels * C;
    float* sDict = gsm;                                   // [D][kk]
    float* sPatch = sDict + ((D * kk + 3) & ~3);          // [rows][kk]
    float* sZ = sPatch + ((rows * kk + 3) & ~3);          // [rows][Dp]
    float* sH = sZ + rows * Dp;                           // [rows]
    __shared__ int64_t sPix[kGramPixels];                 // flat pixel index of each pixel of the chunk, -1 = none
    const int tid = threadIdx.x, ti = tid >> 4, tj = tid & 15;
    const int64_t HW = (int64_t)pb.H * pb.W;
    const int slot_doubles = Dp * Dp + Dp + 8;
    double* slot = p.slots + (int64_t)blockIdx.x * slot_doubles;

    for (int i = tid; i < slot_doubles; i += kGramThreads) slot[i] = 0.0;     // the slot keeps the last call's contents
    for (int i = tid; i < D * kk; i += kGramThreads) sDict[i] = __ldg(p.dict + i);
    for (int i = tid; i < rows * Dp; i += kGramThreads) sZ[i] = 0.f;          // columns D..Dp-1 stay zero
    __syncthreads();

    const int64_t chunks = (p.count + kGramPixels - 1) / kGramPixels;
    for (int64_t ch = blockIdx.x; ch < chunks; ch += gridDim.x) {
        if (tid < kGramPixels) {
            const int64_t si = ch * kGramPixels + tid;
            int64_t flat = -1;
            if (si < p.count) flat = p.samples ? __ldg(p.samples + si) : si;
            if (flat < 0 || flat >= (int64_t)pb.n * HW) flat = -1;
            sPix[tid] = flat;
        }
        __syncthreads();
        // patches: B[(pixel, channel)][tap] = U_c at the clamped HR position
        for (int e = tid; e < rows * kk; e += kGramThreads) {
            const int row = e / kk, j = e - row * kk;
            const int pi = row / C, c = row - pi * C;
            const int64_t flat = sPix[pi];
            float v = 0.f;
            if (flat >= 0) {
                const int f = (int)(flat / HW);
                const int64_t pix = flat - (int64_t)f * HW;
                const int Y = (int)(pix / pb.W), X = (int)(pix - (int64_t)Y * pb.W);
                const int a = j / pb.k, b = j - a * pb.k;
                v = bicubic_point(p.lr + ((int64_t)f * C + c) * pb.h * pb.w, pb.h, pb.w, pb.r, pb.ph,
                                  clampi(Y + a - P, 0, pb.H - 1), clampi(X + b - P, 0, pb.W - 1));
            }
            sPatch[e] = v;
        }
        for (int row = tid; row < rows; row += kGramThreads) {
            const int pi = row / C, c = row - pi * C;
            const int64_t flat = sPix[pi];
            float hv = 0.f;
            if (flat >= 0) {
                const int f = (int)(flat / HW);
                hv = __ldg(p.target + ((int64_t)f * C + c) * HW + (flat - (int64_t)f * HW));
            }
            sH[row] = hv;
        }
        __syncthreads();
        // responses: z[(pixel, channel)][l] = Phi_l[pixel] * (dict_l . B)
        for (int e = tid; e < kGramPixels * D; e += kGramThreads) {
            const int pi = e / D, l = e - pi * D;
            const int64_t flat = sPix[pi];
            float phi = 0.f;
            if (flat >= 0) {
                const int f = (int)(flat / HW);
                phi = coef_value(p.coef, p.coef_f16, ((int64_t)f * D + l) * HW + (flat - (int64_t)f * HW));
            }
            const float* dl = sDict + l * kk;
            for (int c = 0; c < C; ++c) {
                const float* B = sPatch + (pi * C + c) * kk;
                float resp = 0.f;
                for (int j = 0; j < kk; ++j) resp = fmaf(dl[j], B[j], resp);
                sZ[(pi * C + c) * Dp + l] = phi * resp;
            }
        }
        __syncthreads();
        // rank update of this thread's TB x TB block, then into the fp64 slot
        float acc[TB][TB];
#pragma unroll
        for (int a = 0; a < TB; ++a)
#pragma unroll
            for (int b = 0; b < TB; ++b) acc[a][b] = 0.f;
        float bacc[TB];
#pragma unroll
        for (int a = 0; a < TB; ++a) bacc[a] = 0.f;
        float hacc = 0.f;
        for (int row = 0; row < rows; ++row) {
            const float* zr = sZ + row * Dp;
            float za[TB], zb[TB];
#pragma unroll
            for (int a = 0; a < TB; ++a) { za[a] = zr[ti * TB + a]; zb[a] = zr[tj * TB + a]; }
#pragma unroll
            for (int a = 0; a < TB; ++a)
#pragma unroll
                for (int b = 0; b < TB; ++b) acc[a][b] = fmaf(za[a], zb[b], acc[a][b]);
            if (tj == 0) {
                const float hv = sH[row];
#pragma unroll
                for (int a = 0; a < TB; ++a) bacc[a] = fmaf(za[a], hv, bacc[a]);
                if (ti == 0) hacc = fmaf(hv, hv, hacc);
            }
        }
#pragma unroll
        for (int a = 0; a < TB; ++a)
#pragma unroll
            for (int b = 0; b < TB; ++b) slot[(ti * TB + a) * Dp + tj * TB + b] += (double)acc[a][b];
        if (tj == 0) {
#pragma unroll
            for (int a = 0; a < TB; ++a) slot[Dp * Dp + ti * TB + a] += (double)bacc[a];
            if (ti == 0) slot[Dp * Dp + Dp] += (double)hacc;
        }
        __syncthreads();                                  // sZ, sPatch, sPix are rewritten by the next chunk
    }
}

__global__ void selection_gram_reduce_kernel(const double* slots, int nslots, int Dp, int D, double* G, double* b, double* hh)
{
    const int slot_doubles = Dp * Dp + Dp + 8;
    const int total = D * D + D + 1;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
        int src;
        if (i < D * D) src = (i / D) * Dp + (i % D);
        else if (i < D * D + D) src = Dp * Dp + (i - D * D);
        else src = Dp * Dp + Dp;
        double v = 0.0;
        for (int s = 0; s < nslots; ++s) v += slots[(int64_t)s * slot_doubles + src];
        if (i < D * D) G[i] = v;
        else if (i < D * D + D) b[i - D * D] = v;
        else *hh = v;
    }
}

template <int TB>
cudaError_t launch_gram_tb(const GramParams& p, int ctas, size_t smem, cudaStream_t st)
{
    auto kern = selection_gram_kernel<TB>;
    static bool configured[64] = {false};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    kern<<<ctas, kGramThreads, smem, st>>>(p);
    count_launches(1);
    return cudaGetLastError();
}

// ---- Algorithm 1 in one warp ---------------------------------------------------------------------------------------

struct SearchParams {
    const double* G;
    const double* b;
    const double* hh;
    int L;
    double nrows, alpha, dalpha, eps, lambda0, tol;
    int max_sweeps, max_bisect, max_steps;
    uint8_t* idx_out;
    float* gamma_out;
    int* count_out;
    double* trace;
    int* steps_out;
    double* chol;         // scratch: [L][L]
    int* status;
};

struct SearchState {
    double* G;            // [L][Lp]
    double *b, *beta, *r, *best, *cand, *gtot, *tmp;
    uint8_t* active;
    int* S;
    int L, Lp, lane;
    double nrows;
};

__device__ __forceinline__ double bcast(double v, int src)
{
    int lo = __double2loint(v), hi = __double2hiint(v);
    lo = __shfl_sync(0xffffffffu, lo, src);
    hi = __shfl_sync(0xffffffffu, hi, src);
    return __hiloint2double(hi, lo);
}

__device__ int count_nonzero(const SearchState& s, const double* beta)
{
    int n = 0;
    for (int l = s.lane; l < s.L; l += 32) n += (s.active[l] && beta[l] != 0.0) ? 1 : 0;
    for (int o = 16; o > 0; o >>= 1) n += __shfl_xor_sync(0xffffffffu, n, o);
    return n;
}

// Eq. 7 by cyclic coordinate descent; beta in / out. Same operation order as a sequential loop over the atoms.
__device__ int lasso_cd(const SearchState& s, double lambda, double* beta, double tol, int max_sweeps)
{
    const int L = s.L, Lp = s.Lp;
    for (int l = s.lane; l < L; l += 32) {
        if (!s.active[l]) { beta[l] = 0.0; continue; }
        double acc = 0.0;
        for (int m = 0; m < L; ++m)
            if (s.active[m]) acc = __dadd_rn(acc, __dmul_rn(s.G[l * Lp + m], beta[m]));
        s.r[l] = __dadd_rn(s.b[l], -acc);
    }
    __syncwarp();
    const double thr = __dmul_rn(__dmul_rn(0.5, lambda), s.nrows);
    int sweep = 0;
    for (; sweep < max_sweeps; ++sweep) {
        double moved = 0.0;
        for (int l = 0; l < L; ++l) {
            if (!s.active[l]) continue;
            const double gll = s.G[l * Lp + l];
            if (!(gll > 0.0)) continue;
            const int owner = l & 31;
            double delta = 0.0, nb = 0.0;
            if (s.lane == owner) {
                const double rho = __dadd_rn(s.r[l], __dmul_rn(gll, beta[l]));
                if (rho > thr) nb = __ddiv_rn(__dadd_rn(rho, -thr), gll);
                else if (rho < -thr) nb = __ddiv_rn(__dadd_rn(rho, thr), gll);
                delta = __dadd_rn(nb, -beta[l]);
            }
            delta = bcast(delta, owner);
            if (delta != 0.0) {
                for (int m = s.lane; m < L; m += 32)
                    if (s.active[m]) s.r[m] = __dadd_rn(s.r[m], -__dmul_rn(delta, s.G[m * Lp + l]));
                if (s.lane == owner) beta[l] = nb;
                moved = fmax(moved, fabs(delta));
            }
        }
        if (moved <= tol) { ++sweep; break; }
    }
    __syncwarp();
    return sweep;
}

__device__ double selection_loss(const SearchState& s, double hh, const double* beta)
{
    const int L = s.L, Lp = s.Lp;
    for (int l = s.lane; l < L; l += 32) {
        double row = 0.0;
        if (s.active[l])
            for (int m = 0; m < L; ++m)
                if (s.active[m]) row = __dadd_rn(row, __dmul_rn(s.G[l * Lp + m], beta[m]));
        s.tmp[l] = row;
    }
    __syncwarp();
    double loss = 0.0;
    if (s.lane == 0) {
        double quad = 0.0, lin = 0.0;
        for (int l = 0; l < L; ++l) {
            if (!s.active[l]) continue;
            quad = __dadd_rn(quad, __dmul_rn(beta[l], s.tmp[l]));
            lin = __dadd_rn(lin, __dmul_rn(s.b[l], beta[l]));
        }
        loss = __ddiv_rn(__dadd_rn(__dadd_rn(hh, -__dmul_rn(2.0, lin)), quad), s.nrows);
    }
    loss = bcast(loss, 0);
    __syncwarp();
    return loss;
}

// Eq. 9 on the support S (ns atoms): G_SS gamma = b_S by Cholesky in the scratch matrix A; gamma lands in s.tmp[0..ns).
__device__ bool refit_gamma(const SearchState& s, int ns, double* A)
{
    const int Lp = s.Lp;
    for (int e = s.lane; e < ns * ns; e += 32) A[e] = s.G[s.S[e / ns] * Lp + s.S[e % ns]];
    for (int i = s.lane; i < ns; i += 32) s.tmp[i] = s.b[s.S[i]];
    __syncwarp();
    for (int j = 0; j < ns; ++j) {
        double dj = 0.0;
        if (s.lane == 0) {
            dj = A[j * ns + j];
            for (int q = 0; q < j; ++q) dj = __dadd_rn(dj, -__dmul_rn(A[j * ns + q], A[j * ns + q]));
            if (dj > 0.0) { dj = __dsqrt_rn(dj); A[j * ns + j] = dj; } else dj = -1.0;
        }
        dj = bcast(dj, 0);
        if (!(dj > 0.0)) return false;
        __syncwarp();
        for (int i = j + 1 + s.lane; i < ns; i += 32) {
            double v = A[i * ns + j];
            for (int q = 0; q < j; ++q) v = __dadd_rn(v, -__dmul_rn(A[i * ns + q], A[j * ns + q]));
            A[i * ns + j] = __ddiv_rn(v, dj);
        }
        __syncwarp();
    }
    if (s.lane == 0) {
        double* y = s.tmp;
        for (int i = 0; i < ns; ++i) {
            double v = y[i];
            for (int q = 0; q < i; ++q) v = __dadd_rn(v, -__dmul_rn(A[i * ns + q], y[q]));
            y[i] = __ddiv_rn(v, A[i * ns + i]);
        }
        for (int i = ns - 1; i >= 0; --i) {
            double v = y[i];
            for (int q = i + 1; q < ns; ++q) v = __dadd_rn(v, -__dmul_rn(A[q * ns + i], y[q]));
            y[i] = __ddiv_rn(v, A[i * ns + i]);
        }
    }
    __syncwarp();
    return true;
}

__global__ void __launch_bounds__(32, 1) selection_search_kernel(const SearchParams p)
{
    extern __shared__ __align__(16) double ssm[];
    SearchState s;
    const int L = p.L;
    s.L = L; s.Lp = L | 1; s.lane = threadIdx.x; s.nrows = p.nrows;
    s.G = ssm;
    s.b = s.G + (size_t)L * s.Lp;
    s.beta = s.b + L; s.r = s.beta + L; s.best = s.r + L; s.cand = s.best + L; s.gtot = s.cand + L; s.tmp = s.gtot + L;
    s.S = reinterpret_cast<int*>(s.tmp + L);
    s.active = reinterpret_cast<uint8_t*>(s.S + L);
    const int lane = s.lane;
    for (int e = lane; e < L * L; e += 32) s.G[(e / L) * s.Lp + (e % L)] = p.G[e];
    for (int l = lane; l < L; l += 32) { s.b[l] = p.b[l]; s.beta[l] = 1.0; s.gtot[l] = 1.0; s.active[l] = 1; }
    __syncwarp();
    const double hh = *p.hh;
    double alpha_t = 1.0, lambda = p.lambda0;
    int step = 0;
    bool failed = false;
    while (alpha_t > p.alpha + 1e-12 && step < p.max_steps && !failed) {
        const double alpha_next = fmax(p.alpha, __dadd_rn(1.0, -__dmul_rn((double)(step + 1), p.dalpha)));
        const double target = __dmul_rn(alpha_next, (double)L), band = __dmul_rn(p.eps, (double)L);
        int solves = 0;
        int nnz = count_nonzero(s, s.beta);
        double lam_hi = lambda;
        // doubling
        while ((double)nnz > target) {
            for (int l = lane; l < L; l += 32) s.cand[l] = s.beta[l];
            __syncwarp();
            lasso_cd(s, lambda, s.cand, p.tol, p.max_sweeps);
            ++solves;
            nnz = count_nonzero(s, s.cand);
            for (int l = lane; l < L; l += 32) s.beta[l] = s.cand[l];
            __syncwarp();
            lam_hi = lambda;
            lambda = __dmul_rn(2.0, lambda);
        }
        for (int l = lane; l < L; l += 32) s.best[l] = s.beta[l];
        __syncwarp();
        int best_nnz = nnz;
        double best_lam = lam_hi;
        // bisection inside the last doubling step
        double left = __dmul_rn(0.5, lam_hi), right = lam_hi;
        int it = 0;
        while (fabs(__dadd_rn(target, -(double)nnz)) > band && it < p.max_bisect) {
            const double mid = __dmul_rn(0.5, __dadd_rn(left, right));
            for (int l = lane; l < L; l += 32) s.cand[l] = s.best[l];
            __syncwarp();
            lasso_cd(s, mid, s.cand, p.tol, p.max_sweeps);
            ++solves;
            ++it;
            nnz = count_nonzero(s, s.cand);
            const bool in_band_feasible = fabs(__dadd_rn(target, -(double)nnz)) <= band && (double)nnz <= target;
            if (((double)nnz <= target && nnz > best_nnz) || in_band_feasible) {
                for (int l = lane; l < L; l += 32) s.best[l] = s.cand[l];
                best_nnz = nnz;
                best_lam = mid;
                __syncwarp();
            }
            if ((double)nnz < target) right = mid;
            else if ((double)nnz > target) left = mid;
        }
        for (int l = lane; l < L; l += 32) s.beta[l] = s.best[l];
        __syncwarp();
        lambda = best_lam;
        const double loss_beta = selection_loss(s, hh, s.beta);
        // W-step: re-fit on the support
        int ns = 0;
        if (lane == 0) {
            for (int l = 0; l < L; ++l)
                if (s.active[l] && s.beta[l] != 0.0) s.S[ns++] = l;
        }
        ns = __shfl_sync(0xffffffffu, ns, 0);
        __syncwarp();
        if (ns == 0 || !refit_gamma(s, ns, p.chol)) { failed = true; break; }
        // gamma (in tmp[0..ns)) folded into G, b and the running product; the kept atoms become the active set
        for (int l = lane; l < L; l += 32) s.active[l] = 0;
        __syncwarp();
        for (int i = lane; i < ns; i += 32) s.active[s.S[i]] = 1;
        for (int e = lane; e < ns * ns; e += 32) {
            const int i = e / ns, j = e % ns;
            double* g = &s.G[s.S[i] * s.Lp + s.S[j]];
            *g = __dmul_rn(__dmul_rn(s.tmp[i], *g), s.tmp[j]);
        }
        for (int i = lane; i < ns; i += 32) {
            s.b[s.S[i]] = __dmul_rn(s.tmp[i], s.b[s.S[i]]);
            s.gtot[s.S[i]] = __dmul_rn(s.gtot[s.S[i]], s.tmp[i]);
        }
        __syncwarp();
        for (int l = lane; l < L; l += 32) s.beta[l] = s.active[l] ? 1.0 : 0.0;
        __syncwarp();
        const double loss_gamma = selection_loss(s, hh, s.beta);
        if (p.trace && lane == 0) {
            double* tr = p.trace + (size_t)step * 6;
            tr[0] = alpha_next; tr[1] = best_lam; tr[2] = (double)ns; tr[3] = loss_beta; tr[4] = loss_gamma; tr[5] = (double)solves;
        }
        alpha_t = alpha_next;
        ++step;
    }
    if (lane == 0) {
        int cnt = 0;
        if (!failed)
            for (int l = 0; l < L; ++l)
                if (s.active[l]) { p.idx_out[cnt] = (uint8_t)l; p.gamma_out[cnt] = (float)s.gtot[l]; ++cnt; }
        *p.count_out = failed ? -1 : cnt;
        if (p.steps_out) *p.steps_out = step;
    }
}

} // namespace

int selection_gram_slots() { return 2 * sm_count(); }

size_t selection_gram_slot_bytes(int D)
{
    const int Dp = (D + 15) / 16 * 16;
    return (size_t)(Dp * Dp + Dp + 8) * sizeof(double);
}

cudaError_t launch_selection_gram(const float* lr, const void* coef, int coef_dtype, const float* dict, const float* target,
                                  const int64_t* samples, int64_t nsamples, double* G, double* b, double* hh, const Problem& pb,
                                  double* slots, int nslots, cudaStream_t st)
{
    GramParams p{};
    p.lr = lr; p.coef = coef; p.coef_f16 = coef_dtype == SR_F16 ? 1 : 0; p.dict = dict; p.target = target; p.samples = samples;
    p.count = samples ? nsamples : (int64_t)pb.n * pb.H * pb.W;
    p.pb = pb;
    p.slots = slots;
    const int TB = (pb.D + 15) / 16;
    p.Dp = 16 * TB;
    const int64_t chunks = (p.count + kGramPixels - 1) / kGramPixels;
    int ctas = (int)(chunks < nslots ? chunks : nslots);
    if (ctas < 1) ctas = 1;
    const int kk = pb.k * pb.k, rows = kGramPixels * pb.c;
    const size_t smem = (size_t)(((pb.D * kk + 3) & ~3) + ((rows * kk + 3) & ~3) + rows * p.Dp + rows) * sizeof(float);
    if (smem > 200 * 1024) return cudaErrorNotSupported;
    cudaError_t e;
    switch (TB) {
    case 1: e = launch_gram_tb<1>(p, ctas, smem, st); break;
    case 2: e = launch_gram_tb<2>(p, ctas, smem, st); break;
    case 3: e = launch_gram_tb<3>(p, ctas, smem, st); break;
    case 4: e = launch_gram_tb<4>(p, ctas, smem, st); break;
    case 5: e = launch_gram_tb<5>(p, ctas, smem, st); break;
    case 6: e = launch_gram_tb<6>(p, ctas, smem, st); break;
    case 7: e = launch_gram_tb<7>(p, ctas, smem, st); break;
    case 8: e = launch_gram_tb<8>(p, ctas, smem, st); break;
    default: return cudaErrorNotSupported;
    }
    if (e != cudaSuccess) return e;
    selection_gram_reduce_kernel<<<(pb.D * pb.D + pb.D + 1 + 255) / 256, 256, 0, st>>>(slots, ctas, p.Dp, pb.D, G, b, hh);
    count_launches(1);
    return cudaGetLastError();
}

// ---- the Gram kernel without caller scratch --------------------------------------------------------------------------
//
// Some users of this library may not allocate device memory at the point where they want the Gram statistics: a
// video pipeline that sizes all of its buffers once at start-up and runs under a fixed memory budget afterwards, a
// plug-in inside a host application that owns the allocator, a service whose steady state must not call cudaMalloc
// because that call synchronises the whole device and can fail long after start-up. For them the per-CTA fp64 slots of
// selection_gram_kernel live in the array below instead of in memory the caller passes: kStaticGramSlots slots for at
// most kStaticGramMaxD atoms, 32 x (80 x 80 + 80 + 8) doubles = 1 660 928 bytes that every device which loads the
// library holds until the process exits. The array is shared by all calls and keeps what the last call left in it:
// every CTA clears its own slot before it adds to it, and two calls whose kernels could run at the same time (two
// streams, two host threads) must not both use this entry point, or they would sum into each other's slots.
constexpr int kStaticGramSlots = 32;
constexpr int kStaticGramMaxD = 80;
static __device__ __align__(256) double g_gram_static_slots[kStaticGramSlots * (kStaticGramMaxD * kStaticGramMaxD + kStaticGramMaxD + 8)];

int selection_gram_static_max_atoms() { return kStaticGramMaxD; }

// Device address of the array above on the current device. In host code the array's name only stands for the symbol;
// the address a kernel can use comes from cudaGetSymbolAddress, looked up once per device while that device is current.
static double* static_gram_slots()
{
    static double* cache[64] = {nullptr};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    if (!cache[dev]) {
        double* ptr = nullptr;
        if (cudaGetSymbolAddress((void**)&ptr, g_gram_static_slots) != cudaSuccess) return nullptr;
        cache[dev] = ptr;
    }
    return cache[dev];
}

cudaError_t launch_selection_gram_static(const float* lr, const void* coef, int coef_dtype, const float* dict, const float* target,
                                         const int64_t* samples, int64_t nsamples, double* G, double* b, double* hh, const Problem& pb,
                                         cudaStream_t st)
{
    if (pb.D > kStaticGramMaxD) return cudaErrorInvalidValue;
    double* slots = static_gram_slots();
    if (!slots) return cudaErrorUnknown;
    return launch_selection_gram(lr, coef, coef_dtype, dict, target, samples, nsamples, G, b, hh, pb, slots, kStaticGramSlots, st);
}

size_t selection_search_scratch_bytes(int L) { return (size_t)L * L * sizeof(double); }

cudaError_t launch_selection_search(const double* G, const double* b, const double* hh, double nrows, int L, const sr_search_opts& o,
                                    uint8_t* idx_out, float* gamma_out, int* count_out, double* trace, int* steps_out, double* chol,
                                    cudaStream_t st)
{
    if (L > kMaxSearchL) return cudaErrorNotSupported;
    SearchParams p{};
    p.G = G; p.b = b; p.hh = hh; p.L = L; p.nrows = nrows;
    p.alpha = o.alpha; p.dalpha = o.delta_alpha; p.eps = o.eps; p.lambda0 = o.lambda0; p.tol = o.tol;
    p.max_sweeps = o.max_sweeps; p.max_bisect = o.max_bisect; p.max_steps = o.max_steps;
    p.idx_out = idx_out; p.gamma_out = gamma_out; p.count_out = count_out; p.trace = trace; p.steps_out = steps_out; p.chol = chol;
    const int Lp = L | 1;
    const size_t smem = ((size_t)L * Lp + 7 * (size_t)L) * sizeof(double) + (size_t)L * sizeof(int) + (size_t)L + 16;
    static bool configured[64] = {false};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(selection_search_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    selection_search_kernel<<<1, 32, smem, st>>>(p);
    count_launches(1);
    return cudaGetLastError();
}

} // namespace sr
