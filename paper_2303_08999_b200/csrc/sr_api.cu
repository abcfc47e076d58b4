// C ABI entry points: argument validation, path selection, status reporting.
#include <math.h>

#include <atomic>
#include <map>
#include <mutex>
#include <tuple>
#include <vector>

#include "sr_common.cuh"
#include "sr_regress_listed.cuh"
#include "sr_regress_subset.cuh"
#include "sr_producer.cuh"
#include "sr_regress_tc.cuh"
#include "sr_selection.cuh"
#include "sr_umma.cuh"

namespace sr {

__device__ int g_status_word = 0;

static std::atomic<long long> g_launches{0};
void count_launches(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

int* device_status_word()
{
    // One lookup per device, cached (the symbol's address differs per device).
    static int* cache[64] = {nullptr};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    if (!cache[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_status_word) != cudaSuccess) return nullptr;
        cache[dev] = (int*)p;
    }
    return cache[dev];
}

static std::atomic<long long> g_wait_limit{1ll << 31};
static std::atomic<int> g_lose_arrival{0};
static std::atomic<int> g_force_kernel{-1};

long long wait_cycle_limit() { return g_wait_limit.load(std::memory_order_relaxed); }

bool take_injected_lost_arrival()
{
    int n = g_lose_arrival.load(std::memory_order_relaxed);
    while (n > 0 && !g_lose_arrival.compare_exchange_weak(n, n - 1, std::memory_order_relaxed)) {}
    return n > 0;
}

int sm_count()
{
    static int cache[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 1;
    if (cache[dev] <= 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) return 1;
        cache[dev] = n;
    }
    return cache[dev];
}

// Keys cubic-convolution weights (a = -0.75) for every phase of an integer scale, computed in
// double and rounded once. src = (X + 1/2)/r - 1/2 = (2X + 1 - r) / (2r) in exact integers.
// `bilinear`: the same four-tap window with weights (0, 1 - t, t, 0), so every kernel serves both forms.
BicubicPhases make_phases(int r, bool bilinear)
{
    BicubicPhases ph{};
    const double A = -0.75;
    for (int p = 0; p < r && p < kMaxScale; ++p) {
        const int num = 2 * p + 1 - r;                     // numerator of src relative to q = X / r
        const int fl = (num >= 0) ? num / (2 * r) : -((-num + 2 * r - 1) / (2 * r));
        const double t = (double)(num - fl * 2 * r) / (double)(2 * r);
        auto inner = [&](double z) { return ((A + 2.0) * z - (A + 3.0)) * z * z + 1.0; };
        auto outer = [&](double z) { return ((A * z - 5.0 * A) * z + 8.0 * A) * z - 4.0 * A; };
        ph.w[p][0] = bilinear ? 0.f : (float)outer(t + 1.0);
        ph.w[p][1] = bilinear ? (float)(1.0 - t) : (float)inner(t);
        ph.w[p][2] = bilinear ? (float)t : (float)inner(1.0 - t);
        ph.w[p][3] = bilinear ? 0.f : (float)outer(2.0 - t);
        ph.base[p] = fl - 1;
    }
    return ph;
}

static int check_dims(const sr_dims* d, bool need_kD)
{
    if (!d) return SR_ERR_NULL;
    if (d->n < 1 || d->c < 1 || d->h < 1 || d->w < 1) return SR_ERR_SHAPE;
    if (d->scale < 1 || d->scale > kMaxScale) return SR_ERR_UNSUPPORTED;
    if (need_kD) {
        if (d->D < 1) return SR_ERR_SHAPE;
        if (d->D > 256) return SR_ERR_UNSUPPORTED;
        if (d->k < 1 || d->k > kMaxK || (d->k % 2) == 0) return SR_ERR_UNSUPPORTED;
    }
    // keep every flat index inside int64 and every per-plane index inside int32
    const int64_t H = (int64_t)d->h * d->scale, W = (int64_t)d->w * d->scale;
    if (H * W > (int64_t)0x7FFFFFFF) return SR_ERR_SHAPE;
    const int64_t planes = (int64_t)d->n * (need_kD ? (d->D > d->c ? d->D : d->c) : d->c);
    if (planes > ((int64_t)1 << 40) / (H * W)) return SR_ERR_SHAPE;
    return SR_OK;
}

static Problem make_problem(const sr_dims* d, int s, uint32_t flags)
{
    Problem pb{};
    pb.n = d->n; pb.c = d->c; pb.h = d->h; pb.w = d->w; pb.r = d->scale; pb.k = d->k; pb.D = d->D;
    pb.H = d->h * d->scale; pb.W = d->w * d->scale;
    pb.s = s; pb.flags = flags;
    pb.ph = make_phases(d->scale, (flags & SR_UPSAMPLE_BILINEAR) != 0);
    return pb;
}

static bool aligned(const void* p, size_t a) { return ((uintptr_t)p % a) == 0; }
static size_t out_align(uint32_t flags) { return (flags & SR_OUT_U8) ? 1 : ((flags & SR_OUT_F16) ? 2 : 4); }
// one output type at a time; luma-only regression needs the three colour planes
static bool bad_out_flags(uint32_t flags, const sr_dims* d)
{
    return ((flags & SR_OUT_F16) && (flags & SR_OUT_U8)) || ((flags & SR_LUMA_ONLY) && d->c != 3);
}

// Which tensor-core layout takes a dense launch. The second layout (sr_regress_tc.cu: channel-split epilogue, two CTAs
// per SM, several rows per pipeline step) wins where the coefficient stream is light and the epilogue sets the pace:
// few atoms, or 7 x 7 atoms with up to 32 of them; the first layout (sr_umma.cu) streams many atoms faster. Measured
// on the 1080p sweep points (dense, D = 16 / 32 / 72 / 128; k = 3 / 5 / 7).
static bool dense_prefers_second_layout(const Problem& pb) { return pb.D <= 16 || (pb.k == 7 && pb.D <= 32); }

// Which kernel takes a launch from index + value planes when both could. The gather kernel (sr_regress_listed.cu) pays
// s * floor(k^2 / 4) 16-byte shared-memory gathers per pixel and nothing per atom of the dictionary; the first
// tensor-core layout pays for clearing and filling a stage row of D coefficients per pixel and little per listed atom.
// Measured on the 1080p sweep points and the 4K x2 batch (D = 16 / 32 / 72 / 128; k = 3 / 5 / 7; s = 4 / 8 / 16), both
// kernels forced in turn: the gather kernel is 1.0 - 3.7 times faster wherever this returns true, and up to two times
// slower at the far end (k = 7, s = 16, few atoms).
static bool compact_prefers_listed(const Problem& pb)
{
    const int gathers = pb.s * ((pb.k * pb.k + 3) / 4);      // 16-byte units of dictionary per pixel
    if (pb.D > 96 || gathers <= 52) return true;
    if (pb.D >= 64) return gathers <= 104 || (pb.r == 2 && gathers <= 112);
    return pb.r == 2 && gathers <= 56;
}

// ---- which kernel runs a regression, and in which launch shape ----------------------------------------------------------
//
// Every regression call goes through run_regress. Without an entry in the tuning table it takes the kernel and shape
// the host rules pick; sr_tune_dense / sr_tune_selected time every legal alternative on the caller's buffers and record
// the fastest for that problem shape (the block-shape search of Section III-B, restated for this library: the legal
// set comes from shared-memory, tensor-memory and stage-count constraints instead of register-file and warp-scheduler
// limits, and it is small enough to be timed exhaustively instead of by Bayesian optimisation).
enum RegressKernel { kKernelGeneral = 0, kKernelFirstLayout = 1, kKernelSecondLayout = 2, kKernelSubset = 3, kKernelListed = 4 };

struct TuneChoice {
    int kernel = -1;      // -1: host rules
    TcTuning tc;          // second layout: tile height and rows per pipeline step
    int sub_th = 0;       // subset and listed kernels: tile height
};

typedef std::tuple<int, int, int, int, int, int, int, int, int, uint32_t, int> TuneKey;

static TuneKey tune_key(int mode, int coef_dtype, const Problem& pb)
{
    return TuneKey(mode, pb.n, pb.c, pb.h, pb.w, pb.r, pb.k, pb.D, pb.s, pb.flags, coef_dtype);
}

static std::mutex g_tune_mu;
static std::map<TuneKey, TuneChoice> g_tune_table;

static bool tune_lookup(const TuneKey& key, TuneChoice& out)
{
    std::lock_guard<std::mutex> lock(g_tune_mu);
    auto it = g_tune_table.find(key);
    if (it == g_tune_table.end()) return false;
    out = it->second;
    return true;
}

static int selected_mode(const uint8_t* idx, uint32_t flags)
{
    if (flags & SR_IDX_GLOBAL) return kModeGlobal;
    if (flags & SR_COEF_COMPACT) return kModeCompact;
    return idx ? kModeIdx : kModeFusedSelect;
}

struct RegressArgs {
    int mode;
    const float* lr;
    const void* coef;
    int coef_dtype;
    const uint8_t* idx;
    const float* gamma;
    const float* dict;
    float* out;
    Problem pb;
    cudaStream_t st;
};

static bool kernel_supported(int kernel, const RegressArgs& a)
{
    const bool idx_vec_ok = !a.idx || a.mode == kModeGlobal || ((reinterpret_cast<uintptr_t>(a.idx) & 15) == 0);   // 16-byte reads
    if ((a.pb.flags & SR_LUMA_ONLY) && kernel != kKernelGeneral) return false;   // only the general kernel has the luma variant
    switch (kernel) {
    case kKernelSubset: return regress_subset_supported(a.mode, a.coef, a.coef_dtype, a.out, a.pb);
    case kKernelListed: return regress_listed_supported(a.mode, a.coef, a.coef_dtype, a.idx, a.out, a.pb);
    case kKernelSecondLayout: return regress_tc_supported(a.mode, a.coef, a.coef_dtype, a.pb);
    case kKernelFirstLayout: return idx_vec_ok && umma_supported(a.mode, a.coef, a.coef_dtype, a.pb);
    default: return true;
    }
}

// The host rules: small global subsets on the FMA-pipe subset kernel; per-pixel lists with their values on the gather
// kernel; the second tensor-core layout for the other
// global subsets and for dense launches with few atoms; the first layout for the rest it supports; else the general kernel.
static int default_kernel(const RegressArgs& a)
{
    const int forced = g_force_kernel.load(std::memory_order_relaxed);
    if (forced >= 0 && kernel_supported(forced, a)) return forced;
    if (kernel_supported(kKernelSubset, a)) return kKernelSubset;
    const bool first = kernel_supported(kKernelFirstLayout, a), second = kernel_supported(kKernelSecondLayout, a);
    if (kernel_supported(kKernelListed, a) && (!first || compact_prefers_listed(a.pb))) return kKernelListed;
    if (second && (a.mode == kModeGlobal || dense_prefers_second_layout(a.pb) || !first)) return kKernelSecondLayout;
    if (first) return kKernelFirstLayout;
    return kKernelGeneral;
}

static cudaError_t run_kernel(const TuneChoice& c, const RegressArgs& a)
{
    switch (c.kernel) {
    case kKernelSubset: return launch_regress_subset(a.lr, a.coef, a.idx, a.gamma, a.dict, a.out, a.pb, a.st, c.sub_th);
    case kKernelListed: return launch_regress_listed(a.lr, a.coef, a.idx, a.dict, a.out, a.pb, a.st, c.sub_th);
    case kKernelSecondLayout: return launch_regress_tc(a.mode, a.lr, a.coef, a.idx, a.gamma, a.dict, a.out, a.pb, a.st, c.tc);
    case kKernelFirstLayout: return launch_regress_umma(a.mode, a.lr, a.coef, a.idx, a.gamma, a.dict, a.out, a.pb, a.st);
    default: return launch_regress_fma(a.mode, a.lr, a.coef, a.coef_dtype, a.idx, a.gamma, a.dict, a.out, a.pb, a.st);
    }
}

static cudaError_t run_regress(const RegressArgs& a);

// SR_LUMA_ONLY with fp32 output: the one-channel regression of the frame's luma by the ordinary kernels, then the chroma
// put back (sr_luma.cu). Planes 0 and 1 of the frame's own output serve as scratch.
static cudaError_t run_regress_luma(const RegressArgs& a)
{
    const Problem& pb = a.pb;
    const int64_t HW = (int64_t)pb.H * pb.W, hw = (int64_t)pb.h * pb.w;
    const bool compact = a.mode == kModeCompact || (a.mode == kModeGlobal && (pb.flags & SR_COEF_COMPACT));
    const int64_t coef_frame = (int64_t)(compact ? pb.s : pb.D) * HW * (a.coef_dtype == SR_F16 ? 2 : 4);
    const bool idx_planes = a.idx && a.mode != kModeGlobal;
    for (int f = 0; f < pb.n; ++f) {
        const float* lr_f = a.lr + (int64_t)f * 3 * hw;
        float* out_f = a.out + (int64_t)f * 3 * HW;
        float* ylr = out_f + HW;
        cudaError_t e = launch_luma_lr(lr_f, ylr, pb, a.st);
        if (e != cudaSuccess) return e;
        RegressArgs b = a;
        b.lr = ylr;
        b.out = out_f;
        b.coef = static_cast<const uint8_t*>(a.coef) + (int64_t)f * coef_frame;
        if (idx_planes) b.idx = a.idx + (int64_t)f * pb.s * HW;
        b.pb.n = 1;
        b.pb.c = 1;
        b.pb.flags &= ~(uint32_t)(SR_LUMA_ONLY | SR_CLAMP01);
        if ((e = run_regress(b)) != cudaSuccess) return e;
        if ((e = launch_luma_combine(lr_f, out_f, pb, a.st)) != cudaSuccess) return e;
    }
    return cudaSuccess;
}

static cudaError_t run_regress(const RegressArgs& a)
{
    if ((a.pb.flags & SR_LUMA_ONLY) && !(a.pb.flags & (SR_OUT_F16 | SR_OUT_U8))) return run_regress_luma(a);
    TuneChoice c;
    if (tune_lookup(tune_key(a.mode, a.coef_dtype, a.pb), c) && kernel_supported(c.kernel, a)) return run_kernel(c, a);
    c = TuneChoice{};
    c.kernel = default_kernel(a);
    return run_kernel(c, a);
}

// Times `reps` launches of one candidate after one warm-up launch; microseconds per launch, negative on error.
static float time_candidate(const TuneChoice& c, const RegressArgs& a, int reps, cudaEvent_t e0, cudaEvent_t e1)
{
    if (run_kernel(c, a) != cudaSuccess) return -1.f;
    if (cudaEventRecord(e0, a.st) != cudaSuccess) return -1.f;
    for (int i = 0; i < reps; ++i)
        if (run_kernel(c, a) != cudaSuccess) return -1.f;
    if (cudaEventRecord(e1, a.st) != cudaSuccess || cudaEventSynchronize(e1) != cudaSuccess) return -1.f;
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess) return -1.f;
    return ms * 1e3f / (float)reps;
}

static int tune_shape(const RegressArgs& a, int reps, sr_tune_result* res)
{
    if (reps < 1) reps = 1;
    std::vector<TuneChoice> cands;
    if (kernel_supported(kKernelFirstLayout, a)) { TuneChoice c; c.kernel = kKernelFirstLayout; cands.push_back(c); }
    if (kernel_supported(kKernelSecondLayout, a)) {
        TcTuning shapes[64];
        const int n = regress_tc_candidates(a.mode, a.pb, shapes, 64);
        for (int i = 0; i < n; ++i) { TuneChoice c; c.kernel = kKernelSecondLayout; c.tc = shapes[i]; cands.push_back(c); }
    }
    if (kernel_supported(kKernelSubset, a)) {
        int ths[8];
        const int n = regress_subset_candidates(a.pb, ths, 8);
        for (int i = 0; i < n; ++i) { TuneChoice c; c.kernel = kKernelSubset; c.sub_th = ths[i]; cands.push_back(c); }
    }
    if (kernel_supported(kKernelListed, a)) {
        int ths[8];
        const int n = regress_listed_candidates(a.pb, ths, 8);
        for (int i = 0; i < n; ++i) { TuneChoice c; c.kernel = kKernelListed; c.sub_th = ths[i]; cands.push_back(c); }
    }
    if (cands.empty()) { TuneChoice c; c.kernel = kKernelGeneral; cands.push_back(c); }
    cudaEvent_t e0, e1;
    if (cudaEventCreate(&e0) != cudaSuccess) return SR_ERR_CUDA;
    if (cudaEventCreate(&e1) != cudaSuccess) { cudaEventDestroy(e0); return SR_ERR_CUDA; }
    TuneChoice def;
    def.kernel = default_kernel(a);
    const float def_us = time_candidate(def, a, reps, e0, e1);
    int best = -1;
    float best_us = 0.f;
    for (size_t i = 0; i < cands.size(); ++i) {
        const float us = time_candidate(cands[i], a, reps, e0, e1);
        if (us > 0.f && (best < 0 || us < best_us)) { best = (int)i; best_us = us; }
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (best < 0 || def_us < 0.f) return SR_ERR_CUDA;
    TuneChoice pick = cands[best];
    if (def_us <= best_us) { pick = def; best_us = def_us; }        // the host rules' own choice stays unless something beat it
    {
        std::lock_guard<std::mutex> lock(g_tune_mu);
        g_tune_table[tune_key(a.mode, a.coef_dtype, a.pb)] = pick;
    }
    if (res) {
        res->kernel = pick.kernel;
        res->tile_rows = pick.kernel == kKernelSecondLayout ? pick.tc.th : ((pick.kernel == kKernelSubset || pick.kernel == kKernelListed) ? pick.sub_th : 0);
        res->rows_per_step = pick.kernel == kKernelSecondLayout ? pick.tc.group : 0;
        res->candidates = (int32_t)cands.size();
        res->best_us = best_us;
        res->default_us = def_us;
    }
    return SR_OK;
}

} // namespace sr

using namespace sr;

extern "C" {

static int upsample_alone(const float* lr, float* hr, const sr_dims* d, uint32_t flags, void* stream)
{
    if (!lr || !hr || !d) return SR_ERR_NULL;
    if (int e = check_dims(d, false)) return e;
    if (!aligned(lr, 4) || !aligned(hr, 4)) return SR_ERR_ALIGN;
    sr_dims dd = *d;
    dd.k = 1; dd.D = 1;
    const Problem pb = make_problem(&dd, 1, flags);
    return launch_bicubic(lr, hr, pb, (cudaStream_t)stream) == cudaSuccess ? SR_OK : SR_ERR_CUDA;
}

int sr_bicubic_upsample(const float* lr, float* hr, const sr_dims* d, void* stream)
{
    return upsample_alone(lr, hr, d, 0u, stream);
}

int sr_bilinear_upsample(const float* lr, float* hr, const sr_dims* d, void* stream)
{
    return upsample_alone(lr, hr, d, SR_UPSAMPLE_BILINEAR, stream);
}

int sr_dict_regress_dense(const float* lr, const void* coef, int coef_dtype, const float* dict, float* out,
                          const sr_dims* d, uint32_t flags, void* stream)
{
    if (!lr || !coef || !dict || !out || !d) return SR_ERR_NULL;
    if (int e = check_dims(d, true)) return e;
    if (coef_dtype != SR_F32 && coef_dtype != SR_F16) return SR_ERR_UNSUPPORTED;
    if (flags & ~(uint32_t)(SR_CLAMP01 | SR_UPSAMPLE_BILINEAR | SR_OUT_F16 | SR_OUT_U8 | SR_LUMA_ONLY) || bad_out_flags(flags, d)) return SR_ERR_UNSUPPORTED;
    if (!aligned(lr, 4) || !aligned(out, out_align(flags)) || !aligned(dict, 4) || !aligned(coef, coef_dtype == SR_F16 ? 2 : 4))
        return SR_ERR_ALIGN;
    const RegressArgs a{kModeDense, lr, coef, coef_dtype, nullptr, nullptr, dict, out, make_problem(d, d->D, flags), (cudaStream_t)stream};
    return run_regress(a) == cudaSuccess ? SR_OK : SR_ERR_CUDA;
}

int sr_tune_dense(const float* lr, const void* coef, int coef_dtype, const float* dict, float* out, const sr_dims* d,
                  uint32_t flags, int reps, void* stream, sr_tune_result* result)
{
    if (!lr || !coef || !dict || !out || !d) return SR_ERR_NULL;
    if (int e = check_dims(d, true)) return e;
    if (coef_dtype != SR_F32 && coef_dtype != SR_F16) return SR_ERR_UNSUPPORTED;
    if (flags & ~(uint32_t)(SR_CLAMP01 | SR_UPSAMPLE_BILINEAR | SR_OUT_F16 | SR_OUT_U8 | SR_LUMA_ONLY) || bad_out_flags(flags, d)) return SR_ERR_UNSUPPORTED;
    if (!aligned(lr, 4) || !aligned(out, out_align(flags)) || !aligned(dict, 4) || !aligned(coef, coef_dtype == SR_F16 ? 2 : 4))
        return SR_ERR_ALIGN;
    const RegressArgs a{kModeDense, lr, coef, coef_dtype, nullptr, nullptr, dict, out, make_problem(d, d->D, flags), (cudaStream_t)stream};
    return tune_shape(a, reps, result);
}

int sr_dict_select(const void* coef, int coef_dtype, uint8_t* idx, void* sel, const sr_dims* d, int s, uint32_t flags,
                   void* stream)
{
    if (!coef || !idx || !d) return SR_ERR_NULL;
    sr_dims dd = *d;
    dd.c = 1; dd.k = 1;
    if (int e = check_dims(&dd, true)) return e;
    if (coef_dtype != SR_F32 && coef_dtype != SR_F16) return SR_ERR_UNSUPPORTED;
    if (flags != 0) return SR_ERR_UNSUPPORTED;
    if (s < 1 || s > d->D) return SR_ERR_SHAPE;
    const size_t esz = coef_dtype == SR_F16 ? 2 : 4;
    if (!aligned(coef, esz) || (sel && !aligned(sel, esz))) return SR_ERR_ALIGN;
    const Problem pb = make_problem(&dd, s, 0);
    return launch_select(coef, coef_dtype, idx, sel, pb, (cudaStream_t)stream) == cudaSuccess ? SR_OK : SR_ERR_CUDA;
}

int sr_dict_regress_selected(const float* lr, const void* coef_or_sel, int coef_dtype, const uint8_t* idx,
                             const float* gamma, const float* dict, float* out, const sr_dims* d, int s,
                             uint32_t flags, void* stream)
{
    if (!lr || !coef_or_sel || !dict || !out || !d) return SR_ERR_NULL;
    if (int e = check_dims(d, true)) return e;
    if (coef_dtype != SR_F32 && coef_dtype != SR_F16) return SR_ERR_UNSUPPORTED;
    if (flags & ~(uint32_t)(SR_CLAMP01 | SR_IDX_GLOBAL | SR_COEF_COMPACT | SR_UPSAMPLE_BILINEAR | SR_OUT_F16 | SR_OUT_U8 | SR_LUMA_ONLY) || bad_out_flags(flags, d)) return SR_ERR_UNSUPPORTED;
    if (s < 1 || s > d->D) return SR_ERR_SHAPE;
    if ((flags & (SR_IDX_GLOBAL | SR_COEF_COMPACT)) && !idx) return SR_ERR_NULL;
    if (gamma && !(flags & SR_IDX_GLOBAL)) return SR_ERR_UNSUPPORTED;
    if (!aligned(lr, 4) || !aligned(out, out_align(flags)) || !aligned(dict, 4) || (gamma && !aligned(gamma, 4)) ||
        !aligned(coef_or_sel, coef_dtype == SR_F16 ? 2 : 4))
        return SR_ERR_ALIGN;
    const RegressArgs a{selected_mode(idx, flags), lr, coef_or_sel, coef_dtype, idx, gamma, dict, out, make_problem(d, s, flags), (cudaStream_t)stream};
    return run_regress(a) == cudaSuccess ? SR_OK : SR_ERR_CUDA;
}

int sr_tune_selected(const float* lr, const void* coef_or_sel, int coef_dtype, const uint8_t* idx, const float* gamma,
                     const float* dict, float* out, const sr_dims* d, int s, uint32_t flags, int reps, void* stream,
                     sr_tune_result* result)
{
    if (!lr || !coef_or_sel || !dict || !out || !d) return SR_ERR_NULL;
    if (int e = check_dims(d, true)) return e;
    if (coef_dtype != SR_F32 && coef_dtype != SR_F16) return SR_ERR_UNSUPPORTED;
    if (flags & ~(uint32_t)(SR_CLAMP01 | SR_IDX_GLOBAL | SR_COEF_COMPACT | SR_UPSAMPLE_BILINEAR | SR_OUT_F16 | SR_OUT_U8 | SR_LUMA_ONLY) || bad_out_flags(flags, d)) return SR_ERR_UNSUPPORTED;
    if (s < 1 || s > d->D) return SR_ERR_SHAPE;
    if ((flags & (SR_IDX_GLOBAL | SR_COEF_COMPACT)) && !idx) return SR_ERR_NULL;
    if (gamma && !(flags & SR_IDX_GLOBAL)) return SR_ERR_UNSUPPORTED;
    if (!aligned(lr, 4) || !aligned(out, out_align(flags)) || !aligned(dict, 4) || (gamma && !aligned(gamma, 4)) ||
        !aligned(coef_or_sel, coef_dtype == SR_F16 ? 2 : 4))
        return SR_ERR_ALIGN;
    const RegressArgs a{selected_mode(idx, flags), lr, coef_or_sel, coef_dtype, idx, gamma, dict, out, make_problem(d, s, flags), (cudaStream_t)stream};
    return tune_shape(a, reps, result);
}

void sr_tune_reset(void)
{
    std::lock_guard<std::mutex> lock(g_tune_mu);
    g_tune_table.clear();
}

size_t sr_selection_gram_scratch_bytes(const sr_dims* d)
{
    if (!d || d->D < 1 || d->D > 128) return 0;
    return (size_t)selection_gram_slots() * selection_gram_slot_bytes(d->D);
}

int sr_selection_gram(const float* lr, const void* coef, int coef_dtype, const float* dict, const float* target,
                      const int64_t* samples, int64_t nsamples, double* G, double* b, double* hh, const sr_dims* d,
                      uint32_t flags, void* scratch, size_t scratch_bytes, void* stream)
{
    if (!lr || !coef || !dict || !target || !G || !b || !hh || !d || !scratch) return SR_ERR_NULL;
    if (int e = check_dims(d, true)) return e;
    if (d->D > 128 || d->c > 16) return SR_ERR_UNSUPPORTED;
    if (coef_dtype != SR_F32 && coef_dtype != SR_F16) return SR_ERR_UNSUPPORTED;
    if (flags & ~(uint32_t)SR_UPSAMPLE_BILINEAR) return SR_ERR_UNSUPPORTED;
    if (samples && nsamples < 1) return SR_ERR_SHAPE;
    if (!aligned(lr, 4) || !aligned(dict, 4) || !aligned(target, 4) || !aligned(coef, coef_dtype == SR_F16 ? 2 : 4) ||
        !aligned(G, 8) || !aligned(b, 8) || !aligned(hh, 8) || !aligned(scratch, 8) || (samples && !aligned(samples, 8)))
        return SR_ERR_ALIGN;
    const size_t slot = selection_gram_slot_bytes(d->D);
    int nslots = selection_gram_slots();
    if (scratch_bytes < slot) return SR_ERR_SHAPE;
    if (scratch_bytes / slot < (size_t)nslots) nslots = (int)(scratch_bytes / slot);
    const Problem pb = make_problem(d, d->D, flags);
    return launch_selection_gram(lr, coef, coef_dtype, dict, target, samples, nsamples, G, b, hh, pb, static_cast<double*>(scratch),
                                 nslots, (cudaStream_t)stream) == cudaSuccess ? SR_OK : SR_ERR_CUDA;
}

int sr_selection_gram_static(const float* lr, const void* coef, int coef_dtype, const float* dict, const float* target,
                             const int64_t* samples, int64_t nsamples, double* G, double* b, double* hh, const sr_dims* d,
                             uint32_t flags, void* stream)
{
    if (!lr || !coef || !dict || !target || !G || !b || !hh || !d) return SR_ERR_NULL;
    if (int e = check_dims(d, true)) return e;
    if (d->D > selection_gram_static_max_atoms()) return SR_ERR_TOO_LARGE;       // beyond the built-in scratch
    if (d->c > 16) return SR_ERR_UNSUPPORTED;
    if (coef_dtype != SR_F32 && coef_dtype != SR_F16) return SR_ERR_UNSUPPORTED;
    if (flags & ~(uint32_t)SR_UPSAMPLE_BILINEAR) return SR_ERR_UNSUPPORTED;
    if (samples && nsamples < 1) return SR_ERR_SHAPE;
    if (!aligned(lr, 4) || !aligned(dict, 4) || !aligned(target, 4) || !aligned(coef, coef_dtype == SR_F16 ? 2 : 4) ||
        !aligned(G, 8) || !aligned(b, 8) || !aligned(hh, 8) || (samples && !aligned(samples, 8)))
        return SR_ERR_ALIGN;
    const Problem pb = make_problem(d, d->D, flags);
    return launch_selection_gram_static(lr, coef, coef_dtype, dict, target, samples, nsamples, G, b, hh, pb,
                                        (cudaStream_t)stream) == cudaSuccess ? SR_OK : SR_ERR_CUDA;
}

size_t sr_selection_search_scratch_bytes(int32_t D) { return (D < 1 || D > 128) ? 0 : selection_search_scratch_bytes(D); }

int sr_selection_search(const double* G, const double* b, const double* hh, double nrows, int32_t D,
                        const sr_search_opts* o, uint8_t* idx_out, float* gamma_out, int32_t* count_out, double* trace,
                        int32_t* steps_out, void* scratch, size_t scratch_bytes, void* stream)
{
    if (!G || !b || !hh || !o || !idx_out || !gamma_out || !count_out || !scratch) return SR_ERR_NULL;
    if (D < 1 || !(nrows > 0.0)) return SR_ERR_SHAPE;
    if (D > 128) return SR_ERR_UNSUPPORTED;
    if (!(o->alpha > 0.0) || !(o->alpha <= 1.0) || !(o->delta_alpha > 0.0) || !(o->lambda0 > 0.0) || !(o->eps >= 0.0) ||
        !(o->tol >= 0.0) || o->max_sweeps < 1 || o->max_bisect < 0 || o->max_steps < 1)
        return SR_ERR_SHAPE;
    if (!aligned(G, 8) || !aligned(b, 8) || !aligned(hh, 8) || !aligned(scratch, 8) || !aligned(gamma_out, 4) ||
        !aligned(count_out, 4) || (trace && !aligned(trace, 8)) || (steps_out && !aligned(steps_out, 4)))
        return SR_ERR_ALIGN;
    if (scratch_bytes < selection_search_scratch_bytes(D)) return SR_ERR_SHAPE;
    return launch_selection_search(G, b, hh, nrows, D, *o, idx_out, gamma_out, count_out, trace, steps_out,
                                   static_cast<double*>(scratch), (cudaStream_t)stream) == cudaSuccess ? SR_OK : SR_ERR_CUDA;
}

const char* sr_status_string(int status)
{
    switch (status) {
    case SR_OK: return "ok";
    case SR_ERR_NULL: return "a required pointer is NULL";
    case SR_ERR_SHAPE: return "a size is out of range";
    case SR_ERR_UNSUPPORTED: return "unsupported scale, atom size, atom count, dtype or flag";
    case SR_ERR_ALIGN: return "a pointer is misaligned";
    case SR_ERR_CUDA: return "a CUDA call or kernel launch failed";
    case SR_ERR_TIMEOUT: return "a bounded device-side wait expired";
    case SR_ERR_TOO_LARGE: return "the problem is larger than the library's built-in scratch memory";
    default: return "unknown status";
    }
}

int64_t sr_launch_count(void) { return (int64_t)g_launches.load(std::memory_order_relaxed); }

size_t sr_producer_folded_bytes(const sr_dims* d, int cin, int kc)
{
    if (!d || check_dims(d, true) != SR_OK) return 0;
    return producer_folded_bytes(make_problem(d, d->D, 0u), ProducerShape{cin, kc});
}

int sr_producer_fold(const float* wconv, const float* bias, const float* dict, const uint8_t* idx, const float* gamma,
                     int s, void* folded, size_t folded_bytes, const sr_dims* d, int cin, int kc, void* stream)
{
    if (!wconv || !dict || !folded || !d) return SR_ERR_NULL;
    if (int e = check_dims(d, true)) return e;
    if (gamma && !idx) return SR_ERR_UNSUPPORTED;
    if (idx && (s < 1 || s > d->D)) return SR_ERR_SHAPE;
    const Problem pb = make_problem(d, d->D, 0u);
    const ProducerShape ps{cin, kc};
    if (!producer_supported(pb, ps)) return SR_ERR_UNSUPPORTED;
    if (folded_bytes < producer_folded_bytes(pb, ps)) return SR_ERR_SHAPE;
    if (!aligned(wconv, 4) || !aligned(dict, 4) || (bias && !aligned(bias, 4)) || (gamma && !aligned(gamma, 4)) || !aligned(folded, 16))
        return SR_ERR_ALIGN;
    return launch_producer_fold(wconv, bias, dict, idx, gamma, s, folded, pb, ps, (cudaStream_t)stream) == cudaSuccess ? SR_OK : SR_ERR_CUDA;
}

int sr_producer_regress(const float* lr, const void* feat, const void* folded, size_t folded_bytes, float* out,
                        const sr_dims* d, int cin, int kc, uint32_t flags, void* stream)
{
    if (!lr || !feat || !folded || !out || !d) return SR_ERR_NULL;
    if (int e = check_dims(d, true)) return e;
    if (flags & ~(uint32_t)(SR_CLAMP01 | SR_UPSAMPLE_BILINEAR | SR_OUT_F16 | SR_OUT_U8) || bad_out_flags(flags, d)) return SR_ERR_UNSUPPORTED;
    const Problem pb = make_problem(d, d->D, flags);
    const ProducerShape ps{cin, kc};
    if (!producer_supported(pb, ps)) return SR_ERR_UNSUPPORTED;
    if (folded_bytes < producer_folded_bytes(pb, ps)) return SR_ERR_SHAPE;
    if (!aligned(lr, 4) || !aligned(feat, 16) || !aligned(folded, 16) || !aligned(out, 16)) return SR_ERR_ALIGN;
    return launch_producer_regress(lr, feat, folded, out, pb, ps, (cudaStream_t)stream) == cudaSuccess ? SR_OK : SR_ERR_CUDA;
}

int sr_probe_rate(int kind, void* scratch8, double* lane_ops_per_s, void* stream)
{
    if (!scratch8 || !lane_ops_per_s) return SR_ERR_NULL;
    if (kind < 0 || kind > 2) return SR_ERR_UNSUPPORTED;
    if (!aligned(scratch8, 4)) return SR_ERR_ALIGN;
    return probe_rate(kind, static_cast<int*>(scratch8), lane_ops_per_s, (cudaStream_t)stream) == cudaSuccess ? SR_OK : SR_ERR_CUDA;
}

int64_t sr_set_wait_limit(int64_t cycles)
{
    if (cycles < 1) return (int64_t)g_wait_limit.load(std::memory_order_relaxed);
    return (int64_t)g_wait_limit.exchange((long long)cycles, std::memory_order_relaxed);
}

int sr_test_lose_arrival(int launches)
{
    if (launches < 0) return SR_ERR_SHAPE;
    g_lose_arrival.store(launches, std::memory_order_relaxed);
    return SR_OK;
}

int sr_test_force_kernel(int kernel)
{
    if (kernel < -1 || kernel > kKernelListed) return SR_ERR_SHAPE;
    g_force_kernel.store(kernel, std::memory_order_relaxed);
    return SR_OK;
}

int sr_device_status(void* stream, int* out_status)
{
    if (!out_status) return SR_ERR_NULL;
    int* word = device_status_word();
    if (!word) return SR_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    int v = 0;
    if (cudaMemcpyAsync(&v, word, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return SR_ERR_CUDA;
    if (cudaMemsetAsync(word, 0, sizeof(int), st) != cudaSuccess) return SR_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return SR_ERR_CUDA;
    *out_status = v;
    return SR_OK;
}

} // extern "C"
