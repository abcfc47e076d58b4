// C ABI entry points: argument validation, path selection, status reporting.
#include <math.h>

#include <atomic>

#include "sr_common.cuh"
#include "sr_regress_subset.cuh"
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

// Which tensor-core layout takes a dense launch. The second layout (sr_regress_tc.cu: channel-split epilogue, two CTAs
// per SM, several rows per pipeline step) wins where the coefficient stream is light and the epilogue sets the pace:
// few atoms, or 7 x 7 atoms with up to 32 of them; the first layout (sr_umma.cu) streams many atoms faster. Measured
// on the 1080p sweep points (dense, D = 16 / 32 / 72 / 128; k = 3 / 5 / 7).
static bool dense_prefers_second_layout(const Problem& pb) { return pb.D <= 16 || (pb.k == 7 && pb.D <= 32); }

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
    if (flags & ~(uint32_t)(SR_CLAMP01 | SR_UPSAMPLE_BILINEAR | SR_OUT_F16)) return SR_ERR_UNSUPPORTED;
    if (!aligned(lr, 4) || !aligned(out, (flags & SR_OUT_F16) ? 2 : 4) || !aligned(dict, 4) || !aligned(coef, coef_dtype == SR_F16 ? 2 : 4))
        return SR_ERR_ALIGN;
    const Problem pb = make_problem(d, d->D, flags);
    cudaError_t err;
    const bool first_ok = umma_supported(kModeDense, coef, coef_dtype, pb);
    if (regress_tc_supported(kModeDense, coef, coef_dtype, pb) && (dense_prefers_second_layout(pb) || !first_ok))
        err = launch_regress_tc(kModeDense, lr, coef, nullptr, nullptr, dict, out, pb, (cudaStream_t)stream);
    else if (first_ok)
        err = launch_regress_umma(kModeDense, lr, coef, nullptr, nullptr, dict, out, pb, (cudaStream_t)stream);
    else
        err = launch_regress_fma(kModeDense, lr, coef, coef_dtype, nullptr, nullptr, dict, out, pb, (cudaStream_t)stream);
    return err == cudaSuccess ? SR_OK : SR_ERR_CUDA;
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
    if (flags & ~(uint32_t)(SR_CLAMP01 | SR_IDX_GLOBAL | SR_COEF_COMPACT | SR_UPSAMPLE_BILINEAR | SR_OUT_F16)) return SR_ERR_UNSUPPORTED;
    if (s < 1 || s > d->D) return SR_ERR_SHAPE;
    if ((flags & (SR_IDX_GLOBAL | SR_COEF_COMPACT)) && !idx) return SR_ERR_NULL;
    if (gamma && !(flags & SR_IDX_GLOBAL)) return SR_ERR_UNSUPPORTED;
    if (!aligned(lr, 4) || !aligned(out, (flags & SR_OUT_F16) ? 2 : 4) || !aligned(dict, 4) || (gamma && !aligned(gamma, 4)) ||
        !aligned(coef_or_sel, coef_dtype == SR_F16 ? 2 : 4))
        return SR_ERR_ALIGN;
    const Problem pb = make_problem(d, s, flags);
    int mode;
    if (flags & SR_IDX_GLOBAL) mode = kModeGlobal;
    else if (flags & SR_COEF_COMPACT) mode = kModeCompact;
    else mode = idx ? kModeIdx : kModeFusedSelect;
    cudaError_t err;
    const bool idx_vec_ok = !idx || (flags & SR_IDX_GLOBAL) || ((reinterpret_cast<uintptr_t>(idx) & 15) == 0);   // 16-byte reads
    if (regress_subset_supported(mode, coef_or_sel, coef_dtype, out, pb))
        err = launch_regress_subset(lr, coef_or_sel, idx, gamma, dict, out, pb, (cudaStream_t)stream);
    else if (regress_tc_supported(mode, coef_or_sel, coef_dtype, pb))
        err = launch_regress_tc(mode, lr, coef_or_sel, idx, gamma, dict, out, pb, (cudaStream_t)stream);
    else if (idx_vec_ok && umma_supported(mode, coef_or_sel, coef_dtype, pb))
        err = launch_regress_umma(mode, lr, coef_or_sel, idx, gamma, dict, out, pb, (cudaStream_t)stream);
    else
        err = launch_regress_fma(mode, lr, coef_or_sel, coef_dtype, idx, gamma, dict, out, pb, (cudaStream_t)stream);
    return err == cudaSuccess ? SR_OK : SR_ERR_CUDA;
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
