// Regression from per-pixel lists on the fp32 FMA pipe (Section III-A: each pixel keeps only its s selected atoms;
// the call receives their indices and values as planes [n][s][H][W]):
//   out[c][i] = sum_j (sum_{q<s} val[q][i] dict[idx[q][i]][j]) B_{i,c}[j]
// With s of D atoms kept, the assembly F_i = Phi_i D has s k^2 useful multiply-adds per pixel, and a tensor-core tile
// would first have to scatter the lists back into dense rows of D coefficients. This kernel gathers instead: a thread
// owns two neighbouring pixels, reads their lists straight from global memory, fetches each listed atom's k^2 taps from
// a dictionary in shared memory and accumulates the filter in registers (packed fp32 multiply-adds), then applies it
// to the up-sampled tile. F and U never leave the SM.
//
// The gather sets the pace: every lane of a warp wants a different dictionary row, 16 bytes at a time. The dictionary
// is therefore stored eight times, copy p in the 16-byte bank group p of every 128-byte line, and lane l reads copy
// l % 8: the eight lanes that share a shared-memory cycle always hit eight different bank groups, whatever atoms they
// ask for. k^2 is odd: the last tap of every atom sits in a table of its own with one copy per lane (4-byte loads, lane
// l reads bank l), so that no 16-byte gather is spent on a single tap (D * (floor(k^2 / 4) + 1) * 128 bytes: 63 KB for
// 72 atoms of 5 x 5).
// Bound: shared-memory bandwidth of the gather (s * (floor(k^2 / 4) * 16 + 4) bytes per pixel), then the fp32 pipe.
//
// One CTA of 512 threads per SM; its two halves of 256 threads walk different tiles (128 x th pixels, th = 8, 16 or
// 24) with their own tile buffers and their own named barrier, so that one half builds its next up-sampled tile while
// the other filters, and both share the one replicated dictionary. In a half, a warp takes 64 pixels of a row.
#include "sr_regress_listed.cuh"
#include "sr_tile_upsample.cuh"

namespace sr {

namespace {

using namespace tile;

constexpr int kThreads = 512;
constexpr int kHalfThreads = 256;
constexpr int kRowsPerPass = 4;   // a half's eight warps: four rows x two 64-pixel halves of a row

struct ListedParams {
    const float* lr;
    const float* dict;
    void* out;
    const uint8_t* idx;   // [n][s][H][W]
    const __half* val;    // [n][s][H][W]
    Geom g;
    int natoms;           // s
    int half_floats;      // floats of one half's tile buffers (a multiple of 4)
};

__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
__device__ __forceinline__ void bar_sync(int id, int nthreads) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory"); }
__device__ __forceinline__ void prefetch_l2(const void* p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }
__device__ __forceinline__ uint32_t ldg_u16(const uint8_t* p)
{
    uint16_t v;
    asm volatile("ld.global.nc.u16 %0, [%1];" : "=h"(v) : "l"(p));
    return v;
}
__device__ __forceinline__ uint32_t ldg_u32(const void* p)
{
    uint32_t v;
    asm volatile("ld.global.nc.u32 %0, [%1];" : "=r"(v) : "l"(p));
    return v;
}

template <typename OutT> __device__ __forceinline__ void store_pair(OutT* o, float a, float b);
template <> __device__ __forceinline__ void store_pair<float>(float* o, float a, float b) { *reinterpret_cast<float2*>(o) = make_float2(a, b); }
template <> __device__ __forceinline__ void store_pair<__half>(__half* o, float a, float b) { *reinterpret_cast<__half2*>(o) = __floats2half2_rn(a, b); }
template <> __device__ __forceinline__ void store_pair<uint8_t>(uint8_t* o, float a, float b)
{
    *reinterpret_cast<uchar2*>(o) = make_uchar2(to_out<uint8_t>(a), to_out<uint8_t>(b));
}

template <int K, int C, typename OutT>
__global__ void __launch_bounds__(kThreads, 1) regress_listed_kernel(const __grid_constant__ ListedParams p)
{
    constexpr int kk = K * K, P = (K - 1) / 2, UW = tile_uw(P), UW4 = UW / 4;
    constexpr int NU = kk / 4;                    // 16-byte units of a dictionary row: taps 0 .. 4 NU - 1; tap kk - 1 apart
    static_assert(kk == 4 * NU + 1, "k^2 = 1 (mod 4) for odd k");
    constexpr int EP = K <= 5 ? 2 : 1;            // pixels whose filters are held at once (register budget)
    constexpr int NL = (K + 2) / 2;               // 8-byte loads that cover the K + 1 columns of a pixel pair's patches
    extern __shared__ __align__(16) float smem[];
    __shared__ float wpad[kMaxScale][12];

    const Geom& g = p.g;
    const Problem& pb = g.pb;
    const int tid = threadIdx.x, half = tid >> 8, ht = tid & (kHalfThreads - 1), warp = ht >> 5, lane = tid & 31;
    const int dict_units = pb.D * NU * 8;
    float4* sD = reinterpret_cast<float4*>(smem);                                      // [D][NU][8 copies]
    float* sT = smem + 4 * dict_units;                                                 // [D][32 copies]: last tap
    const int last_floats = 32 * pb.D;
    float* hb = sT + last_floats + half * p.half_floats;
    float* sU = hb;                                                                    // [C][uh][UW]
    float* sV = sU + C * g.uh * UW;                                                    // [C][uh][tcols]
    float* sL = sV + C * g.uh * g.tcols;                                               // [C * trows][tcols]

    // ---- set-up: tile buffers start as zeros (the up-sampling passes read a few values beyond the ones they weight)
    for (int i = tid; i < 2 * p.half_floats / 4; i += kThreads)
        reinterpret_cast<float4*>(sT + last_floats)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    fill_wpad(pb, wpad, tid, kThreads);
    for (int i = tid; i < dict_units; i += kThreads) {
        const int u = i >> 3, a = u / NU, j = u - a * NU;
        float v[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) v[e] = __ldg(p.dict + (int64_t)a * kk + 4 * j + e);
        sD[i] = make_float4(v[0], v[1], v[2], v[3]);
    }
    for (int i = tid; i < last_floats; i += kThreads) sT[i] = __ldg(p.dict + (int64_t)(i >> 5) * kk + kk - 1);
    __syncthreads();

    // this thread's part of the up-sampling passes of its half: a group of four columns and a row lane
    const int tc4 = g.tcols >> 2;
    const int v_lane = fast_div(ht, tc4, g.tc4_magic), v_i4 = (ht - v_lane * tc4) * 4, v_lanes = kHalfThreads / tc4;
    const int h_lane = ht / UW4, h_cg = ht - h_lane * UW4, h_lanes = kHalfThreads / UW4;
    const bool clamp01 = (pb.flags & SR_CLAMP01) != 0;
    const int64_t HW = (int64_t)pb.H * pb.W;
    const int bar_id = 1 + half;
    const int rsub = warp >> 1, pp = (warp & 1) * 32 + lane;      // row of a pass, pixel pair of the row
    const float4* my_dict = sD + (lane & 7);
    const float* my_last = sT + lane;

    // lists of the 64 pixels this warp filters in row y of frame f: one 64-byte piece per index plane and one 128-byte
    // line per value plane, asked into L2 a row of work ahead
    auto prefetch_lists = [&](int f, int y, int x64) {
        if (y < pb.H && x64 < pb.W) {
            const int64_t off = (int64_t)f * p.natoms * HW + (int64_t)y * pb.W + x64;
            if (lane < p.natoms) prefetch_l2(p.idx + off + lane * HW);
            else if (lane >= 16 && lane - 16 < p.natoms) prefetch_l2(p.val + off + (lane - 16) * HW);
        }
    };

    // A half's share of the image is a run of 8-row groups (the same number for every half to within one), cut into
    // tiles of up to th rows.
    const int run_end = run_bound(g, 2 * blockIdx.x + half + 1, 2 * gridDim.x);
    int run_cur = run_bound(g, 2 * blockIdx.x + half, 2 * gridDim.x);
    {
        int peek = run_cur;
        LrWindow w0;
        if (next_tile_of_run(g, peek, run_end, w0.f, w0.y0, w0.x0, w0.rows)) {
            lr_window_of_tile<P>(g, w0);
            prefetch_lr_window_of(g, p.lr, w0, sL, ht, kHalfThreads);
        }
    }
    LrWindow w;
    while (next_tile_of_run(g, run_cur, run_end, w.f, w.y0, w.x0, w.rows)) {
        lr_window_of_tile<P>(g, w);
        const int uh = w.rows + 2 * P;
        prefetch_lists(w.f, w.y0 + rsub, w.x0 + 64 * (warp & 1));
        cp_async_wait_all();
        bar_sync(bar_id, kHalfThreads);                      // LR window landed; the previous tile's U is no longer read
        if (v_lane < v_lanes) vertical_pass(g, w, uh, P, sL, sV, v_i4, v_lane, v_lanes);
        bar_sync(bar_id, kHalfThreads);
        {
            int peek = run_cur;
            LrWindow wn;
            if (next_tile_of_run(g, peek, run_end, wn.f, wn.y0, wn.x0, wn.rows)) {
                lr_window_of_tile<P>(g, wn);
                prefetch_lr_window_of(g, p.lr, wn, sL, ht, kHalfThreads);
            }
        }
        if (h_lane < h_lanes) horizontal_pass<P>(g, wpad, w, uh, sV, sU, h_cg, h_lane, h_lanes);
        bar_sync(bar_id, kHalfThreads);                      // the U tile is complete

        const int px0 = w.x0 + 2 * pp;
        for (int row = rsub; row < w.rows; row += kRowsPerPass) {
            if (row + kRowsPerPass < w.rows) prefetch_lists(w.f, w.y0 + row + kRowsPerPass, w.x0 + 64 * (warp & 1));
            if (px0 >= pb.W) continue;                       // columns beyond the image (width not a multiple of 128)
            const int64_t pix = (int64_t)(w.y0 + row) * pb.W + px0;
            const uint8_t* irow = p.idx + (int64_t)w.f * p.natoms * HW + pix;
            const __half* vrow = p.val + (int64_t)w.f * p.natoms * HW + pix;
            float acc[C][2];
#pragma unroll
            for (int c = 0; c < C; ++c) acc[c][0] = acc[c][1] = 0.f;
#pragma unroll
            for (int e0 = 0; e0 < 2; e0 += EP) {
                // ---- the filters of pixels e0 .. e0 + EP - 1: F[e][j] = taps 2 j, 2 j + 1
                float2 F[EP][2 * NU];
                float Fl[EP];                                // the last tap
#pragma unroll
                for (int e = 0; e < EP; ++e)
#pragma unroll
                    for (int j = 0; j < 2 * NU; ++j) F[e][j] = make_float2(0.f, 0.f);
#pragma unroll
                for (int e = 0; e < EP; ++e) Fl[e] = 0.f;
                for (int q0 = 0; q0 < p.natoms; q0 += 8) {
                    uint32_t iw[8], vw[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        iw[j] = vw[j] = 0u;
                        if (q0 + j < p.natoms) {
                            iw[j] = ldg_u16(irow + (q0 + j) * HW);
                            vw[j] = ldg_u32(vrow + (q0 + j) * HW);
                        }
                    }
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        if (q0 + j < p.natoms) {
                            const float2 v2 = __half22float2(*reinterpret_cast<const __half2*>(&vw[j]));
#pragma unroll
                            for (int e = 0; e < EP; ++e) {
                                const int px = e0 + e;
                                const int a = min((int)((iw[j] >> (8 * px)) & 255u), pb.D - 1);
                                const float v = px == 0 ? v2.x : v2.y;
                                const float2 vv = make_float2(v, v);
                                const float4* dr = my_dict + a * (NU * 8);
#pragma unroll
                                for (int u = 0; u < NU; ++u) {
                                    const float4 d = dr[u * 8];
                                    F[e][2 * u] = __ffma2_rn(make_float2(d.x, d.y), vv, F[e][2 * u]);
                                    F[e][2 * u + 1] = __ffma2_rn(make_float2(d.z, d.w), vv, F[e][2 * u + 1]);
                                }
                                Fl[e] = fmaf(my_last[a * 32], v, Fl[e]);
                            }
                        }
                    }
                }
                // ---- applied to the up-sampled tile: pixel px, tap (a, b) reads row (row + a), column 2 pp + px + b
#pragma unroll
                for (int a = 0; a < K; ++a) {
                    // keeps the compiler from hoisting every row's loads above the arithmetic (7 x 7: 21 rows of eight
                    // values, which it then spills)
                    asm volatile("" ::: "memory");
#pragma unroll
                    for (int c = 0; c < C; ++c) {
                        const float2* up = reinterpret_cast<const float2*>(sU + (c * g.uh + row + a) * UW + 2 * pp);
                        float u[2 * NL];
#pragma unroll
                        for (int n = 0; n < NL; ++n) {
                            const float2 t2 = up[n];
                            u[2 * n] = t2.x;
                            u[2 * n + 1] = t2.y;
                        }
#pragma unroll
                        for (int e = 0; e < EP; ++e) {
                            const int px = e0 + e;
#pragma unroll
                            for (int b = 0; b < K; ++b) {
                                const int tap = a * K + b;
                                const float f = tap == kk - 1 ? Fl[e] : ((tap & 1) ? F[e][tap >> 1].y : F[e][tap >> 1].x);
                                acc[c][px] = fmaf(f, u[px + b], acc[c][px]);
                            }
                        }
                    }
                }
            }
            OutT* of = reinterpret_cast<OutT*>(p.out) + (int64_t)w.f * C * HW + pix;
#pragma unroll
            for (int c = 0; c < C; ++c) {
                float v0 = acc[c][0], v1 = acc[c][1];
                if (clamp01) {
                    v0 = fminf(fmaxf(v0, 0.f), 1.f);
                    v1 = fminf(fmaxf(v1, 0.f), 1.f);
                }
                store_pair<OutT>(of + c * HW, v0, v1);
            }
        }
    }
    cp_async_wait_all();
}

struct DeviceInfo { int sms = 0, cc_major = 0, smem_optin = 0; bool ok = false; };

const DeviceInfo& device_info()
{
    static DeviceInfo cache[64];
    static DeviceInfo none;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return none;
    DeviceInfo& d = cache[dev];
    if (!d.ok) {
        if (cudaDeviceGetAttribute(&d.sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return none;
        if (cudaDeviceGetAttribute(&d.cc_major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return none;
        if (cudaDeviceGetAttribute(&d.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) return none;
        d.ok = true;
    }
    return d;
}

constexpr int kStaticReserve = 1024;   // static shared memory (the padded tap table)

struct Plan { int th = 0; size_t smem = 0; int half_floats = 0; int ctas = 0; };

// Shared memory of the replicated dictionary plus two tile sets at tile height th; 0 when it does not fit.
size_t smem_for(const Problem& pb, int th, int& half_floats)
{
    Geom g;
    half_floats = (int)((plan_geom(g, pb, th, nullptr) + 8 + 3) & ~(size_t)3);
    const size_t dict = (size_t)pb.D * (pb.k * pb.k / 4 + 1) * 128;     // the 16-byte units, eight copies each, and the last taps
    const size_t need = dict + 2 * (size_t)half_floats * 4;
    const DeviceInfo& di = device_info();
    return di.ok && need + kStaticReserve <= (size_t)di.smem_optin ? need : 0;
}

// Tile height: every half gets the same run of 8-row groups (to within one) and cuts it into tiles of up to th rows; a
// run costs its rows (in passes of four) plus, per tile, an up-sampled tile of th + k - 1 rows. Units: row passes.
Plan choose_plan(const Problem& pb, int th_forced)
{
    Plan best;
    double best_cost = 0.0;
    const DeviceInfo& di = device_info();
    if (!di.ok) return best;
    for (int th = 24; th >= 8; th -= 8) {
        if (th_forced > 0 && th != th_forced) continue;
        int hf = 0;
        const size_t smem = smem_for(pb, th, hf);
        if (smem == 0) continue;
        Geom g;
        plan_geom(g, pb, th, nullptr);
        const long long groups = g.num_groups;
        const long long halves = groups < 2LL * di.sms ? groups : 2LL * di.sms;
        const long long per_half = (groups + halves - 1) / halves;               // 8-row groups in a half's run
        const long long tiles = (per_half * 8 + th - 1) / th;
        const double cost = (double)per_half * (8 / kRowsPerPass) + (double)tiles * 0.12 * g.uh;
        if (best.th == 0 || cost < best_cost) {
            best.th = th; best.smem = smem; best.half_floats = hf; best.ctas = (int)((halves + 1) / 2);
            best_cost = cost;
        }
    }
    return best;
}

template <int K, int C, typename OutT>
cudaError_t launch_t(const ListedParams& prm, const Plan& pl, cudaStream_t st)
{
    auto kern = regress_listed_kernel<K, C, OutT>;
    static bool configured[64] = {false};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, device_info().smem_optin - kStaticReserve);
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    kern<<<pl.ctas, kThreads, pl.smem, st>>>(prm);
    count_launches(1);
    return cudaGetLastError();
}

template <int K, int C>
cudaError_t launch_o(const ListedParams& prm, const Plan& pl, cudaStream_t st)
{
    if (prm.g.pb.flags & SR_OUT_U8) return launch_t<K, C, uint8_t>(prm, pl, st);
    if (prm.g.pb.flags & SR_OUT_F16) return launch_t<K, C, __half>(prm, pl, st);
    return launch_t<K, C, float>(prm, pl, st);
}

template <int K>
cudaError_t launch_c(const ListedParams& prm, const Plan& pl, cudaStream_t st)
{
    if (prm.g.pb.c == 3) return launch_o<K, 3>(prm, pl, st);
    if (prm.g.pb.c == 1) return launch_o<K, 1>(prm, pl, st);
    return cudaErrorNotSupported;
}

} // namespace

int regress_listed_candidates(const Problem& pb, int* ths, int max_out)
{
    int n = 0;
    for (int th = 24; th >= 8; th -= 8)
        if (choose_plan(pb, th).th == th && n < max_out) ths[n++] = th;
    return n;
}

bool regress_listed_supported(int mode, const void* coef, int coef_dtype, const uint8_t* idx, const void* out, const Problem& pb)
{
    if (mode != kModeCompact || coef_dtype != SR_F16 || pb.s < 1 || pb.s > 16 || pb.D > 256) return false;
    if ((pb.k != 3 && pb.k != 5 && pb.k != 7) || (pb.c != 1 && pb.c != 3) || (pb.W & 1) != 0) return false;
    // one load / store per pixel pair
    if ((reinterpret_cast<uintptr_t>(idx) & 1) != 0 || (reinterpret_cast<uintptr_t>(coef) & 3) != 0) return false;
    if ((reinterpret_cast<uintptr_t>(out) & ((pb.flags & SR_OUT_U8) ? 1 : ((pb.flags & SR_OUT_F16) ? 3 : 7))) != 0) return false;
    const DeviceInfo& di = device_info();
    if (!di.ok || di.cc_major < 9) return false;
    return choose_plan(pb, 0).th > 0;
}

cudaError_t launch_regress_listed(const float* lr, const void* val, const uint8_t* idx, const float* dict, float* out,
                                  const Problem& pb, cudaStream_t st, int th_forced)
{
    Plan pl = choose_plan(pb, th_forced);
    if (pl.th == 0) pl = choose_plan(pb, 0);
    if (pl.th == 0) return cudaErrorNotSupported;
    ListedParams prm{};
    plan_geom(prm.g, pb, pl.th, lr);
    prm.lr = lr; prm.dict = dict; prm.out = out; prm.idx = idx;
    prm.val = static_cast<const __half*>(val);
    prm.natoms = pb.s;
    prm.half_floats = pl.half_floats;
    switch (pb.k) {
    case 3: return launch_c<3>(prm, pl, st);
    case 5: return launch_c<5>(prm, pl, st);
    case 7: return launch_c<7>(prm, pl, st);
    default: return cudaErrorNotSupported;
    }
}

} // namespace sr
