// Regression with a small global atom subset on the fp32 FMA pipe (Section III-A: only the selected atoms of the
// dictionary are kept, Eq. 6; their coefficient channels are re-weighted by gamma, Eq. 9):
//   out[c][i] = sum_j (sum_{q<s} gamma_q Phi[S_q][i] dict[S_q][j]) B_{i,c}[j]      for s <= 8 atoms.
// With so few atoms the assembly F_i = Phi_i D is not a contraction worth a tensor-core tile (s k^2 + c k^2 = 275
// multiply-adds per pixel at s = 8, k = 5, c = 3): a tensor-core pipeline spends longer handing 128-pixel rows from
// role to role than the arithmetic takes. This kernel has no roles: every thread owns four neighbouring pixels of a
// row, reads their s coefficients straight from global memory (8 bytes per plane and thread, 256 contiguous bytes per
// warp), assembles the filter one patch row at a time with packed fp32 multiply-adds against the dictionary (kept in
// shared memory with every tap stored twice, so that one 16-byte broadcast load feeds two packed instructions), and
// applies it to the up-sampled tile. The dictionary stays fp32 (no binary16 split), F and U never leave the SM.
// Bound: the fp32 FMA pipe (s k^2 + c k^2 multiply-adds per pixel).
//
// Tile = 128 x th pixels (th = 8, 16 or 24), 256 threads = 8 warps, warp w takes the tile rows w, w + 8, ...; two
// CTAs per SM, so that one builds its next up-sampled tile while the other one filters.
#include "sr_regress_subset.cuh"
#include "sr_tile_upsample.cuh"

namespace sr {

namespace {

using namespace tile;

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;

struct SubParams {
    const float* lr;
    const float* dict;
    void* out;
    const uint8_t* idx;   // s atom ids
    const float* gamma;   // s weights or nullptr
    const __half* coef;
    Geom g;
    int natoms;           // s
    int planes;           // planes per frame in the coefficient tensor (D, or s when it is compact)
    int gather;           // 1: plane q is plane idx[q] of the full tensor
};

__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_but_one() { asm volatile("cp.async.wait_group 1;" ::: "memory"); }
__device__ __forceinline__ void cp_async_8(void* dst_smem, const void* src)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"((uint32_t)__cvta_generic_to_shared(dst_smem)), "l"(src) : "memory");
}

template <int K, int NQ, int C, typename OutT>
__global__ void __launch_bounds__(kThreads, 2) regress_subset_kernel(const __grid_constant__ SubParams p)
{
    constexpr int kk = K * K, P = (K - 1) / 2, UW = tile_uw(P), UW4 = UW / 4;
    constexpr int NU = (4 + K - 1 + 3) / 4;                  // 16-byte loads that cover a thread's four patches in a U row
    extern __shared__ __align__(16) float smem[];
    __shared__ float wpad[kMaxScale][12];
    __shared__ int64_t plane_off[NQ];

    const Geom& g = p.g;
    const Problem& pb = g.pb;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    float2* sD2 = reinterpret_cast<float2*>(smem);                                     // [kk][NQ]: every tap twice
    float* sU = smem + 2 * kk * NQ;                                                    // [C][uh][UW]
    float* sV = sU + C * g.uh * UW;                                                    // [C][uh][tcols]
    float* sL = sV + C * g.uh * g.tcols;                                               // [C * trows][tcols]
    const int total_floats = 2 * kk * NQ + C * g.uh * UW + C * g.uh * g.tcols + C * g.trows * g.tcols + 8;
    // coefficients of this thread's next two rows of work, [2][NQ][thread] x 8 bytes: fetched with cp.async one row of
    // work ahead (across tiles too), so that their trip from HBM is hidden behind a whole row of arithmetic
    uint2* sPhi = reinterpret_cast<uint2*>(smem + ((total_floats + 3) & ~3));

    // ---- set-up: buffers start as zeros (the up-sampling passes read a few values beyond the ones they weight)
    for (int i = tid; i < total_floats / 4; i += kThreads) reinterpret_cast<float4*>(smem)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    fill_wpad(pb, wpad, tid, kThreads);
    const int64_t plane_elems = (int64_t)pb.H * pb.W;
    if (tid < NQ) {
        int a = tid;
        if (p.gather && tid < p.natoms) a = min((int)__ldg(p.idx + tid), pb.D - 1);
        plane_off[tid] = (int64_t)a * plane_elems;
    }
    __syncthreads();
    for (int i = tid; i < kk * NQ; i += kThreads) {
        const int j = i / NQ, q = i - j * NQ;
        float v = 0.f;
        if (q < p.natoms) {
            const int a = p.idx ? min((int)__ldg(p.idx + q), pb.D - 1) : q;
            v = __ldg(p.dict + (int64_t)a * kk + j) * (p.gamma ? __ldg(p.gamma + q) : 1.f);
        }
        sD2[i] = make_float2(v, v);
    }
    // this thread's part of the up-sampling passes: a group of four columns and a row lane
    const int tc4 = g.tcols >> 2;
    const int v_lane = fast_div(tid, tc4, g.tc4_magic), v_i4 = (tid - v_lane * tc4) * 4, v_lanes = kThreads / tc4;
    const int h_lane = tid / UW4, h_cg = tid - h_lane * UW4, h_lanes = kThreads / UW4;
    const bool clamp01 = (pb.flags & SR_CLAMP01) != 0;

    // The CTA's share of the image is a run of 8-row groups (the same number for every CTA to within one), cut into
    // tiles of up to th rows. The warp's work, in order: tile rows warp, warp + 8, ... of its CTA's tiles. (pf_*) is the
    // next row to fetch coefficients for; it always runs one row of work ahead of the row being computed.
    const int run_end = run_bound(g, blockIdx.x + 1, gridDim.x);
    int run_cur = run_bound(g, blockIdx.x, gridDim.x);
    int pf_cur = run_cur, pf_rows = 0, pf_row = warp, buf = 0;
    const __half* pf_src = nullptr;                          // this lane's four coefficients in row 0 of the tile, plane 0
    auto pf_next_tile = [&]() {
        int f, y0, x0;
        if (!next_tile_of_run(g, pf_cur, run_end, f, y0, x0, pf_rows)) return false;
        const int px = x0 + 4 * lane;
        pf_src = px < pb.W ? p.coef + (int64_t)f * p.planes * plane_elems + (int64_t)y0 * pb.W + px : nullptr;
        return true;
    };
    bool pf_tile = pf_next_tile();
    auto fetch_next = [&](int into) {
        while (pf_tile) {
            if (pf_row < pf_rows) {
                if (pf_src) {
                    const __half* src = pf_src + (int64_t)pf_row * pb.W;
#pragma unroll
                    for (int q = 0; q < NQ; ++q)
                        if (q < p.natoms) cp_async_8(sPhi + (into * NQ + q) * kThreads + tid, src + plane_off[q]);
                }
                pf_row += kWarps;
                break;
            }
            pf_tile = pf_next_tile();
            pf_row = warp;
        }
        cp_async_commit();
    };
    {
        int peek = run_cur;
        LrWindow w0;
        if (next_tile_of_run(g, peek, run_end, w0.f, w0.y0, w0.x0, w0.rows)) {
            lr_window_of_tile<P>(g, w0);
            prefetch_lr_window_of(g, p.lr, w0, sL, tid, kThreads);
        }
    }
    fetch_next(0);
    LrWindow w;
    while (next_tile_of_run(g, run_cur, run_end, w.f, w.y0, w.x0, w.rows)) {
        lr_window_of_tile<P>(g, w);
        const int uh = w.rows + 2 * P;
        cp_async_wait_all();
        __syncthreads();                                     // LR window landed; the previous tile's U is no longer read
        if (v_lane < v_lanes) vertical_pass(g, w, uh, P, sL, sV, v_i4, v_lane, v_lanes);
        __syncthreads();
        {
            int peek = run_cur;
            LrWindow wn;
            if (next_tile_of_run(g, peek, run_end, wn.f, wn.y0, wn.x0, wn.rows)) {
                lr_window_of_tile<P>(g, wn);
                prefetch_lr_window_of(g, p.lr, wn, sL, tid, kThreads);
            }
        }
        if (h_lane < h_lanes) horizontal_pass<P>(g, wpad, w, uh, sV, sU, h_cg, h_lane, h_lanes);
        __syncthreads();                                     // the U tile is complete

        const int px0 = w.x0 + 4 * lane;
        {
            OutT* of = reinterpret_cast<OutT*>(p.out) + (int64_t)w.f * C * plane_elems + px0;
            for (int row = warp; row < w.rows; row += kWarps) {
                const int64_t pix = (int64_t)(w.y0 + row) * pb.W;
                fetch_next(buf ^ 1);                         // the row of work after this one
                cp_async_wait_but_one();                     // this row's coefficients (fetched one row of work ago) have landed
                if (px0 >= pb.W) { buf ^= 1; continue; }     // columns beyond the image (width not a multiple of 128)
                // coefficients of the four pixels: (pixel 0, pixel 1) and (pixel 2, pixel 3) per atom
                float2 phi[NQ][2];
#pragma unroll
                for (int q = 0; q < NQ; ++q) {
                    uint2 raw = make_uint2(0u, 0u);
                    if (q < p.natoms) raw = sPhi[(buf * NQ + q) * kThreads + tid];
                    phi[q][0] = __half22float2(*reinterpret_cast<const __half2*>(&raw.x));
                    phi[q][1] = __half22float2(*reinterpret_cast<const __half2*>(&raw.y));
                }
                buf ^= 1;
                float acc[C][4];
#pragma unroll
                for (int c = 0; c < C; ++c)
#pragma unroll
                    for (int i = 0; i < 4; ++i) acc[c][i] = 0.f;
#pragma unroll
                for (int a = 0; a < K; ++a) {
                    // patch row a of the four filters: F[b][pair] = sum_q dict[q][a][b] * phi[q][pair]
                    float2 F[K][2];
#pragma unroll
                    for (int b = 0; b < K; ++b) {
                        F[b][0] = F[b][1] = make_float2(0.f, 0.f);
                        const float4* dp = reinterpret_cast<const float4*>(sD2 + (a * K + b) * NQ);
#pragma unroll
                        for (int q2 = 0; q2 < NQ / 2; ++q2) {
                            const float4 dd = dp[q2];        // (d, d) of atom 2 q2 and (d, d) of atom 2 q2 + 1
                            F[b][0] = __ffma2_rn(make_float2(dd.x, dd.y), phi[2 * q2][0], F[b][0]);
                            F[b][1] = __ffma2_rn(make_float2(dd.x, dd.y), phi[2 * q2][1], F[b][1]);
                            F[b][0] = __ffma2_rn(make_float2(dd.z, dd.w), phi[2 * q2 + 1][0], F[b][0]);
                            F[b][1] = __ffma2_rn(make_float2(dd.z, dd.w), phi[2 * q2 + 1][1], F[b][1]);
                        }
                    }
                    // applied to row (row + a) of the U tile: pixel i, tap b reads column 4 lane + i + b
#pragma unroll
                    for (int c = 0; c < C; ++c) {
                        const float4* up = reinterpret_cast<const float4*>(sU + (c * g.uh + row + a) * UW + 4 * lane);
                        float u[4 * NU];
#pragma unroll
                        for (int n = 0; n < NU; ++n) {
                            const float4 v = up[n];
                            u[4 * n] = v.x; u[4 * n + 1] = v.y; u[4 * n + 2] = v.z; u[4 * n + 3] = v.w;
                        }
#pragma unroll
                        for (int b = 0; b < K; ++b) {
                            acc[c][0] = fmaf(F[b][0].x, u[b], acc[c][0]);
                            acc[c][1] = fmaf(F[b][0].y, u[b + 1], acc[c][1]);
                            acc[c][2] = fmaf(F[b][1].x, u[b + 2], acc[c][2]);
                            acc[c][3] = fmaf(F[b][1].y, u[b + 3], acc[c][3]);
                        }
                    }
                }
#pragma unroll
                for (int c = 0; c < C; ++c) {
                    float v[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) v[i] = clamp01 ? fminf(fmaxf(acc[c][i], 0.f), 1.f) : acc[c][i];
                    OutT* o = of + c * plane_elems + pix;
                    if constexpr (sizeof(OutT) == 4) {
                        *reinterpret_cast<float4*>(o) = make_float4(v[0], v[1], v[2], v[3]);
                    } else if constexpr (sizeof(OutT) == 1) {
                        *reinterpret_cast<uchar4*>(o) = make_uchar4(to_out<uint8_t>(v[0]), to_out<uint8_t>(v[1]), to_out<uint8_t>(v[2]), to_out<uint8_t>(v[3]));
                    } else {
                        const __half2 h01 = __floats2half2_rn(v[0], v[1]), h23 = __floats2half2_rn(v[2], v[3]);
                        *reinterpret_cast<uint2*>(o) = make_uint2(*reinterpret_cast<const uint32_t*>(&h01), *reinterpret_cast<const uint32_t*>(&h23));
                    }
                }
            }
        }
    }
    cp_async_wait_all();
}

struct DeviceInfo { int sms = 0, cc_major = 0, smem_sm = 0; bool ok = false; };

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
        if (cudaDeviceGetAttribute(&d.smem_sm, cudaDevAttrMaxSharedMemoryPerMultiprocessor, dev) != cudaSuccess) return none;
        d.ok = true;
    }
    return d;
}

constexpr int kStaticReserve = 2048;   // static shared memory + the per-CTA system reservation


// Tile height: every resident CTA gets the same run of 8-row groups (to within one) and cuts it into tiles of up to th
// rows; a warp takes every eighth row of a tile, so a run costs one row pass per group plus, per tile, its up-sampled
// tile (th + k - 1 rows) and three CTA-wide barriers. Units: warp instructions. The per-tile term is set from timings
// (1080p x4, s = 8): a tile's fixed work is about as long as sixteen rows of filtering, so the tallest tile wins.
int choose_th(const Problem& pb, int nq, size_t& smem_bytes, int& ctas, int g_forced_th = 0)
{
    const DeviceInfo& di = device_info();
    const int per_cta = di.smem_sm / 2 - kStaticReserve;
    const int tiles_x = (pb.W + TW - 1) / TW;
    int best_th = 0;
    double best = 0.0;
    for (int th = 24; th >= 8; th -= 8) {
        if (g_forced_th > 0 && th != g_forced_th) continue;
        Geom g;
        const size_t floats = ((plan_geom(g, pb, th, nullptr) + 2 * pb.k * pb.k * nq + 8 + 3) & ~(size_t)3) + 2 * nq * kThreads * 2;
        if (floats * 4 > (size_t)per_cta) continue;
        const long long groups = (long long)g.num_groups;
        const int c = groups < 2LL * di.sms ? (int)groups : 2 * di.sms;
        // a CTA's run of ceil(groups / c) 8-row groups costs its row passes plus one up-sampled tile (th + k - 1 rows
        // and three CTA-wide barriers) per th rows
        const long long per_cta = (groups + c - 1) / c;
        const long long tiles = (per_cta * 8 + th - 1) / th;
        const double row_pass = 8.0 * (nq * pb.k * pb.k * 0.625 + pb.c * pb.k * pb.k * 4 + 80);
        const double cost = (double)per_cta * row_pass + (double)tiles * (2 * row_pass + g.uh * 175.0);
        if (best_th == 0 || cost < best) { best_th = th; best = cost; smem_bytes = floats * 4; ctas = c; }
    }
    (void)tiles_x;
    return best_th;
}

template <int K, int NQ, int C, typename OutT>
cudaError_t launch_t(const SubParams& prm, int ctas, size_t smem, cudaStream_t st)
{
    auto kern = regress_subset_kernel<K, NQ, C, OutT>;
    static bool configured[64] = {false};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!configured[dev]) {
        const DeviceInfo& di = device_info();
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, di.smem_sm / 2 - kStaticReserve);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    kern<<<ctas, kThreads, smem, st>>>(prm);
    count_launches(1);
    return cudaGetLastError();
}

template <int K, int NQ, int C>
cudaError_t launch_o(const SubParams& prm, int ctas, size_t smem, cudaStream_t st)
{
    if (prm.g.pb.flags & SR_OUT_U8) return launch_t<K, NQ, C, uint8_t>(prm, ctas, smem, st);
    if (prm.g.pb.flags & SR_OUT_F16) return launch_t<K, NQ, C, __half>(prm, ctas, smem, st);
    return launch_t<K, NQ, C, float>(prm, ctas, smem, st);
}

template <int K, int NQ>
cudaError_t launch_c(const SubParams& prm, int ctas, size_t smem, cudaStream_t st)
{
    if (prm.g.pb.c == 3) return launch_o<K, NQ, 3>(prm, ctas, smem, st);
    if (prm.g.pb.c == 1) return launch_o<K, NQ, 1>(prm, ctas, smem, st);
    return cudaErrorNotSupported;
}

template <int K>
cudaError_t launch_q(const SubParams& prm, int ctas, size_t smem, cudaStream_t st)
{
    return prm.natoms <= 4 ? launch_c<K, 4>(prm, ctas, smem, st) : launch_c<K, 8>(prm, ctas, smem, st);
}

} // namespace

// Tile heights the problem admits (shared memory of two CTAs per SM); the tile-shape search times these.
int regress_subset_candidates(const Problem& pb, int* ths, int max_out)
{
    int n = 0;
    for (int th = 24; th >= 8; th -= 8) {
        size_t smem;
        int ctas;
        if (choose_th(pb, pb.s <= 4 ? 4 : 8, smem, ctas, th) == th && n < max_out) ths[n++] = th;
    }
    return n;
}

bool regress_subset_supported(int mode, const void* coef, int coef_dtype, const void* out, const Problem& pb)
{
    if ((reinterpret_cast<uintptr_t>(out) & ((pb.flags & SR_OUT_U8) ? 3 : ((pb.flags & SR_OUT_F16) ? 7 : 15))) != 0) return false;   // one store per four pixels
    if (mode != kModeGlobal || pb.s > 8 || coef_dtype != SR_F16) return false;
    if (pb.k > 7 || (pb.c != 1 && pb.c != 3)) return false;
    if ((reinterpret_cast<uintptr_t>(coef) & 7) != 0 || (pb.W & 3) != 0) return false;    // 8-byte loads of four coefficients
    const DeviceInfo& di = device_info();
    if (!di.ok || di.cc_major < 9) return false;
    size_t smem;
    int ctas;
    return choose_th(pb, pb.s <= 4 ? 4 : 8, smem, ctas) > 0;
}

cudaError_t launch_regress_subset(const float* lr, const void* coef, const uint8_t* idx, const float* gamma, const float* dict,
                                  float* out, const Problem& pb, cudaStream_t st, int th_forced)
{
    SubParams prm{};
    size_t smem = 0;
    int ctas = 0;
    const int th = choose_th(pb, pb.s <= 4 ? 4 : 8, smem, ctas, th_forced);
    if (th == 0) return cudaErrorNotSupported;
    plan_geom(prm.g, pb, th, lr);
    prm.lr = lr; prm.dict = dict; prm.out = out; prm.idx = idx; prm.gamma = gamma;
    prm.coef = static_cast<const __half*>(coef);
    prm.natoms = pb.s;
    prm.gather = (pb.flags & SR_COEF_COMPACT) ? 0 : 1;
    prm.planes = prm.gather ? pb.D : pb.s;
    switch (pb.k) {
    case 1: return launch_q<1>(prm, ctas, smem, st);
    case 3: return launch_q<3>(prm, ctas, smem, st);
    case 5: return launch_q<5>(prm, ctas, smem, st);
    case 7: return launch_q<7>(prm, ctas, smem, st);
    default: return cudaErrorNotSupported;
    }
}

} // namespace sr
