// Regression fused with the producer of Phi, for sm_100a.
//
// Section II-A: the coefficient network ends in convolution and pixel-shuffle layers that predict Phi, and the
// regression then forms F_i = Phi_i D (Eq. 2-3) and y_i = F_i B_i^T. When the last layer is a plain convolution (no
// activation after it), the two linear maps compose: with the LR feature vector x(q) around LR pixel q,
//     F_i[j] = sum_l Phi_l(i) D[l][j] = sum_{tap, ci} x(q)[tap][ci] * ( sum_l Wc[l r^2 + phase(i)][ci][tap] D[l][j] ) + b'[phase(i)][j]
// so the per-pixel filter is ONE convolution of the feature map with the folded weights W' = Wc D (r^2 k^2 output
// channels instead of L r^2), and neither Phi (144 bytes per HR pixel at L = 72) nor F ever exists in memory. A global
// atom subset with weights gamma (Section III-A, Eq. 6 / Eq. 9) folds the same way (the sum runs over the subset).
// launch_producer_fold builds W' and b' once per (network, dictionary); launch_producer_regress is the per-frame kernel.
//
// The kernel is an implicit GEMM on the tensor cores: M = 128 LR pixels of a tile (128 / r columns x r rows, so the HR
// tile is 128 x r^2 pixels; at r = 3, 42 x 3 LR pixels = 126 of the 128 rows and an HR tile of 126 x 9), K = kc^2 taps x 32 feature channels, N = the folded filters of a group of phase rows.
//   A: one TMA box per tap and 8-channel group from the channels-last feature map [n][h][w][32] (binary16); boxes that
//      reach outside the map read zeros, which is the convolution's zero padding. K-major, no swizzle.
//   B: W' as binary16, pre-arranged by the fold in the K-major core-matrix order the MMA reads, streamed from L2 by
//      plain bulk copies through a small ring (a step = the taps of one kernel row).
//   bias: b' enters through one extra K-step whose A operand is a constant tile (two columns of ones) and whose B rows
//      hold the binary16 hi and lo parts of b', so the epilogue never touches it.
//   D: fp32 in tensor memory, two buffers of 256 columns; a pass fills one buffer with the filters of RG phase rows
//      (N <= 256) while the epilogue drains the other.
// Epilogue: thread = one LR pixel = one TMEM lane; per HR row of its r x r block and per patch row it loads the r k
// filter taps of its r pixels, reads r + k - 1 neighbouring values of the up-sampled tile per channel (shared memory,
// vector loads) and accumulates r x c outputs; r consecutive output pixels leave as one vector store. Two groups of four
// warps take alternate passes. The up-sampled tile is built per tile by the epilogue warps (stage 1, Section II-A;
// shared code with the other regression kernels).
// Warps: 0 weight stages (bulk copies, one thread), 1 MMA issuer (one thread; owns tensor memory), 2 LR-window
// prefetch (two windows ahead), 3 feature taps (TMA boxes, one thread), 4-7 / 8-11 epilogue groups. One CTA per SM (512 TMEM columns), persistent over tiles.
// Every wait is bounded; on expiry the CTA raises its abort flag, sets the device status word, drains and returns.
#include "sr_ptx.cuh"
#include "sr_producer.cuh"
#include "sr_tile_upsample.cuh"

namespace sr {

namespace {

using namespace ptx;
using namespace tile;

constexpr int kCin = 32;
constexpr int kTapBytes = 128 * kCin * 2;   // one tap of the A operand: 128 pixels x 32 channels, binary16
constexpr int kOnesBytes = 128 * 16 * 2;    // the constant A tile of the bias K-step
constexpr int kUtilThreads = 128, kEpiThreads = 256, kThreads = kUtilThreads + kEpiThreads;
constexpr int kMaxSteps = 9, kMaxStages = 4, kMaxC = 3;
constexpr int kMmaWarp = 1, kLrWarp = 2, kLrThreads = 32, kFeatWarp = 3;

template <int R, int K> struct PG {
    static constexpr int kk = K * K, P = (K - 1) / 2;
    static constexpr int TWD = R == 3 ? 126 : TW;      // HR columns of a tile (a multiple of r)
    static constexpr int TLW = TWD / R;                // LR columns of a tile
    static constexpr int TLH = 128 / TLW;              // LR rows of a tile
    static constexpr int MPIX = TLW * TLH;             // LR pixels of a tile = rows of the MMA in use (128, or 126 at r = 3)
    static constexpr int TH = R * TLH;                 // HR rows of a tile
    static constexpr int FW = R * K;                   // taps of one patch row for the r pixels of an HR row of the block
    static constexpr int FWP = (FW + 3) & ~3;          // padded so that tensor-memory loads stay naturally aligned
    static constexpr int RG = R == 3 ? (3 * K * FWP <= 256 ? 3 : 1)
                                     : ((R % 2 == 0 && 2 * K * FWP <= 256) ? 2 : 1);   // phase rows per pass (N <= 256)
    static constexpr int G = R / RG;                   // passes per tile
    static constexpr bool SPLIT = RG >= 2;             // both epilogue groups work on every pass: group e takes the phase
                                                       // rows of the pass with ryl % 2 == e
    static constexpr int NCOL = RG * K * FWP;          // accumulator columns of a pass
    static constexpr int NG = (NCOL + 15) / 16 * 16;   // N of the MMA
    static constexpr int UW = tile_uw(P, TWD), UW4 = UW / 4;
    static constexpr uint32_t TAP_TX = MPIX * kCin * 2;   // bytes the boxes of one tap bring
    static constexpr int LBO_B = NG * 16;              // bytes between the two 8-channel groups of a K-step of B
    static constexpr int BIAS_BYTES = 2 * LBO_B;       // one K-step
    static constexpr int TAP_B_BYTES = 4 * LBO_B;      // two K-steps (32 channels)
    static_assert(MPIX <= 128 && MPIX > 96 && (SPLIT || (G % 2) == 0) && NG <= 256, "tile or pass shape");
    // accumulator column of tap (a, b) for pixel rx of phase row ryl
    __host__ __device__ static constexpr int col_of(int ryl, int a, int rx, int b) { return (ryl * K + a) * FWP + rx * K + b; }
};

struct ProdParams {
    const float* lr;
    void* out;
    const uint8_t* folded;
    int* status;
    Geom g;
    int kc, ntaps;
    int tps, nsteps;          // taps per pipeline step, steps per pass
    int stages;
    int resident;             // 1: every weight stage of a tile has its own slot; the weights are loaded once per CTA
    uint32_t stage_bytes;
    long long wait_cycles;
    int inject_lost_arrival;
};

struct __align__(16) Ctl {
    uint64_t b_full[kMaxStages], b_empty[kMaxStages];
    uint64_t a_full[kMaxSteps], a_empty[kMaxSteps];
    uint64_t acc_full[2], acc_empty[2];
    uint64_t lr_full[2], lr_empty[2];
    uint64_t drain;
    uint32_t tmem_base;
    WaitCtx wait;
    float wpad[kMaxScale][12];
};

__device__ __forceinline__ void cp_async_mbar_arrive_noinc(uint64_t* bar)
{
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

__device__ __forceinline__ void named_barrier_sync(int id, int nthreads)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

__device__ __forceinline__ bool named_barrier_and(int id, int nthreads, bool pred)
{
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 p, %1, 0;\n\tbarrier.cta.red.and.pred q, %2, %3, p;\n\tselp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(r)
        : "r"((uint32_t)pred), "r"(id), "r"(nthreads)
        : "memory");
    return r != 0;
}

// N (a multiple of 4) consecutive accumulator columns from column `off` (a multiple of 4), in pieces that are aligned
// to their own width. `off` is a constant after unrolling, so only one chain of loads remains.
template <int N>
__device__ __forceinline__ void tmem_ld_natural(uint32_t taddr, int off, float* v)
{
    if constexpr (N >= 16) {
        if ((off & 15) == 0) {
            tmem_ld_x16(taddr + off, v);
            tmem_ld_natural<N - 16>(taddr, off + 16, v + 16);
            return;
        }
    }
    if constexpr (N >= 8) {
        if ((off & 7) == 0) {
            tmem_ld_x8(taddr + off, v);
            tmem_ld_natural<N - 8>(taddr, off + 8, v + 8);
            return;
        }
    }
    if constexpr (N >= 4) {
        tmem_ld_x4(taddr + off, v);
        tmem_ld_natural<N - 4>(taddr, off + 4, v + 4);
    }
}

// R consecutive output pixels as one store.
template <int R, typename OutT> __device__ __forceinline__ void store_pixels(OutT* dst, const float* v);
template <> __device__ __forceinline__ void store_pixels<4, float>(float* dst, const float* v)
{
    *reinterpret_cast<float4*>(dst) = make_float4(v[0], v[1], v[2], v[3]);
}
template <> __device__ __forceinline__ void store_pixels<2, float>(float* dst, const float* v)
{
    *reinterpret_cast<float2*>(dst) = make_float2(v[0], v[1]);
}
template <> __device__ __forceinline__ void store_pixels<4, __half>(__half* dst, const float* v)
{
    const __half2 a = __floats2half2_rn(v[0], v[1]), b = __floats2half2_rn(v[2], v[3]);
    *reinterpret_cast<uint2*>(dst) = make_uint2(*reinterpret_cast<const uint32_t*>(&a), *reinterpret_cast<const uint32_t*>(&b));
}
template <> __device__ __forceinline__ void store_pixels<2, __half>(__half* dst, const float* v)
{
    *reinterpret_cast<__half2*>(dst) = __floats2half2_rn(v[0], v[1]);
}
template <> __device__ __forceinline__ void store_pixels<4, uint8_t>(uint8_t* dst, const float* v)
{
    *reinterpret_cast<uchar4*>(dst) = make_uchar4(to_out<uint8_t>(v[0]), to_out<uint8_t>(v[1]), to_out<uint8_t>(v[2]), to_out<uint8_t>(v[3]));
}
template <> __device__ __forceinline__ void store_pixels<2, uint8_t>(uint8_t* dst, const float* v)
{
    *reinterpret_cast<uchar2*>(dst) = make_uchar2(to_out<uint8_t>(v[0]), to_out<uint8_t>(v[1]));
}

template <> __device__ __forceinline__ void store_pixels<3, float>(float* dst, const float* v)
{
    dst[0] = v[0]; dst[1] = v[1]; dst[2] = v[2];
}
template <> __device__ __forceinline__ void store_pixels<3, __half>(__half* dst, const float* v)
{
    dst[0] = __float2half_rn(v[0]); dst[1] = __float2half_rn(v[1]); dst[2] = __float2half_rn(v[2]);
}
template <> __device__ __forceinline__ void store_pixels<3, uint8_t>(uint8_t* dst, const float* v)
{
    dst[0] = to_out<uint8_t>(v[0]); dst[1] = to_out<uint8_t>(v[1]); dst[2] = to_out<uint8_t>(v[2]);
}

// One phase row (RYL, compile-time) of one pass for one thread: the r pixels of one HR row of this thread's r x r block.
// The tensor-memory loads of patch row a + 1 are issued before the arithmetic of row a, so their latency hides behind it.
//   u_px:   the up-sampled tile at (channel 0, row 0, this block's first column); planes u_plane floats apart
//   out_px: channel 0, first row of the tile, this block's first pixel; channels HW elements apart
template <int R, int K, typename OutT, int RYL>
__device__ __forceinline__ void epilogue_row(const float* u_px, int u_plane, OutT* out_px, int64_t HW, int W, int C, int g,
                                             uint32_t taddr, int yl, int rows_valid, bool in_x, bool clamp01)
{
    using G = PG<R, K>;
    constexpr int UWIN = R + K - 1;                 // neighbouring values of a patch row the r pixels share
    constexpr int UV = R == 4 ? 4 : (R == 2 ? 2 : 1);   // floats per load (16-, 8- or 4-byte aligned at r * xl)
    constexpr int NV = (UWIN + UV - 1) / UV;
    const int yt = R * yl + g * G::RG + RYL;        // row inside the tile
    float acc[kMaxC][R];
#pragma unroll
    for (int ch = 0; ch < kMaxC; ++ch)
#pragma unroll
        for (int rx = 0; rx < R; ++rx) acc[ch][rx] = 0.f;
    float f[2][G::FWP];
    tmem_ld_natural<G::FWP>(taddr, (RYL * K) * G::FWP, f[0]);
#pragma unroll
    for (int a = 0; a < K; ++a) {
        tmem_ld_wait();
        if (a + 1 < K) tmem_ld_natural<G::FWP>(taddr, (RYL * K + a + 1) * G::FWP, f[(a + 1) & 1]);
        const float* fa = f[a & 1];
        float u[kMaxC][NV * UV];
#pragma unroll
        for (int ch = 0; ch < kMaxC; ++ch) {
            if (ch < C) {
                const float* urow = u_px + ch * u_plane + (yt + a) * G::UW;
#pragma unroll
                for (int i = 0; i < NV; ++i) {
                    if constexpr (UV == 4) {
                        const float4 t = *reinterpret_cast<const float4*>(urow + 4 * i);
                        u[ch][4 * i] = t.x; u[ch][4 * i + 1] = t.y; u[ch][4 * i + 2] = t.z; u[ch][4 * i + 3] = t.w;
                    } else if constexpr (UV == 1) {
                        u[ch][i] = urow[i];
                    } else {
                        const float2 t = *reinterpret_cast<const float2*>(urow + 2 * i);
                        u[ch][2 * i] = t.x; u[ch][2 * i + 1] = t.y;
                    }
                }
            }
        }
        // tap by tap across the r x c accumulators, so that consecutive multiply-adds are independent
#pragma unroll
        for (int b = 0; b < K; ++b)
#pragma unroll
            for (int ch = 0; ch < kMaxC; ++ch)
                if (ch < C) {
#pragma unroll
                    for (int rx = 0; rx < R; ++rx) acc[ch][rx] = fmaf(fa[rx * K + b], u[ch][rx + b], acc[ch][rx]);
                }
    }
    if (in_x && yt < rows_valid) {
#pragma unroll
        for (int ch = 0; ch < kMaxC; ++ch) {
            if (ch < C) {
                if (clamp01) {
#pragma unroll
                    for (int rx = 0; rx < R; ++rx) acc[ch][rx] = fminf(fmaxf(acc[ch][rx], 0.f), 1.f);
                }
                store_pixels<R, OutT>(out_px + ch * HW + (int64_t)yt * W, acc[ch]);
            }
        }
    }
}

// One pass of one tile for one thread: the RG phase rows of pass g (group < 0), or those with ryl % 2 == group (split passes).
template <int R, int K, typename OutT>
__device__ __forceinline__ void epilogue_pass(const float* u_px, int u_plane, OutT* out_px, int64_t HW, int W, int C, int g,
                                              uint32_t taddr, int yl, int rows_valid, bool in_x, bool clamp01, int group)
{
    if (group != 1) epilogue_row<R, K, OutT, 0>(u_px, u_plane, out_px, HW, W, C, g, taddr, yl, rows_valid, in_x, clamp01);
    if constexpr (PG<R, K>::RG >= 2) {
        if (group != 0) epilogue_row<R, K, OutT, 1>(u_px, u_plane, out_px, HW, W, C, g, taddr, yl, rows_valid, in_x, clamp01);
    }
    if constexpr (PG<R, K>::RG >= 3) {
        if (group != 1) epilogue_row<R, K, OutT, 2>(u_px, u_plane, out_px, HW, W, C, g, taddr, yl, rows_valid, in_x, clamp01);
    }
}

template <int R, int K, typename OutT>
__global__ void __launch_bounds__(kThreads, 1)
producer_regress_kernel(const __grid_constant__ CUtensorMap map_feat, const __grid_constant__ ProdParams p)
{
    using G = PG<R, K>;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    __shared__ Ctl ctl;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const Problem& pb = p.g.pb;
    const int C = pb.c;

    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* sA = smem;                                           // [ntaps][4 channel groups][128 pixels][8] binary16
    uint8_t* sOnes = sA + (size_t)p.ntaps * kTapBytes;            // [2][128][8]
    uint8_t* sB = sOnes + kOnesBytes;                             // [stages][stage_bytes]
    float* sU = reinterpret_cast<float*>(sB + (size_t)p.stages * p.stage_bytes);   // [C][uh][UW]
    float* sV = sU + C * p.g.uh * G::UW;                          // [C][uh][tcols]
    float* sL = sV + C * p.g.uh * p.g.tcols;                      // [2 buffers][C * trows][tcols]
    const int l_tile = C * p.g.trows * p.g.tcols;                 // floats of one LR window
    const int dyn_bytes = (int)((uint8_t*)(sL + 2 * l_tile) - smem) + 32;

    // ---------------------------------------------------------------- set-up
    if (tid == 0) {
        for (int i = 0; i < kMaxStages; ++i) { mbar_init(&ctl.b_full[i], 1); mbar_init(&ctl.b_empty[i], 1); }
        for (int i = 0; i < kMaxSteps; ++i) { mbar_init(&ctl.a_full[i], 1); mbar_init(&ctl.a_empty[i], 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(&ctl.acc_full[i], 1); mbar_init(&ctl.acc_empty[i], G::SPLIT ? 8 : 4); }
        for (int i = 0; i < 2; ++i) { mbar_init(&ctl.lr_full[i], kLrThreads); mbar_init(&ctl.lr_empty[i], 1); }
        mbar_init(&ctl.drain, 1);
        ctl.wait.abort_flag = 0;
        ctl.wait.limit = p.wait_cycles;
        fence_barrier_init();
        prefetch_tensormap(&map_feat);
    }
    // everything starts as zeros: the up-sampling passes read a few staged values beyond the ones they weight, and the
    // constant tile of the bias step is zero except for its two columns of ones
    {
        uint4* a4 = reinterpret_cast<uint4*>(smem);
        for (int i = tid; i < dyn_bytes / 16; i += kThreads) a4[i] = make_uint4(0, 0, 0, 0);
    }
    fill_wpad(pb, ctl.wpad, tid, kThreads);
    __syncthreads();
    // element (pixel m, channel k) of a K-major operand without swizzle: (k / 8) * (rows * 16) + m * 16 + (k % 8) * 2
    if (tid < 128) *reinterpret_cast<uint32_t*>(sOnes + tid * 16) = 0x3C003C00u;   // k = 0 and k = 1: 1.0, 1.0
    fence_proxy_async_smem();
    __syncwarp();
    if (warp == kMmaWarp) tmem_alloc(&ctl.tmem_base, 512);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = ctl.tmem_base;
    volatile WaitCtx* wc = &ctl.wait;
    const int pc = p.kc / 2;

    // ---------------------------------------------------------------- roles
    if (warp == 0) {
        // ===== weight stages: one bulk copy per step of every pass, through the ring (or once per CTA when resident)
        if (lane == 0) {
            int s = 0;
            uint32_t ph = 0, ti = 0;
            bool ok = true;
            int issued_b = 0;
            bool lose_one = p.inject_lost_arrival != 0 && blockIdx.x == 0;
            for (int t = blockIdx.x; t < p.g.num_tiles && ok; t += gridDim.x, ++ti) {
                for (int g = 0; g < G::G && ok; ++g) {
                    for (int st = 0; st < p.nsteps; ++st) {
                        if (!p.resident && !(ok = mbar_wait(&ctl.b_empty[s], ph ^ 1, wc))) break;
                        if (p.resident && ti > 0) continue;      // resident weights: slot g * nsteps + st was filled for the first tile
                        if (lose_one && (st == 1 || p.nsteps == 1)) {
                            lose_one = false;                    // test hook: this stage never fills
                        } else {
                            mbar_arrive_expect_tx(&ctl.b_full[s], p.stage_bytes);
                            bulk_load_1d(sB + (size_t)s * p.stage_bytes, p.folded + (size_t)(g * p.nsteps + st) * p.stage_bytes,
                                         p.stage_bytes, &ctl.b_full[s]);
                        }
                        ++issued_b;
                        if (++s == p.stages) { s = 0; ph ^= 1; }
                    }
                }
            }
            if (!ok) {
                // wind-down after a failed wait: copies issued into stages that were never consumed may still be
                // travelling; give each a short, bounded time to land before the CTA leaves
                int sj = s;
                uint32_t pj = ph;
                const int in_flight = min(issued_b, p.stages);
                for (int j = 0; j < in_flight; ++j) {
                    if (--sj < 0) { sj += p.stages; pj ^= 1; }
                    mbar_wait_drain(&ctl.b_full[sj], pj);
                }
            }
        }
        __syncwarp();
    } else if (warp == kFeatWarp) {
        // ===== feature taps: TMA boxes of the tile's taps, step by step, as soon as the previous tile's MMAs have read them
        if (lane == 0) {
            uint32_t ti = 0, a_issued = 0, a_parity = 0;      // per step: a box was issued; parity of its phase
            bool ok = true;
            for (int t = blockIdx.x; t < p.g.num_tiles && ok; t += gridDim.x, ++ti) {
                int f, y0, x0, rows;
                decode_tile(p.g, t, f, y0, x0, rows);
                const int ylr0 = y0 / R, xlr0 = x0 / R;
                for (int st = 0; st < p.nsteps; ++st) {
                    if (!(ok = mbar_wait(&ctl.a_empty[st], (ti & 1) ^ 1, wc))) break;
                    const int nt = min(p.tps, p.ntaps - st * p.tps);
                    mbar_arrive_expect_tx(&ctl.a_full[st], (uint32_t)nt * G::TAP_TX);
                    for (int j = 0; j < nt; ++j) {
                        const int tap = st * p.tps + j;
                        const int dy = tap / p.kc, dx = tap - dy * p.kc;
                        uint8_t* dst = sA + (size_t)tap * kTapBytes;
#pragma unroll
                        for (int kg = 0; kg < kCin / 8; ++kg)
                            tma_load_4d(dst + kg * 2048, &map_feat, &ctl.a_full[st], kg * 8, xlr0 + dx - pc, ylr0 + dy - pc, f);
                    }
                    a_issued |= 1u << st;
                    a_parity = (a_parity & ~(1u << st)) | ((ti & 1) << st);
                }
            }
            if (!ok)                                          // wind-down: boxes in flight get a short, bounded time to land
                for (int st = 0; st < p.nsteps; ++st)
                    if (a_issued & (1u << st)) mbar_wait_drain(&ctl.a_full[st], (a_parity >> st) & 1u);
        }
        __syncwarp();
    } else if (warp == kMmaWarp) {
        // ===== MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc_f16(128, G::NG, /*a_mn_major=*/false, /*b_mn_major=*/false);
            // both operands K-major without swizzle: 8 rows x 16 bytes per core matrix, row groups 128 B apart (SBO),
            // the second 8-channel group of a K-step LBO bytes away
            const uint64_t a_desc0 = make_smem_desc(smem_u32(sA), 2048, 128, kSwizzleNone);
            const uint64_t ones_desc = make_smem_desc(smem_u32(sOnes), 2048, 128, kSwizzleNone);
            const uint64_t b_desc0 = make_smem_desc(smem_u32(sB), G::LBO_B, 128, kSwizzleNone);
            int s = 0;
            uint32_t ph = 0, ti = 0, pcount = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < p.g.num_tiles && ok; t += gridDim.x, ++ti) {
                for (int g = 0; g < G::G && ok; ++g, ++pcount) {
                    const uint32_t buf = pcount & 1;
                    if (!(ok = mbar_wait(&ctl.acc_empty[buf], ((pcount >> 1) & 1) ^ 1, wc))) break;
                    const uint32_t taddr = tmem_base + buf * 256u;
                    for (int st = 0; st < p.nsteps; ++st) {
                        if (p.resident) s = g * p.nsteps + st;
                        if ((!p.resident || ti == 0) && !(ok = mbar_wait(&ctl.b_full[s], p.resident ? 0u : ph, wc))) break;
                        if (g == 0 && !(ok = mbar_wait(&ctl.a_full[st], ti & 1, wc))) break;
                        tc_fence_after_sync();
                        const uint64_t bst = b_desc0 + (uint64_t)(((uint32_t)s * p.stage_bytes) >> 4);
                        if (st == 0) mma_f16_ss(taddr, ones_desc, bst, idesc, 0u);       // bias: starts the accumulation
                        const int nt = min(p.tps, p.ntaps - st * p.tps);
                        for (int j = 0; j < nt; ++j) {
                            const int tap = st * p.tps + j;
                            const uint64_t ad = a_desc0 + (uint64_t)((uint32_t)(tap * kTapBytes) >> 4);
                            const uint64_t bd = bst + (uint64_t)((uint32_t)(G::BIAS_BYTES + j * G::TAP_B_BYTES) >> 4);
                            mma_f16_ss(taddr, ad, bd, idesc, 1u);
                            mma_f16_ss(taddr, ad + (4096 >> 4), bd + ((2 * G::LBO_B) >> 4), idesc, 1u);
                        }
                        if (!p.resident) mma_commit(&ctl.b_empty[s]);   // the stage may be refilled once these MMAs have read it
                        if (g == G::G - 1) mma_commit(&ctl.a_empty[st]);   // and, after the tile's last pass, the feature taps
                        if (!p.resident && ++s == p.stages) { s = 0; ph ^= 1; }
                    }
                    if (ok) mma_commit(&ctl.acc_full[buf]);
                }
            }
            // tensor memory is freed only once every MMA issued here has finished
            mma_commit(&ctl.drain);
            mbar_wait_drain(&ctl.drain, 0);
        }
        __syncwarp();
    } else if (warp == kLrWarp) {
        // ===== LR-window prefetch, two buffers: the windows of tiles i + 1 and i + 2 travel while the
        // epilogue works on tile i (a window takes a microsecond or two to arrive from global memory)
        uint32_t ti = 0;
        for (int t = blockIdx.x; t < p.g.num_tiles; t += gridDim.x, ++ti) {
            const uint32_t lb = ti & 1u;
            bool ok = true;
            if (lane == 0) ok = mbar_wait_relaxed(&ctl.lr_empty[lb], ((ti >> 1) & 1u) ^ 1u, wc);
            if (!__shfl_sync(0xffffffffu, (int)ok, 0)) break;
            prefetch_lr_window<G::P, G::TWD>(p.g, p.lr, t, sL + lb * l_tile, tid - kLrWarp * 32, kLrThreads);
            cp_async_mbar_arrive_noinc(&ctl.lr_full[lb]);
        }
        cp_async_wait_all();
    } else if (warp >= 4) {
        // ===== epilogue
        const int e = (warp - 4) >> 2;                       // group: takes the passes with g % 2 == e
        const int quarter = warp & 3;                        // the TMEM lanes this warp may read: 32*quarter..+31
        const int m = quarter * 32 + lane;                   // LR pixel of the tile = TMEM lane
        const bool lane_used = m < G::MPIX;                  // at r = 3 the last two rows of the MMA carry no pixel
        const int yl = lane_used ? m / G::TLW : 0, xl = lane_used ? m - yl * G::TLW : 0;
        const int64_t HW = (int64_t)pb.H * pb.W;
        const bool clamp01 = (pb.flags & SR_CLAMP01) != 0;
        const uint32_t tmem_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
        const int et = tid - kUtilThreads;
        const int tc4 = p.g.tcols >> 2;
        const int v_lane = fast_div(et, tc4, p.g.tc4_magic), v_i4 = (et - v_lane * tc4) * 4, v_lanes = kEpiThreads / tc4;
        const int h_lane = et / G::UW4, h_cg = et - h_lane * G::UW4, h_lanes = kEpiThreads / G::UW4;
        const int u_plane = p.g.uh * G::UW;
        uint32_t ti = 0, pe = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < p.g.num_tiles; t += gridDim.x, ++ti) {
            LrWindow w;
            lr_window<G::P, G::TWD>(p.g, t, w);
            const int uh = w.rows + 2 * G::P;
            const uint32_t lb = ti & 1u;
            ok = ok && mbar_wait_leader(&ctl.lr_full[lb], (ti >> 1) & 1u, wc, true);
            ok = named_barrier_and(1, kEpiThreads, ok);      // LR window landed, previous tile left by every thread
            if (!ok) break;
            if (v_lane < v_lanes) vertical_pass(p.g, w, uh, G::P, sL + lb * l_tile, sV, v_i4, v_lane, v_lanes);
            named_barrier_sync(1, kEpiThreads);
            if (et == 0) mbar_arrive(&ctl.lr_empty[lb]);     // this LR window may be overwritten
            if (h_lane < h_lanes) horizontal_pass<G::P, G::TWD>(p.g, ctl.wpad, w, uh, sV, sU, h_cg, h_lane, h_lanes);
            named_barrier_sync(1, kEpiThreads);              // the U tile is complete
            const bool in_x = lane_used && w.x0 + R * xl < pb.W;
            OutT* out_px = reinterpret_cast<OutT*>(p.out) + (int64_t)w.f * C * HW + (int64_t)w.y0 * pb.W + w.x0 + R * xl;
            // split passes: both groups take every pass (buffers alternate), group e the phase row e of it;
            // otherwise group e takes the passes with g % 2 == e, which always land in buffer e
            for (int g = G::SPLIT ? 0 : e; g < G::G; g += G::SPLIT ? 1 : 2, ++pe) {
                const uint32_t buf = G::SPLIT ? (pe & 1u) : (uint32_t)e;
                ok = mbar_wait_leader(&ctl.acc_full[buf], (G::SPLIT ? (pe >> 1) : pe) & 1u, wc, false);
                if (!ok) break;
                tc_fence_after_sync();
                epilogue_pass<R, K, OutT>(sU + R * xl, u_plane, out_px, HW, pb.W, C, g, tmem_lane + buf * 256u, yl, w.rows, in_x,
                                          clamp01, G::SPLIT ? e : -1);
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&ctl.acc_empty[buf]);   // this warp has read its lanes of the buffer
            }
            // a failed wait is agreed on at the next tile's barrier, so that nobody is left waiting there
        }
    }

    // ---------------------------------------------------------------- teardown
    __syncwarp();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (ctl.wait.abort_flag && tid == 0) atomicExch(p.status, SR_ERR_TIMEOUT);
    if (warp == kMmaWarp) tmem_dealloc(tmem_base, 512);
}

// ---- folding -----------------------------------------------------------------------------------------------------------

struct FoldParams {
    const float* wconv;
    const float* bias;
    const float* dict;
    const uint8_t* idx;
    const float* gamma;
    int natoms, D, cin, kc, ntaps, tps, nsteps;
    uint32_t stage_bytes;
    int64_t total_halves;
};

// One thread per binary16 element of the folded block. Stage (g, st) = [bias K-step][tps taps x two K-steps]; inside a
// K-step pair the element (column n, channel k) sits at (k / 8) * LBO + (n / 8) * 128 + (n % 8) * 16 + (k % 8) * 2.
template <int R, int K>
__global__ void producer_fold_kernel(__half* __restrict__ folded, const __grid_constant__ FoldParams fp)
{
    using G = PG<R, K>;
    const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= fp.total_halves) return;
    const int per_stage = (int)(fp.stage_bytes / 2);
    const int stage = (int)(e / per_stage);
    int rem = (int)(e - (int64_t)stage * per_stage);
    const int g = stage / fp.nsteps, st = stage - g * fp.nsteps;
    const bool is_bias = rem < G::BIAS_BYTES / 2;
    int tap = -1;
    if (!is_bias) {
        rem -= G::BIAS_BYTES / 2;
        const int j = rem / (G::TAP_B_BYTES / 2);
        rem -= j * (G::TAP_B_BYTES / 2);
        tap = st * fp.tps + j;
    }
    const int kg = rem / (G::LBO_B / 2);                     // 8-channel group
    rem -= kg * (G::LBO_B / 2);
    const int n = (rem >> 6) * 8 + ((rem >> 3) & 7);         // column
    const int k = kg * 8 + (rem & 7);                        // channel (or hi / lo slot of the bias step)
    float value = 0.f;
    const int blk = n / G::FWP, i = n - blk * G::FWP;
    const bool col_used = n < G::NCOL && i < G::FW;
    const bool wanted = col_used && (is_bias ? (st == 0 && k < 2 && fp.bias != nullptr) : (tap < fp.ntaps && k < fp.cin));
    if (wanted) {
        const int ryl = blk / K, a = blk - ryl * K;
        const int rx = i / K, b = i - rx * K;
        const int phase = (g * G::RG + ryl) * R + rx;
        const int jj = a * K + b;
        double acc = 0.0;
        for (int q = 0; q < fp.natoms; ++q) {
            const int l = fp.idx ? min((int)fp.idx[q], fp.D - 1) : q;
            const double wgt = (fp.idx && fp.gamma) ? (double)fp.gamma[q] : 1.0;
            const int o = l * R * R + phase;
            const double src = is_bias ? (double)fp.bias[o] : (double)fp.wconv[((int64_t)o * fp.cin + k) * fp.ntaps + tap];
            acc += wgt * src * (double)fp.dict[(int64_t)l * G::kk + jj];
        }
        const float v = (float)acc;
        if (is_bias) {
            const __half hi = __float2half_rn(v);
            value = k == 0 ? __half2float(hi) : v - __half2float(hi);
        } else {
            value = v;
        }
    }
    folded[e] = __float2half_rn(value);
}

// ---- host side -------------------------------------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = [] {
        void* f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            f = nullptr;
        return (EncodeTiledFn)f;
    }();
    return fn;
}

struct DeviceInfo { int cc_major = 0, smem_optin = 0; bool ok = false; };

const DeviceInfo& device_info()
{
    static DeviceInfo cache[64];
    static DeviceInfo none;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return none;
    DeviceInfo& d = cache[dev];
    if (!d.ok) {
        if (cudaDeviceGetAttribute(&d.cc_major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return none;
        if (cudaDeviceGetAttribute(&d.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) return none;
        d.ok = true;
    }
    return d;
}

constexpr int kStaticReserve = 4096;   // static shared memory (control block) + the per-CTA system reservation

struct Plan {
    bool ok = false;
    int ntaps = 0, tps = 0, nsteps = 0, stages = 0, passes = 0, resident = 0;
    uint32_t stage_bytes = 0;
    size_t smem = 0;
};

template <int R, int K>
Plan make_plan_rk(const Problem& pb, const ProducerShape& ps)
{
    using G = PG<R, K>;
    Plan pl;
    const DeviceInfo& di = device_info();
    if (!di.ok) return pl;
    pl.ntaps = ps.kc * ps.kc;
    pl.passes = G::G;
    Geom g;
    // the shared memory is planned for three channels whatever the frame has, so that the layout of the folded block
    // (taps per step) depends on scale, k and the layer only, as the header promises
    Problem pb3 = pb;
    pb3.c = kMaxC;
    const size_t geom_floats = plan_geom(g, pb3, G::TH, nullptr, G::TWD);
    const size_t fixed = 1024 /* alignment slack */ + 32 + (size_t)pl.ntaps * kTapBytes + kOnesBytes +
                         (geom_floats + (size_t)kMaxC * g.trows * g.tcols /* second LR window */) * sizeof(float);
    const size_t per_cta = (size_t)di.smem_optin - kStaticReserve;
    // a step = the taps of one kernel row when two such stages fit, else a single tap
    for (int tps = ps.kc; tps >= 1; tps = (tps > 1 ? 1 : 0)) {
        const uint32_t stage_bytes = (uint32_t)(G::BIAS_BYTES + tps * G::TAP_B_BYTES);
        if (fixed + 2 * (size_t)stage_bytes > per_cta) continue;
        int stages = (int)((per_cta - fixed) / stage_bytes);
        if (stages > kMaxStages) stages = kMaxStages;
        pl.ok = true;
        pl.tps = tps;
        pl.nsteps = (pl.ntaps + tps - 1) / tps;
        // when every stage of a tile fits at once the weights stay in shared memory for the CTA's whole life
        if (stages >= G::G * pl.nsteps) { stages = G::G * pl.nsteps; pl.resident = 1; }
        pl.stages = stages;
        pl.stage_bytes = stage_bytes;
        pl.smem = fixed + (size_t)stages * stage_bytes;
        break;
    }
    if (pl.ok && pl.nsteps > kMaxSteps) pl.ok = false;
    return pl;
}

Plan make_plan(const Problem& pb, const ProducerShape& ps)
{
    if (pb.r == 4) {
        if (pb.k == 3) return make_plan_rk<4, 3>(pb, ps);
        if (pb.k == 5) return make_plan_rk<4, 5>(pb, ps);
        if (pb.k == 7) return make_plan_rk<4, 7>(pb, ps);
    } else if (pb.r == 3) {
        if (pb.k == 3) return make_plan_rk<3, 3>(pb, ps);
        if (pb.k == 5) return make_plan_rk<3, 5>(pb, ps);
    } else if (pb.r == 2) {
        if (pb.k == 3) return make_plan_rk<2, 3>(pb, ps);
        if (pb.k == 5) return make_plan_rk<2, 5>(pb, ps);
        if (pb.k == 7) return make_plan_rk<2, 7>(pb, ps);
    }
    return Plan{};
}

template <int R, int K, typename OutT>
cudaError_t launch_rko(const CUtensorMap& map, const ProdParams& prm, const Plan& pl, cudaStream_t st)
{
    auto kern = producer_regress_kernel<R, K, OutT>;
    static bool configured[64] = {false};   // per template instance and device
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, device_info().smem_optin - kStaticReserve);
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    const int ctas = prm.g.num_tiles < sm_count() ? prm.g.num_tiles : sm_count();
    kern<<<ctas, kThreads, pl.smem, st>>>(map, prm);
    count_launches(1);
    return cudaGetLastError();
}

template <int R, int K>
cudaError_t launch_rk(const CUtensorMap& map, const ProdParams& prm, const Plan& pl, cudaStream_t st)
{
    if (prm.g.pb.flags & SR_OUT_U8) return launch_rko<R, K, uint8_t>(map, prm, pl, st);
    if (prm.g.pb.flags & SR_OUT_F16) return launch_rko<R, K, __half>(map, prm, pl, st);
    return launch_rko<R, K, float>(map, prm, pl, st);
}

template <int R, int K>
cudaError_t fold_rk(__half* folded, const FoldParams& fp, cudaStream_t st)
{
    const int threads = 256;
    const int64_t blocks = (fp.total_halves + threads - 1) / threads;
    producer_fold_kernel<R, K><<<(unsigned)blocks, threads, 0, st>>>(folded, fp);
    count_launches(1);
    return cudaGetLastError();
}

} // namespace

bool producer_supported(const Problem& pb, const ProducerShape& ps)
{
    if (ps.cin != kCin || (ps.kc != 1 && ps.kc != 3)) return false;
    if (pb.c > kMaxC || pb.n > 65535) return false;
    if (pb.flags & SR_LUMA_ONLY) return false;
    const DeviceInfo& di = device_info();
    if (!di.ok || di.cc_major != 10 || !encode_fn()) return false;
    return make_plan(pb, ps).ok;
}

size_t producer_folded_bytes(const Problem& pb, const ProducerShape& ps)
{
    if (!producer_supported(pb, ps)) return 0;
    const Plan pl = make_plan(pb, ps);
    return (size_t)pl.passes * pl.nsteps * pl.stage_bytes;
}

cudaError_t launch_producer_fold(const float* wconv, const float* bias, const float* dict, const uint8_t* idx,
                                 const float* gamma, int s, void* folded, const Problem& pb, const ProducerShape& ps,
                                 cudaStream_t st)
{
    const Plan pl = make_plan(pb, ps);
    if (!pl.ok) return cudaErrorNotSupported;
    FoldParams fp{};
    fp.wconv = wconv; fp.bias = bias; fp.dict = dict; fp.idx = idx; fp.gamma = gamma;
    fp.natoms = idx ? s : pb.D;
    fp.D = pb.D; fp.cin = ps.cin; fp.kc = ps.kc; fp.ntaps = pl.ntaps; fp.tps = pl.tps; fp.nsteps = pl.nsteps;
    fp.stage_bytes = pl.stage_bytes;
    fp.total_halves = (int64_t)pl.passes * pl.nsteps * pl.stage_bytes / 2;
    __half* out = static_cast<__half*>(folded);
    if (pb.r == 4) {
        if (pb.k == 3) return fold_rk<4, 3>(out, fp, st);
        if (pb.k == 5) return fold_rk<4, 5>(out, fp, st);
        if (pb.k == 7) return fold_rk<4, 7>(out, fp, st);
    } else if (pb.r == 3) {
        if (pb.k == 3) return fold_rk<3, 3>(out, fp, st);
        if (pb.k == 5) return fold_rk<3, 5>(out, fp, st);
    } else if (pb.r == 2) {
        if (pb.k == 3) return fold_rk<2, 3>(out, fp, st);
        if (pb.k == 5) return fold_rk<2, 5>(out, fp, st);
        if (pb.k == 7) return fold_rk<2, 7>(out, fp, st);
    }
    return cudaErrorNotSupported;
}

cudaError_t launch_producer_regress(const float* lr, const void* feat, const void* folded, void* out, const Problem& pb,
                                    const ProducerShape& ps, cudaStream_t st)
{
    const Plan pl = make_plan(pb, ps);
    if (!pl.ok || !encode_fn()) return cudaErrorNotSupported;
    ProdParams prm{};
    prm.lr = lr; prm.out = out; prm.folded = static_cast<const uint8_t*>(folded);
    prm.status = device_status_word();
    if (!prm.status) return cudaErrorUnknown;
    const int tw = pb.r == 3 ? 126 : TW, tlw = tw / pb.r, tlh = 128 / tlw;   // the tile shape of PG<R, K>
    plan_geom(prm.g, pb, pb.r * tlh, lr, tw);
    prm.kc = ps.kc; prm.ntaps = pl.ntaps; prm.tps = pl.tps; prm.nsteps = pl.nsteps; prm.stages = pl.stages; prm.resident = pl.resident;
    prm.stage_bytes = pl.stage_bytes;
    prm.wait_cycles = wait_cycle_limit();
    prm.inject_lost_arrival = take_injected_lost_arrival() ? 1 : 0;

    // feature map [n][h][w][cin] binary16; a box is 8 channels x the tile's LR columns x its LR rows
    CUtensorMap map{};
    const cuuint64_t dims[4] = {(cuuint64_t)ps.cin, (cuuint64_t)pb.w, (cuuint64_t)pb.h, (cuuint64_t)pb.n};
    const cuuint64_t strides[3] = {(cuuint64_t)ps.cin * 2, (cuuint64_t)pb.w * ps.cin * 2, (cuuint64_t)pb.h * pb.w * ps.cin * 2};
    const cuuint32_t es[4] = {1, 1, 1, 1};
    const cuuint32_t box[4] = {8, (cuuint32_t)tlw, (cuuint32_t)tlh, 1};
    if (encode_fn()(&map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4, const_cast<void*>(feat), dims, strides, box, es,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return cudaErrorInvalidValue;
    if (pb.r == 4) {
        if (pb.k == 3) return launch_rk<4, 3>(map, prm, pl, st);
        if (pb.k == 5) return launch_rk<4, 5>(map, prm, pl, st);
        if (pb.k == 7) return launch_rk<4, 7>(map, prm, pl, st);
    } else if (pb.r == 3) {
        if (pb.k == 3) return launch_rk<3, 3>(map, prm, pl, st);
        if (pb.k == 5) return launch_rk<3, 5>(map, prm, pl, st);
    } else if (pb.r == 2) {
        if (pb.k == 3) return launch_rk<2, 3>(map, prm, pl, st);
        if (pb.k == 5) return launch_rk<2, 5>(map, prm, pl, st);
        if (pb.k == 7) return launch_rk<2, 7>(map, prm, pl, st);
    }
    return cudaErrorNotSupported;
}

} // namespace sr
