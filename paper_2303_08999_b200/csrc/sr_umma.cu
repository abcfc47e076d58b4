// Fused regression kernel for sm_100a: TMA-streamed coefficient planes, dictionary assembly F = Phi D on the
// tcgen05 tensor cores with fp32 accumulators in tensor memory, bicubic tile + patch dot product + clamp in the
// epilogue. The filter matrix F (TMEM / registers), the up-sampled image U and its patches (shared memory) never
// reach HBM: per HR pixel the kernel reads its coefficients once and writes its c output values once.
//
// One persistent CTA per SM walks HR tiles of 128 x 8 pixels. A tile row (128 pixels of one HR row) is one
// pipeline stage: two TMA boxes of [atoms][64 pixels] binary16 land in shared memory in the 128-byte-swizzled
// MN-major layout the tensor core reads directly (pixels are M, atoms are K), so the planar [n][D][H][W]
// coefficient tensor needs no transpose. The dictionary is the B operand (K-major): its fp32 values are split
// into binary16 hi + lo parts (~22 bits kept) that sit side by side along N, so one MMA per 16 atoms reads the
// coefficient stage once and yields both partial filters; the epilogue adds them. N = 2 x (k*k padded to 16).
//
// Shared-memory bandwidth is the scarce on-chip resource here (TMA fill + operand reads + U tile + patch reads),
// so the epilogue keeps a sliding k x k x 3 window of U in registers and reads each U row once per pixel column.
//
// Warp roles (448 threads):
//   warp 0       TMA producer            full[stage]  <- bytes landed        waits empty[stage]
//   warp 1       MMA issuer, TMEM owner  acc_full[a], empty[stage] <- tcgen05.commit; waits full[stage], acc_empty[a]
//   warps 2-9    U producers             bicubic (separable) of the tile + halo into a double-buffered tile
//   warps 10-13  epilogue                TMEM -> registers (one pixel's filter per thread), patch dot, clamp, store
// Every wait is bounded; on expiry the CTA raises its abort flag, sets the device status word and drains.
#include "sr_ptx.cuh"
#include "sr_umma.cuh"

namespace sr {

namespace {

using namespace ptx;

constexpr int TW = 128, TH = 8;
constexpr int kThreads = 448;
constexpr int kFirstUWarp = 2, kNumUWarps = 8, kFirstEpiWarp = 10, kNumEpiWarps = 4;
constexpr int kMaxStages = 8;
constexpr int kMaxAccSlots = 8;
constexpr int kMaxChannels = 4;
constexpr int kStaticReserve = 5120;   // static shared memory (control block) + alignment, kept out of the dynamic budget

struct UmmaParams {
    const float* lr;
    const float* dict;
    float* out;
    const uint8_t* idx;   // global-subset mode: s atom ids
    const float* gamma;   // global-subset mode: s weights or nullptr
    int* status;
    Problem pb;
    int mode;
    int natoms;           // coefficient planes per pixel that enter the contraction (D, or s for a subset)
    int dpad;             // natoms rounded up to a multiple of 16 (the MMA K extent)
    int per_atom_boxes;   // 1: one TMA box per selected atom (subset of a full tensor); 0: one box covers all atoms
    int stages;
    int trows;            // LR rows a tile can need (rows of the horizontal-pass scratch tile)
    int tcols;            // LR columns a tile can need
    uint32_t r_magic;     // ceil(2^32 / r): floor(x / r) == umulhi(x, r_magic) for 0 <= x < 2^29 (r >= 2)
    uint32_t tcols_magic; // same for tcols
    int tiles_x, tiles_y, num_tiles;
};

struct __align__(16) Ctl {
    uint64_t full[kMaxStages], empty[kMaxStages];
    uint64_t acc_full[kMaxAccSlots], acc_empty[kMaxAccSlots];
    uint64_t u_full[2], u_empty[2];
    uint32_t tmem_base;
    int abort_flag;
    float4 vy_w[TH + 2 * 4];   // per U-tile row: its four vertical tap weights
    float4 hx_w[TW + 2 * 4];   // per U-tile column: its four horizontal tap weights
    int vy_off[TH + 2 * 4];    // per U-tile row: first row of the scratch tile it reads
    int hx_off[TW + 2 * 4];    // per U-tile column: first column of the LR window it reads
    uint8_t atoms[256];        // subset mode: the atom id of each selected plane
};

template <int K> struct Geo {
    static constexpr int kk = K * K;
    static constexpr int NPAD = (kk + 15) / 16 * 16;     // taps padded; hi part in columns [0, NPAD), lo in [NPAD, 2 NPAD)
    static constexpr int NB = 2 * NPAD;                  // N of the MMA
    static constexpr int P = (K - 1) / 2;
    static constexpr int UW = TW + 2 * P, UH = TH + 2 * P;
    static constexpr int LBO_B = (NB / 8) * 128;         // bytes between the two K-halves of a K-step of the B operand
    static constexpr int KSTEP_B = 2 * LBO_B;            // bytes per K-step (16 atoms) of the B operand
    static constexpr int ACC_SLOTS = (512 / NB) < kMaxAccSlots ? (512 / NB) : kMaxAccSlots;
    static constexpr int TMEM_COLS = ACC_SLOTS * NB;     // 256 or 512: a power of two
};

__device__ __forceinline__ int fast_div(int x, int d, uint32_t magic) { return d == 1 ? x : (int)__umulhi((uint32_t)x, magic); }

__device__ __forceinline__ void decode_tile(const UmmaParams& p, int t, int& f, int& y0, int& x0, int& rows)
{
    const int tx = t % p.tiles_x;
    const int rest = t / p.tiles_x;
    const int ty = rest % p.tiles_y;
    f = rest / p.tiles_y;
    y0 = ty * TH;
    x0 = tx * TW;
    rows = min(TH, p.pb.H - y0);
}

// LR pixels a tile (plus patch halo) needs for its bicubic taps: rows lr_lo .. lr_lo + nrows - 1 and columns
// col_lo .. col_lo + ncols - 1 (unclamped; reads clamp them to the image).
struct LrWindow { int f, y0, x0, rows, lr_lo, nrows, col_lo, ncols; };

template <int K>
__device__ __forceinline__ void lr_window(const UmmaParams& p, int t, LrWindow& g)
{
    constexpr int P = (K - 1) / 2;
    const Problem& pb = p.pb;
    decode_tile(p, t, g.f, g.y0, g.x0, g.rows);
    const int Ylo = clampi(g.y0 - P, 0, pb.H - 1), Yhi = clampi(g.y0 + g.rows - 1 + P, 0, pb.H - 1);
    const int qylo = fast_div(Ylo, pb.r, p.r_magic), qyhi = fast_div(Yhi, pb.r, p.r_magic);
    g.lr_lo = qylo + pb.ph.base[Ylo - qylo * pb.r];
    g.nrows = qyhi + pb.ph.base[Yhi - qyhi * pb.r] + 3 - g.lr_lo + 1;      // <= trows
    const int Xlo = clampi(g.x0 - P, 0, pb.W - 1), Xhi = clampi(g.x0 + TW - 1 + P, 0, pb.W - 1);
    const int qxlo = fast_div(Xlo, pb.r, p.r_magic), qxhi = fast_div(Xhi, pb.r, p.r_magic);
    g.col_lo = qxlo + pb.ph.base[Xlo - qxlo * pb.r];
    g.ncols = qxhi + pb.ph.base[Xhi - qxhi * pb.r] + 3 - g.col_lo + 1;     // <= tcols
}

__device__ __forceinline__ void cp_async_f32(float* dst_smem, const float* src)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_u32(dst_smem)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void named_barrier_sync(int id, int nthreads)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// Group-wide AND over a named barrier.
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

// One pixel's filter from tensor memory: F[j] = hi[j] + lo[j] for the taps j < k*k (16 columns at a time).
template <int K>
__device__ __forceinline__ void load_filter(uint32_t taddr, float* F)
{
    using G = Geo<K>;
#pragma unroll
    for (int j0 = 0; j0 < G::NPAD; j0 += 16) {
        if (j0 < G::kk) {
            float h[16], l[16];
            tmem_ld_x16(taddr + j0, h);
            tmem_ld_x16(taddr + G::NPAD + j0, l);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 16; ++i) F[j0 + i] = h[i] + l[i];
        }
    }
}

// y_c = F . B_c for NC channels of one pixel, patch read tap by tap from the shared U tile. Independent
// accumulators per channel and patch-row parity keep the FMA pipe busy instead of one serial chain.
template <int K, int NC>
__device__ __forceinline__ void patch_dot(const float* F, const float* u, int ch_stride, int row_stride, float* dst,
                                          int64_t dst_ch_stride, bool store, bool clamp01)
{
    float acc[NC][2];
#pragma unroll
    for (int c = 0; c < NC; ++c) acc[c][0] = acc[c][1] = 0.f;
#pragma unroll
    for (int a = 0; a < K; ++a)
#pragma unroll
        for (int b = 0; b < K; ++b)
#pragma unroll
            for (int c = 0; c < NC; ++c) acc[c][a & 1] = fmaf(F[a * K + b], u[c * ch_stride + a * row_stride + b], acc[c][a & 1]);
#pragma unroll
    for (int c = 0; c < NC; ++c) {
        float v = acc[c][0] + acc[c][1];
        if (clamp01) v = fminf(fmaxf(v, 0.f), 1.f);
        if (store) dst[c * dst_ch_stride] = v;
    }
}

// Optional role timing (build with -DSR_PROFILE_ROLES): cycles each role spends in total and inside waits,
// written per CTA to the buffer registered with sr_debug_role_profile.
#ifdef SR_PROFILE_ROLES
__device__ long long* g_role_prof = nullptr;
#define PROF_DECL long long prof_t0 = clock64(), prof_wait = 0, prof_tw = 0, prof_mma = 0, prof_commit = 0; bool prof_tmp_ok = true;
#define PROF_WAIT(expr) (prof_tw = clock64(), prof_tmp_ok = (expr), prof_wait += clock64() - prof_tw, prof_tmp_ok)
#define PROF_T(var) long long var = clock64();
#define PROF_ADD(acc, t0) acc += clock64() - (t0);
#define PROF_STORE2(role, a, b) if (g_role_prof) { g_role_prof[(blockIdx.x * 32 + (role)) * 2] = (a); g_role_prof[(blockIdx.x * 32 + (role)) * 2 + 1] = (b); }
#define PROF_STORE(role) if (g_role_prof && lane == 0) { g_role_prof[(blockIdx.x * 32 + (role)) * 2] = clock64() - prof_t0; g_role_prof[(blockIdx.x * 32 + (role)) * 2 + 1] = prof_wait; }
#else
#define PROF_DECL
#define PROF_WAIT(expr) (expr)
#define PROF_STORE(role)
#define PROF_T(var)
#define PROF_ADD(acc, t0)
#define PROF_STORE2(role, a, b)
#endif

template <int K>
__global__ void __launch_bounds__(kThreads, 1)
regress_umma_kernel(const __grid_constant__ CUtensorMap map_all, const __grid_constant__ CUtensorMap map_row,
                    const __grid_constant__ UmmaParams p)
{
    using G = Geo<K>;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    __shared__ Ctl ctl;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const Problem& pb = p.pb;
    const int C = pb.c;
    const int stage_bytes = p.dpad * 256;            // two chunks of [dpad][64 pixels] binary16
    const int chunk_bytes = p.dpad * 128;
    const int ksteps = p.dpad / 16;

    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* sA = smem;
    uint8_t* sB = sA + (size_t)p.stages * stage_bytes;
    float* sU = reinterpret_cast<float*>(sB + (size_t)ksteps * G::KSTEP_B);            // [2][C][UH][UW]
    float* sT = sU + 2 * C * G::UH * G::UW;                                           // [C * trows][UW]
    float* sL = sT + C * p.trows * G::UW;                                             // [2][C * trows][tcols]

    // ---------------------------------------------------------------- set-up
    if (tid == 0) {
        for (int i = 0; i < kMaxStages; ++i) { mbar_init(&ctl.full[i], 1); mbar_init(&ctl.empty[i], 1); }
        for (int i = 0; i < kMaxAccSlots; ++i) { mbar_init(&ctl.acc_full[i], 1); mbar_init(&ctl.acc_empty[i], kNumEpiWarps * 32); }
        for (int i = 0; i < 2; ++i) { mbar_init(&ctl.u_full[i], kNumUWarps * 32); mbar_init(&ctl.u_empty[i], kNumEpiWarps * 32); }
        ctl.abort_flag = 0;
        fence_barrier_init();
        prefetch_tensormap(&map_all);
        prefetch_tensormap(&map_row);
    }
    // B operand: dict (or gamma-weighted subset rows) as binary16 hi | lo along N, K-major, no swizzle.
    // element (column n, atom k) of a K-step: (k%16)/8 * LBO + n/8 * 128 + n%8 * 16 + k%8 * 2
    for (int i = tid; i < p.dpad * G::NPAD; i += kThreads) {
        const int k = i / G::NPAD, n = i - k * G::NPAD;
        float v = 0.f;
        if (k < p.natoms && n < G::kk) {
            if (p.mode == kModeGlobal) {
                const int a = min((int)__ldg(p.idx + k), pb.D - 1);
                v = __ldg(p.dict + (int64_t)a * G::kk + n) * (p.gamma ? __ldg(p.gamma + k) : 1.f);
            } else {
                v = __ldg(p.dict + (int64_t)k * G::kk + n);
            }
        }
        const __half hi = __float2half_rn(v);
        const __half lo = __float2half_rn(v - __half2float(hi));
        const int base = (k >> 4) * G::KSTEP_B + ((k & 15) >> 3) * G::LBO_B + (k & 7) * 2;
        const int nl = n + G::NPAD;
        *reinterpret_cast<__half*>(sB + base + (n >> 3) * 128 + (n & 7) * 16) = hi;
        *reinterpret_cast<__half*>(sB + base + (nl >> 3) * 128 + (nl & 7) * 16) = lo;
    }
    if (p.per_atom_boxes)
        for (int q = tid; q < p.natoms; q += kThreads) ctl.atoms[q] = (uint8_t)min((int)__ldg(p.idx + q), pb.D - 1);
    // Rows of the A stages that no TMA box writes (subset mode: atoms natoms..dpad-1) must read as zero.
    if (p.per_atom_boxes) {
        uint4* a4 = reinterpret_cast<uint4*>(sA);
        const int n16 = p.stages * stage_bytes / 16;
        for (int i = tid; i < n16; i += kThreads) a4[i] = make_uint4(0, 0, 0, 0);
    }
    fence_proxy_async_smem();
    __syncwarp();
    if (warp == 1) tmem_alloc(&ctl.tmem_base, G::TMEM_COLS);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = ctl.tmem_base;
    volatile int* abort_flag = &ctl.abort_flag;
    PROF_DECL

    // ---------------------------------------------------------------- roles
    if (warp == 0) {
        // ===== TMA producer
        if (lane == 0) {
            uint32_t it = 0;
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < p.num_tiles && ok; t += gridDim.x) {
                int f, y0, x0, rows;
                decode_tile(p, t, f, y0, x0, rows);
                for (int r = 0; r < rows; ++r, ++it) {
                    if (!(ok = PROF_WAIT(mbar_wait(&ctl.empty[s], ph ^ 1, abort_flag)))) break;
                    uint8_t* dst = sA + (size_t)s * stage_bytes;
                    if (!p.per_atom_boxes) {
                        mbar_arrive_expect_tx(&ctl.full[s], stage_bytes);
                        tma_load_4d(dst, &map_all, &ctl.full[s], x0, y0 + r, 0, f);
                        tma_load_4d(dst + chunk_bytes, &map_all, &ctl.full[s], x0 + 64, y0 + r, 0, f);
                    } else {
                        mbar_arrive_expect_tx(&ctl.full[s], p.natoms * 256);
                        for (int q = 0; q < p.natoms; ++q) {
                            const int a = ctl.atoms[q];
                            tma_load_4d(dst + q * 128, &map_row, &ctl.full[s], x0, y0 + r, a, f);
                            tma_load_4d(dst + chunk_bytes + q * 128, &map_row, &ctl.full[s], x0 + 64, y0 + r, a, f);
                        }
                    }
                    if (++s == p.stages) { s = 0; ph ^= 1; }
                }
            }
            PROF_STORE(0)
            // drain: every load issued has either been consumed or is waited for here (bounded)
            if (!ok) {
                const uint32_t n = it < (uint32_t)p.stages ? it : (uint32_t)p.stages;
                for (uint32_t j = 0; j < n; ++j) {
                    const uint32_t last = it - 1 - j;   // the most recent use of stage last % stages
                    const long long t0 = clock64();
                    while (!mbar_try_wait(&ctl.full[last % p.stages], (last / p.stages) & 1) && clock64() - t0 < (1ll << 27)) {}
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ===== MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc_f16(128, G::NB, /*a_mn_major=*/true, /*b_mn_major=*/false);
            // A: MN-major, 128-byte swizzle: 8 atoms x 64 pixels per 1024-byte atom; K-groups 1024 B apart (SBO),
            // the second 64-pixel chunk chunk_bytes away (LBO). A K-step of 16 atoms is 2048 B further on.
            // Only the 14-bit start-address field (units of 16 B) changes between stages and K-steps.
            const uint64_t a_desc0 = make_smem_desc(smem_u32(sA), chunk_bytes, 1024, kSwizzle128B);
            const uint64_t b_desc0 = make_smem_desc(smem_u32(sB), G::LBO_B, 128, kSwizzleNone);
            const uint32_t a_stage_step = (uint32_t)stage_bytes >> 4;
            uint32_t it = 0;
            int s = 0, a = 0;
            uint32_t ph = 0, aph = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < p.num_tiles && ok; t += gridDim.x) {
                int f, y0, x0, rows;
                decode_tile(p, t, f, y0, x0, rows);
                for (int r = 0; r < rows; ++r, ++it) {
                    if (!(ok = PROF_WAIT(mbar_wait(&ctl.acc_empty[a], aph ^ 1, abort_flag)))) break;
                    if (!(ok = PROF_WAIT(mbar_wait(&ctl.full[s], ph, abort_flag)))) break;
                    tc_fence_after_sync();
                    const uint32_t taddr = tmem_base + (uint32_t)(a * G::NB);
                    uint64_t ad = a_desc0 + (uint64_t)((uint32_t)s * a_stage_step);
                    uint64_t bd = b_desc0;
                    PROF_T(tm0)
                    for (int ks = 0; ks < ksteps; ++ks) {
                        mma_f16_ss(taddr, ad, bd, idesc, ks > 0);
                        ad += 2048 >> 4;
                        bd += G::KSTEP_B >> 4;
                    }
                    PROF_ADD(prof_mma, tm0)
                    PROF_T(tc0)
                    mma_commit(&ctl.empty[s]);       // the stage may be refilled once these MMAs have read it
                    mma_commit(&ctl.acc_full[a]);    // and the accumulator is complete
                    PROF_ADD(prof_commit, tc0)
                    if (++s == p.stages) { s = 0; ph ^= 1; }
                    if (++a == G::ACC_SLOTS) { a = 0; aph ^= 1; }
                }
            }
            PROF_STORE(1)
            PROF_STORE2(20, prof_mma, prof_commit)
        }
        __syncwarp();
    } else if (warp < kFirstEpiWarp) {
        // ===== U producers: separable bicubic of the tile + halo (clamped HR coordinates), fp32.
        // The LR window of the NEXT tile is fetched with cp.async while this tile is computed. Work is
        // flattened to one output value per loop trip so that every thread of the group stays busy.
        const int ut = tid - kFirstUWarp * 32;
        constexpr int NU = kNumUWarps * 32;
        const int lbuf_floats = C * p.trows * p.tcols;
        auto prefetch_lr = [&](int t, int buf) {
            LrWindow g;
            lr_window<K>(p, t, g);
            float* dstL = sL + buf * lbuf_floats;
            const int total = C * g.nrows * p.tcols;      // rows flattened as ch * nrows + j, pitch tcols
            for (int e = ut; e < total; e += NU) {
                const int row = fast_div(e, p.tcols, p.tcols_magic), i = e - row * p.tcols;
                if (i < g.ncols) {
                    const int ch = (row >= g.nrows) + (row >= 2 * g.nrows) + (row >= 3 * g.nrows);
                    const int j = row - ch * g.nrows;
                    const float* src = p.lr + (((int64_t)g.f * C + ch) * pb.h + clampi(g.lr_lo + j, 0, pb.h - 1)) * pb.w +
                                       clampi(g.col_lo + i, 0, pb.w - 1);
                    cp_async_f32(dstL + e, src);
                }
            }
            cp_async_commit();
        };
        uint32_t ti = 0;
        if ((int)blockIdx.x < p.num_tiles) prefetch_lr(blockIdx.x, 0);
        for (int t = blockIdx.x; t < p.num_tiles; t += gridDim.x, ++ti) {
            LrWindow g;
            lr_window<K>(p, t, g);
            const int ub = ti & 1;
            const uint32_t uph = (ti >> 1) & 1;
            const bool has_next = t + (int)gridDim.x < p.num_tiles;
            // every thread is past the previous tile's passes before its LR buffer, scratch and tables are reused
            bool ok = PROF_WAIT(mbar_wait(&ctl.u_empty[ub], uph ^ 1, abort_flag));
            ok = named_barrier_and(1, NU, ok);
            if (!ok) break;
            if (has_next) prefetch_lr(t + gridDim.x, (ti + 1) & 1);
            const int uh = g.rows + 2 * G::P;
            if (ut < G::UW) {
                const int Xc = clampi(g.x0 - G::P + ut, 0, pb.W - 1);
                const int q = fast_div(Xc, pb.r, p.r_magic), px = Xc - q * pb.r;
                ctl.hx_off[ut] = q + pb.ph.base[px] - g.col_lo;
                ctl.hx_w[ut] = make_float4(pb.ph.w[px][0], pb.ph.w[px][1], pb.ph.w[px][2], pb.ph.w[px][3]);
            } else if (ut - G::UW < uh) {
                const int uy = ut - G::UW;
                const int Yc = clampi(g.y0 - G::P + uy, 0, pb.H - 1);
                const int q = fast_div(Yc, pb.r, p.r_magic), py = Yc - q * pb.r;
                ctl.vy_off[uy] = q + pb.ph.base[py] - g.lr_lo;
                ctl.vy_w[uy] = make_float4(pb.ph.w[py][0], pb.ph.w[py][1], pb.ph.w[py][2], pb.ph.w[py][3]);
            }
            if (has_next) cp_async_wait<1>(); else cp_async_wait<0>();
            named_barrier_sync(1, NU);                       // tables written, this tile's LR window landed
            // horizontal pass: T[row][ux] = sum_b wx[b] * L[row][hx_off[ux] + b], row = ch * nrows + j
            const float* Lb = sL + (ti & 1) * lbuf_floats;
            const int hrows = C * g.nrows;
#pragma unroll 2
            for (int o = ut; o < hrows * G::UW; o += NU) {
                const int row = o / G::UW, ux = o - row * G::UW;
                const float4 w = ctl.hx_w[ux];
                const float* src = Lb + row * p.tcols + ctl.hx_off[ux];
                float v = w.x * src[0];
                v = fmaf(w.y, src[1], v);
                v = fmaf(w.z, src[2], v);
                v = fmaf(w.w, src[3], v);
                sT[o] = v;
            }
            named_barrier_sync(1, NU);
            // vertical pass: U[ch][uy][ux] = sum_a wy[a] * T[ch * nrows + vy_off[uy] + a][ux]
            float* Ub = sU + ub * C * G::UH * G::UW;
            for (int ch = 0; ch < C; ++ch) {
                const float* Tc = sT + ch * g.nrows * G::UW;
                float* Uc = Ub + ch * G::UH * G::UW;
#pragma unroll 2
                for (int o = ut; o < uh * G::UW; o += NU) {
                    const int uy = o / G::UW, ux = o - uy * G::UW;
                    const float4 w = ctl.vy_w[uy];
                    const float* src = Tc + ctl.vy_off[uy] * G::UW + ux;
                    float v = w.x * src[0];
                    v = fmaf(w.y, src[G::UW], v);
                    v = fmaf(w.z, src[2 * G::UW], v);
                    v = fmaf(w.w, src[3 * G::UW], v);
                    Uc[o] = v;
                }
            }
            mbar_arrive(&ctl.u_full[ub]);
        }
        cp_async_wait<0>();
        PROF_STORE(warp)
    } else {
        // ===== epilogue: thread = one pixel column of the tile (TMEM lane), rows in order
        const int quarter = warp & 3;                        // the TMEM lanes this warp may read: 32*quarter..+31
        const int x = quarter * 32 + lane;                   // pixel within the tile row
        const int64_t HW = (int64_t)pb.H * pb.W;
        const bool clamp01 = (pb.flags & SR_CLAMP01) != 0;
        uint32_t it = 0, ti = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < p.num_tiles && ok; t += gridDim.x, ++ti) {
            int f, y0, x0, rows;
            decode_tile(p, t, f, y0, x0, rows);
            const int ub = ti & 1;
            const uint32_t uph = (ti >> 1) & 1;
            ok = PROF_WAIT(__all_sync(0xffffffffu, mbar_wait(&ctl.u_full[ub], uph, abort_flag)));
            if (!ok) break;
            const float* Ub = sU + ub * C * G::UH * G::UW;
            const bool in_x = x0 + x < pb.W;
            float* dst0 = p.out + ((int64_t)f * C) * HW + (int64_t)y0 * pb.W + x0 + x;
            if (K <= 5 && C == 3) {
                // sliding window: the k x k x 3 patch lives in registers; each new row costs 3k shared loads
                float win[3][K][K];
                const float* u0 = Ub + x;
#pragma unroll
                for (int a = 0; a < K - 1; ++a)
#pragma unroll
                    for (int c = 0; c < 3; ++c)
#pragma unroll
                        for (int b = 0; b < K; ++b) win[c][a][b] = u0[(c * G::UH + a) * G::UW + b];
#pragma unroll
                for (int r = 0; r < TH; ++r) {
                    if (r < rows && ok) {
#pragma unroll
                        for (int c = 0; c < 3; ++c)
#pragma unroll
                            for (int b = 0; b < K; ++b) win[c][(r + K - 1) % K][b] = u0[(c * G::UH + r + K - 1) * G::UW + b];
                        const int a_slot = it % G::ACC_SLOTS;
                        const uint32_t aph = (it / G::ACC_SLOTS) & 1;
                        ok = PROF_WAIT(__all_sync(0xffffffffu, mbar_wait(&ctl.acc_full[a_slot], aph, abort_flag)));
                        if (ok) {
                            tc_fence_after_sync();
                            float F[G::NPAD];
                            load_filter<K>(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(a_slot * G::NB), F);
                            tc_fence_before_sync();
                            mbar_arrive(&ctl.acc_empty[a_slot]);
                            float acc[3][2];
#pragma unroll
                            for (int c = 0; c < 3; ++c) acc[c][0] = acc[c][1] = 0.f;
#pragma unroll
                            for (int a = 0; a < K; ++a)
#pragma unroll
                                for (int b = 0; b < K; ++b)
#pragma unroll
                                    for (int c = 0; c < 3; ++c)
                                        acc[c][a & 1] = fmaf(F[a * K + b], win[c][(r + a) % K][b], acc[c][a & 1]);
#pragma unroll
                            for (int c = 0; c < 3; ++c) {
                                float v = acc[c][0] + acc[c][1];
                                if (clamp01) v = fminf(fmaxf(v, 0.f), 1.f);
                                if (in_x) dst0[c * HW + (int64_t)r * pb.W] = v;
                            }
                        }
                        ++it;
                    }
                }
            } else {
                for (int r = 0; r < rows; ++r, ++it) {
                    const int a_slot = it % G::ACC_SLOTS;
                    const uint32_t aph = (it / G::ACC_SLOTS) & 1;
                    ok = PROF_WAIT(__all_sync(0xffffffffu, mbar_wait(&ctl.acc_full[a_slot], aph, abort_flag)));
                    if (!ok) break;
                    tc_fence_after_sync();
                    float F[G::NPAD];
                    load_filter<K>(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(a_slot * G::NB), F);
                    tc_fence_before_sync();
                    mbar_arrive(&ctl.acc_empty[a_slot]);
                    float* dst = dst0 + (int64_t)r * pb.W;
                    const float* u0 = Ub + r * G::UW + x;
                    if (C == 3) {
                        patch_dot<K, 3>(F, u0, G::UH * G::UW, G::UW, dst, HW, in_x, clamp01);
                    } else {
                        for (int ch = 0; ch < C; ++ch)
                            patch_dot<K, 1>(F, u0 + ch * G::UH * G::UW, G::UH * G::UW, G::UW, dst + ch * HW, HW, in_x, clamp01);
                    }
                }
            }
            if (ok) mbar_arrive(&ctl.u_empty[ub]);
        }
        PROF_STORE(warp)
    }

    // ---------------------------------------------------------------- teardown
    __syncwarp();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (ctl.abort_flag && tid == 0) atomicExch(p.status, SR_ERR_TIMEOUT);
    if (warp == 1) tmem_dealloc(tmem_base, G::TMEM_COLS);
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

int trows_for(int k, int r) { return (TH + (k - 1) - 1) / r + 5; }
int tcols_for(int k, int r) { return (TW + (k - 1) - 1) / r + 5; }

template <int K> size_t fixed_smem_bytes(int c, int dpad, int r)
{
    using G = Geo<K>;
    const int trows = trows_for(K, r), tcols = tcols_for(K, r);
    return 1024 /* alignment slack */ + (size_t)(dpad / 16) * G::KSTEP_B +
           (size_t)(2 * c * G::UH * G::UW + c * trows * G::UW + 2 * c * trows * tcols) * sizeof(float);
}

// planes that enter the contraction, and whether they are picked one by one out of a full tensor
void contraction_shape(int mode, const Problem& pb, int& natoms, int& per_atom)
{
    if (mode == kModeGlobal) {
        natoms = pb.s;
        per_atom = (pb.flags & SR_COEF_COMPACT) ? 0 : 1;
    } else {
        natoms = pb.D;
        per_atom = 0;
    }
}

template <int K> int stages_for(int c, int dpad, int r, int smem_optin)
{
    const size_t fixed = fixed_smem_bytes<K>(c, dpad, r) + kStaticReserve;
    if (fixed >= (size_t)smem_optin) return 0;
    const int s = (int)(((size_t)smem_optin - fixed) / ((size_t)dpad * 256));
    return s > kMaxStages ? kMaxStages : s;
}

int stages_for_k(int k, int c, int dpad, int r, int smem_optin)
{
    switch (k) {
    case 1: return stages_for<1>(c, dpad, r, smem_optin);
    case 3: return stages_for<3>(c, dpad, r, smem_optin);
    case 5: return stages_for<5>(c, dpad, r, smem_optin);
    case 7: return stages_for<7>(c, dpad, r, smem_optin);
    default: return 0;
    }
}

template <int K>
cudaError_t launch_k(const CUtensorMap& map_all, const CUtensorMap& map_row, UmmaParams& prm, cudaStream_t st)
{
    const DeviceInfo& di = device_info();
    const size_t smem = fixed_smem_bytes<K>(prm.pb.c, prm.dpad, prm.pb.r) + (size_t)prm.stages * prm.dpad * 256;
    auto kern = regress_umma_kernel<K>;
    static bool configured[64] = {false};   // per template instance and device; the maximum is requested once
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, di.smem_optin - kStaticReserve);
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    const int grid = prm.num_tiles < di.sms ? prm.num_tiles : di.sms;
    kern<<<grid, kThreads, smem, st>>>(map_all, map_row, prm);
    count_launches(1);
    return cudaGetLastError();
}

} // namespace

#ifdef SR_PROFILE_ROLES
extern "C" int sr_debug_role_profile(long long* device_buffer)
{
    return cudaMemcpyToSymbol(g_role_prof, &device_buffer, sizeof(device_buffer)) == cudaSuccess ? 0 : 5;
}
#endif

bool umma_supported(int mode, const void* coef, int coef_dtype, const Problem& pb)
{
    if (mode != kModeDense && mode != kModeGlobal) return false;
    if (coef_dtype != SR_F16) return false;
    if (pb.k > 7 || pb.c > kMaxChannels) return false;
    if ((reinterpret_cast<uintptr_t>(coef) & 15) != 0 || (pb.W & 7) != 0) return false;   // TMA: 16-byte base and pitches
    if (pb.n > 65535) return false;
    const DeviceInfo& di = device_info();
    if (!di.ok || di.cc_major != 10 || !encode_fn()) return false;
    int natoms, per_atom;
    contraction_shape(mode, pb, natoms, per_atom);
    const int dpad = (natoms + 15) / 16 * 16;
    return stages_for_k(pb.k, pb.c, dpad, pb.r, di.smem_optin) >= 2;
}

cudaError_t launch_regress_umma(int mode, const float* lr, const void* coef, const uint8_t* idx, const float* gamma,
                                const float* dict, float* out, const Problem& pb, cudaStream_t st)
{
    const DeviceInfo& di = device_info();
    UmmaParams prm{};
    prm.lr = lr; prm.dict = dict; prm.out = out; prm.idx = idx; prm.gamma = gamma;
    prm.status = device_status_word();
    if (!prm.status) return cudaErrorUnknown;
    prm.pb = pb;
    prm.mode = mode;
    contraction_shape(mode, pb, prm.natoms, prm.per_atom_boxes);
    prm.dpad = (prm.natoms + 15) / 16 * 16;
    prm.stages = stages_for_k(pb.k, pb.c, prm.dpad, pb.r, di.smem_optin);
    prm.trows = trows_for(pb.k, pb.r);
    prm.tcols = tcols_for(pb.k, pb.r);
    prm.r_magic = pb.r > 1 ? (uint32_t)((0x100000000ull + pb.r - 1) / pb.r) : 0u;
    prm.tcols_magic = (uint32_t)((0x100000000ull + prm.tcols - 1) / prm.tcols);
    prm.tiles_x = (pb.W + TW - 1) / TW;
    prm.tiles_y = (pb.H + TH - 1) / TH;
    prm.num_tiles = prm.tiles_x * prm.tiles_y * pb.n;

    // coefficient tensor as seen by TMA: (W, H, planes, n) binary16, innermost first
    const int planes = (mode == kModeGlobal && (pb.flags & SR_COEF_COMPACT)) ? pb.s : pb.D;
    const cuuint64_t dims[4] = {(cuuint64_t)pb.W, (cuuint64_t)pb.H, (cuuint64_t)planes, (cuuint64_t)pb.n};
    const cuuint64_t strides[3] = {(cuuint64_t)pb.W * 2, (cuuint64_t)pb.W * pb.H * 2, (cuuint64_t)pb.W * pb.H * 2 * planes};
    const cuuint32_t es[4] = {1, 1, 1, 1};
    const cuuint32_t box_all[4] = {64, 1, (cuuint32_t)prm.dpad, 1};
    const cuuint32_t box_row[4] = {64, 1, 1, 1};
    CUtensorMap map_all, map_row;
    EncodeTiledFn enc = encode_fn();
    if (enc(&map_all, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4, const_cast<void*>(coef), dims, strides, box_all, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return cudaErrorInvalidValue;
    if (enc(&map_row, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4, const_cast<void*>(coef), dims, strides, box_row, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return cudaErrorInvalidValue;

    switch (pb.k) {
    case 1: return launch_k<1>(map_all, map_row, prm, st);
    case 3: return launch_k<3>(map_all, map_row, prm, st);
    case 5: return launch_k<5>(map_all, map_row, prm, st);
    case 7: return launch_k<7>(map_all, map_row, prm, st);
    default: return cudaErrorNotSupported;
    }
}

} // namespace sr
