// Fused regression kernel for sm_100a: TMA-streamed coefficient planes, dictionary assembly F = Phi D on the
// tcgen05 tensor cores with fp32 accumulators in tensor memory, bicubic tile + patch dot product + clamp in the
// epilogue. The filter matrix F (TMEM / registers), the up-sampled image U and its patches (shared memory) never
// reach HBM: per HR pixel the kernel reads its coefficients once and writes its c output values once.
//
// One persistent CTA per SM walks HR tiles of 128 x 8 pixels. A tile row (128 pixels of one HR row) is one
// pipeline stage: two TMA boxes of [atoms][64 pixels] binary16 land in shared memory in the 128-byte-swizzled
// MN-major layout the tensor core reads directly (pixels are M, atoms are K), so the planar [n][D][H][W]
// coefficient tensor needs no transpose. The dictionary (K-major, split into binary16 hi + lo parts so that its
// fp32 values keep ~22 bits) is the B operand: N = k*k taps padded to a multiple of 16.
//
// Warp roles (448 threads):
//   warp 0      TMA producer            full[stage]  <- bytes landed        waits empty[stage]
//   warp 1      MMA issuer, TMEM owner  acc_full[a], empty[stage] <- tcgen05.commit; waits full[stage], acc_empty[a]
//   warps 2-5   U producers             bicubic (separable) of the tile + halo into a double-buffered tile
//   warps 6-13  epilogue (2 x 4 warps)  TMEM -> registers (one pixel's filter per thread), patch dot, clamp, store
// Every wait is bounded; on expiry the CTA raises its abort flag, sets the device status word and drains.
#include "sr_ptx.cuh"
#include "sr_umma.cuh"

namespace sr {

namespace {

using namespace ptx;

constexpr int TW = 128, TH = 8;
constexpr int kThreads = 448;
constexpr int kFirstUWarp = 2, kNumUWarps = 4, kFirstEpiWarp = 6, kNumEpiWarps = 8;
constexpr int kAccSlots = 8;
constexpr int kMaxStages = 8;
constexpr int kMaxChannels = 4;
constexpr int kStaticReserve = 2048;   // static shared memory (control block) + alignment, kept out of the dynamic budget

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
    int trows;            // rows of the horizontal-pass scratch tile
    int tiles_x, tiles_y, num_tiles;
};

struct __align__(8) Ctl {
    uint64_t full[kMaxStages], empty[kMaxStages];
    uint64_t acc_full[kAccSlots], acc_empty[kAccSlots];
    uint64_t u_full[2], u_empty[2];
    uint32_t tmem_base;
    int abort_flag;
    int vy_row[TH + 2 * 4];    // per U-tile row: first row of the scratch tile it reads
    int vy_phase[TH + 2 * 4];  // and its vertical phase
};

template <int K> struct Geo {
    static constexpr int kk = K * K;
    static constexpr int NPAD = (kk + 15) / 16 * 16;
    static constexpr int P = (K - 1) / 2;
    static constexpr int UW = TW + 2 * P, UH = TH + 2 * P;
    static constexpr int LBO_B = (NPAD / 8) * 128;   // bytes between the two K-halves of a K-step of the B operand
    static constexpr int KSTEP_B = 2 * LBO_B;        // bytes per K-step (16 atoms) of the B operand
    static constexpr int TMEM_COLS = kAccSlots * NPAD;   // 128, 256 or 512: a power of two
};

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
    uint8_t* sBhi = sA + (size_t)p.stages * stage_bytes;
    uint8_t* sBlo = sBhi + (size_t)ksteps * G::KSTEP_B;
    float* sU = reinterpret_cast<float*>(sBlo + (size_t)ksteps * G::KSTEP_B);        // [2][C][UH][UW]
    float* sT = sU + 2 * C * G::UH * G::UW;                                           // [C][trows][UW]

    // ---------------------------------------------------------------- set-up
    if (tid == 0) {
        for (int i = 0; i < kMaxStages; ++i) { mbar_init(&ctl.full[i], 1); mbar_init(&ctl.empty[i], 1); }
        for (int i = 0; i < kAccSlots; ++i) { mbar_init(&ctl.acc_full[i], 1); mbar_init(&ctl.acc_empty[i], 128); }
        for (int i = 0; i < 2; ++i) { mbar_init(&ctl.u_full[i], kNumUWarps * 32); mbar_init(&ctl.u_empty[i], kNumEpiWarps * 32); }
        ctl.abort_flag = 0;
        fence_barrier_init();
        prefetch_tensormap(&map_all);
        prefetch_tensormap(&map_row);
    }
    // B operand: dict (or gamma-weighted subset rows) as binary16 hi + lo, K-major, no swizzle.
    // element (tap n, atom k) of a K-step: (k%16)/8 * LBO + n/8 * 128 + n%8 * 16 + k%8 * 2
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
        const int off = (k >> 4) * G::KSTEP_B + ((k & 15) >> 3) * G::LBO_B + (n >> 3) * 128 + (n & 7) * 16 + (k & 7) * 2;
        *reinterpret_cast<__half*>(sBhi + off) = hi;
        *reinterpret_cast<__half*>(sBlo + off) = lo;
    }
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

    // ---------------------------------------------------------------- roles
    if (warp == 0) {
        // ===== TMA producer
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < p.num_tiles && ok; t += gridDim.x) {
                int f, y0, x0, rows;
                decode_tile(p, t, f, y0, x0, rows);
                for (int r = 0; r < rows; ++r, ++it) {
                    const int s = it % p.stages;
                    const uint32_t ph = (it / p.stages) & 1;
                    if (!(ok = mbar_wait(&ctl.empty[s], ph ^ 1, abort_flag))) break;
                    uint8_t* dst = sA + (size_t)s * stage_bytes;
                    if (!p.per_atom_boxes) {
                        mbar_arrive_expect_tx(&ctl.full[s], stage_bytes);
                        tma_load_4d(dst, &map_all, &ctl.full[s], x0, y0 + r, 0, f);
                        tma_load_4d(dst + chunk_bytes, &map_all, &ctl.full[s], x0 + 64, y0 + r, 0, f);
                    } else {
                        mbar_arrive_expect_tx(&ctl.full[s], p.natoms * 256);
                        for (int q = 0; q < p.natoms; ++q) {
                            const int a = min((int)__ldg(p.idx + q), pb.D - 1);
                            tma_load_4d(dst + q * 128, &map_row, &ctl.full[s], x0, y0 + r, a, f);
                            tma_load_4d(dst + chunk_bytes + q * 128, &map_row, &ctl.full[s], x0 + 64, y0 + r, a, f);
                        }
                    }
                }
            }
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
            constexpr uint32_t idesc = make_idesc_f16(128, G::NPAD, /*a_mn_major=*/true, /*b_mn_major=*/false);
            uint32_t it = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < p.num_tiles && ok; t += gridDim.x) {
                int f, y0, x0, rows;
                decode_tile(p, t, f, y0, x0, rows);
                for (int r = 0; r < rows; ++r, ++it) {
                    const int s = it % p.stages;
                    const uint32_t ph = (it / p.stages) & 1;
                    const int a = it % kAccSlots;
                    const uint32_t aph = (it / kAccSlots) & 1;
                    if (!(ok = mbar_wait(&ctl.acc_empty[a], aph ^ 1, abort_flag))) break;
                    if (!(ok = mbar_wait(&ctl.full[s], ph, abort_flag))) break;
                    tc_fence_after_sync();
                    const uint32_t a_addr = smem_u32(sA + (size_t)s * stage_bytes);
                    const uint32_t taddr = tmem_base + (uint32_t)(a * G::NPAD);
                    for (int ks = 0; ks < ksteps; ++ks) {
                        // A: MN-major, 128-byte swizzle: 8 atoms x 64 pixels per 1024-byte atom; K-groups 1024 B apart
                        // (SBO), the second 64-pixel chunk chunk_bytes away (LBO). A K-step of 16 atoms is 2048 B.
                        const uint64_t ad = make_smem_desc(a_addr + ks * 2048, chunk_bytes, 1024, kSwizzle128B);
                        const uint64_t bh = make_smem_desc(smem_u32(sBhi) + ks * G::KSTEP_B, G::LBO_B, 128, kSwizzleNone);
                        const uint64_t bl = make_smem_desc(smem_u32(sBlo) + ks * G::KSTEP_B, G::LBO_B, 128, kSwizzleNone);
                        mma_f16_ss(taddr, ad, bh, idesc, ks > 0);
                        mma_f16_ss(taddr, ad, bl, idesc, 1u);
                    }
                    mma_commit(&ctl.empty[s]);       // the stage may be refilled once these MMAs have read it
                    mma_commit(&ctl.acc_full[a]);    // and the accumulator is complete
                }
            }
        }
        __syncwarp();
    } else if (warp < kFirstEpiWarp) {
        // ===== U producers: separable bicubic of the tile + halo (clamped HR coordinates), fp32
        const int ut = tid - kFirstUWarp * 32;               // 0..127
        constexpr int NU = kNumUWarps * 32;
        uint32_t ti = 0;
        for (int t = blockIdx.x; t < p.num_tiles; t += gridDim.x, ++ti) {
            int f, y0, x0, rows;
            decode_tile(p, t, f, y0, x0, rows);
            const int ub = ti & 1;
            const uint32_t uph = (ti >> 1) & 1;
            bool ok = mbar_wait(&ctl.u_empty[ub], uph ^ 1, abort_flag);
            ok = named_barrier_and(1, NU, ok);               // also: the previous tile's vertical pass is done
            if (!ok) break;
            const int uh = rows + 2 * G::P;
            // LR rows the tile needs: from the first tap of its first HR row to the last tap of its last HR row
            const int Ylo = clampi(y0 - G::P, 0, pb.H - 1), Yhi = clampi(y0 + rows - 1 + G::P, 0, pb.H - 1);
            const int qlo = Ylo / pb.r, qhi = Yhi / pb.r;
            const int lr_lo = qlo + pb.ph.base[Ylo - qlo * pb.r];
            const int nrows = qhi + pb.ph.base[Yhi - qhi * pb.r] + 3 - lr_lo + 1;   // <= trows
            if (ut < uh) {
                const int Yc = clampi(y0 - G::P + ut, 0, pb.H - 1);
                const int q = Yc / pb.r, py = Yc - q * pb.r;
                ctl.vy_row[ut] = q + pb.ph.base[py] - lr_lo;
                ctl.vy_phase[ut] = py;
            }
            // horizontal pass: T[ch][j][ux] = sum_b wx[b] * lr[ch][clamp(lr_lo + j)][clamp(xb + b)]
            for (int item = ut; item < C * G::UW; item += NU) {
                const int ch = item / G::UW, ux = item - ch * G::UW;
                const int Xc = clampi(x0 - G::P + ux, 0, pb.W - 1);
                const int q = Xc / pb.r, px = Xc - q * pb.r;
                const int xb = q + pb.ph.base[px];
                const int c0 = clampi(xb, 0, pb.w - 1), c1 = clampi(xb + 1, 0, pb.w - 1);
                const int c2 = clampi(xb + 2, 0, pb.w - 1), c3 = clampi(xb + 3, 0, pb.w - 1);
                const float w0 = pb.ph.w[px][0], w1 = pb.ph.w[px][1], w2 = pb.ph.w[px][2], w3 = pb.ph.w[px][3];
                const float* plane = p.lr + ((int64_t)f * C + ch) * pb.h * pb.w;
                float* dstT = sT + (ch * p.trows) * G::UW + ux;
                for (int j = 0; j < nrows; ++j) {
                    const float* row = plane + (int64_t)clampi(lr_lo + j, 0, pb.h - 1) * pb.w;
                    float v = w0 * __ldg(row + c0);
                    v = fmaf(w1, __ldg(row + c1), v);
                    v = fmaf(w2, __ldg(row + c2), v);
                    v = fmaf(w3, __ldg(row + c3), v);
                    dstT[j * G::UW] = v;
                }
            }
            named_barrier_sync(1, NU);
            // vertical pass: U[ch][uy][ux] = sum_a wy[a] * T[ch][vy_row[uy] + a][ux]
            float* Ub = sU + ub * C * G::UH * G::UW;
            for (int item = ut; item < C * G::UW; item += NU) {
                const int ch = item / G::UW, ux = item - ch * G::UW;
                const float* srcT = sT + (ch * p.trows) * G::UW + ux;
                float* dstU = Ub + ch * G::UH * G::UW + ux;
                for (int uy = 0; uy < uh; ++uy) {
                    const int j = ctl.vy_row[uy], py = ctl.vy_phase[uy];
                    float v = pb.ph.w[py][0] * srcT[j * G::UW];
                    v = fmaf(pb.ph.w[py][1], srcT[(j + 1) * G::UW], v);
                    v = fmaf(pb.ph.w[py][2], srcT[(j + 2) * G::UW], v);
                    v = fmaf(pb.ph.w[py][3], srcT[(j + 3) * G::UW], v);
                    dstU[uy * G::UW] = v;
                }
            }
            mbar_arrive(&ctl.u_full[ub]);
        }
    } else {
        // ===== epilogue: thread = one pixel of the tile row (TMEM lane); two groups of four warps alternate rows
        const int quarter = warp & 3;                        // the TMEM lanes this warp may read: 32*quarter..+31
        const int group = (warp - kFirstEpiWarp) >> 2;
        const int x = quarter * 32 + lane;                   // pixel within the tile row
        const int64_t HW = (int64_t)pb.H * pb.W;
        uint32_t it = 0, ti = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < p.num_tiles && ok; t += gridDim.x, ++ti) {
            int f, y0, x0, rows;
            decode_tile(p, t, f, y0, x0, rows);
            const int ub = ti & 1;
            const uint32_t uph = (ti >> 1) & 1;
            ok = __all_sync(0xffffffffu, mbar_wait(&ctl.u_full[ub], uph, abort_flag));
            if (!ok) break;
            const float* Ub = sU + ub * C * G::UH * G::UW;
            const bool in_x = x0 + x < pb.W;
            for (int r = 0; r < rows; ++r, ++it) {
                if ((int)(it & 1) != group) continue;
                const int a = it % kAccSlots;
                const uint32_t aph = (it / kAccSlots) & 1;
                ok = __all_sync(0xffffffffu, mbar_wait(&ctl.acc_full[a], aph, abort_flag));
                if (!ok) break;
                tc_fence_after_sync();
                float F[G::NPAD];
                const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(a * G::NPAD);
#pragma unroll
                for (int j = 0; j < G::NPAD; j += 16) tmem_ld_x16(taddr + j, F + j);
                tmem_ld_wait();
                tc_fence_before_sync();
                mbar_arrive(&ctl.acc_empty[a]);
                float* dst = p.out + ((int64_t)f * C) * HW + (int64_t)(y0 + r) * pb.W + x0 + x;
                for (int ch = 0; ch < C; ++ch) {
                    const float* u = Ub + (ch * G::UH + r) * G::UW + x;
                    float acc = 0.f;
#pragma unroll
                    for (int aa = 0; aa < K; ++aa)
#pragma unroll
                        for (int bb = 0; bb < K; ++bb) acc = fmaf(F[aa * K + bb], u[aa * G::UW + bb], acc);
                    if (pb.flags & SR_CLAMP01) acc = fminf(fmaxf(acc, 0.f), 1.f);
                    if (in_x) dst[ch * HW] = acc;
                }
            }
            if (ok) mbar_arrive(&ctl.u_empty[ub]);
        }
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

template <int K> size_t fixed_smem_bytes(int c, int dpad, int trows)
{
    using G = Geo<K>;
    return 1024 /* alignment slack */ + 2 * (size_t)(dpad / 16) * G::KSTEP_B +
           (size_t)(2 * c * G::UH * G::UW + c * trows * G::UW) * sizeof(float);
}

int trows_for(int k, int r) { return (TH + (k - 1) - 1) / r + 5; }

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
    const size_t fixed = fixed_smem_bytes<K>(c, dpad, trows_for(K, r)) + kStaticReserve;
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
    const size_t smem = fixed_smem_bytes<K>(prm.pb.c, prm.dpad, prm.trows) + (size_t)prm.stages * prm.dpad * 256;
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
