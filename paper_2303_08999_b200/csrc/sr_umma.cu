// Fused regression kernel for sm_100a: coefficient planes streamed with 16-byte asynchronous copies, dictionary
// assembly F = Phi D on the tcgen05 tensor cores with fp32 accumulators in tensor memory, bicubic tile + patch dot
// product + clamp in the epilogue. The filter matrix F (TMEM / registers), the up-sampled image U and its patches
// (shared memory) never reach HBM: per HR pixel the kernel reads its coefficients once and writes its c output
// values once.
//
// One persistent CTA per SM walks HR tiles of 128 x 16 pixels. A tile row (128 pixels of one HR row) is one
// pipeline stage [atoms][128 pixels] binary16, written by cp.async.cg (coalesced 128-bit loads, L1 bypassed)
// straight into the 128-byte-swizzled MN-major layout the tensor core reads (pixels are M, atoms are K), so the
// planar [n][D][H][W] coefficient tensor needs no transpose. (A TMA box over 72 planes 4 MB apart streams at
// ~4.2 TB/s on B200; the same bytes through cp.async reach ~5.5 TB/s, hence this choice.) The dictionary is the
// B operand (K-major): its fp32 values are split into binary16 hi + lo parts (~22 bits kept) that sit side by
// side along N, so one MMA per 16 atoms reads the coefficient stage once and yields both partial filters; the
// epilogue adds them. N = 2 x (k*k padded to 16).
//
// Shared-memory bandwidth and per-warp latency are the scarce on-chip resources, so the epilogue keeps a sliding
// k x k x 3 window of U in registers and reads each U row once per pixel column.
//
// Warp roles (640 threads = five warpgroups; the register file is re-balanced between them with setmaxnreg):
//   warps 0-3    coefficient producers   full[stage] <- cp.async arrivals when the copies land; wait empty[stage]
//   warps 4-5    MMA issuers (warp 4 owns TMEM): one thread each, alternate rows, because the issue loop of a
//                single thread (~600 cycles per row alone, twice that on a busy SM) would otherwise pace the kernel;
//                acc_full[a], empty[stage] <- tcgen05.commit; wait full[stage], acc_empty[a]
//   warps 6-11   U producers             bicubic (separable) of the tile + halo into a double-buffered tile
//   warps 12-19  epilogue (2 x 4 warps)  TMEM -> registers (one pixel's filter per thread), patch dot, clamp, store;
//                                        the two groups own the upper and the lower half of a tile
// Every wait is bounded; on expiry the CTA raises its abort flag, sets the device status word and drains.
#include <stdlib.h>

#include "sr_ptx.cuh"
#include "sr_umma.cuh"

namespace sr {

namespace {

using namespace ptx;

constexpr int TW = 128, TH = 16;
constexpr int kNumLoadWarps = 4, kMmaWarp = 4, kNumMmaWarps = 2;
constexpr int kFirstUWarp = 6, kNumUWarps = 6, kFirstSelWarp = 12, kNumSelWarps = 4, kNumEpiWarps = 8;

// Role layout. The selective variant (per-pixel top-s chosen inside the kernel) inserts one warpgroup of
// "select" warps between the loaders and the MMA issuers: they rewrite each landed stage in place, zeroing the
// coefficients that are not among the pixel's s largest, and the rest of the pipeline is the dense one.
template <bool SEL> struct Cfg {
    static constexpr int kFirstEpiWarp = SEL ? kFirstSelWarp + kNumSelWarps : kFirstSelWarp;   // 16 or 12
    static constexpr int kThreads = (kFirstEpiWarp + kNumEpiWarps) * 32;                        // 768 or 640
    // Registers per thread after setmaxnreg. setmaxnreg only moves registers inside the pool the CTA was given at
    // launch (warps x registers-per-thread the kernel was compiled for), so the re-balanced total must not exceed
    // it: an increase that can never be satisfied would block forever.
    static constexpr int kRegsLaunch = SEL ? 80 : 96;       // 65536 / threads, rounded down to a multiple of 8
    static constexpr int kRegsLoad = 40, kRegsMmaU = SEL ? 56 : 72, kRegsSel = 64, kRegsEpi = SEL ? 128 : 144;
    static constexpr int kNumWarps = kFirstEpiWarp + kNumEpiWarps;
    static constexpr int kPoolAfter = kNumLoadWarps * kRegsLoad + (kFirstSelWarp - kNumLoadWarps) * kRegsMmaU +
                                      (SEL ? kNumSelWarps * kRegsSel : 0) + kNumEpiWarps * kRegsEpi;
    static_assert(kRegsLaunch * kThreads <= 65536, "launch register count does not fit the register file");
    static_assert(kPoolAfter <= kNumWarps * kRegsLaunch, "re-balanced registers exceed the CTA's pool");
};

constexpr int kMaxStages = 10;
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
    int rows_alloc;       // rows a stage chunk really holds: natoms rounded up to 8 (one swizzle group). When this is
                          // below dpad the last K-step's upper 8 rows read whatever follows the chunk; the matching
                          // dictionary rows are zero, so any finite bytes there contribute nothing.
    int planes;           // planes per frame in the coefficient tensor (D, or s when it is compact)
    int sel_s;            // selective variant: atoms kept per pixel
    int tma_rows;         // leading planes of every stage that a TMA box brings in (multiple of 8; 0 = none); the
                          // rest arrive through cp.async, so that both load paths of the SM work side by side
    int gather_planes;    // 1: plane q of the contraction is plane atoms[q] of the tensor (subset of a full tensor)
    const __half* coef;
    int stages;
    int trows;            // LR rows a tile can need (rows of the horizontal-pass scratch tile)
    int tcols;            // LR columns a tile can need
    uint32_t r_magic;     // ceil(2^32 / r): floor(x / r) == umulhi(x, r_magic) for 0 <= x < 2^29 (r >= 2)
    uint32_t tcols_magic; // same for tcols
    int tiles_x, tiles_y, num_tiles;
};

struct __align__(16) Ctl {
    uint64_t full[kMaxStages], empty[kMaxStages];
    uint64_t ready[kMaxStages];   // selective variant: the stage has been masked and may be multiplied
    uint64_t acc_full[kMaxAccSlots], acc_empty[kMaxAccSlots];
    uint64_t u_full[2], u_empty[2];
    uint32_t tmem_base;
    int abort_flag;
    float4 vy_w[TH + 2 * 4];   // per U-tile row: its four vertical tap weights
    float4 wtab[kMaxScale];    // the four tap weights of every phase (copied once from the kernel parameters)
    int vy_off[TH + 2 * 4];    // per U-tile row: first row of the scratch tile it reads
    alignas(16) int hx_off[TW + 2 * 4];   // per U-tile column: first column of the LR window it reads, | phase << 16
    uint8_t atoms[256];        // subset mode: the atom id of each selected plane
};

template <int K> struct Geo {
    static constexpr int kk = K * K;
    static constexpr int NPAD = (kk + 15) / 16 * 16;     // taps padded; hi part in columns [0, NPAD), lo in [NPAD, 2 NPAD)
    static constexpr int NB = 2 * NPAD;                  // N of the MMA
    static constexpr int P = (K - 1) / 2;
    static constexpr int UW = (TW + 2 * P + 3) & ~3;     // U tile width: tile + halo, rounded up to 4 for 16-byte rows
    static constexpr int UH = TH + 2 * P;
    static constexpr int LBO_B = (NB / 8) * 128;         // bytes between the two K-halves of a K-step of the B operand
    static constexpr int KSTEP_B = 2 * LBO_B;            // bytes per K-step (16 atoms) of the B operand
    static constexpr int ACC_SLOTS = (512 / NB) < kMaxAccSlots ? (512 / NB) : kMaxAccSlots;
    // Column of tap (a, b) inside a half of the accumulator: the first K-1 taps of every patch row come first, row by
    // row, so that they can be consumed as aligned pairs by the packed fp32 instructions; the last tap of every row
    // follows as a block of K single columns.
    static constexpr int NPAIRCOLS = K * (K - 1);
    __host__ __device__ static constexpr int col_of(int a, int b) { return b < K - 1 ? a * (K - 1) + b : NPAIRCOLS + a; }
    __host__ __device__ static constexpr int col_of_tap(int j) { return col_of(j / K, j % K); }
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

// Rows of a tile are streamed in the order 0, H, 1, H+1, ... (H = TH/2) so that the two epilogue groups, which
// own the upper and the lower half of the tile, both receive work from the start. Item i of a tile with `rows`
// valid rows maps to a tile row; every role enumerates the same sequence.
constexpr int kHalf = TH / 2;
__device__ __forceinline__ int tile_row_of_item(int i, int rows)
{
    const int h1 = rows > kHalf ? rows - kHalf : 0;      // rows in the lower half
    // the first 2*h1 items alternate between the halves, the rest belong to the upper half
    return i < 2 * h1 ? ((i & 1) ? kHalf + (i >> 1) : (i >> 1)) : i - h1;
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
    const int Xlo = clampi(g.x0 - P, 0, pb.W - 1), Xhi = clampi(g.x0 - P + Geo<K>::UW - 1, 0, pb.W - 1);
    const int qxlo = fast_div(Xlo, pb.r, p.r_magic), qxhi = fast_div(Xhi, pb.r, p.r_magic);
    g.col_lo = qxlo + pb.ph.base[Xlo - qxlo * pb.r];
    g.ncols = qxhi + pb.ph.base[Xhi - qxhi * pb.r] + 3 - g.col_lo + 1;     // <= tcols
}

__device__ __forceinline__ void cp_async_f32(float* dst_smem, const float* src)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_u32(dst_smem)), "l"(src) : "memory");
}
template <int N> __device__ __forceinline__ void setmaxnreg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N> __device__ __forceinline__ void setmaxnreg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }

// 16-byte copy global -> shared, L1 bypassed; src_bytes = 0 writes zeros instead of reading.
__device__ __forceinline__ void cp_async_16(uint32_t dst_smem, const void* src, uint32_t src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst_smem), "l"(src), "r"(src_bytes) : "memory");
}
// Arrives on the mbarrier (without raising its pending count) once all cp.async of this thread so far completed.
__device__ __forceinline__ void cp_async_mbar_arrive_noinc(uint64_t* bar)
{
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// cp.async.wait_group with a run-time count (0..7): at most n of this thread's groups remain in flight.
__device__ __forceinline__ void cp_async_wait_dyn(int n)
{
    switch (n) {
    case 0: cp_async_wait<0>(); break;
    case 1: cp_async_wait<1>(); break;
    case 2: cp_async_wait<2>(); break;
    case 3: cp_async_wait<3>(); break;
    case 4: cp_async_wait<4>(); break;
    case 5: cp_async_wait<5>(); break;
    case 6: cp_async_wait<6>(); break;
    default: cp_async_wait<7>(); break;
    }
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

// One pixel's filter from tensor memory in natural tap order: F[a*K+b] = hi[col] + lo[col], col = col_of(a, b)
// (at most 16 columns at a time).
template <int K>
__device__ __forceinline__ void load_filter(uint32_t taddr, float* F)
{
    using G = Geo<K>;
    float Fc[G::NPAD];                                       // column order
#pragma unroll
    for (int j0 = 0; j0 < G::kk; j0 += 16) {
        constexpr int kTail = G::kk % 16;
        float h[16], l[16];
        if (j0 + 16 <= G::kk) {
            tmem_ld_n<16>(taddr + j0, h);
            tmem_ld_n<16>(taddr + G::NPAD + j0, l);
        } else {
            tmem_ld_n<kTail ? kTail : 16>(taddr + j0, h);
            tmem_ld_n<kTail ? kTail : 16>(taddr + G::NPAD + j0, l);
        }
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 16; ++i)
            if (j0 + i < G::kk) Fc[j0 + i] = h[i] + l[i];
    }
#pragma unroll
    for (int j = 0; j < G::kk; ++j) F[j] = Fc[G::col_of_tap(j)];
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

// ---- per-pixel top-s masking of a staged row (selective variant) -----------------------------------------------------

__device__ __forceinline__ void cx_h2(__half2& a, __half2& b)    // afterwards a >= b in both halves
{
    const __half2 hi = __hmax2(a, b), lo = __hmin2(a, b);
    a = hi;
    b = lo;
}

__device__ __forceinline__ void sort8_desc_h2(__half2 (&k)[8])   // 19 exchanges
{
    cx_h2(k[0], k[1]); cx_h2(k[2], k[3]); cx_h2(k[4], k[5]); cx_h2(k[6], k[7]);
    cx_h2(k[0], k[2]); cx_h2(k[1], k[3]); cx_h2(k[4], k[6]); cx_h2(k[5], k[7]);
    cx_h2(k[1], k[2]); cx_h2(k[5], k[6]);
    cx_h2(k[0], k[4]); cx_h2(k[1], k[5]); cx_h2(k[2], k[6]); cx_h2(k[3], k[7]);
    cx_h2(k[2], k[4]); cx_h2(k[3], k[5]);
    cx_h2(k[1], k[2]); cx_h2(k[3], k[4]); cx_h2(k[5], k[6]);
}

__device__ __forceinline__ void bitonic_merge8_desc_h2(__half2 (&k)[8])
{
#pragma unroll
    for (int d = 4; d >= 1; d >>= 1)
#pragma unroll
        for (int i = 0; i < 8; ++i)
            if ((i & d) == 0) cx_h2(k[i], k[i + d]);
}

__device__ __forceinline__ __half2 h2_from_bits(uint32_t u) { return *reinterpret_cast<__half2*>(&u); }
__device__ __forceinline__ uint32_t bits_from_h2(__half2 h) { return *reinterpret_cast<uint32_t*>(&h); }

// Masks two independent pixel pairs (columns `colA`, `colB`: pointers at (atom 0, two neighbouring pixels) of a
// stage; atom l of a pair sits at col + l*128 + ((c16 ^ (l & 7)) << 4)) so that two sorting networks are in flight
// per thread. Keeps, per pixel, the s (<= 8) coefficients of largest magnitude (ties: lower atom index first) and
// zeroes the rest. Magnitudes are compared as positive binary16 numbers, which orders finite values exactly like
// their bit patterns.
__device__ __forceinline__ void select_mask_stage(uint8_t* colA, uint32_t c16A, uint8_t* colB, uint32_t c16B, int natoms, int s)
{
    auto wordA = [&](int l) -> uint32_t* {
        return reinterpret_cast<uint32_t*>(colA + (uint32_t)l * 128u + (((c16A ^ (uint32_t)(l & 7))) << 4));
    };
    auto wordB = [&](int l) -> uint32_t* {
        return reinterpret_cast<uint32_t*>(colB + (uint32_t)l * 128u + (((c16B ^ (uint32_t)(l & 7))) << 4));
    };
    const __half2 zero = h2_from_bits(0u);
    // The running list starts with 8 - s entries of +infinity: they stay on top, so the s-th largest real
    // magnitude always ends up in slot 7 and no slot has to be picked at run time.
    const __half2 inf = h2_from_bits(0x7C007C00u);
    __half2 topA[8], topB[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) topA[i] = topB[i] = (i < 8 - s) ? inf : zero;
    for (int l0 = 0; l0 < natoms; l0 += 8) {
        __half2 gA[8], gB[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            gA[i] = (l0 + i < natoms) ? h2_from_bits(*wordA(l0 + i) & 0x7FFF7FFFu) : zero;
            gB[i] = (l0 + i < natoms) ? h2_from_bits(*wordB(l0 + i) & 0x7FFF7FFFu) : zero;
        }
        sort8_desc_h2(gA);
        sort8_desc_h2(gB);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            topA[i] = __hmax2(topA[i], gA[7 - i]);
            topB[i] = __hmax2(topB[i], gB[7 - i]);
        }
        bitonic_merge8_desc_h2(topA);
        bitonic_merge8_desc_h2(topB);
    }
    // tau = s-th largest magnitude; need = how many coefficients equal to tau are kept = s - #(magnitudes > tau)
    // = 8 - #(list entries > tau), the virtual infinities included
    const __half2 tauA = topA[7], tauB = topB[7];
    __half2 gtA = zero, gtB = zero;
#pragma unroll
    for (int i = 0; i < 7; ++i) { gtA = __hadd2(gtA, __hgt2(topA[i], tauA)); gtB = __hadd2(gtB, __hgt2(topB[i], tauB)); }
    const __half2 eight = __float2half2_rn(8.f);
    const __half2 needA = __hsub2(eight, gtA), needB = __hsub2(eight, gtB);
    // above tau everything passes; once `need` ties have passed, the threshold moves one ulp up for that pixel
    const uint32_t tA = bits_from_h2(tauA), tB = bits_from_h2(tauB);
    const uint32_t tA1 = tA + 0x00010001u, tB1 = tB + 0x00010001u;     // next representable magnitude (per half)
    uint32_t thrA = tA, thrB = tB;                                     // need >= 1: tau itself is one of the ties
    __half2 cntA = zero, cntB = zero;
#pragma unroll 4
    for (int l = 0; l < natoms; ++l) {
        uint32_t* wa = wordA(l);
        uint32_t* wb = wordB(l);
        const uint32_t a = *wa, b = *wb;
        const __half2 ma = h2_from_bits(a & 0x7FFF7FFFu), mb = h2_from_bits(b & 0x7FFF7FFFu);
        *wa = a & __hge2_mask(ma, h2_from_bits(thrA));
        *wb = b & __hge2_mask(mb, h2_from_bits(thrB));
        cntA = __hadd2(cntA, __heq2(ma, tauA));
        cntB = __hadd2(cntB, __heq2(mb, tauB));
        const uint32_t exA = __hge2_mask(cntA, needA), exB = __hge2_mask(cntB, needB);
        thrA = (tA & ~exA) | (tA1 & exA);
        thrB = (tB & ~exB) | (tB1 & exB);
    }
}

struct EpiCtx {
    int quarter, group, x;
    int64_t HW;
    bool clamp01;
    uint32_t tmem_lane_base;
};

// Position in a tile's streaming order of row j of half `group` (inverse of tile_row_of_item).
__device__ __forceinline__ int item_of_half_row(int j, int group, int h1)
{
    return j < h1 ? 2 * j + group : j + h1;              // beyond h1 only the upper half (group 0) has rows
}

// Epilogue of one half tile (rows j = 0 .. my_rows-1 of the half, top to bottom) for a three-channel image.
// The k x k x 3 patch lives in registers as a sliding window (slot of U row u is u % K, all indices
// compile-time), so each row costs 3 * K shared loads instead of 3 * K * K. Window rows and filter taps are held
// as (K-1)/2 aligned pairs plus one single per patch row, so hi + lo and the patch dot product run on the packed
// fp32 instructions (two lanes per issue slot). Returns false when a wait expired.
template <int K, class CtlT>
__device__ __forceinline__ bool epilogue_half_windowed(CtlT& ctl, const EpiCtx& e, const float* Ub, float* dst0, int W,
                                                       int my_rows, int h1, uint32_t it_base, bool in_x,
                                                       volatile int* abort_flag, long long* wait_cycles = nullptr)
{
    using G = Geo<K>;
    constexpr int NP = (K - 1) / 2;                          // pairs per patch row
    constexpr int NPc = NP > 0 ? NP : 1;
    float2 winp[3][K][NPc];
    float wins[3][K];
    const float* u0 = Ub + e.x;
    auto load_row = [&](int u) {                             // U row u of the half -> window slot u % K
#pragma unroll
        for (int c = 0; c < 3; ++c) {
            const float* src = u0 + (c * G::UH + u) * G::UW;
#pragma unroll
            for (int i = 0; i < NP; ++i) winp[c][u % K][i] = make_float2(src[2 * i], src[2 * i + 1]);
            wins[c][u % K] = src[K - 1];
        }
    };
    bool ok = true;
    if (my_rows > 0) {
#pragma unroll
        for (int u = 0; u < K - 1; ++u) load_row(u);
    }
#pragma unroll
    for (int j = 0; j < kHalf; ++j) {
        if (j < my_rows && ok) {
            load_row(j + K - 1);
            const uint32_t it = it_base + item_of_half_row(j, e.group, h1);
            const int a_slot = it % G::ACC_SLOTS;
            const uint32_t aph = (it / G::ACC_SLOTS) & 1;
#ifdef SR_PROFILE_ROLES
            const long long tw0 = clock64();
#endif
            ok = mbar_wait_warp(&ctl.acc_full[a_slot], aph, abort_flag);
#ifdef SR_PROFILE_ROLES
            if (wait_cycles) *wait_cycles += clock64() - tw0;
#endif
            if (ok) {
                tc_fence_after_sync();
                const uint32_t taddr = e.tmem_lane_base + (uint32_t)(a_slot * G::NB);
                // filter: pair columns [0, K(K-1)) and single columns [K(K-1), K*K) of both halves, summed
                float2 Fp[K][NPc];
                float Fs[K];
                {
                    float2 hp[K * NPc], lp[K * NPc];
                    if (NP > 0) {
                        tmem_ld_n<G::NPAIRCOLS>(taddr, reinterpret_cast<float*>(hp));
                        tmem_ld_n<G::NPAIRCOLS>(taddr + G::NPAD, reinterpret_cast<float*>(lp));
                    }
                    float hs[K], ls[K];
                    tmem_ld_n<K>(taddr + G::NPAIRCOLS, hs);
                    tmem_ld_n<K>(taddr + G::NPAD + G::NPAIRCOLS, ls);
                    tmem_ld_wait();
#pragma unroll
                    for (int a = 0; a < K; ++a) {
#pragma unroll
                        for (int i = 0; i < NP; ++i) Fp[a][i] = __fadd2_rn(hp[a * NP + i], lp[a * NP + i]);
                        Fs[a] = hs[a] + ls[a];
                    }
                }
                tc_fence_before_sync();
                mbar_arrive(&ctl.acc_empty[a_slot]);
                float2 acc2[3][2];
                float accs[3];
#pragma unroll
                for (int c = 0; c < 3; ++c) { acc2[c][0] = acc2[c][1] = make_float2(0.f, 0.f); accs[c] = 0.f; }
#pragma unroll
                for (int a = 0; a < K; ++a)
#pragma unroll
                    for (int c = 0; c < 3; ++c) {
#pragma unroll
                        for (int i = 0; i < NP; ++i)
                            acc2[c][i & 1] = __ffma2_rn(Fp[a][i], winp[c][(j + a) % K][i], acc2[c][i & 1]);
                        accs[c] = fmaf(Fs[a], wins[c][(j + a) % K], accs[c]);
                    }
#pragma unroll
                for (int c = 0; c < 3; ++c) {
                    const float2 t2 = __fadd2_rn(acc2[c][0], acc2[c][1]);
                    float v = (t2.x + t2.y) + accs[c];
                    if (e.clamp01) v = fminf(fmaxf(v, 0.f), 1.f);
                    if (in_x) dst0[c * e.HW + (int64_t)j * W] = v;
                }
            }
        }
    }
    return ok;
}

// Optional role timing (build with -DSR_PROFILE_ROLES): cycles each role spends in total and inside waits,
// written per CTA to the buffer registered with sr_debug_role_profile.
#ifdef SR_PROFILE_ROLES
__device__ long long* g_role_prof = nullptr;
__device__ int g_debug_mode = 0;   // 1: TMA streaming only (no MMA, no U, no epilogue)
#define PROF_DECL long long prof_t0 = clock64(), prof_wait = 0, prof_tw = 0, prof_mma = 0, prof_commit = 0, prof_a = 0, prof_b = 0, prof_c = 0, prof_d = 0; bool prof_tmp_ok = true;
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

template <int K, bool SEL>
__global__ void __launch_bounds__(Cfg<SEL>::kThreads, 1)
regress_umma_kernel(const __grid_constant__ CUtensorMap map_lead, const __grid_constant__ UmmaParams p)
{
    using G = Geo<K>;
    using CF = Cfg<SEL>;
    constexpr int kThreads = CF::kThreads, kFirstEpiWarp = CF::kFirstEpiWarp;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    __shared__ Ctl ctl;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
#ifdef SR_PROFILE_ROLES
    unsigned long long gt_entry; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(gt_entry));
#endif
    const Problem& pb = p.pb;
    const int C = pb.c;
    const int stage_bytes = p.rows_alloc * 256;      // two chunks of [rows_alloc][64 pixels] binary16
    const int chunk_bytes = p.rows_alloc * 128;
    const int ksteps = p.dpad / 16;

    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* sA = smem;
    uint8_t* sB = sA + (size_t)p.stages * stage_bytes;
    float* sU = reinterpret_cast<float*>(sB + (size_t)ksteps * G::KSTEP_B);            // [2][C][UH][UW]
    float* sT = sU + 2 * C * G::UH * G::UW;                                           // [C * trows][UW]
    float* sL = sT + C * p.trows * G::UW;                                             // [2][C * trows][tcols]

    // ---------------------------------------------------------------- set-up
    if (tid == 0) {
        for (int i = 0; i < kMaxStages; ++i) { mbar_init(&ctl.full[i], kNumLoadWarps * 32 + (p.tma_rows > 0 ? 1 : 0)); mbar_init(&ctl.empty[i], 1); mbar_init(&ctl.ready[i], 32); }
        for (int i = 0; i < kMaxAccSlots; ++i) { mbar_init(&ctl.acc_full[i], 1); mbar_init(&ctl.acc_empty[i], 128); }
        for (int i = 0; i < 2; ++i) { mbar_init(&ctl.u_full[i], kNumUWarps * 32); mbar_init(&ctl.u_empty[i], kNumEpiWarps * 32); }
        ctl.abort_flag = 0;
        fence_barrier_init();
        if (p.tma_rows > 0) prefetch_tensormap(&map_lead);
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
        const int nh = n < G::kk ? G::col_of_tap(n) : n;     // tap n lives in column col_of_tap(n) of each half
        const int nl = nh + G::NPAD;
        *reinterpret_cast<__half*>(sB + base + (nh >> 3) * 128 + (nh & 7) * 16) = hi;
        *reinterpret_cast<__half*>(sB + base + (nl >> 3) * 128 + (nl & 7) * 16) = lo;
    }
    if (tid < kMaxScale) ctl.wtab[tid] = make_float4(pb.ph.w[tid][0], pb.ph.w[tid][1], pb.ph.w[tid][2], pb.ph.w[tid][3]);
    if (p.gather_planes)
        for (int q = tid; q < p.natoms; q += kThreads) ctl.atoms[q] = (uint8_t)min((int)__ldg(p.idx + q), pb.D - 1);
    // The copies only ever write rows < natoms of a stage; the padding rows up to dpad must read as zero.
    {
        uint4* a4 = reinterpret_cast<uint4*>(sA);
        const int n16 = p.stages * stage_bytes / 16;
        for (int i = tid; i < n16; i += kThreads) a4[i] = make_uint4(0, 0, 0, 0);
    }
    fence_proxy_async_smem();
    __syncwarp();
    if (warp == kMmaWarp) tmem_alloc(&ctl.tmem_base, G::TMEM_COLS);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = ctl.tmem_base;
    volatile int* abort_flag = &ctl.abort_flag;
    PROF_DECL
#ifdef SR_PROFILE_ROLES
    unsigned long long gt_setup; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(gt_setup));
#endif

    // ---------------------------------------------------------------- roles
#ifdef SR_PROFILE_ROLES
    const int debug_mode = g_debug_mode;
    // debug runs: 1, 2 = streaming only; 3 = loaders + MMA + epilogue handshake only (no U, no TMEM reads, no math)
    const int dm = debug_mode & 15;
    const int my_tiles = ((dm == 1 || dm == 2) && warp > kMmaWarp) || ((dm >= 3 && dm <= 5) && warp > kMmaWarp && warp < kFirstEpiWarp) ? 0 : p.num_tiles;
#else
    const int my_tiles = p.num_tiles;
#endif
    // Each role's branch starts by re-balancing the register file for its warpgroup (all four warps of a
    // warpgroup execute the same setmaxnreg instruction).
    if (warp < kNumLoadWarps) {
        setmaxnreg_dec<CF::kRegsLoad>();
        // ===== coefficient producers: 128 threads, thread = (16-byte column c16 of the 128-pixel row, atom l0 + 8k)
        // A stage is [chunk of 64 pixels][atom][128 B]; within a 1024-byte group of 8 atoms the 16-byte columns are
        // XOR-swizzled with the atom index (the 128-byte swizzle the MMA descriptor names).
        constexpr int NL = kNumLoadWarps * 32;
        const int c16 = tid & 15, l0 = tid >> 4;             // l0 in 0..7: constant (l & 7) for this thread
        const uint32_t dst_thread = (uint32_t)((c16 >> 3) * chunk_bytes + l0 * 128 + (((c16 & 7) ^ l0) << 4));
        const int64_t plane_elems = (int64_t)pb.H * pb.W;
        int s = 0;
        uint32_t ph = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < p.num_tiles && ok; t += gridDim.x) {
            int f, y0, x0, rows;
            decode_tile(p, t, f, y0, x0, rows);
#ifdef SR_PROFILE_ROLES
            if ((debug_mode & 15) == 2) { int rr; decode_tile(p, blockIdx.x % p.tiles_x, f, y0, x0, rr); }   // L2-resident re-reads
#endif
            const int xe = x0 + c16 * 8;                     // first of this thread's 8 pixels
            const uint32_t src_bytes = xe < pb.W ? 16u : 0u; // columns beyond the image are zero-filled
            const __half* src_col = p.coef + (int64_t)f * p.planes * plane_elems + (xe < pb.W ? xe : 0);
            for (int r = 0; r < rows; ++r) {
                ok = PROF_WAIT(mbar_wait(&ctl.empty[s], ph ^ 1, abort_flag));
                if (!ok) break;
                const int yr = y0 + tile_row_of_item(r, rows);
                const __half* src_row = src_col + (int64_t)yr * pb.W;
                uint32_t dst = smem_u32(sA + (size_t)s * stage_bytes) + dst_thread;
                if (p.tma_rows > 0 && tid == 0) {
                    // planes [0, tma_rows) of both 64-pixel chunks: two boxes, bytes counted on the same barrier
                    uint8_t* sdst = sA + (size_t)s * stage_bytes;
                    mbar_arrive_expect_tx(&ctl.full[s], (uint32_t)p.tma_rows * 256u);
                    tma_load_4d(sdst, &map_lead, &ctl.full[s], x0, yr, 0, f);
                    tma_load_4d(sdst + chunk_bytes, &map_lead, &ctl.full[s], x0 + 64, yr, 0, f);
                }
                if (!p.gather_planes) {
                    const int lfirst = p.tma_rows + l0;
                    const __half* src = src_row + lfirst * plane_elems;
                    dst += (uint32_t)p.tma_rows * 128u;
#pragma unroll 3
                    for (int l = lfirst; l < p.natoms; l += 8) {
                        cp_async_16(dst, src, src_bytes);
                        dst += 1024u;
                        src += 8 * plane_elems;
                    }
                } else {
                    for (int l = l0; l < p.natoms; l += 8, dst += 1024u)
                        cp_async_16(dst, src_row + (int)ctl.atoms[l] * plane_elems, src_bytes);
                }
                // asynchronous arrival: counts on full[s] once this thread's copies above have landed
                cp_async_mbar_arrive_noinc(&ctl.full[s]);
                if (++s == p.stages) { s = 0; ph ^= 1; }
            }
        }
        cp_async_wait_all();                                 // nothing of this thread is in flight at exit
        PROF_STORE(warp)
    } else if (warp < kFirstSelWarp) {
      setmaxnreg_dec<CF::kRegsMmaU>();
      if (warp < kMmaWarp + kNumMmaWarps) {
        // ===== MMA issuers: warp kMmaWarp + m takes the rows whose running index is m modulo kNumMmaWarps
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc_f16(128, G::NB, /*a_mn_major=*/true, /*b_mn_major=*/false);
            // A: MN-major, 128-byte swizzle: 8 atoms x 64 pixels per 1024-byte atom; K-groups 1024 B apart (SBO),
            // the second 64-pixel chunk chunk_bytes away (LBO). A K-step of 16 atoms is 2048 B further on.
            // Only the 14-bit start-address field (units of 16 B) changes between stages and K-steps.
            const uint64_t a_desc0 = make_smem_desc(smem_u32(sA), chunk_bytes, 1024, kSwizzle128B);
            const uint64_t b_desc0 = make_smem_desc(smem_u32(sB), G::LBO_B, 128, kSwizzleNone);
            const uint32_t a_stage_step = (uint32_t)stage_bytes >> 4;
            const int me = warp - kMmaWarp;
            // total rows this CTA streams
            uint32_t total = 0;
            for (int t = blockIdx.x; t < p.num_tiles; t += gridDim.x) {
                int f, y0, x0, rows;
                decode_tile(p, t, f, y0, x0, rows);
                total += rows;
            }
            int s = me % p.stages, a = me % G::ACC_SLOTS;
            uint32_t ph = (me / p.stages) & 1, aph = (me / G::ACC_SLOTS) & 1;
            bool ok = true;
            for (uint32_t it = me; it < total && ok; it += kNumMmaWarps) {
#ifdef SR_PROFILE_ROLES
                if ((debug_mode & 15) == 1 || (debug_mode & 15) == 2) {
                    if (!(ok = mbar_wait(&ctl.full[s], ph, abort_flag))) break;
                    mbar_arrive(&ctl.empty[s]);
                    s += kNumMmaWarps; if (s >= p.stages) { s -= p.stages; ph ^= 1; }
                    continue;
                }
#endif
                if (!(ok = PROF_WAIT(mbar_wait(&ctl.acc_empty[a], aph ^ 1, abort_flag)))) break;
                if (!(ok = PROF_WAIT(mbar_wait(SEL ? &ctl.ready[s] : &ctl.full[s], ph, abort_flag)))) break;
                fence_proxy_async_smem();        // the stage was written by cp.async (generic proxy), the MMA reads it through the async proxy
                tc_fence_after_sync();
                const uint32_t taddr = tmem_base + (uint32_t)(a * G::NB);
                uint64_t ad = a_desc0 + (uint64_t)((uint32_t)s * a_stage_step);
                uint64_t bd = b_desc0;
                for (int ks = 0; ks < ksteps; ++ks) {
                    mma_f16_ss(taddr, ad, bd, idesc, ks > 0);
                    ad += 2048 >> 4;
                    bd += G::KSTEP_B >> 4;
                }
                mma_commit(&ctl.empty[s]);       // the stage may be refilled once these MMAs have read it
                mma_commit(&ctl.acc_full[a]);    // and the accumulator is complete
                s += kNumMmaWarps; if (s >= p.stages) { s -= p.stages; ph ^= 1; }
                a += kNumMmaWarps; if (a >= G::ACC_SLOTS) { a -= G::ACC_SLOTS; aph ^= 1; }
            }
            PROF_STORE(warp)
        }
        __syncwarp();
      } else {
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
        if ((int)blockIdx.x < my_tiles) prefetch_lr(blockIdx.x, 0);
        for (int t = blockIdx.x; t < my_tiles; t += gridDim.x, ++ti) {
            LrWindow g;
            lr_window<K>(p, t, g);
            const int ub = ti & 1;
            const uint32_t uph = (ti >> 1) & 1;
            const bool has_next = t + (int)gridDim.x < my_tiles;
            // every thread is past the previous tile's passes before its LR buffer, scratch and tables are reused
            bool ok = PROF_WAIT(mbar_wait(&ctl.u_empty[ub], uph ^ 1, abort_flag));
            ok = named_barrier_and(1, NU, ok);
            if (!ok) break;
            PROF_T(tu0)
            if (has_next) prefetch_lr(t + gridDim.x, (ti + 1) & 1);
            const int uh = g.rows + 2 * G::P;
            for (int i = ut; i < G::UW + uh; i += NU) {
                if (i < G::UW) {
                    const int Xc = clampi(g.x0 - G::P + i, 0, pb.W - 1);
                    const int q = fast_div(Xc, pb.r, p.r_magic), px = Xc - q * pb.r;
                    ctl.hx_off[i] = (q + pb.ph.base[px] - g.col_lo) | (px << 16);
                } else {
                    const int uy = i - G::UW;
                    const int Yc = clampi(g.y0 - G::P + uy, 0, pb.H - 1);
                    const int q = fast_div(Yc, pb.r, p.r_magic), py = Yc - q * pb.r;
                    ctl.vy_off[uy] = q + pb.ph.base[py] - g.lr_lo;
                    ctl.vy_w[uy] = make_float4(pb.ph.w[py][0], pb.ph.w[py][1], pb.ph.w[py][2], pb.ph.w[py][3]);
                }
            }
            if (has_next) cp_async_wait<1>(); else cp_async_wait<0>();
            named_barrier_sync(1, NU);                       // tables written, this tile's LR window landed
            PROF_ADD(prof_a, tu0)
            PROF_T(tu1)
            // horizontal pass: T[row][ux] = sum_b wx[b] * L[row][hx_off[ux] + b], row = ch * nrows + j;
            // four neighbouring columns per trip, one 16-byte store
            const float* Lb = sL + (ti & 1) * lbuf_floats;
            const int hrows = C * g.nrows;
            constexpr int UW4 = G::UW / 4;
#pragma unroll 2
            for (int o = ut; o < hrows * UW4; o += NU) {
                const int row = o / UW4, ux = (o - row * UW4) * 4;
                const int4 op = *reinterpret_cast<const int4*>(&ctl.hx_off[ux]);   // offset | phase << 16, four columns
                const float* Lr = Lb + row * p.tcols;
                float4 out;
                {
                    const float4 w = ctl.wtab[op.x >> 16];
                    const float* src = Lr + (op.x & 0xFFFF);
                    out.x = fmaf(w.w, src[3], fmaf(w.z, src[2], fmaf(w.y, src[1], w.x * src[0])));
                }
                {
                    const float4 w = ctl.wtab[op.y >> 16];
                    const float* src = Lr + (op.y & 0xFFFF);
                    out.y = fmaf(w.w, src[3], fmaf(w.z, src[2], fmaf(w.y, src[1], w.x * src[0])));
                }
                {
                    const float4 w = ctl.wtab[op.z >> 16];
                    const float* src = Lr + (op.z & 0xFFFF);
                    out.z = fmaf(w.w, src[3], fmaf(w.z, src[2], fmaf(w.y, src[1], w.x * src[0])));
                }
                {
                    const float4 w = ctl.wtab[op.w >> 16];
                    const float* src = Lr + (op.w & 0xFFFF);
                    out.w = fmaf(w.w, src[3], fmaf(w.z, src[2], fmaf(w.y, src[1], w.x * src[0])));
                }
                *reinterpret_cast<float4*>(sT + row * G::UW + ux) = out;
            }
            PROF_ADD(prof_b, tu1)
            PROF_T(tu2)
            named_barrier_sync(1, NU);
            PROF_ADD(prof_c, tu2)
            PROF_T(tu3)
            // vertical pass: U[ch][uy][ux] = sum_a wy[a] * T[ch * nrows + vy_off[uy] + a][ux], 16 bytes at a time
            float* Ub = sU + ub * C * G::UH * G::UW;
            for (int ch = 0; ch < C; ++ch) {
                const float* Tc = sT + ch * g.nrows * G::UW;
                float* Uc = Ub + ch * G::UH * G::UW;
#pragma unroll 2
                for (int o = ut; o < uh * UW4; o += NU) {
                    const int uy = o / UW4, ux = (o - uy * UW4) * 4;
                    const float4 w = ctl.vy_w[uy];
                    const float* src = Tc + ctl.vy_off[uy] * G::UW + ux;
                    const float4 t0 = *reinterpret_cast<const float4*>(src);
                    const float4 t1 = *reinterpret_cast<const float4*>(src + G::UW);
                    const float4 t2 = *reinterpret_cast<const float4*>(src + 2 * G::UW);
                    const float4 t3 = *reinterpret_cast<const float4*>(src + 3 * G::UW);
                    float4 out;
                    out.x = fmaf(w.w, t3.x, fmaf(w.z, t2.x, fmaf(w.y, t1.x, w.x * t0.x)));
                    out.y = fmaf(w.w, t3.y, fmaf(w.z, t2.y, fmaf(w.y, t1.y, w.x * t0.y)));
                    out.z = fmaf(w.w, t3.z, fmaf(w.z, t2.z, fmaf(w.y, t1.z, w.x * t0.z)));
                    out.w = fmaf(w.w, t3.w, fmaf(w.z, t2.w, fmaf(w.y, t1.w, w.x * t0.w)));
                    *reinterpret_cast<float4*>(Uc + uy * G::UW + ux) = out;
                }
            }
            PROF_ADD(prof_d, tu3)
            mbar_arrive(&ctl.u_full[ub]);
        }
        cp_async_wait<0>();
        PROF_STORE(warp)
      }
    } else if (SEL && warp < kFirstEpiWarp) {
        setmaxnreg_dec<CF::kRegsSel>();
        // ===== select warps: one warp per stage (32 threads x 2 pixel pairs); warp w takes the stages whose
        // running index is w modulo 4. Per pixel: the s-th largest magnitude tau by sorting networks on packed
        // binary16 magnitudes, then every coefficient below tau, and every tie with tau beyond the first `need` in
        // atom order, is zeroed in place.
        const int me = warp - kFirstSelWarp;
        // this thread's pixel pairs: pixels 2*lane, 2*lane+1 of the first and of the second 64-pixel chunk
        const int px = 2 * lane;
        const uint32_t colA = (uint32_t)((px & 7) * 2), colB = (uint32_t)(chunk_bytes + (px & 7) * 2);
        const uint32_t c16 = (uint32_t)(px >> 3);
        uint32_t total = 0;
        for (int t = blockIdx.x; t < my_tiles; t += gridDim.x) {
            int f, y0, x0, rows;
            decode_tile(p, t, f, y0, x0, rows);
            total += rows;
        }
        int s = me % p.stages;
        uint32_t ph = (me / p.stages) & 1;
        bool ok = true;
        for (uint32_t it = me; it < total && ok; it += kNumSelWarps) {
            ok = mbar_wait_warp(&ctl.full[s], ph, abort_flag);
            if (!ok) break;
            uint8_t* stage = sA + (size_t)s * stage_bytes;
            select_mask_stage(stage + colA, c16, stage + colB, c16, p.natoms, p.sel_s);
            fence_proxy_async_smem();                                    // masked stage -> tensor core (async proxy)
            mbar_arrive(&ctl.ready[s]);
            s += kNumSelWarps;
            while (s >= p.stages) { s -= p.stages; ph ^= 1; }
        }
        PROF_STORE(warp)
    } else {
        setmaxnreg_inc<CF::kRegsEpi>();
        // ===== epilogue: thread = one pixel column of the tile (TMEM lane); two groups of four warps own the
        // upper and the lower half of a tile and walk their rows top to bottom
        EpiCtx e;
        e.quarter = warp & 3;                                // the TMEM lanes this warp may read: 32*quarter..+31
        e.group = (warp - kFirstEpiWarp) >> 2;
        e.x = e.quarter * 32 + lane;                         // pixel within the tile row
        e.HW = (int64_t)pb.H * pb.W;
        e.clamp01 = (pb.flags & SR_CLAMP01) != 0;
        e.tmem_lane_base = tmem_base + ((uint32_t)(e.quarter * 32) << 16);
        uint32_t it_base = 0, ti = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < my_tiles && ok; t += gridDim.x, ++ti) {
            int f, y0, x0, rows;
            decode_tile(p, t, f, y0, x0, rows);
            const int ub = ti & 1;
            const uint32_t uph = (ti >> 1) & 1;
#ifdef SR_PROFILE_ROLES
            if ((debug_mode & 15) == 3) {
                const int h1d = rows > kHalf ? rows - kHalf : 0;
                const int mine = e.group ? h1d : rows - h1d;
                for (int j = 0; j < mine && ok; ++j) {
                    const uint32_t it = it_base + item_of_half_row(j, e.group, h1d);
                    ok = mbar_wait_warp(&ctl.acc_full[it % G::ACC_SLOTS], (it / G::ACC_SLOTS) & 1, abort_flag);
                    if (ok) mbar_arrive(&ctl.acc_empty[it % G::ACC_SLOTS]);
                }
                it_base += rows;
                continue;
            }
            if ((debug_mode & 15) == 4) {
                const int h1d = rows > kHalf ? rows - kHalf : 0;
                const int mine = e.group ? h1d : rows - h1d;
                float sink = 0.f;
                for (int j = 0; j < mine && ok; ++j) {
                    const uint32_t it = it_base + item_of_half_row(j, e.group, h1d);
                    ok = mbar_wait_warp(&ctl.acc_full[it % G::ACC_SLOTS], (it / G::ACC_SLOTS) & 1, abort_flag);
                    if (ok) {
                        tc_fence_after_sync();
                        float F[G::NPAD];
                        load_filter<K>(e.tmem_lane_base + (uint32_t)((it % G::ACC_SLOTS) * G::NB), F);
                        tc_fence_before_sync();
                        mbar_arrive(&ctl.acc_empty[it % G::ACC_SLOTS]);
                        for (int q = 0; q < G::kk; ++q) sink += F[q];
                    }
                }
                if (sink == 123.456f) p.out[0] = sink;
                it_base += rows;
                continue;
            }
            if ((debug_mode & 15) != 5)
#endif
            ok = PROF_WAIT(mbar_wait_warp(&ctl.u_full[ub], uph, abort_flag));
            if (!ok) break;
            const int h1 = rows > kHalf ? rows - kHalf : 0;
            const int my_rows = e.group ? h1 : rows - h1;    // rows of this group's half
            const int r0 = e.group * kHalf;                  // first tile row of the half
            const float* Ub = sU + ub * C * G::UH * G::UW + r0 * G::UW;
            const bool in_x = x0 + e.x < pb.W;
            float* dst0 = p.out + ((int64_t)f * C) * e.HW + (int64_t)(y0 + r0) * pb.W + x0 + e.x;
            if (K <= 5 && C == 3) {
                #ifdef SR_PROFILE_ROLES
                ok = epilogue_half_windowed<K>(ctl, e, Ub, dst0, pb.W, my_rows, h1, it_base, in_x, abort_flag, &prof_wait);
#else
                ok = epilogue_half_windowed<K>(ctl, e, Ub, dst0, pb.W, my_rows, h1, it_base, in_x, abort_flag);
#endif
            } else {
                for (int j = 0; j < my_rows; ++j) {
                    const uint32_t it = it_base + item_of_half_row(j, e.group, h1);
                    const int a_slot = it % G::ACC_SLOTS;
                    const uint32_t aph = (it / G::ACC_SLOTS) & 1;
                    ok = mbar_wait_warp(&ctl.acc_full[a_slot], aph, abort_flag);
                    if (!ok) break;
                    tc_fence_after_sync();
                    float F[G::NPAD];
                    load_filter<K>(e.tmem_lane_base + (uint32_t)(a_slot * G::NB), F);
                    tc_fence_before_sync();
                    mbar_arrive(&ctl.acc_empty[a_slot]);
                    float* dst = dst0 + (int64_t)j * pb.W;
                    const float* u0 = Ub + j * G::UW + e.x;
                    if (C == 3) {
                        patch_dot<K, 3>(F, u0, G::UH * G::UW, G::UW, dst, e.HW, in_x, e.clamp01);
                    } else {
                        for (int ch = 0; ch < C; ++ch)
                            patch_dot<K, 1>(F, u0 + ch * G::UH * G::UW, G::UH * G::UW, G::UW, dst + ch * e.HW, e.HW, in_x, e.clamp01);
                    }
                }
            }
            it_base += rows;
#ifdef SR_PROFILE_ROLES
            if ((debug_mode & 15) == 5) continue;
#endif
            if (ok) mbar_arrive(&ctl.u_empty[ub]);
        }
        PROF_STORE(warp)
    }

    // ---------------------------------------------------------------- teardown
    __syncwarp();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
#ifdef SR_PROFILE_ROLES
    if (tid == 0 && g_role_prof) {
        unsigned long long gt_end; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(gt_end));
        g_role_prof[(blockIdx.x * 32 + 30) * 2] = (long long)(gt_setup - gt_entry);
        g_role_prof[(blockIdx.x * 32 + 30) * 2 + 1] = (long long)(gt_end - gt_entry);
        g_role_prof[(blockIdx.x * 32 + 31) * 2] = (long long)gt_entry;
        g_role_prof[(blockIdx.x * 32 + 31) * 2 + 1] = (long long)gt_end;
    }
#endif
    if (ctl.abort_flag && tid == 0) atomicExch(p.status, SR_ERR_TIMEOUT);
    if (warp == kMmaWarp) tmem_dealloc(tmem_base, G::TMEM_COLS);
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

// Share of a stage's planes that goes through TMA (the rest through cp.async); SR_TMA_SHARE overrides (0..100).
int tma_share_percent()
{
    static int v = [] {
        const char* e = getenv("SR_TMA_SHARE");
        int x = e ? atoi(e) : 50;
        return x < 0 ? 0 : (x > 100 ? 100 : x);
    }();
    return v;
}

int trows_for(int k, int r) { return (TH + (k - 1) - 1) / r + 5; }
int tcols_for(int k, int r) { return (((TW + (k - 1) + 3) & ~3) - 1) / r + 5; }

template <int K> size_t fixed_smem_bytes(int c, int dpad, int r)
{
    using G = Geo<K>;
    const int trows = trows_for(K, r), tcols = tcols_for(K, r);
    return 1024 /* alignment slack */ + (size_t)(dpad / 16) * G::KSTEP_B +
           (size_t)(2 * c * G::UH * G::UW + c * trows * G::UW + 2 * c * trows * tcols) * sizeof(float);
}

// planes that enter the contraction, and whether they are picked one by one out of a full tensor
void contraction_shape(int mode, const Problem& pb, int& natoms, int& gather)
{
    if (mode == kModeGlobal) {
        natoms = pb.s;
        gather = (pb.flags & SR_COEF_COMPACT) ? 0 : 1;
    } else {
        natoms = pb.D;
        gather = 0;
    }
}

template <int K> int stages_for(int c, int dpad, int rows_alloc, int r, int smem_optin)
{
    const size_t fixed = fixed_smem_bytes<K>(c, dpad, r) + kStaticReserve;
    if (fixed >= (size_t)smem_optin) return 0;
    const int s = (int)(((size_t)smem_optin - fixed) / ((size_t)rows_alloc * 256));
    return s > kMaxStages ? kMaxStages : s;
}

// A role that takes every n-th row (two MMA issuers, four select warps) must meet every use of the stages it
// waits on, one after the other: mbarrier waits only know the parity of a phase, so a waiter that skipped a use
// could mistake the phase before last for the one it wants. With the stage count a multiple of n each such warp
// owns a fixed subset of the stages.
int usable_stages(int mode, int stages)
{
    const int n = (mode == kModeFusedSelect) ? kNumSelWarps : kNumMmaWarps;
    return stages / n * n;
}

int stages_for_k(int k, int c, int dpad, int rows_alloc, int r, int smem_optin)
{
    switch (k) {
    case 1: return stages_for<1>(c, dpad, rows_alloc, r, smem_optin);
    case 3: return stages_for<3>(c, dpad, rows_alloc, r, smem_optin);
    case 5: return stages_for<5>(c, dpad, rows_alloc, r, smem_optin);
    case 7: return stages_for<7>(c, dpad, rows_alloc, r, smem_optin);
    default: return 0;
    }
}

template <int K, bool SEL>
cudaError_t launch_ks(const CUtensorMap& map_lead, UmmaParams& prm, cudaStream_t st)
{
    const DeviceInfo& di = device_info();
    const size_t smem = fixed_smem_bytes<K>(prm.pb.c, prm.dpad, prm.pb.r) + (size_t)prm.stages * prm.rows_alloc * 256;
    auto kern = regress_umma_kernel<K, SEL>;
    static bool configured[64] = {false};   // per template instance and device; the maximum is requested once
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, di.smem_optin - kStaticReserve);
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    const int grid = prm.num_tiles < di.sms ? prm.num_tiles : di.sms;
    kern<<<grid, Cfg<SEL>::kThreads, smem, st>>>(map_lead, prm);
    count_launches(1);
    return cudaGetLastError();
}

template <int K>
cudaError_t launch_k(const CUtensorMap& map_lead, UmmaParams& prm, cudaStream_t st)
{
    return prm.mode == kModeFusedSelect ? launch_ks<K, true>(map_lead, prm, st) : launch_ks<K, false>(map_lead, prm, st);
}

} // namespace

#ifdef SR_PROFILE_ROLES
extern "C" int sr_debug_mode(int mode)
{
    return cudaMemcpyToSymbol(g_debug_mode, &mode, sizeof(mode)) == cudaSuccess ? 0 : 5;
}

extern "C" int sr_debug_role_profile(long long* device_buffer)
{
    return cudaMemcpyToSymbol(g_role_prof, &device_buffer, sizeof(device_buffer)) == cudaSuccess ? 0 : 5;
}
#endif

bool umma_supported(int mode, const void* coef, int coef_dtype, const Problem& pb)
{
    if (mode != kModeDense && mode != kModeGlobal && !(mode == kModeFusedSelect && pb.s <= 8)) return false;
    if (coef_dtype != SR_F16) return false;
    if (pb.k > 7 || pb.c > kMaxChannels) return false;
    if ((reinterpret_cast<uintptr_t>(coef) & 15) != 0 || (pb.W & 7) != 0) return false;   // 16-byte copies: aligned base and row pitch
    if (pb.n > 65535) return false;
    const DeviceInfo& di = device_info();
    if (!di.ok || di.cc_major != 10) return false;
    int natoms, gather;
    contraction_shape(mode, pb, natoms, gather);
    const int dpad = (natoms + 15) / 16 * 16;
    return usable_stages(mode, stages_for_k(pb.k, pb.c, dpad, (natoms + 7) / 8 * 8, pb.r, di.smem_optin)) >= 2;
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
    prm.sel_s = pb.s;
    contraction_shape(mode, pb, prm.natoms, prm.gather_planes);
    prm.planes = (mode == kModeGlobal && (pb.flags & SR_COEF_COMPACT)) ? pb.s : pb.D;
    prm.coef = static_cast<const __half*>(coef);
    prm.dpad = (prm.natoms + 15) / 16 * 16;
    prm.rows_alloc = (prm.natoms + 7) / 8 * 8;
    prm.stages = usable_stages(mode, stages_for_k(pb.k, pb.c, prm.dpad, prm.rows_alloc, pb.r, di.smem_optin));
    prm.trows = trows_for(pb.k, pb.r);
    prm.tcols = tcols_for(pb.k, pb.r);
    prm.r_magic = pb.r > 1 ? (uint32_t)((0x100000000ull + pb.r - 1) / pb.r) : 0u;
    prm.tcols_magic = (uint32_t)((0x100000000ull + prm.tcols - 1) / prm.tcols);
    prm.tiles_x = (pb.W + TW - 1) / TW;
    prm.tiles_y = (pb.H + TH - 1) / TH;
    prm.num_tiles = prm.tiles_x * prm.tiles_y * pb.n;

    // Split of the coefficient stream between the SM's two load paths: the leading planes of a stage through one
    // TMA box per 64-pixel chunk, the rest through cp.async. Subsets gathered plane by plane use cp.async only.
    CUtensorMap map_lead{};
    prm.tma_rows = 0;
    if (!prm.gather_planes && encode_fn() && prm.natoms >= 16) {
        int lead = (prm.natoms * tma_share_percent() / 100) / 8 * 8;
        if (lead > 0) {
            const cuuint64_t dims[4] = {(cuuint64_t)pb.W, (cuuint64_t)pb.H, (cuuint64_t)prm.planes, (cuuint64_t)pb.n};
            const cuuint64_t strides[3] = {(cuuint64_t)pb.W * 2, (cuuint64_t)pb.W * pb.H * 2,
                                           (cuuint64_t)pb.W * pb.H * 2 * prm.planes};
            const cuuint32_t es[4] = {1, 1, 1, 1};
            const cuuint32_t box[4] = {64, 1, (cuuint32_t)lead, 1};
            if (encode_fn()(&map_lead, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4, const_cast<void*>(coef), dims, strides, box, es,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS)
                prm.tma_rows = lead;
        }
    }
    switch (pb.k) {
    case 1: return launch_k<1>(map_lead, prm, st);
    case 3: return launch_k<3>(map_lead, prm, st);
    case 5: return launch_k<5>(map_lead, prm, st);
    case 7: return launch_k<7>(map_lead, prm, st);
    default: return cudaErrorNotSupported;
    }
}

} // namespace sr
