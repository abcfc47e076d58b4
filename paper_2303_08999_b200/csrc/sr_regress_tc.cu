// Fused regression kernel for sm_100a, second layout: dense and global-subset modes (Eq. 2-3; Section III-A, Eq. 6
// and Eq. 9 for the subset form).
//
// What it computes is the same as sr_umma.cu: coefficient planes streamed into shared memory in the 128-byte-swizzled
// MN-major layout the tensor core reads (pixels are M, atoms are K), F = Phi D by tcgen05.mma with fp32 accumulators
// in tensor memory, up-sampled tile + patch dot product + clamp in the epilogue; F, the up-sampled image U and its
// patches never reach HBM. What differs is how the SM's warps are spent. Cycle stamps per role on the first layout
// and on an earlier form of this one showed where the time of the modes that stream few bytes goes:
//   - a hand-over through an mbarrier costs the waiting thread 150-250 cycles even when the phase is already
//     complete, and the single-threaded roles (copy issue, MMA issue) run at 20-30 cycles per instruction on a busy
//     SM, so a pipeline that hands over one 128-pixel row at a time is paced by its hand-overs (about 1200 cycles per
//     row and CTA) whatever the row costs. Here a pipeline step is a GROUP of up to four rows: one stage, one pair
//     of waits, one commit for the group;
//   - the epilogue of the first layout (one thread = one pixel, all channels, a k x k x c register window, 144
//     registers) had eight warps in flight. Here an epilogue thread owns one pixel column AND one channel: its window
//     is k x k registers, it fits in 72 registers, 4 x c warps (12 for RGB) work on a row, and the CTA is small
//     enough (128 + 128 c threads, under 112 KB of shared memory, 256 columns of tensor memory) for TWO CTAs per SM:
//     while one builds the up-sampled tile of its next block, the other one filters;
//   - the up-sampled tile was bound by shared-memory cycles (16 scalar loads and four 16-byte weight loads per four
//     output columns). Here the vertical pass runs first, on the LR columns; in the horizontal pass a thread keeps
//     its four columns for the whole tile, holds their taps as one 4 x 7 weight matrix in registers and reads seven
//     values per four outputs;
//   - the tile height th (<= 16) is a launch parameter, chosen on the host so that the tiles divide evenly among the
//     resident CTAs;
//   - with few atoms (<= 32) the binary16 hi and lo halves of the dictionary are stacked along K instead of N: the
//     tensor core adds them, the epilogue reads k*k columns instead of 2 k*k. With at most 8 atoms the second K-group
//     of the one MMA re-reads the same eight staged planes (stride 0 in the descriptor), so hi and lo cost a single
//     K-step.
// Warp roles: 0-1 coefficient loaders (TMA boxes for the leading planes of a stage, 16-byte cp.async for the rest),
// 2 MMA issuer (one thread; owns the tensor memory), 3 LR-window prefetch, 4.. epilogue (quarter = warp % 4 of the
// 128 pixel columns, channel = (warp - 4) / 4).
// Every wait is bounded; on expiry the CTA raises its abort flag, sets the device status word, drains and returns.
#include "sr_ptx.cuh"
#include "sr_regress_tc.cuh"
#include "sr_tile_upsample.cuh"

namespace sr {

namespace {

using namespace ptx;
using namespace tile;

constexpr int kMaxTH = 16;
constexpr int kUtilThreads = 128;
constexpr int kLoadThreads = 64;
constexpr int kMmaWarp = 2, kLrWarp = 3;
constexpr int kMaxStages = 8;
constexpr int kMaxC = 3;
constexpr int kMaxGroupRows = 4;

template <int K, bool HILO> struct Geo {
    static constexpr int kk = K * K;
    static constexpr int NPAD = (kk + 15) / 16 * 16;     // taps padded to the MMA's N granule
    static constexpr int NB = HILO ? 2 * NPAD : NPAD;    // N of the MMA: hi | lo side by side, or one of them
    static constexpr int P = (K - 1) / 2;
    static constexpr int UW = (TW + 2 * P + 3) & ~3;     // U tile width: tile + halo, rounded up to 4 for 16-byte rows
    static constexpr int UW4 = UW / 4;
    static constexpr int LBO_B = (NB / 8) * 128;         // bytes between the two K-halves of a K-step of the B operand
    static constexpr int KSTEP_B = 2 * LBO_B;            // bytes per K-step (16 rows) of the B operand
    static constexpr int TMEM_COLS = K >= 7 ? 512 : 256; // 256: two CTAs share the SM's 512 columns
    static constexpr int ACC_SLOTS = TMEM_COLS / NB;     // 2 .. 16
    static constexpr int MAX_GROUP = (ACC_SLOTS / 2) < kMaxGroupRows ? (ACC_SLOTS / 2) : kMaxGroupRows;   // rows per group: two groups in flight
    // Column of tap (a, b) inside a half of the accumulator: the first K-1 taps of every patch row come first, row by
    // row, so that they are consumed as aligned pairs by the packed fp32 instructions; the last tap of every row
    // follows as a block of K single columns.
    static constexpr int NPAIRCOLS = K * (K - 1);
    __host__ __device__ static constexpr int col_of(int a, int b) { return b < K - 1 ? a * (K - 1) + b : NPAIRCOLS + a; }
    __host__ __device__ static constexpr int col_of_tap(int j) { return col_of(j / K, j % K); }
    static constexpr int kCtasPerSm = K >= 7 ? 1 : 2;
    static constexpr int kRegsUtil = 40;
    static constexpr int kRegsEpi = K >= 7 ? 152 : 72;
    static constexpr int kThreadsMax = kUtilThreads + 128 * kMaxC;
    static constexpr int kRegsLaunch = 65536 / (kThreadsMax * kCtasPerSm) / 8 * 8;
    static_assert(kUtilThreads * kRegsUtil + 128 * kMaxC * kRegsEpi <= kThreadsMax * kRegsLaunch, "re-balanced registers exceed the CTA's pool");
    static_assert(kUtilThreads * kRegsUtil + 128 * kRegsEpi <= (kUtilThreads + 128) * kRegsLaunch, "re-balanced registers exceed the pool of a one-channel CTA");
};

struct TcParams {
    const float* lr;
    const float* dict;
    void* out;
    const uint8_t* idx;   // global-subset mode: s atom ids
    const float* gamma;   // global-subset mode: s weights or nullptr
    const __half* coef;
    int* status;
    Geom g;               // problem, tile height and the sizes that follow from it
    int mode;
    int natoms;           // coefficient planes per pixel that enter the contraction (D, or s for a subset)
    int dpad;             // natoms rounded up to a multiple of 16 (the MMA K extent)
    int rows_alloc;       // rows a stage chunk holds: natoms rounded up to 8 (one swizzle group)
    int planes;           // planes per frame in the coefficient tensor (D, or s when it is compact)
    int tma_rows;         // leading planes of every stage row that a TMA box brings in (multiple of 8; 0 = none)
    int gather_planes;    // 1: plane q of the contraction is plane atoms[q] of the tensor (subset of a full tensor)
    int alias8;           // 1: at most 8 atoms, hi and lo share one K-step (the A descriptor's K-group stride is 0)
    int stages;
    int group;            // tile rows per pipeline step: 1, 2 or 4
    long long wait_cycles;
    int inject_lost_arrival;
};

struct __align__(16) Ctl {
    uint64_t full[kMaxStages], empty[kMaxStages];
    uint64_t acc_full[2], acc_empty[2];
    uint64_t lr_full, lr_empty;
    uint64_t drain;
    uint32_t tmem_base;
    WaitCtx wait;
    float wpad[kMaxScale][12]; // the four tap weights of every phase between zeros: 0 0 0 w0 w1 w2 w3 0 0 0
    uint8_t atoms[256];        // subset mode: the atom id of each selected plane
};

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

// Epilogue of one tile for one (pixel column, channel): rows j = 0 .. rows-1 top to bottom. The k x k patch lives
// in registers as a sliding window (slot of U row u is u % K, all indices compile-time inside a block of K rows), so
// each row costs K shared loads. Window rows and filter taps are held as (K-1)/2 aligned pairs plus one single per
// patch row for the packed fp32 instructions. With HILO the accumulator is read in chunks of at most 16 columns from
// both halves, and both are multiplied into the same sums (no filter registers, no additions).
// Rows come in groups of `group` (two accumulator sets alternate): one wait before a group's first row, one arrival
// after its last. `gi` counts the CTA's groups. Returns false when a wait expired.
template <int K, bool HILO, typename OutT, class CtlT>
__device__ __forceinline__ bool epilogue_tile(CtlT& ctl, const float* Uc, OutT* dst, int W, int rows, int group, uint32_t& gi,
                                              uint32_t tmem_lane_base, bool in_x, bool clamp01, int lane, volatile WaitCtx* wc)
{
    using G = Geo<K, HILO>;
    constexpr int NP = (K - 1) / 2;                          // pairs per patch row
    constexpr int NPc = NP > 0 ? NP : 1;
    float2 winp[K][NPc];
    float wins[K];
    auto load_row = [&](int slot, int u) {                   // U row u of the tile -> window slot `slot` = u % K
        const float* src = Uc + u * G::UW;
#pragma unroll
        for (int i = 0; i < NP; ++i) winp[slot][i] = make_float2(src[2 * i], src[2 * i + 1]);
        wins[slot] = src[K - 1];
    };
    bool ok = true;
#pragma unroll
    for (int u = 0; u < K - 1; ++u) load_row(u, u);
    constexpr int NBLK = (kMaxTH + K - 1) / K;
    const int gmask = group - 1;
#pragma unroll 1
    for (int jb = 0; jb < NBLK * K; jb += K) {
#pragma unroll
        for (int jj = 0; jj < K; ++jj) {
            const int j = jb + jj;
            if (j < rows && ok) {
                load_row((jj + K - 1) % K, j + K - 1);
                const int in_group = j & gmask;
                const uint32_t gs = gi & 1;
                if (in_group == 0) ok = mbar_wait_leader(&ctl.acc_full[gs], (gi >> 1) & 1, wc, true);
                if (ok) {
                    tc_fence_after_sync();
                    const uint32_t taddr = tmem_lane_base + (gs * (uint32_t)group + (uint32_t)in_group) * G::NB;
                    float2 acc2[2];
                    float accs = 0.f;
                    acc2[0] = acc2[1] = make_float2(0.f, 0.f);
                    if constexpr (!HILO) {
                        float f[G::kk];
                        tmem_ld_n<G::kk>(taddr, f);
                        tmem_ld_wait();
#pragma unroll
                        for (int col = 0; col < G::kk; ++col) {
                            if (col < G::NPAIRCOLS) {
                                if ((col & 1) == 0) {        // columns col, col + 1 are one pair: taps (a, 2 pi), (a, 2 pi + 1)
                                    const int pr = col / 2, a = pr / NPc, pi = pr % NPc;
                                    acc2[pr & 1] = __ffma2_rn(make_float2(f[col], f[col + 1]), winp[(jj + a) % K][pi], acc2[pr & 1]);
                                }
                            } else {
                                accs = fmaf(f[col], wins[(jj + col - G::NPAIRCOLS) % K], accs);
                            }
                        }
                    } else {
#pragma unroll
                        for (int c0 = 0; c0 < G::kk; c0 += 16) {
                            constexpr int kTail = G::kk % 16;
                            float h[16], l[16];
                            if (c0 + 16 <= G::kk) {
                                tmem_ld_n<16>(taddr + c0, h);
                                tmem_ld_n<16>(taddr + G::NPAD + c0, l);
                            } else {
                                tmem_ld_n<kTail ? kTail : 16>(taddr + c0, h);
                                tmem_ld_n<kTail ? kTail : 16>(taddr + G::NPAD + c0, l);
                            }
                            tmem_ld_wait();
#pragma unroll
                            for (int i = 0; i < 16; ++i) {
                                const int col = c0 + i;
                                if (col < G::NPAIRCOLS) {
                                    if ((col & 1) == 0) {
                                        const int pr = col / 2, a = pr / NPc, pi = pr % NPc;
                                        const float2 w = winp[(jj + a) % K][pi];
                                        acc2[pr & 1] = __ffma2_rn(make_float2(h[i], h[i + 1]), w, acc2[pr & 1]);
                                        acc2[pr & 1] = __ffma2_rn(make_float2(l[i], l[i + 1]), w, acc2[pr & 1]);
                                    }
                                } else if (col < G::kk) {
                                    const int a = col - G::NPAIRCOLS;
                                    accs = fmaf(h[i], wins[(jj + a) % K], accs);
                                    accs = fmaf(l[i], wins[(jj + a) % K], accs);
                                }
                            }
                        }
                    }
                    if (in_group == gmask || j == rows - 1) {    // the group's accumulators have been read
                        tc_fence_before_sync();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&ctl.acc_empty[gs]);
                        ++gi;
                    }
                    const float2 t2 = __fadd2_rn(acc2[0], acc2[1]);
                    float v = (t2.x + t2.y) + accs;
                    if (clamp01) v = fminf(fmaxf(v, 0.f), 1.f);
                    if (in_x) *dst = to_out<OutT>(v);
                    dst += W;
                }
            }
        }
    }
    return ok;
}

template <int K, bool HILO, typename OutT>
__global__ void __launch_bounds__(Geo<K, HILO>::kThreadsMax, Geo<K, HILO>::kCtasPerSm)
regress_tc_kernel(const __grid_constant__ CUtensorMap map_lead, const __grid_constant__ TcParams p)
{
    using G = Geo<K, HILO>;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    __shared__ Ctl ctl;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int nthreads = blockDim.x;
    const Problem& pb = p.g.pb;
    const int C = pb.c;
    const int row_bytes = p.rows_alloc * 256;        // one tile row: two chunks of [rows_alloc][64 pixels] binary16
    const int chunk_bytes = p.rows_alloc * 128;
    const int stage_bytes = p.group * row_bytes;
    const int ksteps = p.dpad / 16;
    const int nbsteps = HILO ? ksteps : (p.alias8 ? 1 : 2 * ksteps);

    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* sA = smem;
    uint8_t* sB = sA + (size_t)p.stages * stage_bytes;
    float* sU = reinterpret_cast<float*>(sB + (size_t)nbsteps * G::KSTEP_B);          // [C][uh][UW]
    float* sV = sU + C * p.g.uh * G::UW;                                                // [C][uh][tcols]
    float* sL = sV + C * p.g.uh * p.g.tcols;                                              // [C * trows][tcols]
    const int dyn_bytes = (int)((uint8_t*)(sL + C * p.g.trows * p.g.tcols) - smem) + 32;  // + a few values read past the last row

    // ---------------------------------------------------------------- set-up
    if (tid == 0) {
        for (int i = 0; i < kMaxStages; ++i) { mbar_init(&ctl.full[i], kLoadThreads + (p.tma_rows > 0 ? 1 : 0)); mbar_init(&ctl.empty[i], 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(&ctl.acc_full[i], 1); mbar_init(&ctl.acc_empty[i], 4 * C); }
        mbar_init(&ctl.lr_full, 32);
        mbar_init(&ctl.lr_empty, 1);
        mbar_init(&ctl.drain, 1);
        ctl.wait.abort_flag = 0;
        ctl.wait.limit = p.wait_cycles;
        fence_barrier_init();
        if (p.tma_rows > 0) prefetch_tensormap(&map_lead);
    }
    // Everything starts as zeros: the copies only ever write rows < natoms of a stage (the padding rows up to dpad must
    // read as zero), only the taps of real atoms are written into the B operand below, and the up-sampling passes read
    // a few staged values beyond the ones they weight (times zero: they must be finite).
    {
        uint4* a4 = reinterpret_cast<uint4*>(smem);
        for (int i = tid; i < dyn_bytes / 16; i += nthreads) a4[i] = make_uint4(0, 0, 0, 0);
    }
    fill_wpad(pb, ctl.wpad, tid, nthreads);
    if (p.gather_planes)
        for (int q = tid; q < p.natoms; q += nthreads) ctl.atoms[q] = (uint8_t)min((int)__ldg(p.idx + q), pb.D - 1);
    __syncthreads();
    // B operand: dict (or gamma-weighted subset rows) as binary16 hi and lo parts, K-major, no swizzle.
    // element (column n, row k) of a K-step: (k%16)/8 * LBO + n/8 * 128 + n%8 * 16 + k%8 * 2
    //   HILO:        K-step k/16, hi in column col, lo in column NPAD + col
    //   stacked:     K-steps 2 (k/16) (hi) and 2 (k/16) + 1 (lo), column col
    //   alias8:      one K-step, hi in row k, lo in row k + 8
    for (int i = tid; i < p.natoms * G::kk; i += nthreads) {
        const int k = i / G::kk, n = i - k * G::kk;
        float v;
        if (p.mode == kModeGlobal) {
            const int a = min((int)__ldg(p.idx + k), pb.D - 1);
            v = __ldg(p.dict + (int64_t)a * G::kk + n) * (p.gamma ? __ldg(p.gamma + k) : 1.f);
        } else {
            v = __ldg(p.dict + (int64_t)k * G::kk + n);
        }
        const __half hi = __float2half_rn(v);
        const __half lo = __float2half_rn(v - __half2float(hi));
        const int col = G::col_of_tap(n);
        const int in_step = ((k & 15) >> 3) * G::LBO_B + (k & 7) * 2;
        if (HILO) {
            uint8_t* base = sB + (k >> 4) * G::KSTEP_B + in_step;
            const int cl = col + G::NPAD;
            *reinterpret_cast<__half*>(base + (col >> 3) * 128 + (col & 7) * 16) = hi;
            *reinterpret_cast<__half*>(base + (cl >> 3) * 128 + (cl & 7) * 16) = lo;
        } else if (p.alias8) {
            uint8_t* base = sB + (col >> 3) * 128 + (col & 7) * 16 + (k & 7) * 2;
            *reinterpret_cast<__half*>(base) = hi;
            *reinterpret_cast<__half*>(base + G::LBO_B) = lo;
        } else {
            uint8_t* base = sB + (k >> 4) * 2 * G::KSTEP_B + in_step + (col >> 3) * 128 + (col & 7) * 16;
            *reinterpret_cast<__half*>(base) = hi;
            *reinterpret_cast<__half*>(base + G::KSTEP_B) = lo;
        }
    }
    fence_proxy_async_smem();
    __syncwarp();
    if (warp == kMmaWarp) tmem_alloc(&ctl.tmem_base, G::TMEM_COLS);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = ctl.tmem_base;
    volatile WaitCtx* wc = &ctl.wait;

    // ---------------------------------------------------------------- roles
    if (warp < 4) {
        setmaxnreg_dec<G::kRegsUtil>();
        if (warp < 2) {
            // ===== coefficient loaders. Thread = (16-byte column c16 of the 128-pixel row, atoms l0 + 4k).
            // A stage row is [chunk of 64 pixels][atom][128 B]; within a 1024-byte group of 8 atoms the 16-byte columns
            // are XOR-swizzled with the atom index (the 128-byte swizzle the MMA descriptor names).
            const int lt = tid;
            const int c16 = lt & 15, l0 = lt >> 4;
            const uint32_t dst_thread0 = (uint32_t)((c16 >> 3) * chunk_bytes + l0 * 128 + (((c16 & 7) ^ l0) << 4));
            const uint32_t dst_thread1 = (uint32_t)((c16 >> 3) * chunk_bytes + (l0 + 4) * 128 + (((c16 & 7) ^ (l0 + 4)) << 4));
            const int64_t plane_elems = (int64_t)pb.H * pb.W;
            // a subset of at most 8 planes: this thread's planes are l0 and l0 + 4, their offsets stay in registers
            const bool few = p.gather_planes && p.natoms <= 8;
            const int64_t goff0 = few && l0 < p.natoms ? (int64_t)ctl.atoms[l0] * plane_elems : 0;
            const int64_t goff1 = few && l0 + 4 < p.natoms ? (int64_t)ctl.atoms[l0 + 4] * plane_elems : 0;
            const bool has0 = l0 < p.natoms, has1 = l0 + 4 < p.natoms;
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            bool lose_one = p.inject_lost_arrival != 0 && blockIdx.x == 0 && tid == 1;
            int issued = 0;
            for (int t = blockIdx.x; t < p.g.num_tiles && ok; t += gridDim.x) {
                int f, y0, x0, rows;
                decode_tile(p.g, t, f, y0, x0, rows);
                const int xe = x0 + c16 * 8;                     // first of this thread's 8 pixels
                const uint32_t src_bytes = xe < pb.W ? 16u : 0u; // columns beyond the image are zero-filled
                const __half* src_row = p.coef + (int64_t)f * p.planes * plane_elems + (int64_t)y0 * pb.W + (xe < pb.W ? xe : 0);
                for (int r0 = 0; r0 < rows; r0 += p.group) {
                    const int nr = min(p.group, rows - r0);
                    ok = mbar_wait_leader(&ctl.empty[s], ph ^ 1, wc, false);
                    if (!ok) break;
                    uint32_t stage_s = smem_u32(sA + (size_t)s * stage_bytes);
                    if (p.tma_rows > 0 && lt == 0) {
                        // planes [0, tma_rows) of both 64-pixel chunks of every row: two boxes per row, bytes counted
                        // on the same barrier
                        uint8_t* sdst = sA + (size_t)s * stage_bytes;
                        mbar_arrive_expect_tx(&ctl.full[s], (uint32_t)(nr * p.tma_rows) * 256u);
                        for (int i = 0; i < nr; ++i, sdst += row_bytes) {
                            tma_load_4d(sdst, &map_lead, &ctl.full[s], x0, y0 + r0 + i, 0, f);
                            tma_load_4d(sdst + chunk_bytes, &map_lead, &ctl.full[s], x0 + 64, y0 + r0 + i, 0, f);
                        }
                    }
                    for (int i = 0; i < nr; ++i, src_row += pb.W, stage_s += (uint32_t)row_bytes) {
                        if (few) {
                            if (has0) cp_async_16(stage_s + dst_thread0, src_row + goff0, src_bytes);
                            if (has1) cp_async_16(stage_s + dst_thread1, src_row + goff1, src_bytes);
                        } else if (!p.gather_planes) {
                            const __half* src = src_row + (p.tma_rows + l0) * plane_elems;
                            uint32_t dst0 = stage_s + dst_thread0 + (uint32_t)p.tma_rows * 128u;
                            uint32_t dst1 = stage_s + dst_thread1 + (uint32_t)p.tma_rows * 128u;
#pragma unroll 2
                            for (int l = p.tma_rows + l0; l < p.natoms; l += 8) {
                                cp_async_16(dst0, src, src_bytes);
                                if (l + 4 < p.natoms) cp_async_16(dst1, src + 4 * plane_elems, src_bytes);
                                dst0 += 1024u;
                                dst1 += 1024u;
                                src += 8 * plane_elems;
                            }
                        } else {
                            uint32_t dst0 = stage_s + dst_thread0, dst1 = stage_s + dst_thread1;
                            for (int l = l0; l < p.natoms; l += 8, dst0 += 1024u, dst1 += 1024u) {
                                cp_async_16(dst0, src_row + (int)ctl.atoms[l] * plane_elems, src_bytes);
                                if (l + 4 < p.natoms) cp_async_16(dst1, src_row + (int)ctl.atoms[l + 4] * plane_elems, src_bytes);
                            }
                        }
                    }
                    // asynchronous arrival: counts on full[s] once this thread's copies above have landed
                    if (lose_one) lose_one = false;
                    else cp_async_mbar_arrive_noinc(&ctl.full[s]);
                    ++issued;
                    if (++s == p.stages) { s = 0; ph ^= 1; }
                }
            }
            cp_async_wait_all();                                 // nothing of this thread is in flight at exit
            if (!ok && lt == 0 && p.tma_rows > 0) {
                // wind-down after a failed wait: boxes issued into stages that were never consumed may still be
                // travelling; give each a short, bounded time to land before the CTA leaves
                int sj = s;
                uint32_t pj = ph;
                const int in_flight = min(issued, p.stages);
                for (int j = 0; j < in_flight; ++j) {
                    if (--sj < 0) { sj += p.stages; pj ^= 1; }
                    mbar_wait_drain(&ctl.full[sj], pj);
                }
            }
        } else if (warp == kMmaWarp) {
            // ===== MMA issuer
            if (lane == 0) {
                constexpr uint32_t idesc = make_idesc_f16(128, G::NB, /*a_mn_major=*/true, /*b_mn_major=*/false);
                // A: MN-major, 128-byte swizzle: 8 atoms x 64 pixels per 1024-byte atom; K-groups 1024 B apart (SBO),
                // the second 64-pixel chunk chunk_bytes away (LBO). A K-step of 16 atoms is 2048 B further on.
                // alias8: the second K-group re-reads the first one (SBO 0) and meets the lo rows of the B operand.
                const uint64_t a_desc0 = make_smem_desc(smem_u32(sA), chunk_bytes, p.alias8 ? 0 : 1024, kSwizzle128B);
                const uint64_t b_desc0 = make_smem_desc(smem_u32(sB), G::LBO_B, 128, kSwizzleNone);
                const uint32_t a_stage_step = (uint32_t)stage_bytes >> 4, a_row_step = (uint32_t)row_bytes >> 4;
                int s = 0;
                uint32_t ph = 0, gi = 0;
                bool ok = true;
                for (int t = blockIdx.x; t < p.g.num_tiles && ok; t += gridDim.x) {
                    int f, y0, x0, rows;
                    decode_tile(p.g, t, f, y0, x0, rows);
                    for (int r0 = 0; r0 < rows; r0 += p.group, ++gi) {
                        const int nr = min(p.group, rows - r0);
                        const uint32_t gs = gi & 1;
                        if (!(ok = mbar_wait(&ctl.acc_empty[gs], ((gi >> 1) & 1) ^ 1, wc))) break;
                        if (!(ok = mbar_wait(&ctl.full[s], ph, wc))) break;
                        fence_proxy_async_smem();    // the stage was written by cp.async (generic proxy), the MMA reads it through the async proxy
                        tc_fence_after_sync();
                        uint64_t arow = a_desc0 + (uint64_t)((uint32_t)s * a_stage_step);
                        uint32_t taddr = tmem_base + gs * (uint32_t)(p.group * G::NB);
                        for (int i = 0; i < nr; ++i, arow += a_row_step, taddr += G::NB) {
                            uint64_t ad = arow, bd = b_desc0;
                            if (HILO || p.alias8) {
                                for (int ks = 0; ks < ksteps; ++ks) {
                                    mma_f16_ss(taddr, ad, bd, idesc, ks > 0);
                                    ad += 2048 >> 4;
                                    bd += G::KSTEP_B >> 4;
                                }
                            } else {
                                for (int ks = 0; ks < ksteps; ++ks) {
                                    mma_f16_ss(taddr, ad, bd, idesc, ks > 0);
                                    mma_f16_ss(taddr, ad, bd + (G::KSTEP_B >> 4), idesc, 1u);
                                    ad += 2048 >> 4;
                                    bd += 2 * (G::KSTEP_B >> 4);
                                }
                            }
                        }
                        mma_commit(&ctl.empty[s]);       // the stage may be refilled once these MMAs have read it
                        mma_commit(&ctl.acc_full[gs]);   // and the group's accumulators are complete
                        if (++s == p.stages) { s = 0; ph ^= 1; }
                    }
                }
                // tensor memory is freed only once every MMA issued here has finished
                mma_commit(&ctl.drain);
                mbar_wait_drain(&ctl.drain, 0);
            }
            __syncwarp();
        } else if (warp == kLrWarp) {
            // ===== LR-window prefetch: the window of tile i + 1 travels while the epilogue works on tile i
            uint32_t ti = 0;
            for (int t = blockIdx.x; t < p.g.num_tiles; t += gridDim.x, ++ti) {
                bool ok = true;
                if (lane == 0) ok = mbar_wait_relaxed(&ctl.lr_empty, (ti & 1) ^ 1, wc);
                if (!__shfl_sync(0xffffffffu, (int)ok, 0)) break;
                prefetch_lr_window<G::P>(p.g, p.lr, t, sL, lane, 32);
                cp_async_mbar_arrive_noinc(&ctl.lr_full);
            }
            cp_async_wait_all();
        }
    } else {
        setmaxnreg_inc<G::kRegsEpi>();
        // ===== epilogue: thread = (pixel column of the tile = TMEM lane, channel)
        const int quarter = warp & 3;                        // the TMEM lanes this warp may read: 32*quarter..+31
        const int ch = (warp - 4) >> 2;
        const int x = quarter * 32 + lane;                   // pixel within the tile row
        const int64_t HW = (int64_t)pb.H * pb.W;
        const bool clamp01 = (pb.flags & SR_CLAMP01) != 0;
        const uint32_t tmem_lane_base = tmem_base + ((uint32_t)(quarter * 32) << 16);
        const int NE = nthreads - kUtilThreads;
        const int et = tid - kUtilThreads;
        // this thread's part of the up-sampling passes: a group of four columns and a row lane
        const int tc4 = p.g.tcols >> 2;
        const int v_lane = fast_div(et, tc4, p.g.tc4_magic), v_i4 = (et - v_lane * tc4) * 4, v_lanes = NE / tc4;
        const int h_lane = et / G::UW4, h_cg = et - h_lane * G::UW4, h_lanes = NE / G::UW4;
        uint32_t gi = 0, ti = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < p.g.num_tiles; t += gridDim.x, ++ti) {
            LrWindow g;
            lr_window<G::P>(p.g, t, g);
            const int uh = g.rows + 2 * G::P;
            ok = ok && mbar_wait_leader(&ctl.lr_full, ti & 1, wc, true);
            ok = named_barrier_and(1, NE, ok);               // LR window landed, previous tile left by every thread
            if (!ok) break;
            if (v_lane < v_lanes) vertical_pass(p.g, g, uh, G::P, sL, sV, v_i4, v_lane, v_lanes);
            named_barrier_sync(1, NE);
            if (et == 0) mbar_arrive(&ctl.lr_empty);         // the LR window may be overwritten
            if (h_lane < h_lanes) horizontal_pass<G::P>(p.g, ctl.wpad, g, uh, sV, sU, h_cg, h_lane, h_lanes);
            named_barrier_sync(1, NE);                       // the U tile is complete
            const bool in_x = g.x0 + x < pb.W;
            OutT* dst = reinterpret_cast<OutT*>(p.out) + ((int64_t)g.f * C + ch) * HW + (int64_t)g.y0 * pb.W + g.x0 + x;
            ok = epilogue_tile<K, HILO, OutT>(ctl, sU + ch * p.g.uh * G::UW + x, dst, pb.W, g.rows, p.group, gi, tmem_lane_base, in_x,
                                              clamp01, lane, wc);
        }
    }

    // ---------------------------------------------------------------- teardown
    __syncwarp();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (ctl.wait.abort_flag && tid == 0) atomicExch(p.status, SR_ERR_TIMEOUT);
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

struct DeviceInfo { int sms = 0, cc_major = 0, smem_sm = 0, smem_optin = 0; bool ok = false; };

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
        if (cudaDeviceGetAttribute(&d.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) return none;
        d.ok = true;
    }
    return d;
}

constexpr int kStaticReserve = 4096;   // static shared memory (control block) + the per-CTA system reservation

// Shape of a launch: everything the host decides.
struct Plan {
    bool ok = false;
    bool hilo = false;
    int natoms = 0, gather = 0, dpad = 0, rows_alloc = 0, alias8 = 0;
    int th = 0, group = 0, stages = 0;
    size_t smem = 0;
    int ctas = 0;
};

template <int K, bool HILO>
size_t fixed_smem_bytes(const Problem& pb, int nbsteps, int th)
{
    using G = Geo<K, HILO>;
    Geom g;
    return 1024 /* alignment slack */ + 32 + (size_t)nbsteps * G::KSTEP_B + plan_geom(g, pb, th, nullptr) * sizeof(float);
}

// Planes that enter the contraction, and whether they are picked one by one out of a full tensor.
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

// Tile height, rows per pipeline step and stage count. The tiles of a launch are dealt round-robin to the resident
// CTAs, so the launch takes as long as the CTA with the most tiles: cost(th) = ceil(tiles(th) / CTAs) * (steps(th) *
// hand-over + th + per-tile work that does not shrink with the tile), in units of one tile row.
template <int K, bool HILO>
Plan make_plan_k(int mode, const Problem& pb, const TcTuning& tune)
{
    using G = Geo<K, HILO>;
    Plan pl;
    const DeviceInfo& di = device_info();
    if (!di.ok) return pl;
    contraction_shape(mode, pb, pl.natoms, pl.gather);
    pl.hilo = HILO;
    pl.dpad = (pl.natoms + 15) / 16 * 16;
    pl.rows_alloc = (pl.natoms + 7) / 8 * 8;
    pl.alias8 = (!HILO && pl.natoms <= 8) ? 1 : 0;
    const int ksteps = pl.dpad / 16;
    const int nbsteps = HILO ? ksteps : (pl.alias8 ? 1 : 2 * ksteps);
    const int per_cta = G::kCtasPerSm == 2 ? di.smem_sm / 2 - kStaticReserve : di.smem_optin - kStaticReserve;
    const int tiles_x = (pb.W + TW - 1) / TW;
    const int ctas_max = di.sms * G::kCtasPerSm;
    const size_t row_bytes = (size_t)pl.rows_alloc * 256;
    double best = 0.0;
    for (int th = kMaxTH; th >= 4; --th) {
        if (tune.th > 0 && th != tune.th) continue;
        const size_t fixed = fixed_smem_bytes<K, HILO>(pb, nbsteps, th);
        // rows per step: as many as leave three stages (two at the least)
        int group = 0, stages = 0;
        for (int gr = G::MAX_GROUP; gr >= 1; gr >>= 1) {
            if (tune.group > 0 && gr != tune.group) continue;
            if (fixed + 2 * gr * row_bytes > (size_t)per_cta) continue;
            const int st = (int)(((size_t)per_cta - fixed) / (gr * row_bytes));
            if (st < 3 && gr > 1 && tune.group == 0) continue;
            group = gr;
            stages = st > kMaxStages ? kMaxStages : st;
            break;
        }
        if (group == 0) continue;
        const long long tiles = (long long)tiles_x * ((pb.H + th - 1) / th) * pb.n;
        const int ctas = tiles < ctas_max ? (int)tiles : ctas_max;
        const long long waves = (tiles + ctas - 1) / ctas;
        const int steps = (th + group - 1) / group;
        const double cost = (double)waves * (th + 0.75 * steps + 2.5);
        if (!pl.ok || cost < best) {
            pl.ok = true;
            best = cost;
            pl.th = th; pl.group = group; pl.stages = stages;
            pl.smem = fixed + (size_t)stages * group * row_bytes;
            pl.ctas = ctas;
        }
    }
    return pl;
}

// hi and lo halves stacked along K while the atoms are few (the extra MMAs are cheap then); side by side along N otherwise
bool use_hilo(int natoms) { return natoms > 32; }

Plan make_plan(int mode, const Problem& pb, const TcTuning& g_tune)
{
    int natoms, gather;
    contraction_shape(mode, pb, natoms, gather);
    const bool hilo = use_hilo(natoms);
    switch (pb.k) {
    case 1: return hilo ? make_plan_k<1, true>(mode, pb, g_tune) : make_plan_k<1, false>(mode, pb, g_tune);
    case 3: return hilo ? make_plan_k<3, true>(mode, pb, g_tune) : make_plan_k<3, false>(mode, pb, g_tune);
    case 5: return hilo ? make_plan_k<5, true>(mode, pb, g_tune) : make_plan_k<5, false>(mode, pb, g_tune);
    case 7: return hilo ? make_plan_k<7, true>(mode, pb, g_tune) : make_plan_k<7, false>(mode, pb, g_tune);
    default: return Plan{};
    }
}

template <int K, bool HILO, typename OutT>
cudaError_t launch_kho(const CUtensorMap& map_lead, const TcParams& prm, const Plan& pl, cudaStream_t st)
{
    using G = Geo<K, HILO>;
    auto kern = regress_tc_kernel<K, HILO, OutT>;
    static bool configured[64] = {false};   // per template instance and device
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!configured[dev]) {
        const DeviceInfo& di = device_info();
        const int lim = G::kCtasPerSm == 2 ? di.smem_sm / 2 - kStaticReserve : di.smem_optin - kStaticReserve;
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, lim);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    kern<<<pl.ctas, kUtilThreads + 128 * prm.g.pb.c, pl.smem, st>>>(map_lead, prm);
    count_launches(1);
    return cudaGetLastError();
}

template <int K, bool HILO>
cudaError_t launch_kh(const CUtensorMap& map_lead, const TcParams& prm, const Plan& pl, cudaStream_t st)
{
    if (prm.g.pb.flags & SR_OUT_U8) return launch_kho<K, HILO, uint8_t>(map_lead, prm, pl, st);
    if (prm.g.pb.flags & SR_OUT_F16) return launch_kho<K, HILO, __half>(map_lead, prm, pl, st);
    return launch_kho<K, HILO, float>(map_lead, prm, pl, st);
}

template <int K>
cudaError_t launch_k(const CUtensorMap& map_lead, const TcParams& prm, const Plan& pl, cudaStream_t st)
{
    return pl.hilo ? launch_kh<K, true>(map_lead, prm, pl, st) : launch_kh<K, false>(map_lead, prm, pl, st);
}

} // namespace

// Every legal launch shape of this path for the problem: tile heights 4..16 x rows per pipeline step {1, 2, 4}, kept
// when the shared memory of a CTA (stages, B operand, up-sampling buffers), its tensor-memory columns (two groups of
// accumulators) and the stage count (>= 2) allow it. The tile-shape search times these.
int regress_tc_candidates(int mode, const Problem& pb, TcTuning* out, int max_out)
{
    int n = 0;
    for (int th = kMaxTH; th >= 4; --th)
        for (int group = kMaxGroupRows; group >= 1; group >>= 1) {
            TcTuning t;
            t.th = th;
            t.group = group;
            const Plan pl = make_plan(mode, pb, t);
            if (pl.ok && pl.th == th && pl.group == group && n < max_out) out[n++] = t;
        }
    return n;
}

bool regress_tc_supported(int mode, const void* coef, int coef_dtype, const Problem& pb)
{
    if (mode != kModeDense && mode != kModeGlobal) return false;
    if (coef_dtype != SR_F16) return false;
    if (pb.k > 7 || pb.c > kMaxC) return false;
    if ((reinterpret_cast<uintptr_t>(coef) & 15) != 0 || (pb.W & 7) != 0) return false;   // 16-byte copies: aligned base and row pitch
    if (pb.n > 65535) return false;
    const DeviceInfo& di = device_info();
    if (!di.ok || di.cc_major != 10) return false;
    return make_plan(mode, pb, TcTuning{}).ok;
}

cudaError_t launch_regress_tc(int mode, const float* lr, const void* coef, const uint8_t* idx, const float* gamma,
                              const float* dict, float* out, const Problem& pb, cudaStream_t st, const TcTuning& tune)
{
    const Plan pl = make_plan(mode, pb, tune);
    if (!pl.ok) return cudaErrorNotSupported;
    TcParams prm{};
    prm.lr = lr; prm.dict = dict; prm.out = out; prm.idx = idx; prm.gamma = gamma;
    prm.coef = static_cast<const __half*>(coef);
    prm.status = device_status_word();
    if (!prm.status) return cudaErrorUnknown;
    plan_geom(prm.g, pb, pl.th, lr);
    prm.mode = mode;
    prm.natoms = pl.natoms; prm.gather_planes = pl.gather; prm.dpad = pl.dpad; prm.rows_alloc = pl.rows_alloc;
    prm.alias8 = pl.alias8;
    prm.planes = (mode == kModeGlobal && (pb.flags & SR_COEF_COMPACT)) ? pb.s : pb.D;
    prm.stages = pl.stages;
    prm.group = pl.group;
    prm.wait_cycles = wait_cycle_limit();
    prm.inject_lost_arrival = take_injected_lost_arrival() ? 1 : 0;

    // Split of the coefficient stream between the SM's two load paths: the leading planes of a stage row through one
    // TMA box per 64-pixel chunk, the rest through cp.async. Subsets gathered plane by plane use cp.async only.
    CUtensorMap map_lead{};
    prm.tma_rows = 0;
    if (!prm.gather_planes && encode_fn() && prm.natoms >= 16) {
        const int lead = (prm.natoms / 2) / 8 * 8;
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
    case 1: return launch_k<1>(map_lead, prm, pl, st);
    case 3: return launch_k<3>(map_lead, prm, pl, st);
    case 5: return launch_k<5>(map_lead, prm, pl, st);
    case 7: return launch_k<7>(map_lead, prm, pl, st);
    default: return cudaErrorNotSupported;
    }
}

} // namespace sr
