// Thin wrappers over the sm_100a PTX this library uses: mbarrier, TMA (cp.async.bulk.tensor), tcgen05
// (tensor-core MMA with TMEM accumulators). Every wait is bounded: after a cycle budget it gives up and
// reports failure so that a kernel can set its status word, drain and return instead of spinning forever.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace sr {
namespace ptx {

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// ---- mbarrier ------------------------------------------------------------------------------------------------------

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}

__device__ __forceinline__ void fence_barrier_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

__device__ __forceinline__ void mbar_arrive(uint64_t* bar)
{
    asm volatile("{\n\t.reg .b64 st;\n\tmbarrier.arrive.shared::cta.b64 st, [%0];\n\t}" ::"r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes)
{
    asm volatile("{\n\t.reg .b64 st;\n\tmbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1;\n\t}" ::"r"(smem_u32(bar)),
                 "r"(bytes)
                 : "memory");
}

// One try: the hardware may park the thread for up to ~`hint_ns` before answering, which keeps a waiting
// warp out of the issue slots without delaying its wake-up when the phase completes.
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity, uint32_t hint_ns = 2000u)
{
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(smem_u32(bar)), "r"(parity), "r"(hint_ns)
        : "memory");
    return done != 0;
}

// Default cycle budget of one wait (about a second at B200 clocks); the host can lower it per launch.
constexpr long long kWaitCycleLimit = 1ll << 31;
// Budget of the waits a CTA makes while it winds down after a failed wait (copies and MMAs still in flight finish
// within microseconds; a phase that can never complete must not hold the exit up for long).
constexpr long long kDrainCycleLimit = 1ll << 21;

// Per-CTA state of the bounded waits (shared memory): the flag a thread raises when its wait ran out, which every
// other wait of the CTA polls, and the cycle budget of one wait.
struct WaitCtx {
    int abort_flag;
    int reserved;
    long long limit;
};

// Whole-warp wait: lane 0 polls, the result is broadcast. Returns the same value in every lane.
__device__ __forceinline__ bool mbar_wait_warp(uint64_t* bar, uint32_t parity, volatile WaitCtx* wc);

// Waits for the phase with the given parity to complete. Returns false when the budget ran out or
// another thread of the CTA has already raised the abort flag.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile WaitCtx* wc)
{
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    const long long limit = const_cast<const WaitCtx*>(wc)->limit;   // fixed for the launch: read once, not per poll
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        if (wc->abort_flag) return false;
        if (clock64() - t0 > limit) {
            wc->abort_flag = 1;
            return false;
        }
    }
}

// The same wait for roles that have time to spare: between tests the thread sleeps, so that its polling does not take
// issue slots and shared-memory cycles from the warps that set the pace.
__device__ __forceinline__ bool mbar_wait_relaxed(uint64_t* bar, uint32_t parity, volatile WaitCtx* wc)
{
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    const long long limit = const_cast<const WaitCtx*>(wc)->limit;
    while (true) {
        __nanosleep(64);
        if (mbar_try_wait(bar, parity)) return true;
        if (wc->abort_flag) return false;
        if (clock64() - t0 > limit) {
            wc->abort_flag = 1;
            return false;
        }
    }
}

// Whole-warp wait in which only lane 0 polls (the other lanes block at the warp barrier and take no issue slots or
// shared-memory cycles meanwhile). Lane 0's successful test is an acquire; the warp barrier orders it before what the
// other lanes do next. `relaxed`: lane 0 sleeps between tests. Returns the same value in every lane.
__device__ __forceinline__ bool mbar_wait_leader(uint64_t* bar, uint32_t parity, volatile WaitCtx* wc, bool relaxed)
{
    int ok = 1;
    if ((threadIdx.x & 31) == 0) ok = (relaxed ? mbar_wait_relaxed(bar, parity, wc) : mbar_wait(bar, parity, wc)) ? 1 : 0;
    ok = __shfl_sync(0xffffffffu, ok, 0);
    __syncwarp();
    return ok != 0;
}

// A wait of the wind-down after a failure: own short budget, ignores (and never raises) the abort flag.
__device__ __forceinline__ bool mbar_wait_drain(uint64_t* bar, uint32_t parity)
{
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (clock64() - t0 > kDrainCycleLimit) return false;
    }
    return true;
}

__device__ __forceinline__ bool mbar_wait_warp(uint64_t* bar, uint32_t parity, volatile WaitCtx* wc)
{
    int ok = 1;
    if ((threadIdx.x & 31) == 0) ok = mbar_wait(bar, parity, wc) ? 1 : 0;
    ok = __shfl_sync(0xffffffffu, ok, 0);
    // Lanes other than 0 did not observe the barrier themselves: one successful test gives them the acquire. The
    // phase lane 0 saw complete cannot be left behind before this warp has used it, so that test succeeds; a lane
    // whose test fails all the same falls back to the bounded wait, and the warp agrees on the outcome.
    if (ok && !mbar_try_wait(bar, parity, 0u)) ok = mbar_wait(bar, parity, wc) ? 1 : 0;
    return __all_sync(0xffffffffu, ok != 0);
}

// Whole-warp wait in which every lane tests the barrier itself (one shared-memory round trip when the phase is
// already complete, against three for mbar_wait_warp: lane 0's test, the shuffle, the other lanes' test). `seen`:
// the result of a test issued earlier (true = the phase was already complete then, nothing left to do).
__device__ __forceinline__ bool mbar_wait_lanes(uint64_t* bar, uint32_t parity, volatile WaitCtx* wc, bool seen)
{
    if (__all_sync(0xffffffffu, seen)) return true;
    return mbar_wait(bar, parity, wc);
}

// The same, with an outcome the whole warp agrees on (the vote is only taken when the early test had failed): for
// callers whose next instruction is warp-collective.
__device__ __forceinline__ bool mbar_wait_lanes_uniform(uint64_t* bar, uint32_t parity, volatile WaitCtx* wc, bool seen)
{
    if (__all_sync(0xffffffffu, seen)) return true;
    return __all_sync(0xffffffffu, mbar_wait(bar, parity, wc));
}

// ---- proxies / fences ----------------------------------------------------------------------------------------------

// Makes shared-memory writes of the generic proxy visible to the async proxy (TMA, tcgen05.mma operands).
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tc_fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// ---- TMA -----------------------------------------------------------------------------------------------------------

__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* map)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)map) : "memory");
}

// 4-D tiled load global -> shared, completion on an mbarrier (bytes counted as transaction bytes).
// c0 (innermost coordinate) times the element size must be a multiple of 16 bytes.
__device__ __forceinline__ void tma_load_4d(void* dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1, int c2, int c3)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(smem_u32(dst)), "l"((uint64_t)map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}

// 1-D bulk copy global -> shared, completion on an mbarrier (bytes counted as transaction bytes). Both addresses
// 16-byte aligned, the size a multiple of 16 bytes.
__device__ __forceinline__ void bulk_load_1d(void* dst, const void* src, uint32_t bytes, uint64_t* bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

// ---- tensor memory -------------------------------------------------------------------------------------------------

// Whole warp. Writes the TMEM base address of `ncols` columns (power of two >= 32) to *dst (shared memory).
__device__ __forceinline__ void tmem_alloc(uint32_t* dst, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst)), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}

// ---- tcgen05.mma ---------------------------------------------------------------------------------------------------

enum SmemLayout : uint64_t { kSwizzleNone = 0, kSwizzle128B = 2, kSwizzle64B = 4, kSwizzle32B = 6 };

// Shared-memory matrix descriptor. Addresses and offsets in bytes (multiples of 16).
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint64_t layout)
{
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;            // descriptor version of this architecture
    d |= layout << 61;
    return d;
}

// Instruction descriptor for kind::f16: fp16 A and B, fp32 accumulator, M x N tile.
__host__ __device__ constexpr uint32_t make_idesc_f16(int M, int N, bool a_mn_major, bool b_mn_major)
{
    return (1u << 4)                          // accumulator format: f32
           | (0u << 7) | (0u << 10)           // A, B format: f16
           | ((a_mn_major ? 1u : 0u) << 15) | ((b_mn_major ? 1u : 0u) << 16)
           | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// D[tmem] (+)= A[smem] * B[smem]; one thread issues.
__device__ __forceinline__ void mma_f16_ss(uint32_t taddr, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(taddr), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// Arrives on the mbarrier once every tcgen05.mma issued so far by this thread has completed.
__device__ __forceinline__ void mma_commit(uint64_t* bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// TMEM -> registers: this warp's 32 lanes, 16 consecutive 32-bit columns per thread.
__device__ __forceinline__ void tmem_ld_x16(uint32_t taddr, float* v)
{
    uint32_t* r = reinterpret_cast<uint32_t*>(v);
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}

__device__ __forceinline__ void tmem_ld_x8(uint32_t taddr, float* v)
{
    uint32_t* r = reinterpret_cast<uint32_t*>(v);
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr)
                 : "memory");
}

__device__ __forceinline__ void tmem_ld_x4(uint32_t taddr, float* v)
{
    uint32_t* r = reinterpret_cast<uint32_t*>(v);
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(taddr)
                 : "memory");
}

__device__ __forceinline__ void tmem_ld_x1(uint32_t taddr, float* v)
{
    uint32_t* r = reinterpret_cast<uint32_t*>(v);
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];" : "=r"(r[0]) : "r"(taddr) : "memory");
}

// Loads N (1..16) consecutive columns with the fewest instructions of width 16, 8, 4, 1.
template <int N>
__device__ __forceinline__ void tmem_ld_n(uint32_t taddr, float* v)
{
    if constexpr (N >= 16) {
        tmem_ld_x16(taddr, v);
        if constexpr (N > 16) tmem_ld_n<N - 16>(taddr + 16, v + 16);
    } else if constexpr (N >= 8) {
        tmem_ld_x8(taddr, v);
        if constexpr (N > 8) tmem_ld_n<N - 8>(taddr + 8, v + 8);
    } else if constexpr (N >= 4) {
        tmem_ld_x4(taddr, v);
        if constexpr (N > 4) tmem_ld_n<N - 4>(taddr + 4, v + 4);
    } else if constexpr (N >= 1) {
        tmem_ld_x1(taddr, v);
        if constexpr (N > 1) tmem_ld_n<N - 1>(taddr + 1, v + 1);
    }
}

} // namespace ptx
} // namespace sr
