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

// The kernel is instantiated for two tile heights: 16 rows for the dense / global-subset modes (less halo work
// per pixel) and 8 rows for the selective mode, whose smaller U tile leaves room for eight coefficient stages.
namespace th16 {
#define SR_UMMA_TH 16
#include "sr_umma_impl.inc"
#undef SR_UMMA_TH
} // namespace th16

namespace th8 {
#define SR_UMMA_TH 8
#include "sr_umma_impl.inc"
#undef SR_UMMA_TH
} // namespace th8

} // namespace

// Tile height per mode: 16 rows wherever the shape still leaves the selective pipeline its eight stages (dense and
// global-subset modes always; the in-kernel selection when the single U buffer it needs fits), else 8 rows.
static bool tall_tiles(int mode, const void* coef, int coef_dtype, const Problem& pb)
{
    if (!th8::is_selective(mode)) return true;
    return th16::supported(mode, coef, coef_dtype, pb) && th16::stage_count(mode, pb) >= 8;
}

bool umma_supported(int mode, const void* coef, int coef_dtype, const Problem& pb)
{
    return tall_tiles(mode, coef, coef_dtype, pb) ? th16::supported(mode, coef, coef_dtype, pb) : th8::supported(mode, coef, coef_dtype, pb);
}

cudaError_t launch_regress_umma(int mode, const float* lr, const void* coef, const uint8_t* idx, const float* gamma,
                                const float* dict, float* out, const Problem& pb, cudaStream_t st)
{
    return tall_tiles(mode, coef, SR_F16, pb) ? th16::launch(mode, lr, coef, idx, gamma, dict, out, pb, st)
                                               : th8::launch(mode, lr, coef, idx, gamma, dict, out, pb, st);
}

} // namespace sr
