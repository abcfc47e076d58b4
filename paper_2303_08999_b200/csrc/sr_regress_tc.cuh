// Tensor-core regression path, second layout (channel-split epilogue, two CTAs per SM): declarations.
#pragma once
#include "sr_common.cuh"

namespace sr {

// True when this path can run the problem (dense and global-subset modes, binary16 coefficients, aligned, c <= 3).
bool regress_tc_supported(int mode, const void* coef, int coef_dtype, const Problem& pb);

// Launch shape; a zero leaves the choice to the host's cost model.
struct TcTuning {
    int th = 0;      // tile height, 4..16
    int group = 0;   // tile rows per pipeline step: 1, 2 or 4
};

cudaError_t launch_regress_tc(int mode, const float* lr, const void* coef, const uint8_t* idx, const float* gamma,
                              const float* dict, float* out, const Problem& pb, cudaStream_t st, const TcTuning& tune = TcTuning{});

// Every launch shape the problem admits (shared memory, tensor memory, stage count); returns how many were written.
int regress_tc_candidates(int mode, const Problem& pb, TcTuning* out, int max_out);

} // namespace sr
