// Tensor-core (tcgen05 + TMEM + TMA) regression path: declarations.
#pragma once
#include "sr_common.cuh"

namespace sr {

// True when the tensor-core path can run this problem (dtype, alignment, sizes); otherwise the FMA path is used.
bool umma_supported(int mode, const void* coef, int coef_dtype, const Problem& pb);

cudaError_t launch_regress_umma(int mode, const float* lr, const void* coef, const uint8_t* idx, const float* gamma,
                                const float* dict, float* out, const Problem& pb, cudaStream_t st);

} // namespace sr
