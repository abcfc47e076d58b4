// Tensor-core regression path (placeholder until the tcgen05 kernel lands: reports "not supported").
#include "sr_umma.cuh"

namespace sr {

bool umma_supported(int, const void*, int, const Problem&) { return false; }

cudaError_t launch_regress_umma(int, const float*, const void*, const uint8_t*, const float*, const float*, float*,
                                const Problem&, cudaStream_t)
{
    return cudaErrorNotSupported;
}

} // namespace sr
