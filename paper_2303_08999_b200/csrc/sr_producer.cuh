// Regression fused with the producer of Phi (last convolution + pixel-shuffle of the coefficient network): declarations.
#pragma once
#include "sr_common.cuh"

namespace sr {

// Shape of the producer layer. cin = feature channels of the LR map, kc = side of the convolution kernel.
struct ProducerShape {
    int cin, kc;
};

// True when the fused kernel runs the problem: scale 2, 3 or 4, k in {3, 5, 7} (k <= 5 at scale 3), c <= 3, cin = 32,
// kc in {1, 3}.
bool producer_supported(const Problem& pb, const ProducerShape& ps);

// Bytes of the folded-weights block for the problem (0 when it is not supported).
size_t producer_folded_bytes(const Problem& pb, const ProducerShape& ps);

// Folds the dictionary (all atoms, or the subset idx[s] with weights gamma[s]) into the convolution's weights and bias
// and writes them in the order the fused kernel streams them.
cudaError_t launch_producer_fold(const float* wconv, const float* bias, const float* dict, const uint8_t* idx,
                                 const float* gamma, int s, void* folded, const Problem& pb, const ProducerShape& ps,
                                 cudaStream_t st);

// The fused kernel: features -> (tensor cores) per-pixel filters -> filtered, up-sampled image.
cudaError_t launch_producer_regress(const float* lr, const void* feat, const void* folded, void* out, const Problem& pb,
                                    const ProducerShape& ps, cudaStream_t st);

} // namespace sr
