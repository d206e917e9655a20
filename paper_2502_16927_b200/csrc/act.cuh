// Activation sigma of the BigMac expert (Eq. 4) and its derivative, fp32, device side.
#pragma once
#include "bigmac.h"

namespace bigmac {

__device__ __forceinline__ float act_apply(int act, float z) {
    switch (act) {
        case BIGMAC_ACT_RELU: return z > 0.0f ? z : 0.0f;
        case BIGMAC_ACT_GELU_ERF: return 0.5f * z * (1.0f + erff(z * 0.70710678118654752f));
        case BIGMAC_ACT_GELU_TANH: {
            const float w = 0.79788456080286536f * (z + 0.044715f * z * z * z);
            return 0.5f * z * (1.0f + tanhf(w));
        }
        default: return z;
    }
}

__device__ __forceinline__ float act_grad(int act, float z) {
    switch (act) {
        case BIGMAC_ACT_RELU: return z > 0.0f ? 1.0f : 0.0f;
        case BIGMAC_ACT_GELU_ERF: {
            const float cdf = 0.5f * (1.0f + erff(z * 0.70710678118654752f));
            const float pdf = 0.39894228040143268f * expf(-0.5f * z * z);
            return cdf + z * pdf;
        }
        case BIGMAC_ACT_GELU_TANH: {
            const float w = 0.79788456080286536f * (z + 0.044715f * z * z * z);
            const float th = tanhf(w);
            const float dw = 0.79788456080286536f * (1.0f + 0.134145f * z * z);
            return 0.5f * (1.0f + th) + 0.5f * z * (1.0f - th * th) * dw;
        }
        default: return 1.0f;
    }
}

}  // namespace bigmac
