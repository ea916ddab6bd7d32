// Learnable (causal) Monarch matrices built from polynomial coefficients and the convolution through them (internal header).
#pragma once
#include <cuda_runtime.h>

#include "m2_plan.h"

namespace m2b {

// order-2 plans with N1 == N2 = b, 2 <= b <= 64
bool covered(const m2_plan* plan);
// L | R | L^-1 | R^-1, each [b][b][b] complex fp32; -1 for plans not covered
int64_t factors_bytes(const m2_plan* plan);
int32_t build(const m2_plan* plan, const float* Lt, const float* Rt, int masked, void* factors, cudaStream_t stream);
int32_t spectrum(const m2_plan* plan, const void* factors, const float* k, int64_t H, int64_t n, void* kf, cudaStream_t stream);
int32_t conv_fwd(const m2_plan* plan, const void* factors, const void* x, const void* kf, void* y, int64_t B, int64_t H, int64_t n,
                 cudaStream_t stream);

}  // namespace m2b
