// Tensor-core Monarch matmul for 64 x 64 blocks (internal header).
#pragma once
#include <cuda_runtime.h>

#include "m2_plan.h"

namespace m2mm {
bool covered(const m2_plan* plan);
int64_t workspace_bytes(const m2_plan* plan, int64_t T);
cudaError_t prepare(const m2_plan* plan);
// two passes (R then L) exchanging the intermediate through `ws` (workspace_bytes(plan, T) bytes); Y may be X.
// Kmul != nullptr: Y = sigma(K (.) M X) with K [Hk][4096] bf16, row t uses K[t % Hk], sigma = ReLU if relu else identity
int32_t matmul(const m2_plan* plan, const void* X, const void* L, const void* R, void* Y, int64_t T, void* ws, const void* Kmul,
               int64_t Hk, int relu, cudaStream_t stream);
// the same two launches in the mode of m2_selftest_bounded_wait_matmul: nothing is issued to the tensor core, every wait for it
// gives up after a few polls, Y and ws are not written
int32_t matmul_wait_selftest(const m2_plan* plan, const void* X, const void* L, const void* R, void* Y, int64_t T, void* ws,
                             cudaStream_t stream);
// gradients with respect to L and R on the tensor cores (fp32 results, bf16 intermediate); ws: wgrad_workspace_bytes
int64_t wgrad_workspace_bytes(const m2_plan* plan, int64_t T);
int32_t wgrad(const m2_plan* plan, const void* X, const void* G, const void* L, const void* R, float* dL, float* dR, int64_t T, void* ws,
              cudaStream_t stream);
}  // namespace m2mm
