// Tensor-core Monarch product on a matrix whose columns are the vectors (internal header).
#pragma once
#include <cuda_runtime.h>

#include "m2_plan.h"

namespace m2c {
// order-2 bf16 plans whose two factors are multiples of 64 (up to 1024), d a multiple of 8
bool covered(const m2_plan* plan, int64_t d);
// Y[bt] = sigma(K (.) M X[bt]) for Bt matrices [N][d]; Kmul: [N][d] (shared by the batch) or nullptr; ws: Bt * N * d bf16 values
int32_t apply(const m2_plan* plan, const void* X, const void* L, const void* R, const void* Kmul, int relu, void* Y, int64_t Bt,
              int64_t d, void* ws, cudaStream_t stream);
// O[bt] = W V[bt]: W [c][c] (outputs x inputs), V, O [Bt][c][cols] with cols contiguous; c a multiple of 64, cols of 8, bf16
bool dense_covered(const m2_plan* plan, int64_t c, int64_t cols);
int32_t dense(const m2_plan* plan, const void* W, const void* V, void* O, int64_t Bt, int64_t c, int64_t cols, cudaStream_t stream);
}  // namespace m2c
