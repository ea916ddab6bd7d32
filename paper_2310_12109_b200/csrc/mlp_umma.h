// Tensor-core block-diagonal MLP of the M2 block, 192 -> 768 -> 192 per block (internal header).
#pragma once
#include <cuda_runtime.h>

#include "m2_plan.h"

namespace m2mlp {
// C / nblk == 192 inputs per block and expand * 192 == 768 hidden per block
bool covered(int C, int nblk, int expand);
// y[tokens][C] = per block j: W_down[j] GELU(W_up[j] z[:, block j]); z, y bf16 (may alias: a CTA reads its tile
// of z before it writes the same tile of y); W_up [nblk][768][192], W_down [nblk][192][768] bf16; `status`
// receives M2_ERR_TIMEOUT if a bounded wait expires
// z_channel_first_T != 0: z is [tokens / T][C][T] (channel-first, T a multiple of 128 that divides tokens) instead of
// [tokens][C]; y is [tokens][C] either way (and must then not alias z)
int32_t launch(const void* z, const void* Wup, const void* Wdn, void* y, int C, int nblk, long long tokens, int32_t* status,
               cudaStream_t stream, long long z_channel_first_T = 0);
}  // namespace m2mlp
