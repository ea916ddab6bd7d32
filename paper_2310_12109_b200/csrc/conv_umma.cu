#include "conv_umma.h"

namespace m2u {
cudaError_t create_tables(m2_plan*) { return cudaSuccess; }
void destroy_tables(m2_plan*) {}
int32_t conv_fwd(const m2_plan*, const void*, const void*, void*, int64_t, int64_t, int64_t, int32_t, cudaStream_t) {
    return M2_ERR_UNSUPPORTED;
}
}  // namespace m2u
