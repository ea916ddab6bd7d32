// Plan object and host-side integer tables of the Monarch library (internal header).
#pragma once
#include <cstdint>
#include <vector>

#include "../../include/m2.h"

struct m2_umma_tables;  // device constants of the tensor-core convolution path (conv_umma.cu)

struct m2_plan {
    int64_t N = 0;
    int32_t p = 0;
    int32_t dims[4] = {1, 1, 1, 1};
    int32_t dtype = M2_FP32;
    int32_t sign = +1;
    int32_t device = -1;

    // integer tables (App. D notation): bit-exact contract with the oracle
    std::vector<int32_t> perm, perm_inv, digit_rev;
    std::vector<std::vector<int32_t>> tw_exp;  // tw_exp[s-1], s = 1..p-1

    // device side
    int32_t* d_status = nullptr;  // error word set by kernels (bounded waits, self checks)
    float2* d_roots[4] = {nullptr, nullptr, nullptr, nullptr};  // omega_{Na}^j, j < Na, per stage
    m2_umma_tables* umma = nullptr;

    mutable const char* last_kernel = "none";
    mutable int64_t launches = 0;
};

// sigma_(b,N)(i) = (i mod b) * (N / b) + i / b
inline void m2_fill_stride_perm(int64_t b, int64_t N, std::vector<int32_t>& out) {
    out.resize(N);
    for (int64_t i = 0; i < N; ++i) out[i] = (int32_t)((i % b) * (N / b) + i / b);
}
