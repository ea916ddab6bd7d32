// C ABI of libm2: plan management, host-side validation, dispatch to the kernels.
#include <cuda_runtime.h>

#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "blocky_monarch.h"
#include "conv_umma.h"
#include "generic_kernels.h"
#include "cols_umma.h"
#include "matmul_umma.h"
#include "mlp_umma.h"
#include "m2_plan.h"

// Scratch of m2_block_fwd_static: the intermediate z of the block forward for callers that cannot
// allocate.  In host code this name is only a handle for cudaGetSymbolAddress, never a device pointer.
static __device__ __align__(256) unsigned char g_block_static_scratch[M2_STATIC_SCRATCH_BYTES];

namespace {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) ok = false;
        if (ok && prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard() {
        if (prev >= 0) cudaSetDevice(prev);
    }
};

void build_tables(m2_plan* pl) {
    const int64_t N = pl->N;
    const int p = pl->p;
    const int64_t N1 = pl->dims[0];
    m2_fill_stride_perm(N1, N, pl->perm);
    m2_fill_stride_perm(N / N1, N, pl->perm_inv);
    // plan position [k1][k2]..[kp] row-major -> k = k1 + N1 k2 + ..
    pl->digit_rev.resize(N);
    for (int64_t pos = 0; pos < N; ++pos) {
        int64_t rem = pos, k = 0;
        int64_t digit[4];
        for (int a = p - 1; a >= 0; --a) {
            digit[a] = rem % pl->dims[a];
            rem /= pl->dims[a];
        }
        int64_t w = 1;
        for (int a = 0; a < p; ++a) {
            k += w * digit[a];
            w *= pl->dims[a];
        }
        pl->digit_rev[pos] = (int32_t)k;
    }
    // twiddle exponents: before digit n_{s+1} is contracted (s = 1..p-1) the element at position
    // [k1]..[ks][n_{s+1}]..[np] is scaled by omega_{N1..N_{s+1}}^{ n_{s+1} * (k1 + N1 k2 + ..) }
    pl->tw_exp.assign(p > 1 ? p - 1 : 0, std::vector<int32_t>());
    for (int s = 1; s < p; ++s) {
        std::vector<int32_t>& t = pl->tw_exp[s - 1];
        t.resize(N);
        int64_t Mcur = 1;
        for (int a = 0; a <= s; ++a) Mcur *= pl->dims[a];
        for (int64_t pos = 0; pos < N; ++pos) {
            int64_t rem = pos;
            int64_t digit[4];
            for (int a = p - 1; a >= 0; --a) {
                digit[a] = rem % pl->dims[a];
                rem /= pl->dims[a];
            }
            int64_t kappa = 0, w = 1;
            for (int a = 0; a < s; ++a) {
                kappa += w * digit[a];
                w *= pl->dims[a];
            }
            t[pos] = (int32_t)((digit[s] * kappa) % Mcur);
        }
    }
}

m2g::ConvShape conv_shape(const m2_plan* pl, int64_t B, int64_t H, int64_t n) {
    m2g::ConvShape s;
    s.p = pl->p;
    for (int a = 0; a < 3; ++a) {
        s.dims[a] = a < pl->p ? pl->dims[a] : 1;
        s.roots[a] = a < pl->p ? pl->d_roots[a] : nullptr;
    }
    s.sign = pl->sign;
    s.B = B;
    s.H = H;
    s.n = n;
    s.stride_b = H * n;
    s.stride_h = n;
    s.stride_e = 1;
    return s;
}

int32_t check_conv_args(const m2_plan* plan, const void* x, const void* kf, void* y, int64_t B, int64_t H, int64_t n,
                        int32_t mode) {
    if (!plan) return M2_ERR_INVALID_ARG;
    if (B < 0 || H < 0 || n <= 0) return M2_ERR_INVALID_ARG;
    if ((!x || !kf || !y) && B * H != 0) return M2_ERR_INVALID_ARG;  // empty batches may carry null pointers
    if (plan->device < 0) return M2_ERR_NO_DEVICE;
    if (mode == M2_CAUSAL) {
        if (2 * n > plan->N) return M2_ERR_INVALID_ARG;
    } else if (mode == M2_CIRCULAR) {
        if (n != plan->N) return M2_ERR_INVALID_ARG;
    } else {
        return M2_ERR_INVALID_ARG;
    }
    if (plan->p < 2 || plan->p > 3) return M2_ERR_UNSUPPORTED;
    if (!aligned16(x) || !aligned16(kf) || !aligned16(y)) return M2_ERR_ALIGNMENT;
    if (B * H > 0x7fffffffLL) return M2_ERR_UNSUPPORTED;
    return M2_OK;
}

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
void* g_static_ptr[kMaxDevices] = {nullptr};   // per device: address of g_block_static_scratch

}  // namespace

extern "C" {

int32_t m2_plan_create(m2_plan** out, int64_t N, int32_t p, const int32_t* factors, int32_t dtype, int32_t sign,
                       int32_t device) {
    if (!out) return M2_ERR_INVALID_ARG;
    *out = nullptr;
    if (!factors || p < 1 || p > 3 || N <= 0 || N > (1 << 24)) return M2_ERR_INVALID_ARG;
    if (dtype != M2_FP32 && dtype != M2_BF16) return M2_ERR_INVALID_ARG;
    if (sign != 1 && sign != -1) return M2_ERR_INVALID_ARG;
    int64_t prod = 1;
    for (int a = 0; a < p; ++a) {
        if (factors[a] <= 0) return M2_ERR_INVALID_ARG;
        prod *= factors[a];
    }
    if (prod != N) return M2_ERR_INVALID_ARG;
    m2_plan* pl = new (std::nothrow) m2_plan();
    if (!pl) return M2_ERR_INVALID_ARG;
    pl->N = N;
    pl->p = p;
    for (int a = 0; a < p; ++a) pl->dims[a] = factors[a];
    pl->dtype = dtype;
    pl->sign = sign;
    pl->device = device;
    build_tables(pl);
    if (device >= 0) {
        DeviceGuard g(device);
        bool ok = g.ok;
        if (ok) ok = cudaMalloc(&pl->d_status, sizeof(int32_t)) == cudaSuccess;
        if (ok) ok = cudaMemset(pl->d_status, 0, sizeof(int32_t)) == cudaSuccess;
        for (int a = 0; a < p && ok; ++a) {
            const int Na = pl->dims[a];
            std::vector<float2> r(Na);
            for (int j = 0; j < Na; ++j) {
                const double ang = 2.0 * M_PI * (double)j / (double)Na;
                r[j] = make_float2((float)std::cos(ang), (float)(sign * std::sin(ang)));
            }
            ok = cudaMalloc(&pl->d_roots[a], sizeof(float2) * Na) == cudaSuccess &&
                 cudaMemcpy(pl->d_roots[a], r.data(), sizeof(float2) * Na, cudaMemcpyHostToDevice) == cudaSuccess;
        }
        if (ok) ok = m2u::create_tables(pl) == cudaSuccess;
        if (ok) ok = m2u3::create_tables(pl) == cudaSuccess;
        if (ok) ok = m2mm::prepare(pl) == cudaSuccess;
        if (ok) ok = cudaDeviceSynchronize() == cudaSuccess;
        if (!ok) {
            cudaGetLastError();
            m2_plan_destroy(pl);
            return M2_ERR_CUDA;
        }
    }
    *out = pl;
    return M2_OK;
}

int32_t m2_plan_destroy(m2_plan* plan) {
    if (!plan) return M2_ERR_INVALID_ARG;
    if (plan->device >= 0) {
        DeviceGuard g(plan->device);
        cudaDeviceSynchronize();
        m2u::destroy_tables(plan);
        m2u3::destroy_tables(plan);
        if (plan->d_status) cudaFree(plan->d_status);
        for (int a = 0; a < 4; ++a)
            if (plan->d_roots[a]) cudaFree(plan->d_roots[a]);
    }
    delete plan;
    return M2_OK;
}

int32_t m2_plan_get_table(const m2_plan* plan, int32_t which, int32_t* host_out, int64_t len) {
    if (!plan || !host_out || len != plan->N) return M2_ERR_INVALID_ARG;
    const std::vector<int32_t>* src = nullptr;
    if (which == M2_TABLE_PERM) src = &plan->perm;
    else if (which == M2_TABLE_PERM_INV) src = &plan->perm_inv;
    else if (which == M2_TABLE_DIGIT_REV) src = &plan->digit_rev;
    else if (which > M2_TABLE_TW_EXP && which < M2_TABLE_TW_EXP + plan->p) src = &plan->tw_exp[which - M2_TABLE_TW_EXP - 1];
    if (!src) return M2_ERR_INVALID_ARG;
    std::memcpy(host_out, src->data(), sizeof(int32_t) * (size_t)len);
    return M2_OK;
}

int64_t m2_spectrum_bytes(const m2_plan* plan, int64_t H) {
    if (!plan || H < 0) return -1;
    return H * plan->N * (int64_t)sizeof(float2) * (m2u::has_private_spectrum(plan) ? 2 : 1);
}

int32_t m2_kernel_spectrum(const m2_plan* plan, const float* k_dev, int64_t H, int64_t n, void* kf_dev, void* stream) {
    if (!plan || !k_dev || !kf_dev) return M2_ERR_INVALID_ARG;
    if (plan->device < 0) return M2_ERR_NO_DEVICE;
    if (H < 0 || n <= 0 || n > plan->N) return M2_ERR_INVALID_ARG;
    if (plan->p < 2 || plan->p > 3) return M2_ERR_UNSUPPORTED;
    if (!aligned16(kf_dev)) return M2_ERR_ALIGNMENT;
    DeviceGuard g(plan->device);
    if (!g.ok) return M2_ERR_CUDA;
    m2g::ConvShape s = conv_shape(plan, 1, H, n);
    cudaError_t e = m2g::launch_spectrum(s, k_dev, kf_dev, (cudaStream_t)stream);
    if (e == cudaErrorInvalidValue) return M2_ERR_UNSUPPORTED;
    if (e != cudaSuccess) return M2_ERR_CUDA;
    if (m2u::relayout_spectrum(plan, kf_dev, H, (cudaStream_t)stream) != cudaSuccess) return M2_ERR_CUDA;
    plan->last_kernel = "spectrum_generic_fp32";
    plan->launches += (H > 0) * (m2u::has_private_spectrum(plan) ? 2 : 1);
    return M2_OK;
}

int32_t m2_spectrum_to_natural(const m2_plan* plan, const void* kf_dev, int64_t H, float* out_dev, void* stream) {
    if (!plan || !kf_dev || !out_dev || H < 0) return M2_ERR_INVALID_ARG;
    if (plan->device < 0) return M2_ERR_NO_DEVICE;
    DeviceGuard g(plan->device);
    if (!g.ok) return M2_ERR_CUDA;
    m2g::ConvShape s = conv_shape(plan, 1, H, plan->N);
    if (m2g::launch_spectrum_to_natural(s, kf_dev, out_dev, (cudaStream_t)stream) != cudaSuccess) return M2_ERR_CUDA;
    plan->launches += (H > 0);
    return M2_OK;
}

int64_t m2_conv_bwd_workspace_bytes(const m2_plan* plan, int64_t B, int64_t H) {
    if (!plan || B < 0 || H < 0) return -1;
    const int64_t u2 = m2u::conv_wgrad_workspace_bytes(plan, B, H), u3 = m2u3::conv_wgrad_workspace_bytes(plan, B, H);
    const int64_t umma = u2 > u3 ? u2 : u3, generic = m2g::conv_wgrad_scratch_bytes(plan->N, H);
    return umma > generic ? umma : generic;
}

int32_t m2_monarch_conv_bwd_kernel(const m2_plan* plan, const void* x_dev, const void* g_dev, float* dk_dev, int64_t B, int64_t H,
                                   int64_t n, int32_t mode, void* ws_dev, int64_t ws_bytes, void* stream) {
    // same argument rules as the forward call (dk plays the part of the output for the null / alignment checks)
    int32_t st = check_conv_args(plan, x_dev, g_dev, dk_dev, B, H, n, mode);
    if (st != M2_OK) return st;
    if (H > 0 && !dk_dev) return M2_ERR_INVALID_ARG;   // an empty batch still writes zeros
    DeviceGuard g(plan->device);
    if (!g.ok) return M2_ERR_CUDA;
    if (H == 0) return M2_OK;
    if (ws_dev && !aligned16(ws_dev)) return M2_ERR_ALIGNMENT;
    m2g::ConvShape s = conv_shape(plan, B, H, n);
    const int64_t need = m2u::conv_wgrad_workspace_bytes(plan, B, H);
    if (need > 0 && B > 0 && ws_dev && ws_bytes >= need) {   // tensor-core transforms and products, CUDA-core sum + inverse
        int parts = 0;
        st = m2u::conv_wgrad_partials(plan, x_dev, g_dev, ws_dev, B, H, n, mode, &parts, (cudaStream_t)stream);
        if (st == M2_OK) {
            st = m2u::conv_wgrad_finish(plan, ws_dev, parts, dk_dev, H, n, (cudaStream_t)stream);
            if (st != M2_OK) return st;
            plan->last_kernel = "conv_wgrad_umma_o2_512";
            return M2_OK;
        }
        if (st != M2_ERR_UNSUPPORTED) return st;
    }
    const int64_t need3 = m2u3::conv_wgrad_workspace_bytes(plan, B, H);
    if (need3 > 0 && B > 0 && ws_dev && ws_bytes >= need3) {   // N = 32768: the order-3 tensor-core kernel, three launches
        st = m2u3::conv_wgrad(plan, x_dev, g_dev, dk_dev, B, H, n, mode, ws_dev, (cudaStream_t)stream);
        if (st != M2_ERR_UNSUPPORTED) return st;
    }
    const cudaError_t e = m2g::launch_conv_wgrad(s, plan->dtype == M2_BF16, x_dev, g_dev, dk_dev, ws_dev, ws_bytes, (cudaStream_t)stream);
    if (e == cudaErrorInvalidValue) return M2_ERR_UNSUPPORTED;
    if (e != cudaSuccess) return M2_ERR_CUDA;
    plan->last_kernel = "conv_wgrad_generic";
    plan->launches += 1;
    return M2_OK;
}

int32_t m2_spectrum_conjugate(const m2_plan* plan, const void* kf_in_dev, int64_t H, void* kf_out_dev, void* stream) {
    if (!plan || !kf_in_dev || !kf_out_dev || H < 0) return M2_ERR_INVALID_ARG;
    if (plan->device < 0) return M2_ERR_NO_DEVICE;
    if (!aligned16(kf_in_dev) || !aligned16(kf_out_dev)) return M2_ERR_ALIGNMENT;
    DeviceGuard g(plan->device);
    if (!g.ok) return M2_ERR_CUDA;
    const long long values = H * plan->N;   // complex values per layout; N is even for every plan with a device path
    if (plan->N % 2 != 0) return M2_ERR_UNSUPPORTED;
    if (m2g::launch_spectrum_conj(kf_in_dev, kf_out_dev, values, m2u::has_private_spectrum(plan) ? values : 0, (cudaStream_t)stream) !=
        cudaSuccess)
        return M2_ERR_CUDA;
    plan->launches += (H > 0);
    return M2_OK;
}

// y = conv(k[h / kf_group], x[b][h]); arguments beyond kf_group checked here
static int32_t conv_fwd_grouped(const m2_plan* plan, const void* x_dev, const void* kf_dev, void* y_dev, int64_t B, int64_t H, int64_t n,
                                int32_t mode, int64_t kf_group, void* stream) {
    int32_t st = check_conv_args(plan, x_dev, kf_dev, y_dev, B, H, n, mode);
    if (st != M2_OK) return st;
    if (kf_group < 1 || kf_group > 0x7fffffffLL || H % kf_group != 0) return M2_ERR_INVALID_ARG;
    DeviceGuard g(plan->device);
    if (!g.ok) return M2_ERR_CUDA;
    if (B * H == 0) return M2_OK;
    // tensor-core path where a kernel exists for the shape, CUDA-core path otherwise
    int32_t ust = m2u::conv_fwd(plan, x_dev, kf_dev, y_dev, B, H, n, mode, (cudaStream_t)stream, (int)kf_group);
    if (ust == M2_ERR_UNSUPPORTED && kf_group == 1) ust = m2u3::conv_fwd(plan, x_dev, kf_dev, y_dev, B, H, n, mode, (cudaStream_t)stream);
    if (ust == M2_OK) return M2_OK;
    if (ust != M2_ERR_UNSUPPORTED) return ust;
    m2g::ConvShape s = conv_shape(plan, B, H, n);
    s.kf_group = (int)kf_group;
    cudaError_t e = m2g::launch_conv(s, plan->dtype == M2_BF16, x_dev, kf_dev, y_dev, nullptr, (cudaStream_t)stream);
    if (e == cudaErrorInvalidValue) return M2_ERR_UNSUPPORTED;
    if (e != cudaSuccess) return M2_ERR_CUDA;
    plan->last_kernel = plan->dtype == M2_BF16 ? "conv_generic_bf16io" : "conv_generic_fp32";
    plan->launches += 1;
    return M2_OK;
}

int32_t m2_monarch_conv_fwd(const m2_plan* plan, const void* x_dev, const void* kf_dev, void* y_dev, int64_t B,
                            int64_t H, int64_t n, int32_t mode, void* stream) {
    return conv_fwd_grouped(plan, x_dev, kf_dev, y_dev, B, H, n, mode, 1, stream);
}

int32_t m2_monarch_conv_fwd_grouped(const m2_plan* plan, const void* x_dev, const void* kf_dev, void* y_dev, int64_t B, int64_t H,
                                    int64_t n, int32_t mode, int64_t kf_group, void* stream) {
    return conv_fwd_grouped(plan, x_dev, kf_dev, y_dev, B, H, n, mode, kf_group, stream);
}

int32_t m2_selftest_bounded_wait(const m2_plan* plan, const void* x_dev, const void* kf_dev, void* y_dev, int64_t B, int64_t H, int64_t n,
                                 int32_t mode, void* stream) {
    int32_t st = check_conv_args(plan, x_dev, kf_dev, y_dev, B, H, n, mode);
    if (st != M2_OK) return st;
    DeviceGuard g(plan->device);
    if (!g.ok) return M2_ERR_CUDA;
    if (B * H == 0) return M2_ERR_UNSUPPORTED;
    return m2u::conv_fwd_wait_selftest(plan, x_dev, kf_dev, y_dev, B, H, n, mode, (cudaStream_t)stream);
}

int32_t m2_monarch_conv_fwd_host(const m2_plan* plan, const void* x_host, const void* kf_dev, void* y_host,
                                 void* x_dev_scratch, void* y_dev_scratch, int64_t B, int64_t H, int64_t n, int32_t mode,
                                 void* stream) {
    if (!x_host || !y_host) return M2_ERR_INVALID_ARG;
    int32_t st = check_conv_args(plan, x_dev_scratch, kf_dev, y_dev_scratch, B, H, n, mode);
    if (st != M2_OK) return st;
    DeviceGuard g(plan->device);
    if (!g.ok) return M2_ERR_CUDA;
    const size_t bytes = (size_t)B * H * n * (plan->dtype == M2_BF16 ? 2 : 4);
    if (bytes == 0) return M2_OK;
    if (cudaMemcpyAsync(x_dev_scratch, x_host, bytes, cudaMemcpyHostToDevice, (cudaStream_t)stream) != cudaSuccess)
        return M2_ERR_CUDA;
    st = m2_monarch_conv_fwd(plan, x_dev_scratch, kf_dev, y_dev_scratch, B, H, n, mode, stream);
    if (st != M2_OK) return st;
    if (cudaMemcpyAsync(y_host, y_dev_scratch, bytes, cudaMemcpyDeviceToHost, (cudaStream_t)stream) != cudaSuccess)
        return M2_ERR_CUDA;
    return M2_OK;
}

static int32_t check_matmul_args(const m2_plan* plan, const void* X, const void* L, const void* R, void* Y, int64_t T) {
    if (!plan || T < 0) return M2_ERR_INVALID_ARG;
    if ((!X || !L || !R || !Y) && T != 0) return M2_ERR_INVALID_ARG;  // an empty batch may carry null pointers
    if (plan->device < 0) return M2_ERR_NO_DEVICE;
    if (plan->p != 2) return M2_ERR_UNSUPPORTED;
    if (!aligned16(X) || !aligned16(L) || !aligned16(R) || !aligned16(Y)) return M2_ERR_ALIGNMENT;
    if (T > 0x7fffffffLL) return M2_ERR_UNSUPPORTED;
    return M2_OK;
}

int64_t m2_matmul_workspace_bytes(const m2_plan* plan, int64_t T) {
    if (!plan || T < 0) return -1;
    return m2mm::workspace_bytes(plan, T);
}

// Y = sigma(K (.) M X) (K == nullptr: Y = M X); arguments already checked, device already current
static int32_t matmul_impl(const m2_plan* plan, const void* X_dev, const void* L_dev, const void* R_dev, void* Y_dev, int64_t T,
                           void* ws_dev, int64_t ws_bytes, const void* K_dev, int64_t Hk, int relu, cudaStream_t stream) {
    if (T == 0) return M2_OK;
    if (m2mm::covered(plan) && ws_dev && ws_bytes >= m2mm::workspace_bytes(plan, T))
        return m2mm::matmul(plan, X_dev, L_dev, R_dev, Y_dev, T, ws_dev, K_dev, Hk, relu, stream);
    cudaError_t e = m2g::launch_matmul(plan->dims[0], plan->dims[1], T, plan->dtype == M2_BF16, X_dev, L_dev, R_dev, Y_dev, K_dev,
                                       Hk > 0 ? Hk : 1, relu, stream);
    if (e == cudaErrorInvalidValue) return M2_ERR_UNSUPPORTED;
    if (e != cudaSuccess) return M2_ERR_CUDA;
    plan->last_kernel = "matmul_generic";
    plan->launches += 1;
    return M2_OK;
}

int32_t m2_monarch_matmul(const m2_plan* plan, const void* X_dev, const void* L_dev, const void* R_dev, void* Y_dev,
                          int64_t T, void* ws_dev, int64_t ws_bytes, void* stream) {
    int32_t st = check_matmul_args(plan, X_dev, L_dev, R_dev, Y_dev, T);
    if (st != M2_OK) return st;
    if (ws_dev && !aligned16(ws_dev)) return M2_ERR_ALIGNMENT;
    DeviceGuard g(plan->device);
    if (!g.ok) return M2_ERR_CUDA;
    return matmul_impl(plan, X_dev, L_dev, R_dev, Y_dev, T, ws_dev, ws_bytes, nullptr, 1, 0, (cudaStream_t)stream);
}

int32_t m2_monarch_apply_order_p(const m2_plan* plan, const void* X_dev, const void* const* W_dev, void* Y_dev, int64_t T, void* stream) {
    if (!plan || T < 0 || !W_dev) return M2_ERR_INVALID_ARG;
    if (plan->device < 0) return M2_ERR_NO_DEVICE;
    if (plan->p < 1 || plan->p > 4) return M2_ERR_UNSUPPORTED;
    if ((!X_dev || !Y_dev) && T != 0) return M2_ERR_INVALID_ARG;
    for (int a = 0; a < plan->p; ++a) {
        if (!W_dev[a] && T != 0) return M2_ERR_INVALID_ARG;
        if (!aligned16(W_dev[a])) return M2_ERR_ALIGNMENT;
    }
    if (!aligned16(X_dev) || !aligned16(Y_dev)) return M2_ERR_ALIGNMENT;
    if (T > 0x7fffffffLL) return M2_ERR_UNSUPPORTED;
    if (T == 0) return M2_OK;
    DeviceGuard g(plan->device);
    if (!g.ok) return M2_ERR_CUDA;
    cudaError_t e = m2g::launch_order_p(plan->dims, plan->p, T, plan->dtype == M2_BF16, X_dev, W_dev, Y_dev, (cudaStream_t)stream);
    if (e == cudaErrorInvalidValue) return M2_ERR_UNSUPPORTED;
    if (e != cudaSuccess) return M2_ERR_CUDA;
    plan->last_kernel = "monarch_order_p_generic";
    plan->launches += 1;
    return M2_OK;
}

int32_t m2_selftest_bounded_wait_matmul(const m2_plan* plan, const void* X_dev, const void* L_dev, const void* R_dev, void* Y_dev,
                                        int64_t T, void* ws_dev, int64_t ws_bytes, void* stream) {
    int32_t st = check_matmul_args(plan, X_dev, L_dev, R_dev, Y_dev, T);
    if (st != M2_OK) return st;
    if (ws_dev && !aligned16(ws_dev)) return M2_ERR_ALIGNMENT;
    DeviceGuard g(plan->device);
    if (!g.ok) return M2_ERR_CUDA;
    if (T == 0 || !m2mm::covered(plan) || !ws_dev || ws_bytes < m2mm::workspace_bytes(plan, T)) return M2_ERR_UNSUPPORTED;
    return m2mm::matmul_wait_selftest(plan, X_dev, L_dev, R_dev, Y_dev, T, ws_dev, (cudaStream_t)stream);
}

int32_t m2_monarch_mix(const m2_plan* plan, const void* X_dev, const void* K_dev, int64_t Hk, int32_t act, const void* La_dev,
                       const void* Ra_dev, const void* Lb_dev, const void* Rb_dev, void* Y_dev, int64_t T, void* ws_dev,
                       int64_t ws_bytes, void* stream) {
    int32_t st = check_matmul_args(plan, X_dev, La_dev, Ra_dev, Y_dev, T);
    if (st != M2_OK) return st;
    if (act != M2_ACT_NONE && act != M2_ACT_RELU) return M2_ERR_INVALID_ARG;
    if (T > 0 && (!K_dev || !Lb_dev || !Rb_dev || Hk < 1)) return M2_ERR_INVALID_ARG;
    if (!aligned16(K_dev) || !aligned16(Lb_dev) || !aligned16(Rb_dev) || (ws_dev && !aligned16(ws_dev))) return M2_ERR_ALIGNMENT;
    DeviceGuard g(plan->device);
    if (!g.ok) return M2_ERR_CUDA;
    // the intermediate sigma(K (.) M_a X) lives in Y: every kernel of the second product reads its tokens before it writes them
    st = matmul_impl(plan, X_dev, La_dev, Ra_dev, Y_dev, T, ws_dev, ws_bytes, K_dev, Hk, act == M2_ACT_RELU, (cudaStream_t)stream);
    if (st != M2_OK) return st;
    return matmul_impl(plan, Y_dev, Lb_dev, Rb_dev, Y_dev, T, ws_dev, ws_bytes, nullptr, 1, 0, (cudaStream_t)stream);
}

static int64_t round256(int64_t v) { return (v + 255) / 256 * 256; }

// Y[bt] = sigma(K (.) M X[bt]) on [Bt][N][d]; arguments already checked, device already current
static int32_t cols_impl(const m2_plan* plan, const void* X_dev, const void* L_dev, const void* R_dev, const void* K_dev, int relu, void* Y_dev,
                         int64_t Bt, int64_t d, void* ws_dev, cudaStream_t stream) {
    int32_t st = m2c::apply(plan, X_dev, L_dev, R_dev, K_dev, relu, Y_dev, Bt, d, ws_dev, stream);
    if (st != M2_ERR_UNSUPPORTED) return st;
    const cudaError_t e = m2g::launch_monarch_cols(plan->dims[0], plan->dims[1], Bt, (int)d, plan->dtype == M2_BF16, X_dev, L_dev, R_dev, K_dev,
                                                   relu, Y_dev, ws_dev, stream);
    if (e == cudaErrorInvalidValue) return M2_ERR_UNSUPPORTED;
    if (e != cudaSuccess) return M2_ERR_CUDA;
    plan->last_kernel = "monarch_cols_generic";
    plan->launches += 2;
    return M2_OK;
}

int32_t m2_monarch_cols(const m2_plan* plan, const void* X_dev, const void* L_dev, const void* R_dev, const void* K_dev, int32_t act,
                        void* Y_dev, int64_t Bt, int64_t d, void* ws_dev, int64_t ws_bytes, void* stream) {
    if (!plan || Bt < 0 || d < 0) return M2_ERR_INVALID_ARG;
    if (act != M2_ACT_NONE && act != M2_ACT_RELU) return M2_ERR_INVALID_ARG;
    if (plan->device < 0) return M2_ERR_NO_DEVICE;
    if (plan->p != 2) return M2_ERR_UNSUPPORTED;
    const int64_t elems = Bt * plan->N * d;
    if (elems == 0) return M2_OK;
    if (!X_dev || !L_dev || !R_dev || !Y_dev || !ws_dev) return M2_ERR_INVALID_ARG;
    if (!aligned16(X_dev) || !aligned16(L_dev) || !aligned16(R_dev) || !aligned16(K_dev) || !aligned16(Y_dev) || !aligned16(ws_dev))
        return M2_ERR_ALIGNMENT;
    const bool bf = plan->dtype == M2_BF16;
    if (ws_bytes < elems * (bf ? 2 : 4)) return M2_ERR_INVALID_ARG;
    if (d > 0x7fffffffLL) return M2_ERR_UNSUPPORTED;
    DeviceGuard g(plan->device);
    if (!g.ok) return M2_ERR_CUDA;
    return cols_impl(plan, X_dev, L_dev, R_dev, K_dev, act == M2_ACT_RELU, Y_dev, Bt, d, ws_dev, (cudaStream_t)stream);
}

int64_t m2_layer_scratch_bytes(const m2_plan* plan_n, const m2_plan* plan_d, int64_t B) {
    if (!plan_n || !plan_d || B < 0) return -1;
    const int64_t es = plan_n->dtype == M2_BF16 ? 2 : 4;
    return 3 * round256(B * plan_n->N * plan_d->N * es) + round256(plan_n->N * plan_d->N * es);
}

int32_t m2_layer_fwd(const m2_plan* plan_n, const m2_plan* plan_d, const void* x_dev, const void* const* factors, const void* n_kernel_dev,
                     const void* d_kernel_dev, const float* gamma_dev, const float* beta_dev, float eps, void* y_dev, int64_t B,
                     void* scratch_dev, int64_t scratch_bytes, void* ws_dev, int64_t ws_bytes, void* stream) {
    if (!plan_n || !plan_d || !factors || B < 0 || !(eps >= 0.f)) return M2_ERR_INVALID_ARG;
    if (plan_n->device < 0 || plan_d->device < 0) return M2_ERR_NO_DEVICE;
    if (plan_n->p != 2 || plan_d->p != 2) return M2_ERR_UNSUPPORTED;
    if (plan_n->dtype != plan_d->dtype || plan_n->device != plan_d->device) return M2_ERR_INVALID_ARG;
    const int64_t n = plan_n->N, d = plan_d->N;
    if (B > 65535 || B * n > 0x7fffffffLL || B * d > 0x7fffffffLL) return M2_ERR_UNSUPPORTED;
    if (B == 0) return M2_OK;
    for (int i = 0; i < 8; ++i)
        if (!factors[i] || !aligned16(factors[i])) return factors[i] ? M2_ERR_ALIGNMENT : M2_ERR_INVALID_ARG;
    if (!x_dev || !n_kernel_dev || !d_kernel_dev || !gamma_dev || !beta_dev || !y_dev || !scratch_dev) return M2_ERR_INVALID_ARG;
    if (!aligned16(x_dev) || !aligned16(n_kernel_dev) || !aligned16(d_kernel_dev) || !aligned16(y_dev) || !aligned16(scratch_dev) ||
        (ws_dev && !aligned16(ws_dev)))
        return M2_ERR_ALIGNMENT;
    const bool bf = plan_n->dtype == M2_BF16;
    const int64_t tensor_bytes = B * n * d * (bf ? 2 : 4);
    if (scratch_bytes < m2_layer_scratch_bytes(plan_n, plan_d, B)) return M2_ERR_INVALID_ARG;
    DeviceGuard g(plan_n->device);
    if (!g.ok) return M2_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    unsigned char* sc = static_cast<unsigned char*>(scratch_dev);
    void* s1 = sc;                                   // [B, n, d]: relu(K_n (.) M1 x)      (or [B, d, n] on the transposing route)
    void* s2 = sc + round256(tensor_bytes);          // [B, n, d]: x~
    void* s3 = sc + 2 * round256(tensor_bytes);      // [B, n, d]: the intermediate between the two factors of M1 / M2
    void* kt = sc + 3 * round256(tensor_bytes);      // [n, d]: the sequence kernel with the channels contiguous
    // Sequence mix.  x is [B, n, d] with the channels contiguous, i.e. the COLUMNS of each [n, d] matrix are the vectors M1, M2
    // act on: no transposition of the activations, only of the [d, n] kernel parameter.
    if (m2g::launch_transpose_any(n_kernel_dev, kt, 1, (int)d, (int)n, bf, st) != cudaSuccess) return M2_ERR_CUDA;
    int32_t rc = cols_impl(plan_n, x_dev, factors[0], factors[1], kt, 1, s1, B, d, s3, st);
    if (rc == M2_OK) rc = cols_impl(plan_n, s1, factors[2], factors[3], nullptr, 0, s2, B, d, s3, st);
    int extra = 2;   // launches beyond the products: kernel transpose + normalisation
    if (rc == M2_ERR_UNSUPPORTED) {   // n too large for the CUDA-core column kernel: transpose the activations instead
        if (m2g::launch_transpose_any(x_dev, s1, B, (int)n, (int)d, bf, st) != cudaSuccess) return M2_ERR_CUDA;
        rc = matmul_impl(plan_n, s1, factors[0], factors[1], s1, B * d, ws_dev, ws_bytes, n_kernel_dev, d, 1, st);
        if (rc == M2_OK) rc = matmul_impl(plan_n, s1, factors[2], factors[3], s1, B * d, ws_dev, ws_bytes, nullptr, 1, 0, st);
        if (rc != M2_OK) return rc;
        if (m2g::launch_transpose_any(s1, s2, B, (int)d, (int)n, bf, st) != cudaSuccess) return M2_ERR_CUDA;
        extra = 4;
    }
    if (rc != M2_OK) return rc;
    rc = matmul_impl(plan_d, s2, factors[4], factors[5], y_dev, B * n, ws_dev, ws_bytes, d_kernel_dev, 1, 1, st);
    if (rc == M2_OK) rc = matmul_impl(plan_d, y_dev, factors[6], factors[7], y_dev, B * n, ws_dev, ws_bytes, nullptr, 1, 0, st);
    if (rc != M2_OK) return rc;
    if (m2g::launch_add_layernorm(y_dev, s2, gamma_dev, beta_dev, y_dev, B * n, (int)d, eps, bf, st) != cudaSuccess) return M2_ERR_CUDA;
    plan_n->launches += extra;   // (the products count themselves on their plans)
    plan_n->last_kernel = "layer_fwd";
    return M2_OK;
}

int64_t m2_bert_mixer_scratch_bytes(const m2_plan* plan, int64_t B, int64_t d) {
    if (!plan || B < 0 || d < 0) return -1;
    return 8 * round256(B * d * plan->N * (plan->dtype == M2_BF16 ? 2 : 4));
}

int32_t m2_bert_mixer_fwd(const m2_plan* plan, const void* x_dev, const void* const* W, const float* const* w_short, const void* kf_dev,
                          const void* kf_res_dev, void* y_dev, int64_t B, int64_t d, void* scratch_dev, int64_t scratch_bytes, void* stream) {
    if (!plan || !W || !w_short || B < 0 || d <= 0) return M2_ERR_INVALID_ARG;
    if (plan->device < 0) return M2_ERR_NO_DEVICE;
    const int64_t n = plan->N;   // bidirectional: circular convolution over the whole plan length
    if (B > 65535 || d > 65535 || B * d * n > 0x7fffffffffLL) return M2_ERR_UNSUPPORTED;
    if (B == 0) return M2_OK;
    for (int i = 0; i < 4; ++i)
        if (!W[i] || !aligned16(W[i])) return W[i] ? M2_ERR_ALIGNMENT : M2_ERR_INVALID_ARG;
    for (int i = 0; i < 3; ++i)
        if (!w_short[i]) return M2_ERR_INVALID_ARG;
    if (!x_dev || !kf_dev || !kf_res_dev || !y_dev || !scratch_dev) return M2_ERR_INVALID_ARG;
    if (!aligned16(x_dev) || !aligned16(y_dev) || !aligned16(scratch_dev)) return M2_ERR_ALIGNMENT;
    if (scratch_bytes < m2_bert_mixer_scratch_bytes(plan, B, d)) return M2_ERR_INVALID_ARG;
    DeviceGuard g(plan->device);
    if (!g.ok) return M2_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    const bool bf = plan->dtype == M2_BF16;
    const int64_t tb = round256(B * d * n * (bf ? 2 : 4));
    unsigned char* sc = static_cast<unsigned char*>(scratch_dev);
    void *xT = sc, *Pq = sc + tb, *Pk = sc + 2 * tb, *Pv = sc + 3 * tb, *QK = sc + 4 * tb, *C = sc + 5 * tb, *Cr = sc + 6 * tb, *Z = sc + 7 * tb;
    auto dense = [&](const void* Wm, const void* V, void* O) -> int32_t {   // O[b] = Wm V[b] on [B][d][n]
        int32_t rc = m2c::dense(plan, Wm, V, O, B, d, n, st);
        if (rc != M2_ERR_UNSUPPORTED) return rc;
        const cudaError_t e = m2g::launch_dense_cols(Wm, V, O, B, (int)d, (int)n, bf, st);
        if (e == cudaErrorInvalidValue) return M2_ERR_UNSUPPORTED;
        if (e != cudaSuccess) return M2_ERR_CUDA;
        plan->launches += 1;
        return M2_OK;
    };
    if (m2g::launch_transpose_any(x_dev, xT, B, (int)n, (int)d, bf, st) != cudaSuccess) return M2_ERR_CUDA;   // channel-first from here on
    int32_t rc = dense(W[0], xT, Pq);
    if (rc == M2_OK) rc = dense(W[1], xT, Pk);
    if (rc == M2_OK) rc = dense(W[2], xT, Pv);
    if (rc != M2_OK) return rc;
    if (m2g::launch_gate_in(Pq, Pk, w_short[0], w_short[1], QK, B, (int)d, (int)n, bf, st) != cudaSuccess) return M2_ERR_CUDA;
    // the residual convolution first; on the N = 512 tensor-core plan the main convolution then applies the gate and adds the
    // residual in its last hand-off (one kernel less and one tensor less through memory)
    rc = m2_monarch_conv_fwd(plan, xT, kf_res_dev, Cr, B, d, n, M2_CIRCULAR, stream);
    if (rc != M2_OK) return rc;
    bool fused_out = false;
    if (bf && n == 512 && m2u::has_private_spectrum(plan) && !m2u3::covered(plan)) {
        rc = m2u::conv_gate_fwd(plan, QK, kf_dev, w_short[2], Z, B, d, st, Pv, Cr);
        if (rc == M2_OK) fused_out = true;
        else if (rc != M2_ERR_UNSUPPORTED) return rc;
    }
    if (!fused_out) {
        rc = m2_monarch_conv_fwd(plan, QK, kf_dev, C, B, d, n, M2_CIRCULAR, stream);
        if (rc != M2_OK) return rc;
        if (m2g::launch_gate_out(Pv, w_short[2], C, Cr, Z, B, (int)d, (int)n, bf, st) != cudaSuccess) return M2_ERR_CUDA;
        plan->launches += 1;
    }
    rc = dense(W[3], Z, Pq);
    if (rc != M2_OK) return rc;
    if (m2g::launch_transpose_any(Pq, y_dev, B, (int)d, (int)n, bf, st) != cudaSuccess) return M2_ERR_CUDA;
    plan->launches += 3;   // the two transposes and the input gate (the products, convolutions and the output gate count themselves)
    plan->last_kernel = fused_out ? "bert_mixer_fwd_fused_gate" : "bert_mixer_fwd";
    return M2_OK;
}

// heads of 16 channels on the N = 512 tensor-core plan: outer product, long convolution and contraction are one kernel and the
// dh-times larger tensors do not exist
static bool hyena_heads_fused(const m2_plan* plan, int64_t n, int64_t d, int64_t dh) {
    return plan->dtype == M2_BF16 && m2u::has_private_spectrum(plan) && !m2u3::covered(plan) && dh == 16 && d % 16 == 0 && n % 16 == 0 &&
           n <= 256;
}

int64_t m2_hyena_scratch_bytes(const m2_plan* plan, int64_t B, int64_t n, int64_t d, int64_t dh) {
    if (!plan || B < 0 || n < 0 || d < 0 || dh <= 0) return -1;
    const int64_t big = hyena_heads_fused(plan, n, d, dh) ? 0 : 2 * dh;
    return (7 + big) * round256(B * d * n * (plan->dtype == M2_BF16 ? 2 : 4));
}

int32_t m2_hyena_heads_fwd(const m2_plan* plan, const void* u_dev, const void* const* W, const void* kf1_dev, const void* kf2_dev,
                           const void* kf3_dev, const void* kf_long_dev, void* y_dev, int64_t B, int64_t n, int64_t d, int64_t dh,
                           void* scratch_dev, int64_t scratch_bytes, void* stream) {
    if (!plan || !W || B < 0 || n <= 0 || d <= 0 || dh <= 0 || d % dh != 0) return M2_ERR_INVALID_ARG;
    if (plan->device < 0) return M2_ERR_NO_DEVICE;
    if (2 * n > plan->N) return M2_ERR_INVALID_ARG;   // causal: N >= 2 n
    if (B > 65535 || B * d * dh * n > 0x7fffffffffLL || d > 65535) return M2_ERR_UNSUPPORTED;
    if (B == 0) return M2_OK;
    for (int i = 0; i < 4; ++i)
        if (!W[i] || !aligned16(W[i])) return W[i] ? M2_ERR_ALIGNMENT : M2_ERR_INVALID_ARG;
    if (!u_dev || !kf1_dev || !kf2_dev || !kf3_dev || !kf_long_dev || !y_dev || !scratch_dev) return M2_ERR_INVALID_ARG;
    if (!aligned16(u_dev) || !aligned16(y_dev) || !aligned16(scratch_dev)) return M2_ERR_ALIGNMENT;
    if (scratch_bytes < m2_hyena_scratch_bytes(plan, B, n, d, dh)) return M2_ERR_INVALID_ARG;
    DeviceGuard g(plan->device);
    if (!g.ok) return M2_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    const bool bf = plan->dtype == M2_BF16;
    const int64_t tb = round256(B * d * n * (bf ? 2 : 4));
    unsigned char* sc = static_cast<unsigned char*>(scratch_dev);
    void *uT = sc, *P1 = sc + tb, *P2 = sc + 2 * tb, *P3 = sc + 3 * tb, *C1 = sc + 4 * tb, *C2 = sc + 5 * tb, *C3 = sc + 6 * tb;
    void *XV = sc + 7 * tb, *XVc = sc + (7 + dh) * tb;
    auto dense = [&](const void* Wm, const void* V, void* O) -> int32_t {   // O[b] = Wm V[b] on [B][d][n]
        int32_t rc = m2c::dense(plan, Wm, V, O, B, d, n, st);
        if (rc != M2_ERR_UNSUPPORTED) return rc;
        const cudaError_t e = m2g::launch_dense_cols(Wm, V, O, B, (int)d, (int)n, bf, st);
        if (e == cudaErrorInvalidValue) return M2_ERR_UNSUPPORTED;
        if (e != cudaSuccess) return M2_ERR_CUDA;
        plan->launches += 1;
        return M2_OK;
    };
    // channel-first from here on: every projection, convolution and head product works on rows of n positions
    if (m2g::launch_transpose_any(u_dev, uT, B, (int)n, (int)d, bf, st) != cudaSuccess) return M2_ERR_CUDA;
    int32_t rc = dense(W[0], uT, P1);
    if (rc == M2_OK) rc = dense(W[1], uT, P2);
    if (rc == M2_OK) rc = dense(W[2], uT, P3);
    if (rc == M2_OK) rc = m2_monarch_conv_fwd(plan, P1, kf1_dev, C1, B, d, n, M2_CAUSAL, stream);
    if (rc == M2_OK) rc = m2_monarch_conv_fwd(plan, P2, kf2_dev, C2, B, d, n, M2_CAUSAL, stream);
    if (rc == M2_OK) rc = m2_monarch_conv_fwd(plan, P3, kf3_dev, C3, B, d, n, M2_CAUSAL, stream);
    if (rc != M2_OK) return rc;
    if (hyena_heads_fused(plan, n, d, dh)) {
        rc = m2u::conv_heads_fwd(plan, C1, C2, C3, kf_long_dev, P1, B, d, dh, n, st);
        if (rc != M2_OK) return rc;
    } else {
        if (m2g::launch_heads_outer(C2, C3, XV, B, (int)d, (int)dh, (int)n, bf, st) != cudaSuccess) return M2_ERR_CUDA;
        rc = conv_fwd_grouped(plan, XV, kf_long_dev, XVc, B, d * dh, n, M2_CAUSAL, dh * dh, stream);   // dh^2 channels share a head's kernel
        if (rc != M2_OK) return rc;
        if (m2g::launch_heads_reduce(C1, XVc, P1, B, (int)d, (int)dh, (int)n, bf, st) != cudaSuccess) return M2_ERR_CUDA;
        plan->launches += 2;
    }
    rc = dense(W[3], P1, P2);
    if (rc != M2_OK) return rc;
    if (m2g::launch_transpose_any(P2, y_dev, B, (int)d, (int)n, bf, st) != cudaSuccess) return M2_ERR_CUDA;
    plan->launches += 2;   // the two transposes (the products, convolutions and head kernels count themselves)
    plan->last_kernel = hyena_heads_fused(plan, n, d, dh) ? "hyena_heads_fwd_fused" : "hyena_heads_fwd";
    return M2_OK;
}

int32_t m2_blocks_transpose(const m2_plan* plan, const void* W_in_dev, void* W_out_dev, int64_t nblocks, int64_t rows, int64_t cols,
                            void* stream) {
    if (!plan || nblocks < 0 || rows <= 0 || cols <= 0 || rows > 65536 || cols > 65536) return M2_ERR_INVALID_ARG;
    if ((!W_in_dev || !W_out_dev) && nblocks > 0) return M2_ERR_INVALID_ARG;
    if (plan->device < 0) return M2_ERR_NO_DEVICE;
    if (!aligned16(W_in_dev) || !aligned16(W_out_dev)) return M2_ERR_ALIGNMENT;
    DeviceGuard g(plan->device);
    if (!g.ok) return M2_ERR_CUDA;
    if (m2g::launch_blocks_transpose(W_in_dev, W_out_dev, nblocks, (int)rows, (int)cols, plan->dtype == M2_BF16, (cudaStream_t)stream) !=
        cudaSuccess)
        return M2_ERR_CUDA;
    plan->launches += (nblocks > 0);
    return M2_OK;
}

int64_t m2_matmul_bwd_workspace_bytes(const m2_plan* plan, int64_t T) {
    if (!plan || plan->p != 2 || T < 0) return -1;
    const int64_t generic = T * plan->N * 4, umma = m2mm::wgrad_workspace_bytes(plan, T);
    return generic > umma ? generic : umma;
}

int32_t m2_monarch_matmul_bwd_weights(const m2_plan* plan, const void* X_dev, const void* G_dev, const void* L_dev, const void* R_dev,
                                      float* dL_dev, float* dR_dev, int64_t T, void* ws_dev, int64_t ws_bytes, void* stream) {
    int32_t st = check_matmul_args(plan, X_dev, L_dev, R_dev, dL_dev, T);
    if (st != M2_OK) return st;
    if (!dL_dev || !dR_dev || (T > 0 && !G_dev)) return M2_ERR_INVALID_ARG;   // the gradients are written (zeros) even for T == 0
    if (!aligned16(G_dev) || !aligned16(dR_dev) || !aligned16(ws_dev)) return M2_ERR_ALIGNMENT;
    if (T > 0 && (!ws_dev || ws_bytes < m2_matmul_bwd_workspace_bytes(plan, T))) return M2_ERR_INVALID_ARG;
    DeviceGuard g(plan->device);
    if (!g.ok) return M2_ERR_CUDA;
    if (m2mm::covered(plan)) return m2mm::wgrad(plan, X_dev, G_dev, L_dev, R_dev, dL_dev, dR_dev, T, ws_dev, (cudaStream_t)stream);
    cudaError_t e = m2g::launch_matmul_wgrad(plan->dims[0], plan->dims[1], T, plan->dtype == M2_BF16, X_dev, G_dev, L_dev, R_dev, dL_dev,
                                             dR_dev, (float*)ws_dev, (cudaStream_t)stream);
    if (e == cudaErrorInvalidValue) return M2_ERR_UNSUPPORTED;
    if (e != cudaSuccess) return M2_ERR_CUDA;
    plan->last_kernel = "matmul_wgrad_generic";
    plan->launches += T > 0 ? 4 : 2;
    return M2_OK;
}

int32_t m2_monarch_matmul_host(const m2_plan* plan, const void* X_host, const void* L_dev, const void* R_dev,
                               void* Y_host, void* X_dev_scratch, void* Y_dev_scratch, int64_t T, void* ws_dev,
                               int64_t ws_bytes, void* stream) {
    if (!X_host || !Y_host) return M2_ERR_INVALID_ARG;
    int32_t st = check_matmul_args(plan, X_dev_scratch, L_dev, R_dev, Y_dev_scratch, T);
    if (st != M2_OK) return st;
    DeviceGuard g(plan->device);
    if (!g.ok) return M2_ERR_CUDA;
    const size_t bytes = (size_t)T * plan->N * (plan->dtype == M2_BF16 ? 2 : 4);
    if (bytes == 0) return M2_OK;
    if (cudaMemcpyAsync(X_dev_scratch, X_host, bytes, cudaMemcpyHostToDevice, (cudaStream_t)stream) != cudaSuccess)
        return M2_ERR_CUDA;
    st = m2_monarch_matmul(plan, X_dev_scratch, L_dev, R_dev, Y_dev_scratch, T, ws_dev, ws_bytes, stream);
    if (st != M2_OK) return st;
    if (cudaMemcpyAsync(Y_host, Y_dev_scratch, bytes, cudaMemcpyDeviceToHost, (cudaStream_t)stream) != cudaSuccess)
        return M2_ERR_CUDA;
    return M2_OK;
}

namespace {

// Sequence mix + gate of the M2 block, z[B][T][C] = gate3(x) (.) circular_conv(x, k) along T.  Plans the tensor-core
// order-2 kernel covers take the channel-first route: x -> xT[B][C][T] (in z), long convolution on the tensor cores
// (into y, which the MLP overwrites afterwards), then the gate kernel transposes back into z.  Other plans run the
// strided CUDA-core kernel.  Returns the number of launches to add to the plan's count or a negative status.
// true when the block forward keeps z channel-first, [B][C][T]: the tensor-core sequence mixer (N = 512) feeding the tensor-core
// MLP.  One transposition (x to channel-first) is then all that stands between the caller's layout and the kernels'.
bool block_z_channel_first(const m2_plan* plan, int64_t T, int64_t C, int32_t nblk, int32_t expand) {
    return plan->dtype == M2_BF16 && m2u::has_private_spectrum(plan) && !m2u3::covered(plan) && T == 512 && C % 64 == 0 &&
           m2mlp::covered((int)C, nblk, expand);
}

int32_t block_mix_gate(const m2_plan* plan, const void* x_dev, const void* kf_dev, const float* w_short_dev, void* z, void* y_scratch,
                       int64_t B, int64_t T, int64_t C, cudaStream_t stream, bool* tensor_core, bool channel_first) {
    *tensor_core = false;
    if (channel_first) {   // x -> channel-first in z; convolution and gate in one kernel, in place
        if (m2g::launch_transpose_btc(x_dev, z, B, (int)T, (int)C, stream) != cudaSuccess) return -M2_ERR_CUDA;
        const int32_t st = m2u::conv_gate_fwd(plan, z, kf_dev, w_short_dev, z, B, C, stream);
        if (st != M2_OK) return -st;
        *tensor_core = true;
        return 1;   // (the convolution counts its own launch)
    }
    if (m2u::has_private_spectrum(plan) && !m2u3::covered(plan) && T == 512 && C % 64 == 0) {
        if (m2g::launch_transpose_btc(x_dev, z, B, (int)T, (int)C, stream) != cudaSuccess) return -M2_ERR_CUDA;
        const int32_t st = m2u::conv_fwd(plan, z, kf_dev, y_scratch, B, C, T, M2_CIRCULAR, stream);
        if (st != M2_OK) return -st;
        if (m2g::launch_gate_transpose(x_dev, y_scratch, w_short_dev, z, B, (int)T, (int)C, stream) != cudaSuccess) return -M2_ERR_CUDA;
        *tensor_core = true;
        return 2;   // (the convolution counts its own launch)
    }
    m2g::ConvShape s = conv_shape(plan, B, C, T);
    s.stride_b = T * C;
    s.stride_h = 1;
    s.stride_e = C;
    const cudaError_t e = m2g::launch_conv(s, true, x_dev, kf_dev, z, w_short_dev, stream);
    if (e == cudaErrorInvalidValue) return -M2_ERR_UNSUPPORTED;
    if (e != cudaSuccess) return -M2_ERR_CUDA;
    return 1;
}

}  // namespace

int32_t m2_block_z_channel_first(const m2_plan* plan, int64_t T, int64_t C, int32_t nblk, int32_t expand) {
    if (!plan || C <= 0 || nblk <= 0 || expand <= 0 || C % nblk != 0) return 0;
    return block_z_channel_first(plan, T, C, nblk, expand) ? 1 : 0;
}

int32_t m2_block_fwd(const m2_plan* plan, const void* x_dev, const void* kf_dev, const float* w_short_dev,
                     const void* W_up_dev, const void* W_down_dev, void* z_dev, void* y_dev, int64_t B, int64_t T,
                     int64_t C, int32_t nblk, int32_t expand, void* stream) {
    if (!plan || !x_dev || !kf_dev || !w_short_dev || !W_up_dev || !W_down_dev || !z_dev || !y_dev)
        return M2_ERR_INVALID_ARG;
    if (plan->device < 0) return M2_ERR_NO_DEVICE;
    if (B < 0 || C <= 0 || nblk <= 0 || expand <= 0 || C % nblk != 0 || T != plan->N) return M2_ERR_INVALID_ARG;
    if (plan->dtype != M2_BF16 || plan->p < 2 || plan->p > 3) return M2_ERR_UNSUPPORTED;
    if (B > 0x7fffffffLL / T || B * T > 0x7fffffffffLL / C) return M2_ERR_UNSUPPORTED;   // token and element counts stay far from wrapping
    if (!aligned16(x_dev) || !aligned16(kf_dev) || !aligned16(W_up_dev) || !aligned16(W_down_dev) || !aligned16(z_dev) ||
        !aligned16(y_dev))
        return M2_ERR_ALIGNMENT;
    DeviceGuard g(plan->device);
    if (!g.ok) return M2_ERR_CUDA;
    if (B == 0) return M2_OK;
    bool tc_mix = false;
    const bool zcf = block_z_channel_first(plan, T, C, nblk, expand);
    const int32_t nl = block_mix_gate(plan, x_dev, kf_dev, w_short_dev, z_dev, y_dev, B, T, C, (cudaStream_t)stream, &tc_mix, zcf);
    if (nl < 0) return -nl;
    cudaError_t e = cudaSuccess;
    if (m2mlp::covered((int)C, nblk, expand)) {   // tensor-core MLP for 192 -> 768 -> 192 blocks
        const int32_t st = m2mlp::launch(z_dev, W_up_dev, W_down_dev, y_dev, (int)C, nblk, B * T, plan->d_status, (cudaStream_t)stream, zcf ? T : 0);
        if (st != M2_OK) return st;
        plan->last_kernel = tc_mix ? "block_conv_umma_mlp_umma" : "block_conv_generic_mlp_umma";
    } else {
        e = m2g::launch_mlp(z_dev, W_up_dev, W_down_dev, y_dev, (int)C, nblk, expand, B * T, (cudaStream_t)stream);
        if (e == cudaErrorInvalidValue) return M2_ERR_UNSUPPORTED;
        if (e != cudaSuccess) return M2_ERR_CUDA;
        plan->last_kernel = tc_mix ? "block_conv_umma_mlp_generic" : "block_generic";
    }
    plan->launches += nl + 1;
    return M2_OK;
}

int32_t m2_block_fwd_static(const m2_plan* plan, const void* x_dev, const void* kf_dev, const float* w_short_dev,
                            const void* W_up_dev, const void* W_down_dev, void* y_dev, int64_t B, int64_t T, int64_t C,
                            int32_t nblk, int32_t expand, void* stream) {
    if (!plan || !x_dev || !kf_dev || !w_short_dev || !W_up_dev || !W_down_dev || !y_dev) return M2_ERR_INVALID_ARG;
    if (plan->device < 0) return M2_ERR_NO_DEVICE;
    if (B < 0 || C <= 0 || nblk <= 0 || expand <= 0 || C % nblk != 0 || T != plan->N) return M2_ERR_INVALID_ARG;
    if (plan->dtype != M2_BF16 || plan->p < 2 || plan->p > 3) return M2_ERR_UNSUPPORTED;
    if (B > (int64_t)M2_STATIC_SCRATCH_BYTES / 2 / T / C) return M2_ERR_UNSUPPORTED;   // z would not fit the fixed array (no product that could wrap)
    if (!aligned16(x_dev) || !aligned16(kf_dev) || !aligned16(W_up_dev) || !aligned16(W_down_dev) || !aligned16(y_dev))
        return M2_ERR_ALIGNMENT;
    if (plan->device >= kMaxDevices) return M2_ERR_UNSUPPORTED;
    DeviceGuard g(plan->device);
    if (!g.ok) return M2_ERR_CUDA;
    // Device address of the array, looked up once per device with that device current (no allocation).
    void* z = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_static_mutex);
        if (!g_static_ptr[plan->device]) {
            void* p = nullptr;
            if (cudaGetSymbolAddress(&p, g_block_static_scratch) != cudaSuccess || !p) {
                cudaGetLastError();
                return M2_ERR_CUDA;
            }
            g_static_ptr[plan->device] = p;
        }
        z = g_static_ptr[plan->device];
    }
    if (B == 0) return M2_OK;
    // Same launches as m2_block_fwd; every element of z[B, T, C] is written before it is read, so the array's
    // previous contents never matter.
    bool tc_mix = false;
    const bool zcf = block_z_channel_first(plan, T, C, nblk, expand);
    const int32_t nl = block_mix_gate(plan, x_dev, kf_dev, w_short_dev, z, y_dev, B, T, C, (cudaStream_t)stream, &tc_mix, zcf);
    if (nl < 0) return -nl;
    cudaError_t e = cudaSuccess;
    if (m2mlp::covered((int)C, nblk, expand)) {
        const int32_t st = m2mlp::launch(z, W_up_dev, W_down_dev, y_dev, (int)C, nblk, B * T, plan->d_status, (cudaStream_t)stream, zcf ? T : 0);
        if (st != M2_OK) return st;
        plan->last_kernel = tc_mix ? "block_conv_umma_mlp_umma_static" : "block_conv_generic_mlp_umma_static";
    } else {
        e = m2g::launch_mlp(z, W_up_dev, W_down_dev, y_dev, (int)C, nblk, expand, B * T, (cudaStream_t)stream);
        if (e == cudaErrorInvalidValue) return M2_ERR_UNSUPPORTED;
        if (e != cudaSuccess) return M2_ERR_CUDA;
        plan->last_kernel = tc_mix ? "block_conv_umma_mlp_generic_static" : "block_generic_static";
    }
    plan->launches += nl + 1;
    return M2_OK;
}

int64_t m2_blocky_factors_bytes(const m2_plan* plan) { return plan ? m2b::factors_bytes(plan) : -1; }

int32_t m2_blocky_monarch(const m2_plan* plan, const float* Lt_dev, const float* Rt_dev, int32_t causal_mask, void* factors_dev,
                          void* stream) {
    if (!plan || !Lt_dev || !Rt_dev || !factors_dev) return M2_ERR_INVALID_ARG;
    if (plan->device < 0) return M2_ERR_NO_DEVICE;
    if (!m2b::covered(plan)) return M2_ERR_UNSUPPORTED;
    if (!aligned16(factors_dev)) return M2_ERR_ALIGNMENT;
    DeviceGuard g(plan->device);
    if (!g.ok) return M2_ERR_CUDA;
    return m2b::build(plan, Lt_dev, Rt_dev, causal_mask != 0, factors_dev, (cudaStream_t)stream);
}

int32_t m2_blocky_kernel_spectrum(const m2_plan* plan, const void* factors_dev, const float* k_dev, int64_t H, int64_t n,
                                  void* kf_dev, void* stream) {
    if (!plan || !factors_dev || H < 0 || n <= 0) return M2_ERR_INVALID_ARG;
    if ((!k_dev || !kf_dev) && H > 0) return M2_ERR_INVALID_ARG;
    if (plan->device < 0) return M2_ERR_NO_DEVICE;
    if (!m2b::covered(plan)) return M2_ERR_UNSUPPORTED;
    if (n > plan->N) return M2_ERR_INVALID_ARG;
    if (!aligned16(factors_dev) || !aligned16(kf_dev)) return M2_ERR_ALIGNMENT;
    if (H > 0x7fffffffLL) return M2_ERR_UNSUPPORTED;
    DeviceGuard g(plan->device);
    if (!g.ok) return M2_ERR_CUDA;
    return m2b::spectrum(plan, factors_dev, k_dev, H, n, kf_dev, (cudaStream_t)stream);
}

int32_t m2_blocky_monarch_conv_fwd(const m2_plan* plan, const void* factors_dev, const void* x_dev, const void* kf_dev,
                                   void* y_dev, int64_t B, int64_t H, int64_t n, void* stream) {
    if (!plan || !factors_dev || B < 0 || H < 0 || n <= 0) return M2_ERR_INVALID_ARG;
    if ((!x_dev || !kf_dev || !y_dev) && B * H != 0) return M2_ERR_INVALID_ARG;
    if (plan->device < 0) return M2_ERR_NO_DEVICE;
    if (!m2b::covered(plan)) return M2_ERR_UNSUPPORTED;
    if (2 * n > plan->N) return M2_ERR_INVALID_ARG;   // the theorem's padding: N >= 2 n
    if (!aligned16(factors_dev) || !aligned16(x_dev) || !aligned16(kf_dev) || !aligned16(y_dev)) return M2_ERR_ALIGNMENT;
    if (B * H > 0x7fffffffLL) return M2_ERR_UNSUPPORTED;
    DeviceGuard g(plan->device);
    if (!g.ok) return M2_ERR_CUDA;
    return m2b::conv_fwd(plan, factors_dev, x_dev, kf_dev, y_dev, B, H, n, (cudaStream_t)stream);
}

const char* m2_status_string(int32_t status) {
    switch (status) {
        case M2_OK: return "ok";
        case M2_ERR_INVALID_ARG: return "invalid argument";
        case M2_ERR_UNSUPPORTED: return "unsupported shape or type";
        case M2_ERR_ALIGNMENT: return "device pointer not 16-byte aligned";
        case M2_ERR_CUDA: return "CUDA call failed";
        case M2_ERR_TIMEOUT: return "device-side wait timed out";
        case M2_ERR_NO_DEVICE: return "plan has no device";
        case M2_ERR_SINGULAR: return "a block of a learnable Monarch factor is singular";
        default: return "unknown status";
    }
}

int32_t m2_last_device_status(const m2_plan* plan, int32_t* out) {
    if (!plan || !out) return M2_ERR_INVALID_ARG;
    if (plan->device < 0) return M2_ERR_NO_DEVICE;
    DeviceGuard g(plan->device);
    if (!g.ok) return M2_ERR_CUDA;
    if (cudaDeviceSynchronize() != cudaSuccess) return M2_ERR_CUDA;
    if (cudaMemcpy(out, plan->d_status, sizeof(int32_t), cudaMemcpyDeviceToHost) != cudaSuccess) return M2_ERR_CUDA;
    if (cudaMemset(plan->d_status, 0, sizeof(int32_t)) != cudaSuccess) return M2_ERR_CUDA;
    return M2_OK;
}

const char* m2_last_kernel_name(const m2_plan* plan) { return plan ? plan->last_kernel : "none"; }

int64_t m2_launch_count(const m2_plan* plan) { return plan ? plan->launches : -1; }

}  // extern "C"
