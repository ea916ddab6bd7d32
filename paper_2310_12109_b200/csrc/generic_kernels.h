// Launch wrappers of the CUDA-core kernels (internal header).
#pragma once
#include <cuda_runtime.h>

namespace m2g {

struct ConvShape {
    int p;
    int dims[3];
    int sign;
    long long B, H, n;
    // element (b, h, i) of x / y lives at b*stride_b + h*stride_h + i*stride_e
    long long stride_b, stride_h, stride_e;
    const float2* roots[3];  // device: omega_{Na}^j per stage
    int kf_group = 1;        // channel h is multiplied by spectrum row h / kf_group
};

cudaError_t launch_conv(const ConvShape& s, bool bf16_io, const void* x, const void* kf, void* y, const float* gate_w,
                        cudaStream_t st);
cudaError_t launch_spectrum(const ConvShape& s, const float* k, void* kf, cudaStream_t st);
cudaError_t launch_spectrum_to_natural(const ConvShape& s, const void* kf, float* out, cudaStream_t st);
// Kmul != nullptr: Y = sigma(K (.) M X), K [Hk][N] of the I/O type, row t uses K[t % Hk], sigma = ReLU if relu else identity
cudaError_t launch_matmul(int N1, int N2, long long T, bool bf16_io, const void* X, const void* L, const void* R, void* Y,
                          const void* Kmul, long long Hk, int relu, cudaStream_t st);
// order-p product in the direct form: W[a] = [N / dims[a]][dims[a]][dims[a]], block id = row-major (k_1..k_{a-1}, n_{a+1}..n_p)
cudaError_t launch_order_p(const int* dims, int p, long long T, bool bf16_io, const void* X, const void* const* W, void* Y, cudaStream_t st);
cudaError_t launch_mlp(const void* z, const void* Wup, const void* Wdn, void* y, int C, int nblk, int expand,
                       long long tokens, cudaStream_t st);

// M2 block helpers (bf16): x[B][T][C] -> xT[B][C][T];  z[b][t][c] = gate3(x)[b][t][c] * vT[b][c][t]  (T, C multiples of 64)
cudaError_t launch_transpose_btc(const void* x, void* xT, long long B, int T, int C, cudaStream_t st);
cudaError_t launch_gate_transpose(const void* x, const void* vT, const float* w, void* z, long long B, int T, int C, cudaStream_t st);

// dk[H, n] (fp32) = gradient of sum_b <conv(k, x_b), g_b> with respect to k; x, g: [B, H, n] contiguous
constexpr long long kWgradScratchBlocks = 296;   // blocks (two per SM) that walk the channels when rows do not fit in shared memory
// bytes of global scratch launch_conv_wgrad needs (0 when three complex rows of N fit in shared memory)
long long conv_wgrad_scratch_bytes(long long N, long long H);
cudaError_t launch_conv_wgrad(const ConvShape& s, bool bf16_io, const void* x, const void* g, float* dk, void* scratch, long long scratch_bytes,
                              cudaStream_t st);
// out[b][c][r] = in[b][r][c] for nblocks blocks of rows x cols elements (fp32 or bf16)
cudaError_t launch_blocks_transpose(const void* in, void* out, long long nblocks, int rows, int cols, bool bf16, cudaStream_t st);
// dL[N1][N2][N2], dR[N2][N1][N1] (fp32) of sum_t <M x_t, g_t>; ws: T*N floats (4 launches)
cudaError_t launch_matmul_wgrad(int N1, int N2, long long T, bool bf16_io, const void* X, const void* G, const void* L, const void* R,
                                float* dL, float* dR, float* ws, cudaStream_t st);
// out[b][c][r] = in[b][r][c], any sizes, fp32 or bf16
cudaError_t launch_transpose_any(const void* in, void* out, long long B, int R, int C, bool bf16, cudaStream_t st);
// y[row] = LayerNorm(a[row] + b[row]) * gamma + beta over d values (y may alias a or b)
cudaError_t launch_add_layernorm(const void* a, const void* b, const float* gamma, const float* beta, void* y, long long rows, int d,
                                 float eps, bool bf16, cudaStream_t st);
// Y = sigma(K (.) M X) for Bt matrices [N][d] whose columns are the vectors (CUDA cores; ws: Bt*N*d values of the I/O type)
cudaError_t launch_monarch_cols(int N1, int N2, long long Bt, int d, bool bf16_io, const void* X, const void* L, const void* R, const void* Kmul,
                                int relu, void* Y, void* ws, cudaStream_t st);
// heads of the M2 Hyena layer on channel-first tensors [B][channels][n]: outer product per position and its contraction with X1
cudaError_t launch_heads_outer(const void* X2, const void* V, void* XV, long long B, int d, int dh, int n, bool bf16, cudaStream_t st);
cudaError_t launch_heads_reduce(const void* X1, const void* XVc, void* O, long long B, int d, int dh, int n, bool bf16, cudaStream_t st);
// O[bt] = W V[bt]: W [c][c] (outputs x inputs), V, O [Bt][c][cols], CUDA cores
cudaError_t launch_dense_cols(const void* W, const void* V, void* O, long long Bt, int c, int cols, bool bf16, cudaStream_t st);
// gated mixer pieces on channel-first tensors [B][d][n]; DW3 = width-3 depthwise filter, zero padded, weights [d][3] fp32:
// QK = DW3(Pq) * DW3(Pk);  Z = DW3(Pv) * C + Cr  (Z must not be one of its inputs)
cudaError_t launch_gate_in(const void* Pq, const void* Pk, const float* wq, const float* wk, void* QK, long long B, int d, int n, bool bf16,
                           cudaStream_t st);
cudaError_t launch_gate_out(const void* Pv, const float* wv, const void* C, const void* Cr, void* Z, long long B, int d, int n, bool bf16,
                            cudaStream_t st);
// conjugates a spectrum buffer: plan-order part (interleaved re, im) followed by the tensor-core kernels' private part
cudaError_t launch_spectrum_conj(const void* in, void* out, long long plan_order_values, long long private_values, cudaStream_t st);

}  // namespace m2g
