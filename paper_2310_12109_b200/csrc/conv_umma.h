// Tensor-core (tcgen05 / TMEM / TMA) Monarch convolution path (internal header).
#pragma once
#include <cuda_runtime.h>

#include "m2_plan.h"

namespace m2u {

// Builds the device constants of the tensor-core path for plans it covers (no-op otherwise).
cudaError_t create_tables(m2_plan* plan);
void destroy_tables(m2_plan* plan);

// Returns M2_ERR_UNSUPPORTED when no tensor-core kernel covers the request (caller falls back to
// the CUDA-core kernels), M2_OK after enqueueing, another status on failure.
// kf_group: channel h is multiplied by spectrum row h / kf_group (the buffer then holds H / kf_group rows).
int32_t conv_fwd(const m2_plan* plan, const void* x, const void* kf, void* y, int64_t B, int64_t H, int64_t n,
                 int32_t mode, cudaStream_t stream, int kf_group = 1);
// The circular convolution of [B][H][512] rows followed by the M2 block's depthwise gate, in one kernel:
//   y[b][h][t] = conv(x[b][h], k[h])[t] * (w_gate[h][0] x[b][h][t-1] + w_gate[h][1] x[b][h][t] + w_gate[h][2] x[b][h][t+1])
// (zero padded at both ends of a row; w_gate [H][3] fp32).  y may be x: the rows are then replaced in place.
// gate_rows != nullptr: the gate is formed from these rows [B][H][512] instead of x; addend != nullptr: rows [B][H][512] added
// after the gate, y = conv(x, k) * gate + addend (neither may be y).
int32_t conv_gate_fwd(const m2_plan* plan, const void* x, const void* kf, const float* w_gate, void* y, int64_t B, int64_t H,
                      cudaStream_t stream, const void* gate_rows = nullptr, const void* addend = nullptr);
// The core of the M2 Hyena layer with heads of dh = 16 channels, in one kernel (no d_h-times larger tensor in memory):
//   y[b][h dh + j][t] = sum_i X1[b][h dh + i][t] (k_h * (X2[b][h dh + i] V[b][h dh + j]))[t],   causal, t < n <= 256,
// X1, X2, V, y: [B][d][n] bf16; kf_heads: the spectrum of the d / dh head kernels.  M2_ERR_UNSUPPORTED for other shapes.
int32_t conv_heads_fwd(const m2_plan* plan, const void* X1, const void* X2, const void* V, const void* kf_heads, void* y, int64_t B,
                       int64_t d, int64_t dh, int64_t n, cudaStream_t stream);
// The row-pair kernel launched so that every pipeline's first bounded wait runs out with nothing in flight (no copy is
// issued, a few polls per wait): the kernel leaves through its abort path, sets M2_ERR_TIMEOUT in the plan's status
// word, writes nothing to y.  Needs B > 8 (the row-pair kernel); M2_ERR_UNSUPPORTED otherwise.
int32_t conv_fwd_wait_selftest(const m2_plan* plan, const void* x, const void* kf, void* y, int64_t B, int64_t H, int64_t n,
                               int32_t mode, cudaStream_t stream);

// Kernel gradient, tensor-core part: partial[b group][h][512] = sum over the group's 8 rows of conj(M x) (.) M g in plan
// order (complex fp32, conv_wgrad_workspace_bytes(plan, B, H) bytes); *parts = number of b groups.
int64_t conv_wgrad_workspace_bytes(const m2_plan* plan, int64_t B, int64_t H);
int32_t conv_wgrad_partials(const m2_plan* plan, const void* x, const void* g, void* partial, int64_t B, int64_t H, int64_t n,
                            int32_t mode, int* parts, cudaStream_t stream);
// ... and dk[H][n] (fp32) = Re M^-1(sum of the parts)[0:n) / N from them (CUDA cores, fp32)
int32_t conv_wgrad_finish(const m2_plan* plan, const void* partial, int parts, float* dk, int64_t H, int64_t n, cudaStream_t stream);

}  // namespace m2u

// Order-3 kernel for N = 32768 = 32^3, causal n = 16384 (conv_umma3.cu); same contract as m2u.
namespace m2u3 {
bool covered(const m2_plan* plan);
cudaError_t create_tables(m2_plan* plan);
void destroy_tables(m2_plan* plan);
cudaError_t relayout_spectrum(const m2_plan* plan, void* kf, int64_t H, cudaStream_t stream);
int32_t conv_fwd(const m2_plan* plan, const void* x, const void* kf, void* y, int64_t B, int64_t H, int64_t n,
                 int32_t mode, cudaStream_t stream);
// kernel gradient dk[H][16384] (fp32) through the same kernel: the row pairs' conjugated spectra, then the convolution of the
// g pairs with them, then the sum over a channel's pairs; ws: conv_wgrad_workspace_bytes(plan, B, H) bytes
int64_t conv_wgrad_workspace_bytes(const m2_plan* plan, int64_t B, int64_t H);
int32_t conv_wgrad(const m2_plan* plan, const void* x, const void* g, float* dk, int64_t B, int64_t H, int64_t n, int32_t mode, void* ws,
                   cudaStream_t stream);
}  // namespace m2u3

namespace m2u {

// Plans the tensor-core path covers keep a second copy of the spectrum in the layout its kernel
// reads (appended to the plan-order copy); relayout_spectrum fills it.
bool has_private_spectrum(const m2_plan* plan);
cudaError_t relayout_spectrum(const m2_plan* plan, void* kf, int64_t H, cudaStream_t stream);

}  // namespace m2u
