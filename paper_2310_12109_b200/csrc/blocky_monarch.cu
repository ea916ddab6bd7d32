// Learnable (causal) Monarch matrices from polynomial coefficients, block size b = sqrt(N) (App. D.5):
//
//   Alg. BlockyMonarch      coefficient matrices Lt, Rt [N][b]  ->  block-diagonal factors L, R of M = P L P R P
//                           L[k1][k2][n2] = l_{n2}(w_N^{k2 b + k1}),   l_j(Z)     = sum_a Lt[a][j] Z^a
//                           R[n2][k1][n1] = r~_{n2,n1}(w_b^{k1}),      r~_{c,j}(Y) = sum_a Rt[c b + a][j] Y^a
//   Lemma on masking        zero patterns on Lt, Rt that make the basis degrees causal (optional, applied while reading)
//   Alg. BlockMonarchConv   f = M^-1 ((M k') (.) (M u'))[0:n), k' and u' zero padded to N
//
// The factors are complex fp32, [block][out][in] interleaved (re, im).  They and their block inverses are built once per
// weight update: evaluation of the polynomials in fp64 (the exponent of the root is reduced exactly before sincospi),
// Gauss-Jordan with partial pivoting in fp64 for the inverses, results rounded to fp32.  The convolution keeps one row in
// shared memory as complex fp32 and runs the four block-diagonal stages (R, L, L^-1, R^-1) as length-b dot products; the
// stride permutations are index arithmetic.  M^-1 = P R^-1 P L^-1 P for square N.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "blocky_monarch.h"

namespace m2b {

constexpr double kPi = 3.14159265358979323846;

// ---- Alg. BlockyMonarch -------------------------------------------------------------------------------------------------

// one thread per entry of L: L[k1][k2][n2] = sum_a Lt'[a][n2] w_N^{(k2 b + k1) a}; amax = b when the mask keeps only the top block
__global__ void blocky_L_kernel(const float* __restrict__ Lt, float2* __restrict__ L, int b, int amax, int masked, double sgn) {
    const int N = b * b;
    const long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    if (e >= (long long)N * b) return;
    const int n2 = (int)(e % b), k2 = (int)((e / b) % b), k1 = (int)(e / N);
    const long long pt = (long long)k2 * b + k1;   // the evaluation point w_N^pt
    double re = 0.0, im = 0.0;
    for (int a = 0; a < amax; ++a) {
        if (masked && a < n2) continue;            // l_j keeps the coefficients a >= j of the top block only
        const double c = (double)Lt[(size_t)a * b + n2];
        double s_, c_;
        sincospi(2.0 * (double)((pt * a) % N) / (double)N, &s_, &c_);
        re += c * c_;
        im += c * s_;
    }
    L[e] = make_float2((float)re, (float)(sgn * im));
}

// one thread per entry of R: R[n2][k1][n1] = sum_a Rt'[n2 b + a][n1] w_b^{k1 a}
__global__ void blocky_R_kernel(const float* __restrict__ Rt, float2* __restrict__ R, int b, int masked, double sgn) {
    const int N = b * b, h = b / 2;
    const long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    if (e >= (long long)N * b) return;
    const int n1 = (int)(e % b), k1 = (int)((e / b) % b), n2 = (int)(e / N);
    double re = 0.0, im = 0.0;
    for (int a = 0; a < b; ++a) {
        if (masked && (a < n1 || (a >= h && n1 < h))) continue;   // minimum degree n1; degree < b/2 for the first half of the columns
        const double c = (double)Rt[((size_t)n2 * b + a) * b + n1];
        double s_, c_;
        sincospi(2.0 * (double)((k1 * a) % b) / (double)b, &s_, &c_);
        re += c * c_;
        im += c * s_;
    }
    R[e] = make_float2((float)re, (float)(sgn * im));
}

// Inverse of every b x b complex block: Gauss-Jordan with partial pivoting on the augmented matrix [A | I] in fp64, one thread
// block per matrix, the augmented rows in shared memory.  A pivot smaller than 1e-12 of the largest entry of the block marks
// it singular: M2_ERR_SINGULAR goes to the status word and the block's inverse is written as zeros.
__global__ void block_inverse_kernel(const float2* __restrict__ A, float2* __restrict__ Ainv, int b, int32_t* __restrict__ status) {
    extern __shared__ double2 aug[];   // [b][2 b]
    __shared__ int piv_row;
    __shared__ double piv_mag, scale_all;
    __shared__ int singular;
    const int blk = blockIdx.x, tid = threadIdx.x, nt = blockDim.x, w = 2 * b;
    const float2* src = A + (size_t)blk * b * b;
    if (tid == 0) {
        singular = 0;
        scale_all = 0.0;
    }
    __syncthreads();
    double mx = 0.0;
    for (int i = tid; i < b * b; i += nt) {
        const int r = i / b, c = i % b;
        const float2 v = src[i];
        aug[r * w + c] = make_double2((double)v.x, (double)v.y);
        aug[r * w + b + c] = make_double2(r == c ? 1.0 : 0.0, 0.0);
        mx = fmax(mx, fmax(fabs((double)v.x), fabs((double)v.y)));
    }
    // largest entry (for the singularity threshold): a few atomics on a shared word
    atomicMax(reinterpret_cast<unsigned long long*>(&scale_all), (unsigned long long)__double_as_longlong(mx));   // non-negative doubles order like integers
    __syncthreads();
    for (int p = 0; p < b; ++p) {
        if (tid == 0) {   // pivot search down column p (b <= 64: serial is fine, this runs once per weight update)
            int best = p;
            double bm = -1.0;
            for (int r = p; r < b; ++r) {
                const double2 v = aug[r * w + p];
                const double m = v.x * v.x + v.y * v.y;
                if (m > bm) {
                    bm = m;
                    best = r;
                }
            }
            piv_row = best;
            piv_mag = bm;
            if (!(bm > 1e-24 * scale_all * scale_all)) singular = 1;
        }
        __syncthreads();
        if (singular) break;
        const int pr = piv_row;
        if (pr != p)
            for (int c = tid; c < w; c += nt) {
                const double2 t = aug[p * w + c];
                aug[p * w + c] = aug[pr * w + c];
                aug[pr * w + c] = t;
            }
        __syncthreads();
        const double2 pv = aug[p * w + p];
        const double inv = 1.0 / (pv.x * pv.x + pv.y * pv.y);
        const double2 ip = make_double2(pv.x * inv, -pv.y * inv);   // 1 / pivot
        __syncthreads();
        for (int c = tid; c < w; c += nt) {
            const double2 v = aug[p * w + c];
            aug[p * w + c] = make_double2(v.x * ip.x - v.y * ip.y, v.x * ip.y + v.y * ip.x);
        }
        __syncthreads();
        // eliminate column p from every other row: thread -> (row, column) pairs; the multipliers are read before any write to
        // column p because column p of the other rows is only written (to zero) by the threads that own it, after the barrier below
        for (int i = tid; i < b * w; i += nt) {
            const int r = i / w, c = i % w;
            if (r == p || c == p) continue;
            const double2 f = aug[r * w + p], q = aug[p * w + c];
            double2 v = aug[r * w + c];
            v.x -= f.x * q.x - f.y * q.y;
            v.y -= f.x * q.y + f.y * q.x;
            aug[r * w + c] = v;
        }
        __syncthreads();
        for (int r = tid; r < b; r += nt)
            if (r != p) aug[r * w + p] = make_double2(0.0, 0.0);
        __syncthreads();
    }
    float2* dst = Ainv + (size_t)blk * b * b;
    for (int i = tid; i < b * b; i += nt) {
        const int r = i / b, c = i % b;
        const double2 v = aug[r * w + b + c];
        dst[i] = singular ? make_float2(0.f, 0.f) : make_float2((float)v.x, (float)v.y);
    }
    if (singular && tid == 0) atomicExch(status, (int32_t)M2_ERR_SINGULAR);
}

// ---- Alg. BlockMonarchConv ------------------------------------------------------------------------------------------------

template <typename IO>
__device__ __forceinline__ float load_io(const IO* p) { return (float)*p; }
template <>
__device__ __forceinline__ float load_io<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }
__device__ __forceinline__ void store_io(float* p, float v) { *p = v; }
__device__ __forceinline__ void store_io(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

// out[o] = sum_i W[blk][j][i] * in[..] for one block-diagonal stage on a row held in shared memory.
//   FIRST : blk = low digit of the input (stride-1 index), i = high digit: in[i * b + blk]; written to out[j * b + blk]  (R, R^-1)
//   !FIRST: blk = high digit, i = low digit: in[blk * b + i]; written to out[blk * b + j]                                (L, L^-1)
template <bool FIRST>
__device__ __forceinline__ void stage(const float2* __restrict__ W, const float2* in, float2* out, int b, int tid, int nt) {
    const int N = b * b;
    for (int o = tid; o < N; o += nt) {
        int blk, j;
        if (FIRST) {
            blk = o % b;
            j = o / b;
        } else {
            blk = o / b;
            j = o % b;
        }
        const float2* wrow = W + ((size_t)blk * b + j) * b;
        float re = 0.f, im = 0.f;
        for (int i = 0; i < b; ++i) {
            const float2 w = __ldg(wrow + i);
            const float2 v = FIRST ? in[i * b + blk] : in[blk * b + i];
            re = fmaf(w.x, v.x, fmaf(-w.y, v.y, re));
            im = fmaf(w.x, v.y, fmaf(w.y, v.x, im));
        }
        out[o] = make_float2(re, im);
    }
}

// SPECTRUM: row = k[h][0:n) (fp32), writes kf[h][k1 b + k2] = (M k')[k2 b + k1] (plan order, complex fp32).
// else     : row = x[(b_, h)][0:n), y = Re(M^-1 (kf[h] (.) M x'))[0:n).
template <typename IO, bool SPECTRUM>
__global__ void __launch_bounds__(256)
blocky_conv_kernel(const IO* __restrict__ x, const float2* __restrict__ kf, IO* __restrict__ y, float2* __restrict__ kf_out,
                   const float2* __restrict__ L, const float2* __restrict__ R, const float2* __restrict__ Linv,
                   const float2* __restrict__ Rinv, int b, int H, int n) {
    extern __shared__ float2 rowbuf[];   // two rows of N complex values
    const int N = b * b, tid = threadIdx.x, nt = blockDim.x;
    float2 *v0 = rowbuf, *v1 = rowbuf + N;
    const long long row = blockIdx.x;
    const int h = (int)(row % H);
    const IO* src = x + (size_t)row * n;
    for (int i = tid; i < N; i += nt) v0[i] = make_float2(i < n ? load_io<IO>(src + i) : 0.f, 0.f);
    __syncthreads();
    stage<true>(R, v0, v1, b, tid, nt);    // [n1][n2] -> [k1][n2]
    __syncthreads();
    stage<false>(L, v1, v0, b, tid, nt);   // [k1][n2] -> [k1][k2]   (plan order; the last P is left to the indices)
    __syncthreads();
    if (SPECTRUM) {
        float2* dst = kf_out + (size_t)row * N;
        for (int i = tid; i < N; i += nt) dst[i] = v0[i];
        return;
    }
    const float2* kr = kf + (size_t)h * N;
    for (int i = tid; i < N; i += nt) {
        const float2 a = v0[i], c = kr[i];
        v0[i] = make_float2(a.x * c.x - a.y * c.y, a.x * c.y + a.y * c.x);
    }
    __syncthreads();
    stage<false>(Linv, v0, v1, b, tid, nt);   // [k1][k2] -> [k1][n2]
    __syncthreads();
    stage<true>(Rinv, v1, v0, b, tid, nt);    // [k1][n2] -> [n1][n2]: natural order
    __syncthreads();
    IO* dst = y + (size_t)row * n;
    for (int i = tid; i < n; i += nt) store_io(dst + i, v0[i].x);
}

// ---- host side ---------------------------------------------------------------------------------------------------------

bool covered(const m2_plan* pl) { return pl->p == 2 && pl->dims[0] == pl->dims[1] && pl->dims[0] >= 2 && pl->dims[0] <= 64; }

int64_t factors_bytes(const m2_plan* pl) { return covered(pl) ? 4LL * pl->N * pl->dims[0] * (int64_t)sizeof(float2) : -1; }

int32_t build(const m2_plan* pl, const float* Lt, const float* Rt, int masked, void* factors, cudaStream_t st) {
    if (!covered(pl)) return M2_ERR_UNSUPPORTED;
    const int b = pl->dims[0];
    const long long per = (long long)pl->N * b;
    float2* L = static_cast<float2*>(factors);
    float2 *R = L + per, *Linv = L + 2 * per, *Rinv = L + 3 * per;
    const unsigned grid = (unsigned)((per + 255) / 256);
    const double sgn = pl->sign >= 0 ? 1.0 : -1.0;
    blocky_L_kernel<<<grid, 256, 0, st>>>(Lt, L, b, masked ? b : (int)pl->N, masked, sgn);
    blocky_R_kernel<<<grid, 256, 0, st>>>(Rt, R, b, masked, sgn);
    const size_t smem = (size_t)b * 2 * b * sizeof(double2);
    if (cudaFuncSetAttribute(block_inverse_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return M2_ERR_CUDA;
    block_inverse_kernel<<<(unsigned)b, 256, smem, st>>>(L, Linv, b, pl->d_status);
    block_inverse_kernel<<<(unsigned)b, 256, smem, st>>>(R, Rinv, b, pl->d_status);
    if (cudaGetLastError() != cudaSuccess) return M2_ERR_CUDA;
    pl->last_kernel = "blocky_monarch_build";
    pl->launches += 4;
    return M2_OK;
}

template <typename IO, bool SPECTRUM>
static int32_t launch_rows(const m2_plan* pl, const void* factors, const void* x, const void* kf, void* y, void* kf_out, long long rows,
                           int H, int n, cudaStream_t st) {
    const int b = pl->dims[0];
    const long long per = (long long)pl->N * b;
    const float2* L = static_cast<const float2*>(factors);
    const size_t smem = (size_t)2 * pl->N * sizeof(float2);
    auto kern = blocky_conv_kernel<IO, SPECTRUM>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return M2_ERR_CUDA;
    kern<<<(unsigned)rows, 256, smem, st>>>((const IO*)x, (const float2*)kf, (IO*)y, (float2*)kf_out, L, L + per, L + 2 * per, L + 3 * per, b,
                                             H, n);
    return cudaGetLastError() == cudaSuccess ? M2_OK : M2_ERR_CUDA;
}

int32_t spectrum(const m2_plan* pl, const void* factors, const float* k, int64_t H, int64_t n, void* kf, cudaStream_t st) {
    if (!covered(pl)) return M2_ERR_UNSUPPORTED;
    if (H == 0) return M2_OK;
    const int32_t rc = launch_rows<float, true>(pl, factors, k, nullptr, nullptr, kf, H, (int)H, (int)n, st);
    if (rc == M2_OK) {
        pl->last_kernel = "blocky_monarch_spectrum";
        pl->launches += 1;
    }
    return rc;
}

int32_t conv_fwd(const m2_plan* pl, const void* factors, const void* x, const void* kf, void* y, int64_t B, int64_t H, int64_t n,
                 cudaStream_t st) {
    if (!covered(pl)) return M2_ERR_UNSUPPORTED;
    if (B * H == 0) return M2_OK;
    const int32_t rc = pl->dtype == M2_BF16
                           ? launch_rows<__nv_bfloat16, false>(pl, factors, x, kf, y, nullptr, B * H, (int)H, (int)n, st)
                           : launch_rows<float, false>(pl, factors, x, kf, y, nullptr, B * H, (int)H, (int)n, st);
    if (rc == M2_OK) {
        pl->last_kernel = "blocky_monarch_conv";
        pl->launches += 1;
    }
    return rc;
}

}  // namespace m2b
