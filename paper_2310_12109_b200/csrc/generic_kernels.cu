// CUDA-core (fp32 FMA) kernels: the fp32 path, the kernel spectrum, and the general-shape path for
// sizes the tensor-core kernels do not cover.  One thread block owns one (batch, channel) row and
// keeps it in shared memory from the load to the store; every Monarch stage is an in-place
// contraction of one index digit (the stride permutations of M = P L P^T R P only decide which
// digit a stage contracts, so they are address arithmetic here, never a data movement pass).
#include <cuda_bf16.h>

#include <cstdint>
#include <cuda_runtime.h>

#include "generic_kernels.h"

namespace m2g {

struct Dims {
    int p;
    int d[3];
    int N;
    float sgn;  // +1 / -1: omega = exp(sgn 2 pi i / M)
};

__device__ __forceinline__ float2 cmul(float2 a, float2 b) {
    return make_float2(a.x * b.x - a.y * b.y, a.x * b.y + a.y * b.x);
}

// storage traits: complex value kept as float2 or as a bf16 pair
template <typename ST>
struct Store;
template <>
struct Store<float2> {
    static __device__ __forceinline__ float2 ld(const float2* p) { return *p; }
    static __device__ __forceinline__ void st(float2* p, float2 v) { *p = v; }
};
template <>
struct Store<__nv_bfloat162> {
    static __device__ __forceinline__ float2 ld(const __nv_bfloat162* p) { return __bfloat1622float2(*p); }
    static __device__ __forceinline__ void st(__nv_bfloat162* p, float2 v) { *p = __float22bfloat162_rn(v); }
};

template <typename T>
__device__ __forceinline__ float to_f32(T v);
template <>
__device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <>
__device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T>
__device__ __forceinline__ T from_f32(float v);
template <>
__device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <>
__device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// omega_M^e with e already reduced to [0, M)
__device__ __forceinline__ float2 twiddle(int e, int M, float sgn) {
    float s, c;
    sincospif(2.0f * (float)e / (float)M, &s, &c);
    return make_float2(c, sgn * s);
}

// One Monarch-DFT stage, in place on buf (plan-position layout [d0][d1][d2]).
//   forward (INV = false), stage a: contract n_a with F_{Na} (Corollary "DFT is M": block = F times the
//     twiddle diagonal); the twiddle of the NEXT stage is applied to the outputs so every element
//     costs one sincos:  out[k_a] = tw_{a+1}(n_{a+1}, kappa + Mprev k_a) * sum_{n_a} w^{k_a n_a} buf[n_a]
//   inverse (INV = true), stage a: out[n_a] = conj(tw_a(n_a, kappa)) * sum_{k_a} conj(w^{k_a n_a}) buf[k_a]
// The N outputs of a stage are produced in chunks of blockDim * ITEMS; a chunk is always a union of
// whole fibers, so its writes cannot disturb the inputs of another chunk.  Within a chunk every
// thread first computes its outputs into registers, then the block synchronises, then writes.
template <typename ST, int ITEMS, bool INV>
__device__ __forceinline__ void stage(ST* buf, const Dims& D, int a, const float2* __restrict__ roots) {
    const int Na = D.d[a];
    int sa = 1;
    for (int j = a + 1; j < D.p; ++j) sa *= D.d[j];
    int Mprev = 1;
    for (int j = 0; j < a; ++j) Mprev *= D.d[j];
    const int Mcur = Mprev * Na;
    const int G = blockDim.x * ITEMS;          // outputs per chunk (G >= N: a single chunk)
    const int F = G / Na;                      // fibers per chunk when G < N
    const int nchunks = (D.N + G - 1) / G;
    for (int c = 0; c < nchunks; ++c) {
        float2 acc[ITEMS];
        int pos[ITEMS];
#pragma unroll
        for (int it = 0; it < ITEMS; ++it) {
            const int i = threadIdx.x + it * blockDim.x;
            int o;
            if (nchunks == 1 || sa < F) {
                o = c * G + i;
            } else {
                const int per_hi = sa / F;     // chunks per value of hi
                o = (c / per_hi) * Na * sa + (i / F) * sa + (c % per_hi) * F + (i % F);
            }
            pos[it] = o;
            acc[it] = make_float2(0.f, 0.f);
            if (o < D.N) {
                const int lo = o % sa;
                const int oa = (o / sa) % Na;
                const int hi = o / (sa * Na);
                const ST* fib = buf + hi * Na * sa + lo;
                float2 s = make_float2(0.f, 0.f);
                for (int j = 0; j < Na; ++j) {
                    float2 w = roots[(oa * j) % Na];
                    if (INV) w.y = -w.y;
                    const float2 v = Store<ST>::ld(fib + j * sa);
                    s.x = fmaf(w.x, v.x, s.x);
                    s.x = fmaf(-w.y, v.y, s.x);
                    s.y = fmaf(w.x, v.y, s.y);
                    s.y = fmaf(w.y, v.x, s.y);
                }
                if (!INV) {
                    if (a + 1 < D.p) {
                        // hi is empty (a = 0) or the single digit k_1 (a = 1)
                        const int kappa = hi + Mprev * oa;
                        const int Nn = D.d[a + 1];
                        const int nn = lo / (sa / Nn);
                        const int Mn = Mcur * Nn;
                        const int e = (int)(((long long)nn * kappa) % Mn);
                        s = cmul(s, twiddle(e, Mn, D.sgn));
                    }
                } else if (a > 0) {
                    int kappa;
                    if (a == 1) kappa = hi;
                    else kappa = hi / D.d[1] + D.d[0] * (hi % D.d[1]);  // a = 2: hi = k_1 * N_2 + k_2
                    const int e = (int)(((long long)oa * kappa) % Mcur);
                    s = cmul(s, twiddle(e, Mcur, -D.sgn));
                }
                acc[it] = s;
            }
        }
        __syncthreads();
#pragma unroll
        for (int it = 0; it < ITEMS; ++it)
            if (pos[it] < D.N) Store<ST>::st(buf + pos[it], acc[it]);
        __syncthreads();
    }
}

struct Roots {
    const float2* r[3];
};

// Fused Monarch convolution for one row per block (Eq. 2 / Alg. BlockMonarchConv with M = F_N):
// load + zero pad, forward stages, spectrum multiply (plan order on both sides, so no permutation),
// inverse stages, real part, truncate, store.  Strides let the same kernel read a [B, T, C] tensor
// along T (the M2 block) -- then gate_w != nullptr adds the width-3 depthwise gate before the store.
template <typename IO, typename ST, int ITEMS>
__global__ void __launch_bounds__(1024) conv_row_kernel(const IO* __restrict__ x, const float2* __restrict__ kf, IO* __restrict__ y, Dims D,
                                Roots R, int H, int n, long long row_stride_b, long long row_stride_h,
                                long long elem_stride, const float* __restrict__ gate_w, int kf_group) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    ST* buf = reinterpret_cast<ST*>(smem_raw);
    const int row = blockIdx.x;
    const int h = row % H;
    const int b = row / H;
    const IO* xr = x + b * row_stride_b + h * row_stride_h;
    IO* yr = y + b * row_stride_b + h * row_stride_h;
    for (int i = threadIdx.x; i < D.N; i += blockDim.x) {
        float v = (i < n) ? to_f32<IO>(xr[(long long)i * elem_stride]) : 0.f;
        Store<ST>::st(buf + i, make_float2(v, 0.f));
    }
    __syncthreads();
    for (int a = 0; a < D.p; ++a) stage<ST, ITEMS, false>(buf, D, a, R.r[a]);
    const float2* kr = kf + (long long)(h / kf_group) * D.N;
    for (int i = threadIdx.x; i < D.N; i += blockDim.x) Store<ST>::st(buf + i, cmul(Store<ST>::ld(buf + i), kr[i]));
    __syncthreads();
    for (int a = D.p - 1; a >= 0; --a) stage<ST, ITEMS, true>(buf, D, a, R.r[a]);
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        float v = Store<ST>::ld(buf + i).x;
        if (gate_w != nullptr) {
            const float w0 = gate_w[h * 3 + 0], w1 = gate_w[h * 3 + 1], w2 = gate_w[h * 3 + 2];
            float g = w1 * to_f32<IO>(xr[(long long)i * elem_stride]);
            if (i > 0) g = fmaf(w0, to_f32<IO>(xr[(long long)(i - 1) * elem_stride]), g);
            if (i + 1 < n) g = fmaf(w2, to_f32<IO>(xr[(long long)(i + 1) * elem_stride]), g);
            v *= g;
        }
        yr[(long long)i * elem_stride] = from_f32<IO>(v);
    }
}

// Gradient with respect to the kernel: dk[h] = M^-1 ( sum_b conj(M x'_b) (.) M g'_b ) [0:n) / N, one block per channel,
// the batch walked sequentially; x, g rows and the accumulated product stay in shared memory (3 complex fp32 rows) -- or, for
// N too large for that, in a per-block slice of a global scratch buffer (gscratch != nullptr; blocks then walk the channels).
template <typename IO, int ITEMS>
__global__ void __launch_bounds__(1024) conv_wgrad_kernel(const IO* __restrict__ x, const IO* __restrict__ g, float* __restrict__ dk, Dims D,
                                                          Roots R, int B, int H, int n, float2* gscratch) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float2* bx = gscratch ? gscratch + (size_t)blockIdx.x * 3 * D.N : reinterpret_cast<float2*>(smem_raw);
    float2* bg = bx + D.N;
    float2* acc = bg + D.N;
    for (int h = blockIdx.x; h < H; h += gridDim.x) {
    __syncthreads();   // the previous channel's result has been read
    for (int i = threadIdx.x; i < D.N; i += blockDim.x) acc[i] = make_float2(0.f, 0.f);
    for (int b = 0; b < B; ++b) {
        const IO* xr = x + ((long long)b * H + h) * n;
        const IO* gr = g + ((long long)b * H + h) * n;
        for (int i = threadIdx.x; i < D.N; i += blockDim.x) {
            bx[i] = make_float2(i < n ? to_f32<IO>(xr[i]) : 0.f, 0.f);
            bg[i] = make_float2(i < n ? to_f32<IO>(gr[i]) : 0.f, 0.f);
        }
        __syncthreads();
        for (int a = 0; a < D.p; ++a) stage<float2, ITEMS, false>(bx, D, a, R.r[a]);
        for (int a = 0; a < D.p; ++a) stage<float2, ITEMS, false>(bg, D, a, R.r[a]);
        for (int i = threadIdx.x; i < D.N; i += blockDim.x) {   // every thread owns the same positions in every round
            const float2 xv = bx[i], gv = bg[i], av = acc[i];
            acc[i] = make_float2(av.x + xv.x * gv.x + xv.y * gv.y, av.y + xv.x * gv.y - xv.y * gv.x);   // += conj(x_f) g_f
        }
        __syncthreads();
    }
    for (int a = D.p - 1; a >= 0; --a) stage<float2, ITEMS, true>(acc, D, a, R.r[a]);
    const float inv = 1.0f / (float)D.N;
    for (int i = threadIdx.x; i < n; i += blockDim.x) dk[(long long)h * n + i] = acc[i].x * inv;
    }
}

// k_f = F_N pad(k) / N per channel, in plan order, computed in place in the output buffer (global
// memory, one block per channel): runs once per weight update, not on the hot path.
template <int ITEMS>
__global__ void __launch_bounds__(1024) spectrum_kernel(const float* __restrict__ k, float2* __restrict__ kf, Dims D, Roots R, int n) {
    const int h = blockIdx.x;
    float2* buf = kf + (long long)h * D.N;
    for (int i = threadIdx.x; i < D.N; i += blockDim.x)
        buf[i] = make_float2(i < n ? k[(long long)h * n + i] : 0.f, 0.f);
    __syncthreads();
    for (int a = 0; a < D.p; ++a) stage<float2, ITEMS, false>(buf, D, a, R.r[a]);
    const float inv = 1.0f / (float)D.N;
    for (int i = threadIdx.x; i < D.N; i += blockDim.x) {
        float2 v = buf[i];
        buf[i] = make_float2(v.x * inv, v.y * inv);
    }
}

__global__ void spectrum_to_natural_kernel(const float2* __restrict__ kf, float2* __restrict__ out, Dims D, long long total) {
    long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    if (i >= total) return;
    const int pos = (int)(i % D.N);
    const long long h = i / D.N;
    // plan position (k1, k2, k3) row-major -> k = k1 + N1 k2 + N1 N2 k3
    int rem = pos, k = 0;
    int digits[3] = {0, 0, 0};
    for (int a = D.p - 1; a >= 0; --a) {
        digits[a] = rem % D.d[a];
        rem /= D.d[a];
    }
    int w = 1;
    for (int a = 0; a < D.p; ++a) {
        k += w * digits[a];
        w *= D.d[a];
    }
    float2 v = kf[i];
    out[h * D.N + k] = make_float2(v.x * (float)D.N, v.y * (float)D.N);
}

// Order-2 Monarch matmul, TT tokens per block, fp32 accumulate (Sec. 3.1):
//   z[n2][k1] = sum_{n1} R[n2][k1][n1] x[n1*N2 + n2];  y[k2*N1 + k1] = sum_{n2} L[k1][k2][n2] z[n2][k1]
template <typename IO, int TT>
__global__ void matmul_tokens_kernel(const IO* __restrict__ X, const IO* __restrict__ L, const IO* __restrict__ Rw,
                                     IO* __restrict__ Y, int N1, int N2, long long T, const IO* __restrict__ Kmul, long long Hk, int relu) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int N = N1 * N2;
    float* xs = reinterpret_cast<float*>(smem_raw);  // [TT][N]
    float* zs = xs + TT * N;                          // [TT][N], index n2*N1 + k1
    const long long t0 = (long long)blockIdx.x * TT;
    for (int i = threadIdx.x; i < TT * N; i += blockDim.x) {
        const long long t = t0 + i / N;
        xs[i] = (t < T) ? to_f32<IO>(X[t * N + (i % N)]) : 0.f;
    }
    __syncthreads();
    for (int o = threadIdx.x; o < N; o += blockDim.x) {
        const int k1 = o % N1, n2 = o / N1;
        const IO* w = Rw + ((long long)n2 * N1 + k1) * N1;
        float acc[TT];
#pragma unroll
        for (int t = 0; t < TT; ++t) acc[t] = 0.f;
        for (int n1 = 0; n1 < N1; ++n1) {
            const float wv = to_f32<IO>(w[n1]);
#pragma unroll
            for (int t = 0; t < TT; ++t) acc[t] = fmaf(wv, xs[t * N + n1 * N2 + n2], acc[t]);
        }
#pragma unroll
        for (int t = 0; t < TT; ++t) zs[t * N + o] = acc[t];
    }
    __syncthreads();
    for (int o = threadIdx.x; o < N; o += blockDim.x) {
        const int k1 = o % N1, k2 = o / N1;
        const IO* w = L + ((long long)k1 * N2 + k2) * N2;
        float acc[TT];
#pragma unroll
        for (int t = 0; t < TT; ++t) acc[t] = 0.f;
        for (int n2 = 0; n2 < N2; ++n2) {
            const float wv = to_f32<IO>(w[n2]);
#pragma unroll
            for (int t = 0; t < TT; ++t) acc[t] = fmaf(wv, zs[t * N + n2 * N1 + k1], acc[t]);
        }
#pragma unroll
        for (int t = 0; t < TT; ++t)
            if (t0 + t < T) {
                float v = acc[t];
                if (Kmul) {   // y = sigma(K (.) M x): the first half of the M2 operator (Eq. 2)
                    v *= to_f32<IO>(Kmul[((t0 + t) % Hk) * N + o]);
                    if (relu) v = fmaxf(v, 0.f);
                }
                Y[(t0 + t) * N + o] = from_f32<IO>(v);
            }
    }
}

// Block-diagonal MLP with GELU (Eq. 3 with block-diagonal M_3, M_4): per (token tile, block)
//   hid = GELU(W_up[j] z_j),  y_j = W_down[j] hid.   The hidden activations never leave the SM.
template <int TT>
__global__ void mlp_blockdiag_kernel(const __nv_bfloat16* __restrict__ z, const __nv_bfloat16* __restrict__ Wup,
                                     const __nv_bfloat16* __restrict__ Wdn, __nv_bfloat16* __restrict__ y, int C,
                                     int nblk, int expand, long long tokens) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int ci = C / nblk, hi = expand * ci;
    float* zs = reinterpret_cast<float*>(smem_raw);  // [TT][ci]
    float* hs = zs + TT * ci;                         // [TT][hi]
    const int j = blockIdx.y;
    const long long t0 = (long long)blockIdx.x * TT;
    for (int i = threadIdx.x; i < TT * ci; i += blockDim.x) {
        const long long t = t0 + i / ci;
        zs[i] = (t < tokens) ? __bfloat162float(z[t * C + j * ci + (i % ci)]) : 0.f;
    }
    __syncthreads();
    for (int o = threadIdx.x; o < hi; o += blockDim.x) {
        const __nv_bfloat16* w = Wup + ((long long)j * hi + o) * ci;
        float acc[TT];
#pragma unroll
        for (int t = 0; t < TT; ++t) acc[t] = 0.f;
        for (int i = 0; i < ci; ++i) {
            const float wv = __bfloat162float(w[i]);
#pragma unroll
            for (int t = 0; t < TT; ++t) acc[t] = fmaf(wv, zs[t * ci + i], acc[t]);
        }
#pragma unroll
        for (int t = 0; t < TT; ++t) {
            const float v = acc[t];
            hs[t * hi + o] = 0.5f * v * (1.0f + erff(v * 0.70710678118654752f));
        }
    }
    __syncthreads();
    for (int o = threadIdx.x; o < ci; o += blockDim.x) {
        const __nv_bfloat16* w = Wdn + ((long long)j * ci + o) * hi;
        float acc[TT];
#pragma unroll
        for (int t = 0; t < TT; ++t) acc[t] = 0.f;
        for (int i = 0; i < hi; ++i) {
            const float wv = __bfloat162float(w[i]);
#pragma unroll
            for (int t = 0; t < TT; ++t) acc[t] = fmaf(wv, hs[t * hi + i], acc[t]);
        }
#pragma unroll
        for (int t = 0; t < TT; ++t)
            if (t0 + t < tokens) y[(t0 + t) * C + j * ci + o] = __float2bfloat16_rn(acc[t]);
    }
}

static Dims make_dims(const ConvShape& s) {
    Dims D;
    D.p = s.p;
    D.N = 1;
    for (int a = 0; a < 3; ++a) {
        D.d[a] = a < s.p ? s.dims[a] : 1;
        D.N *= D.d[a];
    }
    D.sgn = s.sign >= 0 ? 1.f : -1.f;
    return D;
}

// items per thread and block size.  Small or odd N: one output per thread.  N <= 2048: two.
// Larger N: 1024 threads x 4 outputs per chunk; then every dimension must be a power of two and N a
// multiple of 4096 so that chunks are unions of whole fibers.
static bool pick_launch(const Dims& D, int& items, int& threads) {
    const int N = D.N;
    if (N % 2 != 0 || N < 128) {
        items = 1;
        threads = N;
        return N >= 1 && N <= 1024;
    }
    if (N <= 2048) {
        items = 2;
        threads = N / 2;
        return true;
    }
    items = 4;
    threads = 1024;
    if (N % 4096 != 0) return false;
    for (int a = 0; a < D.p; ++a)
        if ((D.d[a] & (D.d[a] - 1)) != 0 || D.d[a] > 4096) return false;
    return true;
}

template <typename IO, typename ST>
static cudaError_t launch_conv_t(const ConvShape& s, const void* x, const void* kf, void* y, const float* gate_w,
                                 cudaStream_t st) {
    Dims D = make_dims(s);
    Roots R{{s.roots[0], s.roots[1], s.roots[2]}};
    int items, threads;
    if (!pick_launch(D, items, threads)) return cudaErrorInvalidValue;
    const size_t smem = (size_t)D.N * sizeof(ST);
    const long long rows = (long long)s.B * s.H;
    if (rows == 0) return cudaSuccess;
#define M2_LAUNCH_CONV(IT)                                                                                         \
    {                                                                                                              \
        auto kern = conv_row_kernel<IO, ST, IT>;                                                                   \
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);        \
        if (e != cudaSuccess) return e;                                                                            \
        kern<<<(unsigned)rows, threads, smem, st>>>((const IO*)x, (const float2*)kf, (IO*)y, D, R, (int)s.H,       \
                                                    (int)s.n, s.stride_b, s.stride_h, s.stride_e, gate_w,          \
                                                    s.kf_group > 0 ? s.kf_group : 1);                              \
    }
    switch (items) {
        case 1: M2_LAUNCH_CONV(1) break;
        case 2: M2_LAUNCH_CONV(2) break;
        case 4: M2_LAUNCH_CONV(4) break;
        default: return cudaErrorInvalidValue;
    }
#undef M2_LAUNCH_CONV
    return cudaGetLastError();
}

cudaError_t launch_conv(const ConvShape& s, bool bf16_io, const void* x, const void* kf, void* y, const float* gate_w,
                        cudaStream_t st) {
    long long N = 1;
    for (int a = 0; a < s.p; ++a) N *= s.dims[a];
    if (!bf16_io) {
        if (N * 8 > 200 * 1024) return cudaErrorInvalidValue;
        return launch_conv_t<float, float2>(s, x, kf, y, gate_w, st);
    }
    if (N * 8 <= 160 * 1024) return launch_conv_t<__nv_bfloat16, float2>(s, x, kf, y, gate_w, st);
    if (N * 4 > 200 * 1024) return cudaErrorInvalidValue;
    return launch_conv_t<__nv_bfloat16, __nv_bfloat162>(s, x, kf, y, gate_w, st);
}

cudaError_t launch_spectrum(const ConvShape& s, const float* k, void* kf, cudaStream_t st) {
    Dims D = make_dims(s);
    Roots R{{s.roots[0], s.roots[1], s.roots[2]}};
    int items, threads;
    if (!pick_launch(D, items, threads)) return cudaErrorInvalidValue;
    if (s.H == 0) return cudaSuccess;
    switch (items) {
        case 1: spectrum_kernel<1><<<(unsigned)s.H, threads, 0, st>>>(k, (float2*)kf, D, R, (int)s.n); break;
        case 2: spectrum_kernel<2><<<(unsigned)s.H, threads, 0, st>>>(k, (float2*)kf, D, R, (int)s.n); break;
        case 4: spectrum_kernel<4><<<(unsigned)s.H, threads, 0, st>>>(k, (float2*)kf, D, R, (int)s.n); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

cudaError_t launch_spectrum_to_natural(const ConvShape& s, const void* kf, float* out, cudaStream_t st) {
    Dims D = make_dims(s);
    const long long total = (long long)s.H * D.N;
    if (total == 0) return cudaSuccess;
    spectrum_to_natural_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>((const float2*)kf, (float2*)out, D, total);
    return cudaGetLastError();
}

template <typename IO>
static cudaError_t launch_matmul_t(int N1, int N2, long long T, const void* X, const void* L, const void* R, void* Y,
                                   const void* Kmul, long long Hk, int relu, cudaStream_t st) {
    constexpr int TT = 4;
    const int N = N1 * N2;
    const size_t smem = (size_t)2 * TT * N * sizeof(float);
    if (smem > 200 * 1024) return cudaErrorInvalidValue;
    if (T == 0) return cudaSuccess;
    auto kern = matmul_tokens_kernel<IO, TT>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    int threads = N < 512 ? ((N + 31) / 32) * 32 : 512;
    kern<<<(unsigned)((T + TT - 1) / TT), threads, smem, st>>>((const IO*)X, (const IO*)L, (const IO*)R, (IO*)Y, N1, N2, T,
                                                                   (const IO*)Kmul, Hk, relu);
    return cudaGetLastError();
}

cudaError_t launch_matmul(int N1, int N2, long long T, bool bf16_io, const void* X, const void* L, const void* R, void* Y,
                          const void* Kmul, long long Hk, int relu, cudaStream_t st) {
    return bf16_io ? launch_matmul_t<__nv_bfloat16>(N1, N2, T, X, L, R, Y, Kmul, Hk, relu, st)
                   : launch_matmul_t<float>(N1, N2, T, X, L, R, Y, Kmul, Hk, relu, st);
}

// Order-p Monarch product in the direct form (Eq. 1; App. D.6, "p-variate Monarch"), TT tokens per block, fp32 accumulate:
// stage a = 1..p contracts the input digit n_a into the output digit k_a with the block chosen by
// (k_1..k_{a-1}, n_{a+1}..n_p) -- its id is the row-major flattening of that tuple, W[a-1] is [N / N_a][N_a out][N_a in].
// The row stays in shared memory as an array with axes (k_1..k_{a-1}, n_a..n_p), first axis most significant; a stage
// works in place: the elements of one block differ only in axis a (stride s_a = N_{a+1} .. N_p), a warp owns a block,
// reads its N_a inputs (broadcast reads) into up to 8 outputs per lane and writes them back after the warp has
// finished reading.  The result leaves in natural order k = k_1 + N_1 k_2 + ...
struct OrderPArgs {
    const void* W[4];
    int dims[4];
    int p;
};

template <typename IO, int TT>
__global__ void __launch_bounds__(512) monarch_order_p_kernel(const IO* __restrict__ X, IO* __restrict__ Y, OrderPArgs A, int N, long long T) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float* v = reinterpret_cast<float*>(smem_raw);   // [TT][N]
    const long long t0 = (long long)blockIdx.x * TT;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    for (int i = threadIdx.x; i < TT * N; i += blockDim.x) {
        const long long t = t0 + i / N;
        v[i] = (t < T) ? to_f32<IO>(X[t * N + (i % N)]) : 0.f;
    }
    __syncthreads();
    int sa = N;
    for (int a = 0; a < A.p; ++a) {
        const int Na = A.dims[a];
        sa /= Na;                                    // stride of axis a
        const IO* Wa = reinterpret_cast<const IO*>(A.W[a]);
        const int nblocks = N / Na;
        for (int b = warp; b < nblocks; b += nwarps) {
            const int base = (b / sa) * (Na * sa) + (b % sa);
            const IO* wb = Wa + (long long)b * Na * Na;
            float acc[8][TT];
#pragma unroll
            for (int j = 0; j < 8; ++j)
#pragma unroll
                for (int t = 0; t < TT; ++t) acc[j][t] = 0.f;
            for (int i = 0; i < Na; ++i) {
                float xv[TT];
#pragma unroll
                for (int t = 0; t < TT; ++t) xv[t] = v[t * N + base + i * sa];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const int o = lane + 32 * j;
                    if (o < Na) {
                        const float wv = to_f32<IO>(wb[(long long)o * Na + i]);
#pragma unroll
                        for (int t = 0; t < TT; ++t) acc[j][t] = fmaf(wv, xv[t], acc[j][t]);
                    }
                }
            }
            __syncwarp();   // every lane has read the block's inputs
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int o = lane + 32 * j;
                if (o < Na)
#pragma unroll
                    for (int t = 0; t < TT; ++t) v[t * N + base + o * sa] = acc[j][t];
            }
        }
        __syncthreads();
    }
    // axes (k_1..k_p), first most significant  ->  natural order, k_1 least significant
    for (int i = threadIdx.x; i < N; i += blockDim.x) {
        int rest = i, nat = 0, w = N;
        for (int a = 0, mul = 1; a < A.p; ++a) {
            w /= A.dims[a];
            const int k = rest / w;
            rest -= k * w;
            nat += k * mul;
            mul *= A.dims[a];
        }
#pragma unroll
        for (int t = 0; t < TT; ++t)
            if (t0 + t < T) Y[(t0 + t) * N + nat] = from_f32<IO>(v[t * N + i]);
    }
}

template <typename IO>
static cudaError_t launch_order_p_t(const OrderPArgs& A, int N, long long T, const void* X, void* Y, cudaStream_t st) {
    if (T == 0) return cudaSuccess;
    const bool four = (size_t)4 * N * sizeof(float) <= 160 * 1024;
    const size_t smem = (size_t)(four ? 4 : 1) * N * sizeof(float);
    if (smem > 200 * 1024) return cudaErrorInvalidValue;
    const int threads = N < 512 * 8 ? 128 : 512;
    cudaError_t e;
    if (four) {
        auto kern = monarch_order_p_kernel<IO, 4>;
        if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
        kern<<<(unsigned)((T + 3) / 4), threads, smem, st>>>((const IO*)X, (IO*)Y, A, N, T);
    } else {
        auto kern = monarch_order_p_kernel<IO, 1>;
        if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
        kern<<<(unsigned)T, threads, smem, st>>>((const IO*)X, (IO*)Y, A, N, T);
    }
    return cudaGetLastError();
}

cudaError_t launch_order_p(const int* dims, int p, long long T, bool bf16_io, const void* X, const void* const* W, void* Y, cudaStream_t st) {
    if (p < 1 || p > 4) return cudaErrorInvalidValue;
    OrderPArgs A;
    long long N = 1;
    for (int a = 0; a < 4; ++a) {
        A.W[a] = a < p ? W[a] : nullptr;
        A.dims[a] = a < p ? dims[a] : 1;
        if (a < p && (dims[a] < 1 || dims[a] > 256)) return cudaErrorInvalidValue;   // 8 outputs per lane
        N *= A.dims[a];
    }
    A.p = p;
    if (N > (1 << 20)) return cudaErrorInvalidValue;
    return bf16_io ? launch_order_p_t<__nv_bfloat16>(A, (int)N, T, X, Y, st) : launch_order_p_t<float>(A, (int)N, T, X, Y, st);
}

cudaError_t launch_mlp(const void* z, const void* Wup, const void* Wdn, void* y, int C, int nblk, int expand,
                       long long tokens, cudaStream_t st) {
    constexpr int TT = 8;
    const int ci = C / nblk, hi = expand * ci;
    const size_t smem = (size_t)TT * (ci + hi) * sizeof(float);
    if (smem > 200 * 1024) return cudaErrorInvalidValue;
    if (tokens == 0) return cudaSuccess;
    auto kern = mlp_blockdiag_kernel<TT>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    dim3 grid((unsigned)((tokens + TT - 1) / TT), (unsigned)nblk);
    kern<<<grid, 256, smem, st>>>((const __nv_bfloat16*)z, (const __nv_bfloat16*)Wup, (const __nv_bfloat16*)Wdn,
                                  (__nv_bfloat16*)y, C, nblk, expand, tokens);
    return cudaGetLastError();
}

// Launch with programmatic stream serialization (the kernel starts with griddepcontrol.launch_dependents / .wait): its CTAs
// may be placed while the previous kernel's last CTAs still run, and the next kernel's while this one's do.
template <typename... KArgs, typename... Args>
static cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}
__device__ __forceinline__ void pdl_prologue() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");   // everything the stream produced before is complete
}

// ---- channel-last <-> channel-first helpers of the M2 block (Sec. 5.1; Eq. 2 runs along the sequence) -----------------
// 64 x 64 bf16 tile transposes through shared memory.  The tile is kept as 32-bit words (two neighbouring columns of one
// row) with a row pitch of 33 words: the 16-byte global loads land as four conflict-free word stores, and the transposed
// side gathers, for one column and 8 consecutive rows, 8 words (2-way conflicts at worst) of which it keeps one half.
constexpr int kTrPitch = 33;

// tile[row][col pair] <- 8 columns (one 16-byte load) of one row
__device__ __forceinline__ void tr_put(uint32_t* tile, int row, int ch, const uint4& v) {
    uint32_t* p = tile + row * kTrPitch + 4 * ch;
    p[0] = v.x;
    p[1] = v.y;
    p[2] = v.z;
    p[3] = v.w;
}
// 8 consecutive rows 8 rb .. 8 rb + 7 of column col -> one 16-byte vector
__device__ __forceinline__ uint4 tr_get(const uint32_t* tile, int rb, int col) {
    const uint32_t* p = tile + (8 * rb) * kTrPitch + (col >> 1);
    const uint32_t sel = (col & 1) ? 0x7632u : 0x5410u;   // high or low halves of two words
    uint4 o;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(o.x) : "r"(p[0 * kTrPitch]), "r"(p[1 * kTrPitch]), "r"(sel));
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(o.y) : "r"(p[2 * kTrPitch]), "r"(p[3 * kTrPitch]), "r"(sel));
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(o.z) : "r"(p[4 * kTrPitch]), "r"(p[5 * kTrPitch]), "r"(sel));
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(o.w) : "r"(p[6 * kTrPitch]), "r"(p[7 * kTrPitch]), "r"(sel));
    return o;
}

// x[B][T][C] -> xT[B][C][T]; both sides move 16 bytes per thread and whole 128-byte rows per 8 threads.
__global__ void __launch_bounds__(256) transpose_btc_kernel(const __nv_bfloat16* __restrict__ x, __nv_bfloat16* __restrict__ xT, int T, int C) {
    __shared__ uint32_t tile[64 * kTrPitch];   // [t][c pair]
    pdl_prologue();
    const int t0 = blockIdx.x * 64, c0 = blockIdx.y * 64;
    const long long b = blockIdx.z;
    const __nv_bfloat16* src = x + (b * T + t0) * (long long)C + c0;
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        const int i = threadIdx.x + 256 * r, tt = i >> 3, ch = i & 7;   // 8 channels c0 + 8 ch .. of row tt
        tr_put(tile, tt, ch, *reinterpret_cast<const uint4*>(src + (long long)tt * C + 8 * ch));
    }
    __syncthreads();
    __nv_bfloat16* dst = xT + (b * C + c0) * (long long)T + t0;
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        const int i = threadIdx.x + 256 * r, cc = i >> 3, tb = i & 7;   // 8 positions t0 + 8 tb .. of channel cc
        *reinterpret_cast<uint4*>(dst + (long long)cc * T + 8 * tb) = tr_get(tile, tb, cc);
    }
}

// z[b][t][c] = (w[c][0] x[b][t-1][c] + w[c][1] x[b][t][c] + w[c][2] x[b][t+1][c]) * v[b][c][t]: the width-3 depthwise
// gate (zero padded) times the long-convolution output, which arrives channel-first and leaves channel-last.
__global__ void __launch_bounds__(256) gate_transpose_kernel(const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ vT,
                                                             const float* __restrict__ w, __nv_bfloat16* __restrict__ z, int T, int C) {
    __shared__ uint32_t tile[64 * kTrPitch];   // [c][t pair]: v as it arrives
    pdl_prologue();   // the convolution's output is complete
    const int t0 = blockIdx.x * 64, c0 = blockIdx.y * 64;
    const long long b = blockIdx.z;
    const __nv_bfloat16* src = vT + (b * C + c0) * (long long)T + t0;
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        const int i = threadIdx.x + 256 * r, cc = i >> 3, ch = i & 7;   // 8 positions t0 + 8 ch .. of channel cc
        tr_put(tile, cc, ch, *reinterpret_cast<const uint4*>(src + (long long)cc * T + 8 * ch));
    }
    __syncthreads();
    const __nv_bfloat16* xb = x + b * (long long)T * C;
    __nv_bfloat16* zb = z + b * (long long)T * C;
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        const int i = threadIdx.x + 256 * r, tt = i >> 3, cb = i & 7, t = t0 + tt, c = c0 + 8 * cb;
        const uint4 xm = *reinterpret_cast<const uint4*>(xb + (long long)t * C + c);
        uint4 xl = make_uint4(0u, 0u, 0u, 0u), xr = make_uint4(0u, 0u, 0u, 0u);   // bf16 zeros outside the sequence
        if (t > 0) xl = *reinterpret_cast<const uint4*>(xb + (long long)(t - 1) * C + c);
        if (t + 1 < T) xr = *reinterpret_cast<const uint4*>(xb + (long long)(t + 1) * C + c);
        const uint4 vv = tr_get(tile, cb, tt);   // channels c .. c + 7 at position t
        const __nv_bfloat16 *em = reinterpret_cast<const __nv_bfloat16*>(&xm), *el = reinterpret_cast<const __nv_bfloat16*>(&xl),
                            *er = reinterpret_cast<const __nv_bfloat16*>(&xr), *ev = reinterpret_cast<const __nv_bfloat16*>(&vv);
        uint4 out;
        __nv_bfloat16* eo = reinterpret_cast<__nv_bfloat16*>(&out);
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const float* wc = w + (c + k) * 3;
            float g = wc[1] * __bfloat162float(em[k]);
            g = fmaf(wc[0], __bfloat162float(el[k]), g);
            g = fmaf(wc[2], __bfloat162float(er[k]), g);
            eo[k] = __float2bfloat16_rn(g * __bfloat162float(ev[k]));
        }
        *reinterpret_cast<uint4*>(zb + (long long)t * C + c) = out;
    }
}

cudaError_t launch_transpose_btc(const void* x, void* xT, long long B, int T, int C, cudaStream_t st) {
    if (T % 64 != 0 || C % 64 != 0) return cudaErrorInvalidValue;
    if (B == 0) return cudaSuccess;
    return launch_pdl(transpose_btc_kernel, dim3(T / 64, C / 64, (unsigned)B), dim3(256), st, (const __nv_bfloat16*)x, (__nv_bfloat16*)xT, T, C);
}

cudaError_t launch_gate_transpose(const void* x, const void* vT, const float* w, void* z, long long B, int T, int C, cudaStream_t st) {
    if (T % 64 != 0 || C % 64 != 0) return cudaErrorInvalidValue;
    if (B == 0) return cudaSuccess;
    return launch_pdl(gate_transpose_kernel, dim3(T / 64, C / 64, (unsigned)B), dim3(256), st, (const __nv_bfloat16*)x, (const __nv_bfloat16*)vT, w,
                      (__nv_bfloat16*)z, T, C);
}

// conj of a spectrum buffer: `pairs` interleaved complex values (re, im), then `quads` values of the tensor-core
// kernels' layouts (re, re', im, im')
__global__ void spectrum_conj_kernel(const float4* __restrict__ in, float4* __restrict__ out, long long pair_quads, long long total) {
    const long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    if (i >= total) return;
    const float4 v = in[i];
    out[i] = i < pair_quads ? make_float4(v.x, -v.y, v.z, -v.w) : make_float4(v.x, v.y, -v.z, -v.w);
}

cudaError_t launch_spectrum_conj(const void* in, void* out, long long plan_order_values, long long private_values, cudaStream_t st) {
    // plan_order_values complex values (even); private_values complex values stored as (re, re', im, im') quads
    const long long pair_quads = plan_order_values / 2, total = pair_quads + private_values / 2;
    if (total == 0) return cudaSuccess;
    spectrum_conj_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>((const float4*)in, (float4*)out, pair_quads, total);
    return cudaGetLastError();
}

long long conv_wgrad_scratch_bytes(long long N, long long H) {
    if ((size_t)N * sizeof(float2) * 3 <= 200 * 1024) return 0;   // fits in shared memory
    return (H < kWgradScratchBlocks ? H : kWgradScratchBlocks) * 3 * N * (long long)sizeof(float2);
}

cudaError_t launch_conv_wgrad(const ConvShape& s, bool bf16_io, const void* x, const void* g, float* dk, void* scratch, long long scratch_bytes,
                              cudaStream_t st) {
    Dims D = make_dims(s);
    Roots R{{s.roots[0], s.roots[1], s.roots[2]}};
    int items, threads;
    if (!pick_launch(D, items, threads)) return cudaErrorInvalidValue;
    size_t smem = (size_t)D.N * sizeof(float2) * 3;
    unsigned grid = (unsigned)s.H;
    float2* gs = nullptr;
    const long long need = conv_wgrad_scratch_bytes(D.N, s.H);
    if (need > 0) {   // rows too long for shared memory: per-block slices of the caller's scratch buffer
        if (!scratch || scratch_bytes < need) return cudaErrorInvalidValue;
        gs = reinterpret_cast<float2*>(scratch);
        smem = 0;
        grid = (unsigned)(s.H < kWgradScratchBlocks ? s.H : kWgradScratchBlocks);
    }
    if (s.H == 0) return cudaSuccess;
#define M2_LAUNCH_WGRAD(IO, IT)                                                                                   \
    {                                                                                                             \
        auto kern = conv_wgrad_kernel<IO, IT>;                                                                    \
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);       \
        if (e != cudaSuccess) return e;                                                                           \
        kern<<<grid, threads, smem, st>>>((const IO*)x, (const IO*)g, dk, D, R, (int)s.B, (int)s.H, (int)s.n, gs); \
    }
    if (bf16_io) {
        switch (items) {
            case 1: M2_LAUNCH_WGRAD(__nv_bfloat16, 1) break;
            case 2: M2_LAUNCH_WGRAD(__nv_bfloat16, 2) break;
            case 4: M2_LAUNCH_WGRAD(__nv_bfloat16, 4) break;
            default: return cudaErrorInvalidValue;
        }
    } else {
        switch (items) {
            case 1: M2_LAUNCH_WGRAD(float, 1) break;
            case 2: M2_LAUNCH_WGRAD(float, 2) break;
            case 4: M2_LAUNCH_WGRAD(float, 4) break;
            default: return cudaErrorInvalidValue;
        }
    }
#undef M2_LAUNCH_WGRAD
    return cudaGetLastError();
}

// out[b][c][r] = in[b][r][c]: block-wise transpose of a block-diagonal factor
template <typename T>
__global__ void blocks_transpose_kernel(const T* __restrict__ in, T* __restrict__ out, int rows, int cols, long long total) {
    const long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x;   // index into out
    if (i >= total) return;
    const int r = (int)(i % rows);
    const int c = (int)((i / rows) % cols);
    const long long b = i / ((long long)rows * cols);
    out[i] = in[(b * rows + r) * cols + c];
}

cudaError_t launch_blocks_transpose(const void* in, void* out, long long nblocks, int rows, int cols, bool bf16, cudaStream_t st) {
    const long long total = nblocks * rows * cols;
    if (total == 0) return cudaSuccess;
    const unsigned grid = (unsigned)((total + 255) / 256);
    if (bf16)
        blocks_transpose_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>((const __nv_bfloat16*)in, (__nv_bfloat16*)out, rows, cols, total);
    else
        blocks_transpose_kernel<float><<<grid, 256, 0, st>>>((const float*)in, (float*)out, rows, cols, total);
    return cudaGetLastError();
}

// First stage of the matmul or of its transpose, fp32 result in index order n2*N1 + k1 (Sec. 3.1):
//   BWD == false: v[n2][k1] = sum_{n1} R[n2][k1][n1] x[n1*N2 + n2]      (W = R, in = X)
//   BWD == true : v[n2][k1] = sum_{k2} L[k1][k2][n2] g[k2*N1 + k1]      (W = L, in = G)
template <typename IO, int TT, bool BWD>
__global__ void matmul_stage1_kernel(const IO* __restrict__ in, const IO* __restrict__ W, float* __restrict__ out, int N1, int N2,
                                     long long T) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int N = N1 * N2;
    float* xs = reinterpret_cast<float*>(smem_raw);  // [TT][N]
    const long long t0 = (long long)blockIdx.x * TT;
    for (int i = threadIdx.x; i < TT * N; i += blockDim.x) {
        const long long t = t0 + i / N;
        xs[i] = (t < T) ? to_f32<IO>(in[t * N + (i % N)]) : 0.f;
    }
    __syncthreads();
    for (int o = threadIdx.x; o < N; o += blockDim.x) {
        const int k1 = o % N1, n2 = o / N1;
        float acc[TT];
#pragma unroll
        for (int t = 0; t < TT; ++t) acc[t] = 0.f;
        if (!BWD) {
            const IO* w = W + ((long long)n2 * N1 + k1) * N1;
            for (int n1 = 0; n1 < N1; ++n1) {
                const float wv = to_f32<IO>(w[n1]);
#pragma unroll
                for (int t = 0; t < TT; ++t) acc[t] = fmaf(wv, xs[t * N + n1 * N2 + n2], acc[t]);
            }
        } else {
            const IO* w = W + (long long)k1 * N2 * N2 + n2;
            for (int k2 = 0; k2 < N2; ++k2) {
                const float wv = to_f32<IO>(w[(long long)k2 * N2]);
#pragma unroll
                for (int t = 0; t < TT; ++t) acc[t] = fmaf(wv, xs[t * N + k2 * N1 + k1], acc[t]);
            }
        }
#pragma unroll
        for (int t = 0; t < TT; ++t)
            if (t0 + t < T) out[(t0 + t) * N + o] = acc[t];
    }
}

// C[b][i][j] = sum_t A[t*N + b*sAb + i*sAi] * B[t*N + b*sBb + j*sBj], i < I, j < J: one 32 x 32 tile of one block per
// CTA, the whole token range walked in chunks of 32 by the same CTA (fixed summation order: deterministic).
template <typename TA, typename TB>
__global__ void __launch_bounds__(256) outer_accum_kernel(const TA* __restrict__ A, const TB* __restrict__ B, float* __restrict__ C, int N,
                                                          long long T, int I, int J, int sAb, int sAi, int sBb, int sBj) {
    __shared__ float as[32][33], bs[32][33];
    const int b = blockIdx.x, i0 = blockIdx.y * 32, j0 = blockIdx.z * 32;
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;   // outputs (i0 + ty + 16 a, j0 + tx + 16 c)
    float acc[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
    for (long long t0 = 0; t0 < T; t0 += 32) {
        for (int e = threadIdx.x; e < 1024; e += 256) {
            const int tt = e / 32, c = e % 32;
            const long long t = t0 + tt;
            as[tt][c] = (t < T && i0 + c < I) ? to_f32<TA>(A[t * N + (long long)b * sAb + (long long)(i0 + c) * sAi]) : 0.f;
            bs[tt][c] = (t < T && j0 + c < J) ? to_f32<TB>(B[t * N + (long long)b * sBb + (long long)(j0 + c) * sBj]) : 0.f;
        }
        __syncthreads();
#pragma unroll 8
        for (int tt = 0; tt < 32; ++tt) {
            const float a0 = as[tt][ty], a1 = as[tt][ty + 16], b0 = bs[tt][tx], b1 = bs[tt][tx + 16];
            acc[0][0] = fmaf(a0, b0, acc[0][0]);
            acc[0][1] = fmaf(a0, b1, acc[0][1]);
            acc[1][0] = fmaf(a1, b0, acc[1][0]);
            acc[1][1] = fmaf(a1, b1, acc[1][1]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
        for (int c = 0; c < 2; ++c) {
            const int i = i0 + ty + 16 * a, j = j0 + tx + 16 * c;
            if (i < I && j < J) C[((long long)b * I + i) * J + j] = acc[a][c];
        }
}

template <typename IO>
static cudaError_t launch_matmul_wgrad_t(int N1, int N2, long long T, const IO* X, const IO* G, const IO* L, const IO* R, float* dL,
                                         float* dR, float* ws, cudaStream_t st) {
    constexpr int TT = 4;
    const int N = N1 * N2;
    const size_t smem = (size_t)TT * N * sizeof(float);
    if (smem > 200 * 1024 || N1 > 65535 * 32 || N2 > 65535 * 32) return cudaErrorInvalidValue;
    auto fwd = matmul_stage1_kernel<IO, TT, false>;
    auto bwd = matmul_stage1_kernel<IO, TT, true>;
    cudaError_t e = cudaFuncSetAttribute(fwd, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(bwd, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const int threads = N < 512 ? ((N + 31) / 32) * 32 : 512;
    const unsigned tiles = (unsigned)((T + TT - 1) / TT);
    const unsigned t1 = (unsigned)((N1 + 31) / 32), t2 = (unsigned)((N2 + 31) / 32);
    if (T > 0) fwd<<<tiles, threads, smem, st>>>(X, R, ws, N1, N2, T);                    // ws = v1[t][n2][k1]
    // dL[k1][k2][n2] = sum_t g[t][k2*N1 + k1] v1[t][n2*N1 + k1]
    outer_accum_kernel<IO, float><<<dim3(N1, t2, t2), 256, 0, st>>>(G, ws, dL, N, T, N2, N2, 1, N1, 1, N1);
    if (T > 0) bwd<<<tiles, threads, smem, st>>>(G, L, ws, N1, N2, T);                    // ws = dv1[t][n2][k1]
    // dR[n2][k1][n1] = sum_t dv1[t][n2*N1 + k1] x[t][n1*N2 + n2]
    outer_accum_kernel<float, IO><<<dim3(N2, t1, t1), 256, 0, st>>>(ws, X, dR, N, T, N1, N1, N1, 1, 1, N2);
    return cudaGetLastError();
}

cudaError_t launch_matmul_wgrad(int N1, int N2, long long T, bool bf16_io, const void* X, const void* G, const void* L, const void* R,
                                float* dL, float* dR, float* ws, cudaStream_t st) {
    return bf16_io ? launch_matmul_wgrad_t<__nv_bfloat16>(N1, N2, T, (const __nv_bfloat16*)X, (const __nv_bfloat16*)G,
                                                          (const __nv_bfloat16*)L, (const __nv_bfloat16*)R, dL, dR, ws, st)
                   : launch_matmul_wgrad_t<float>(N1, N2, T, (const float*)X, (const float*)G, (const float*)L, (const float*)R, dL, dR,
                                                  ws, st);
}

// out[b][c][r] = in[b][r][c] for any sizes and both I/O types: 32 x 32 tiles through shared memory
template <typename T>
__global__ void __launch_bounds__(256) transpose_any_kernel(const T* __restrict__ in, T* __restrict__ out, int R, int C) {
    __shared__ T tile[32][33];
    const long long b = blockIdx.z;
    const int r0 = blockIdx.y * 32, c0 = blockIdx.x * 32;
    const int tx = threadIdx.x % 32, ty = threadIdx.x / 32;
    for (int i = ty; i < 32; i += 8)
        if (r0 + i < R && c0 + tx < C) tile[i][tx] = in[(b * R + r0 + i) * C + c0 + tx];
    __syncthreads();
    for (int i = ty; i < 32; i += 8)
        if (c0 + i < C && r0 + tx < R) out[(b * C + c0 + i) * R + r0 + tx] = tile[tx][i];
}

cudaError_t launch_transpose_any(const void* in, void* out, long long B, int R, int C, bool bf16, cudaStream_t st) {
    if (B == 0 || R == 0 || C == 0) return cudaSuccess;
    if (B > 65535 || (R + 31) / 32 > 65535) return cudaErrorInvalidValue;
    if (bf16 && R % 64 == 0 && C % 64 == 0) return launch_transpose_btc(in, out, B, R, C, st);
    const dim3 grid((C + 31) / 32, (R + 31) / 32, (unsigned)B);
    if (bf16)
        transpose_any_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>((const __nv_bfloat16*)in, (__nv_bfloat16*)out, R, C);
    else
        transpose_any_kernel<float><<<grid, 256, 0, st>>>((const float*)in, (float*)out, R, C);
    return cudaGetLastError();
}

// y[row] = LayerNorm(a[row] + b[row]) * gamma + beta over d values per row (biased variance, fp32 statistics, two passes
// over registers-or-L1-resident data); one 128-thread block per row; y may be a or b.
template <typename IO>
__global__ void __launch_bounds__(128) add_layernorm_kernel(const IO* a, const IO* b, const float* __restrict__ gamma,
                                                            const float* __restrict__ beta, IO* y, int d, float eps) {
    __shared__ float red[4];
    const long long row = blockIdx.x;
    const IO* ar = a + row * d;
    const IO* br = b + row * d;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    auto block_sum = [&](float v) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        __syncthreads();   // red[] may still be read from the previous reduction
        if (lane == 0) red[w] = v;
        __syncthreads();
        return red[0] + red[1] + red[2] + red[3];
    };
    float s = 0.f;
    for (int i = threadIdx.x; i < d; i += 128) s += to_f32<IO>(ar[i]) + to_f32<IO>(br[i]);
    const float mean = block_sum(s) / (float)d;
    float q = 0.f;
    for (int i = threadIdx.x; i < d; i += 128) {
        const float v = to_f32<IO>(ar[i]) + to_f32<IO>(br[i]) - mean;
        q = fmaf(v, v, q);
    }
    const float rstd = rsqrtf(block_sum(q) / (float)d + eps);
    for (int i = threadIdx.x; i < d; i += 128) {
        const float v = to_f32<IO>(ar[i]) + to_f32<IO>(br[i]) - mean;
        y[row * d + i] = from_f32<IO>(fmaf(v * rstd, gamma[i], beta[i]));
    }
}

cudaError_t launch_add_layernorm(const void* a, const void* b, const float* gamma, const float* beta, void* y, long long rows, int d,
                                 float eps, bool bf16, cudaStream_t st) {
    if (rows == 0) return cudaSuccess;
    if (rows > 0x7fffffffLL) return cudaErrorInvalidValue;
    if (bf16)
        add_layernorm_kernel<__nv_bfloat16><<<(unsigned)rows, 128, 0, st>>>((const __nv_bfloat16*)a, (const __nv_bfloat16*)b, gamma, beta,
                                                                           (__nv_bfloat16*)y, d, eps);
    else
        add_layernorm_kernel<float><<<(unsigned)rows, 128, 0, st>>>((const float*)a, (const float*)b, gamma, beta, (float*)y, d, eps);
    return cudaGetLastError();
}

// One block-diagonal factor applied to a matrix whose columns are the vectors (V, O: [Bt][N][d], d contiguous):
//   O[row o*so + j*sjo][c] = sigma(K[that row][c] * sum_i W[j][o][i] * V[row i*si + j*sj][c]),  one thread per output element
template <typename IO>
__global__ void __launch_bounds__(128) cols_stage_kernel(const IO* __restrict__ W, const IO* __restrict__ V, IO* __restrict__ O,
                                                         const IO* __restrict__ Kmul, int relu, int nin, int nout, long long N, int d, long long si,
                                                         long long sj, long long so, long long sjo) {
    const int c = blockIdx.x * 128 + threadIdx.x;
    if (c >= d) return;
    const int j = blockIdx.y / nout, o = blockIdx.y % nout;
    const long long bt = blockIdx.z;
    const IO* w = W + ((long long)j * nout + o) * nin;
    const IO* v = V + (bt * N + j * sj) * d + c;
    float acc = 0.f;
    for (int i = 0; i < nin; ++i) acc = fmaf(to_f32<IO>(w[i]), to_f32<IO>(v[(long long)i * si * d]), acc);
    const long long row = o * so + j * sjo;
    if (Kmul) {
        acc *= to_f32<IO>(Kmul[row * d + c]);
        if (relu) acc = fmaxf(acc, 0.f);
    }
    O[(bt * N + row) * d + c] = from_f32<IO>(acc);
}

// Y = sigma(K (.) P L P^T R P X) on [Bt][N][d] through the intermediate ws ([Bt][N][d], rows k1*N2 + n2)
cudaError_t launch_monarch_cols(int N1, int N2, long long Bt, int d, bool bf16_io, const void* X, const void* L, const void* R, const void* Kmul,
                                int relu, void* Y, void* ws, cudaStream_t st) {
    const long long N = (long long)N1 * N2;
    if (Bt == 0 || d == 0) return cudaSuccess;
    if (Bt > 65535 || N > 65535) return cudaErrorInvalidValue;   // grid limits of this simple kernel
    const dim3 grid((d + 127) / 128, (unsigned)N, (unsigned)Bt);
    if (bf16_io) {
        using T = __nv_bfloat16;
        cols_stage_kernel<T><<<grid, 128, 0, st>>>((const T*)R, (const T*)X, (T*)ws, nullptr, 0, N1, N1, N, d, N2, 1, N2, 1);
        cols_stage_kernel<T><<<grid, 128, 0, st>>>((const T*)L, (const T*)ws, (T*)Y, (const T*)Kmul, relu, N2, N2, N, d, 1, N2, N1, 1);
    } else {
        cols_stage_kernel<float><<<grid, 128, 0, st>>>((const float*)R, (const float*)X, (float*)ws, nullptr, 0, N1, N1, N, d, N2, 1, N2, 1);
        cols_stage_kernel<float><<<grid, 128, 0, st>>>((const float*)L, (const float*)ws, (float*)Y, (const float*)Kmul, relu, N2, N2, N, d, 1, N2,
                                                       N1, 1);
    }
    return cudaGetLastError();
}

// Heads of the M2 Hyena layer, channel-first tensors [B][channels][n] (n contiguous):
//   outer : XV[b][(h dh + i) dh + j][t] = X2[b][h dh + i][t] * V[b][h dh + j][t]
//   reduce: O[b][h dh + j][t] = sum_i X1[b][h dh + i][t] * XVc[b][(h dh + i) dh + j][t]
// one thread per output element (fp32 arithmetic, one rounding on the way out)
template <typename IO>
__global__ void heads_outer_kernel(const IO* __restrict__ X2, const IO* __restrict__ V, IO* __restrict__ XV, int d, int dh, int n,
                                   long long total) {
    const long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x;   // over B * d * dh * n
    if (e >= total) return;
    const int t = (int)(e % n);
    const long long ch = (e / n) % ((long long)d * dh), b = e / ((long long)n * d * dh);
    const int j = (int)(ch % dh), hi = (int)(ch / dh);   // hi = h dh + i
    const int hj = (hi / dh) * dh + j;
    XV[e] = from_f32<IO>(to_f32<IO>(X2[(b * d + hi) * n + t]) * to_f32<IO>(V[(b * d + hj) * n + t]));
}

template <typename IO>
__global__ void heads_reduce_kernel(const IO* __restrict__ X1, const IO* __restrict__ XVc, IO* __restrict__ O, int d, int dh, int n,
                                    long long total) {
    const long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x;   // over B * d * n
    if (e >= total) return;
    const int t = (int)(e % n);
    const int c = (int)((e / n) % d);
    const long long b = e / ((long long)n * d);
    const int h = c / dh, j = c % dh;
    float acc = 0.f;
    for (int i = 0; i < dh; ++i)
        acc = fmaf(to_f32<IO>(X1[(b * d + h * dh + i) * n + t]), to_f32<IO>(XVc[((b * d + h * dh + i) * dh + j) * n + t]), acc);
    O[e] = from_f32<IO>(acc);
}

// The same on bf16 rows whose length is a multiple of 8: 16-byte accesses, one thread per (b, h dh + i, 8 positions) for the
// outer product (its X2 piece is reused for all j) and per (b, h dh + j, 8 positions) for the contraction.
__device__ __forceinline__ void bf16x8_to_f32(const uint4& v, float* f) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        f[2 * q] = __uint_as_float(w[q] << 16);
        f[2 * q + 1] = __uint_as_float(w[q] & 0xffff0000u);
    }
}
__device__ __forceinline__ uint4 f32_to_bf16x8(const float* f) {
    uint32_t w[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        __nv_bfloat162 p = __floats2bfloat162_rn(f[2 * q], f[2 * q + 1]);
        w[q] = *reinterpret_cast<uint32_t*>(&p);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

__global__ void __launch_bounds__(256) heads_outer_bf16x8_kernel(const uint4* __restrict__ X2, const uint4* __restrict__ V, uint4* __restrict__ XV,
                                                                 int d, int dh, int n8, long long total) {
    pdl_prologue();
    const long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x;   // over B * d * n8
    if (e >= total) return;
    const int t8 = (int)(e % n8);
    const int hi = (int)((e / n8) % d);
    const long long b = e / ((long long)n8 * d);
    float a[8], v[8], o[8];
    bf16x8_to_f32(X2[e], a);
    const int h0 = (hi / dh) * dh;
    for (int j = 0; j < dh; ++j) {
        bf16x8_to_f32(V[(b * d + h0 + j) * n8 + t8], v);
#pragma unroll
        for (int q = 0; q < 8; ++q) o[q] = a[q] * v[q];
        XV[((b * d + hi) * dh + j) * n8 + t8] = f32_to_bf16x8(o);
    }
}

__global__ void __launch_bounds__(256) heads_reduce_bf16x8_kernel(const uint4* __restrict__ X1, const uint4* __restrict__ XVc, uint4* __restrict__ O,
                                                                  int d, int dh, int n8, long long total) {
    pdl_prologue();
    const long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x;   // over B * d * n8
    if (e >= total) return;
    const int t8 = (int)(e % n8);
    const int c = (int)((e / n8) % d);
    const long long b = e / ((long long)n8 * d);
    const int h0 = (c / dh) * dh, j = c % dh;
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f}, a[8], v[8];
    for (int i = 0; i < dh; ++i) {
        bf16x8_to_f32(X1[(b * d + h0 + i) * n8 + t8], a);
        bf16x8_to_f32(XVc[((b * d + h0 + i) * dh + j) * n8 + t8], v);
#pragma unroll
        for (int q = 0; q < 8; ++q) acc[q] = fmaf(a[q], v[q], acc[q]);
    }
    O[e] = f32_to_bf16x8(acc);
}

cudaError_t launch_heads_outer(const void* X2, const void* V, void* XV, long long B, int d, int dh, int n, bool bf16, cudaStream_t st) {
    const long long total = B * d * dh * n;
    if (total == 0) return cudaSuccess;
    if (bf16 && n % 8 == 0) {
        const long long t8 = B * d * (n / 8);
        return launch_pdl(heads_outer_bf16x8_kernel, dim3((unsigned)((t8 + 255) / 256)), dim3(256), st, (const uint4*)X2, (const uint4*)V, (uint4*)XV, d, dh,
                          n / 8, t8);
    }
    const unsigned grid = (unsigned)((total + 255) / 256);
    if (bf16)
        heads_outer_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>((const __nv_bfloat16*)X2, (const __nv_bfloat16*)V, (__nv_bfloat16*)XV, d, dh, n, total);
    else
        heads_outer_kernel<float><<<grid, 256, 0, st>>>((const float*)X2, (const float*)V, (float*)XV, d, dh, n, total);
    return cudaGetLastError();
}

cudaError_t launch_heads_reduce(const void* X1, const void* XVc, void* O, long long B, int d, int dh, int n, bool bf16, cudaStream_t st) {
    const long long total = B * d * n;
    if (total == 0) return cudaSuccess;
    if (bf16 && n % 8 == 0) {
        const long long t8 = B * d * (n / 8);
        return launch_pdl(heads_reduce_bf16x8_kernel, dim3((unsigned)((t8 + 255) / 256)), dim3(256), st, (const uint4*)X1, (const uint4*)XVc, (uint4*)O, d,
                          dh, n / 8, t8);
    }
    const unsigned grid = (unsigned)((total + 255) / 256);
    if (bf16)
        heads_reduce_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>((const __nv_bfloat16*)X1, (const __nv_bfloat16*)XVc, (__nv_bfloat16*)O, d, dh, n, total);
    else
        heads_reduce_kernel<float><<<grid, 256, 0, st>>>((const float*)X1, (const float*)XVc, (float*)O, d, dh, n, total);
    return cudaGetLastError();
}

// O[bt] = W V[bt] on the CUDA cores: W [c][c] (outputs x inputs), V, O [Bt][c][cols] (one block-diagonal stage with a single block)
cudaError_t launch_dense_cols(const void* W, const void* V, void* O, long long Bt, int c, int cols, bool bf16, cudaStream_t st) {
    if (Bt == 0 || c == 0 || cols == 0) return cudaSuccess;
    if (Bt > 65535 || c > 65535) return cudaErrorInvalidValue;
    const dim3 grid((cols + 127) / 128, (unsigned)c, (unsigned)Bt);
    if (bf16)
        cols_stage_kernel<__nv_bfloat16><<<grid, 128, 0, st>>>((const __nv_bfloat16*)W, (const __nv_bfloat16*)V, (__nv_bfloat16*)O, nullptr, 0, c, c, c,
                                                               cols, 1, 0, 1, 0);
    else
        cols_stage_kernel<float><<<grid, 128, 0, st>>>((const float*)W, (const float*)V, (float*)O, nullptr, 0, c, c, c, cols, 1, 0, 1, 0);
    return cudaGetLastError();
}

// Gated mixer pieces on channel-first tensors [B][d][n] (n contiguous); DW3(a; w)[t] = w0 a[t-1] + w1 a[t] + w2 a[t+1], zero padded:
//   gate_in : QK[b][c][t] = DW3(Pq[b][c]; wq[c])[t] * DW3(Pk[b][c]; wk[c])[t]
//   gate_out: Z[b][c][t]  = DW3(Pv[b][c]; wv[c])[t] * C[b][c][t] + Cr[b][c][t]
// one thread per element, fp32 arithmetic, one rounding on the way out (Z may alias Pv's buffer only if it does not: it reads
// neighbours, so the output must be a different buffer)
template <typename IO>
__device__ __forceinline__ float dw3_at(const IO* __restrict__ row, const float* __restrict__ w, int t, int n) {
    float g = w[1] * to_f32<IO>(row[t]);
    if (t > 0) g = fmaf(w[0], to_f32<IO>(row[t - 1]), g);
    if (t + 1 < n) g = fmaf(w[2], to_f32<IO>(row[t + 1]), g);
    return g;
}

template <typename IO>
__global__ void gate_in_kernel(const IO* __restrict__ Pq, const IO* __restrict__ Pk, const float* __restrict__ wq, const float* __restrict__ wk,
                               IO* __restrict__ QK, int d, int n, long long total) {
    const long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x;   // over B * d * n
    if (e >= total) return;
    const int t = (int)(e % n);
    const long long rowi = e / n;
    const int c = (int)(rowi % d);
    QK[e] = from_f32<IO>(dw3_at<IO>(Pq + rowi * n, wq + 3 * c, t, n) * dw3_at<IO>(Pk + rowi * n, wk + 3 * c, t, n));
}

template <typename IO>
__global__ void gate_out_kernel(const IO* __restrict__ Pv, const float* __restrict__ wv, const IO* __restrict__ C, const IO* __restrict__ Cr,
                                IO* __restrict__ Z, int d, int n, long long total) {
    const long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    if (e >= total) return;
    const int t = (int)(e % n);
    const long long rowi = e / n;
    const int c = (int)(rowi % d);
    Z[e] = from_f32<IO>(fmaf(dw3_at<IO>(Pv + rowi * n, wv + 3 * c, t, n), to_f32<IO>(C[e]), to_f32<IO>(Cr[e])));
}

// bf16 rows whose length is a multiple of 8: 8 positions per thread (one 16-byte piece plus the two neighbours)
__device__ __forceinline__ void dw3_x8(const __nv_bfloat16* __restrict__ row, const float* __restrict__ w, int t0, int n, float* g) {
    float a[10];
    bf16x8_to_f32(*reinterpret_cast<const uint4*>(row + t0), a + 1);
    a[0] = t0 > 0 ? __bfloat162float(row[t0 - 1]) : 0.f;
    a[9] = t0 + 8 < n ? __bfloat162float(row[t0 + 8]) : 0.f;
#pragma unroll
    for (int q = 0; q < 8; ++q) g[q] = fmaf(w[0], a[q], fmaf(w[1], a[q + 1], w[2] * a[q + 2]));
}

__global__ void __launch_bounds__(256) gate_in_bf16x8_kernel(const __nv_bfloat16* __restrict__ Pq, const __nv_bfloat16* __restrict__ Pk,
                                                             const float* __restrict__ wq, const float* __restrict__ wk,
                                                             __nv_bfloat16* __restrict__ QK, int d, int n, long long total8) {
    pdl_prologue();
    const long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x;   // over B * d * n / 8
    if (e >= total8) return;
    const int n8 = n / 8, t0 = (int)(e % n8) * 8;
    const long long rowi = e / n8;
    const int c = (int)(rowi % d);
    float gq[8], gk[8];
    dw3_x8(Pq + rowi * n, wq + 3 * c, t0, n, gq);
    dw3_x8(Pk + rowi * n, wk + 3 * c, t0, n, gk);
#pragma unroll
    for (int q = 0; q < 8; ++q) gq[q] *= gk[q];
    *reinterpret_cast<uint4*>(QK + rowi * n + t0) = f32_to_bf16x8(gq);
}

__global__ void __launch_bounds__(256) gate_out_bf16x8_kernel(const __nv_bfloat16* __restrict__ Pv, const float* __restrict__ wv,
                                                              const __nv_bfloat16* __restrict__ C, const __nv_bfloat16* __restrict__ Cr,
                                                              __nv_bfloat16* __restrict__ Z, int d, int n, long long total8) {
    pdl_prologue();
    const long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    if (e >= total8) return;
    const int n8 = n / 8, t0 = (int)(e % n8) * 8;
    const long long rowi = e / n8;
    const int c = (int)(rowi % d);
    float gv[8], cv[8], rv[8];
    dw3_x8(Pv + rowi * n, wv + 3 * c, t0, n, gv);
    bf16x8_to_f32(*reinterpret_cast<const uint4*>(C + rowi * n + t0), cv);
    bf16x8_to_f32(*reinterpret_cast<const uint4*>(Cr + rowi * n + t0), rv);
#pragma unroll
    for (int q = 0; q < 8; ++q) gv[q] = fmaf(gv[q], cv[q], rv[q]);
    *reinterpret_cast<uint4*>(Z + rowi * n + t0) = f32_to_bf16x8(gv);
}

cudaError_t launch_gate_in(const void* Pq, const void* Pk, const float* wq, const float* wk, void* QK, long long B, int d, int n, bool bf16,
                           cudaStream_t st) {
    const long long total = B * d * n;
    if (total == 0) return cudaSuccess;
    if (bf16 && n % 8 == 0) {
        return launch_pdl(gate_in_bf16x8_kernel, dim3((unsigned)((total / 8 + 255) / 256)), dim3(256), st, (const __nv_bfloat16*)Pq,
                          (const __nv_bfloat16*)Pk, wq, wk, (__nv_bfloat16*)QK, d, n, total / 8);
    }
    const unsigned grid = (unsigned)((total + 255) / 256);
    if (bf16)
        gate_in_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>((const __nv_bfloat16*)Pq, (const __nv_bfloat16*)Pk, wq, wk, (__nv_bfloat16*)QK, d, n, total);
    else
        gate_in_kernel<float><<<grid, 256, 0, st>>>((const float*)Pq, (const float*)Pk, wq, wk, (float*)QK, d, n, total);
    return cudaGetLastError();
}

cudaError_t launch_gate_out(const void* Pv, const float* wv, const void* C, const void* Cr, void* Z, long long B, int d, int n, bool bf16,
                            cudaStream_t st) {
    const long long total = B * d * n;
    if (total == 0) return cudaSuccess;
    if (bf16 && n % 8 == 0) {
        return launch_pdl(gate_out_bf16x8_kernel, dim3((unsigned)((total / 8 + 255) / 256)), dim3(256), st, (const __nv_bfloat16*)Pv, wv,
                          (const __nv_bfloat16*)C, (const __nv_bfloat16*)Cr, (__nv_bfloat16*)Z, d, n, total / 8);
    }
    const unsigned grid = (unsigned)((total + 255) / 256);
    if (bf16)
        gate_out_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>((const __nv_bfloat16*)Pv, wv, (const __nv_bfloat16*)C, (const __nv_bfloat16*)Cr,
                                                             (__nv_bfloat16*)Z, d, n, total);
    else
        gate_out_kernel<float><<<grid, 256, 0, st>>>((const float*)Pv, wv, (const float*)C, (const float*)Cr, (float*)Z, d, n, total);
    return cudaGetLastError();
}

}  // namespace m2g
