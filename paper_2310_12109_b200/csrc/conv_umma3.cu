// Tensor-core Monarch convolution, order 3, N = 32768 = 32 x 32 x 32, causal with n = 16384, bf16 in /
// fp32 accumulate / bf16 out (the long M2-GPT-shaped mixer).
//
// y = Re( M^-1 ( k_f (.) M pad(x) ) ), M = F_N as an order-3 Monarch matrix (Eq. 1, Eq. 2; App. D.6
// "p-variate Monarch"; Corollary "DFT is M" generalised: stage a contracts digit n_a with F_32 after a
// twiddle diagonal).  One CTA per SM works on one PAIR of batch rows of the same channel at a time:
// because the kernel k is real, the two real rows ride as the real and imaginary part of one complex
// row (F^-1(F(xa + i xb) . k_f) = ya + i yb), which halves every stage.  Zero padding makes the upper
// half of digit n1 zero on the way in and unneeded on the way out, so the first stage has K = 32 and
// the last N = 32.
//
// A stage is 8 UMMA tiles (M = 128 lanes = 128 values of the two digits that are not being contracted,
// N = 64 = (re|im) x 32 outputs, K = 64 = (re|im) x 32 inputs); the 8 accumulators fill the 512 TMEM
// columns.  After each stage all 512 threads read their lanes back, apply the twiddle (or the
// spectrum) in fp32, round to bf16 and write the next stage's A operand straight into its UMMA layout
// in the one 128 KB operand buffer -- that write is the stride permutation.  Lane orders are chosen so
// that the eight lanes of a quarter-warp always land in one 128-byte swizzle row (128B-swizzled,
// M-major operands) or in one core matrix (K-major operand of the first inverse stage): conflict-free.
//
//   stage   contracts   lanes of D (tile j, lane t)                      hand-off after it
//   S1      n1 (K=32)   n2 = 4j + t/32, n3 = t%32                        w_1024^{n2 k1}            -> A2
//   S2      n2          k1 = 8(2(j&1)+t/64) + t%8, n3 = 8(j/2) + (t/8)%8 w_N^{n3 (k1 + 32 k2)}     -> A3
//   S3      n3          k2 = 8(2(j&1)+t/64) + t%8, k1 = 8(j/2) + (t/8)%8 spectrum k_f              -> A4 (K-major)
//   S3'     k3          same lanes, columns n3                           conj w_N^{n3 (k1+32 k2)}  -> A5
//   S2'     k2          n3 = 8(2(j&1)+t/64) + t%8, k1 = 8(j/2) + (t/8)%8 conj w_1024^{n2 k1}       -> A6
//   S1'     k1 (N=32)   n2 = 8(j/2) + t%8, n3 = 8(2(j&1)+t/64) + (t/8)%8 round, stage (64B-swizzled box image), TMA store
//
// The fp32 arithmetic of the hand-offs is packed (fma.rn.f32x2: two complex products in five instructions); the
// twiddles w_N^{n3 (k1 + 32 k2)} are geometric sequences in k2 (resp. n3) and run as packed chains stepping by rho^2.
#include <cuda.h>
#include <cuda_bf16.h>

#include <cmath>
#include <cstring>
#include <vector>

#include "conv_umma.h"
#include "ptx_sm100.cuh"
#include "tma_host.h"

namespace m2u3 {

using namespace sm100;

constexpr int kThreads = 512;
constexpr int kN = 32768;
// shared memory map
constexpr int OFF_A = 0;                 // operand buffer (also the output staging)   131072
constexpr int OFF_X = 131072;            // packed input pair, S1's A operand            65536
constexpr int OFF_CONST = 196608;        // B1 4096 | BF 8192 | BI 8192 | B6 4096 | tw 8704
constexpr int CONST_BYTES = 4096 + 8192 + 8192 + 4096 + 8704;
constexpr int OFF_B1 = OFF_CONST, OFF_BF = OFF_B1 + 4096, OFF_BI = OFF_BF + 8192, OFF_B6 = OFF_BI + 8192;
constexpr int OFF_TW = OFF_B6 + 4096;    // w_1024^{a b}: row a = 17 float4 (cos b, cos b+1, sin b, sin b+1), b even
constexpr int OFF_BAR = OFF_CONST + CONST_BYTES;   // bar_mma, flag, tmem ptr
constexpr int SMEM_BYTES = OFF_BAR + 64;
static_assert(SMEM_BYTES <= 232448, "shared memory budget");

struct Tables {
    void* d_const = nullptr;   // CONST_BYTES
    float2* d_tn = nullptr;    // w_N^{a b}, a, b < 32, row stride 32
};

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float2 cmul(float2 a, float2 b) { return make_float2(a.x * b.x - a.y * b.y, a.x * b.y + a.y * b.x); }
__device__ __forceinline__ float2 conjf(float2 a) { return make_float2(a.x, -a.y); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, uint32_t src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_store(void* gdst, uint32_t ssrc, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst), "r"(ssrc), "r"(bytes) : "memory");
}

// 128-byte-swizzled M-major operand: 64-element M blocks 8192 B apart, groups of 8 K rows 1024 B apart
__device__ __forceinline__ uint32_t a_off(int mb, int kgroup, int krow, int mchunk) {
    return (uint32_t)(mb * 8192 + kgroup * 1024 + krow * 128 + ((mchunk ^ krow) << 4));
}

// reads the 64 columns (re 0..31 | im 32..63) of this thread's lane in one accumulator tile
__device__ __forceinline__ void load_tile(uint32_t taddr, float* re, float* im) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        tmem_ld8(taddr + 8 * i, re + 8 * i);
        tmem_ld8(taddr + 32 + 8 * i, im + 8 * i);
    }
    tmem_ld_wait();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        tmem_ld_fence8(re + 8 * i);
        tmem_ld_fence8(im + 8 * i);
    }
}

// Two neighbouring complex values (re pair a0 a1, im pair b0 b1) times (c + i s) given as packed pairs c2, s2;
// the products leave as bf16 pairs.  Packed fp32 arithmetic: 5 instructions for the two complex products.
__device__ __forceinline__ void cmul2_pack(float a0, float a1, float b0, float b1, uint64_t c2, uint64_t s2, uint32_t& pr, uint32_t& pi) {
    const uint64_t a2 = pk2(a0, a1), b2 = pk2(b0, b1);
    const uint64_t r2 = fma2(sub2(0ull, b2), s2, mul2(a2, c2));   // a c - b s
    const uint64_t i2 = fma2(b2, c2, mul2(a2, s2));               // a s + b c
    float x0, x1, y0, y1;
    upk2(r2, x0, x1);
    upk2(i2, y0, y1);
    pr = pack_bf16(x0, x1);
    pi = pack_bf16(y0, y1);
}
// the same times the conjugate (c - i s)
__device__ __forceinline__ void cmul2_conj_pack(float a0, float a1, float b0, float b1, uint64_t c2, uint64_t s2, uint32_t& pr, uint32_t& pi) {
    const uint64_t a2 = pk2(a0, a1), b2 = pk2(b0, b1);
    const uint64_t r2 = fma2(b2, s2, mul2(a2, c2));               // a c + b s
    const uint64_t i2 = fma2(sub2(0ull, a2), s2, mul2(b2, c2));   // b c - a s
    float x0, x1, y0, y1;
    upk2(r2, x0, x1);
    upk2(i2, y0, y1);
    pr = pack_bf16(x0, x1);
    pi = pack_bf16(y0, y1);
}

// 8 complex values times f, f rho, ..., f rho^7: the factors of neighbouring values run as one packed chain that
// steps by rho^2 (three steps per call)
__device__ __forceinline__ void geometric8_pack(const float* re, const float* im, float2 f, float2 rho, uint4& pr, uint4& pi) {
    const float2 g = cmul(f, rho), q = cmul(rho, rho);
    uint64_t fr = pk2(f.x, g.x), fi = pk2(f.y, g.y);
    const uint64_t qr = pk2(q.x, q.x), qi = pk2(q.y, q.y), nqi = pk2(-q.y, -q.y);
    uint32_t r_[4], i_[4];
#pragma unroll
    for (int p = 0; p < 4; ++p) {
        cmul2_pack(re[2 * p], re[2 * p + 1], im[2 * p], im[2 * p + 1], fr, fi, r_[p], i_[p]);
        if (p < 3) {
            const uint64_t nr = fma2(fi, nqi, mul2(fr, qr)), ni = fma2(fi, qr, mul2(fr, qi));
            fr = nr;
            fi = ni;
        }
    }
    pr = make_uint4(r_[0], r_[1], r_[2], r_[3]);
    pi = make_uint4(i_[0], i_[1], i_[2], i_[3]);
}

// loads one packed input pair (rows a and b of channel h) into the S1 operand layout
__device__ __forceinline__ void load_pair(uint32_t s_x, const __nv_bfloat16* xa, const __nv_bfloat16* xb, bool has_b) {
    // 4096 chunks of 16 bytes: chunk = (c, n1 < 16, pc = p / 8)
    for (int ch = threadIdx.x; ch < 4096; ch += kThreads) {
        const int pc = ch & 127, n1 = (ch >> 7) & 15, c = ch >> 11;
        const int k = c * 16 + n1;
        const uint32_t dst = s_x + (uint32_t)((pc >> 3) * 4096 + (k >> 3) * 1024 + (k & 7) * 128 + (((pc & 7) ^ (k & 7)) << 4));
        const __nv_bfloat16* src = (c == 0 ? xa : xb) + n1 * 1024 + pc * 8;
        cp_async16(dst, (c == 0 || has_b) ? (const void*)src : (const void*)xa, (c == 0 || has_b) ? 16u : 0u);
    }
    cp_async_commit();
}

// MODE 0: the convolution.  kf_per_pair != 0: the spectrum block is selected by the row pair instead of by the channel (the
//         kernel-gradient path: every pair is multiplied by its own conj(M x) / N).
// MODE 1: only the forward transform: conj(M (xa + i xb)) / N of every row pair is written to spec_out in the layout hand-off 3
//         reads (pair index in place of the channel); no output rows.
template <int MODE>
__global__ void __launch_bounds__(kThreads, 1)
conv32k_kernel(const __grid_constant__ CUtensorMap map_y, const __nv_bfloat16* __restrict__ x, const float4* __restrict__ kfu,
               const uint4* __restrict__ consts, const float2* __restrict__ tn, int B, int H, int32_t* __restrict__ status,
               int kf_per_pair, float4* __restrict__ spec_out) {
    extern __shared__ __align__(1024) unsigned char smem[];
    const int tid = threadIdx.x;
    const int wg = tid >> 7, t = tid & 127, warp = t >> 5;
    const bool issuer = t == 32 * wg;   // one UMMA-issuing thread per warpgroup, each on a different scheduler
    const uint32_t s_base = smem_u32(smem);
    const uint32_t bar_mma = s_base + OFF_BAR, s_tptr = s_base + OFF_BAR + 16;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + OFF_BAR + 8);
    const size_t row_elems = 16384;

    const int bpairs = (B + 1) / 2;
    const int pairs = H * bpairs;
    int pr_i = blockIdx.x;
    if (tid == 0) {
        mbar_init(bar_mma, 4);   // one commit per warpgroup's issuing thread
        *abort_flag = 0;
        fence_barrier_init();
    }
    // Programmatic dependent launch: the next kernel's CTAs may take over SMs as this grid's CTAs leave them; the
    // plan-owned constants and the TMEM allocation do not depend on anything the stream ran before.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    {
        uint4* dst = reinterpret_cast<uint4*>(smem + OFF_CONST);
        for (int i = tid; i < CONST_BYTES / 16; i += kThreads) dst[i] = consts[i];
    }
    if (tid < 32) tmem_alloc(s_tptr, 512);
    asm volatile("griddepcontrol.wait;" ::: "memory");   // producers of x / the spectrum and earlier users of y are done
    if (pr_i < pairs) {
        const int h = pr_i / bpairs, b0 = (pr_i % bpairs) * 2;
        load_pair(s_base + OFF_X, x + ((size_t)b0 * H + h) * row_elems, x + ((size_t)(b0 + 1) * H + h) * row_elems, b0 + 1 < B);
    }
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(smem + OFF_BAR + 16);
    const uint32_t t_lane = tmem + ((uint32_t)(warp * 32) << 16);
    const float4* tw4 = reinterpret_cast<const float4*>(smem + OFF_TW);   // row a: tw4[a * 17 + b / 2]
    auto tw_at = [&](int a, int b) {                                       // w_1024^{a b} as one complex value
        const float* p = reinterpret_cast<const float*>(tw4 + a * 17 + (b >> 1)) + (b & 1);
        return make_float2(p[0], p[2]);
    };

    constexpr uint32_t ID_S1 = instr_desc_bf16(128, 64, true, false);
    constexpr uint32_t ID_MM = instr_desc_bf16(128, 64, true, false);    // M-major A, N = 64
    constexpr uint32_t ID_KM = instr_desc_bf16(128, 64, false, false);   // K-major A, N = 64
    constexpr uint32_t ID_S6 = instr_desc_bf16(128, 32, true, false);    // last stage, N = 32

    uint32_t ph = 0;
    bool ok = true, aborted = false, store_pending = false;

#define M2_STAGE_SYNC()                                   \
    fence_proxy_async();                                  \
    tc_fence_before();                                    \
    if (__syncthreads_or(!ok)) {                          \
        aborted = true;                                   \
        break;                                            \
    }
#define M2_WAIT_MMA()                  \
    ok = mbar_wait(bar_mma, ph);       \
    ph ^= 1;                           \
    tc_fence_after();

    for (; pr_i < pairs; pr_i += gridDim.x) {
        const int h = pr_i / bpairs, b0 = (pr_i % bpairs) * 2;
        const bool has_b = b0 + 1 < B;
        // the pair's input has landed (every thread waits for its own copies, then the block syncs)
        cp_async_wait_all();
        M2_STAGE_SYNC()
        const int kidx = kf_per_pair ? pr_i : h;   // which 256 KB spectrum block this pair is multiplied by
        // pull this pair's 256 KB of spectrum towards L2 now; hand-off 3 reads it five stages later
        if (MODE == 0 && (t & 7) == 0) {
#pragma unroll 1
            for (int jj = 0; jj < 2; ++jj) {
                const float4* kp = kfu + ((size_t)(kidx * 8 + wg + 4 * jj) * 16) * 128 + t;
#pragma unroll
                for (int q = 0; q < 16; ++q) asm volatile("prefetch.global.L2 [%0];" ::"l"(kp + q * 128));
            }
        }
        // ---- S1: contract n1 (K = 32: the zero half is skipped) -----------------------------------------
        if (issuer) {   // one thread of every warpgroup issues the UMMAs of the two tiles its warpgroup hands off
            if (tid == 0 && store_pending) {   // the previous pair's output staging must be read out before A is reused
                tma_store_wait_read0();
                store_pending = false;
            }
            tc_fence_after();
#pragma unroll
            for (int jj = 0; jj < 2; ++jj)
#pragma unroll
                for (int s = 0; s < 2; ++s)
                    umma_f16(tmem + (wg + 4 * jj) * 64, smem_desc_sw128(s_base + OFF_X + (wg + 4 * jj) * 8192 + s * 2048, 4096, 1024),
                             smem_desc(s_base + OFF_B1 + s * 256, 128, 512), ID_S1, s > 0);
            umma_commit(bar_mma);
        }
        M2_WAIT_MMA()
        {   // the input buffer is free again: start fetching the next pair
            const int nx = pr_i + gridDim.x;
            if (ok && nx < pairs) {
                const int hn = nx / bpairs, bn = (nx % bpairs) * 2;
                load_pair(s_base + OFF_X, x + ((size_t)bn * H + hn) * row_elems, x + ((size_t)(bn + 1) * H + hn) * row_elems, bn + 1 < B);
            }
        }
        // ---- h1: w_1024^{n2 k1}; A2[(n3, k1)][(c, n2)] -----------------------------------------------------
        if (ok) {
#pragma unroll 1
            for (int jj = 0; jj < 2; ++jj) {
                const int j = wg + 4 * jj;
                const int n2 = 4 * j + (t >> 5), n3 = t & 31;
                float re[32], im[32];
                load_tile(t_lane + j * 64, re, im);
                const float4* twr = tw4 + n2 * 17;   // warp-uniform row
#pragma unroll
                for (int hi = 0; hi < 4; ++hi) {
                    uint32_t r_[4], i_[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const float4 w = twr[4 * hi + q];
                        cmul2_pack(re[8 * hi + 2 * q], re[8 * hi + 2 * q + 1], im[8 * hi + 2 * q], im[8 * hi + 2 * q + 1], pk2(w.x, w.y),
                                   pk2(w.z, w.w), r_[q], i_[q]);
                    }
                    const int mb = (n3 >> 3) * 4 + hi;
                    *reinterpret_cast<uint4*>(smem + OFF_A + a_off(mb, (n2 >> 3), n2 & 7, n3 & 7)) = make_uint4(r_[0], r_[1], r_[2], r_[3]);
                    *reinterpret_cast<uint4*>(smem + OFF_A + a_off(mb, 4 + (n2 >> 3), n2 & 7, n3 & 7)) = make_uint4(i_[0], i_[1], i_[2], i_[3]);
                }
            }
        }
        M2_STAGE_SYNC()
        // ---- S2: contract n2 -----------------------------------------------------------------------------------
        if (issuer) {
            tc_fence_after();
#pragma unroll
            for (int jj = 0; jj < 2; ++jj)
#pragma unroll
                for (int s = 0; s < 4; ++s)
                    umma_f16(tmem + (wg + 4 * jj) * 64, smem_desc_sw128(s_base + OFF_A + (wg + 4 * jj) * 16384 + s * 2048, 8192, 1024),
                             smem_desc(s_base + OFF_BF + s * 256, 128, 1024), ID_MM, s > 0);
            umma_commit(bar_mma);
        }
        // (the first factor of hand-off 2 comes from L2: the first tile's is asked for before the wait for the UMMAs, the second
        // tile's while the first is worked on; tile wg + 4 has the same k1 and n3 larger by 16)
        const float2* tn_h2 = tn + (((wg >> 1) << 3) + ((t >> 3) & 7)) * 32 + ((2 * (wg & 1) + (t >> 6)) << 3) + (t & 7);
        float2 f0_next = __ldg(tn_h2);
        M2_WAIT_MMA()
        // ---- h2: w_N^{n3 (k1 + 32 k2)} = w_N^{n3 k1} (w_1024^{n3})^{k2}; A3[(k1, k2)][(c, n3)] --------------------
        if (ok) {
#pragma unroll 1
            for (int jj = 0; jj < 2; ++jj) {
                const int j = wg + 4 * jj;
                const int k1 = ((2 * (j & 1) + (t >> 6)) << 3) + (t & 7), n3 = ((j >> 1) << 3) + ((t >> 3) & 7);
                const float2 f0 = f0_next;
                if (jj == 0) f0_next = __ldg(tn_h2 + 16 * 32);
                float re[32], im[32];
                load_tile(t_lane + j * 64, re, im);
                const float2 rho = tw_at(n3, 1);
#pragma unroll
                for (int hi = 0; hi < 4; ++hi) {
                    uint4 pr, pi;
                    geometric8_pack(re + 8 * hi, im + 8 * hi, hi == 0 ? f0 : cmul(f0, tw_at(n3, 8 * hi)), rho, pr, pi);
                    const int mb = (k1 >> 3) * 4 + hi;
                    *reinterpret_cast<uint4*>(smem + OFF_A + a_off(mb, (n3 >> 3), n3 & 7, k1 & 7)) = pr;
                    *reinterpret_cast<uint4*>(smem + OFF_A + a_off(mb, 4 + (n3 >> 3), n3 & 7, k1 & 7)) = pi;
                }
            }
        }
        M2_STAGE_SYNC()
        // ---- S3: contract n3 -----------------------------------------------------------------------------------
        if (issuer) {
            tc_fence_after();
#pragma unroll
            for (int jj = 0; jj < 2; ++jj)
#pragma unroll
                for (int s = 0; s < 4; ++s)
                    umma_f16(tmem + (wg + 4 * jj) * 64, smem_desc_sw128(s_base + OFF_A + (wg + 4 * jj) * 16384 + s * 2048, 8192, 1024),
                             smem_desc(s_base + OFF_BF + s * 256, 128, 1024), ID_MM, s > 0);
            umma_commit(bar_mma);
        }
        // ---- h3: spectrum multiply (k_f holds 1/N); A4 K-major: row = lane, K = (c, k3).  All of a tile's spectrum
        //      values are requested before the wait for the UMMAs, the second tile's while the first is worked on. ------
        if constexpr (MODE == 1) {
            // the spectrum of the pair, conjugated and scaled by 1 / N, in the layout hand-off 3 reads it back in
            M2_WAIT_MMA()
            if (ok) {
                const float inv = 1.0f / (float)kN;
#pragma unroll 1
                for (int jj = 0; jj < 2; ++jj) {
                    const int j = wg + 4 * jj;
                    float4* dst = spec_out + ((size_t)(pr_i * 8 + j) * 16) * 128 + t;
                    float re[32], im[32];
                    load_tile(t_lane + j * 64, re, im);
#pragma unroll
                    for (int q = 0; q < 16; ++q)
                        dst[q * 128] = make_float4(re[2 * q] * inv, re[2 * q + 1] * inv, -im[2 * q] * inv, -im[2 * q + 1] * inv);
                }
            }
            continue;   // the next pair's first barrier orders these accumulator reads before its UMMAs
        }
        {
            const float4* kp0 = kfu + ((size_t)(kidx * 8 + wg) * 16) * 128 + t;
            float4 w[16];
#pragma unroll
            for (int q = 0; q < 16; ++q) w[q] = __ldg(kp0 + q * 128);
            M2_WAIT_MMA()
            if (ok) {
#pragma unroll
                for (int jj = 0; jj < 2; ++jj) {
                    const int j = wg + 4 * jj;
                    unsigned char* rowp = smem + OFF_A + j * 16384 + (t >> 3) * 1024 + (t & 7) * 16;
#pragma unroll
                    for (int hi = 0; hi < 4; ++hi) {
                        float re[8], im[8];
                        tmem_ld8(t_lane + j * 64 + 8 * hi, re);
                        tmem_ld8(t_lane + j * 64 + 32 + 8 * hi, im);
                        tmem_ld_wait();
                        tmem_ld_fence8(re);
                        tmem_ld_fence8(im);
                        uint32_t r_[4], i_[4];
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const float4 ww = w[4 * hi + q];
                            if (jj == 0) w[4 * hi + q] = __ldg(kp0 + (size_t)4 * 16 * 128 + (4 * hi + q) * 128);   // tile wg + 4
                            cmul2_pack(re[2 * q], re[2 * q + 1], im[2 * q], im[2 * q + 1], pk2(ww.x, ww.y), pk2(ww.z, ww.w), r_[q], i_[q]);
                        }
                        *reinterpret_cast<uint4*>(rowp + hi * 128) = make_uint4(r_[0], r_[1], r_[2], r_[3]);
                        *reinterpret_cast<uint4*>(rowp + (4 + hi) * 128) = make_uint4(i_[0], i_[1], i_[2], i_[3]);
                    }
                }
            }
        }
        M2_STAGE_SYNC()
        // ---- S3': contract k3 with conj F ---------------------------------------------------------------------------
        if (issuer) {
            tc_fence_after();
#pragma unroll
            for (int jj = 0; jj < 2; ++jj)
#pragma unroll
                for (int s = 0; s < 4; ++s)
                    umma_f16(tmem + (wg + 4 * jj) * 64, smem_desc(s_base + OFF_A + (wg + 4 * jj) * 16384 + s * 256, 128, 1024),
                             smem_desc(s_base + OFF_BI + s * 256, 128, 1024), ID_KM, s > 0);
            umma_commit(bar_mma);
        }
        // (hand-off 4's factors w_N^{m k1}, m = 1, 8, 16, 24: the same way; tile wg + 4 has k1 larger by 16)
        const float2* tn_h4 = tn + ((wg >> 1) << 3) + ((t >> 3) & 7);
        float2 g_next[4];
        g_next[0] = __ldg(tn_h4 + 32);
#pragma unroll
        for (int hi = 1; hi < 4; ++hi) g_next[hi] = __ldg(tn_h4 + 8 * hi * 32);
        M2_WAIT_MMA()
        // ---- h4: conj w_N^{n3 (k1 + 32 k2)}; A5[(k1, n3)][(c, k2)] -----------------------------------------------------
        if (ok) {
#pragma unroll 1
            for (int jj = 0; jj < 2; ++jj) {
                const int j = wg + 4 * jj;
                const int k2 = ((2 * (j & 1) + (t >> 6)) << 3) + (t & 7), k1 = ((j >> 1) << 3) + ((t >> 3) & 7);
                float2 g[4];
#pragma unroll
                for (int hi = 0; hi < 4; ++hi) g[hi] = g_next[hi];
                if (jj == 0) {
                    g_next[0] = __ldg(tn_h4 + 16 + 32);
#pragma unroll
                    for (int hi = 1; hi < 4; ++hi) g_next[hi] = __ldg(tn_h4 + 16 + 8 * hi * 32);
                }
                float re[32], im[32];
                load_tile(t_lane + j * 64, re, im);
                // rho^m = conj( w_N^{m k1} w_1024^{m k2} )
                const float2 rho = conjf(cmul(g[0], tw_at(1, k2)));
#pragma unroll
                for (int hi = 0; hi < 4; ++hi) {
                    float2 f = make_float2(1.f, 0.f);
                    if (hi > 0) f = conjf(cmul(g[hi], tw_at(8 * hi, k2)));
                    uint4 pr, pi;
                    geometric8_pack(re + 8 * hi, im + 8 * hi, f, rho, pr, pi);
                    const int mb = (k1 >> 3) * 4 + hi;
                    *reinterpret_cast<uint4*>(smem + OFF_A + a_off(mb, (k2 >> 3), k2 & 7, k1 & 7)) = pr;
                    *reinterpret_cast<uint4*>(smem + OFF_A + a_off(mb, 4 + (k2 >> 3), k2 & 7, k1 & 7)) = pi;
                }
            }
        }
        M2_STAGE_SYNC()
        // ---- S2': contract k2 with conj F ---------------------------------------------------------------------------
        if (issuer) {
            tc_fence_after();
#pragma unroll
            for (int jj = 0; jj < 2; ++jj)
#pragma unroll
                for (int s = 0; s < 4; ++s)
                    umma_f16(tmem + (wg + 4 * jj) * 64, smem_desc_sw128(s_base + OFF_A + (wg + 4 * jj) * 16384 + s * 2048, 8192, 1024),
                             smem_desc(s_base + OFF_BI + s * 256, 128, 1024), ID_MM, s > 0);
            umma_commit(bar_mma);
        }
        M2_WAIT_MMA()
        // ---- h5: conj w_1024^{n2 k1}; A6[(n2, n3)][(c, k1)] --------------------------------------------------------------
        if (ok) {
#pragma unroll 1
            for (int jj = 0; jj < 2; ++jj) {
                const int j = wg + 4 * jj;
                const int n3 = ((2 * (j & 1) + (t >> 6)) << 3) + (t & 7), k1 = ((j >> 1) << 3) + ((t >> 3) & 7);
                float re[32], im[32];
                load_tile(t_lane + j * 64, re, im);
                const float4* twr = tw4 + k1 * 17;
#pragma unroll
                for (int hi = 0; hi < 4; ++hi) {
                    uint32_t r_[4], i_[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const float4 w = twr[4 * hi + q];
                        cmul2_conj_pack(re[8 * hi + 2 * q], re[8 * hi + 2 * q + 1], im[8 * hi + 2 * q], im[8 * hi + 2 * q + 1], pk2(w.x, w.y),
                                        pk2(w.z, w.w), r_[q], i_[q]);
                    }
                    const int mb = hi * 4 + (n3 >> 3);
                    *reinterpret_cast<uint4*>(smem + OFF_A + a_off(mb, (k1 >> 3), k1 & 7, n3 & 7)) = make_uint4(r_[0], r_[1], r_[2], r_[3]);
                    *reinterpret_cast<uint4*>(smem + OFF_A + a_off(mb, 4 + (k1 >> 3), k1 & 7, n3 & 7)) = make_uint4(i_[0], i_[1], i_[2], i_[3]);
                }
            }
        }
        M2_STAGE_SYNC()
        // ---- S1': contract k1 with conj F, outputs n1 < 16 only (N = 32) ----------------------------------------------
        if (issuer) {
            tc_fence_after();
#pragma unroll
            for (int jj = 0; jj < 2; ++jj)
#pragma unroll
                for (int s = 0; s < 4; ++s)
                    umma_f16(tmem + (wg + 4 * jj) * 64, smem_desc_sw128(s_base + OFF_A + (wg + 4 * jj) * 16384 + s * 2048, 8192, 1024),
                             smem_desc(s_base + OFF_B6 + s * 256, 128, 1024), ID_S6, s > 0);
            umma_commit(bar_mma);
        }
        M2_WAIT_MMA()
        // ---- h6: round; stage both rows in the (now free) operand buffer; bulk store ------------------------------------
        if (ok) {
#pragma unroll 1
            for (int jj = 0; jj < 2; ++jj) {
                const int j = wg + 4 * jj;
                const int n2 = ((j >> 1) << 3) + (t & 7), n3 = ((2 * (j & 1) + (t >> 6)) << 3) + ((t >> 3) & 7);
                float v[32];
#pragma unroll
                for (int i = 0; i < 4; ++i) tmem_ld8(t_lane + j * 64 + 8 * i, v + 8 * i);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 4; ++i) tmem_ld_fence8(v + 8 * i);
                // staging = the TMA store's 64-byte-swizzled box image (rows of 32 n3; chunk index XOR bits 7..8 of the
                // address): a warp's 8 n2 x 4 n3 then hit 16 different banks instead of 4
                unsigned char* oa = smem + OFF_A + ((n2 * 64 + n3 * 2) ^ (((n2 >> 1) & 3) << 4));
#pragma unroll
                for (int n1 = 0; n1 < 16; ++n1) {
                    *reinterpret_cast<__nv_bfloat16*>(oa + n1 * 2048) = __float2bfloat16_rn(v[n1]);
                    *reinterpret_cast<__nv_bfloat16*>(oa + 32768 + n1 * 2048) = __float2bfloat16_rn(v[16 + n1]);
                }
            }
        }
        M2_STAGE_SYNC()
        if (tid == 0) {
            // y as [rows of 32 elements]: a batch row is 512 of them, a box 256
            const int ra = (b0 * H + h) * 512;
            tma_store_2d(&map_y, s_base + OFF_A, 0, ra);
            tma_store_2d(&map_y, s_base + OFF_A + 16384, 0, ra + 256);
            if (has_b) {
                const int rb = ((b0 + 1) * H + h) * 512;
                tma_store_2d(&map_y, s_base + OFF_A + 32768, 0, rb);
                tma_store_2d(&map_y, s_base + OFF_A + 49152, 0, rb + 256);
            }
            tma_store_commit();
            store_pending = true;
        }
    }
#undef M2_STAGE_SYNC
#undef M2_WAIT_MMA
    // ---- teardown ---------------------------------------------------------------------------------------------------
    cp_async_wait_all();
    if (tid == 0) {
        if (aborted) atomicExch(status, (int32_t)M2_ERR_TIMEOUT);
        tma_store_wait_all0();
    }
    tc_fence_before();
    __syncthreads();
    if (tid < 32) tmem_dealloc(tmem, 512);
}

// spectrum in the layout h3 reads: kfu[h][tile j][q = k3 / 2][lane t] = (re(2q), re(2q + 1), im(2q), im(2q + 1))
// for (k1, k2) = lane map of D3; plan order is [k1][k2][k3].
__global__ void relayout_spectrum3_kernel(const float2* __restrict__ kf, float4* __restrict__ kfu, long long total) {
    const long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x;   // over H * 8 * 16 * 128
    if (i >= total) return;
    const int t = (int)(i & 127), q = (int)((i >> 7) & 15), j = (int)((i >> 11) & 7);
    const long long h = i >> 14;
    const int k2 = ((2 * (j & 1) + (t >> 6)) << 3) + (t & 7), k1 = ((j >> 1) << 3) + ((t >> 3) & 7);
    const float2* src = kf + h * kN + (k1 * 32 + k2) * 32 + 2 * q;
    kfu[i] = make_float4(src[0].x, src[1].x, src[0].y, src[1].y);
}

// ---- host side ---------------------------------------------------------------------------------------------------

static uint16_t bf16_bits(double v) {
    float f = (float)v;
    uint32_t b;
    std::memcpy(&b, &f, 4);
    b += 0x7FFFu + ((b >> 16) & 1u);
    return (uint16_t)(b >> 16);
}
// K-major operand image of an [N][K] matrix (8 x 8 core matrices, K-adjacent 128 B apart)
static void put_kmajor(std::vector<uint16_t>& img, int K, int n, int k, double v) {
    const size_t byte = (size_t)(n / 8) * (K / 8) * 128 + (size_t)(k / 8) * 128 + (n % 8) * 16 + (k % 8) * 2;
    img[byte / 2] = bf16_bits(v);
}

bool covered(const m2_plan* pl) {
    return pl->dtype == M2_BF16 && pl->p == 3 && pl->dims[0] == 32 && pl->dims[1] == 32 && pl->dims[2] == 32;
}

cudaError_t create_tables(m2_plan* pl) {
    if (!covered(pl)) return cudaSuccess;
    const double sg = pl->sign >= 0 ? 1.0 : -1.0;
    std::vector<uint16_t> B1(2048), BF(4096), BI(4096), B6(2048);
    // complex 32-point DFT as a real matrix: in (a + ib), F = cs + i sn:  re = cs a - sn b,  im = sn a + cs b
    auto fill = [&](std::vector<uint16_t>& img, int K, int n_out, int n_in, bool inverse) {
        for (int co = 0; co < 2; ++co)
            for (int o = 0; o < n_out; ++o)
                for (int ci = 0; ci < 2; ++ci)
                    for (int i = 0; i < n_in; ++i) {
                        const double th = 2.0 * M_PI * ((o * i) % 32) / 32.0;
                        const double cs = std::cos(th), sn = (inverse ? -sg : sg) * std::sin(th);
                        const double v = co == 0 ? (ci == 0 ? cs : -sn) : (ci == 0 ? sn : cs);
                        put_kmajor(img, K, co * n_out + o, ci * n_in + i, v);
                    }
    };
    fill(B1, 32, 32, 16, false);   // [N = (c, k1) 64][K = (c, n1 < 16) 32]
    fill(BF, 64, 32, 32, false);   // [64][64]
    fill(BI, 64, 32, 32, true);    // conjugate
    fill(B6, 64, 16, 32, true);    // [N = (c, n1 < 16) 32][K = (c, k1) 64], conjugate
    std::vector<float> tw(32 * 17 * 4, 0.f), tn(32 * 32 * 2);
    for (int a = 0; a < 32; ++a)
        for (int b = 0; b < 32; ++b) {
            const double t1 = 2.0 * M_PI * ((a * b) % 1024) / 1024.0, t2 = 2.0 * M_PI * ((a * b) % kN) / (double)kN;
            tw[(a * 17 + b / 2) * 4 + (b & 1)] = (float)std::cos(t1);
            tw[(a * 17 + b / 2) * 4 + 2 + (b & 1)] = (float)(sg * std::sin(t1));
            tn[(a * 32 + b) * 2] = (float)std::cos(t2);
            tn[(a * 32 + b) * 2 + 1] = (float)(sg * std::sin(t2));
        }
    std::vector<unsigned char> blob(CONST_BYTES);
    std::memcpy(blob.data(), B1.data(), 4096);
    std::memcpy(blob.data() + 4096, BF.data(), 8192);
    std::memcpy(blob.data() + 12288, BI.data(), 8192);
    std::memcpy(blob.data() + 20480, B6.data(), 4096);
    std::memcpy(blob.data() + 24576, tw.data(), 8704);
    Tables* tb = new Tables();
    cudaError_t e = cudaMalloc(&tb->d_const, CONST_BYTES);
    if (e == cudaSuccess) e = cudaMemcpy(tb->d_const, blob.data(), CONST_BYTES, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMalloc(&tb->d_tn, tn.size() * sizeof(float));
    if (e == cudaSuccess) e = cudaMemcpy(tb->d_tn, tn.data(), tn.size() * sizeof(float), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(conv32k_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(conv32k_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    if (e != cudaSuccess) {
        if (tb->d_const) cudaFree(tb->d_const);
        if (tb->d_tn) cudaFree(tb->d_tn);
        delete tb;
        return e;
    }
    pl->umma = reinterpret_cast<m2_umma_tables*>(tb);
    return cudaSuccess;
}

void destroy_tables(m2_plan* pl) {
    if (!pl->umma || !covered(pl)) return;
    Tables* tb = reinterpret_cast<Tables*>(pl->umma);
    if (tb->d_const) cudaFree(tb->d_const);
    if (tb->d_tn) cudaFree(tb->d_tn);
    delete tb;
    pl->umma = nullptr;
}

cudaError_t relayout_spectrum(const m2_plan* pl, void* kf, int64_t H, cudaStream_t stream) {
    if (!pl->umma || !covered(pl) || H == 0) return cudaSuccess;
    const long long total = H * 16384;
    float4* kfu = reinterpret_cast<float4*>(static_cast<unsigned char*>(kf) + (size_t)H * kN * 8);
    relayout_spectrum3_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>((const float2*)kf, kfu, total);
    return cudaGetLastError();
}

int32_t conv_fwd(const m2_plan* pl, const void* x, const void* kf, void* y, int64_t B, int64_t H, int64_t n, int32_t mode,
                 cudaStream_t stream) {
    if (!pl->umma || !covered(pl)) return M2_ERR_UNSUPPORTED;
    if (mode != M2_CAUSAL || n != 16384) return M2_ERR_UNSUPPORTED;
    Tables* tb = reinterpret_cast<Tables*>(pl->umma);
    int dev = 0, sms = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const long long pairs = H * ((B + 1) / 2);
    const int grid = (int)(pairs < sms ? pairs : sms);
    const float4* kfu = reinterpret_cast<const float4*>(static_cast<const unsigned char*>(kf) + (size_t)H * kN * 8);
    alignas(64) CUtensorMap my;
    {
        const cuuint64_t gdim[2] = {32, (cuuint64_t)(B * H * 512)};
        const cuuint64_t gstr[1] = {64};
        const cuuint32_t box[2] = {32, 256};
        if (!tma_host::encode_sw64_bf16(&my, y, 2, gdim, gstr, box)) return M2_ERR_UNSUPPORTED;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, conv32k_kernel<0>, my, (const __nv_bfloat16*)x, kfu, (const uint4*)tb->d_const, (const float2*)tb->d_tn,
                           (int)B, (int)H, pl->d_status, 0, (float4*)nullptr) != cudaSuccess)
        return M2_ERR_CUDA;
    pl->last_kernel = "conv_umma_o3_32k";
    pl->launches += 1;
    return M2_OK;
}

// dk[h][i] = sum over the row pairs of channel h of the pair's first output row (fp32 sum of bf16 values, pairs in index order);
// 8 consecutive positions per thread
__global__ void wgrad_pair_sum_kernel(const __nv_bfloat16* __restrict__ rows, float* __restrict__ dk, int B, int H, long long total8) {
    const long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x;   // over H * 16384 / 8
    if (e >= total8) return;
    const long long h = e >> 11, i = (e & 2047) * 8;
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    for (int b = 0; b < B; b += 2) {
        const uint4 v = *reinterpret_cast<const uint4*>(rows + ((long long)b * H + h) * 16384 + i);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            acc[2 * q] += __uint_as_float(w[q] << 16);
            acc[2 * q + 1] += __uint_as_float(w[q] & 0xffff0000u);
        }
    }
    float4* dst = reinterpret_cast<float4*>(dk + h * 16384 + i);
    dst[0] = make_float4(acc[0], acc[1], acc[2], acc[3]);
    dst[1] = make_float4(acc[4], acc[5], acc[6], acc[7]);
}

// Kernel gradient on the tensor cores: with z_p = xa + i xb and w_p = ga + i gb for the row pairs p of a channel,
//   M^-1( conj(M z_p) (.) M w_p ) = (corr(xa, ga) + corr(xb, gb)) + i (corr(xa, gb) - corr(xb, ga)),
// both parts real sequences, so the first output row of the convolution kernel run on the g pairs with the spectrum
// conj(M z_p) / N is the pair's contribution to dk; the pairs of a channel are then added.
// ws: spectra [pairs][256 KB] | output rows [B][H][16384] bf16.
int64_t conv_wgrad_workspace_bytes(const m2_plan* pl, int64_t B, int64_t H) {
    if (!pl->umma || !covered(pl)) return 0;
    return H * ((B + 1) / 2) * 262144 + B * H * 16384 * 2;
}

int32_t conv_wgrad(const m2_plan* pl, const void* x, const void* g, float* dk, int64_t B, int64_t H, int64_t n, int32_t mode, void* ws,
                   cudaStream_t stream) {
    if (!pl->umma || !covered(pl)) return M2_ERR_UNSUPPORTED;
    if (mode != M2_CAUSAL || n != 16384 || B == 0) return M2_ERR_UNSUPPORTED;
    Tables* tb = reinterpret_cast<Tables*>(pl->umma);
    int dev = 0, sms = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const long long pairs = H * ((B + 1) / 2);
    if (pairs > 0x7ffffff) return M2_ERR_UNSUPPORTED;
    float4* spec = reinterpret_cast<float4*>(ws);
    __nv_bfloat16* rows = reinterpret_cast<__nv_bfloat16*>(static_cast<unsigned char*>(ws) + pairs * 262144);
    alignas(64) CUtensorMap my;
    {
        const cuuint64_t gdim[2] = {32, (cuuint64_t)(B * H * 512)};
        const cuuint64_t gstr[1] = {64};
        const cuuint32_t box[2] = {32, 256};
        if (!tma_host::encode_sw64_bf16(&my, rows, 2, gdim, gstr, box)) return M2_ERR_UNSUPPORTED;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(pairs < sms ? pairs : sms));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, conv32k_kernel<1>, my, (const __nv_bfloat16*)x, (const float4*)nullptr, (const uint4*)tb->d_const,
                           (const float2*)tb->d_tn, (int)B, (int)H, pl->d_status, 1, spec) != cudaSuccess)
        return M2_ERR_CUDA;
    if (cudaLaunchKernelEx(&cfg, conv32k_kernel<0>, my, (const __nv_bfloat16*)g, (const float4*)spec, (const uint4*)tb->d_const,
                           (const float2*)tb->d_tn, (int)B, (int)H, pl->d_status, 1, (float4*)nullptr) != cudaSuccess)
        return M2_ERR_CUDA;
    const long long total8 = H * 2048;
    wgrad_pair_sum_kernel<<<(unsigned)((total8 + 255) / 256), 256, 0, stream>>>(rows, dk, (int)B, (int)H, total8);
    if (cudaGetLastError() != cudaSuccess) return M2_ERR_CUDA;
    pl->last_kernel = "conv_wgrad_umma_o3_32k";
    pl->launches += 3;
    return M2_OK;
}

}  // namespace m2u3
