// Tensor-core Monarch convolution, order 2, N = 512 = 32 x 16, bf16 in / fp32 accumulate / bf16 out.
//
// y = Re( M^-1 ( k_f (.) M pad(x) ) ) with M = P L P^T R P = F_N (Eq. 2; Corollary "DFT is M").  Every
// Monarch stage is a dense contraction over one index digit and runs as a tcgen05 UMMA with the
// accumulator in TMEM; the stride permutations never move data on their own: they are the choice of
// which digit an operand's K dimension walks, expressed in the TMA box and in where the hand-off
// threads write the next operand.
//
// A "unit" is 8 batch entries of one channel (8 rows x 512).  128 TMEM lanes = 8 rows x 16 values of the
// digit that is NOT being contracted, so each thread owns whole complex numbers (re and im sit in
// different TMEM columns of its lane) and the twiddle / spectrum multiplies are thread-local fp32:
//
//   S1   D1[(r,n2)][(c,k1)]   = sum_n1  x[r][n1][n2] * F32[(c,k1)][n1]           A: M-major, 32B-swizzled (the TMA box as it lies)
//   h1   twiddle w_N^{n2 k1} (fp32), round to bf16, write A2[(r,k1)][(c,n2)]         M-major
//   S2   D2[(r,k1)][(c,k2)]   = sum_(c,n2) A2 * F16                              two M=128 halves
//   h2   multiply by k_f[h][k1][k2] (fp32, 1/N folded in), write A3[(r,k1)][(c,k2)]  K-major
//   S2'  D3[(r,k1)][(c,n2)]   = sum_(c,k2) A3 * conj(F16)
//   h3   conj twiddle, write A4[(r,n2)][(c,k1)]                                      M-major
//   S1'  D4[(r,n2)][n1]       = Re sum_(c,k1) A4 * conj(F32)
//   h4   round to bf16 and store y[r][n1*16 + n2] from registers (a warp instruction writes two full 32-byte sectors).
//
// One CTA per SM keeps the constant operands once and runs kGroups independent unit pipelines of 128
// threads (own mbarriers, 64 TMEM columns, 28 KB of shared memory each), so one pipeline's UMMA / TMA /
// barrier latency is covered by the others' fp32 work.  Units are handed out by a device-wide counter; the kernel is
// launched with programmatic stream serialization (set-up overlaps the previous kernel's tail).  All waits are bounded.
#include "conv_umma.h"

#include <cuda.h>
#include <cuda_bf16.h>

#include <cmath>
#include <cstdlib>
#include <cstring>
#include <vector>

#include "ptx_sm100.cuh"
#include "tma_host.h"

namespace m2u {

using namespace sm100;

constexpr int kRows = 8;             // rows (batch entries) per unit
constexpr int kGroups = 7;           // independent warpgroups per CTA, each running its own unit loop (72 registers per thread)
constexpr int kThreads = 128 * kGroups;
constexpr int kTmemColsPerGroup = 64;
constexpr int kTmemCols = 512;       // allocation must be a power of two >= kGroups * 64
// shared memory map (bytes): constants shared by the CTA, then one slice per warpgroup
constexpr int OFF_CONST = 0;         // B1 4096 | B2 2048 | B3 2048 | B4 4096 | twA 4096 | twB 4096
constexpr int CONST_BYTES = 20480;
constexpr int OFF_B1 = OFF_CONST, OFF_B2 = OFF_B1 + 4096, OFF_B3 = OFF_B2 + 2048, OFF_B4 = OFF_B3 + 2048;
constexpr int OFF_TWA = OFF_B4 + 4096, OFF_TWB = OFF_TWA + 4096;
constexpr int OFF_BAR = OFF_CONST + CONST_BYTES;   // per group: bar_x, bar_mma, bar_k, flag (32 B each, up to 16 groups); tmem ptr at +512
constexpr int OFF_GROUP = OFF_BAR + 1024;   // keeps every group slice 1024-byte aligned
constexpr int G_X = 0;               // one box [r][n1][16 n2], 32-byte swizzled   8192
constexpr int G_A = 8192;            // A2 / A3 / A4                        16384
constexpr int G_KF = 24576;          // spectrum row of the unit's channel  4096
constexpr int GROUP_BYTES = 28672;
constexpr int SMEM_BYTES = OFF_GROUP + kGroups * GROUP_BYTES;
static_assert(kGroups * 32 <= 512 && kGroups * kTmemColsPerGroup <= kTmemCols && SMEM_BYTES <= 232448, "per-CTA budgets");

struct Tables {
    void* d_const = nullptr;  // CONST_BYTES
    void* d_const_p = nullptr;  // constants of the row-pair kernel
    int* d_sched = nullptr;   // {next unit, pipelines finished}; zero between launches
};

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}


// Multiplies 8 complex values (re[], im[]) by 8 complex factors given as 4 float4 (c0, c1, s0, s1) -- the
// factors of two neighbouring values -- and packs real and imaginary parts as bf16 pairs.
__device__ __forceinline__ void cmul_pack8(const float* re, const float* im, const float4* w, uint4& pr, uint4& pi) {
    uint32_t r_[4], i_[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const uint64_t a2 = pk2(re[2 * q], re[2 * q + 1]), b2 = pk2(im[2 * q], im[2 * q + 1]);
        const uint64_t c2 = pk2(w[q].x, w[q].y), s2 = pk2(w[q].z, w[q].w);
        const uint64_t r2 = fma2(sub2(0ull, b2), s2, mul2(a2, c2));   // a c - b s
        const uint64_t i2 = fma2(b2, c2, mul2(a2, s2));               // a s + b c
        float x0, x1, y0, y1;
        upk2(r2, x0, x1);
        upk2(i2, y0, y1);
        r_[q] = pack_bf16(x0, x1);
        i_[q] = pack_bf16(y0, y1);
    }
    pr = make_uint4(r_[0], r_[1], r_[2], r_[3]);
    pi = make_uint4(i_[0], i_[1], i_[2], i_[3]);
}

// block-wide barrier among the 128 threads of one warpgroup that also ORs a predicate
__device__ __forceinline__ bool group_sync_or(int wg, bool pred, volatile int* flag) {
    if (pred) *flag = 1;
    asm volatile("bar.sync %0, 128;" ::"r"(wg + 1) : "memory");
    return *flag != 0;
}

__global__ void __launch_bounds__(kThreads, 1)
conv512_kernel(const __grid_constant__ CUtensorMap map_x, __nv_bfloat16* __restrict__ y,
               const float4* __restrict__ kfu, const uint4* __restrict__ consts, int B, int H, int n,
               int32_t* __restrict__ status, int* __restrict__ sched, int kf_group) {
    extern __shared__ __align__(1024) unsigned char smem_all[];
    const int wg = threadIdx.x >> 7;          // warpgroup = independent unit pipeline
    const int tid = threadIdx.x & 127;
    const int warp = tid >> 5;                // warp within the group = TMEM lane quarter
    // the thread that issues this pipeline's UMMAs and copies; its warp differs from group to group so that
    // the extra work spreads over the SM's four schedulers
    const bool leader = tid == 32 * (wg & 3);
    const uint32_t s_all = smem_u32(smem_all);
    unsigned char* smem = smem_all + OFF_GROUP + wg * GROUP_BYTES;   // this group's slice
    const uint32_t s_base = s_all + OFF_GROUP + wg * GROUP_BYTES;
    const uint32_t bar_x = s_all + OFF_BAR + wg * 32, bar_mma = bar_x + 8, bar_k = bar_x + 16;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_all + OFF_BAR + wg * 32 + 24);
    volatile int* next_slot = reinterpret_cast<volatile int*>(smem_all + OFF_BAR + wg * 32 + 28);
    const uint32_t s_tptr = s_all + OFF_BAR + 512;

    const int bgroups0 = (B + kRows - 1) / kRows;
    const int units0 = H * bgroups0;
    int u = blockIdx.x * kGroups + wg;
    const int ustride = gridDim.x * kGroups;
    if (leader) {
        mbar_init(bar_x, 1);
        mbar_init(bar_mma, 1);
        mbar_init(bar_k, 1);
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tensormap(&map_x);
    }
    // Programmatic dependent launch: the next kernel on the stream may start its CTAs as this grid's CTAs leave
    // their SMs; everything above the wait below touches only plan-owned constants and this CTA's own resources.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    bool x_pending = false, k_pending = false;
    // constants -> shared memory
    {
        uint4* dst = reinterpret_cast<uint4*>(smem_all + OFF_CONST);
        for (int i = threadIdx.x; i < CONST_BYTES / 16; i += kThreads) dst[i] = consts[i];
    }
    if (threadIdx.x < 32) tmem_alloc(s_tptr, kTmemCols);
    // everything the stream ran before this kernel (the producer of x and of the spectrum, the previous launch's
    // reset of the scheduler words, readers of y) is complete and visible from here on
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (leader && u < units0) {   // first loads
        mbar_expect_tx(bar_x, 8192);
        tma_load_4d(s_base + G_X, &map_x, 0, 0, u % H, (u / H) * kRows, bar_x);
        x_pending = true;
        mbar_expect_tx(bar_k, 4096);
        bulk_load(s_base + G_KF, kfu + (size_t)((u % H) / kf_group) * 256, 4096, bar_k);
        k_pending = true;
    }
    fence_proxy_async();   // the constant matrices are read by the async proxy (UMMA)
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_cta = *reinterpret_cast<volatile uint32_t*>(smem_all + OFF_BAR + 512);
    const uint32_t tmem = tmem_cta + wg * kTmemColsPerGroup;
    const uint32_t t_lane = tmem + ((uint32_t)(warp * 32) << 16);   // this warp's 32 lanes
    const uint32_t T1 = 0, T2 = 0;   // every stage's accumulator reuses the same 64 columns

    const int units = units0;
    constexpr uint32_t ID_S1 = instr_desc_bf16(128, 64, true, false);
    constexpr uint32_t ID_S2 = instr_desc_bf16(128, 32, true, false);
    constexpr uint32_t ID_S2I = instr_desc_bf16(128, 32, false, false);
    constexpr uint32_t ID_S1I = instr_desc_bf16(128, 32, true, false);
    const int n1_valid = n / 16;
    const int k1steps = (n1_valid + 15) / 16;   // causal input: digits n1 >= n/16 are zero -> skipped

    uint32_t ph_x = 0, ph_m = 0, ph_k = 0;
    bool ok = true, aborted = false;
    // Units beyond the first two are handed out by a device-wide counter (sched[0]): pipelines that finish early take more.
    // The last pipeline to leave (sched[1] counts them) zeroes both words for the next launch on this plan.
    int un = u + ustride;   // the second unit is static too
    int un2 = units;        // thread 0: the unit after next, claimed one whole unit ahead so the atomic's latency is never waited for
    while (u < units) {
        const int h = u % H;
        const int b0 = (u / H) * kRows;
        // ---- S1 ---------------------------------------------------------------------------------
        if (leader) {
            ok = mbar_wait(bar_x, ph_x);
            x_pending = false;
            if (ok) {
                tc_fence_after();
#pragma unroll 1
                for (int s = 0; s < k1steps; ++s)
                    umma_f16(tmem + T1, smem_desc_sw32(s_base + G_X + s * 512, 1024, 256),
                             smem_desc(s_all + OFF_B1 + s * 256, 128, 512), ID_S1, s > 0);
                umma_commit(bar_mma);
            }
        }
        ph_x ^= 1;
        // ---- h1: twiddle, A2 ---------------------------------------------------------------------
        ok = ok && mbar_wait(bar_mma, ph_m);
        ph_m ^= 1;
        tc_fence_after();
        if (leader) un2 = 2 * ustride + atomicAdd(sched, 1);   // consumed at the end of this unit
        if (leader && ok && un < units) {   // the x tile is free: fetch the next unit's
            mbar_expect_tx(bar_x, 8192);
            tma_load_4d(s_base + G_X, &map_x, 0, 0, un % H, (un / H) * kRows, bar_x);
            x_pending = true;
        }
        if (ok) {
            const int r = tid >> 4, n2 = tid & 15, n2hi = n2 >> 3, n2lo = n2 & 7;   // lane = r * 16 + n2: the row order of the input box
            const float4* twA = reinterpret_cast<const float4*>(smem_all + OFF_TWA) + n2;
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {   // two batches of 16 complex values keep the register count down
                float re[16], im[16];
#pragma unroll
                for (int jj = 0; jj < 2; ++jj) {
                    tmem_ld8(t_lane + T1 + 16 * hh + 8 * jj, re + 8 * jj);
                    tmem_ld8(t_lane + T1 + 32 + 16 * hh + 8 * jj, im + 8 * jj);
                }
                tmem_ld_wait();
#pragma unroll
                for (int jj = 0; jj < 2; ++jj) {
                    tmem_ld_fence8(re + 8 * jj);
                    tmem_ld_fence8(im + 8 * jj);
                }
#pragma unroll
                for (int jj = 0; jj < 2; ++jj) {
                    const int j = 2 * hh + jj;
                    float4 w[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) w[q] = twA[(4 * j + q) * 16];
                    uint4 pr, pi;
                    cmul_pack8(re + 8 * jj, im + 8 * jj, w, pr, pi);
                    unsigned char* base = smem + G_A + (r * 4 + j) * 512 + n2lo * 16;
                    *reinterpret_cast<uint4*>(base + (0 + n2hi) * 128) = pr;
                    *reinterpret_cast<uint4*>(base + (2 + n2hi) * 128) = pi;
                }
            }
        }
        fence_proxy_async();
        tc_fence_before();
        if (group_sync_or(wg, !ok, abort_flag)) {
            aborted = true;
            break;
        }
        // ---- S2 ---------------------------------------------------------------------------------
        if (leader) {
            tc_fence_after();
#pragma unroll
            for (int hf = 0; hf < 2; ++hf)
#pragma unroll
                for (int s = 0; s < 2; ++s)
                    umma_f16(tmem + T2 + hf * 32, smem_desc(s_base + G_A + hf * 8192 + s * 256, 128, 512),
                             smem_desc(s_all + OFF_B2 + s * 256, 128, 512), ID_S2, s > 0);
            umma_commit(bar_mma);
        }
        // ---- h2: spectrum multiply, A3 -------------------------------------------------------------
        ok = mbar_wait(bar_k, ph_k);          // the channel's spectrum row has landed
        ph_k ^= 1;
        if (leader) k_pending = false;
        ok = ok && mbar_wait(bar_mma, ph_m);
        ph_m ^= 1;
        tc_fence_after();
        if (ok) {
            const int k1 = tid & 31;
            const float4* kfs = reinterpret_cast<const float4*>(smem + G_KF) + k1;
            // both row halves (hf) of a thread share k1, hence the spectrum values: load them once per chunk
#pragma unroll
            for (int g = 0; g < 2; ++g) {
                float re[16], im[16];
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    tmem_ld8(t_lane + T2 + hf * 32 + 8 * g, re + 8 * hf);
                    tmem_ld8(t_lane + T2 + hf * 32 + 16 + 8 * g, im + 8 * hf);
                }
                float4 w[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) w[q] = kfs[(g * 4 + q) * 32];
                tmem_ld_wait();
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    tmem_ld_fence8(re + 8 * hf);
                    tmem_ld_fence8(im + 8 * hf);
                }
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    const int m = hf * 128 + tid;
                    unsigned char* rowp = smem + G_A + (m >> 3) * 512 + (m & 7) * 16;
                    uint4 pr, pi;
                    cmul_pack8(re + 8 * hf, im + 8 * hf, w, pr, pi);
                    *reinterpret_cast<uint4*>(rowp + g * 128) = pr;
                    *reinterpret_cast<uint4*>(rowp + (2 + g) * 128) = pi;
                }
            }
        }
        fence_proxy_async();
        tc_fence_before();
        if (group_sync_or(wg, !ok, abort_flag)) {
            aborted = true;
            break;
        }
        // ---- S2' --------------------------------------------------------------------------------
        if (leader) {
            tc_fence_after();
#pragma unroll
            for (int hf = 0; hf < 2; ++hf)
#pragma unroll
                for (int s = 0; s < 2; ++s)
                    umma_f16(tmem + T1 + hf * 32, smem_desc(s_base + G_A + hf * 8192 + s * 256, 128, 512),
                             smem_desc(s_all + OFF_B3 + s * 256, 128, 512), ID_S2I, s > 0);
            umma_commit(bar_mma);
            if (un < units) {                 // the spectrum tile is free: fetch the next unit's
                mbar_expect_tx(bar_k, 4096);
                bulk_load(s_base + G_KF, kfu + (size_t)((un % H) / kf_group) * 256, 4096, bar_k);
                k_pending = true;
            }
        }
        // ---- h3: conjugate twiddle, A4 --------------------------------------------------------------
        ok = mbar_wait(bar_mma, ph_m);
        ph_m ^= 1;
        tc_fence_after();
        if (ok) {
            const int k1 = tid & 31;
            const float4* twB = reinterpret_cast<const float4*>(smem_all + OFF_TWB) + k1;
#pragma unroll
            for (int g = 0; g < 2; ++g) {   // the twiddles depend on (k1, n2) only: shared by both row halves
                float re[16], im[16];
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    tmem_ld8(t_lane + T1 + hf * 32 + 8 * g, re + 8 * hf);
                    tmem_ld8(t_lane + T1 + hf * 32 + 16 + 8 * g, im + 8 * hf);
                }
                float4 w[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) w[q] = twB[(4 * g + q) * 32];
                tmem_ld_wait();
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    tmem_ld_fence8(re + 8 * hf);
                    tmem_ld_fence8(im + 8 * hf);
                }
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    const int r = hf * 4 + (tid >> 5);
                    uint4 pr, pi;
                    cmul_pack8(re + 8 * hf, im + 8 * hf, w, pr, pi);
                    unsigned char* base = smem + G_A + (r * 2 + g) * 1024 + (k1 >> 3) * 128 + (k1 & 7) * 16;
                    *reinterpret_cast<uint4*>(base) = pr;
                    *reinterpret_cast<uint4*>(base + 512) = pi;
                }
            }
        }
        fence_proxy_async();
        tc_fence_before();
        if (group_sync_or(wg, !ok, abort_flag)) {
            aborted = true;
            break;
        }
        // ---- S1' --------------------------------------------------------------------------------
        if (leader) {
            tc_fence_after();
#pragma unroll
            for (int s = 0; s < 4; ++s)
                umma_f16(tmem + T2, smem_desc(s_base + G_A + s * 256, 128, 1024),
                         smem_desc(s_all + OFF_B4 + s * 256, 128, 1024), ID_S1I, s > 0);
            umma_commit(bar_mma);
        }
        // ---- h4: round and store: lane (r, n2) holds y[r][n1*16 + n2] for all n1; a warp writes two full
        //      32-byte sectors per instruction --------------------------------------------------------
        ok = mbar_wait(bar_mma, ph_m);
        ph_m ^= 1;
        tc_fence_after();
        if (ok) {
            const int r = tid >> 4, n2 = tid & 15;
            float v[32];
#pragma unroll
            for (int g = 0; g < 4; ++g) tmem_ld8(t_lane + T2 + 8 * g, v + 8 * g);
            tmem_ld_wait();
#pragma unroll
            for (int g = 0; g < 4; ++g) tmem_ld_fence8(v + 8 * g);
            if (b0 + r < B) {
                __nv_bfloat16* yr = y + ((size_t)(b0 + r) * H + h) * n + n2;
#pragma unroll
                for (int i = 0; i < 32; ++i)
                    if (i < n1_valid) yr[i * 16] = __float2bfloat16_rn(v[i]);
            }
        }
        if (leader) *next_slot = un2;
        tc_fence_before();
        if (group_sync_or(wg, !ok, abort_flag)) {
            aborted = true;
            break;
        }
        u = un;
        un = *next_slot;   // written by thread 0 before the barrier above
    }
    // ---- teardown: nothing of ours may still be in flight when the TMEM and the CTA go away ----------
    if (leader) {
        if (aborted) atomicExch(status, (int32_t)M2_ERR_TIMEOUT);
        if (x_pending) mbar_wait(bar_x, ph_x);
        if (k_pending) mbar_wait(bar_k, ph_k);
        __threadfence();
        if (atomicAdd(sched + 1, 1) == ustride - 1) {   // last pipeline out: reset the scheduler words
            sched[0] = 0;
            sched[1] = 0;
            __threadfence();
        }
    }
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x < 32) tmem_dealloc(tmem_cta, kTmemCols);
}

// ---- the same pipeline on PAIRS of batch rows ------------------------------------------------------------------------
//
// k is real, so two batch rows of one channel ride as the real and the imaginary part of one complex row:
// F^-1(k_f (.) F(xa + i xb)) = ya + i yb.  A unit is then 16 batch rows = 8 complex rows: the first stage contracts
// K = (re | im) x n1 = 64 and the last one produces both parts (N = 64), everything between is unchanged, so the three
// fp32 hand-offs between the stages are paid once per two rows.  6 pipelines of 32 KB (the spectrum values come straight
// from global memory / L2, requested before the accumulator wait).
constexpr int kGroupsP = 6;
constexpr int kThreadsP = 128 * kGroupsP;
constexpr int P_OFF_B1 = 0, P_OFF_B2 = 8192, P_OFF_B3 = 10240, P_OFF_B4 = 12288, P_OFF_TWA = 20480, P_OFF_TWB = 24576;
constexpr int P_CONST_BYTES = 28672;
constexpr int P_OFF_BAR = P_CONST_BYTES;          // per group 32 B; tmem ptr at +512
constexpr int P_OFF_GROUP = P_OFF_BAR + 1024;
constexpr int P_G_X = 0;                          // re tile 8192 | im tile 8192 (one box [r][n1][16 n2] each, 32-byte swizzled)
constexpr int P_G_A = 16384;                      // A2 / A3 / A4   16384
constexpr int P_GROUP_BYTES = 32768;
constexpr int P_SMEM_BYTES = P_OFF_GROUP + kGroupsP * P_GROUP_BYTES;
static_assert(kGroupsP * 32 <= 512 && kGroupsP * kTmemColsPerGroup <= kTmemCols && P_SMEM_BYTES <= 232448 && P_OFF_GROUP % 1024 == 0,
              "per-CTA budgets");

//
// GATE (the M2 block's sequence mixer, Eq. 2 with the depthwise gate of Sec. 5.1): the rows leave multiplied by the width-3
// depthwise convolution of the INPUT row, y[t] <- y[t] (w[h][0] x[t-1] + w[h][1] x[t] + w[h][2] x[t+1]), zero padded at both ends
// of the row.  xg = the input rows again ([B][H][512], read from L2 in the last hand-off: the unit's tile in shared memory has
// long been replaced by the next unit's), w_gate = [H][3] fp32.  The output may be written over the input (map_y over the same rows
// as map_x): a unit's rows are read for the last time before its stores are issued, and no other unit touches them.  The gate may
// also be taken from other rows than the convolution's input (xg need not be what map_x covers), and vh != nullptr names rows
// [B][H][512] that are added after the gate: y <- y gate + vh (the gated M2-BERT sequence mixer: V (.) conv(k, Q (.) K) + conv(k_res, x)).
//
// HEADS (MODE 2; the core of the M2 Hyena layer with heads of dh = 16 channels, GPT appendix): a unit is one (batch entry b, channel
// hj = head * 16 + j) and its 16 rows are the sequences X2[b][head * 16 + i][t] V[b][hj][t], i = 0 .. 15, of the head's outer
// product -- formed in shared memory from the TMA-loaded X2 rows (map_x boxes span 8 CHANNELS of one batch entry) and the V row
// (vh) before the first stage -- and what leaves is their causal convolution with the head's kernel contracted with X1 (xg):
//   y[b][hj][t] = sum_i X1[b][head * 16 + i][t] (k_head * (X2_i V_j))[t],   t < n <= 256.
// The d_h-times larger tensor of the outer product and of its convolution never exists in memory.  kf_group = dh selects the
// head's spectrum row.  Nothing is staged or stored by TMA in this mode: a unit's result is one row of n values.
template <int MODE>
__global__ void __launch_bounds__(kThreadsP, 1)
conv512p_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_y, __nv_bfloat16* __restrict__ y,
               const float4* __restrict__ kfu, const uint4* __restrict__ consts, int B, int H, int n,
               int32_t* __restrict__ status, int* __restrict__ sched, int selftest, int kf_group,
               const __nv_bfloat16* __restrict__ xg, const float* __restrict__ w_gate, const __nv_bfloat16* __restrict__ vh) {
    constexpr bool GATE = MODE == 1, HEADS = MODE == 2;
    extern __shared__ __align__(1024) unsigned char smem_all[];
    const int wg = threadIdx.x >> 7;          // warpgroup = independent unit pipeline
    const int tid = threadIdx.x & 127;
    const int warp = tid >> 5;                // warp within the group = TMEM lane quarter
    // the thread that issues this pipeline's UMMAs and copies; its warp differs from group to group so that
    // the extra work spreads over the SM's four schedulers
    const bool leader = tid == 32 * (wg & 3);
    // a second issuing thread, two schedulers further on, takes the second half of the stages that have two independent halves
    const bool leader2 = tid == 32 * ((wg + 2) & 3);
    const uint32_t s_all = smem_u32(smem_all);
    unsigned char* smem = smem_all + P_OFF_GROUP + wg * P_GROUP_BYTES;   // this group's slice
    const uint32_t s_base = s_all + P_OFF_GROUP + wg * P_GROUP_BYTES;
    const uint32_t bar_x = s_all + P_OFF_BAR + wg * 32, bar_mma = bar_x + 8;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_all + P_OFF_BAR + wg * 32 + 24);
    volatile int* next_slot = reinterpret_cast<volatile int*>(smem_all + P_OFF_BAR + wg * 32 + 28);
    const uint32_t s_tptr = s_all + P_OFF_BAR + 512;

    const int bgroups0 = HEADS ? B : (B + 2 * kRows - 1) / (2 * kRows);   // 16 batch rows = 8 complex rows per unit (HEADS: 16 channels of one entry)
    const int units0 = H * bgroups0;
    // pipeline-major numbering: a partial last round of units spreads over all CTAs instead of filling the first ones
    int u = wg * gridDim.x + blockIdx.x;
    const int ustride = gridDim.x * kGroupsP;
    if (leader) {
        mbar_init(bar_x, 1);
        mbar_init(bar_mma, 2);   // both issuing threads commit in every stage
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tensormap(&map_x);
        prefetch_tensormap(&map_y);
        // Pull this pipeline's first input tiles towards L2 now, while the previous kernel on the stream is still finishing:
        // a prefetch returns no data, and L2 is where that kernel's writes land, so the copies issued after the wait below
        // see them whatever it wrote.
        if (!selftest && u < units0) {
            if (HEADS) {
                const int hb = ((u % H) / kf_group) * kf_group, bb = u / H;
                tma_prefetch_4d(&map_x, 0, 0, hb, bb);
                tma_prefetch_4d(&map_x, 0, 0, hb + kRows, bb);
            } else {
                const int hh = u % H, bb = (u / H) * 2 * kRows;
                tma_prefetch_4d(&map_x, 0, 0, hh, bb);
                tma_prefetch_4d(&map_x, 0, 0, hh, bb + kRows);
            }
        }
    }
    // Programmatic dependent launch: the next kernel on the stream may start its CTAs as this grid's CTAs leave
    // their SMs; everything above the wait below touches only plan-owned constants and this CTA's own resources.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    bool x_pending = false;
    // Self-test of the bounded waits (selftest != 0): no input copy is ever issued and every wait gives up after a few polls,
    // so each pipeline's first wait -- on a barrier nothing will arrive on, with nothing in flight -- runs out and the pipeline
    // leaves through the abort path below exactly as it would after a lost copy.
    const uint32_t wlim = selftest ? 16u : (1u << 22);
    // constants -> shared memory
    {
        uint4* dst = reinterpret_cast<uint4*>(smem_all);
        for (int i = threadIdx.x; i < P_CONST_BYTES / 16; i += kThreadsP) dst[i] = consts[i];
    }
    if (threadIdx.x < 32) tmem_alloc(s_tptr, kTmemCols);
    // everything the stream ran before this kernel (the producer of x and of the spectrum, the previous launch's
    // reset of the scheduler words, readers of y) is complete and visible from here on
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // rows b0 .. b0+7 are the real parts and rows b0+8 .. b0+15 the imaginary parts of the unit's 8 complex rows (boxes
    // past the end of the batch read zeros).  A box is [8 rows][32 n1][16 n2] with 32-byte rows, 32-byte swizzled: as it lies
    // it is the M-major operand of S1 with M = (row, n2) -- 16-element M blocks 1 KB apart, groups of 8 n1 256 B apart.
    auto load_unit = [&](int v) {
        if (selftest) return;
        mbar_expect_tx(bar_x, 16384);
        if (HEADS) {   // the head's 16 X2 rows of batch entry v / H: two boxes of 8 channels
            const int hb = ((v % H) / kf_group) * kf_group, bb = v / H;
            tma_load_4d(s_base + P_G_X, &map_x, 0, 0, hb, bb, bar_x);
            tma_load_4d(s_base + P_G_X + 8192, &map_x, 0, 0, hb + kRows, bb, bar_x);
        } else {
            const int hh = v % H, bb = (v / H) * 2 * kRows;
            tma_load_4d(s_base + P_G_X, &map_x, 0, 0, hh, bb, bar_x);
            tma_load_4d(s_base + P_G_X + 8192, &map_x, 0, 0, hh, bb + kRows, bar_x);
        }
        x_pending = true;
    };
    if (leader && u < units0) {   // first loads
        load_unit(u);
    }
    fence_proxy_async();   // the constant matrices are read by the async proxy (UMMA)
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_cta = *reinterpret_cast<volatile uint32_t*>(smem_all + P_OFF_BAR + 512);
    const uint32_t tmem = tmem_cta + wg * kTmemColsPerGroup;
    const float4* kfu_k1 = kfu + (threadIdx.x & 31);
    const uint32_t t_lane = tmem + ((uint32_t)(warp * 32) << 16);   // this warp's 32 lanes
    const uint32_t T1 = 0, T2 = 0;   // every stage's accumulator reuses the same 64 columns

    const int units = units0;
    constexpr uint32_t ID_S1 = instr_desc_bf16(128, 64, true, false);
    constexpr uint32_t ID_S2 = instr_desc_bf16(128, 32, true, false);
    constexpr uint32_t ID_S2I = instr_desc_bf16(128, 32, false, false);
    constexpr uint32_t ID_S1I = instr_desc_bf16(64, 64, false, true);
    const int n1_valid = n / 16;
    const int k1steps = (n1_valid + 15) / 16;   // causal input: digits n1 >= n/16 are zero -> skipped

    uint32_t ph_x = 0, ph_m = 0;
    bool ok = true, aborted = false;
    // Units beyond the first two are handed out by a device-wide counter (sched[0]): pipelines that finish early take more.
    // The last pipeline to leave (sched[1] counts them) zeroes both words for the next launch on this plan.
    int un = u + ustride;   // the second unit is static too
    int un2 = units;        // thread 0: the unit after next, claimed one whole unit ahead so the atomic's latency is never waited for
    while (u < units) {
        const int h = u % H;
        const int b0 = HEADS ? u / H : (u / H) * 2 * kRows;
        if (HEADS) {
            // ---- h0: the X2 rows have landed; every row times the V row of this unit's channel, in place.  Thread (row r, n1) owns
            //      the 32-byte run of 16 positions t = 16 n1 .. of its row in both boxes (rows i = r and i = 8 + r). ----
            const int r = tid >> 4, n1 = tid & 15, sw = (n1 >> 2) & 1;
            uint4 va = make_uint4(0u, 0u, 0u, 0u), vb = va;
            if (16 * n1 < n) {   // (asked for before the wait for the tile: the two latencies overlap)
                const uint4* vrow = reinterpret_cast<const uint4*>(vh + ((size_t)b0 * H + h) * n + 16 * n1);
                va = __ldg(vrow);
                vb = __ldg(vrow + 1);
            }
            ok = mbar_wait(bar_x, ph_x, wlim);
            x_pending = false;
            if (ok) {
                if (16 * n1 < n) {
                    const uint32_t vw[8] = {va.x, va.y, va.z, va.w, vb.x, vb.y, vb.z, vb.w};
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        unsigned char* row = smem + P_G_X + c * 8192 + r * 1024 + n1 * 32;
#pragma unroll
                        for (int q = 0; q < 2; ++q) {   // q = half of the run: positions 8 q .. 8 q + 7
                            uint4* cell = reinterpret_cast<uint4*>(row + ((q ^ sw) << 4));
                            const uint4 xv = *cell;
                            const uint32_t xw[4] = {xv.x, xv.y, xv.z, xv.w};
                            uint32_t o[4];
#pragma unroll
                            for (int k = 0; k < 4; ++k)
                                o[k] = pack_bf16(__uint_as_float(xw[k] << 16) * __uint_as_float(vw[4 * q + k] << 16),
                                                 __uint_as_float(xw[k] & 0xffff0000u) * __uint_as_float(vw[4 * q + k] & 0xffff0000u));
                            *cell = make_uint4(o[0], o[1], o[2], o[3]);
                        }
                    }
                }
            }
            fence_proxy_async();   // the products are read by the tensor core
            if (group_sync_or(wg, !ok, abort_flag)) {
                aborted = true;
                break;
            }
        }
        // ---- S1 ---------------------------------------------------------------------------------
        if (leader) {
            if (!HEADS) ok = mbar_wait(bar_x, ph_x, wlim);
            x_pending = false;
            if (ok) {
                tc_fence_after();
#pragma unroll
                for (int c = 0; c < 2; ++c)   // K = (re | im part of the input) x n1
#pragma unroll 1
                    for (int s = 0; s < k1steps; ++s)
                        umma_f16(tmem + T1, smem_desc_sw32(s_base + P_G_X + c * 8192 + s * 512, 1024, 256),
                                 smem_desc(s_all + P_OFF_B1 + (2 * c + s) * 256, 128, 1024), ID_S1, (c | s) > 0);
                // S1 does not touch the operand buffer, hand-off 1 (which waits for this commit) overwrites it: the previous
                // unit's output stores must have read their staging area by then, and they do so while S1 runs
                tma_store_wait_read0();
                umma_commit(bar_mma);
            }
        }
        if (leader2) umma_commit(bar_mma);   // (nothing of its own to track in this stage)
        ph_x ^= 1;
        // ---- h1: twiddle, A2 ---------------------------------------------------------------------
        ok = ok && mbar_wait(bar_mma, ph_m, wlim);
        ph_m ^= 1;
        tc_fence_after();
        if (leader) un2 = 2 * ustride + atomicAdd(sched, 1);   // consumed at the end of this unit
        if (leader && ok && un < units) {   // the x tile is free: fetch the next unit's
            load_unit(un);
        }
        if (ok) {
            const int r = tid >> 4, n2 = tid & 15, n2hi = n2 >> 3, n2lo = n2 & 7;   // lane = r * 16 + n2: the row order of the input boxes
            const float4* twA = reinterpret_cast<const float4*>(smem_all + P_OFF_TWA) + n2;
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {   // two batches of 16 complex values keep the register count down
                float re[16], im[16];
#pragma unroll
                for (int jj = 0; jj < 2; ++jj) {
                    tmem_ld8(t_lane + T1 + 16 * hh + 8 * jj, re + 8 * jj);
                    tmem_ld8(t_lane + T1 + 32 + 16 * hh + 8 * jj, im + 8 * jj);
                }
                tmem_ld_wait();
#pragma unroll
                for (int jj = 0; jj < 2; ++jj) {
                    tmem_ld_fence8(re + 8 * jj);
                    tmem_ld_fence8(im + 8 * jj);
                }
#pragma unroll
                for (int jj = 0; jj < 2; ++jj) {
                    const int j = 2 * hh + jj;
                    float4 w[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) w[q] = twA[(4 * j + q) * 16];
                    uint4 pr, pi;
                    cmul_pack8(re + 8 * jj, im + 8 * jj, w, pr, pi);
                    unsigned char* base = smem + P_G_A + (r * 4 + j) * 512 + n2lo * 16;
                    *reinterpret_cast<uint4*>(base + (0 + n2hi) * 128) = pr;
                    *reinterpret_cast<uint4*>(base + (2 + n2hi) * 128) = pi;
                }
            }
        }
        fence_proxy_async();
        tc_fence_before();
        if (group_sync_or(wg, !ok, abort_flag)) {
            aborted = true;
            break;
        }
        // ---- S2 ---------------------------------------------------------------------------------
        if (leader || leader2) {
            tc_fence_after();
            const int hf = leader ? 0 : 1;
#pragma unroll
            for (int s = 0; s < 2; ++s)
                umma_f16(tmem + T2 + hf * 32, smem_desc(s_base + P_G_A + hf * 8192 + s * 256, 128, 512),
                         smem_desc(s_all + P_OFF_B2 + s * 256, 128, 512), ID_S2, s > 0);
            umma_commit(bar_mma);
        }
        // ---- h2: spectrum multiply, A3 -------------------------------------------------------------
        float4 kw[8];   // this thread's 16 spectrum values (k1 fixed), requested before the accumulator is waited for
#pragma unroll
        for (int q = 0; q < 8; ++q) kw[q] = __ldg(kfu_k1 + (size_t)(h / kf_group) * 256 + q * 32);
        ok = mbar_wait(bar_mma, ph_m, wlim);
        ph_m ^= 1;
        tc_fence_after();
        if (ok) {
            // both row halves (hf) of a thread share k1, hence the spectrum values
#pragma unroll
            for (int g = 0; g < 2; ++g) {
                float re[16], im[16];
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    tmem_ld8(t_lane + T2 + hf * 32 + 8 * g, re + 8 * hf);
                    tmem_ld8(t_lane + T2 + hf * 32 + 16 + 8 * g, im + 8 * hf);
                }
                float4 w[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) w[q] = kw[g * 4 + q];
                tmem_ld_wait();
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    tmem_ld_fence8(re + 8 * hf);
                    tmem_ld_fence8(im + 8 * hf);
                }
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    const int m = hf * 128 + tid;
                    unsigned char* rowp = smem + P_G_A + (m >> 3) * 512 + (m & 7) * 16;
                    uint4 pr, pi;
                    cmul_pack8(re + 8 * hf, im + 8 * hf, w, pr, pi);
                    *reinterpret_cast<uint4*>(rowp + g * 128) = pr;
                    *reinterpret_cast<uint4*>(rowp + (2 + g) * 128) = pi;
                }
            }
        }
        fence_proxy_async();
        tc_fence_before();
        if (group_sync_or(wg, !ok, abort_flag)) {
            aborted = true;
            break;
        }
        // ---- S2' --------------------------------------------------------------------------------
        if (leader || leader2) {
            tc_fence_after();
            const int hf = leader ? 0 : 1;
#pragma unroll
            for (int s = 0; s < 2; ++s)
                umma_f16(tmem + T1 + hf * 32, smem_desc(s_base + P_G_A + hf * 8192 + s * 256, 128, 512),
                         smem_desc(s_all + P_OFF_B3 + s * 256, 128, 512), ID_S2I, s > 0);
            umma_commit(bar_mma);
        }
        // ---- h3: conjugate twiddle, A4 --------------------------------------------------------------
        ok = mbar_wait(bar_mma, ph_m, wlim);
        ph_m ^= 1;
        tc_fence_after();
        if (ok) {
            const int k1 = tid & 31;
            const float4* twB = reinterpret_cast<const float4*>(smem_all + P_OFF_TWB) + k1;
#pragma unroll
            for (int g = 0; g < 2; ++g) {   // the twiddles depend on (k1, n2) only: shared by both row halves
                float re[16], im[16];
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    tmem_ld8(t_lane + T1 + hf * 32 + 8 * g, re + 8 * hf);
                    tmem_ld8(t_lane + T1 + hf * 32 + 16 + 8 * g, im + 8 * hf);
                }
                float4 w[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) w[q] = twB[(4 * g + q) * 32];
                tmem_ld_wait();
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    tmem_ld_fence8(re + 8 * hf);
                    tmem_ld_fence8(im + 8 * hf);
                }
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    const int r = hf * 4 + (tid >> 5);
                    uint4 pr, pi;
                    cmul_pack8(re + 8 * hf, im + 8 * hf, w, pr, pi);
                    unsigned char* base = smem + P_G_A + (r * 2 + g) * 1024 + (k1 >> 3) * 128 + (k1 & 7) * 16;
                    *reinterpret_cast<uint4*>(base) = pr;
                    *reinterpret_cast<uint4*>(base + 512) = pi;
                }
            }
        }
        fence_proxy_async();
        tc_fence_before();
        if (group_sync_or(wg, !ok, abort_flag)) {
            aborted = true;
            break;
        }
        // ---- S1' --------------------------------------------------------------------------------
        if (leader || leader2) {
            tc_fence_after();
            // the conjugated F_32 image is the A operand here (M = (re | im) x n1 = 64) and the data the B operand (N = 4 rows x 16 n2),
            // so that a thread of the last hand-off owns whole 32-byte runs of the output; the second half of the rows goes to
            // lanes 16..31 of every lane quarter (an M = 64 accumulator keeps row m in lane m % 16 + 32 (m / 16))
            const int hf = leader ? 0 : 1;
#pragma unroll
            for (int s = 0; s < 4; ++s)
                umma_f16(tmem + T2 + ((uint32_t)(16 * hf) << 16), smem_desc(s_all + P_OFF_B4 + s * 256, 128, 1024),
                         smem_desc(s_base + P_G_A + hf * 8192 + s * 256, 128, 1024), ID_S1I, s > 0);
            umma_commit(bar_mma);
        }
        // ---- h4: round and stage: a lane holds, for one n1 of the real-part rows or of the imaginary-part rows, the 16 n2 of
        //      four rows: 32-byte runs of y[r][n1*16 + n2].  The operand buffer (free now) takes the two boxes
        //      [8 rows][32 n1][16 n2] in the 32-byte-swizzled image of the TMA stores (16-byte chunk XOR bit 7 of the address):
        //      a quarter-warp's eight 16-byte stores fall into eight different bank groups ---------------
        // (HEADS: the X1 values this thread will need -- its four rows at its 16 positions -- come from L2 and are asked for before
        // the wait for the last stage)
        uint4 x1v[HEADS ? 8 : 1];
        if (HEADS) {
            const int m = 16 * warp + (tid & 15), c = m >> 5, n1 = m & 31, rh = (tid >> 4) & 1;
#pragma unroll
            for (int rl = 0; rl < 8; ++rl) x1v[rl] = make_uint4(0u, 0u, 0u, 0u);
            if ((warp & 1) == 0 && 16 * n1 < n) {
                const int hb = (h / kf_group) * kf_group;
#pragma unroll
                for (int rl = 0; rl < 4; ++rl) {
                    const uint4* xrow = reinterpret_cast<const uint4*>(xg + ((size_t)b0 * H + hb + kRows * c + 4 * rh + rl) * n + 16 * n1);
                    x1v[2 * rl] = __ldg(xrow);
                    x1v[2 * rl + 1] = __ldg(xrow + 1);
                }
            }
        }
        ok = mbar_wait(bar_mma, ph_m, wlim);
        ph_m ^= 1;
        tc_fence_after();
        float hacc[HEADS ? 16 : 1];
        if (ok) {
            // lane l of warp w holds output row m = 16 w + l % 16 = (c, n1) for the rows r = 4 (l / 16) .. + 3: 16 n2 per row
            const int m = 16 * warp + (tid & 15), c = m >> 5, n1 = m & 31, rh = (tid >> 4) & 1;
            unsigned char* st = smem + P_G_A + c * 8192 + (4 * rh) * 1024 + n1 * 32;
            const int sw = (n1 >> 2) & 1;
            if (HEADS) {
                // contraction with X1: this thread's four rows i = 8 c + 4 rh + (0 .. 3) at its 16 positions; positions past n do not exist
#pragma unroll
                for (int j = 0; j < 16; ++j) hacc[j] = 0.f;
                // (a warp holds n1 = 0 .. 15 or 16 .. 31: the second kind has nothing below position 256 and skips the tensor-memory
                // loads as a whole warp; a single lane whose positions lie past n only skips its own global loads)
                const bool lane_live = 16 * n1 < n;
                if ((warp & 1) == 0) {
#pragma unroll
                    for (int rl = 0; rl < 4; ++rl) {   // one row at a time
                        const uint4 xa = x1v[2 * rl], xb = x1v[2 * rl + 1];
                        float v[16];
                        tmem_ld8(t_lane + T2 + 16 * rl, v);
                        tmem_ld8(t_lane + T2 + 16 * rl + 8, v + 8);
                        tmem_ld_wait();
                        tmem_ld_fence8(v);
                        tmem_ld_fence8(v + 8);
                        const uint32_t xw[8] = {xa.x, xa.y, xa.z, xa.w, xb.x, xb.y, xb.z, xb.w};
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            hacc[2 * j] = fmaf(v[2 * j], __uint_as_float(xw[j] << 16), hacc[2 * j]);
                            hacc[2 * j + 1] = fmaf(v[2 * j + 1], __uint_as_float(xw[j] & 0xffff0000u), hacc[2 * j + 1]);
                        }
                    }
                }
                // the other four rows of this half sit 16 lanes further on; the half c = 1 hands its sums over through the operand buffer
#pragma unroll
                for (int j = 0; j < 16; ++j) hacc[j] += __shfl_xor_sync(0xffffffffu, hacc[j], 16);
                if (c == 1 && rh == 0 && lane_live) {
                    float4* xch = reinterpret_cast<float4*>(smem + P_G_A) + n1 * 4;
#pragma unroll
                    for (int j = 0; j < 4; ++j) xch[j] = make_float4(hacc[4 * j], hacc[4 * j + 1], hacc[4 * j + 2], hacc[4 * j + 3]);
                }
            }
            float w0 = 0.f, w1 = 0.f, w2 = 0.f;
            if (GATE) {
                w0 = __ldg(w_gate + 3 * h);
                w1 = __ldg(w_gate + 3 * h + 1);
                w2 = __ldg(w_gate + 3 * h + 2);
            }
#pragma unroll
            for (int g = 0; g < (HEADS ? 0 : 2); ++g) {   // two rows at a time
                // GATE: the 16 input values under this thread's run and their two neighbours, for both rows (requested before the
                // accumulator is read so that the two latencies overlap)
                uint4 xa[2], xb[2], aa[2], ab[2];
                unsigned short xl[2], xr[2];
                if (GATE) {
#pragma unroll
                    for (int rr = 0; rr < 2; ++rr) {
                        const int brow = b0 + kRows * c + 4 * rh + 2 * g + rr;
                        xa[rr] = xb[rr] = aa[rr] = ab[rr] = make_uint4(0u, 0u, 0u, 0u);
                        xl[rr] = xr[rr] = 0;
                        if (brow < B) {
                            const __nv_bfloat16* xrow = xg + ((size_t)brow * H + h) * 512 + 16 * n1;
                            xa[rr] = __ldg(reinterpret_cast<const uint4*>(xrow));
                            xb[rr] = __ldg(reinterpret_cast<const uint4*>(xrow) + 1);
                            if (n1 > 0) xl[rr] = __ldg(reinterpret_cast<const unsigned short*>(xrow) - 1);
                            if (n1 < 31) xr[rr] = __ldg(reinterpret_cast<const unsigned short*>(xrow) + 16);
                            if (vh != nullptr) {
                                const uint4* arow = reinterpret_cast<const uint4*>(vh + ((size_t)brow * H + h) * 512 + 16 * n1);
                                aa[rr] = __ldg(arow);
                                ab[rr] = __ldg(arow + 1);
                            }
                        }
                    }
                }
                float v[32];
#pragma unroll
                for (int q = 0; q < 4; ++q) tmem_ld8(t_lane + T2 + 32 * g + 8 * q, v + 8 * q);
                tmem_ld_wait();
#pragma unroll
                for (int q = 0; q < 4; ++q) tmem_ld_fence8(v + 8 * q);
                if (GATE) {
#pragma unroll
                    for (int rr = 0; rr < 2; ++rr) {
                        const uint32_t xw[8] = {xa[rr].x, xa[rr].y, xa[rr].z, xa[rr].w, xb[rr].x, xb[rr].y, xb[rr].z, xb[rr].w};
                        float xv[18];   // x[t0 - 1 .. t0 + 16]; a bf16 is the upper half of its fp32
                        xv[0] = __uint_as_float((uint32_t)xl[rr] << 16);
                        xv[17] = __uint_as_float((uint32_t)xr[rr] << 16);
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            xv[1 + 2 * j] = __uint_as_float(xw[j] << 16);
                            xv[2 + 2 * j] = __uint_as_float(xw[j] & 0xffff0000u);
                        }
                        const uint32_t aw[8] = {aa[rr].x, aa[rr].y, aa[rr].z, aa[rr].w, ab[rr].x, ab[rr].y, ab[rr].z, ab[rr].w};
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            const float add = (j & 1) ? __uint_as_float(aw[j >> 1] & 0xffff0000u) : __uint_as_float(aw[j >> 1] << 16);
                            v[16 * rr + j] = fmaf(v[16 * rr + j], fmaf(w2, xv[j + 2], fmaf(w1, xv[j + 1], w0 * xv[j])), add);
                        }
                    }
                }
#pragma unroll
                for (int q = 0; q < 4; ++q) {   // q = (row, half of the n2 range): one 16-byte chunk of the row's 32-byte run
                    const uint4 pk = make_uint4(pack_bf16(v[8 * q], v[8 * q + 1]), pack_bf16(v[8 * q + 2], v[8 * q + 3]),
                                                pack_bf16(v[8 * q + 4], v[8 * q + 5]), pack_bf16(v[8 * q + 6], v[8 * q + 7]));
                    *reinterpret_cast<uint4*>(st + (2 * g + (q >> 1)) * 1024 + (((q & 1) ^ sw) << 4)) = pk;
                }
            }
        }
        if (leader) *next_slot = un2;
        fence_proxy_async();   // the staged rows are read by the TMA stores
        tc_fence_before();
        if (group_sync_or(wg, !ok, abort_flag)) {
            aborted = true;
            break;
        }
        if (HEADS) {
            if (tid < 16 && 16 * tid < n) {   // rows 0 .. 7 summed: add the other half's sums, round, store this lane's 16 positions
                const float4* xch = reinterpret_cast<const float4*>(smem + P_G_A) + tid * 4;
                uint32_t o[8];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float4 t4 = xch[j];
                    o[2 * j] = pack_bf16(hacc[4 * j] + t4.x, hacc[4 * j + 1] + t4.y);
                    o[2 * j + 1] = pack_bf16(hacc[4 * j + 2] + t4.z, hacc[4 * j + 3] + t4.w);
                }
                uint4* dst = reinterpret_cast<uint4*>(y + ((size_t)b0 * H + h) * n + 16 * tid);
                dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
                dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
            }
        } else if (leader) {   // rows past the batch and positions past n are clipped by the tensor map
            tma_store_4d(&map_y, s_base + P_G_A, 0, 0, h, b0);
            if (b0 + kRows < B) tma_store_4d(&map_y, s_base + P_G_A + 8192, 0, 0, h, b0 + kRows);
            tma_store_commit();
        }
        u = un;
        un = *next_slot;   // written by thread 0 before the barrier above
    }
    // ---- teardown: nothing of ours may still be in flight when the TMEM and the CTA go away ----------
    if (leader) {
        if (aborted) atomicExch(status, (int32_t)M2_ERR_TIMEOUT);
        if (x_pending) mbar_wait(bar_x, ph_x, wlim);
        tma_store_wait_read0();
        __threadfence();
        if (atomicAdd(sched + 1, 1) == ustride - 1) {   // last pipeline out: reset the scheduler words
            sched[0] = 0;
            sched[1] = 0;
            __threadfence();
        }
    }
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x < 32) tmem_dealloc(tmem_cta, kTmemCols);
}

// ---- gradient with respect to the kernel k ---------------------------------------------------------------------------
//
//   dk[h] = M^-1 ( sum_b conj(M x_b) (.) M g_b ) [0:n)          (the transpose of Eq. 2 with respect to k)
//
// The forward half of the pipeline above (S1, twiddle, S2) runs on the x tile and on the g tile of a unit (8 batch
// entries of one channel) side by side: 128 TMEM columns per pipeline, 4 pipelines per CTA.  Each thread then holds the
// two spectra of its rows at the same (k1, k2), forms conj(X) G in fp32, adds its two rows, the four warps' sums are
// added through shared memory, and the unit's [k1][k2] sum goes to partial[b group][h] in plan order.  A CUDA-core
// kernel adds the b groups in order and applies M^-1 in fp32 (one block per channel).
constexpr int kGroupsW = 4;
constexpr int kThreadsW = 128 * kGroupsW;
constexpr int WG_X = 0;              // x tile 8192 | g tile 8192 (one box [r][n1][16 n2] each, 32-byte swizzled)
constexpr int WG_A = 16384;          // A2 of x 16384 | A2 of g 16384; afterwards the four warps' sums [warp][k2][33 k1] float2
constexpr int W_GROUP_BYTES = 49152;
constexpr int W_SMEM_BYTES = OFF_GROUP + kGroupsW * W_GROUP_BYTES;
static_assert(W_SMEM_BYTES <= 232448 && 4 * 16 * 33 * 8 <= 32768, "per-CTA budgets");

__global__ void __launch_bounds__(kThreadsW, 1)
convwgrad512_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_g, float2* __restrict__ partial,
                    const uint4* __restrict__ consts, int B, int H, int n, int32_t* __restrict__ status) {
    extern __shared__ __align__(1024) unsigned char smem_all[];
    const int wg = threadIdx.x >> 7, tid = threadIdx.x & 127, warp = tid >> 5;
    const bool leader = tid == 32 * (wg & 3);
    const uint32_t s_all = smem_u32(smem_all);
    unsigned char* smem = smem_all + OFF_GROUP + wg * W_GROUP_BYTES;
    const uint32_t s_base = s_all + OFF_GROUP + wg * W_GROUP_BYTES;
    const uint32_t bar_x = s_all + OFF_BAR + wg * 32, bar_mma = bar_x + 8;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_all + OFF_BAR + wg * 32 + 24);
    const uint32_t s_tptr = s_all + OFF_BAR + 512;
    const int bgroups = (B + kRows - 1) / kRows;
    const int units = H * bgroups;
    const int ustride = gridDim.x * kGroupsW;
    int u = wg * gridDim.x + blockIdx.x;   // pipeline-major: a partial last round spreads over all CTAs
    if (leader) {
        mbar_init(bar_x, 1);
        mbar_init(bar_mma, 1);
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tensormap(&map_x);
        prefetch_tensormap(&map_g);
    }
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    {
        uint4* dst = reinterpret_cast<uint4*>(smem_all + OFF_CONST);
        for (int i = threadIdx.x; i < CONST_BYTES / 16; i += kThreadsW) dst[i] = consts[i];
    }
    if (threadIdx.x < 32) tmem_alloc(s_tptr, kTmemCols);
    asm volatile("griddepcontrol.wait;" ::: "memory");
    bool x_pending = false;
    auto load_unit = [&](int v) {   // both tiles of unit v, one barrier phase
        mbar_expect_tx(bar_x, 16384);
        const int hh = v % H, bb = (v / H) * kRows;
        tma_load_4d(s_base + WG_X, &map_x, 0, 0, hh, bb, bar_x);          // boxes [8 rows][32 n1][16 n2], 32-byte swizzled
        tma_load_4d(s_base + WG_X + 8192, &map_g, 0, 0, hh, bb, bar_x);
        x_pending = true;
    };
    if (leader && u < units) load_unit(u);
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_cta = *reinterpret_cast<volatile uint32_t*>(smem_all + OFF_BAR + 512);
    const uint32_t tmem = tmem_cta + wg * 128;
    const uint32_t t_lane = tmem + ((uint32_t)(warp * 32) << 16);
    constexpr uint32_t ID_S1 = instr_desc_bf16(128, 64, true, false);
    constexpr uint32_t ID_S2 = instr_desc_bf16(128, 32, true, false);
    const int k1steps = (n / 16 + 15) / 16;
    uint32_t ph_x = 0, ph_m = 0;
    bool ok = true, aborted = false;
    while (u < units) {
        const int h = u % H, bg = u / H;
        const int un = u + ustride;
        // ---- S1 on both tiles -----------------------------------------------------------------------
        if (leader) {
            ok = mbar_wait(bar_x, ph_x);
            x_pending = false;
            if (ok) {
                tc_fence_after();
#pragma unroll
                for (int tt = 0; tt < 2; ++tt)
#pragma unroll 1
                    for (int s = 0; s < k1steps; ++s)
                        umma_f16(tmem + 64 * tt, smem_desc_sw32(s_base + WG_X + tt * 8192 + s * 512, 1024, 256),
                                 smem_desc(s_all + OFF_B1 + s * 256, 128, 512), ID_S1, s > 0);
                umma_commit(bar_mma);
            }
        }
        ph_x ^= 1;
        ok = ok && mbar_wait(bar_mma, ph_m);
        ph_m ^= 1;
        tc_fence_after();
        if (leader && ok && un < units) load_unit(un);   // the tiles are free
        // ---- h1: twiddle, A2 of x and of g ---------------------------------------------------------------
        if (ok) {
            const int r = tid >> 4, n2 = tid & 15, n2hi = n2 >> 3, n2lo = n2 & 7;   // lane = r * 16 + n2: the row order of the input boxes
            const float4* twA = reinterpret_cast<const float4*>(smem_all + OFF_TWA) + n2;
#pragma unroll 1
            for (int tt = 0; tt < 2; ++tt)
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    float re[16], im[16];
#pragma unroll
                    for (int jj = 0; jj < 2; ++jj) {
                        tmem_ld8(t_lane + 64 * tt + 16 * hh + 8 * jj, re + 8 * jj);
                        tmem_ld8(t_lane + 64 * tt + 32 + 16 * hh + 8 * jj, im + 8 * jj);
                    }
                    tmem_ld_wait();
#pragma unroll
                    for (int jj = 0; jj < 2; ++jj) {
                        tmem_ld_fence8(re + 8 * jj);
                        tmem_ld_fence8(im + 8 * jj);
                    }
#pragma unroll
                    for (int jj = 0; jj < 2; ++jj) {
                        const int j = 2 * hh + jj;
                        float4 w[4];
#pragma unroll
                        for (int q = 0; q < 4; ++q) w[q] = twA[(4 * j + q) * 16];
                        uint4 pr, pi;
                        cmul_pack8(re + 8 * jj, im + 8 * jj, w, pr, pi);
                        unsigned char* base = smem + WG_A + tt * 16384 + (r * 4 + j) * 512 + n2lo * 16;
                        *reinterpret_cast<uint4*>(base + (0 + n2hi) * 128) = pr;
                        *reinterpret_cast<uint4*>(base + (2 + n2hi) * 128) = pi;
                    }
                }
        }
        fence_proxy_async();
        tc_fence_before();
        if (group_sync_or(wg, !ok, abort_flag)) {
            aborted = true;
            break;
        }
        // ---- S2 on both ---------------------------------------------------------------------------------
        if (leader) {
            tc_fence_after();
#pragma unroll
            for (int tt = 0; tt < 2; ++tt)
#pragma unroll
                for (int hf = 0; hf < 2; ++hf)
#pragma unroll
                    for (int s = 0; s < 2; ++s)
                        umma_f16(tmem + 64 * tt + hf * 32, smem_desc(s_base + WG_A + tt * 16384 + hf * 8192 + s * 256, 128, 512),
                                 smem_desc(s_all + OFF_B2 + s * 256, 128, 512), ID_S2, s > 0);
            umma_commit(bar_mma);
        }
        ok = mbar_wait(bar_mma, ph_m);
        ph_m ^= 1;
        tc_fence_after();
        // ---- conj(X) G, summed over this thread's two rows, then over the four warps ------------------------------
        float2* red = reinterpret_cast<float2*>(smem + WG_A);   // [warp][k2][33]: both A2 buffers are free now
        if (ok) {
            const int k1 = tid & 31;
#pragma unroll
            for (int g = 0; g < 2; ++g) {
                float sr[8], si[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) sr[q] = si[q] = 0.f;
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    float xr[8], xi[8], gr[8], gi[8];
                    tmem_ld8(t_lane + hf * 32 + 8 * g, xr);
                    tmem_ld8(t_lane + hf * 32 + 16 + 8 * g, xi);
                    tmem_ld8(t_lane + 64 + hf * 32 + 8 * g, gr);
                    tmem_ld8(t_lane + 64 + hf * 32 + 16 + 8 * g, gi);
                    tmem_ld_wait();
                    tmem_ld_fence8(xr);
                    tmem_ld_fence8(xi);
                    tmem_ld_fence8(gr);
                    tmem_ld_fence8(gi);
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        sr[q] = fmaf(xr[q], gr[q], fmaf(xi[q], gi[q], sr[q]));
                        si[q] = fmaf(xr[q], gi[q], fmaf(-xi[q], gr[q], si[q]));
                    }
                }
#pragma unroll
                for (int q = 0; q < 8; ++q) red[(warp * 16 + 8 * g + q) * 33 + k1] = make_float2(sr[q], si[q]);
            }
        }
        tc_fence_before();
        if (group_sync_or(wg, !ok, abort_flag)) {
            aborted = true;
            break;
        }
        {
            float2* dst = partial + ((size_t)bg * H + h) * 512;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int p = tid + 128 * i, k1 = p >> 4, k2 = p & 15;   // plan order
                float2 a = red[(0 * 16 + k2) * 33 + k1];
#pragma unroll
                for (int w = 1; w < 4; ++w) {
                    const float2 b = red[(w * 16 + k2) * 33 + k1];
                    a.x += b.x;
                    a.y += b.y;
                }
                dst[p] = a;
            }
        }
        if (group_sync_or(wg, false, abort_flag)) {   // the sums are read: the next unit's h1 may overwrite them
            aborted = true;
            break;
        }
        u = un;
    }
    if (leader) {
        if (aborted) atomicExch(status, (int32_t)M2_ERR_TIMEOUT);
        if (x_pending) mbar_wait(bar_x, ph_x);
    }
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x < 32) tmem_dealloc(tmem_cta, kTmemCols);
}

// spectrum re-layout for this kernel: kfu[h][k2/2][k1] = (re(k2 even), re(k2 odd), im(even), im(odd)) from plan order
__global__ void relayout_spectrum_kernel(const float2* __restrict__ kf, float4* __restrict__ kfu, long long total) {
    const long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x;   // over H * 8 * 32
    if (i >= total) return;
    const int k1 = (int)(i & 31), q = (int)((i >> 5) & 7);
    const long long h = i >> 8;
    const float2 a = kf[h * 512 + k1 * 16 + 2 * q], b = kf[h * 512 + k1 * 16 + 2 * q + 1];
    kfu[i] = make_float4(a.x, b.x, a.y, b.y);
}

// ---- host side ---------------------------------------------------------------------------------------

static uint16_t bf16_bits(double v) {
    float f = (float)v;
    uint32_t b;
    std::memcpy(&b, &f, 4);
    b += 0x7FFFu + ((b >> 16) & 1u);
    return (uint16_t)(b >> 16);
}

// K-major operand image: element (n, k) of an [N][K] matrix, 8 x 8 core matrices of 128 bytes,
// K-adjacent core matrices 128 bytes apart, N-adjacent ones (K/8)*128 bytes apart.
static void put_kmajor(std::vector<uint16_t>& img, int K, int n, int k, double v) {
    const size_t byte = (size_t)(n / 8) * (K / 8) * 128 + (size_t)(k / 8) * 128 + (n % 8) * 16 + (k % 8) * 2;
    img[byte / 2] = bf16_bits(v);
}

static bool covered(const m2_plan* pl) {
    return pl->dtype == M2_BF16 && pl->p == 2 && pl->dims[0] == 32 && pl->dims[1] == 16;
}

cudaError_t create_tables(m2_plan* pl) {
    if (!covered(pl)) return cudaSuccess;
    const int N1 = 32, N2 = 16, N = 512;
    const double sg = pl->sign >= 0 ? 1.0 : -1.0;
    std::vector<uint16_t> B1(2048), B2(1024), B3(1024), B4(2048);
    std::vector<float> twA(1024), twB(1024);
    // B1: [N = (c,k1) 64][K = n1 32]: F32[k1,n1] = cos + i sg sin
    for (int c = 0; c < 2; ++c)
        for (int k1 = 0; k1 < N1; ++k1)
            for (int n1 = 0; n1 < N1; ++n1) {
                const double th = 2.0 * M_PI * ((k1 * n1) % N1) / N1;
                put_kmajor(B1, 32, c * 32 + k1, n1, c == 0 ? std::cos(th) : sg * std::sin(th));
            }
    // B2: [N = (c',k2) 32][K = (c,n2) 32]: (a + ib)(cos + i s) -> re: cos a - s b ; im: s a + cos b
    // B3: the same with the conjugate matrix: [N = (c',n2) 32][K = (c,k2) 32]
    for (int co = 0; co < 2; ++co)
        for (int o = 0; o < N2; ++o)
            for (int ci = 0; ci < 2; ++ci)
                for (int i = 0; i < N2; ++i) {
                    const double th = 2.0 * M_PI * ((o * i) % N2) / N2;
                    const double cs = std::cos(th), sn = sg * std::sin(th);
                    double f, g;
                    if (co == 0) { f = ci == 0 ? cs : -sn; g = ci == 0 ? cs : sn; }
                    else         { f = ci == 0 ? sn : cs;  g = ci == 0 ? -sn : cs; }
                    put_kmajor(B2, 32, co * 16 + o, ci * 16 + i, f);
                    put_kmajor(B3, 32, co * 16 + o, ci * 16 + i, g);
                }
    // B4: [N = n1 32][K = (c,k1) 64]: Re( conj(F32)[n1,k1] (a + ib) ) = cos a + s b
    for (int n1 = 0; n1 < N1; ++n1)
        for (int c = 0; c < 2; ++c)
            for (int k1 = 0; k1 < N1; ++k1) {
                const double th = 2.0 * M_PI * ((k1 * n1) % N1) / N1;
                put_kmajor(B4, 64, n1, c * 32 + k1, c == 0 ? std::cos(th) : sg * std::sin(th));
            }
    // twiddles w_N^{n2 k1}: twA[k1/2][n2] = (cos(k1 even), cos(k1 odd), sin(even), sin(odd)); twB[n2/2][k1] likewise, conjugated
    for (int k1 = 0; k1 < N1; ++k1)
        for (int n2 = 0; n2 < N2; ++n2) {
            const double th = 2.0 * M_PI * ((n2 * k1) % N) / N;
            const float cs = (float)std::cos(th), sn = (float)(sg * std::sin(th));
            const size_t ia = ((size_t)(k1 / 2) * 16 + n2) * 4 + (k1 % 2);
            twA[ia] = cs;
            twA[ia + 2] = sn;
            const size_t ib = ((size_t)(n2 / 2) * 32 + k1) * 4 + (n2 % 2);
            twB[ib] = cs;
            twB[ib + 2] = -sn;
        }
    std::vector<unsigned char> blob(CONST_BYTES);
    std::memcpy(blob.data(), B1.data(), 4096);
    std::memcpy(blob.data() + 4096, B2.data(), 2048);
    std::memcpy(blob.data() + 6144, B3.data(), 2048);
    std::memcpy(blob.data() + 8192, B4.data(), 4096);
    std::memcpy(blob.data() + 12288, twA.data(), 4096);
    std::memcpy(blob.data() + 16384, twB.data(), 4096);
    // row-pair kernel: B1p [N = (c,k1) 64][K = (c',n1) 64] = F32 on complex input; B4p [N = (c',n1) 64][K = (c,k1) 64] = conj(F32)
    std::vector<uint16_t> B1p(4096), B4p(4096);
    for (int co = 0; co < 2; ++co)
        for (int o = 0; o < N1; ++o)
            for (int ci = 0; ci < 2; ++ci)
                for (int i = 0; i < N1; ++i) {
                    const double th = 2.0 * M_PI * ((o * i) % N1) / N1;
                    const double cs = std::cos(th), sn = sg * std::sin(th);
                    // (a + ib)(cs + i sn): re = cs a - sn b, im = sn a + cs b;   conjugate: re = cs a + sn b, im = -sn a + cs b
                    put_kmajor(B1p, 64, co * 32 + o, ci * 32 + i, co == 0 ? (ci == 0 ? cs : -sn) : (ci == 0 ? sn : cs));
                    put_kmajor(B4p, 64, co * 32 + o, ci * 32 + i, co == 0 ? (ci == 0 ? cs : sn) : (ci == 0 ? -sn : cs));
                }
    std::vector<unsigned char> blob_p(P_CONST_BYTES);
    std::memcpy(blob_p.data() + P_OFF_B1, B1p.data(), 8192);
    std::memcpy(blob_p.data() + P_OFF_B2, B2.data(), 2048);
    std::memcpy(blob_p.data() + P_OFF_B3, B3.data(), 2048);
    std::memcpy(blob_p.data() + P_OFF_B4, B4p.data(), 8192);
    std::memcpy(blob_p.data() + P_OFF_TWA, twA.data(), 4096);
    std::memcpy(blob_p.data() + P_OFF_TWB, twB.data(), 4096);
    Tables* t = new Tables();
    cudaError_t e = cudaMalloc(&t->d_const, CONST_BYTES);
    if (e == cudaSuccess) e = cudaMalloc(&t->d_const_p, P_CONST_BYTES);
    if (e == cudaSuccess) e = cudaMemcpy(t->d_const_p, blob_p.data(), P_CONST_BYTES, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(conv512p_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, P_SMEM_BYTES);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(conv512p_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, P_SMEM_BYTES);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(conv512p_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, P_SMEM_BYTES);
    if (e == cudaSuccess) e = cudaMemcpy(t->d_const, blob.data(), CONST_BYTES, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMalloc(&t->d_sched, 2 * sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(t->d_sched, 0, 2 * sizeof(int));
    if (e == cudaSuccess) e = cudaFuncSetAttribute(conv512_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(convwgrad512_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, W_SMEM_BYTES);
    if (e != cudaSuccess) {
        if (t->d_const) cudaFree(t->d_const);
        if (t->d_const_p) cudaFree(t->d_const_p);
        if (t->d_sched) cudaFree(t->d_sched);
        delete t;
        return e;
    }
    pl->umma = reinterpret_cast<m2_umma_tables*>(t);
    return cudaSuccess;
}

void destroy_tables(m2_plan* pl) {
    if (!pl->umma || !covered(pl)) return;
    Tables* t = reinterpret_cast<Tables*>(pl->umma);
    if (t->d_const) cudaFree(t->d_const);
    if (t->d_const_p) cudaFree(t->d_const_p);
    if (t->d_sched) cudaFree(t->d_sched);
    delete t;
    pl->umma = nullptr;
}

// x / y viewed as [b][h][n1][n2] with n2 innermost; box = the 16 n2 of a row (32 bytes, 32-byte swizzle), all 32 n1, one h, 8 b
static bool make_map_rows32(CUtensorMap* map, const void* ptr, int64_t B, int64_t H, int64_t n) {
    const cuuint64_t gdim[4] = {16, (cuuint64_t)(n / 16), (cuuint64_t)H, (cuuint64_t)B};
    const cuuint64_t gstr[3] = {32, (cuuint64_t)n * 2, (cuuint64_t)H * n * 2};
    const cuuint32_t box[4] = {16, 32, 1, (cuuint32_t)kRows};
    return tma_host::encode_sw32_bf16(map, ptr, 4, gdim, gstr, box);
}

static int32_t conv_fwd_impl(const m2_plan* pl, const void* x, const void* kf, void* y, int64_t B, int64_t H, int64_t n, int32_t mode,
                             cudaStream_t stream, int selftest, int kf_group, const float* w_gate = nullptr, const void* gate_rows = nullptr,
                             const void* addend = nullptr) {
    if (!pl->umma || !covered(pl)) return M2_ERR_UNSUPPORTED;
    // rows must be whole multiples of the inner digit and 16-byte pitched for TMA
    if (n % 16 != 0 || (mode == M2_CIRCULAR && n != 512) || n > 512) return M2_ERR_UNSUPPORTED;
    Tables* t = reinterpret_cast<Tables*>(pl->umma);
    int dev = 0, sms = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const bool pairs = B > kRows || w_gate != nullptr;   // two batch rows per complex row once there are more than 8 (the gated form has this kernel only)
    if (w_gate != nullptr && (mode != M2_CIRCULAR || kf_group != 1)) return M2_ERR_UNSUPPORTED;
    if (selftest && !pairs) return M2_ERR_UNSUPPORTED;
    const long long units = pairs ? H * ((B + 2 * kRows - 1) / (2 * kRows)) : H * ((B + kRows - 1) / kRows);
    const int groups = pairs ? kGroupsP : kGroups;
    const long long ctas = (units + groups - 1) / groups;
    const int grid = (int)(ctas < sms ? ctas : sms);
    // the kernels' own spectrum layout follows the plan-order copy of the H / kf_group spectrum rows
    const float4* kfu = reinterpret_cast<const float4*>(static_cast<const unsigned char*>(kf) + (size_t)(H / kf_group) * 512 * 8);
    // launched with programmatic stream serialization: its CTAs may take over SMs that the previous kernel's CTAs
    // have left while that kernel's last CTAs still run (the kernel waits for it before touching its data)
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(pairs ? kThreadsP : kThreads);
    cfg.dynamicSmemBytes = pairs ? P_SMEM_BYTES : SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (pairs) {
        alignas(64) CUtensorMap my;
        if (!make_map_rows32(&my, y, B, H, n)) return M2_ERR_UNSUPPORTED;
        alignas(64) CUtensorMap mx32;   // the row-pair kernel reads whole 32-byte rows of 16 n2
        if (!make_map_rows32(&mx32, x, B, H, n)) return M2_ERR_UNSUPPORTED;
        const cudaError_t le =
            w_gate != nullptr
                ? cudaLaunchKernelEx(&cfg, conv512p_kernel<1>, mx32, my, (__nv_bfloat16*)y, kfu, (const uint4*)t->d_const_p, (int)B, (int)H,
                                     (int)n, pl->d_status, t->d_sched, selftest, kf_group, (const __nv_bfloat16*)(gate_rows ? gate_rows : x), w_gate,
                                     (const __nv_bfloat16*)addend)
                : cudaLaunchKernelEx(&cfg, conv512p_kernel<0>, mx32, my, (__nv_bfloat16*)y, kfu, (const uint4*)t->d_const_p, (int)B, (int)H,
                                     (int)n, pl->d_status, t->d_sched, selftest, kf_group, (const __nv_bfloat16*)nullptr, (const float*)nullptr,
                                     (const __nv_bfloat16*)nullptr);
        if (le != cudaSuccess) return M2_ERR_CUDA;
    } else {
        alignas(64) CUtensorMap mx;
        if (!make_map_rows32(&mx, x, B, H, n)) return M2_ERR_UNSUPPORTED;
        if (cudaLaunchKernelEx(&cfg, conv512_kernel, mx, (__nv_bfloat16*)y, kfu, (const uint4*)t->d_const, (int)B, (int)H, (int)n, pl->d_status,
                               t->d_sched, kf_group) != cudaSuccess)
            return M2_ERR_CUDA;
    }
    pl->last_kernel = w_gate != nullptr ? "conv_umma_o2_512_pairs_gated" : pairs ? "conv_umma_o2_512_pairs" : "conv_umma_o2_512_rows";
    pl->launches += 1;
    return M2_OK;
}

int32_t conv_fwd(const m2_plan* pl, const void* x, const void* kf, void* y, int64_t B, int64_t H, int64_t n, int32_t mode,
                 cudaStream_t stream, int kf_group) {
    return conv_fwd_impl(pl, x, kf, y, B, H, n, mode, stream, 0, kf_group);
}

int32_t conv_gate_fwd(const m2_plan* pl, const void* x, const void* kf, const float* w_gate, void* y, int64_t B, int64_t H,
                      cudaStream_t stream, const void* gate_rows, const void* addend) {
    if (w_gate == nullptr) return M2_ERR_INVALID_ARG;
    return conv_fwd_impl(pl, x, kf, y, B, H, 512, M2_CIRCULAR, stream, 0, 1, w_gate, gate_rows, addend);
}

int32_t conv_heads_fwd(const m2_plan* pl, const void* X1, const void* X2, const void* V, const void* kf_heads, void* y, int64_t B,
                       int64_t d, int64_t dh, int64_t n, cudaStream_t stream) {
    if (!pl->umma || !covered(pl)) return M2_ERR_UNSUPPORTED;
    if (dh != 2 * kRows || d % dh != 0 || n % 16 != 0 || n > 256 || n <= 0) return M2_ERR_UNSUPPORTED;
    if (B == 0) return M2_OK;
    if (B * d > 0x7fffffffLL) return M2_ERR_UNSUPPORTED;
    Tables* t = reinterpret_cast<Tables*>(pl->umma);
    int dev = 0, sms = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const long long units = B * d, ctas = (units + kGroupsP - 1) / kGroupsP;
    // X2 [B][d][n] as (16 n2 | n1 | channel | batch entry); a box takes 8 channels of one entry, digits n1 >= n / 16 read zeros
    alignas(64) CUtensorMap mx, my;
    const cuuint64_t gdim[4] = {16, (cuuint64_t)(n / 16), (cuuint64_t)d, (cuuint64_t)B};
    const cuuint64_t gstr[3] = {32, (cuuint64_t)n * 2, (cuuint64_t)d * n * 2};
    const cuuint32_t box[4] = {16, 32, (cuuint32_t)kRows, 1};
    if (!tma_host::encode_sw32_bf16(&mx, X2, 4, gdim, gstr, box)) return M2_ERR_UNSUPPORTED;
    if (!make_map_rows32(&my, y, B, d, n)) return M2_ERR_UNSUPPORTED;   // (not used by this mode; a valid map all the same)
    const float4* kfu = reinterpret_cast<const float4*>(static_cast<const unsigned char*>(kf_heads) + (size_t)(d / dh) * 512 * 8);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(ctas < sms ? ctas : sms));
    cfg.blockDim = dim3(kThreadsP);
    cfg.dynamicSmemBytes = P_SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, conv512p_kernel<2>, mx, my, (__nv_bfloat16*)y, kfu, (const uint4*)t->d_const_p, (int)B, (int)d, (int)n,
                           pl->d_status, t->d_sched, 0, (int)dh, (const __nv_bfloat16*)X1, (const float*)nullptr,
                           (const __nv_bfloat16*)V) != cudaSuccess)
        return M2_ERR_CUDA;
    pl->last_kernel = "conv_umma_o2_512_heads";
    pl->launches += 1;
    return M2_OK;
}

int32_t conv_fwd_wait_selftest(const m2_plan* pl, const void* x, const void* kf, void* y, int64_t B, int64_t H, int64_t n, int32_t mode,
                               cudaStream_t stream) {
    return conv_fwd_impl(pl, x, kf, y, B, H, n, mode, stream, 1, 1);
}

// dk[h] = Re M^-1 ( sum_p partial[p][h][:] ) [0:n) / 512 for N = 512 = 32 x 16: the parts added in index order, then the two
// inverse stages in fp32 (conj F_16 over k2 with the conjugated twiddle, conj F_32 over k1, real part); one block per channel
__global__ void __launch_bounds__(256) wgrad512_finish_kernel(const float2* __restrict__ partial, int parts, float* __restrict__ dk,
                                                              const float2* __restrict__ roots32, const float2* __restrict__ roots16, int H, int n,
                                                              float sgn) {
    __shared__ float2 a[512], bb[512], r32[32], r16[16];
    const int h = blockIdx.x, tid = threadIdx.x;
    if (tid < 32) r32[tid] = roots32[tid];
    if (tid < 16) r16[tid] = roots16[tid];
    for (int i = tid; i < 512; i += 256) {
        float2 v = make_float2(0.f, 0.f);
        for (int p = 0; p < parts; ++p) {
            const float2 w = partial[((size_t)p * H + h) * 512 + i];
            v.x += w.x;
            v.y += w.y;
        }
        a[i] = v;
    }
    __syncthreads();
    for (int o = tid; o < 512; o += 256) {   // (k1, n2) = sum_k2 conj(w_16^{k2 n2}) a[k1][k2], times conj(w_512^{n2 k1})
        const int k1 = o >> 4, n2 = o & 15;
        float sr = 0.f, si = 0.f;
#pragma unroll
        for (int k2 = 0; k2 < 16; ++k2) {
            const float2 w = r16[(k2 * n2) & 15], v = a[k1 * 16 + k2];   // conj(w) v = (wx vx + wy vy) + i (wx vy - wy vx)
            sr = fmaf(w.x, v.x, fmaf(w.y, v.y, sr));
            si = fmaf(w.x, v.y, fmaf(-w.y, v.x, si));
        }
        float ts, tc;
        sincospif(2.0f * (float)((n2 * k1) & 511) / 512.0f, &ts, &tc);
        ts *= sgn;   // w_512^{n2 k1} = tc + i ts; multiply by its conjugate
        bb[o] = make_float2(sr * tc + si * ts, si * tc - sr * ts);
    }
    __syncthreads();
    for (int t = tid; t < 512; t += 256) {   // y[n1*16 + n2] = Re sum_k1 conj(w_32^{k1 n1}) bb[k1][n2]
        const int n1 = t >> 4, n2 = t & 15;
        float acc = 0.f;
#pragma unroll
        for (int k1 = 0; k1 < 32; ++k1) {
            const float2 w = r32[(k1 * n1) & 31], v = bb[k1 * 16 + n2];
            acc = fmaf(w.x, v.x, fmaf(w.y, v.y, acc));
        }
        if (t < n) dk[(size_t)h * n + t] = acc * (1.0f / 512.0f);
    }
}

int64_t conv_wgrad_workspace_bytes(const m2_plan* pl, int64_t B, int64_t H) {
    return pl->umma && covered(pl) ? ((B + kRows - 1) / kRows) * H * 512 * 8 : 0;
}

// partial[b group][h][512] (plan order) = sum over the group's rows of conj(M x) (.) M g; returns the number of b groups in *parts
int32_t conv_wgrad_partials(const m2_plan* pl, const void* x, const void* g, void* partial, int64_t B, int64_t H, int64_t n, int32_t mode,
                            int* parts, cudaStream_t stream) {
    if (!pl->umma || !covered(pl)) return M2_ERR_UNSUPPORTED;
    if (n % 16 != 0 || (mode == M2_CIRCULAR && n != 512) || n > 512) return M2_ERR_UNSUPPORTED;
    Tables* t = reinterpret_cast<Tables*>(pl->umma);
    alignas(64) CUtensorMap mx, mg;
    if (!make_map_rows32(&mx, x, B, H, n) || !make_map_rows32(&mg, g, B, H, n)) return M2_ERR_UNSUPPORTED;
    int dev = 0, sms = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const long long bgroups = (B + kRows - 1) / kRows, units = H * bgroups;
    const long long ctas = (units + kGroupsW - 1) / kGroupsW;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(ctas < sms ? ctas : sms));
    cfg.blockDim = dim3(kThreadsW);
    cfg.dynamicSmemBytes = W_SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, convwgrad512_kernel, mx, mg, (float2*)partial, (const uint4*)t->d_const, (int)B, (int)H, (int)n,
                           pl->d_status) != cudaSuccess)
        return M2_ERR_CUDA;
    *parts = (int)bgroups;
    pl->launches += 1;
    return M2_OK;
}

// the second launch of the kernel gradient: dk from the partial sums
int32_t conv_wgrad_finish(const m2_plan* pl, const void* partial, int parts, float* dk, int64_t H, int64_t n, cudaStream_t stream) {
    if (!pl->umma || !covered(pl)) return M2_ERR_UNSUPPORTED;
    if (H == 0) return M2_OK;
    wgrad512_finish_kernel<<<(unsigned)H, 256, 0, stream>>>((const float2*)partial, parts, dk, pl->d_roots[0], pl->d_roots[1], (int)H, (int)n,
                                                            pl->sign >= 0 ? 1.0f : -1.0f);
    if (cudaGetLastError() != cudaSuccess) return M2_ERR_CUDA;
    pl->launches += 1;
    return M2_OK;
}

bool has_private_spectrum(const m2_plan* pl) { return pl->umma != nullptr && (covered(pl) || m2u3::covered(pl)); }

cudaError_t relayout_spectrum(const m2_plan* pl, void* kf, int64_t H, cudaStream_t stream) {
    if (m2u3::covered(pl)) return m2u3::relayout_spectrum(pl, kf, H, stream);
    if (!has_private_spectrum(pl) || H == 0) return cudaSuccess;
    const long long total = H * 256;
    float4* kfu = reinterpret_cast<float4*>(static_cast<unsigned char*>(kf) + (size_t)H * 512 * 8);
    relayout_spectrum_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>((const float2*)kf, kfu, total);
    return cudaGetLastError();
}


}  // namespace m2u
