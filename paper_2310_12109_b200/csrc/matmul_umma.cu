// Tensor-core order-2 Monarch matmul for 64 x 64 blocks (N = 4096), bf16 in / fp32 accumulate / bf16 out.
//
//   y[t][k2*64 + k1] = sum_{n2} L[k1][k2][n2] * sum_{n1} R[n2][k1][n1] * x[t][n1*64 + n2]      (Sec. 3.1)
//
// Both block-diagonal factors are batches of 64 independent GEMMs [tokens x 64] x [64 x 64]; the batch
// index is the CONTIGUOUS index of the data each factor reads (n2 for R, k1 for L after the middle
// permutation), so neither operand of a tensor-core GEMM can be taken from memory as it lies.  The two
// factors therefore run as two passes of one kernel that exchange the intermediate through a workspace
// laid out in 16 KB blocks z[token tile][n2 / 8][k1][t % 128][n2 % 8] (it mostly stays in the 126 MB L2): what the
// pass-1 CTA (token tile, n2 group) writes is one contiguous 128 KB slab, and what the pass-2 CTA (token tile, k1
// group) reads are eight contiguous 16 KB pieces of eight such slabs:
//
//   pass 1 (R): a CTA owns 128 tokens x 8 consecutive n2.  Threads read 16-byte pieces of x (8 values of
//               n2 for one (t, n1)), transpose 8 x 8 blocks in registers (the permutation P) and write the
//               K-major, 128-byte-swizzled UMMA operand A_{n2}[t][n1]; 8 UMMA groups (M = 128 tokens,
//               N = 64 = k1, K = 64 = n1) fill the 512 TMEM columns; the epilogue gathers, for every k1,
//               the 8 values of n2 from the 8 accumulators as one 16-byte piece (the permutation P^T); the
//               CTA's pieces [k1][t][16 B] are its slab of z and are stored from registers, 512 bytes per warp.
//   pass 2 (L): a CTA owns 128 tokens x 8 consecutive k1; eight bulk copies bring [n2 / 8][k1 % 8][t][16 B] into shared
//               memory, which IS the K-major operand of every k1 without swizzle (core matrix = 8 tokens x 16 bytes,
//               next K chunk 16 KB further); same UMMAs with L's blocks; the epilogue stages 16-byte pieces of
//               y[t][k2][k1] and one dimension-permuting TMA store scatters them (the last P).
#include <cuda.h>
#include <cuda_bf16.h>

#include <cstring>

#include "generic_kernels.h"
#include "matmul_umma.h"
#include "ptx_sm100.cuh"
#include "tma_host.h"

namespace m2mm {

using namespace sm100;

constexpr int kThreads = 512;
constexpr int kTileT = 128;   // tokens per CTA
constexpr int kGroup = 8;     // blocks per CTA
constexpr int OFF_A = 0;                   // 8 operands [128 t][64] bf16, swizzled   131072
constexpr int OFF_B = 131072;              // 8 weight blocks [64][64] bf16, swizzled   65536
constexpr int OFF_BAR = 196608;            // bar_mma, tmem ptr, bar_in
constexpr int SMEM_BYTES = OFF_BAR + 64;

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, uint32_t src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit_wait() {
    asm volatile("cp.async.commit_group;" ::: "memory");
    asm volatile("cp.async.wait_group 0;" ::: "memory");
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, uint32_t src, int c0, int c1, int c2) {
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];" ::"l"(map), "r"(src), "r"(c0),
                 "r"(c1), "r"(c2)
                 : "memory");
}
__device__ __forceinline__ void bulk_store(void* gdst, uint32_t ssrc, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst), "r"(ssrc), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t r;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
    return r;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
// byte offset of 16-byte chunk kc of row r in a K-major operand with 128-byte rows and the 128B swizzle
__device__ __forceinline__ uint32_t sw_off(int r, int kc) { return (uint32_t)((r >> 3) * 1024 + (r & 7) * 128 + ((kc ^ (r & 7)) << 4)); }

// PASS 1: in = x[T][64 n1][64 n2], W = R[n2][k1][n1], out = z[T][64 k1][64 n2]
// PASS 2: in = z[T][64 k1][64 n2], W = L[k1][k2][n2], out = y[T][64 k2][64 k1]
template <int PASS>
__global__ void __launch_bounds__(kThreads, 1)
monarch64_pass_kernel(const __nv_bfloat16* __restrict__ in, const __nv_bfloat16* __restrict__ W,
                      const __grid_constant__ CUtensorMap map_out, __nv_bfloat16* __restrict__ zout, long long T,
                      int32_t* __restrict__ status, const __nv_bfloat16* __restrict__ Kmul, long long Hk, int relu) {
    extern __shared__ __align__(1024) unsigned char smem[];
    const int tid = threadIdx.x;
    const int wg = tid >> 7, t = tid & 127, warp = t >> 5;
    const uint32_t s_base = smem_u32(smem);
    const uint32_t bar_mma = s_base + OFF_BAR, s_tptr = s_base + OFF_BAR + 16, bar_in = s_base + OFF_BAR + 24;
    // the 8 CTAs that share the 128-byte lines of one token tile are neighbours in launch order, so the
    // 16-byte pieces of a line are fetched / written while the line is still in L2
    const long long t0 = (long long)blockIdx.y * kTileT;
    const int grp = blockIdx.x;   // which 8 consecutive blocks (n2 in pass 1, k1 in pass 2)

    if (tid == 0) {
        mbar_init(bar_mma, 1);
        mbar_init(bar_in, 1);
        fence_barrier_init();
    }
    if (tid < 32) tmem_alloc(s_tptr, 512);
    // Programmatic dependent launch: the next kernel's CTAs may take over SMs as this grid's CTAs leave them.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    // weight blocks -> swizzled K-major B operands ([64 out][64 in], rows of 128 bytes)
    for (int c = tid; c < kGroup * 64 * 8; c += kThreads) {
        const int kc = c & 7, o = (c >> 3) & 63, bl = c >> 9;
        cp_async16(s_base + OFF_B + bl * 8192 + sw_off(o, kc), W + ((size_t)(grp * kGroup + bl) * 64 + o) * 64 + kc * 8, 16u);
    }
    // The weights are the caller's and were complete before this call; everything else (pass 1's z for pass 2, the
    // producer of x, earlier readers of the buffers written here) is awaited now.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (PASS == 1) {
        // unit = (token tt, group g of 8 consecutive n1): 8 loads of 16 bytes (8 values of n2 each), an 8 x 8
        // transpose in registers, 8 stores (one per n2) of the 8 n1 values = chunk g of row tt of A_{n2}
#pragma unroll 1
        for (int u = tid; u < kTileT * 8; u += kThreads) {
            const int g = u & 7, tt = u >> 3;
            uint4 v[8];
            const bool live = t0 + tt < T;
            const uint4* src = reinterpret_cast<const uint4*>(in + (size_t)(t0 + tt) * 4096 + (size_t)(8 * g) * 64 + grp * 8);
#pragma unroll
            for (int i = 0; i < 8; ++i) {   // cached in L2 only: the other half of every 32-byte sector belongs to another SM
                v[i] = make_uint4(0u, 0u, 0u, 0u);
                if (live)
                    asm volatile("ld.global.cg.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v[i].x), "=r"(v[i].y), "=r"(v[i].z), "=r"(v[i].w) : "l"(src + i * 8));
            }
            const uint32_t* w = reinterpret_cast<const uint32_t*>(v);   // w[i*4 + j]: n1 = 8g+i, n2 = 2j, 2j+1
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                uint4 lo, hi;
                lo.x = prmt(w[0 * 4 + j], w[1 * 4 + j], 0x5410); hi.x = prmt(w[0 * 4 + j], w[1 * 4 + j], 0x7632);
                lo.y = prmt(w[2 * 4 + j], w[3 * 4 + j], 0x5410); hi.y = prmt(w[2 * 4 + j], w[3 * 4 + j], 0x7632);
                lo.z = prmt(w[4 * 4 + j], w[5 * 4 + j], 0x5410); hi.z = prmt(w[4 * 4 + j], w[5 * 4 + j], 0x7632);
                lo.w = prmt(w[6 * 4 + j], w[7 * 4 + j], 0x5410); hi.w = prmt(w[6 * 4 + j], w[7 * 4 + j], 0x7632);
                *reinterpret_cast<uint4*>(smem + OFF_A + (2 * j) * 16384 + sw_off(tt, g)) = lo;
                *reinterpret_cast<uint4*>(smem + OFF_A + (2 * j + 1) * 16384 + sw_off(tt, g)) = hi;
            }
        }
    } else if (tid == 0) {
        // z block (token tile, n2 group kc, k1 group grp) = [k1 % 8][t][8 n2] = 16 KB: chunk kc of every operand row
        mbar_expect_tx(bar_in, 8 * 16384);
        const unsigned char* zb = reinterpret_cast<const unsigned char*>(in) + (size_t)blockIdx.y * (8 * 131072) + (size_t)grp * 16384;
        for (int kc = 0; kc < 8; ++kc) bulk_load(s_base + OFF_A + kc * 16384, zb + (size_t)kc * 131072, 16384, bar_in);
    }
    cp_async_commit_wait();
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(smem + OFF_BAR + 16);

    if (tid == 0) {
        constexpr uint32_t IDESC = instr_desc_bf16(128, 64, false, false);
        bool in_ok = true;
        if (PASS == 2) in_ok = mbar_wait(bar_in, 0);
        if (in_ok) {
#pragma unroll 1
            for (int bl = 0; bl < kGroup; ++bl)
#pragma unroll
                for (int s = 0; s < 4; ++s)
                    umma_f16(tmem + bl * 64,
                             PASS == 1 ? smem_desc_sw128(s_base + OFF_A + bl * 16384 + s * 32, 16, 1024)
                                       : smem_desc(s_base + OFF_A + bl * 2048 + s * 32768, 16384, 128),
                             smem_desc_sw128(s_base + OFF_B + bl * 8192 + s * 32, 16, 1024), IDESC, s > 0);
        }
        umma_commit(bar_mma);   // (with no UMMA issued it completes at once; the missing input is reported below)
        if (!in_ok) atomicExch(status, (int32_t)M2_ERR_TIMEOUT);
    }
    const bool ok = mbar_wait(bar_mma, 0);
    tc_fence_after();
    // epilogue: lane = token; warpgroup wg takes output columns [16 wg, 16 wg + 16); for every output index o the 8
    // accumulators give the 8 consecutive block indices -> one 16-byte piece.  The pieces are staged in the (now free)
    // operand buffer with consecutive lanes writing to different banks, then leave through the copy engine:
    //   pass 1: the pieces [k1][t][16 B] are this CTA's contiguous slab of z and go straight from registers to global
    //           memory (a warp's 32 tokens are 512 contiguous bytes);
    //   pass 2: y[t][k2][k1]     -- staged as [k2][t][16 B]; one TMA store whose tensor map lists the dimensions as
    //                               (k1, t, k2) scatters the pieces (rows past T are clipped by the map).
    unsigned char* zslab = PASS == 1 ? reinterpret_cast<unsigned char*>(zout) + ((size_t)blockIdx.y * 8 + grp) * 131072 : nullptr;
    if (ok) {
        const uint32_t t_lane = tmem + ((uint32_t)(warp * 32) << 16);
#pragma unroll 1
        for (int gk = 0; gk < 2; ++gk) {
            const int o0 = 16 * wg + 8 * gk;
            float v[8][8];
#pragma unroll
            for (int bl = 0; bl < 8; ++bl) tmem_ld8(t_lane + bl * 64 + o0, v[bl]);
            tmem_ld_wait();
#pragma unroll
            for (int bl = 0; bl < 8; ++bl) tmem_ld_fence8(v[bl]);
            if (PASS == 2 && Kmul != nullptr && t0 + t < T) {
                // y = sigma(K (.) M x) (first half of the M2 operator, Eq. 2): the 8 accumulators of one kk are the 8
                // consecutive k1 of output index k2*64 + k1 -> one 16-byte piece of the kernel row
                const __nv_bfloat16* krow = Kmul + (size_t)((t0 + t) % Hk) * 4096 + 8 * grp;
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    const uint4 kp = *reinterpret_cast<const uint4*>(krow + (o0 + kk) * 64);
                    const uint32_t kw[4] = {kp.x, kp.y, kp.z, kp.w};
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        float a = v[2 * q][kk] * __uint_as_float(kw[q] << 16);
                        float b = v[2 * q + 1][kk] * __uint_as_float(kw[q] & 0xffff0000u);
                        v[2 * q][kk] = relu ? fmaxf(a, 0.f) : a;
                        v[2 * q + 1][kk] = relu ? fmaxf(b, 0.f) : b;
                    }
                }
            }
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
                const uint4 p = make_uint4(pack_bf16(v[0][kk], v[1][kk]), pack_bf16(v[2][kk], v[3][kk]),
                                           pack_bf16(v[4][kk], v[5][kk]), pack_bf16(v[6][kk], v[7][kk]));
                if (PASS == 1)   // z slab [k1][token][16 B]: a warp's 32 tokens are 512 contiguous bytes, stored as they are
                    *reinterpret_cast<uint4*>(zslab + (o0 + kk) * 2048 + t * 16) = p;
                else             // [k2][token][16 B], scattered to y by the TMA store below
                    *reinterpret_cast<uint4*>(smem + OFF_A + (o0 + kk) * 2048 + t * 16) = p;
            }
        }
    }
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    if (PASS == 2 && tid == 0 && ok) {
        tma_store_3d(&map_out, s_base + OFF_A, 8 * grp, (int)t0, 0);
        tma_store_commit();
        tma_store_wait_read0();   // the staging buffer dies with the CTA
    }
    __syncthreads();
    if (!ok && tid == 0) atomicExch(status, (int32_t)M2_ERR_TIMEOUT);
    if (tid < 32) tmem_dealloc(tmem, 512);
}

bool covered(const m2_plan* pl);
int64_t workspace_bytes(const m2_plan* pl, int64_t T);

// ---- the forward passes: 64 tokens x 16 blocks per CTA ------------------------------------------------------------------
//
// The cost of both passes is the number of memory requests for the pieces of x (pass 1) and of y (pass 2) that a CTA owning
// g consecutive blocks touches: 2 g bytes of every 128-byte line.  With g = 16 a piece is a whole 32-byte sector -- half as
// many requests as with g = 8 -- and the tile shrinks to 64 tokens so that the 16 operands still fill 128 KB:
//
//   UMMA         M = 64 (tokens), N = 64, K = 64 per block; row r of an accumulator lives in TMEM lane (r % 16) + 32 (r / 16),
//                so the accumulators of blocks 8..15 sit at lane offset 16 in the columns of blocks 0..7: 16 accumulators in
//                512 columns, and in the epilogue lanes 0..15 of a warp hold blocks 0..7 and lanes 16..31 blocks 8..15 of
//                the same 16 tokens.
//   weights      16 blocks of 8 KB do not fit beside the operands: they stream through a ring of kSlots buffers, one TMA
//                tile per block (128-byte swizzle = the K-major operand image), re-filled as the UMMAs release them.
//   workspace    z[64-token tile][k1][n2 / 8][t % 64][n2 % 8]: per (tile, k1) 8 KB that ARE the K-major operand of block k1
//                in pass 2 without swizzle (core matrix = 8 tokens x 16 bytes; next K chunk 1 KB further).  The pass-1 CTA
//                (tile, n2 group) writes 2 KB of each of them straight from registers; the pass-2 CTA (tile, k1 group)
//                fetches its 16 operands as 128 contiguous KB.
//   pass 1 in    one (token, 8 consecutive n1) per thread: 8 loads of 32 bytes, a 16 x 8 transpose in registers (PRMT; this
//                is P), 16 stores of 16 bytes into the swizzled operands A_{n2}[t][n1].
//   pass 2 out   y[t][k2][16 k1]: a thread's 8 accumulators of one k2 are 16 bytes, the lane 16 further holds the other half
//                of the sector; stored from registers (the last P).
constexpr int kTile2 = 64;                    // tokens per CTA
constexpr int kGroup2 = 16;                   // blocks per CTA
constexpr int kSlots = 11;                    // weight ring
constexpr int kIssuers = 4;                   // UMMA-issuing threads
constexpr int F_OFF_A = 0;                    // 16 operands [64 t][64] bf16                         131072
constexpr int F_OFF_W = 131072;               // kSlots weight blocks [64][64] bf16, swizzled         90112
constexpr int F_OFF_BAR = F_OFF_W + kSlots * 8192;   // full[kSlots], empty[kSlots], bar_mma, bar_in, tmem ptr
constexpr int F_SMEM_BYTES = F_OFF_BAR + 256;
static_assert(F_SMEM_BYTES <= 232448 && (2 * kSlots + 4) * 8 + 24 <= 256, "shared-memory budget of the forward passes");

// PASS 1: in = x[T][64 n1][64 n2], weights R[n2][k1][n1], out = workspace z
// PASS 2: in = workspace z, weights L[k1][k2][n2], out = y[T][64 k2][64 k1] (optionally sigma(K (.) y))
//
// Persistent: CTA c of a grid that is a multiple of 4 walks the items c, c + grid, .. of (token tile, block group) pairs numbered
// group-fastest, so its block group is c % 4 for good (the weights stay) and the 4 CTAs that share a tile's lines work on it at
// the same time.  Of the 16 weight blocks, 5..10 own ring slots 5..10; blocks 0..4 and 11..15 take turns in slots 0..4: a tile
// runs the blocks that are resident first (0..10 on even iterations, 15..5 on odd ones) and the other five as their slots are
// re-filled -- 5 block loads per tile.  The phases of consecutive tiles overlap: the loads of tile i + 1 are in flight (in
// registers in pass 1, as bulk copies into the operand buffer in pass 2) while the accumulators of tile i are drained.
template <int PASS>
__global__ void __launch_bounds__(kThreads, 1)
monarch64_fwd_kernel(const __nv_bfloat16* __restrict__ in, const __grid_constant__ CUtensorMap map_w, __nv_bfloat16* __restrict__ out,
                     long long T, int32_t* __restrict__ status, const __nv_bfloat16* __restrict__ Kmul, long long Hk, int relu) {
    extern __shared__ __align__(1024) unsigned char smem[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t s_base = smem_u32(smem);
    const uint32_t bar_full = s_base + F_OFF_BAR, bar_empty = bar_full + 8 * kSlots, bar_mma = bar_empty + 8 * kSlots;
    const uint32_t bar_in = bar_mma + 8, s_tptr = bar_mma + 16, bar_go = bar_mma + 48;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + F_OFF_BAR + (2 * kSlots + 2) * 8 + 8);
    const int grp = blockIdx.x & 3;                                   // which 16 consecutive blocks (n2 in pass 1, k1 in pass 2)
    const long long ntiles = (T + kTile2 - 1) / kTile2, nitems = 4 * ntiles;
    long long item = blockIdx.x;
    if (tid == 0) {
        for (int i = 0; i < 2 * kSlots + 2; ++i) mbar_init(bar_full + 8 * i, i == 2 * kSlots ? kIssuers : 1);   // bar_mma: one arrival per issuer
        *abort_flag = 0;
        mbar_init(bar_go, 1);
        fence_barrier_init();
        prefetch_tensormap(&map_w);
    }
    if (warp == 2) tmem_alloc(s_tptr, 512);
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    __syncthreads();   // barriers initialised before anyone arms them
    // weight block b -> ring slot b % kSlots (the weights are the caller's and were complete before this call)
    auto load_block = [&](int b) {
        const uint32_t slot = (uint32_t)(b % kSlots);
        mbar_expect_tx(bar_full + 8 * slot, 8192);
        tma_load_2d(s_base + F_OFF_W + slot * 8192, &map_w, 0, (grp * kGroup2 + b) * 64, bar_full + 8 * slot);
    };
    volatile int* fills = abort_flag + 1;   // thread 32: fills requested so far for slots 0..4
    if (tid == 32)
        for (int b = 0; b < kSlots; ++b) {
            load_block(b);
            if (b < 5) fills[b] = 1;
        }
    // this CTA's quarter of a tile's lines, pulled towards L2 as whole lines well before the 32-byte pieces are read
    auto prefetch_item = [&](long long it) {
        if (PASS == 1 && it < nitems) {
            const long long t0p = (it >> 2) * kTile2;
            const long long rows = T - t0p < kTile2 ? T - t0p : kTile2;
            const long long share = rows * 8192 / 4;
            bulk_prefetch_l2(reinterpret_cast<const unsigned char*>(in) + t0p * 8192 + grp * share, (uint32_t)share);
        }
    };
    if (tid == 64) {
        prefetch_item(item);
        prefetch_item(item + gridDim.x);
    }
    // everything else (pass 1's z for pass 2, the producer of x, earlier readers of the buffers written here) is awaited now
    asm volatile("griddepcontrol.wait;" ::: "memory");

    // pass 1: one (token, 8 consecutive n1) per thread, 8 loads of 32 bytes
    const int g = tid & 7, tt_in = tid >> 3;
    uint32_t w[8][8];   // w[i][j]: n1 = 8 g + i, n2 = 16 grp + 2 j, 2 j + 1
    auto load_x = [&](long long it) {
        const long long t0l = (it >> 2) * kTile2;
        const bool live = t0l + tt_in < T;
        const unsigned char* src = reinterpret_cast<const unsigned char*>(in) + (size_t)(t0l + tt_in) * 8192 + (size_t)(8 * g) * 128 + grp * 32;
#pragma unroll
        for (int i = 0; i < 8; ++i) {   // cached in L2 only: the rest of every line belongs to other SMs
            if (live) {
                asm volatile("ld.global.cg.v8.u32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                             : "=r"(w[i][0]), "=r"(w[i][1]), "=r"(w[i][2]), "=r"(w[i][3]), "=r"(w[i][4]), "=r"(w[i][5]), "=r"(w[i][6]), "=r"(w[i][7])
                             : "l"(src + i * 128));
            } else {
#pragma unroll
                for (int j = 0; j < 8; ++j) w[i][j] = 0u;
            }
        }
    };
    // the 16 x 8 transpose in registers (this is P) and the 16 stores into the swizzled operands A_{n2}[t][n1]
    auto store_a = [&]() {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            uint4 lo, hi;
            lo.x = prmt(w[0][j], w[1][j], 0x5410); hi.x = prmt(w[0][j], w[1][j], 0x7632);
            lo.y = prmt(w[2][j], w[3][j], 0x5410); hi.y = prmt(w[2][j], w[3][j], 0x7632);
            lo.z = prmt(w[4][j], w[5][j], 0x5410); hi.z = prmt(w[4][j], w[5][j], 0x7632);
            lo.w = prmt(w[6][j], w[7][j], 0x5410); hi.w = prmt(w[6][j], w[7][j], 0x7632);
            *reinterpret_cast<uint4*>(smem + F_OFF_A + (2 * j) * 8192 + sw_off(tt_in, g)) = lo;
            *reinterpret_cast<uint4*>(smem + F_OFF_A + (2 * j + 1) * 8192 + sw_off(tt_in, g)) = hi;
        }
    };
    // pass 2: the 16 operands of (tile, k1 group) are 128 contiguous KB of the workspace
    auto load_z = [&](long long it) {
        mbar_expect_tx(bar_in, kGroup2 * 8192);
        const unsigned char* zb = reinterpret_cast<const unsigned char*>(in) + ((size_t)(it >> 2) * 64 + (size_t)grp * kGroup2) * 8192;
        for (int b = 0; b < kGroup2; ++b) bulk_load(s_base + F_OFF_A + b * 8192, zb + (size_t)b * 8192, 8192, bar_in);
    };
    bool z_pending = false;
    uint32_t z_par = 0;   // thread 0: parity of the operand copy in flight
    if (item < nitems) {
        if (PASS == 1) {
            load_x(item);
            store_a();
        } else if (tid == 0) {
            load_z(item);
            z_pending = true;
        }
    }
    const uint32_t tmem_slot = F_OFF_BAR + (2 * kSlots + 2) * 8;
    uint32_t it_n = 0;   // iterations done: parities of bar_mma, bar_in and of the alternating ring slots
    bool ok = true;
#pragma unroll 1
    for (; item < nitems; item += gridDim.x, ++it_n) {
        const long long tile = item >> 2, t0 = tile * kTile2, next = item + gridDim.x;
        // the operands of this tile are complete (pass 1) and the previous tile's accumulators have been read
        fence_proxy_async();
        tc_fence_before();
        if (__syncthreads_or(*abort_flag)) break;   // a wait ran out somewhere: every thread leaves here, together
        tc_fence_after();
        const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(smem + tmem_slot);
        const bool odd = (it_n & 1u) != 0;
        // UMMA issue.  One thread issues an instruction of this size every ~57 cycles while the tensor core can take one every ~32:
        // four threads (lane 0 of warps 4..7, one per scheduler) issue the positions p = i, i + 4, .. concurrently.  Position p
        // runs block p on even iterations and 15 - p on odd ones: first the blocks whose weights are resident, then the five
        // whose slots are re-filled meanwhile; a slot is released by a commit of the thread that used it.
        if (lane == 0 && warp >= 4 && warp < 4 + kIssuers) {
            constexpr uint32_t IDESC = instr_desc_bf16(64, 64, false, false);
            bool ok_in = true;
            if (PASS == 2) ok_in = mbar_wait(bar_in, it_n & 1u);
            tc_fence_after();
#pragma unroll 1
            for (int p = warp - 4; p < kGroup2 && ok_in; p += kIssuers) {
                const int b = odd ? kGroup2 - 1 - p : p;
                const uint32_t slot = (uint32_t)(b % kSlots);
                // Slots 5..10 are filled once (waited for on the first iteration).  Slots 0..4 are filled once before the loop and once
                // in every iteration: the first five positions use fill number it_n (there since the previous iteration), the last
                // five fill number it_n + 1 (requested in this iteration).
                if (p >= 5 && p < kSlots) {
                    if (it_n == 0) ok_in = mbar_wait(bar_full + 8 * slot, 0);
                } else {
                    ok_in = mbar_wait(bar_full + 8 * slot, (p < 5 ? it_n : it_n + 1u) & 1u);
                }
                if (!ok_in) break;
                tc_fence_after();
                const uint32_t d = tmem + ((uint32_t)(16 * (b >> 3)) << 16) + (uint32_t)(b & 7) * 64;
                const uint64_t ad = PASS == 1 ? smem_desc_sw128(s_base + F_OFF_A + b * 8192, 16, 1024) : smem_desc(s_base + F_OFF_A + b * 8192, 1024, 128);
                const uint64_t bd = smem_desc_sw128(s_base + F_OFF_W + slot * 8192, 16, 1024);
                constexpr uint64_t a_step = PASS == 1 ? 2 : 128;   // per K step of 16: 32 bytes of a swizzled row, or two 1 KB chunks (in 16-byte units)
#pragma unroll
                for (int s = 0; s < 4; ++s) umma_f16(d, ad + s * a_step, bd + s * 2, IDESC, s > 0);
                if (p < 5) umma_commit(bar_empty + 8 * slot);   // the slot's other block may come in
            }
            umma_commit(bar_mma);   // (with nothing issued it completes at once; the missing input is reported here)
            if (!ok_in) {
                atomicExch(status, (int32_t)M2_ERR_TIMEOUT);
                *abort_flag = 1;
            }
        } else if (tid == 32) {   // re-fill slots 0..4 with the blocks this tile runs last: 11..15 on even iterations, 4..0 on odd ones
#pragma unroll 1
            for (int p = kSlots; p < kGroup2; ++p) {
                const int b = odd ? kGroup2 - 1 - p : p;
                if (!mbar_wait(bar_empty + 8 * (b % kSlots), it_n & 1u)) {
                    atomicExch(status, (int32_t)M2_ERR_TIMEOUT);
                    *abort_flag = 1;
                    break;
                }
                load_block(b);
                ++fills[b % kSlots];
            }
            if (PASS == 1) mbar_arrive(bar_go);   // (also after a failed wait: nobody is left waiting for this)
        } else if (tid == 64) {
            prefetch_item(next + gridDim.x);
        }
        __syncwarp();   // the lanes that share a warp with an issuing or producing thread must not spin on a barrier while it works
        // pass 1: the next tile's pieces are requested now and arrive while this tile's accumulators are computed and drained --
        // but only once the five weight blocks this tile still needs have been requested: behind 64 K piece requests they would
        // arrive thousands of cycles late, and the last UMMAs wait for them
        if (PASS == 1 && next < nitems) {
            if (tid != 32 && !mbar_wait(bar_go, it_n & 1u)) *abort_flag = 1;
            load_x(next);
        }
        ok = mbar_wait(bar_mma, it_n & 1u);
        tc_fence_after();
        // pass 2: the operand buffer is free again: the next tile's operands come in while this tile is stored
        if (PASS == 2 && tid == 0) {
            z_pending = false;
            if (ok && next < nitems) {
                load_z(next);
                z_pending = true;
                z_par = (it_n + 1u) & 1u;
            }
        }
        // epilogue: lane l of lane quarter q holds token 16 q + (l & 15) of block set l >> 4 (blocks 8 set .. 8 set + 7); the four warps
        // of a quarter split the 64 output columns.  For every output index the 8 accumulators of a thread are 8 consecutive block
        // indices: one 16-byte piece.
        if (ok) {
            const int q = warp & 3, c4 = warp >> 2, tt = 16 * q + (lane & 15), set = lane >> 4;
            const uint32_t t_lane = tmem + ((uint32_t)(q * 32) << 16);
            const bool live = t0 + tt < T;
            unsigned char* dst;
            if (PASS == 1)   // z[tile][k1][octet 2 grp + set][tt][16 B]
                dst = reinterpret_cast<unsigned char*>(out) + (size_t)tile * (64 * 8192) + (size_t)(2 * grp + set) * 1024 + tt * 16;
            else             // y[t][k2][16 grp + 8 set ..]
                dst = reinterpret_cast<unsigned char*>(out) + (size_t)(t0 + tt) * 8192 + (size_t)(16 * grp + 8 * set) * 2;
#pragma unroll 1
            for (int gk = 0; gk < 4; ++gk) {
                const int o0 = 16 * c4 + 4 * gk;
                float v[8][4];
#pragma unroll
                for (int bl = 0; bl < 8; ++bl) tmem_ld4(t_lane + bl * 64 + o0, v[bl]);
                tmem_ld_wait();
#pragma unroll
                for (int bl = 0; bl < 8; ++bl) tmem_ld_fence4(v[bl]);
                if (PASS == 2 && Kmul != nullptr && live) {
                    // y = sigma(K (.) M x) (first half of the M2 operator, Eq. 2): the 8 accumulators of one output index are 8
                    // consecutive k1 -> one 16-byte piece of the kernel row
                    const __nv_bfloat16* krow = Kmul + (size_t)((t0 + tt) % Hk) * 4096 + 16 * grp + 8 * set;
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) {
                        const uint4 kp = *reinterpret_cast<const uint4*>(krow + (o0 + kk) * 64);
                        const uint32_t kw[4] = {kp.x, kp.y, kp.z, kp.w};
#pragma unroll
                        for (int pp = 0; pp < 4; ++pp) {
                            float a = v[2 * pp][kk] * __uint_as_float(kw[pp] << 16);
                            float bb = v[2 * pp + 1][kk] * __uint_as_float(kw[pp] & 0xffff0000u);
                            v[2 * pp][kk] = relu ? fmaxf(a, 0.f) : a;
                            v[2 * pp + 1][kk] = relu ? fmaxf(bb, 0.f) : bb;
                        }
                    }
                }
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {
                    const uint4 pk = make_uint4(pack_bf16(v[0][kk], v[1][kk]), pack_bf16(v[2][kk], v[3][kk]),
                                                pack_bf16(v[4][kk], v[5][kk]), pack_bf16(v[6][kk], v[7][kk]));
                    if (PASS == 1)   // whole tiles of the workspace are written (rows past T are zeros)
                        *reinterpret_cast<uint4*>(dst + (size_t)(o0 + kk) * 8192) = pk;
                    else if (live)
                        *reinterpret_cast<uint4*>(dst + (size_t)(o0 + kk) * 128) = pk;
                }
            }
        }
        if (!ok && tid == 0) {
            atomicExch(status, (int32_t)M2_ERR_TIMEOUT);
            *abort_flag = 1;
        }
        // pass 1: the operand buffer is free (this tile's UMMAs are complete): the next tile's operands go in
        if (PASS == 1 && ok && next < nitems) store_a();
    }
    // teardown: nothing of ours may be in flight when the CTA goes away (only after a wait ran out can anything be left)
    if (PASS == 2 && tid == 0 && z_pending) mbar_wait(bar_in, z_par);
    if (tid == 32)
        for (int sl = 0; sl < 5; ++sl)
            if (fills[sl] > 0) mbar_wait(bar_full + 8 * sl, (uint32_t)(fills[sl] - 1) & 1u);
    tc_fence_before();
    __syncthreads();
    if (warp == 2) tmem_dealloc(*reinterpret_cast<volatile uint32_t*>(smem + tmem_slot), 512);
}

// ---- gradients with respect to the weight blocks ------------------------------------------------------------------
//
//   D_b[m][a] = sum_t Z_b[t][m] * V_b[t][a]        for the 64 blocks b, contraction over ALL tokens
//
// V = x or the upstream gradient g, read as [t][a][b] with the block index b contiguous (exactly what pass 1 reads), and
// Z = the intermediate in the workspace layout [token tile][m / 8][b][t % 128][m % 8] that pass 1 writes:
//   dR[n2][k1][n1] = sum_t dv[t][n2][k1] x[t][n1][n2]:  V = x (b = n2, a = n1),  Z = pass 1 of (g, L^T) (m = k1)
//   dL[k1][k2][n2] = sum_t g[t][k2][k1] v[t][n2][k1]:   V = g (b = k1, a = k2),  Z = pass 1 of (x, R)   (m = n2), D = dL[k1]^T
// With the tokens as the K dimension both operands lie in shared memory as the forward kernels already produce them: the
// 128-byte-swizzled tile [t][a] that pass 1 builds from 16-byte pieces of V is an N-major B operand (a row = one t), and a
// workspace block [t][8 m] is a column of M-major core matrices (8 consecutive t x 16 bytes) of the A operand.
// A CTA owns 8 consecutive blocks and one share of the 64-token half tiles, accumulates its 8 [64 x 64] partial results in
// TMEM (M = 64: rows in lanes 0..15 of every lane quarter) over its whole share and writes them once; a second kernel adds
// the shares in a fixed order.
constexpr int WG_OFF_X = 0;           // 8 operands [64 t][64 a] bf16, swizzled rows of 128 bytes            65536
constexpr int WG_OFF_Z = 65536;       // [m / 8][block 8][64 t][16 B]                                         65536
constexpr int WG_OFF_BAR = 131072;
constexpr int WG_SMEM = WG_OFF_BAR + 64;
constexpr int kWgSplits = 18;         // 8 block groups x 18 shares = 144 CTAs
constexpr size_t kWgPartialBytes = (size_t)kWgSplits * 64 * 4096 * 4;

__global__ void __launch_bounds__(kThreads, 1)
monarch64_wgrad_kernel(const __nv_bfloat16* __restrict__ in, const __nv_bfloat16* __restrict__ zin, float* __restrict__ partial,
                       long long T, int units, int32_t* __restrict__ status) {
    extern __shared__ __align__(1024) unsigned char smem[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t s_base = smem_u32(smem);
    const uint32_t bar_mma = s_base + WG_OFF_BAR, s_tptr = s_base + WG_OFF_BAR + 16, bar_in = s_base + WG_OFF_BAR + 24;
    const int grp = blockIdx.x, split = blockIdx.y, nsplit = gridDim.y;
    if (tid == 0) {
        mbar_init(bar_mma, 1);
        mbar_init(bar_in, 1);
        fence_barrier_init();
    }
    if (tid < 32) tmem_alloc(s_tptr, 512);
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");   // the workspace was written by the kernel before this one
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(smem + WG_OFF_BAR + 16);
    constexpr uint32_t IDESC = instr_desc_bf16(64, 64, true, true);
    uint32_t ph = 0;
    bool ok = true;
    int it = 0;
#pragma unroll 1
    for (int u = split; u < units; u += nsplit, ++it) {
        const int tile = u >> 1, half = u & 1;
        const long long t0 = (long long)tile * kTileT + half * 64;
        if (tid == 0) {   // 64 tokens of the 8 blocks' workspace columns: 64 pieces of 1 KB
            mbar_expect_tx(bar_in, 65536);
            const unsigned char* zb = reinterpret_cast<const unsigned char*>(zin) + (size_t)tile * (8 * 131072) + (size_t)grp * 16384 + half * 1024;
            for (int kc = 0; kc < 8; ++kc)
                for (int bl = 0; bl < 8; ++bl)
                    bulk_load(s_base + WG_OFF_Z + kc * 8192 + bl * 1024, zb + (size_t)kc * 131072 + bl * 2048, 1024, bar_in);
        }
        {   // one (token, group of 8 a) per thread: 8 pieces of 16 bytes, 8 x 8 transpose, 8 stores (see pass 1)
            const int g = tid & 7, tt = tid >> 3;
            uint4 v[8];
            const bool live = t0 + tt < T;
            const uint4* src = reinterpret_cast<const uint4*>(in + (size_t)(t0 + tt) * 4096 + (size_t)(8 * g) * 64 + grp * 8);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                v[i] = make_uint4(0u, 0u, 0u, 0u);
                if (live)
                    asm volatile("ld.global.cg.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v[i].x), "=r"(v[i].y), "=r"(v[i].z), "=r"(v[i].w) : "l"(src + i * 8));
            }
            const uint32_t* w = reinterpret_cast<const uint32_t*>(v);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                uint4 lo, hi;
                lo.x = prmt(w[0 * 4 + j], w[1 * 4 + j], 0x5410); hi.x = prmt(w[0 * 4 + j], w[1 * 4 + j], 0x7632);
                lo.y = prmt(w[2 * 4 + j], w[3 * 4 + j], 0x5410); hi.y = prmt(w[2 * 4 + j], w[3 * 4 + j], 0x7632);
                lo.z = prmt(w[4 * 4 + j], w[5 * 4 + j], 0x5410); hi.z = prmt(w[4 * 4 + j], w[5 * 4 + j], 0x7632);
                lo.w = prmt(w[6 * 4 + j], w[7 * 4 + j], 0x5410); hi.w = prmt(w[6 * 4 + j], w[7 * 4 + j], 0x7632);
                *reinterpret_cast<uint4*>(smem + WG_OFF_X + (2 * j) * 8192 + sw_off(tt, g)) = lo;
                *reinterpret_cast<uint4*>(smem + WG_OFF_X + (2 * j + 1) * 8192 + sw_off(tt, g)) = hi;
            }
        }
        fence_proxy_async();
        tc_fence_before();
        __syncthreads();
        if (tid == 0) {
            tc_fence_after();
            const bool in_ok = mbar_wait(bar_in, ph);
            if (in_ok) {
#pragma unroll 1
                for (int bl = 0; bl < kGroup; ++bl)
#pragma unroll
                    for (int s = 0; s < 4; ++s)   // 16 tokens per instruction
                        umma_f16(tmem + bl * 64, smem_desc(s_base + WG_OFF_Z + bl * 1024 + s * 256, 128, 8192),
                                 smem_desc_sw128(s_base + WG_OFF_X + bl * 8192 + s * 2048, 8192, 1024), IDESC, (it > 0 || s > 0) ? 1u : 0u);
            }
            umma_commit(bar_mma);
            if (!in_ok) atomicExch(status, (int32_t)M2_ERR_TIMEOUT);
        }
        ok = mbar_wait(bar_mma, ph);   // both operand buffers are free again
        ph ^= 1;
        tc_fence_after();
        if (!__syncthreads_and(ok)) {
            ok = false;
            break;
        }
    }
    // the 8 accumulators: row r of a block sits in lane (r % 16) of lane quarter r / 16; warpgroup wg takes blocks 2 wg, 2 wg + 1
    if (ok && it > 0) {
        const int q = warp & 3, wg = warp >> 2, r = 16 * q + lane;
        const uint32_t t_lane = tmem + ((uint32_t)(q * 32) << 16);
#pragma unroll 1
        for (int bb = 0; bb < 2; ++bb) {
            const int bl = 2 * wg + bb;
            float* dst = partial + (((size_t)split * 64 + grp * 8 + bl) * 64 + r) * 64;
#pragma unroll 1
            for (int c0 = 0; c0 < 64; c0 += 8) {
                float v[8];
                tmem_ld8(t_lane + bl * 64 + c0, v);
                tmem_ld_wait();
                tmem_ld_fence8(v);
                if (lane < 16) {
                    *reinterpret_cast<float4*>(dst + c0) = make_float4(v[0], v[1], v[2], v[3]);
                    *reinterpret_cast<float4*>(dst + c0 + 4) = make_float4(v[4], v[5], v[6], v[7]);
                }
            }
        }
    }
    if (!ok && tid == 0) atomicExch(status, (int32_t)M2_ERR_TIMEOUT);
    tc_fence_before();
    __syncthreads();
    if (tid < 32) tmem_dealloc(tmem, 512);
}

// out[b][i][j] = sum_s partial[s][b][i][j]  (transposed: partial[s][b][j][i]), shares added in index order
__global__ void wgrad_reduce_kernel(const float* __restrict__ partial, float* __restrict__ out, int nsplit, int transposed) {
    const int e = blockIdx.x * blockDim.x + threadIdx.x;   // < 64 * 4096
    const int b = e >> 12, i = (e >> 6) & 63, j = e & 63;
    const int src = transposed ? (b << 12) + (j << 6) + i : e;
    float acc = 0.f;
    for (int s = 0; s < nsplit; ++s) acc += partial[(size_t)s * (64 * 4096) + src];
    out[e] = acc;
}

int64_t wgrad_workspace_bytes(const m2_plan* pl, int64_t T) {
    return covered(pl) ? workspace_bytes(pl, T) + (int64_t)kWgPartialBytes + 64 * 4096 * 2 : 0;
}

int32_t wgrad(const m2_plan* pl, const void* X, const void* G, const void* L, const void* R, float* dL, float* dR, int64_t T, void* ws,
              cudaStream_t stream) {
    if (!covered(pl)) return M2_ERR_UNSUPPORTED;
    const int units = (int)(2 * ((T + kTileT - 1) / kTileT));
    const int nsplit = units < kWgSplits ? units : kWgSplits;
    unsigned char* zws = static_cast<unsigned char*>(ws);
    float* partial = reinterpret_cast<float*>(zws + workspace_bytes(pl, T));
    __nv_bfloat16* Lt = reinterpret_cast<__nv_bfloat16*>(zws + workspace_bytes(pl, T) + kWgPartialBytes);
    if (T == 0) {
        wgrad_reduce_kernel<<<1024, 256, 0, stream>>>(partial, dL, 0, 0);
        wgrad_reduce_kernel<<<1024, 256, 0, stream>>>(partial, dR, 0, 0);
        pl->launches += 2;
        return cudaGetLastError() == cudaSuccess ? M2_OK : M2_ERR_CUDA;
    }
    alignas(64) CUtensorMap unused;
    memset(&unused, 0, sizeof(unused));   // pass 1 never touches its map
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t p1 = {};
    p1.gridDim = dim3(8, (unsigned)((T + kTileT - 1) / kTileT));
    p1.blockDim = dim3(kThreads);
    p1.dynamicSmemBytes = SMEM_BYTES;
    p1.stream = stream;
    p1.attrs = attr;
    p1.numAttrs = 1;
    cudaLaunchConfig_t wg = p1;
    wg.gridDim = dim3(8, (unsigned)nsplit);
    wg.dynamicSmemBytes = WG_SMEM;
    const __nv_bfloat16 *x = (const __nv_bfloat16*)X, *g = (const __nv_bfloat16*)G;
    // dL: v = R-stage of x, then sum_t v (x) g per block k1
    if (cudaLaunchKernelEx(&p1, monarch64_pass_kernel<1>, x, (const __nv_bfloat16*)R, unused, (__nv_bfloat16*)zws, (long long)T, pl->d_status,
                           (const __nv_bfloat16*)nullptr, 1LL, 0) != cudaSuccess)
        return M2_ERR_CUDA;
    if (cudaLaunchKernelEx(&wg, monarch64_wgrad_kernel, g, (const __nv_bfloat16*)zws, partial, (long long)T, units, pl->d_status) != cudaSuccess)
        return M2_ERR_CUDA;
    wgrad_reduce_kernel<<<1024, 256, 0, stream>>>(partial, dL, nsplit, 1);
    // dR: dv = L^T-stage of g, then sum_t dv (x) x per block n2
    if (m2g::launch_blocks_transpose(L, Lt, 64, 64, 64, true, stream) != cudaSuccess) return M2_ERR_CUDA;
    if (cudaLaunchKernelEx(&p1, monarch64_pass_kernel<1>, g, (const __nv_bfloat16*)Lt, unused, (__nv_bfloat16*)zws, (long long)T, pl->d_status,
                           (const __nv_bfloat16*)nullptr, 1LL, 0) != cudaSuccess)
        return M2_ERR_CUDA;
    if (cudaLaunchKernelEx(&wg, monarch64_wgrad_kernel, x, (const __nv_bfloat16*)zws, partial, (long long)T, units, pl->d_status) != cudaSuccess)
        return M2_ERR_CUDA;
    wgrad_reduce_kernel<<<1024, 256, 0, stream>>>(partial, dR, nsplit, 0);
    if (cudaGetLastError() != cudaSuccess) return M2_ERR_CUDA;
    pl->last_kernel = "matmul_wgrad_umma_64x64";
    pl->launches += 7;
    return M2_OK;
}

bool covered(const m2_plan* pl) { return pl->dtype == M2_BF16 && pl->p == 2 && pl->dims[0] == 64 && pl->dims[1] == 64; }

// whole token tiles: the last tile's slab is written in full
int64_t workspace_bytes(const m2_plan* pl, int64_t T) { return covered(pl) ? ((T + kTileT - 1) / kTileT) * kTileT * 4096 * 2 : 0; }

cudaError_t prepare(const m2_plan* pl) {
    if (!covered(pl)) return cudaSuccess;
    cudaError_t e = cudaFuncSetAttribute(monarch64_pass_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(monarch64_pass_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(monarch64_wgrad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, WG_SMEM);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(monarch64_fwd_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, F_SMEM_BYTES);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(monarch64_fwd_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, F_SMEM_BYTES);
    return e;
}

// 128 tokens x 8 blocks per CTA (16-byte pieces): serves inputs that are only 16-byte aligned
static int32_t matmul_g8(const m2_plan* pl, const void* X, const void* L, const void* R, void* Y, int64_t T, void* ws, const void* Kmul,
               int64_t Hk, int relu, cudaStream_t stream) {
    if (!covered(pl)) return M2_ERR_UNSUPPORTED;
    if (T == 0) return M2_OK;
    dim3 grid(8, (unsigned)((T + kTileT - 1) / kTileT));
    // y[t][k2][k1] seen as (k1 64 | t, stride 8 KB | k2, stride 128 B); box = 8 k1 x 128 tokens x 64 k2
    alignas(64) CUtensorMap my;
    const cuuint64_t gdim[3] = {64, (cuuint64_t)T, 64}, gstr[2] = {8192, 128};
    const cuuint32_t box[3] = {8, (cuuint32_t)kTileT, 64};
    if (!tma_host::encode_bf16(&my, Y, 3, gdim, gstr, box)) return M2_ERR_UNSUPPORTED;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, monarch64_pass_kernel<1>, (const __nv_bfloat16*)X, (const __nv_bfloat16*)R, my, (__nv_bfloat16*)ws,
                           (long long)T, pl->d_status, (const __nv_bfloat16*)nullptr, 1LL, 0) != cudaSuccess)
        return M2_ERR_CUDA;
    if (cudaLaunchKernelEx(&cfg, monarch64_pass_kernel<2>, (const __nv_bfloat16*)ws, (const __nv_bfloat16*)L, my,
                           (__nv_bfloat16*)nullptr, (long long)T, pl->d_status, (const __nv_bfloat16*)Kmul, (long long)(Hk > 0 ? Hk : 1),
                           relu) != cudaSuccess)
        return M2_ERR_CUDA;
    pl->last_kernel = "matmul_umma_64x64_g8";
    pl->launches += 2;
    return M2_OK;
}

int32_t matmul(const m2_plan* pl, const void* X, const void* L, const void* R, void* Y, int64_t T, void* ws, const void* Kmul,
               int64_t Hk, int relu, cudaStream_t stream) {
    if (!covered(pl)) return M2_ERR_UNSUPPORTED;
    if (T == 0) return M2_OK;
    // the 32-byte loads of pass 1 want x on a 32-byte boundary (torch allocations are; a view need not be)
    if ((reinterpret_cast<uintptr_t>(X) & 31u) != 0) return matmul_g8(pl, X, L, R, Y, T, ws, Kmul, Hk, relu, stream);
    // weight blocks as TMA tiles: [64 blocks x 64 rows][64] bf16, one box = one block, 128-byte swizzle
    alignas(64) CUtensorMap mr, ml;
    const cuuint64_t gdim[2] = {64, 64 * 64}, gstr[1] = {128};
    const cuuint32_t box[2] = {64, 64};
    if (!tma_host::encode_sw128_bf16(&mr, R, 2, gdim, gstr, box) || !tma_host::encode_sw128_bf16(&ml, L, 2, gdim, gstr, box))
        return M2_ERR_UNSUPPORTED;
    cudaLaunchConfig_t cfg = {};
    int dev = 0, sms = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const long long nitems = 4 * ((T + kTile2 - 1) / kTile2);
    const long long ctas = (sms / 4) * 4 > 4 ? (sms / 4) * 4 : 4;   // a multiple of 4: a CTA keeps its block group
    cfg.gridDim = dim3((unsigned)(nitems < ctas ? nitems : ctas));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = F_SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, monarch64_fwd_kernel<1>, (const __nv_bfloat16*)X, mr, (__nv_bfloat16*)ws, (long long)T, pl->d_status,
                           (const __nv_bfloat16*)nullptr, 1LL, 0) != cudaSuccess)
        return M2_ERR_CUDA;
    if (cudaLaunchKernelEx(&cfg, monarch64_fwd_kernel<2>, (const __nv_bfloat16*)ws, ml, (__nv_bfloat16*)Y, (long long)T, pl->d_status,
                           (const __nv_bfloat16*)Kmul, (long long)(Hk > 0 ? Hk : 1), relu) != cudaSuccess)
        return M2_ERR_CUDA;
    pl->last_kernel = "matmul_umma_64x64";
    pl->launches += 2;
    return M2_OK;
}

}  // namespace m2mm
