// Tensor-core order-2 Monarch matmul for 64 x 64 blocks (N = 4096), bf16 in / fp32 accumulate / bf16 out.
//
//   y[t][k2*64 + k1] = sum_{n2} L[k1][k2][n2] * sum_{n1} R[n2][k1][n1] * x[t][n1*64 + n2]      (Sec. 3.1)
//
// Both block-diagonal factors are batches of 64 independent GEMMs [tokens x 64] x [64 x 64]; the batch
// index is the CONTIGUOUS index of the data each factor reads (n2 for R, k1 for L after the middle
// permutation), so neither operand of a tensor-core GEMM can be taken from memory as it lies.  The two
// factors therefore run as two passes that exchange the intermediate through a caller workspace.  Two
// generations of pass kernels live in this file:
//
//   monarch64_fwd_kernel<1|2>   the forward path (further down): 32 tokens x 16 blocks per item, 32-byte pieces,
//                               weights resident, loading / draining / issuing warps.
//   monarch64_pass_kernel<1|2>  128 tokens x 8 blocks per CTA, 16-byte pieces (described next): serves inputs that are
//                               only 16-byte aligned, and the weight gradients, whose kernel reads its workspace layout
//                               z[token tile][n2 / 8][k1][t % 128][n2 % 8]:
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

// ---- the forward passes: 32 tokens x 16 blocks per item ------------------------------------------------------------------
//
// The cost of both passes is the number of memory requests for the pieces of x (pass 1) and of y (pass 2) that a CTA owning
// g consecutive blocks touches: 2 g bytes of every 128-byte line.  With g = 16 a piece is a whole 32-byte sector.  An SM takes
// such requests at a fixed rate (and a warp that issues them is blocked while they queue), so everything else a tile needs
// runs underneath them, in other warps:
//
//   UMMA         the WEIGHT block is the A operand (M = 64 output indices, K = 64) and the tile's data the B operand (N = 32
//                tokens): D_b[out][t].  Row r of an M = 64 accumulator lives in TMEM lane (r % 16) + 32 (r / 16), so blocks
//                8..15 sit at lane offset 16 in the columns of blocks 0..7: a tile's 16 accumulators take 256 columns, and
//                the 512 columns hold TWO tiles -- the UMMAs of tile i run while the accumulators of tile i - 1 are drained.
//   weights      all 16 blocks of the CTA's group stay in shared memory (128 KB, one TMA tile per block, 128-byte swizzle =
//                the K-major operand image); the 16 operands of a 32-token tile take the other 64 KB.
//   roles        warps 0..7 load (global -> registers -> operand buffer), warps 8..15 drain (TMEM -> registers -> global),
//                lane 0 of warps 16 and 17 issues 8 blocks each (32 UMMAs, ~60 cycles of the thread's time per instruction,
//                about what the tensor core needs for them).  They meet only through mbarriers.
//   workspace    z[32-token tile][n2 / 16][t % 32][k1][n2 % 16]: 32-byte pieces with k1 running fastest.  In pass 1 lane l of a
//                draining warp holds output index k1 = 16 q + l % 16 of blocks 8 (l / 16) .. + 7, i.e. 16 bytes of a piece, and a
//                warp store is 512 contiguous bytes; in pass 2 the CTA (tile, k1 group) reads, for every (n2 / 16, t), 16 pieces
//                = 512 contiguous bytes, and a piece is 32 bytes of row t of the K-major operand of its block as it lies.
//   pass 1 in    one (token, 8 consecutive n1) per loading thread: 8 loads of 32 bytes, a 16 x 8 transpose in registers (PRMT;
//                this is P), 16 stores of 16 bytes into the swizzled operands B_{n2}[t][n1].
//   pass 2 out   y[t][k2][16 k1]: a thread's 8 accumulators of one token are 16 bytes, the lane 16 further holds the other half
//                of the sector.  Each draining warp stages [4 tokens][its 16 k2][32 B] in shared memory (the 32-byte-swizzled
//                image of a TMA box: no bank conflicts) and lane 0 sends it off with one tensor store (the last P): the 2048
//                sectors a tile scatters over 2048 lines never pass through the load/store unit, whose request rate is
//                what the loads need; rows past T are clipped by the tensor map.
constexpr int kTok = 32;                      // tokens per item
constexpr int kGroup2 = 16;                   // blocks per CTA
constexpr int F_OFF_A = 0;                    // 16 operands [32 t][64] bf16, swizzled rows of 128 bytes      65536
constexpr int F_OFF_W = 65536;                // 16 weight blocks [64][64] bf16, swizzled                     131072
constexpr int kLoadWarps = 8, kDrainWarps = 8, kIssueWarps = 2;
constexpr int F_OFF_ST = F_OFF_W + kGroup2 * 8192;    // pass 2: per draining warp two staging buffers [4 t][16 k2][32 B]  32768
constexpr int F_OFF_BAR = F_OFF_ST + kDrainWarps * 4096;   // bar_w, bar_mma[2], tmem ptr, abort flag, bar_opnd, bar_tfree[2]
constexpr int F_SMEM_BYTES = F_OFF_BAR + 64;
constexpr int kFwdThreads = 32 * (kLoadWarps + kDrainWarps + kIssueWarps);
constexpr size_t kTileBytes = (size_t)kTok * 8192;    // a tile of x, z or y
static_assert(F_SMEM_BYTES <= 232448, "shared-memory budget of the forward passes");

// PASS 1: in = x[T][64 n1][64 n2], weights R[n2][k1][n1], out = workspace z
// PASS 2: in = workspace z, weights L[k1][k2][n2], out = y[T][64 k2][64 k1] (optionally sigma(K (.) y))
//
// Persistent: CTA c of a grid that is a multiple of 4 walks the items c, c + grid, .. of (token tile, block group) pairs numbered
// group-fastest, so its block group is c % 4 for good (the weights stay) and the 4 CTAs that share a tile's lines work on it at
// the same time.  Tile i of a CTA uses accumulator set i % 2:
//   loading warps   wait for the UMMAs of tile i - 1 (operand buffer free), write tile i's operands from their registers, arrive on
//                   bar_opnd, request tile i + 1;
//   issuing threads wait for bar_opnd (operands of tile i) and bar_tfree[i % 2] (set drained of tile i - 2), issue, commit to
//                   bar_mma[i % 2];
//   draining warps  wait for bar_mma[i % 2], move the set to global memory, arrive on bar_tfree[i % 2].
template <int PASS>
__global__ void __launch_bounds__(kFwdThreads, 1)
monarch64_fwd_kernel(const __nv_bfloat16* __restrict__ in, const __grid_constant__ CUtensorMap map_w,
                     const __grid_constant__ CUtensorMap map_y, __nv_bfloat16* __restrict__ out, long long T,
                     int32_t* __restrict__ status, const __nv_bfloat16* __restrict__ Kmul, long long Hk, int relu, int selftest) {
    extern __shared__ __align__(1024) unsigned char smem[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t s_base = smem_u32(smem);
    const uint32_t bar_w = s_base + F_OFF_BAR, bar_mma = bar_w + 8, s_tptr = bar_w + 24, bar_opnd = bar_w + 40, bar_tfree = bar_w + 48;
    // selftest: the issuing threads issue and commit nothing and every wait for them gives up after a few polls, so that all
    // roles leave through their abort paths with nothing of theirs in flight
    const uint32_t wlim = selftest ? 64u : (1u << 22);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + F_OFF_BAR + 32);
    const int grp = blockIdx.x & 3;                                   // which 16 consecutive blocks (n2 in pass 1, k1 in pass 2)
    const long long ntiles = (T + kTok - 1) / kTok, nitems = 4 * ntiles;
    long long item = blockIdx.x;
    // pass 2 walks the tiles from the last to the first: what pass 1 wrote last is what the L2 still holds
    auto tile_of = [&](long long it) { return PASS == 1 ? it >> 2 : ntiles - 1 - (it >> 2); };
    if (tid == 0) {
        mbar_init(bar_w, 1);
        mbar_init(bar_mma, kIssueWarps);       // one arrival per issuing thread
        mbar_init(bar_mma + 8, kIssueWarps);
        mbar_init(bar_opnd, kLoadWarps);       // one arrival per loading warp
        mbar_init(bar_tfree, kDrainWarps);     // one arrival per draining warp
        mbar_init(bar_tfree + 8, kDrainWarps);
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tensormap(&map_w);
        if (PASS == 2) prefetch_tensormap(&map_y);
    }
    if (warp == 2) tmem_alloc(s_tptr, 512);
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    __syncthreads();   // barriers initialised before anyone arms them
    // the weights are the caller's and were complete before this call
    if (tid == 32) {
        mbar_expect_tx(bar_w, kGroup2 * 8192);
        for (int b = 0; b < kGroup2; ++b) tma_load_2d(s_base + F_OFF_W + b * 8192, &map_w, 0, (grp * kGroup2 + b) * 64, bar_w);
    }
    // this CTA's quarter of a tile's lines, pulled towards L2 as whole lines well before the pieces are read (the four CTAs that
    // share a tile ask for a quarter each).  L2 is where the previous kernel's writes land, so nothing stale can be fetched.
    auto prefetch_item = [&](long long it) {
        if (it < nitems) {
            const long long t0p = tile_of(it) * kTok;
            const long long rows = PASS == 2 || T - t0p >= kTok ? kTok : T - t0p;   // (whole tiles of the workspace exist)
            const long long share = rows * 8192 / 4;
            bulk_prefetch_l2(reinterpret_cast<const unsigned char*>(in) + t0p * 8192 + grp * share, (uint32_t)share);
        }
    };
    if (tid == 33) {
        prefetch_item(item);
        prefetch_item(item + gridDim.x);
    }
    // everything else (pass 1's z for pass 2, the producer of x, earlier readers of the buffers written here) is awaited now
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(smem + F_OFF_BAR + 24);
    uint32_t it_n = 0;        // tiles begun: tile it_n of this CTA uses accumulator set it_n % 2 and phase it_n / 2 of that set's barriers
    bool ok = true;
    auto timed_out = [&]() {
        atomicExch(status, (int32_t)M2_ERR_TIMEOUT);
        *abort_flag = 1;
    };

    if (warp < kLoadWarps) {
        // ---- loading warps: the 2048 pieces of an item, 8 per thread ----
        // Pass 1: (token tid / 8, n1 = 8 (tid % 8) + i), a piece = 16 consecutive n2; the quarter-warp that shared memory serves a
        // 16-byte store in writes the 8 chunks of one row: no bank conflicts.
        // Pass 2: (token 16 (warp / 4) + 8 (i / 4) + lane % 8, k1 = 4 (warp % 4) + lane / 8 of the group, n2 / 16 = i % 4): a warp reads 8
        // whole lines, and a quarter-warp stores to 8 different rows.
        const int t_in = PASS == 1 ? tid >> 3 : 16 * (warp >> 2) + (lane & 7);
        const int sub = PASS == 1 ? tid & 7 : 4 * (warp & 3) + (lane >> 3);
        uint32_t w[8][8];
        auto load_in = [&](long long it) {
            const long long tile = tile_of(it);
            if (PASS == 1) {
                const bool live = tile * kTok + t_in < T;
                const unsigned char* src =
                    reinterpret_cast<const unsigned char*>(in) + (size_t)(tile * kTok + t_in) * 8192 + (size_t)(8 * sub) * 128 + grp * 32;
#pragma unroll
                for (int i = 0; i < 8; ++i) {   // cached in L2 only: the rest of every line belongs to other SMs
                    if (live) {
                        asm volatile("ld.global.cg.v8.u32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                                     : "=r"(w[i][0]), "=r"(w[i][1]), "=r"(w[i][2]), "=r"(w[i][3]), "=r"(w[i][4]), "=r"(w[i][5]), "=r"(w[i][6]), "=r"(w[i][7])
                                     : "l"(src + i * 128));
                    } else {
#pragma unroll
                        for (int m = 0; m < 8; ++m) w[i][m] = 0u;
                    }
                }
            } else {   // whole tiles of the workspace were written
                const unsigned char* src =
                    reinterpret_cast<const unsigned char*>(in) + (size_t)tile * kTileBytes + (size_t)t_in * 2048 + (size_t)(16 * grp + sub) * 32;
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    asm volatile("ld.global.cg.v8.u32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                                 : "=r"(w[i][0]), "=r"(w[i][1]), "=r"(w[i][2]), "=r"(w[i][3]), "=r"(w[i][4]), "=r"(w[i][5]), "=r"(w[i][6]), "=r"(w[i][7])
                                 : "l"(src + (size_t)(i & 3) * 65536 + (size_t)(i >> 2) * (8 * 2048)));
            }
        };
        auto store_opnd = [&]() {
            if (PASS == 1) {   // the 16 x 8 transpose in registers (this is P): 16 bytes = 8 consecutive n1 of one (t, n2)
                unsigned char* dst = smem + F_OFF_A + sw_off(t_in, sub);
#pragma unroll
                for (int m = 0; m < 8; ++m) {
                    uint4 lo, hi;
                    lo.x = prmt(w[0][m], w[1][m], 0x5410); hi.x = prmt(w[0][m], w[1][m], 0x7632);
                    lo.y = prmt(w[2][m], w[3][m], 0x5410); hi.y = prmt(w[2][m], w[3][m], 0x7632);
                    lo.z = prmt(w[4][m], w[5][m], 0x5410); hi.z = prmt(w[4][m], w[5][m], 0x7632);
                    lo.w = prmt(w[6][m], w[7][m], 0x5410); hi.w = prmt(w[6][m], w[7][m], 0x7632);
                    *reinterpret_cast<uint4*>(dst + (2 * m) * 4096) = lo;
                    *reinterpret_cast<uint4*>(dst + (2 * m + 1) * 4096) = hi;
                }
            } else {           // a piece is 32 bytes of row t of block k1's operand as it lies
                unsigned char* dst = smem + F_OFF_A + sub * 4096;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int t = t_in + 8 * (i >> 2), c = 2 * (i & 3);
                    *reinterpret_cast<uint4*>(dst + sw_off(t, c)) = make_uint4(w[i][0], w[i][1], w[i][2], w[i][3]);
                    *reinterpret_cast<uint4*>(dst + sw_off(t, c + 1)) = make_uint4(w[i][4], w[i][5], w[i][6], w[i][7]);
                }
            }
        };
        if (item < nitems) load_in(item);
#pragma unroll 1
        for (; item < nitems; item += gridDim.x, ++it_n) {
            if (__any_sync(~0u, *abort_flag != 0)) break;
            // the UMMAs of the previous tile have read the operand buffer
            if (it_n > 0) ok = __all_sync(~0u, mbar_wait(bar_mma + 8 * ((it_n - 1u) & 1u), ((it_n - 1u) >> 1) & 1u, wlim));
            if (!ok) break;
            store_opnd();
            fence_proxy_async();   // operands visible to the tensor core
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_opnd);
            // the next tile's pieces are requested now and arrive while this one is computed
            if (item + gridDim.x < nitems) load_in(item + gridDim.x);
            if (tid == 33) prefetch_item(item + 2 * (long long)gridDim.x);
        }
        if (!ok && lane == 0) timed_out();
    } else if (warp < kLoadWarps + kDrainWarps) {
        // ---- draining warps: lane l of lane quarter q = warp % 4 holds output index 16 q + (l & 15) of blocks 8 (l >> 4) .. + 7; the two
        // warps of a quarter split the 32 tokens.  For every token the 8 accumulators of a thread are 8 consecutive block indices:
        // one 16-byte piece. ----
        const int q = warp & 3, c2 = (warp - kLoadWarps) >> 2, r = 16 * q + (lane & 15), set = lane >> 4;
#pragma unroll 1
        for (; item < nitems; item += gridDim.x, ++it_n) {
            if (__any_sync(~0u, *abort_flag != 0)) break;
            const uint32_t p = it_n & 1u;
            const long long tile = tile_of(item), t0 = tile * kTok + 16 * c2;
            ok = __all_sync(~0u, mbar_wait(bar_mma + 8 * p, (it_n >> 1) & 1u, wlim));
            if (!ok) break;
            tc_fence_after();
            const uint32_t t_lane = tmem + ((uint32_t)(q * 32) << 16) + p * 256u + 16u * c2;
            // pass 1: z[tile][grp][t][k1][32 B], straight from registers, 512 contiguous bytes per warp store
            unsigned char* dst = reinterpret_cast<unsigned char*>(out) + (size_t)tile * kTileBytes + (size_t)grp * 65536 + (size_t)(16 * c2) * 2048 + r * 32 + set * 16;
            // pass 2: this warp's staging buffers; chunk (16 bytes) index XOR bit 7 of the address = the 32-byte swizzle of the box
            const uint32_t st_warp = F_OFF_ST + (uint32_t)(warp - kLoadWarps) * 4096u;
            const uint32_t st_lane = (uint32_t)(lane & 15) * 32u + (uint32_t)((set ^ ((lane >> 2) & 1)) << 4);
#pragma unroll 1
            for (int h = 0; h < 4; ++h) {
                float v[8][4];
#pragma unroll
                for (int bl = 0; bl < 8; ++bl) tmem_ld4(t_lane + bl * 32 + 4 * h, v[bl]);
                if (PASS == 2) {   // the buffer of two rounds ago has been read by its store
                    if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                    __syncwarp();
                }
                tmem_ld_wait();
#pragma unroll
                for (int bl = 0; bl < 8; ++bl) tmem_ld_fence4(v[bl]);
                if (PASS == 2 && Kmul != nullptr) {
                    // y = sigma(K (.) M x) (first half of the M2 operator, Eq. 2): the 8 accumulators of one token are 8 consecutive k1
                    // -> one 16-byte piece of the kernel row
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) {
                        const long long t = t0 + 4 * h + kk;
                        if (t < T) {
                            const uint4 kp = *reinterpret_cast<const uint4*>(Kmul + (size_t)(t % Hk) * 4096 + r * 64 + 16 * grp + 8 * set);
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
                }
                unsigned char* stg = smem + st_warp + (uint32_t)(h & 1) * 2048u + st_lane;
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {
                    const uint4 pk = make_uint4(pack_bf16(v[0][kk], v[1][kk]), pack_bf16(v[2][kk], v[3][kk]),
                                                pack_bf16(v[4][kk], v[5][kk]), pack_bf16(v[6][kk], v[7][kk]));
                    if (PASS == 1)   // whole tiles of the workspace are written (rows past T are zeros)
                        *reinterpret_cast<uint4*>(dst + (size_t)(4 * h + kk) * 2048) = pk;
                    else
                        *reinterpret_cast<uint4*>(stg + kk * 512) = pk;
                }
                if (PASS == 2) {
                    fence_proxy_async();   // staged rows visible to the copy engine
                    __syncwarp();
                    if (lane == 0 && t0 + 4 * h < T) {   // (a box that starts past T has nothing to store)
                        tma_store_3d(&map_y, s_base + st_warp + (uint32_t)(h & 1) * 2048u, 16 * grp, 16 * q, (int)(t0 + 4 * h));
                        tma_store_commit();
                    }
                }
            }
            // the set may be overwritten: this warp's TMEM loads are complete
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_tfree + 8 * p);
        }
        if (PASS == 2 && lane == 0) tma_store_wait_all0();   // this thread's stores are complete before shared memory goes away
        if (!ok && lane == 0) timed_out();
    } else if (lane == 0) {
        // ---- issuing threads ----
        constexpr uint32_t IDESC = instr_desc_bf16(64, kTok, false, false);
        constexpr int kPer = kGroup2 / kIssueWarps;
        const int b0 = (warp - kLoadWarps - kDrainWarps) * kPer;
        ok = mbar_wait(bar_w, 0);
#pragma unroll 1
        for (; item < nitems && ok && *abort_flag == 0; item += gridDim.x, ++it_n) {
            const uint32_t p = it_n & 1u;
            ok = mbar_wait(bar_opnd, p, wlim);
            if (ok && it_n >= 2) ok = mbar_wait(bar_tfree + 8 * p, ((it_n - 2u) >> 1) & 1u, wlim);
            if (!ok) break;
            if (selftest) continue;
            tc_fence_after();
#pragma unroll 1
            for (int b = b0; b < b0 + kPer; ++b) {
                const uint32_t d = tmem + ((uint32_t)(16 * (b >> 3)) << 16) + p * 256u + (uint32_t)(b & 7) * kTok;
                const uint64_t ad = smem_desc_sw128(s_base + F_OFF_W + b * 8192, 16, 1024);
                const uint64_t bd = smem_desc_sw128(s_base + F_OFF_A + b * 4096, 16, 1024);
#pragma unroll
                for (int s = 0; s < 4; ++s) umma_f16(d, ad + s * 2, bd + s * 2, IDESC, s > 0);   // K step of 16: 32 bytes of a swizzled row
            }
            umma_commit(bar_mma + 8 * p);
        }
        if (!ok) timed_out();
    }
    // teardown: the weight copy is the only thing that can still be in flight (after a wait ran out)
    if (tid == 32) mbar_wait(bar_w, 0);
    tc_fence_before();
    __syncthreads();
    if (warp == 2) tmem_dealloc(tmem, 512);
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

static int32_t matmul_impl(const m2_plan* pl, const void* X, const void* L, const void* R, void* Y, int64_t T, void* ws, const void* Kmul,
                           int64_t Hk, int relu, int selftest, cudaStream_t stream) {
    if (!covered(pl)) return M2_ERR_UNSUPPORTED;
    if (T == 0) return selftest ? M2_ERR_UNSUPPORTED : M2_OK;
    // the 32-byte loads of pass 1 want x on a 32-byte boundary (torch allocations are; a view need not be)
    if ((reinterpret_cast<uintptr_t>(X) & 31u) != 0)
        return selftest ? M2_ERR_UNSUPPORTED : matmul_g8(pl, X, L, R, Y, T, ws, Kmul, Hk, relu, stream);
    // weight blocks as TMA tiles: [64 blocks x 64 rows][64] bf16, one box = one block, 128-byte swizzle
    alignas(64) CUtensorMap mr, ml, my;
    const cuuint64_t gdim[2] = {64, 64 * 64}, gstr[1] = {128};
    const cuuint32_t box[2] = {64, 64};
    if (!tma_host::encode_sw128_bf16(&mr, R, 2, gdim, gstr, box) || !tma_host::encode_sw128_bf16(&ml, L, 2, gdim, gstr, box))
        return M2_ERR_UNSUPPORTED;
    // y[t][k2][k1] seen as (k1 64 | k2, stride 128 B | t, stride 8 KB); box = 16 k1 x 16 k2 x 4 tokens, 32-byte swizzle
    const cuuint64_t ydim[3] = {64, 64, (cuuint64_t)T}, ystr[2] = {128, 8192};
    const cuuint32_t ybox[3] = {16, 16, 4};
    if (!tma_host::encode_sw32_bf16(&my, Y, 3, ydim, ystr, ybox)) return M2_ERR_UNSUPPORTED;
    cudaLaunchConfig_t cfg = {};
    int dev = 0, sms = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const long long nitems = 4 * ((T + kTok - 1) / kTok);
    const long long ctas = (sms / 4) * 4 > 4 ? (sms / 4) * 4 : 4;   // a multiple of 4: a CTA keeps its block group
    cfg.gridDim = dim3((unsigned)(nitems < ctas ? nitems : ctas));
    cfg.blockDim = dim3(kFwdThreads);
    cfg.dynamicSmemBytes = F_SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, monarch64_fwd_kernel<1>, (const __nv_bfloat16*)X, mr, my, (__nv_bfloat16*)ws, (long long)T, pl->d_status,
                           (const __nv_bfloat16*)nullptr, 1LL, 0, selftest) != cudaSuccess)
        return M2_ERR_CUDA;
    if (cudaLaunchKernelEx(&cfg, monarch64_fwd_kernel<2>, (const __nv_bfloat16*)ws, ml, my, (__nv_bfloat16*)Y, (long long)T, pl->d_status,
                           (const __nv_bfloat16*)Kmul, (long long)(Hk > 0 ? Hk : 1), relu, selftest) != cudaSuccess)
        return M2_ERR_CUDA;
    pl->last_kernel = "matmul_umma_64x64";
    pl->launches += 2;
    return M2_OK;
}

int32_t matmul(const m2_plan* pl, const void* X, const void* L, const void* R, void* Y, int64_t T, void* ws, const void* Kmul,
               int64_t Hk, int relu, cudaStream_t stream) {
    return matmul_impl(pl, X, L, R, Y, T, ws, Kmul, Hk, relu, 0, stream);
}

int32_t matmul_wait_selftest(const m2_plan* pl, const void* X, const void* L, const void* R, void* Y, int64_t T, void* ws,
                             cudaStream_t stream) {
    return matmul_impl(pl, X, L, R, Y, T, ws, nullptr, 1, 0, 1, stream);
}

}  // namespace m2mm
