// Tensor-core block-diagonal MLP of the M2 block (Eq. 3 with block-diagonal M_3, M_4; Sec. 5.1: M2-BERT's dense
// layers replaced by block-diagonal ones):  y_j = W_down[j] GELU(W_up[j] z_j)  per token and block j, erf-form GELU,
// for blocks of 192 inputs / 768 hidden / 192 outputs (d = 768, 4 blocks, expansion 4).  bf16 operands, fp32
// accumulation in TMEM, the hidden activations are rounded to bf16 and never leave the SM.
//
// An item = 128 tokens x one block.  The hidden dimension is walked in 6 chunks of 128:
//   S1(c)  D1[c % 2][128 tok][128 hid] = Z[128][192] * W_up[j][chunk c]^T        12 UMMAs (M128 N128 K16)
//   E1(c)  TMEM -> registers -> GELU -> bf16 -> back into TMEM, over the first 64 columns of the D1 buffer it came from
//          (two values per column): G[128 tok][128 hid] is the A operand of S2 and never touches shared memory
//   S2(c)  D2[128 tok][192 out] += G * W_down[j][:, chunk c]^T                     8 UMMAs (M128 N192 K16, A from TMEM)
// and at the end of an item D2 -> bf16 -> staging -> TMA stores.
//
// Persistent: one CTA per SM walks the items c, c + grid, ..; all barriers count chunks across items, so the weight
// chunks, the activations and the first UMMAs of the next item are under way while the GELU warps finish and store the
// current one (a CTA per item spent a third of its time launching, setting up and draining).  Warp roles: warp 0 feeds
// the activation tiles and the weight chunks by TMA (W_up chunks double-buffered), warp 1 issues the UMMAs and runs
// S1(c + 1) ahead of E1(c) (two D1 buffers), warps 2..17 are the GELU warps (lane quarter = warp % 4, 32 of the 128
// chunk columns each).  Shared-memory operands are K-major with the 128-byte swizzle, written by TMA.  Every wait is
// bounded; a role that gave up keeps arriving at the GELU warps' block barriers so that nobody is left behind.
#include <cuda.h>

#include <atomic>
#include <cuda_bf16.h>

#include "mlp_umma.h"
#include "ptx_sm100.cuh"
#include "tma_host.h"

namespace m2mlp {

using namespace sm100;

constexpr int kCI = 192, kHID = 768, kCO = 192, kChunk = 128, kChunks = kHID / kChunk, kTileT = 128;
constexpr int kEpiWarps = 16, kThreads = 64 + 32 * kEpiWarps;
constexpr int OFF_Z = 0;                    // 3 K-blocks [128][64] bf16                               49152
constexpr int OFF_W1 = 49152;               // 2 buffers x 3 K-blocks [128 hid][64]                   98304
constexpr int OFF_W2 = 147456;              // 2 K-blocks [192 out][64]                               49152
constexpr int OFF_ST = 196608;              // output staging: 2 buffers [128 tok][64]                32768
constexpr int OFF_BAR = 229376;
constexpr int SMEM_BYTES = OFF_BAR + 192;
static_assert(SMEM_BYTES <= 232448, "shared memory budget");
// mbarriers (8 bytes each) from OFF_BAR
enum { B_Z = 0, B_W1F = 1, B_W1E = 3, B_W2F = 5, B_W2E = 6, B_D1F = 7, B_D1E = 9, B_GF = 11, B_ZE = 12, B_D2F = 13, B_D2E = 14, B_COUNT = 15 };

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
                 "l"(map), "r"(c0), "r"(c1), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(dst),
                 "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
// GELU(v) = v Phi(v), Phi the standard normal distribution function = (1 + erf(v / sqrt 2)) / 2.  Phi(v) - 1/2 is odd:
// Phi(v) = 1/2 + v Q(v^2) with Q a degree-9 polynomial in x = v^2 / 8 - 1 fitted on |v| <= 4 (Chebyshev least squares);
// beyond 4 the argument is clamped (Phi(4) = 1 - 3e-5).  Absolute error of GELU 2.3e-5 inside, <= 4e-5 |v| outside:
// far below the bf16 rounding of the hidden activations.  Two neighbouring values are evaluated together with packed
// fp32 arithmetic: 13 packed and 4 scalar instructions per pair, nothing on the special-function unit.
__device__ __forceinline__ void gelu2(float v0, float v1, float& g0, float& g1) {
    const float c0 = fminf(fmaxf(v0, -4.0f), 4.0f), c1 = fminf(fmaxf(v1, -4.0f), 4.0f);
    const uint64_t vc = pk2(c0, c1);
    const uint64_t x = fma2(mul2(vc, vc), pk2(0.125f, 0.125f), pk2(-1.0f, -1.0f));
    uint64_t q = pk2(-0.0006410883506760001f, -0.0006410883506760001f);
    q = fma2(q, x, pk2(0.0015863177832216024f, 0.0015863177832216024f));
    q = fma2(q, x, pk2(-0.002556844847276807f, -0.002556844847276807f));
    q = fma2(q, x, pk2(0.005862586200237274f, 0.005862586200237274f));
    q = fma2(q, x, pk2(-0.012616137973964214f, -0.012616137973964214f));
    q = fma2(q, x, pk2(0.02264878712594509f, 0.02264878712594509f));
    q = fma2(q, x, pk2(-0.03683827072381973f, -0.03683827072381973f));
    q = fma2(q, x, pk2(0.05591851472854614f, 0.05591851472854614f));
    q = fma2(q, x, pk2(-0.08432330191135406f, -0.08432330191135406f));
    q = fma2(q, x, pk2(0.1759500801563263f, 0.1759500801563263f));
    const uint64_t phi = fma2(vc, q, pk2(0.5f, 0.5f));
    upk2(mul2(pk2(v0, v1), phi), g0, g1);
}
__device__ __forceinline__ uint32_t gelu2_pack(float v0, float v1) {
    float g0, g1;
    gelu2(v0, v1, g0, g1);
    return pack_bf16(g0, g1);
}
// byte offset of 16-byte chunk kc of row r in a K-major block with 128-byte rows and the 128B swizzle
__device__ __forceinline__ uint32_t sw_off(int r, int kc) { return (uint32_t)((r >> 3) * 1024 + (r & 7) * 128 + ((kc ^ (r & 7)) << 4)); }

// ZCF: the activations arrive channel-first, z[b][c][t] (T positions per batch entry, a multiple of 128), as the sequence mixer
// leaves them: an item's tile is then two boxes [192 channels][64 tokens], the tokens contiguous -- as they lie the two 64-token
// blocks of an M-major A operand (K = the channels) -- and nothing has to be transposed between the mixer and the MLP.
template <bool ZCF>
__global__ void __launch_bounds__(kThreads, 1)
mlp_umma_kernel(const __grid_constant__ CUtensorMap map_z, const __grid_constant__ CUtensorMap map_w1,
                const __grid_constant__ CUtensorMap map_w2, const __grid_constant__ CUtensorMap map_y, int32_t* __restrict__ status,
                int nblk, int nitems, int T) {
    extern __shared__ __align__(1024) unsigned char smem[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t s_base = smem_u32(smem);
    const uint32_t bars = s_base + OFF_BAR, s_tptr = s_base + OFF_BAR + 8 * B_COUNT;
    auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
    // this CTA's items: item(q) = blockIdx.x + q * gridDim.x  ->  block j = item % nblk, token tile = item / nblk
    const int nq = ((int)blockIdx.x < nitems) ? (nitems - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
    const int total = nq * kChunks;                // chunks of all items, counted through by every role
    auto item_j = [&](int q) { return (int)((blockIdx.x + (unsigned)q * gridDim.x) % (unsigned)nblk); };
    auto item_t0 = [&](int q) { return (int)((blockIdx.x + (unsigned)q * gridDim.x) / (unsigned)nblk) * kTileT; };

    if (tid == 0) {
        mbar_init(bar(B_Z), 1);
        mbar_init(bar(B_ZE), 1);
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar(B_W1F + i), 1);
            mbar_init(bar(B_W1E + i), 1);
            mbar_init(bar(B_D1F + i), 1);
            mbar_init(bar(B_D1E + i), kEpiWarps);   // one arrival per GELU warp
        }
        mbar_init(bar(B_W2F), 1);
        mbar_init(bar(B_W2E), 1);
        mbar_init(bar(B_GF), kEpiWarps);
        mbar_init(bar(B_D2F), 1);
        mbar_init(bar(B_D2E), kEpiWarps);
        fence_barrier_init();
        prefetch_tensormap(&map_z);
        prefetch_tensormap(&map_w1);
        prefetch_tensormap(&map_w2);
        prefetch_tensormap(&map_y);
    }
    if (warp == 1) tmem_alloc(s_tptr, 512);
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    asm volatile("griddepcontrol.wait;" ::: "memory");   // the producer of z (and earlier readers of y) are done
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(smem + OFF_BAR + 8 * B_COUNT);
    const uint32_t D1 = tmem, D2 = tmem + 256;            // D1 buffers at columns 0 and 128, D2 at 256..447
    bool ok = true;

    if (warp == 0) {
        // ---- TMA producer: three streams that advance independently (activation tiles, W_up chunks two ahead of the
        //      UMMAs, the single W_down buffer as soon as S2 has read it), so none waits behind another's barrier ----
        if (lane == 0) {
            int zq = 0, g1 = 0, g2 = 0;
            uint32_t idle = 0;
            while ((zq < nq || g1 < total || g2 < total) && idle < (1u << 22)) {
                bool progressed = false;
                if (zq < nq && (zq < 1 || mbar_try_wait(bar(B_ZE), (zq - 1) & 1))) {                                  // the last S1 of item zq - 1 has read Z
                    mbar_expect_tx(bar(B_Z), 49152);
                    if (ZCF) {
                        const int tt = item_t0(zq);
                        for (int mb = 0; mb < 2; ++mb)
                            tma_load_3d(s_base + OFF_Z + mb * 24576, &map_z, tt % T + 64 * mb, item_j(zq) * kCI, tt / T, bar(B_Z));
                    } else {
                        for (int kb = 0; kb < 3; ++kb)
                            tma_load_2d(s_base + OFF_Z + kb * 16384, &map_z, item_j(zq) * kCI + kb * 64, item_t0(zq), bar(B_Z));
                    }
                    ++zq;
                    progressed = true;
                }
                if (g1 < total && (g1 < 2 || mbar_try_wait(bar(B_W1E + (g1 & 1)), ((g1 >> 1) - 1) & 1))) {            // S1(g1 - 2) has read the buffer
                    const int bb = g1 & 1, c = g1 % kChunks, jj = item_j(g1 / kChunks);
                    mbar_expect_tx(bar(B_W1F + bb), 49152);
                    for (int kb = 0; kb < 3; ++kb)
                        tma_load_2d(s_base + OFF_W1 + bb * 49152 + kb * 16384, &map_w1, kb * 64, jj * kHID + c * kChunk, bar(B_W1F + bb));
                    ++g1;
                    progressed = true;
                }
                if (g2 < total && (g2 < 1 || mbar_try_wait(bar(B_W2E), (g2 - 1) & 1))) {                               // S2(g2 - 1) has read the chunk
                    const int c = g2 % kChunks, jj = item_j(g2 / kChunks);
                    mbar_expect_tx(bar(B_W2F), 49152);
                    for (int kb = 0; kb < 2; ++kb)
                        tma_load_2d(s_base + OFF_W2 + kb * 24576, &map_w2, c * kChunk + kb * 64, jj * kCO, bar(B_W2F));
                    ++g2;
                    progressed = true;
                }
                idle = progressed ? 0 : idle + 1;
            }
            if (zq < nq || g1 < total || g2 < total) ok = false;
        }
    } else if (warp == 1) {
        // ---- UMMA issuer ---------------------------------------------------------------------------------------------
        if (lane == 0) {
            constexpr uint32_t ID1 = instr_desc_bf16(128, 128, ZCF, false), ID2 = instr_desc_bf16(128, 192, false, false);
            auto s1 = [&](int g) {   // D1[g % 2] = Z * W_up chunk g
                const int b = g & 1;
                ok = mbar_wait(bar(B_W1F + b), (g >> 1) & 1);
                if (ok && g >= 2) ok = mbar_wait(bar(B_D1E + b), ((g >> 1) - 1) & 1);   // the GELU warps have read D1[b]
                if (!ok) return;
                tc_fence_after();
#pragma unroll 1
                for (int kb = 0; kb < 3; ++kb)
#pragma unroll
                    for (int s = 0; s < 4; ++s)
                        umma_f16(D1 + b * 128,
                                 ZCF ? smem_desc_sw128(s_base + OFF_Z + (kb * 4 + s) * 2048, 24576, 1024)   // 16 channels = 16 rows of 128 bytes
                                     : smem_desc_sw128(s_base + OFF_Z + kb * 16384 + s * 32, 16, 1024),
                                 smem_desc_sw128(s_base + OFF_W1 + b * 49152 + kb * 16384 + s * 32, 16, 1024), ID1, (kb | s) != 0);
                umma_commit(bar(B_D1F + b));
                umma_commit(bar(B_W1E + b));
                if (g % kChunks == kChunks - 1) umma_commit(bar(B_ZE));   // the item's last S1: its activation tile is free after it
            };
            if (total > 0) {
                ok = mbar_wait(bar(B_Z), 0);
                if (ok) s1(0);
            }
            for (int g = 0; g < total && ok; ++g) {
                const int c = g % kChunks, q = g / kChunks;
                if (c + 1 < kChunks) s1(g + 1);
                if (!ok) break;
                ok = mbar_wait(bar(B_GF), g & 1) && mbar_wait(bar(B_W2F), g & 1);
                if (ok && c == 0 && q > 0) ok = mbar_wait(bar(B_D2E), (q - 1) & 1);   // the previous item's D2 has been read
                if (!ok) break;
                tc_fence_after();
                // A = G in tensor memory: the first 64 columns of D1[g % 2], 8 columns per K step of 16
#pragma unroll 1
                for (int kb = 0; kb < 2; ++kb)
#pragma unroll
                    for (int s = 0; s < 4; ++s)
                        umma_f16_ta(D2, D1 + (g & 1) * 128 + (kb * 4 + s) * 8,
                                    smem_desc_sw128(s_base + OFF_W2 + kb * 24576 + s * 32, 16, 1024), ID2, (c | kb | s) != 0);
                umma_commit(bar(B_W2E));
                if (c == kChunks - 1) {
                    umma_commit(bar(B_D2F));
                    if (g + 1 < total) {   // the next item's first S1 follows this item's last S2
                        ok = mbar_wait(bar(B_Z), (q + 1) & 1);
                        if (ok) s1(g + 1);
                    }
                }
            }
        }
    } else {
        // ---- GELU warps: lane quarter qq = warp % 4 (a TMEM rule), column slice sl = 32 of the chunk's 128 columns ----
        const int ew = warp - 2, qq = warp & 3, sl = ew >> 2;
        const int row = qq * 32 + lane;                                   // token within the tile
        const uint32_t t_lane = tmem + ((uint32_t)(qq * 32) << 16);
        const bool storer = ew == 0 && lane == 0;                         // issues the output stores
        for (int g = 0; g < total; ++g) {
            const int b = g & 1, c = g % kChunks, q = g / kChunks;
            if (ok) ok = mbar_wait(bar(B_D1F + b), (g >> 1) & 1);
            if (ok) {
                tc_fence_after();
                float v[32];
#pragma unroll
                for (int i = 0; i < 4; ++i) tmem_ld8(t_lane + b * 128 + sl * 32 + 8 * i, v + 8 * i);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 4; ++i) tmem_ld_fence8(v + 8 * i);
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(B_D1E + b));                  // this warp has read its part of D1[b]
                uint32_t pk[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) pk[i] = gelu2_pack(v[2 * i], v[2 * i + 1]);
                // G goes back into tensor memory over the first 64 columns of D1[b]: every GELU warp must have read the buffer
                ok = mbar_wait(bar(B_D1E + b), (g >> 1) & 1);
                if (ok) {
                    tc_fence_after();
                    tmem_st8(t_lane + b * 128 + sl * 16, pk);
                    tmem_st8(t_lane + b * 128 + sl * 16 + 8, pk + 8);
                    tmem_st_wait();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar(B_GF));
                }
            }
            if (c != kChunks - 1) continue;
            // ---- output of item q: D2 -> bf16 -> staging -> TMA stores.  The 24 chunks (16 bytes) of a 192-column row
            //      belong to three K-blocks of 64 columns; K-blocks 0 and 1 are staged in the two 16 KB buffers and sent,
            //      K-block 2 follows in the first buffer once its store has read it.  The block barriers are passed by
            //      every GELU warp whatever happened before. ----
            if (ok) ok = mbar_wait(bar(B_D2F), q & 1);
            uint4 keep[6];
            if (ok) {
                tc_fence_after();
#pragma unroll
                for (int h = 0; h < 2; ++h) {                                // 48 of the 192 output columns per slice: 6 chunks
                    float w[24];
#pragma unroll
                    for (int i = 0; i < 3; ++i) tmem_ld8(t_lane + 256 + sl * 48 + h * 24 + 8 * i, w + 8 * i);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 3; ++i) tmem_ld_fence8(w + 8 * i);
#pragma unroll
                    for (int i = 0; i < 3; ++i)
                        keep[h * 3 + i] = make_uint4(pack_bf16(w[8 * i], w[8 * i + 1]), pack_bf16(w[8 * i + 2], w[8 * i + 3]),
                                                     pack_bf16(w[8 * i + 4], w[8 * i + 5]), pack_bf16(w[8 * i + 6], w[8 * i + 7]));
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(B_D2E));                      // D2 may be overwritten by the next item
            }
            if (storer) tma_store_wait_read0();                              // the previous item's stores have read the staging buffers
            asm volatile("bar.sync 1, %0;" ::"n"(32 * kEpiWarps) : "memory");
            if (ok) {
#pragma unroll
                for (int i = 0; i < 6; ++i) {
                    const int kc = sl * 6 + i;                               // 16-byte chunk of the 192-column row
                    if (kc < 16) *reinterpret_cast<uint4*>(smem + OFF_ST + (kc >> 3) * 16384 + sw_off(row, kc & 7)) = keep[i];
                }
                fence_proxy_async();
            }
            asm volatile("bar.sync 1, %0;" ::"n"(32 * kEpiWarps) : "memory");
            if (storer && ok) {
                for (int kb = 0; kb < 2; ++kb) tma_store_2d(&map_y, s_base + OFF_ST + kb * 16384, item_j(q) * kCO + kb * 64, item_t0(q));
                tma_store_commit();
                tma_store_wait_read0();
            }
            asm volatile("bar.sync 1, %0;" ::"n"(32 * kEpiWarps) : "memory");
            if (ok) {
#pragma unroll
                for (int i = 0; i < 6; ++i) {
                    const int kc = sl * 6 + i;
                    if (kc >= 16) *reinterpret_cast<uint4*>(smem + OFF_ST + sw_off(row, kc & 7)) = keep[i];
                }
                fence_proxy_async();
            }
            asm volatile("bar.sync 1, %0;" ::"n"(32 * kEpiWarps) : "memory");
            if (storer && ok) {
                tma_store_2d(&map_y, s_base + OFF_ST, item_j(q) * kCO + 128, item_t0(q));
                tma_store_commit();
            }
        }
        if (storer) tma_store_wait_all0();                                   // complete before shared memory goes away
    }
    if (!ok) atomicExch(status, (int32_t)M2_ERR_TIMEOUT);
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, 512);
}

bool covered(int C, int nblk, int expand) { return nblk > 0 && C / nblk == kCI && C % nblk == 0 && expand * kCI == kHID; }

cudaError_t prepare() {
    cudaError_t e = cudaFuncSetAttribute(mlp_umma_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(mlp_umma_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    return e;
}

int32_t launch(const void* z, const void* Wup, const void* Wdn, void* y, int C, int nblk, long long tokens, int32_t* status,
               cudaStream_t stream, long long z_channel_first_T) {
    if (tokens == 0) return M2_OK;
    const long long T = z_channel_first_T;
    if (T != 0 && (T < 0 || T % kTileT != 0 || tokens % T != 0 || T > 0x7fffffffLL)) return M2_ERR_INVALID_ARG;
    int dev_id = 0;
    {   // the shared-memory opt-in is per device (setting it twice is harmless; the flag itself is race-free)
        static std::atomic<bool> prepared[64];
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return M2_ERR_CUDA;
        if (!prepared[dev].load(std::memory_order_acquire)) {
            if (prepare() != cudaSuccess) return M2_ERR_CUDA;
            prepared[dev].store(true, std::memory_order_release);
        }
        dev_id = dev;
    }
    alignas(64) CUtensorMap mz, mw1, mw2, my;
    {   // activations [tokens][C]: box = 64 columns x 128 tokens, 128B swizzle (rows past the end: zero-filled / clipped)
        const cuuint64_t gdim[2] = {(cuuint64_t)C, (cuuint64_t)tokens}, gstr[1] = {(cuuint64_t)C * 2};
        const cuuint32_t box[2] = {64, (cuuint32_t)kTileT};
        if (!tma_host::encode_sw128_bf16(&my, y, 2, gdim, gstr, box)) return M2_ERR_UNSUPPORTED;
        if (T == 0) {
            if (!tma_host::encode_sw128_bf16(&mz, z, 2, gdim, gstr, box)) return M2_ERR_UNSUPPORTED;
        } else {   // z[b][c][t]: box = 64 tokens x the block's 192 channels of one batch entry
            const cuuint64_t zdim[3] = {(cuuint64_t)T, (cuuint64_t)C, (cuuint64_t)(tokens / T)}, zstr[2] = {(cuuint64_t)T * 2, (cuuint64_t)C * T * 2};
            const cuuint32_t zbox[3] = {64, (cuuint32_t)kCI, 1};
            if (!tma_host::encode_sw128_bf16(&mz, z, 3, zdim, zstr, zbox)) return M2_ERR_UNSUPPORTED;
        }
    }
    {   // W_up [nblk * 768 hidden][192 in]: box = 64 x 128 rows;  W_down [nblk * 192 out][768 hidden]: box = 64 x 192 rows
        const cuuint64_t g1[2] = {(cuuint64_t)kCI, (cuuint64_t)nblk * kHID}, s1[1] = {(cuuint64_t)kCI * 2};
        const cuuint32_t b1[2] = {64, (cuuint32_t)kChunk};
        const cuuint64_t g2[2] = {(cuuint64_t)kHID, (cuuint64_t)nblk * kCO}, s2[1] = {(cuuint64_t)kHID * 2};
        const cuuint32_t b2[2] = {64, (cuuint32_t)kCO};
        if (!tma_host::encode_sw128_bf16(&mw1, Wup, 2, g1, s1, b1) || !tma_host::encode_sw128_bf16(&mw2, Wdn, 2, g2, s2, b2))
            return M2_ERR_UNSUPPORTED;
    }
    cudaLaunchConfig_t cfg = {};
    const long long nitems = ((tokens + kTileT - 1) / kTileT) * nblk;
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev_id) != cudaSuccess || sms < 1 || nitems > 0x7fffffffLL) return M2_ERR_CUDA;
    cfg.gridDim = dim3((unsigned)(nitems < sms ? nitems : sms));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t le = T != 0 ? cudaLaunchKernelEx(&cfg, mlp_umma_kernel<true>, mz, mw1, mw2, my, status, nblk, (int)nitems, (int)T)
                                  : cudaLaunchKernelEx(&cfg, mlp_umma_kernel<false>, mz, mw1, mw2, my, status, nblk, (int)nitems, 1);
    if (le != cudaSuccess) return M2_ERR_CUDA;
    return M2_OK;
}

}  // namespace m2mlp
