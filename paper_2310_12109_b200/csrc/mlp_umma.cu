// Tensor-core block-diagonal MLP of the M2 block (Eq. 3 with block-diagonal M_3, M_4; Sec. 5.1: M2-BERT's dense
// layers replaced by block-diagonal ones):  y_j = W_down[j] GELU(W_up[j] z_j)  per token and block j, erf-form GELU,
// for blocks of 192 inputs / 768 hidden / 192 outputs (d = 768, 4 blocks, expansion 4).  bf16 operands, fp32
// accumulation in TMEM, the hidden activations are rounded to bf16 and never leave the SM.
//
// One CTA = 128 tokens x one block.  The hidden dimension is walked in 6 chunks of 128:
//   S1(c)  D1[c % 2][128 tok][128 hid] = Z[128][192] * W_up[j][chunk c]^T        12 UMMAs (M128 N128 K16)
//   E1(c)  TMEM -> registers -> GELU -> bf16 -> G[128 tok][128 hid] (UMMA operand, shared memory)
//   S2(c)  D2[128 tok][192 out] += G * W_down[j][:, chunk c]^T                     8 UMMAs (M128 N192 K16)
// and at the end D2 -> bf16 -> staging -> TMA store.  Warp roles: warp 0 feeds the weight chunks by TMA (W_up
// chunks double-buffered), warp 1 issues the UMMAs and runs S1(c + 1) ahead of E1(c) (two D1 buffers), warps 2..17
// are the GELU warps (lane quarter = warp % 4, 32 of the 128 chunk columns each).  All operands are K-major with the
// 128-byte swizzle, written by TMA (Z, weights) or by the GELU warps (G).  Every wait is bounded.
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
constexpr int OFF_Z = 0;                    // 3 K-blocks [128][64] bf16 (also the output staging)   49152
constexpr int OFF_W1 = 49152;               // 2 buffers x 3 K-blocks [128 hid][64]                   98304
constexpr int OFF_W2 = 147456;              // 2 K-blocks [192 out][64]                               49152
constexpr int OFF_G = 196608;               // 2 K-blocks [128 tok][64]                               32768
constexpr int OFF_BAR = 229376;
constexpr int SMEM_BYTES = OFF_BAR + 192;
static_assert(SMEM_BYTES <= 232448, "shared memory budget");
// mbarriers (8 bytes each) from OFF_BAR
enum { B_Z = 0, B_W1F = 1, B_W1E = 3, B_W2F = 5, B_W2E = 6, B_D1F = 7, B_D1E = 9, B_GF = 11, B_GE = 12, B_D2F = 13, B_COUNT = 14 };

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
                 "l"(map), "r"(c0), "r"(c1), "r"(bar)
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

__global__ void __launch_bounds__(kThreads, 1)
mlp_umma_kernel(const __grid_constant__ CUtensorMap map_z, const __grid_constant__ CUtensorMap map_w1,
                const __grid_constant__ CUtensorMap map_w2, const __grid_constant__ CUtensorMap map_y, int32_t* __restrict__ status) {
    extern __shared__ __align__(1024) unsigned char smem[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t s_base = smem_u32(smem);
    const uint32_t bars = s_base + OFF_BAR, s_tptr = s_base + OFF_BAR + 8 * B_COUNT;
    auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
    const int j = blockIdx.y;                      // block of the block-diagonal factors
    const int t0 = blockIdx.x * kTileT;            // first token of the tile

    if (tid == 0) {
        mbar_init(bar(B_Z), 1);
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar(B_W1F + i), 1);
            mbar_init(bar(B_W1E + i), 1);
            mbar_init(bar(B_D1F + i), 1);
            mbar_init(bar(B_D1E + i), kEpiWarps);   // one arrival per GELU warp
        }
        mbar_init(bar(B_W2F), 1);
        mbar_init(bar(B_W2E), 1);
        mbar_init(bar(B_GF), kEpiWarps);
        mbar_init(bar(B_GE), 1);
        mbar_init(bar(B_D2F), 1);
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
        // ---- TMA producer ------------------------------------------------------------------------------------------
        if (lane == 0) {
            mbar_expect_tx(bar(B_Z), 49152);
            for (int kb = 0; kb < 3; ++kb) tma_load_2d(s_base + OFF_Z + kb * 16384, &map_z, j * kCI + kb * 64, t0, bar(B_Z));
            // The two weight streams advance independently (a W_up chunk two ahead of the UMMAs, the single W_down
            // buffer as soon as S2 has read it), so neither waits behind the other's barrier.
            int c1 = 0, c2 = 0;
            uint32_t idle = 0;
            while ((c1 < kChunks || c2 < kChunks) && idle < (1u << 22)) {
                bool progressed = false;
                if (c1 < kChunks && (c1 < 2 || mbar_try_wait(bar(B_W1E + (c1 & 1)), ((c1 >> 1) - 1) & 1))) {   // S1(c1 - 2) has read the buffer
                    const int bb = c1 & 1;
                    mbar_expect_tx(bar(B_W1F + bb), 49152);
                    for (int kb = 0; kb < 3; ++kb)
                        tma_load_2d(s_base + OFF_W1 + bb * 49152 + kb * 16384, &map_w1, kb * 64, j * kHID + c1 * kChunk, bar(B_W1F + bb));
                    ++c1;
                    progressed = true;
                }
                if (c2 < kChunks && (c2 < 1 || mbar_try_wait(bar(B_W2E), (c2 - 1) & 1))) {                        // S2(c2 - 1) has read the chunk
                    mbar_expect_tx(bar(B_W2F), 49152);
                    for (int kb = 0; kb < 2; ++kb)
                        tma_load_2d(s_base + OFF_W2 + kb * 24576, &map_w2, c2 * kChunk + kb * 64, j * kCO, bar(B_W2F));
                    ++c2;
                    progressed = true;
                }
                idle = progressed ? 0 : idle + 1;
            }
            if (c1 < kChunks || c2 < kChunks) ok = false;
        }
    } else if (warp == 1) {
        // ---- UMMA issuer ---------------------------------------------------------------------------------------------
        if (lane == 0) {
            constexpr uint32_t ID1 = instr_desc_bf16(128, 128, false, false), ID2 = instr_desc_bf16(128, 192, false, false);
            auto s1 = [&](int c) {   // D1[c % 2] = Z * W_up chunk c
                const int b = c & 1;
                ok = mbar_wait(bar(B_W1F + b), (c >> 1) & 1);
                if (ok && c >= 2) ok = mbar_wait(bar(B_D1E + b), ((c >> 1) - 1) & 1);   // the GELU warps have read D1[b]
                if (!ok) return;
                tc_fence_after();
#pragma unroll 1
                for (int kb = 0; kb < 3; ++kb)
#pragma unroll
                    for (int s = 0; s < 4; ++s)
                        umma_f16(D1 + b * 128, smem_desc_sw128(s_base + OFF_Z + kb * 16384 + s * 32, 16, 1024),
                                 smem_desc_sw128(s_base + OFF_W1 + b * 49152 + kb * 16384 + s * 32, 16, 1024), ID1, (kb | s) != 0);
                umma_commit(bar(B_D1F + b));
                umma_commit(bar(B_W1E + b));
            };
            ok = mbar_wait(bar(B_Z), 0);
            if (ok) s1(0);
            for (int c = 0; c < kChunks && ok; ++c) {
                if (c + 1 < kChunks) s1(c + 1);
                if (!ok) break;
                ok = mbar_wait(bar(B_GF), c & 1) && mbar_wait(bar(B_W2F), c & 1);
                if (!ok) break;
                tc_fence_after();
#pragma unroll 1
                for (int kb = 0; kb < 2; ++kb)
#pragma unroll
                    for (int s = 0; s < 4; ++s)
                        umma_f16(D2, smem_desc_sw128(s_base + OFF_G + kb * 16384 + s * 32, 16, 1024),
                                 smem_desc_sw128(s_base + OFF_W2 + kb * 24576 + s * 32, 16, 1024), ID2, (c | kb | s) != 0);
                umma_commit(bar(B_GE));
                umma_commit(bar(B_W2E));
                if (c == kChunks - 1) umma_commit(bar(B_D2F));
            }
        }
    } else {
        // ---- GELU warps: lane quarter q = warp % 4 (a TMEM rule), column slice sl = 32 of the chunk's 128 columns ----
        const int ew = warp - 2, q = warp & 3, sl = ew >> 2;
        const int row = q * 32 + lane;                                   // token within the tile
        const uint32_t t_lane = tmem + ((uint32_t)(q * 32) << 16);
        for (int c = 0; c < kChunks && ok; ++c) {
            const int b = c & 1;
            ok = mbar_wait(bar(B_D1F + b), (c >> 1) & 1);
            if (!ok) break;
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
            uint4 pk[4];
#pragma unroll
            for (int i = 0; i < 4; ++i)
                pk[i] = make_uint4(gelu2_pack(v[8 * i], v[8 * i + 1]), gelu2_pack(v[8 * i + 2], v[8 * i + 3]),
                                   gelu2_pack(v[8 * i + 4], v[8 * i + 5]), gelu2_pack(v[8 * i + 6], v[8 * i + 7]));
            if (c >= 1) ok = mbar_wait(bar(B_GE), (c - 1) & 1);          // S2(c - 1) has read G
            if (!ok) break;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int kc = sl * 4 + i;                               // 16-byte chunk of the 128-column row
                *reinterpret_cast<uint4*>(smem + OFF_G + (kc >> 3) * 16384 + sw_off(row, kc & 7)) = pk[i];
            }
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(B_GF));
        }
        // ---- output: D2 -> bf16 -> staging (the Z buffer, free since the last S1) -> TMA store ---------------------
        if (ok) ok = mbar_wait(bar(B_D2F), 0);
        if (ok) {
            tc_fence_after();
#pragma unroll 1
            for (int h = 0; h < 2; ++h) {                                // 48 of the 192 output columns per slice: 6 chunks
                float w[24];
#pragma unroll
                for (int i = 0; i < 3; ++i) tmem_ld8(t_lane + 256 + sl * 48 + h * 24 + 8 * i, w + 8 * i);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 3; ++i) tmem_ld_fence8(w + 8 * i);
#pragma unroll
                for (int i = 0; i < 3; ++i) {
                    const int kc = sl * 6 + h * 3 + i;                   // 16-byte chunk of the 192-column row: 24 of them
                    *reinterpret_cast<uint4*>(smem + OFF_Z + (kc >> 3) * 16384 + sw_off(row, kc & 7)) =
                        make_uint4(pack_bf16(w[8 * i], w[8 * i + 1]), pack_bf16(w[8 * i + 2], w[8 * i + 3]),
                                   pack_bf16(w[8 * i + 4], w[8 * i + 5]), pack_bf16(w[8 * i + 6], w[8 * i + 7]));
                }
            }
            fence_proxy_async();
        }
        asm volatile("bar.sync 1, %0;" ::"n"(32 * kEpiWarps) : "memory");
        if (ok && ew == 0 && lane == 0) {
            for (int kb = 0; kb < 3; ++kb) tma_store_2d(&map_y, s_base + OFF_Z + kb * 16384, j * kCO + kb * 64, t0);
            tma_store_commit();
            tma_store_wait_all0();
        }
    }
    if (!ok) atomicExch(status, (int32_t)M2_ERR_TIMEOUT);
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, 512);
}

bool covered(int C, int nblk, int expand) { return nblk > 0 && C / nblk == kCI && C % nblk == 0 && expand * kCI == kHID; }

cudaError_t prepare() { return cudaFuncSetAttribute(mlp_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES); }

int32_t launch(const void* z, const void* Wup, const void* Wdn, void* y, int C, int nblk, long long tokens, int32_t* status,
               cudaStream_t stream) {
    if (tokens == 0) return M2_OK;
    {   // the shared-memory opt-in is per device (setting it twice is harmless; the flag itself is race-free)
        static std::atomic<bool> prepared[64];
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return M2_ERR_CUDA;
        if (!prepared[dev].load(std::memory_order_acquire)) {
            if (prepare() != cudaSuccess) return M2_ERR_CUDA;
            prepared[dev].store(true, std::memory_order_release);
        }
    }
    alignas(64) CUtensorMap mz, mw1, mw2, my;
    {   // activations [tokens][C]: box = 64 columns x 128 tokens, 128B swizzle (rows past the end: zero-filled / clipped)
        const cuuint64_t gdim[2] = {(cuuint64_t)C, (cuuint64_t)tokens}, gstr[1] = {(cuuint64_t)C * 2};
        const cuuint32_t box[2] = {64, (cuuint32_t)kTileT};
        if (!tma_host::encode_sw128_bf16(&mz, z, 2, gdim, gstr, box) || !tma_host::encode_sw128_bf16(&my, y, 2, gdim, gstr, box))
            return M2_ERR_UNSUPPORTED;
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
    cfg.gridDim = dim3((unsigned)((tokens + kTileT - 1) / kTileT), (unsigned)nblk);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, mlp_umma_kernel, mz, mw1, mw2, my, status) != cudaSuccess) return M2_ERR_CUDA;
    return M2_OK;
}

}  // namespace m2mlp
