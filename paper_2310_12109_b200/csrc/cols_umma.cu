// Monarch matrix times a matrix whose COLUMNS are the vectors:  Y = sigma(K (.) M X),  X, Y, K: [N][d] row-major,
// M = P L P^T R P with N = N1 * N2 (Sec. 3.1; this is Eq. 2's M X with X in R^{N x d} as the paper writes it, and the layout
// of its operator benchmark, Table 2: N = 4K .. 256K, block size sqrt(N), d = 768 columns).
//
// With the d columns contiguous, both block-diagonal factors are plain batched GEMMs over rows and no element ever has
// to be transposed:
//   stage(W, V)[row o*so + j][c] = sum_i W[j][o][i] * V[row i*si + j*sj][c]
//   z = stage(R, x): N2 blocks of N1 x N1, block j = n2 reads the rows n1*N2 + n2 (a strided set) and writes the rows k1*N2 + n2
//   y = stage(L, z): N1 blocks of N2 x N2, block j = k1 reads the rows k1*N2 + n2 (consecutive) and writes the rows k2*N1 + k1
// so the stride permutations are nothing but the strides of two TMA tensor maps.  One kernel serves both stages:
// a CTA computes the tile [128 outputs o][NC columns] of one block j:  A = W[j] rows (K-major, 128B-swizzled TMA boxes
// of 64 inputs), B = 64 input rows x NC columns (N-major: a row of the operand is a row of V), accumulator in TMEM
// (M = 128, or 64 for blocks of 64; N = NC <= 256), K = the block size walked in chunks of 64 through a three-stage TMA ring;
// the epilogue applies the optional factor K (.) and ReLU in fp32, rounds to bf16, stages the tile in the swizzled image of
// the TMA store boxes and stores it to its rows.  One persistent CTA per SM with a producer warp, an issuing warp
// and four epilogue warps; two accumulators in TMEM, so a tile's epilogue overlaps the next tile's UMMAs.  Block sizes are
// multiples of 64 (an output tile past the end of a block is clipped by the store's tensor map), d a multiple of 8 (a ragged
// last column tile is zero-filled on the way in and clipped on the way out).  All waits are bounded.
#include <cuda.h>

#include <atomic>
#include <cuda_bf16.h>

#include <cstring>

#include "cols_umma.h"
#include "ptx_sm100.cuh"
#include "tma_host.h"

namespace m2c {

using namespace sm100;

constexpr int kThreads = 192;               // warps 0..3: epilogue (the four TMEM lane quarters); warp 4: TMA producer; warp 5: UMMA issuer
constexpr int kStages = 3;
constexpr int STAGE_BYTES = 49152;          // A chunk [128][64] 16384 | B chunk [64][256] 32768
constexpr int OFF_OUT = kStages * STAGE_BYTES;   // output staging: up to 4 boxes [128][64] bf16   65536
constexpr int OFF_BAR = OFF_OUT + 65536;    // full[3], empty[3], acc_full[2], acc_empty[2], tmem ptr, abort flag
constexpr int SMEM_BYTES = OFF_BAR + 128;
static_assert(SMEM_BYTES <= 232448, "shared memory budget");

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
                 "l"(map), "r"(c0), "r"(c1), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// barrier among the 128 epilogue threads that also ANDs a predicate (every thread gets the same answer)
__device__ __forceinline__ bool epilogue_sync_and(bool pred) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %1, 0;\n\t"
        "bar.red.and.pred p, 1, 128, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(r)
        : "r"((uint32_t)pred)
        : "memory");
    return r != 0;
}

// Persistent: CTA p works on tiles p, p + gridDim.x, ...; tile index = ((bt * b + j) * otiles + ot) * ctiles + ct, so the
// CTAs running at the same time share the block's weights or its input rows in L2.  The producer runs ahead through the
// three-stage ring across tile boundaries; the accumulator is double-buffered in TMEM, so a tile's epilogue overlaps the
// next tile's UMMAs.
__global__ void __launch_bounds__(kThreads, 1)
monarch_cols_stage_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_v,
                          const __grid_constant__ CUtensorMap map_o, const __nv_bfloat16* __restrict__ Kmul, int relu, int b, int nb, int krs_o, int d,
                          int nc, int m, int tiles, int32_t* __restrict__ status) {   // b: block size, nb: number of blocks
    extern __shared__ __align__(1024) unsigned char smem[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t s_base = smem_u32(smem);
    const uint32_t bar_full = s_base + OFF_BAR, bar_empty = bar_full + 24, bar_accf = bar_full + 48, bar_acce = bar_full + 64;
    const uint32_t s_tptr = bar_full + 80;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + OFF_BAR + 88);
    const int otiles = (b + 127) / 128, ctiles = (d + nc - 1) / nc;   // the last column tile may be ragged: TMA zero-fills / clips it
    const int chunks = b / 64, nq = nc / 64;
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(bar_accf + 8 * a, 1);
            mbar_init(bar_acce + 8 * a, 4);   // one arrival per epilogue warp
        }
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tensormap(&map_w);
        prefetch_tensormap(&map_v);
        prefetch_tensormap(&map_o);
    }
    if (warp == 5) tmem_alloc(s_tptr, (uint32_t)(2 * nc));   // 128, 256 or 512 columns: two accumulators
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    asm volatile("griddepcontrol.wait;" ::: "memory");   // V may have been written by the kernel before this one
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(smem + OFF_BAR + 80);

    if (warp == 4) {
        // ---- TMA producer ----------------------------------------------------------------------------------------------
        if (lane == 0) {
            const uint32_t stage_tx = (uint32_t)(m * 128 + nq * 8192);
            uint32_t n = 0;   // chunks issued so far
            bool ok = true;
            for (int t = blockIdx.x; t < tiles && ok; t += gridDim.x) {
                const int ct = t % ctiles, ot = (t / ctiles) % otiles, j = (t / (ctiles * otiles)) % nb, bt = t / (ctiles * otiles * nb);
                for (int kc = 0; kc < chunks; ++kc, ++n) {
                    const int s = n % kStages;
                    if (n >= kStages) ok = mbar_wait(bar_empty + 8 * s, ((n / kStages) - 1) & 1);   // the UMMAs have read the buffer
                    if (!ok || *abort_flag) {
                        ok = false;
                        break;
                    }
                    const uint32_t sb = s_base + s * STAGE_BYTES, bf = bar_full + 8 * s;
                    mbar_expect_tx(bf, stage_tx);
                    tma_load_2d(sb, &map_w, kc * 64, j * b + ot * 128, bf);                                          // W[j][o tile][64 inputs]
                    for (int q = 0; q < nq; ++q) tma_load_4d(sb + 16384 + q * 8192, &map_v, ct * nc + 64 * q, kc * 64, j, bt, bf);   // 64 input rows
                }
            }
            if (!ok) {
                *abort_flag = 1;
                atomicExch(status, (int32_t)M2_ERR_TIMEOUT);
            }
        }
    } else if (warp == 5) {
        // ---- UMMA issuer -----------------------------------------------------------------------------------------------
        if (lane == 0) {
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(nc >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
            uint32_t n = 0;
            int it = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < tiles && ok; t += gridDim.x, ++it) {
                const int acc = it & 1;
                if (it >= 2) ok = mbar_wait(bar_acce + 8 * acc, ((it >> 1) - 1) & 1);   // the epilogue has read this accumulator
                if (!ok) break;
                tc_fence_after();
                for (int kc = 0; kc < chunks; ++kc, ++n) {
                    const int s = n % kStages;
                    ok = mbar_wait(bar_full + 8 * s, (n / kStages) & 1);
                    if (!ok || *abort_flag) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t sb = s_base + s * STAGE_BYTES;
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)   // 16 inputs per instruction
                        umma_f16(tmem + acc * nc, smem_desc_sw128(sb + ks * 32, 16, 1024), smem_desc_sw128(sb + 16384 + ks * 2048, 8192, 1024),
                                 idesc, (kc | ks) != 0);
                    umma_commit(bar_empty + 8 * s);
                }
                if (ok) umma_commit(bar_accf + 8 * acc);
            }
            if (!ok) {
                *abort_flag = 1;
                atomicExch(status, (int32_t)M2_ERR_TIMEOUT);
            }
        }
    } else {
        // ---- epilogue warps: accumulator row r = output o; M = 128: lane r; M = 64: lane (r % 16) + 32 (r / 16) -------------------
        const bool valid = m == 128 || lane < 16;
        const int r = m == 128 ? tid : warp * 16 + (lane & 15);
        const uint32_t t_lane = tmem + ((uint32_t)(warp * 32) << 16);
        unsigned char* stg = smem + OFF_OUT;
        int it = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < tiles && ok; t += gridDim.x, ++it) {
            const int ct = t % ctiles, ot = (t / ctiles) % otiles, j = (t / (ctiles * otiles)) % nb, bt = t / (ctiles * otiles * nb);
            const int acc = it & 1, o = ot * 128 + r, c0 = ct * nc;
            // the factor K (.) for this thread's row, requested while the tile's UMMAs still run
            uint4 kreg[32];
            if (Kmul != nullptr && valid) {
                const uint4* krow = reinterpret_cast<const uint4*>(Kmul + ((size_t)o * krs_o + j) * d + c0);   // K is shared by the batch
#pragma unroll
                for (int e = 0; e < 32; ++e)
                    if (e < nq * 8) kreg[e] = c0 + 8 * e < d ? __ldg(krow + e) : make_uint4(0u, 0u, 0u, 0u);   // d is a multiple of 8
            }
            ok = mbar_wait(bar_accf + 8 * acc, (it >> 1) & 1);
            tc_fence_after();
            if (tid == 0) tma_store_wait_read0();   // the previous tile's stores have read the staging area
            ok = epilogue_sync_and(ok && *abort_flag == 0);
            if (!ok) break;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                if (q >= nq) break;
                unsigned char* box = stg + q * (m * 128);   // [m rows][64 columns], 128-byte rows, 16-byte chunks XOR (row % 8)
#pragma unroll
                for (int hq = 0; hq < 2; ++hq) {
                    float v[32];
#pragma unroll
                    for (int c8 = 0; c8 < 4; ++c8) tmem_ld8(t_lane + acc * nc + q * 64 + (hq * 4 + c8) * 8, v + 8 * c8);
                    tmem_ld_wait();
#pragma unroll
                    for (int c8 = 0; c8 < 4; ++c8) tmem_ld_fence8(v + 8 * c8);
                    if (valid) {
#pragma unroll
                        for (int c8 = 0; c8 < 4; ++c8) {
                            float* w = v + 8 * c8;
                            if (Kmul != nullptr) {
                                const uint4 kp = kreg[q * 8 + hq * 4 + c8];
                                const uint32_t kw[4] = {kp.x, kp.y, kp.z, kp.w};
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    w[2 * e] *= __uint_as_float(kw[e] << 16);
                                    w[2 * e + 1] *= __uint_as_float(kw[e] & 0xffff0000u);
                                }
                                if (relu) {
#pragma unroll
                                    for (int e = 0; e < 8; ++e) w[e] = fmaxf(w[e], 0.f);
                                }
                            }
                            *reinterpret_cast<uint4*>(box + (r >> 3) * 1024 + (r & 7) * 128 + (((hq * 4 + c8) ^ (r & 7)) << 4)) =
                                make_uint4(pack_bf16(w[0], w[1]), pack_bf16(w[2], w[3]), pack_bf16(w[4], w[5]), pack_bf16(w[6], w[7]));
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_acce + 8 * acc);   // this warp has read its part of the accumulator
            fence_proxy_async();
            asm volatile("bar.sync 1, 128;" ::: "memory");
            if (tid == 0) {
                for (int q = 0; q < nq; ++q) tma_store_4d(&map_o, s_base + OFF_OUT + q * (m * 128), c0 + 64 * q, ot * 128, j, bt);
                tma_store_commit();
            }
        }
        if (tid == 0) tma_store_wait_read0();   // the staging area dies with the CTA
        if (!ok && lane == 0) {
            *abort_flag = 1;
            atomicExch(status, (int32_t)M2_ERR_TIMEOUT);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 5) tmem_dealloc(tmem, (uint32_t)(2 * nc));
}

bool covered(const m2_plan* pl, int64_t d) {
    if (pl->dtype != M2_BF16 || pl->p != 2) return false;
    // blocks of whole 64-input chunks (an output tile past the end of a block computes rows that the store's tensor map clips),
    // rows of whole 16-byte pieces
    for (int a = 0; a < 2; ++a)
        if (pl->dims[a] < 64 || pl->dims[a] > 1024 || pl->dims[a] % 64 != 0) return false;
    return d > 0 && d % 8 == 0;
}

cudaError_t prepare() {
    // per-device opt-in; setting the attribute twice is harmless, so host threads only need the flag itself to be race-free
    static std::atomic<bool> done[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64 && done[dev].load(std::memory_order_acquire)) return cudaSuccess;
    e = cudaFuncSetAttribute(monarch_cols_stage_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    if (e == cudaSuccess && dev >= 0 && dev < 64) done[dev].store(true, std::memory_order_release);
    return e;
}

// one stage: nb blocks of b x b; out rows o*so + j = W[j] applied to the rows i*si + j*sj of V (N = rows per matrix of the batch)
static int32_t stage(const m2_plan* pl, int64_t N, const void* W, const void* V, void* O, const void* Kmul, int relu, int64_t Bt, int64_t d,
                     int b, int nb, int64_t si, int64_t sj, int64_t so, cudaStream_t stream) {
    const int m = b == 64 ? 64 : 128;
    const int nc = d > 128 ? 256 : d > 64 ? 128 : 64;   // columns per tile
    alignas(64) CUtensorMap mw, mv, mo;
    {
        const cuuint64_t gdim[2] = {(cuuint64_t)b, (cuuint64_t)nb * b}, gstr[1] = {(cuuint64_t)b * 2};
        const cuuint32_t box[2] = {64, (cuuint32_t)m};
        if (!tma_host::encode_sw128_bf16(&mw, W, 2, gdim, gstr, box)) return M2_ERR_UNSUPPORTED;
    }
    {
        const cuuint64_t gdim[4] = {(cuuint64_t)d, (cuuint64_t)b, (cuuint64_t)nb, (cuuint64_t)Bt};
        const cuuint64_t gstr[3] = {(cuuint64_t)(si * d * 2), (cuuint64_t)(sj * d * 2), (cuuint64_t)N * d * 2};
        const cuuint32_t box[4] = {64, 64, 1, 1};
        if (!tma_host::encode_sw128_bf16(&mv, V, 4, gdim, gstr, box)) return M2_ERR_UNSUPPORTED;
    }
    {
        const cuuint64_t gdim[4] = {(cuuint64_t)d, (cuuint64_t)b, (cuuint64_t)nb, (cuuint64_t)Bt};
        const cuuint64_t gstr[3] = {(cuuint64_t)(so * d * 2), (cuuint64_t)d * 2, (cuuint64_t)N * d * 2};
        const cuuint32_t box[4] = {64, (cuuint32_t)m, 1, 1};
        if (!tma_host::encode_sw128_bf16(&mo, O, 4, gdim, gstr, box)) return M2_ERR_UNSUPPORTED;
    }
    const long long tiles = Bt * nb * ((b + 127) / 128) * ((d + nc - 1) / nc);
    if (tiles > 0x7fffffffLL) return M2_ERR_UNSUPPORTED;
    int dev = 0, sms = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(tiles < sms ? tiles : sms));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, monarch_cols_stage_kernel, mw, mv, mo, (const __nv_bfloat16*)Kmul, relu, b, nb, (int)so, (int)d, nc, m,
                           (int)tiles, pl->d_status) != cudaSuccess)
        return M2_ERR_CUDA;
    return M2_OK;
}

int32_t apply(const m2_plan* pl, const void* X, const void* L, const void* R, const void* Kmul, int relu, void* Y, int64_t Bt, int64_t d,
              void* ws, cudaStream_t stream) {
    if (!covered(pl, d)) return M2_ERR_UNSUPPORTED;
    if (Bt > 65535) return M2_ERR_UNSUPPORTED;
    if (Bt == 0) return M2_OK;
    if (prepare() != cudaSuccess) return M2_ERR_CUDA;
    const int N1 = pl->dims[0], N2 = pl->dims[1];
    int32_t st = stage(pl, pl->N, R, X, ws, nullptr, 0, Bt, d, N1, N2, N2, 1, N2, stream);   // z[k1*N2 + n2]: N2 blocks R[n2] on the rows n1*N2 + n2
    if (st != M2_OK) return st;
    st = stage(pl, pl->N, L, ws, Y, Kmul, relu, Bt, d, N2, N1, 1, N2, N1, stream);           // y[k2*N1 + k1]: N1 blocks L[k1] on the rows k1*N2 + n2
    if (st != M2_OK) return st;
    pl->last_kernel = "monarch_cols_umma";
    pl->launches += 2;
    return M2_OK;
}

// A dense matrix is a block-diagonal one with a single block: O[bt] = W V[bt] for Bt matrices V [c][cols] (cols contiguous),
// W: [c][c] row-major (outputs x inputs).  pl only lends its status word and launch counter.
bool dense_covered(const m2_plan* pl, int64_t c, int64_t cols) {
    return pl->dtype == M2_BF16 && c >= 64 && c <= 4096 && c % 64 == 0 && cols > 0 && cols % 8 == 0;
}

int32_t dense(const m2_plan* pl, const void* W, const void* V, void* O, int64_t Bt, int64_t c, int64_t cols, cudaStream_t stream) {
    if (!dense_covered(pl, c, cols) || Bt > 65535) return M2_ERR_UNSUPPORTED;
    if (Bt == 0) return M2_OK;
    if (prepare() != cudaSuccess) return M2_ERR_CUDA;
    const int32_t st = stage(pl, c, W, V, O, nullptr, 0, Bt, cols, (int)c, 1, 1, c, 1, stream);   // (the block stride is never used: one block)
    if (st == M2_OK) pl->launches += 1;
    return st;
}

}  // namespace m2c
