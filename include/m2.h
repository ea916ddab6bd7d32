/*
 * m2.h -- C ABI of the B200 Monarch Mixer hot-path library (libm2.so).
 *
 * Two operations of "Monarch Mixer" (arXiv 2310.12109) and the helpers around them:
 *
 *   Monarch matmul   y = P L P^T R P x                         (Sec. 3.1; Eq. 1 for order p)
 *   Monarch conv     y = M^-1 ( (M k) (.) (M x) ),  M = F_N     (Eq. 2; App. D.3 Def. "matrix
 *                    factored as an order-p Monarch matrix        convolution"; Alg. BlockMonarchConv;
 *                    with twiddle diagonals                       Corollary "DFT is M", App. D.5)
 *
 * Conventions (App. D notation).  N = N1*N2*..*Np.  A length-N vector is indexed
 * n = (..(n1*N2 + n2)*N3 + ..) on input (n1 most significant) and k = k1 + N1*k2 + N1*N2*k3 + ..
 * on output (k1 least significant).  "Plan order" stores the tensor [k1][k2]..[kp] row-major.
 * P = P_(N1,N) is the stride permutation (P x)[i] = x[sigma(i)], sigma(i) = (i mod N1)*(N/N1) + i/N1.
 * omega_M = exp(sign * 2 pi i / M); the paper uses sign = +1.
 *
 * General rules.  Every function returns an m2_status (0 = OK) and never throws.  Pointers named
 * *_dev are device pointers on the plan's device, *_host are host pointers.  The caller owns every
 * data buffer; the library owns the plan and its device tables.  `stream` is a cudaStream_t passed
 * as void* (NULL = the legacy default stream).  Arguments are validated on the host before
 * anything is launched; on an error nothing has been enqueued.  The hot calls never synchronise
 * the stream and never allocate.  All device buffers must be 16-byte aligned and contiguous.
 * Work is ordered by the stream as usual: a call sees everything enqueued on `stream` before it.  (The
 * tensor-core kernels are launched so that their thread blocks may take over SMs while the previous
 * kernel's last blocks still run; they wait for that kernel before touching any data.)
 */
#ifndef M2_H_
#define M2_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct m2_plan m2_plan;

enum m2_status {
    M2_OK = 0,
    M2_ERR_INVALID_ARG = 1, /* null pointer, bad size, sizes inconsistent with the plan */
    M2_ERR_UNSUPPORTED = 2, /* valid request the library has no kernel for */
    M2_ERR_ALIGNMENT = 3,   /* a device pointer is not 16-byte aligned */
    M2_ERR_CUDA = 4,        /* a CUDA runtime / driver call failed */
    M2_ERR_TIMEOUT = 5,     /* a bounded device-side wait ran out (read via m2_last_device_status) */
    M2_ERR_NO_DEVICE = 6,   /* the plan was created host-only (device < 0) */
    M2_ERR_SINGULAR = 7     /* a block of a learnable Monarch factor could not be inverted (read via m2_last_device_status) */
};

enum m2_dtype { M2_FP32 = 0, M2_BF16 = 1 };
enum m2_conv_mode { M2_CAUSAL = 0, M2_CIRCULAR = 1 };
enum m2_table {
    M2_TABLE_PERM = 0,      /* sigma_(N1,N)                      (App. D notation)            */
    M2_TABLE_PERM_INV = 1,  /* its inverse, sigma_(N/N1,N)       (P_(b,N)^T = P_(N/b,N))       */
    M2_TABLE_DIGIT_REV = 2, /* plan position -> natural frequency k = k1 + N1 k2 + ..         */
    M2_TABLE_TW_EXP = 16    /* M2_TABLE_TW_EXP + s, s = 1..p-1: exponent e of the twiddle
                               omega_{N1..N_{s+1}}^e applied at plan position pos before the
                               digit n_{s+1} is contracted: e = n_{s+1} * (k1 + N1 k2 + .. ) mod
                               (N1..N_{s+1}), indexed by the row-major position
                               [k1]..[k_s][n_{s+1}]..[n_p]                                     */
};

/* Creates a plan for length N = factors[0]*..*factors[p-1] (p = 2 or 3 for the convolution; the
 * matmul uses p = 2).  dtype is the storage type of x / y (M2_FP32: float, M2_BF16: bfloat16);
 * every sum is accumulated in fp32.  (Between stages bf16 plans round: the tensor-core kernels re-round the
 * operands of every stage to bf16, and the general-shape convolution kernel, for 20480 < N <= 51200 where
 * a complex fp32 row no longer fits in shared memory, keeps the row between its stages as bf16 pairs.)  sign = +1 (paper) or -1.  device >= 0: CUDA device ordinal, tables
 * are uploaded (the call synchronises).  device < 0: host-only plan, usable only with
 * m2_plan_get_table.  (Eq. 1: the factorisation N = N1..Np with block size N^(1/p); Corollary
 * "DFT is M": the twiddles.)  A plan carries a little device state of its own (a status word, work
 * counters of its kernels): calls on one plan must be ordered on the GPU -- one stream, or events
 * between streams; use one plan per stream for calls that may overlap.  A plan also carries host-side
 * bookkeeping (launch count, name of the last kernel) that is not synchronised: do not use one plan from
 * two host threads at the same time (give each thread its own plan; the library's global state -- the
 * per-device kernel attributes and the static scratch address -- is safe to reach from several threads). */
int32_t m2_plan_create(m2_plan** out, int64_t N, int32_t p, const int32_t* factors, int32_t dtype,
                       int32_t sign, int32_t device);
int32_t m2_plan_destroy(m2_plan* plan);

/* Copies one integer table (enum m2_table) into host_out[0..len); len must equal N. */
int32_t m2_plan_get_table(const m2_plan* plan, int32_t which, int32_t* host_out, int64_t len);

/* Bytes of the spectrum buffer m2_kernel_spectrum writes for H channels. */
int64_t m2_spectrum_bytes(const m2_plan* plan, int64_t H);

/* k_f = M * pad(k) per channel (Alg. BlockMonarchConv, the line k_f <- M k; Eq. 2's K_1 given in
 * frequency space).  k_dev: [H, n] float32, n <= N, zero padded to N.  kf_dev: m2_spectrum_bytes
 * bytes; the format is private to the plan (complex fp32, plan order, with the 1/N of M^-1 folded
 * in).  Computed in fp32 whatever the plan dtype; meant to run once per weight update. */
int32_t m2_kernel_spectrum(const m2_plan* plan, const float* k_dev, int64_t H, int64_t n, void* kf_dev,
                           void* stream);

/* Test helper: converts a spectrum buffer to natural frequency order, unnormalised (= F_N pad(k)),
 * interleaved (re, im) float32 [H, N, 2]. */
int32_t m2_spectrum_to_natural(const m2_plan* plan, const void* kf_dev, int64_t H, float* out_dev,
                               void* stream);

/* kf_out = conj(kf_in), in every layout the buffer holds (kf_out may be kf_in).  With the conjugated
 * spectrum m2_monarch_conv_fwd computes the transpose of the convolution: for an upstream gradient g of y,
 * dx = M^-1 ( conj(k_f) (.) M pad(g) ) [0:n) is the gradient with respect to x (k is real, so conj(F k)
 * is the spectrum of the index-reversed kernel: the transposed circulant, resp. the transposed Toeplitz
 * matrix T_k of App. D.3 once zero padded).  The paper trains through this operator (Sec. 5) without
 * writing the backward pass out. */
int32_t m2_spectrum_conjugate(const m2_plan* plan, const void* kf_in_dev, int64_t H, void* kf_out_dev,
                              void* stream);

/* Gradient with respect to the kernel: for an upstream gradient g of y,
 *   dk[h][u] = sum_b sum_t g[b][h][t] x[b][h][t - u]  =  M^-1 ( sum_b conj(M pad(x_b)) (.) M pad(g_b) ) [0:n)
 * (the convolution of Eq. 2 is linear in k; indices mod N for M2_CIRCULAR, t >= u for M2_CAUSAL).
 * x_dev, g_dev: [B, H, n] in the plan dtype; dk_dev: [H, n] float32.
 * ws_dev: optional caller-owned workspace of m2_conv_bwd_workspace_bytes(plan, B, H) bytes (16-byte aligned; 0 bytes
 * means this plan has no kernel that uses one).  With it, plans the tensor-core path covers (bf16, N = 512 = 32 x 16)
 * run both forward transforms and the products conj(M x) (.) M g on the tensor cores (intermediates rounded to bf16
 * like the forward pass), 8 batch rows at a time, and a CUDA-core kernel adds the groups in order and applies M^-1 in
 * fp32; for N = 32768 = 32^3 (causal, n = 16384) the order-3 convolution kernel is run twice (the row pairs' conjugated
 * spectra, then the convolution of the g pairs with them) and the pairs' rows are added.  Otherwise, or with a workspace
 * too small for those, everything runs on the CUDA cores in fp32, one thread block per channel with its three complex
 * rows in shared memory (N up to 8192) or, for longer rows, in the workspace (at least 24 N bytes per channel for up to
 * 296 channels; M2_ERR_UNSUPPORTED without it).  m2_conv_bwd_workspace_bytes returns the largest of these needs.  All
 * paths are deterministic.  (The paper trains through the operator, Sec. 5, without writing the
 * backward pass out.) */
int64_t m2_conv_bwd_workspace_bytes(const m2_plan* plan, int64_t B, int64_t H);
int32_t m2_monarch_conv_bwd_kernel(const m2_plan* plan, const void* x_dev, const void* g_dev, float* dk_dev, int64_t B,
                                   int64_t H, int64_t n, int32_t mode, void* ws_dev, int64_t ws_bytes, void* stream);

/* y = Re( M^-1 ( k_f (.) M pad(x) ) )[0:n)  (Eq. 2 with M_1 = F, M_2 = F^-1; App. D.3).
 * x_dev, y_dev: [B, H, n] in the plan dtype; kf_dev from m2_kernel_spectrum with the same H.
 * mode M2_CAUSAL: n <= N/2, x zero padded to N, first n outputs kept (Thm 3 / App. D.3 review).
 * mode M2_CIRCULAR: n == N. */
int32_t m2_monarch_conv_fwd(const m2_plan* plan, const void* x_dev, const void* kf_dev, void* y_dev, int64_t B,
                            int64_t H, int64_t n, int32_t mode, void* stream);

/* The same convolution with one kernel shared by kf_group consecutive channels: channel h is multiplied by row h / kf_group
 * of the spectrum, which m2_kernel_spectrum computed for H / kf_group kernels (H must be a multiple of kf_group).  This is how
 * the heads of the M2 Hyena layer (App. "GPT Causal Language Modeling") use one long kernel for the dh^2 sequences of a head's
 * outer product without the spectrum being repeated dh^2 times. */
int32_t m2_monarch_conv_fwd_grouped(const m2_plan* plan, const void* x_dev, const void* kf_dev, void* y_dev, int64_t B,
                                    int64_t H, int64_t n, int32_t mode, int64_t kf_group, void* stream);

/* Same operation from host buffers: copies x_host -> x_dev (scratch the caller provides), runs the
 * convolution, copies y_dev -> y_host, all on `stream`; returns without synchronising.  x_host and
 * y_host should be pinned for the copies to be asynchronous. */
int32_t m2_monarch_conv_fwd_host(const m2_plan* plan, const void* x_host, const void* kf_dev, void* y_host,
                                 void* x_dev_scratch, void* y_dev_scratch, int64_t B, int64_t H, int64_t n,
                                 int32_t mode, void* stream);

/* Order-2 Monarch matmul per token (Sec. 3.1, M = P L P^T R P; weight layout of the
 * blockdiag_matmul listing, [block][out][in]):
 *   y[t][k2*N1 + k1] = sum_{n2} L[k1][k2][n2] * sum_{n1} R[n2][k1][n1] * x[t][n1*N2 + n2].
 * X_dev, Y_dev: [T, N] in the plan dtype; L_dev: [N1][N2][N2], R_dev: [N2][N1][N1], same dtype.
 * R is applied first.  (The listing's parameter called L is applied first and so plays R's role.)
 * ws_dev: caller-owned device workspace of at least m2_matmul_workspace_bytes(plan, T) bytes for the
 * intermediate between the two factors (16-byte aligned); with ws_dev == NULL or ws_bytes too small the
 * call uses the slower kernels that need none.  bf16 plans with 64 x 64 blocks run on the tensor cores; their fastest
 * kernels read X in 32-byte pieces and want X_dev on a 32-byte boundary (any fresh allocation is; a view at an odd
 * 16-byte offset falls back to kernels with 16-byte pieces, same results). */
int64_t m2_matmul_workspace_bytes(const m2_plan* plan, int64_t T);
int32_t m2_monarch_matmul(const m2_plan* plan, const void* X_dev, const void* L_dev, const void* R_dev,
                          void* Y_dev, int64_t T, void* ws_dev, int64_t ws_bytes, void* stream);
int32_t m2_monarch_matmul_host(const m2_plan* plan, const void* X_host, const void* L_dev, const void* R_dev,
                               void* Y_host, void* X_dev_scratch, void* Y_dev_scratch, int64_t T, void* ws_dev,
                               int64_t ws_bytes, void* stream);

/* The M2 operator with general (learnable) Monarch matrices, Eq. 2 / the sequence- and feature-mixing lines of the M2
 * layer listing:  Y = M_b sigma(K (.) M_a X),  M_a = P La P^T Ra P,  M_b = P Lb P^T Rb P,  sigma = identity or ReLU.
 * X_dev, Y_dev: [T, N] in the plan dtype (Y_dev may be X_dev; Y_dev also holds the intermediate);
 * K_dev: [Hk, N] in the plan dtype, row t of X takes row t mod Hk of K (one kernel row per channel with the rows of X
 * ordered (batch, channel): Hk = channels; one shared row: Hk = 1).  Factors as in m2_monarch_matmul; ws_dev/ws_bytes
 * as there (m2_matmul_workspace_bytes(plan, T)).  The product K (.) M_a X and sigma are taken in fp32 on the fp32
 * accumulator; the intermediate is then rounded to the plan dtype. */
#define M2_ACT_NONE 0
#define M2_ACT_RELU 1
int32_t m2_monarch_mix(const m2_plan* plan, const void* X_dev, const void* K_dev, int64_t Hk, int32_t act,
                       const void* La_dev, const void* Ra_dev, const void* Lb_dev, const void* Rb_dev, void* Y_dev,
                       int64_t T, void* ws_dev, int64_t ws_bytes, void* stream);

/* The basic M2 layer (App. "Implementation", the MonarchMixerLayer listing), x: [B, n, d] in the plans' dtype:
 *   x~  = (M2 relu(K_n (.) M1 x^T))^T        mix along the sequence;  K_n = n_kernel_dev [d, n]
 *   y   = M4 relu(k_d (.) M3 x~)             mix along the features;  k_d = d_kernel_dev [1, d]
 *   out = LayerNorm(y + x~) * gamma + beta   over d, biased variance, eps inside the root; gamma, beta fp32 [d]
 * plan_n: order-2 plan of length n (M1, M2), plan_d: order-2 plan of length d (M3, M4); same dtype and device.
 * factors: HOST array of 8 device pointers {L1, R1, L2, R2, L3, R3, L4, R4}, each pair as in m2_monarch_matmul
 * (R is applied first; the listing's parameter called L is the one applied first, i.e. this library's R).
 * y_dev: [B, n, d] (must not overlap x_dev).  scratch_dev: m2_layer_scratch_bytes(plan_n, plan_d, B) bytes, caller-owned.
 * ws_dev / ws_bytes: optional matmul workspace, at least the larger of m2_matmul_workspace_bytes(plan_n, B d) and
 * m2_matmul_workspace_bytes(plan_d, B n); NULL selects the kernels that need none.
 * The sequence mix runs through the columns-as-vectors kernels (m2_monarch_cols: x is [n, d] per batch entry with the
 * channels contiguous, so nothing but the [d, n] kernel parameter is transposed); the feature mix through the
 * rows-as-vectors kernels (m2_monarch_mix); the residual add and the normalisation are one kernel. */
int64_t m2_layer_scratch_bytes(const m2_plan* plan_n, const m2_plan* plan_d, int64_t B);
int32_t m2_layer_fwd(const m2_plan* plan_n, const m2_plan* plan_d, const void* x_dev, const void* const* factors,
                     const void* n_kernel_dev, const void* d_kernel_dev, const float* gamma_dev, const float* beta_dev,
                     float eps, void* y_dev, int64_t B, void* scratch_dev, int64_t scratch_bytes, void* ws_dev,
                     int64_t ws_bytes, void* stream);

/* The Monarch product on matrices whose COLUMNS are the vectors -- Eq. 2's M X with X in R^{N x d} stored row-major, the
 * layout of the paper's operator benchmark (Table 2: N = 4K .. 256K, block size sqrt(N), 768 columns):
 *   Y[bt] = sigma(K (.) (M X[bt])),  M = P L P^T R P,  bt < Bt,  sigma = identity or ReLU (M2_ACT_*).
 * X_dev, Y_dev: [Bt, N, d] in the plan dtype, d contiguous (Y_dev must not overlap X_dev); K_dev: [N, d], shared by the
 * batch, or NULL (then sigma is not applied either: Y = M X).  L_dev, R_dev as in m2_monarch_matmul.  ws_dev: caller-owned,
 * at least Bt N d elements of the plan dtype (the intermediate between the two factors), 16-byte aligned.
 * The M2 operator M_b (K (.) M_a X) is two calls, the first with K, the second without.
 * With the columns contiguous both factors are batched GEMMs over rows and the stride permutations are strides of TMA
 * tensor maps: bf16 plans whose factors N1, N2 are multiples of 64 (up to 1024) with d a multiple of 8 run on the tensor cores, two
 * launches per call; everything else on a CUDA-core kernel (N <= 65535, else M2_ERR_UNSUPPORTED). */
int32_t m2_monarch_cols(const m2_plan* plan, const void* X_dev, const void* L_dev, const void* R_dev, const void* K_dev,
                        int32_t act, void* Y_dev, int64_t Bt, int64_t d, void* ws_dev, int64_t ws_bytes, void* stream);

/* The gated bidirectional sequence mixer of M2-BERT (Sec. 5.1 in words; Sec. 3.2's V (.) M2 (K1 (.) M1 (Q (.) K)) with M1, M2
 * the DFT and its inverse), x: [B, n, d] with n = the plan length (circular convolutions):
 *   Q, K, V = DW3(x W_q), DW3(x W_k), DW3(x W_v)    dense projections, then width-3 depthwise filters along the sequence
 *                                                   (DW3(a)[t] = w0 a[t-1] + w1 a[t] + w2 a[t+1], zero padded)
 *   y = ( V (.) conv(k, Q (.) K) + conv(k_res, x) ) W_o
 * (the paper gives this block in words and a figure: where the residual convolution taps the input and the output
 * projection are this library's reading).
 * W: HOST array of 4 device pointers {W_q, W_k, W_v, W_o}, each [d][d] stored outputs x inputs; w_short: HOST array of 3
 * device pointers to fp32 [d][3] filters (q, k, v); kf_dev, kf_res_dev: m2_kernel_spectrum of k and k_res [d, n].
 * y_dev: [B, n, d] (must not overlap x_dev); scratch_dev: m2_bert_mixer_scratch_bytes(plan, B, d) bytes, caller-owned.
 * After one transposition everything runs channel-first: projections = the single-block column-layout kernel, the two
 * convolutions = m2_monarch_conv_fwd, two elementwise kernels for the filters and gates. */
int64_t m2_bert_mixer_scratch_bytes(const m2_plan* plan, int64_t B, int64_t d);
int32_t m2_bert_mixer_fwd(const m2_plan* plan, const void* x_dev, const void* const* W, const float* const* w_short,
                          const void* kf_dev, const void* kf_res_dev, void* y_dev, int64_t B, int64_t d, void* scratch_dev,
                          int64_t scratch_bytes, void* stream);

/* The M2 Hyena layer with heads (App. "GPT Causal Language Modeling", the algorithm of that name), u: [B, n, d]:
 *   X1, X2, V = u W_X1, u W_X2, u W_V;  X1~, X2~, V~ = causal Monarch convolution of every channel with a short kernel;
 *   per head of dh channels: XV[t] = X2~[t] V~[t]^T, each of its dh^2 sequences through the causal Monarch convolution with
 *   the head's long kernel; O[t] = X1~[t] XV[t];  y = concat(O) W_O.
 * plan: the convolution plan, N >= 2 n (the convolutions are m2_monarch_conv_fwd in M2_CAUSAL mode on channel-first rows).
 * W: HOST array of 4 device pointers {W_X1, W_X2, W_V, W_O}, each [d][d] stored outputs x inputs (y[o] = sum_i W[o][i] u[i]).
 * kf1_dev, kf2_dev, kf3_dev: m2_kernel_spectrum of the short kernels [d, n];  kf_long_dev: m2_kernel_spectrum of the long
 * kernels, one row per head: [d / dh, n] (the dh^2 sequences of a head share its row: m2_monarch_conv_fwd_grouped).
 * y_dev: [B, n, d] (must not overlap u_dev).  scratch_dev: m2_hyena_scratch_bytes(plan, B, n, d, dh) bytes, caller-owned
 * ((7 + 2 dh) tensors of B d n elements; 7 for heads of dh = 16 on the bf16 N = 512 plan with n a multiple of 16 up to 256, where
 * outer product, long convolution and contraction are one tensor-core kernel and the dh-times larger tensors do not exist).
 * The projections are the single-block case of the column-layout Monarch kernel (tensor cores for d a multiple of 64 up
 * to 4096 and n a multiple of 8, bf16), so after one transposition everything runs channel-first. */
int64_t m2_hyena_scratch_bytes(const m2_plan* plan, int64_t B, int64_t n, int64_t d, int64_t dh);
int32_t m2_hyena_heads_fwd(const m2_plan* plan, const void* u_dev, const void* const* W, const void* kf1_dev,
                           const void* kf2_dev, const void* kf3_dev, const void* kf_long_dev, void* y_dev, int64_t B,
                           int64_t n, int64_t d, int64_t dh, void* scratch_dev, int64_t scratch_bytes, void* stream);

/* W_out[b][c][r] = W_in[b][r][c]: block-wise transpose of a block-diagonal factor of nblocks blocks of rows x cols
 * elements of the plan dtype (W_out must not overlap W_in).  It gives the gradient of the Monarch matmul with
 * respect to its input: M^T = P^T R^T P L^T P^T (Sec. 3.1 transposed) is again an order-2 Monarch product, so for an
 * upstream gradient G of Y
 *   dX = m2_monarch_matmul(plan', G, L' = blocks_transpose(R), R' = blocks_transpose(L), ...)
 * where plan' has the factors in the opposite order (N2, N1) -- the same plan when N1 == N2 -- and L', R' have
 * the shapes of R, L.  (The paper trains through the operator, Sec. 5, without writing the backward pass out.) */
int32_t m2_blocks_transpose(const m2_plan* plan, const void* W_in_dev, void* W_out_dev, int64_t nblocks, int64_t rows,
                            int64_t cols, void* stream);

/* Order-p Monarch product Y_t = M X_t in the direct form (Eq. 1; App. D.6, "p-variate Monarch") for a plan of any order
 * p = 1..3 with arbitrary (learnable) blocks.  With the input index n = (n_1, .., n_p), n_1 most significant, stage
 * a = 1..p contracts the digit n_a into the output digit k_a with the block chosen by (k_1, .., k_{a-1}, n_{a+1}, .., n_p);
 * the output index is k = k_1 + N_1 k_2 + .. (natural order).  W_dev: HOST array of p DEVICE pointers; W_dev[a-1] is
 * [N / N_a][N_a out][N_a in] of the plan dtype, the block id being the row-major flattening of
 * (k_1, .., k_{a-1}, n_{a+1}, .., n_p).  (For p >= 3 the paper gives the block index as a tuple only: this linear order is
 * this library's reading.)  For p = 2, W_dev = {R, L} gives exactly m2_monarch_matmul.  X_dev, Y_dev: [T, N] of the plan
 * dtype, must not overlap; fp32 accumulation, the row stays in fp32 between the stages.  One CUDA-core kernel; needs
 * every N_a <= 256 and N <= 51200 (M2_ERR_UNSUPPORTED otherwise).  T == 0 is a no-op. */
int32_t m2_monarch_apply_order_p(const m2_plan* plan, const void* X_dev, const void* const* W_dev, void* Y_dev, int64_t T,
                                 void* stream);

/* Gradients of sum_t <Y_t, G_t>, Y = M X with M = P L P^T R P (Sec. 3.1), with respect to the blocks of L and R:
 *   dL[k1][k2][n2] = sum_t G[t][k2 N1 + k1] v[t][n2][k1],           v  = R-stage of the forward pass,
 *   dR[n2][k1][n1] = sum_t dv[t][n2][k1] X[t][n1 N2 + n2],          dv = L^T-stage applied to G.
 * X_dev, G_dev: [T, N], L_dev, R_dev as in m2_monarch_matmul (plan dtype); dL_dev [N1][N2][N2] and dR_dev [N2][N1][N1]
 * are fp32 and overwritten (zeros for T == 0).  ws_dev: caller-owned, at least m2_matmul_bwd_workspace_bytes(plan, T)
 * bytes (at least 4 T N: it holds v, then dv; bf16 plans with 64 x 64 blocks add room for the partial sums of the
 * token shares and one transposed factor), 16-byte aligned; too small or NULL with T > 0: M2_ERR_INVALID_ARG.
 * bf16 plans with 64 x 64 blocks run on the tensor cores with the tokens as the contraction dimension (v and dv pass
 * through bf16 like the forward intermediate; partial sums per token share in fp32, added in a fixed order); every
 * other plan runs four fp32 CUDA-core kernels with a fixed summation order.  Both are deterministic.  (The paper
 * trains through the operator, Sec. 5, without writing the backward pass out.) */
int64_t m2_matmul_bwd_workspace_bytes(const m2_plan* plan, int64_t T);
int32_t m2_monarch_matmul_bwd_weights(const m2_plan* plan, const void* X_dev, const void* G_dev, const void* L_dev,
                                      const void* R_dev, float* dL_dev, float* dR_dev, int64_t T, void* ws_dev,
                                      int64_t ws_bytes, void* stream);

/* M2 block forward for the M2-BERT-base shape (Eq. 2-3; Sec. 5.1): along the sequence, per channel,
 * v = circular Monarch conv of x with the channel's kernel; gate g = depthwise conv of width 3
 * (centred, zero padded); z = g (.) v; then the block-diagonal MLP y = bd(W_down) GELU(bd(W_up) z)
 * with nblk blocks (exact erf GELU).  x_dev, y_dev: [B, T, C] bf16 with T == N of the plan;
 * kf_dev: spectrum of k[C, T]; w_short_dev: [C, 3] float32; W_up_dev: [nblk, E*C/nblk, C/nblk] bf16;
 * W_down_dev: [nblk, C/nblk, E*C/nblk] bf16; z_dev: B*T*C bf16 of scratch that receives z.  z_dev and y_dev
 * must not overlap x_dev or each other; both are also used as scratch while the call runs.
 * Layout of z on return: [B, T, C] like x, except where m2_block_z_channel_first(plan, T, C, nblk, E) returns 1: there
 * z is left channel-first, [B, C, T], the layout the tensor-core sequence mixer works in and the tensor-core MLP reads
 * as it lies (bf16 plans with N = 512 = 32 x 16 and blocks of 192 -> 768 -> 192; x is transposed once on the way in,
 * convolution and gate are one kernel, nothing is transposed back).  The query is host-only arithmetic on the plan and
 * the shape; it returns 0 for bad arguments. */
int32_t m2_block_z_channel_first(const m2_plan* plan, int64_t T, int64_t C, int32_t nblk, int32_t expand);
int32_t m2_block_fwd(const m2_plan* plan, const void* x_dev, const void* kf_dev, const float* w_short_dev,
                     const void* W_up_dev, const void* W_down_dev, void* z_dev, void* y_dev, int64_t B,
                     int64_t T, int64_t C, int32_t nblk, int32_t expand, void* stream);

/* The same block forward as m2_block_fwd for callers that must not allocate device memory and have
 * no scratch buffer of their own to hand in.  (The paper has no counterpart: this is a deployment
 * variant, not a different operation.)  Typical callers: a serving process whose framework has
 * already taken all device memory into its own pool, so a cudaMalloc here would fail or eat into that
 * pool's reserve; or a latency-critical loop that cannot afford the device-wide synchronisation a
 * cudaMalloc / cudaFree implies.  The intermediate z lives in a fixed array inside the library:
 * M2_STATIC_SCRATCH_BYTES of device memory on every GPU that loads libm2.so, held until the process exits.
 *
 *  - B*T*C*2 bytes must not exceed M2_STATIC_SCRATCH_BYTES, else M2_ERR_UNSUPPORTED (nothing is launched).
 *  - The call allocates nothing and frees nothing.  The first call on each device looks up the address of
 *    the array (once per device, kept afterwards); make that first call before any stream capture begins.
 *  - All calls on a device share the one array.  It keeps whatever the previous call left in it; that is
 *    harmless because every call overwrites the part it later reads, nothing needs to start at zero.
 *    Two calls whose kernels overlap on the GPU (different streams without ordering between them) race on it:
 *    order them on one stream or with events.
 *  - Arguments, shapes, dtypes and results are otherwise exactly those of m2_block_fwd; z is not returned. */
#define M2_STATIC_SCRATCH_BYTES (8u * 1024u * 1024u)
int32_t m2_block_fwd_static(const m2_plan* plan, const void* x_dev, const void* kf_dev, const float* w_short_dev,
                            const void* W_up_dev, const void* W_down_dev, void* y_dev, int64_t B, int64_t T,
                            int64_t C, int32_t nblk, int32_t expand, void* stream);

/* Learnable (causal) Monarch matrices from polynomial coefficients, block size b = sqrt(N) (App. D.5: Alg. BlockyMonarch; the
 * lemma on masking and basis degrees; Alg. BlockMonarchConv; the theorem on causal block Monarch convolution).  `plan` is an
 * order-2 plan with N1 = N2 = b, 2 <= b <= 64 (M2_ERR_UNSUPPORTED otherwise).
 *
 * m2_blocky_monarch: Lt_dev, Rt_dev are float32 [N][b] coefficient matrices: column j of Lt holds the coefficients of
 *   l_j(Z) = sum_a Lt[a][j] Z^a; Rt is b stacked [b][b] blocks, column j of block c holds r~_{c,j}(Y) = sum_a Rt[c b + a][j] Y^a.
 *   It writes the factor set of M = P L P R P into factors_dev (m2_blocky_factors_bytes(plan) bytes, caller-owned, 16-byte
 *   aligned, opaque): L[k1][k2][n2] = l_{n2}(w_N^{k2 b + k1}), R[n2][k1][n1] = r~_{n2,n1}(w_b^{k1}) -- so that column
 *   j1 b + j0 of M is the basis polynomial l_{j0}(Z) r~_{j0,j1}(Z^b) on the N-th roots of unity -- and the block inverses of
 *   both (M^-1 = P R^-1 P L^-1 P).  Of the two formulas App. D.5 prints for the blocks of L this is the one used in the proof
 *   that the DFT is such an M.  causal_mask != 0 applies the lemma's zero patterns while reading: of Lt only entries
 *   [a][j] with j <= a < b survive; of every block of Rt entry [a][j] is dropped where a < j, or a >= b/2 and j < b/2; the
 *   diagonals must be non-zero.  Evaluation and inversion run in fp64, the results are stored as complex fp32.  A block that
 *   cannot be inverted sets M2_ERR_SINGULAR in the plan's status word (m2_last_device_status) and leaves zeros as its inverse.
 *   Meant to run once per weight update.
 * m2_blocky_kernel_spectrum: kf_dev[h] = M (k[h], 0) in plan order, complex fp32 [H][N] (k_dev float32 [H][n], n <= N).
 * m2_blocky_monarch_conv_fwd: y = Re( M^-1 ( kf[h] (.) M (x, 0) ) )[0:n) per row; x_dev, y_dev [B][H][n] in the plan dtype,
 *   2 n <= N.  With masked factors the map x -> y is causal (f[i] depends on x[0..i] only) and its imaginary part vanishes;
 *   with the DFT's coefficients (identity blocks in Rt, identity on top of Lt) it is the causal convolution.  CUDA-core
 *   kernels, fp32 arithmetic: a general M has no fast structure beyond its two block-diagonal factors. */
int64_t m2_blocky_factors_bytes(const m2_plan* plan);
int32_t m2_blocky_monarch(const m2_plan* plan, const float* Lt_dev, const float* Rt_dev, int32_t causal_mask, void* factors_dev,
                          void* stream);
int32_t m2_blocky_kernel_spectrum(const m2_plan* plan, const void* factors_dev, const float* k_dev, int64_t H, int64_t n,
                                  void* kf_dev, void* stream);
int32_t m2_blocky_monarch_conv_fwd(const m2_plan* plan, const void* factors_dev, const void* x_dev, const void* kf_dev,
                                   void* y_dev, int64_t B, int64_t H, int64_t n, void* stream);

/* Self-test of the device-side bounded waits (the paper has no counterpart; a test and diagnosis aid).  Every wait
 * inside the tensor-core kernels -- for a TMA copy, for a tensor-core commit -- gives up after a fixed number of
 * polls; the pipeline that gave up sets M2_ERR_TIMEOUT in the plan's status word, waits (again bounded) for its own
 * copies in flight, releases its tensor memory and returns, so that the context stays usable.  This call launches the
 * row-pair N = 512 convolution kernel with the arguments of m2_monarch_conv_fwd in a mode where no input copy is issued
 * and every wait gives up after a few polls: each pipeline's first wait runs out with nothing in flight and the kernel
 * leaves through that abort path.  y_dev is not written.  Afterwards m2_last_device_status reports M2_ERR_TIMEOUT
 * (and resets it) and the plan serves ordinary calls as before.  Needs a bf16 plan with N = 512 = 32 x 16 and B > 8;
 * M2_ERR_UNSUPPORTED otherwise. */
int32_t m2_selftest_bounded_wait(const m2_plan* plan, const void* x_dev, const void* kf_dev, void* y_dev, int64_t B,
                                 int64_t H, int64_t n, int32_t mode, void* stream);

/* The same self-test for the tensor-core Monarch matmul (bf16 plans with 64 x 64 blocks): launches the two passes of
 * m2_monarch_matmul with its arguments in a mode where the issuing threads give the tensor core nothing and every wait
 * for it gives up after a few polls, so that the loading, draining and issuing warps of every CTA leave through their
 * abort paths.  Y_dev and ws_dev are not written.  Afterwards m2_last_device_status reports M2_ERR_TIMEOUT (and resets
 * it) and the plan serves ordinary calls as before.  Needs T > 0, X_dev on a 32-byte boundary and a workspace of
 * m2_matmul_workspace_bytes(plan, T) bytes; M2_ERR_UNSUPPORTED otherwise. */
int32_t m2_selftest_bounded_wait_matmul(const m2_plan* plan, const void* X_dev, const void* L_dev, const void* R_dev,
                                        void* Y_dev, int64_t T, void* ws_dev, int64_t ws_bytes, void* stream);

const char* m2_status_string(int32_t status);

/* Reads (synchronously) the device status word kernels set when a bounded wait expires or a
 * self-check fails; 0 = clean.  Resets it. */
int32_t m2_last_device_status(const m2_plan* plan, int32_t* out);

/* Which implementation the last hot call on this plan dispatched to (a static string such as
 * "conv_generic_fp32" or "conv_umma_o2"); for tests and the benchmark's report. */
const char* m2_last_kernel_name(const m2_plan* plan);

/* Number of kernels the library has launched on this plan since creation. */
int64_t m2_launch_count(const m2_plan* plan);

#ifdef __cplusplus
}
#endif
#endif /* M2_H_ */
