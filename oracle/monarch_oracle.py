"""CPU oracle for the Monarch Mixer hot path (arXiv 2310.12109).

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain, double-precision
statement of what the GPU library must compute.  Only the tests, the smoke
check and the benchmark's CPU-baseline leg may import it; the product path
never does, and this module imports nothing from the product package.

Two tiers:

* Tier 1 -- the plain definitions the method reaches exactly (up to rounding):
  stride permutation matrices, block-diagonal matrices, the dense product
  ``P L P^T R P``, the DFT matrix, direct O(N^2) circular / causal convolution,
  and the element-wise pieces of the M2 block (depthwise conv, GELU, dense
  block-diagonal MLP).
* Tier 2 -- the method step by step in the paper's order: factored Monarch
  apply (permute, block-diagonal multiply, permute, ...), the Monarch factors
  that make ``M = F_N`` (Corollary "DFT is M", App. D.5), and the Monarch
  convolution ``M^-1 (M k  (.)  M u)`` (Eq. 2, Def. "matrix convolution",
  Alg. BlockMonarchConv).  Tier 2 is itself pinned to tier 1 by the CPU tests.

All arithmetic is float64 / complex128.  Index conventions (App. D notation):
``N = N1*N2*...*Np``; the input index is ``n = (..(n1*N2 + n2)*N3 + ..)`` with
n1 most significant; the natural output index is ``k = k1 + N1*k2 + N1*N2*k3``
with k1 least significant.  "Plan order" is the tensor ``[k1][k2]..[kp]`` stored
row-major.

Pins (see tests/test_oracle_*.py): permutation closed forms and inverses,
``M == F_N`` entry-wise, numpy's FFT (a different algorithm) for large N,
brute-force convolution sums, Parseval, delta / shift kernels, causality,
explicit dense products on tiny N.  Unpinned by the paper: the linear order of
order-p block ids for p >= 3 with arbitrary (non-DFT) blocks, and the wiring of
the M2 block composition (gate, short conv alignment, block count) -- marked
"parity unpinned" at the functions concerned.
"""
from __future__ import annotations

import math

import numpy as np

# ----------------------------------------------------------------------------
# Tier 1: definitions
# ----------------------------------------------------------------------------


def stride_perm(b: int, N: int) -> np.ndarray:
    """sigma_(b,N)(i) = i0 * N/b + i1 for i = i1*b + i0 (App. D notation, item on
    the permutation class P_(b,N))."""
    if b <= 0 or N % b != 0:
        raise ValueError("b must divide N")
    i = np.arange(N, dtype=np.int64)
    i0 = i % b
    i1 = i // b
    return i0 * (N // b) + i1


def perm_matrix(b: int, N: int) -> np.ndarray:
    """P_(b,N): the N x N matrix whose i-th row is e_{sigma_(b,N)(i)}, so that
    (P x)[i] = x[sigma(i)] (App. D notation)."""
    P = np.zeros((N, N))
    P[np.arange(N), stride_perm(b, N)] = 1.0
    return P


def apply_perm(b: int, N: int, x: np.ndarray) -> np.ndarray:
    """(P_(b,N) x) along the last axis."""
    return x[..., stride_perm(b, N)]


def blockdiag_dense(W: np.ndarray) -> np.ndarray:
    """Dense matrix of a block-diagonal factor.  W has shape [nblocks, out, in]
    (the weight layout of the paper's blockdiag_matmul listing, App. A)."""
    nb, o, i = W.shape
    D = np.zeros((nb * o, nb * i), dtype=W.dtype)
    for b in range(nb):
        D[b * o:(b + 1) * o, b * i:(b + 1) * i] = W[b]
    return D


def monarch_dense(L: np.ndarray, R: np.ndarray) -> np.ndarray:
    """Dense order-2 Monarch matrix M = P L P^T R P (Sec. 3.1) with P = P_(N1,N).

    R: [N2, N1, N1] (N2 blocks, applied first), L: [N1, N2, N2] (N1 blocks).
    For square N (N1 == N2) P^T = P and this is the paper's M = P L P R P."""
    N2, N1, _ = R.shape
    assert R.shape == (N2, N1, N1) and L.shape == (N1, N2, N2)
    N = N1 * N2
    P = perm_matrix(N1, N)
    return P @ blockdiag_dense(L) @ P.T @ blockdiag_dense(R) @ P


def dft_matrix(N: int, sign: int = +1) -> np.ndarray:
    """F_N[i, j] = omega_N^{i j}, omega_N = exp(sign * 2 pi i / N).  The paper uses
    sign = +1 (App. D, definition of the roots of unity)."""
    idx = np.arange(N)
    # reduce the exponent modulo N in integers so large N stays accurate
    e = (np.outer(idx, idx) % N).astype(np.float64)
    return np.exp(sign * 2j * np.pi * e / N)


def direct_circular_conv(k: np.ndarray, x: np.ndarray) -> np.ndarray:
    """y[t] = sum_{u=0}^{N-1} k[u] x[(t-u) mod N], along the last axis."""
    N = x.shape[-1]
    assert k.shape[-1] == N
    y = np.zeros(np.broadcast_shapes(k.shape, x.shape), dtype=np.result_type(k, x))
    t = np.arange(N)
    for u in range(N):
        y += k[..., u:u + 1] * x[..., (t - u) % N]
    return y


def direct_causal_conv(k: np.ndarray, x: np.ndarray) -> np.ndarray:
    """y[t] = sum_{u=0}^{t} k[u] x[t-u], 0 <= t < n: multiplication by the lower
    triangular Toeplitz matrix of k (App. D.3, review of causal maps)."""
    n = x.shape[-1]
    assert k.shape[-1] == n
    y = np.zeros(np.broadcast_shapes(k.shape, x.shape), dtype=np.result_type(k, x))
    for u in range(n):
        y[..., u:] += k[..., u:u + 1] * x[..., :n - u]
    return y


def direct_circular_conv_adjoint(k: np.ndarray, g: np.ndarray) -> np.ndarray:
    """Transpose of the circulant map x -> direct_circular_conv(k, x) applied to g:
    dx[s] = sum_{t=0}^{N-1} g[t] k[(t-s) mod N] (the gradient of <y, g> with respect to x)."""
    N = g.shape[-1]
    out = np.zeros(np.broadcast_shapes(k.shape, g.shape), dtype=np.result_type(k, g))
    for s_ in range(N):
        idx = (np.arange(N) - s_) % N
        out[..., s_] = np.sum(g * k[..., idx], axis=-1)
    return out


def direct_causal_conv_adjoint(k: np.ndarray, g: np.ndarray) -> np.ndarray:
    """Transpose of the lower-triangular Toeplitz map of direct_causal_conv (App. D.3, T_k):
    dx[s] = sum_{t=s}^{n-1} g[t] k[t-s], 0 <= s < n."""
    n = g.shape[-1]
    out = np.zeros(np.broadcast_shapes(k.shape, g.shape), dtype=np.result_type(k, g))
    for s_ in range(n):
        out[..., s_] = np.sum(g[..., s_:] * k[..., : n - s_], axis=-1)
    return out


def depthwise_conv3_same(x: np.ndarray, w: np.ndarray) -> np.ndarray:
    """Short depthwise convolution of width 3 along the sequence, centred, zero
    padded: g[b,t,c] = w[c,0] x[b,t-1,c] + w[c,1] x[b,t,c] + w[c,2] x[b,t+1,c].
    x: [B, T, C], w: [C, 3].  (Sec. 5.1 mentions the short conv only in words;
    alignment is this build's reading -- parity unpinned.)"""
    B, T, C = x.shape
    g = w[:, 1] * x
    g[:, 1:, :] += w[:, 0] * x[:, :-1, :]
    g[:, :-1, :] += w[:, 2] * x[:, 1:, :]
    return g


def gelu_erf(v: np.ndarray) -> np.ndarray:
    """GELU(v) = v/2 * (1 + erf(v / sqrt 2)), evaluated with math.erf."""
    erf = np.vectorize(math.erf, otypes=[np.float64])
    return 0.5 * v * (1.0 + erf(v / math.sqrt(2.0)))


def blockdiag_apply(W: np.ndarray, x: np.ndarray) -> np.ndarray:
    """Multiplication by the block-diagonal matrix diag(W[0], .., W[nb-1]) of Sec. 3.1 along the last axis: the vector
    is cut into nb consecutive segments and segment b is multiplied by its own block W[b] (out x in), one block after
    the other."""
    nb, o, i = W.shape
    assert x.shape[-1] == nb * i
    out = np.empty(x.shape[:-1] + (nb * o,), dtype=np.result_type(W.dtype, x.dtype))
    for b in range(nb):
        seg = x[..., b * i:(b + 1) * i]                       # the inputs of block b
        out[..., b * o:(b + 1) * o] = seg @ W[b].T            # (W[b] seg) for every leading index
    return out


# ----------------------------------------------------------------------------
# Tier 2: the method, step by step
# ----------------------------------------------------------------------------


def monarch_apply(L: np.ndarray, R: np.ndarray, x: np.ndarray, stages: dict | None = None) -> np.ndarray:
    """y = P L P^T R P x along the last axis, evaluated as the paper evaluates it
    (Sec. 3.1 and the MonarchMatrix listing): permute, block-diagonal multiply
    with R, permute, block-diagonal multiply with L, permute.  No dense N x N
    matrix is formed.  `stages`, if given, receives every intermediate."""
    N2, N1, _ = R.shape
    N = N1 * N2
    assert x.shape[-1] == N and L.shape == (N1, N2, N2)
    v0 = apply_perm(N1, N, x)            # [n2][n1]
    v1 = blockdiag_apply(R, v0)          # [n2][k1]
    v2 = apply_perm(N2, N, v1)           # P^T = P_(N/N1, N): [k1][n2]
    v3 = blockdiag_apply(L, v2)          # [k1][k2]   (plan order)
    y = apply_perm(N1, N, v3)            # [k2][k1]   (natural order)
    if stages is not None:
        stages.update(after_P=v0, after_R=v1, after_Pt=v2, after_L=v3, out=y)
    return y


def monarch_apply_transpose(L: np.ndarray, R: np.ndarray, g: np.ndarray) -> np.ndarray:
    """M^T g along the last axis for M = P L P^T R P (Sec. 3.1): the gradient of <M x, g> with respect to x.
    M^T = P^T R^T P L^T P^T with block-wise transposes; written with the inverse permutations explicitly."""
    N1, N2 = L.shape[0], R.shape[0]
    N = N1 * N2
    lead = g.shape[:-1]
    v = g.reshape(*lead, N2, N1)                      # g[k2, k1]; P^T: back to blocks indexed by k1
    v = np.swapaxes(v, -1, -2)                        # [k1][k2]
    v = np.einsum("bkn,...bk->...bn", L, v)           # L^T per block k1: [k1][n2]
    v = np.swapaxes(v, -1, -2)                        # P: [n2][k1]
    v = np.einsum("bkn,...bk->...bn", R, v)           # R^T per block n2: [n2][n1]
    v = np.swapaxes(v, -1, -2)                        # P^T: [n1][n2]
    return v.reshape(*lead, N)


def monarch_mix(La, Ra, Lb, Rb, K: np.ndarray, x: np.ndarray, act: str = "none") -> np.ndarray:
    """The M2 operator y = M_b sigma(K (.) M_a x) along the last axis (Eq. 2 with general Monarch matrices; the M2
    layer listing applies it once along the sequence and once along the features with sigma = ReLU).  x: [T, N];
    K: [Hk, N], row t of x takes row t mod Hk of K (Hk = T: one kernel row per row; Hk = 1: one shared row)."""
    assert act in ("none", "relu")
    T = x.shape[0]
    mid = K[np.arange(T) % K.shape[0]] * monarch_apply(La, Ra, x)
    if act == "relu":
        mid = np.maximum(mid, 0.0)
    return monarch_apply(Lb, Rb, mid)


def monarch_cols(L, R, X: np.ndarray, K: np.ndarray | None = None, act: str = "none") -> np.ndarray:
    """Y = sigma(K (.) M X) for X [.., N, d] whose COLUMNS are the vectors (Eq. 2's M X with X in R^{N x d}); K: [N, d]
    or None (then no sigma either).  The Monarch apply itself is monarch_apply along axis -2."""
    Y = np.swapaxes(monarch_apply(L, R, np.swapaxes(X, -1, -2)), -1, -2)
    if K is not None:
        Y = K * Y
        if act == "relu":
            Y = np.maximum(Y, 0.0)
    return Y


def layer_norm(v: np.ndarray, gamma: np.ndarray, beta: np.ndarray, eps: float = 1e-5) -> np.ndarray:
    """LayerNorm over the last axis: (v - mean) / sqrt(var + eps) * gamma + beta with the biased variance."""
    mu = v.mean(axis=-1, keepdims=True)
    var = ((v - mu) ** 2).mean(axis=-1, keepdims=True)
    return (v - mu) / np.sqrt(var + eps) * gamma + beta


def m2_layer(x: np.ndarray, p: dict, eps: float = 1e-5, stages: dict | None = None) -> np.ndarray:
    """The basic M2 layer (App. "Implementation", the MonarchMixerLayer listing), x: [B, n, d]:
        x~ = (M2 relu(K_n (.) M1 x^T))^T                 mix along the sequence, K_n: [d, n]
        y  = M4 relu(k_d (.) M3 x~)                      mix along the features, k_d: [1, d]
        out = LayerNorm(y + x~).
    p: factors "L1","R1",..,"L4","R4" in this library's convention (R is applied first: the listing's parameter
    called L), "n_kernel", "d_kernel", "gamma", "beta"."""
    B, n, d = x.shape
    xT = np.swapaxes(x, 1, 2).reshape(B * d, n)                                        # rows (b, channel)
    u = monarch_mix(p["L1"], p["R1"], p["L2"], p["R2"], p["n_kernel"], xT, "relu")     # row (b, c) takes K_n[c]
    xt = np.swapaxes(u.reshape(B, d, n), 1, 2)                                         # [B, n, d]
    y = monarch_mix(p["L3"], p["R3"], p["L4"], p["R4"], p["d_kernel"], xt.reshape(B * n, d), "relu").reshape(B, n, d)
    out = layer_norm(y + xt, p["gamma"], p["beta"], eps)
    if stages is not None:
        stages.update(x_tilde=xt, y=y)
    return out


def m2_bert_mixer(x: np.ndarray, p: dict, dims: tuple, stages: dict | None = None) -> np.ndarray:
    """The gated bidirectional sequence mixer of M2-BERT (Sec. 5.1 in words; Sec. 3.2's "more expressive layer"
    V (.) M2 (K1 (.) M1 (Q (.) K)) with M1, M2 the DFT and its inverse), x: [B, n, d], n = prod(dims):
        Q, K, V = DW3(x W_q), DW3(x W_k), DW3(x W_v)          dense projections, then the short depthwise convolutions
        y = ( V (.) circconv(k, Q (.) K) + circconv(k_res, x) ) W_o     gated convolution + residual convolution, output projection
    Weights act as x @ W ([d_in, d_out]); k, k_res: [d, n]; w_q, w_k, w_v: [d, 3].
    (The paper gives this block in words and a figure only: where the residual convolution taps the input and the output
    projection are this build's reading -- parity of the composition unpinned.)"""
    cm = lambda a: np.swapaxes(a, 1, 2)
    Q = depthwise_conv3_same(x @ p["W_q"], p["w_q"])
    K = depthwise_conv3_same(x @ p["W_k"], p["w_k"])
    V = depthwise_conv3_same(x @ p["W_v"], p["w_v"])
    C = monarch_conv(p["k"][None], cm(Q * K), dims, causal=False)            # [B, d, n]
    Cr = monarch_conv(p["k_res"][None], cm(x), dims, causal=False)
    Z = V * cm(C) + cm(Cr)
    if stages is not None:
        stages.update(Q=Q, K=K, V=V, C=C, Cr=Cr, Z=Z)
    return Z @ p["W_o"]


def m2_hyena_heads(u: np.ndarray, p: dict, dims: tuple, dh: int, stages: dict | None = None) -> np.ndarray:
    """The M2 Hyena layer with heads (App. "GPT Causal Language Modeling", the algorithm of that name), u: [B, n, d]:
        X1, X2, V = u W_X1, u W_X2, u W_V                                     (dense projections)
        X1~, X2~, V~ = causal Monarch convolution of each channel with the short kernels K1, K2, K3 [d, n]
        per head h (d_h channels): XV[t] = X2~[t] V~[t]^T (d_h x d_h per position), each of its d_h^2 sequences through the
        causal Monarch convolution with the head's long kernel K_long[h]; O[t] = X1~[t] XV[t]  (row vector times matrix)
        y = concat_h(O) W_O.
    Weights act as u @ W with W: [d_in, d_out].  The convolutions are monarch_conv with the plan's factorisation `dims`
    (N = prod(dims) >= 2 n)."""
    B, n, d = u.shape
    Hh = d // dh
    assert Hh * dh == d
    cm = lambda a: np.swapaxes(a, 1, 2)                                       # [B, n, d] <-> [B, d, n]
    X1, X2, V = u @ p["W_x1"], u @ p["W_x2"], u @ p["W_v"]
    X1c = monarch_conv(p["K1"][None], cm(X1), dims, causal=True)             # [B, d, n]
    X2c = monarch_conv(p["K2"][None], cm(X2), dims, causal=True)
    Vc = monarch_conv(p["K3"][None], cm(V), dims, causal=True)
    x2h, vh, x1h = (a.reshape(B, Hh, dh, n) for a in (X2c, Vc, X1c))
    XV = np.einsum("bhit,bhjt->bhijt", x2h, vh)                              # outer product per position
    XVc = monarch_conv(p["K_long"][None, :, None, None, :], XV, dims, causal=True)
    O = np.einsum("bhit,bhijt->bhjt", x1h, XVc).reshape(B, d, n)
    y = cm(O) @ p["W_o"]
    if stages is not None:
        stages.update(X1c=X1c, X2c=X2c, Vc=Vc, XVc=XVc, O=O)
    return y


def monarch_weight_grads(L: np.ndarray, R: np.ndarray, x: np.ndarray, g: np.ndarray):
    """Gradients of sum_t <M x_t, g_t> with respect to the blocks of L and R for M = P L P^T R P (Sec. 3.1), by the
    chain rule through the stages of monarch_apply: with v0 = P x ([n2][n1]), v1 = R v0 ([n2][k1]) and the upstream
    gradient read in plan order gv[k1][k2] = g[k2 N1 + k1],
        dL[k1][k2][n2] = sum_t gv[t][k1][k2] v1[t][n2][k1]
        dv1[t][n2][k1] = sum_k2 L[k1][k2][n2] gv[t][k1][k2]
        dR[n2][k1][n1] = sum_t dv1[t][n2][k1] v0[t][n2][n1].
    x, g: [T, N].  Returns (dL, dR) with the shapes of L and R."""
    N2, N1, _ = R.shape
    T = x.shape[0]
    v0 = np.swapaxes(x.reshape(T, N1, N2), 1, 2)          # [t][n2][n1]
    v1 = np.einsum("nki,tni->tnk", R, v0)                 # [t][n2][k1]
    gv = np.swapaxes(g.reshape(T, N2, N1), 1, 2)          # [t][k1][k2]
    dL = np.einsum("tkq,tnk->kqn", gv, v1)                # [k1][k2][n2]
    dv1 = np.einsum("kqn,tkq->tnk", L, gv)                # [t][n2][k1]
    dR = np.einsum("tnk,tni->nki", dv1, v0)               # [n2][k1][n1]
    return dL, dR


def monarch_apply_order_p(blocks: list, dims: tuple, x: np.ndarray) -> np.ndarray:
    """Order-p Monarch apply in the direct form (App. D.6, "p-variate Monarch"):
    stage a (a = 1..p) contracts input digit n_a into output digit k_a with the
    block selected by (k1..k_{a-1}, n_{a+1}..n_p); blocks[a-1] has shape
    [prod(dims)/dims[a-1], dims[a-1], dims[a-1]] with the block id the row-major
    flattening of (k1, .., k_{a-1}, n_{a+1}, .., n_p).  Output in natural order
    k = k1 + N1 k2 + ...   (For p >= 3 with arbitrary blocks the paper gives the
    block index as a tuple only; the linear order here is this build's reading --
    parity unpinned.  The DFT instance does not depend on it.)"""
    p = len(dims)
    N = int(np.prod(dims))
    lead = x.shape[:-1]
    v = x.reshape(*lead, *dims)          # axes: n1..np
    nl = len(lead)
    for a in range(p):
        Na = dims[a]
        W = blocks[a].reshape(*dims[:a], *dims[a + 1:], Na, Na)   # (k1..k_{a-1}, n_{a+1}..np, out, in)
        # move the contracted axis last on the data
        vt = np.moveaxis(v, nl + a, -1)                           # (lead, k1..k_{a-1}, n_{a+1}..np, n_a)
        out = np.einsum("...oi,...i->...o", W, vt)                # per-block mat-vec
        v = np.moveaxis(out, -1, nl + a)
    # v axes are k1..kp; natural order has kp most significant
    perm = list(range(nl)) + [nl + a for a in reversed(range(p))]
    return np.transpose(v, perm).reshape(*lead, N)


def monarch_dft_factors(N1: int, N2: int, sign: int = +1):
    """Block-diagonal factors with P L P^T R P = F_N, N = N1 N2 (Corollary "DFT is
    M": l_{j1}(Z) = Z^{j1}, r~_{j1,j0}(Z) = Z^{j0}).  Every block of R is F_{N1};
    block k1 of L evaluates Z^{n2} at omega_N^{k1 + N1 k2}, i.e.
    L[k1][k2, n2] = omega_N^{(k1 + N1 k2) n2} = (F_{N2} diag(omega_N^{k1 n2}))[k2, n2]."""
    N = N1 * N2
    R = np.broadcast_to(dft_matrix(N1, sign), (N2, N1, N1)).copy()
    k1 = np.arange(N1)[:, None, None]
    k2 = np.arange(N2)[None, :, None]
    n2 = np.arange(N2)[None, None, :]
    e = ((k1 + N1 * k2) * n2) % N
    L = np.exp(sign * 2j * np.pi * e / N)
    return L, R


def monarch_dft_factors_order_p(dims: tuple, sign: int = +1) -> list:
    """Order-p generalisation of the corollary: stage a's block with id
    (k1..k_{a-1}, n_{a+1}..) is F_{Na} with its columns scaled by the twiddle
    omega_{N1..Na}^{n_a (k1 + N1 k2 + .. + N1..N_{a-2} k_{a-1})}; independent of
    the trailing n digits."""
    p = len(dims)
    blocks = []
    for a in range(p):
        Na = dims[a]
        Mprev = int(np.prod(dims[:a]))         # N1..N_{a-1}
        Mcur = Mprev * Na
        trail = int(np.prod(dims[a + 1:]))
        # kappa = k1 + N1 k2 + ... enumerated in block-id (row-major k1..k_{a-1}) order
        kappa = np.zeros((1,), dtype=np.int64)
        w = 1
        for j in range(a):
            kappa = (kappa[:, None] + w * np.arange(dims[j])[None, :]).reshape(-1)
            w *= dims[j]
        ka = np.arange(Na)[None, :, None]
        na = np.arange(Na)[None, None, :]
        e = (na * (kappa[:, None, None] + Mprev * ka)) % Mcur
        B = np.exp(sign * 2j * np.pi * e / Mcur)              # [Mprev, Na, Na]
        B = np.repeat(B[:, None], trail, axis=1).reshape(Mprev * trail, Na, Na)
        blocks.append(B)
    return blocks


def monarch_inverse_factors(L: np.ndarray, R: np.ndarray):
    """Block inverses: (P L P^T R P)^-1 = P^T R^-1 P L^-1 P^T with R^-1, L^-1 block
    diagonal (each block inverted on its own)."""
    return np.linalg.inv(L), np.linalg.inv(R)


def monarch_inverse_apply(Linv: np.ndarray, Rinv: np.ndarray, y: np.ndarray) -> np.ndarray:
    """x = P^T R^-1 P L^-1 P^T y (the factors of monarch_apply undone in reverse)."""
    N2, N1, _ = Rinv.shape
    N = N1 * N2
    v3 = apply_perm(N2, N, y)            # P^T: natural [k2][k1] -> [k1][k2]
    v2 = blockdiag_apply(Linv, v3)       # [k1][n2]
    v1 = apply_perm(N1, N, v2)           # P:   [n2][k1]
    v0 = blockdiag_apply(Rinv, v1)       # [n2][n1]
    return apply_perm(N2, N, v0)         # P^T: [n1][n2]


def plan_order_index(dims: tuple) -> np.ndarray:
    """pos -> natural frequency k for plan order: position ((k1*N2+k2)*N3+..)
    holds frequency k1 + N1 k2 + N1 N2 k3 + ...   (a digit reversal)."""
    p = len(dims)
    grids = np.meshgrid(*[np.arange(d) for d in dims], indexing="ij")
    k = np.zeros_like(grids[0])
    w = 1
    for a in range(p):
        k = k + w * grids[a]
        w *= dims[a]
    return k.reshape(-1).astype(np.int64)


def monarch_dft(x: np.ndarray, dims: tuple, sign: int = +1, plan_order: bool = False) -> np.ndarray:
    """F_N x by the factored Monarch apply (order len(dims)).  With plan_order the
    last permutation is left out and the result stays as [k1][k2].. row-major."""
    blocks = monarch_dft_factors_order_p(dims, sign)
    y = monarch_apply_order_p(blocks, dims, x.astype(np.complex128))
    if plan_order:
        return y[..., plan_order_index(dims)]
    return y


def monarch_conv(k: np.ndarray, x: np.ndarray, dims: tuple, causal: bool, sign: int = +1,
                 stages: dict | None = None) -> np.ndarray:
    """Monarch convolution f = M^-1 (M k' (.) M u') with M the Monarch-DFT
    (Alg. BlockMonarchConv with the corollary's factors; Eq. 2).

    causal: k, x have length n <= N/2; both are zero padded to N = prod(dims) and
    the first n outputs are kept (App. D.3 review; Thm 3).  Otherwise n == N and
    the result is the circular convolution.  k: [..., n] broadcastable against
    x: [..., n] (kernel per channel, shared over the batch)."""
    N = int(np.prod(dims))
    n = x.shape[-1]
    assert k.shape[-1] == n
    if causal:
        assert 2 * n <= N
        kp = np.concatenate([k, np.zeros((*k.shape[:-1], N - n))], axis=-1)
        xp = np.concatenate([x, np.zeros((*x.shape[:-1], N - n))], axis=-1)
    else:
        assert n == N
        kp, xp = k, x
    blocks = monarch_dft_factors_order_p(dims, sign)
    k_f = monarch_apply_order_p(blocks, dims, kp.astype(np.complex128))
    u_f = monarch_apply_order_p(blocks, dims, xp.astype(np.complex128))
    prod = k_f * u_f
    # M^-1 = conj(M) / N for the DFT: apply the conjugated factors, scale by 1/N
    cblocks = [np.conj(B) for B in blocks]
    f = monarch_apply_order_p(cblocks, dims, prod) / N
    if stages is not None:
        stages.update(k_f=k_f, u_f=u_f, prod=prod, f=f)
    return np.real(f[..., :n])


def monarch_conv_adjoint(k: np.ndarray, g: np.ndarray, dims: tuple, causal: bool, sign: int = +1) -> np.ndarray:
    """Gradient of <monarch_conv(k, x), g> with respect to x: the same Monarch convolution with the
    conjugated kernel spectrum, M^-1 (conj(M k') (.) M g') (k real: conj(F k) = F of the index-reversed
    kernel, which is the transposed circulant; zero padding makes the causal case exact for n <= N/2)."""
    N = int(np.prod(dims))
    n = g.shape[-1]
    assert k.shape[-1] == n
    if causal:
        assert 2 * n <= N
        kp = np.concatenate([k, np.zeros((*k.shape[:-1], N - n))], axis=-1)
        gp = np.concatenate([g, np.zeros((*g.shape[:-1], N - n))], axis=-1)
    else:
        assert n == N
        kp, gp = k, g
    blocks = monarch_dft_factors_order_p(dims, sign)
    k_f = monarch_apply_order_p(blocks, dims, kp.astype(np.complex128))
    g_f = monarch_apply_order_p(blocks, dims, gp.astype(np.complex128))
    f = monarch_apply_order_p([np.conj(B) for B in blocks], dims, np.conj(k_f) * g_f) / N
    return np.real(f[..., :n])


def direct_conv_kernel_grad(x: np.ndarray, g: np.ndarray, causal: bool) -> np.ndarray:
    """Gradient of sum_b <conv(k, x[b]), g[b]> with respect to k (the convolution is linear in k):
    dk[h, u] = sum_b sum_t g[b, h, t] x[b, h, t - u], indices taken mod N for the circular convolution and
    restricted to t >= u for the causal one.  x, g: [B, H, n]; result [H, n]."""
    B, H, n = x.shape
    dk = np.zeros((H, n), dtype=np.result_type(x, g))
    for u in range(n):
        if causal:
            dk[:, u] = np.sum(g[:, :, u:] * x[:, :, : n - u], axis=(0, 2))
        else:
            dk[:, u] = np.sum(g * np.roll(x, u, axis=-1), axis=(0, 2))
    return dk


def monarch_conv_kernel_grad(x: np.ndarray, g: np.ndarray, dims: tuple, causal: bool, sign: int = +1) -> np.ndarray:
    """The same gradient through the Monarch-DFT: dk = M^-1 ( sum_b conj(M x'_b) (.) M g'_b ) [0:n)
    (x real; zero padded to N = prod(dims) in the causal case)."""
    N = int(np.prod(dims))
    n = x.shape[-1]
    if causal:
        assert 2 * n <= N
        pad = np.zeros((*x.shape[:-1], N - n))
        xp, gp = np.concatenate([x, pad], axis=-1), np.concatenate([g, pad], axis=-1)
    else:
        assert n == N
        xp, gp = x, g
    blocks = monarch_dft_factors_order_p(dims, sign)
    x_f = monarch_apply_order_p(blocks, dims, xp.astype(np.complex128))
    g_f = monarch_apply_order_p(blocks, dims, gp.astype(np.complex128))
    acc = np.sum(np.conj(x_f) * g_f, axis=0)
    f = monarch_apply_order_p([np.conj(Bk) for Bk in blocks], dims, acc) / N
    return np.real(f[..., :n])


def m2_block_forward(x, k, w_short, W_up, W_down, dims=(32, 16)):
    """M2 block forward as configured for the M2-BERT-base shape (Sec. 5.1, Eq. 2-3):
    gate g = depthwise-conv3(x); long mix v = circular Monarch conv of x with k
    along the sequence per channel; z = g (.) v; MLP y = bd(W_down) GELU(bd(W_up) z)
    with 4-block block-diagonal matrices.  x: [B, T, C]; k: [C, T]; w_short: [C, 3];
    W_up: [4, 4C/4, C/4]; W_down: [4, C/4, 4C/4].  (Composition is this build's
    reading of the paper's prose -- parity unpinned; every piece is pinned.)"""
    g = depthwise_conv3_same(x, w_short)
    xt = np.transpose(x, (0, 2, 1))                       # [B, C, T]
    v = monarch_conv(k[None], xt, dims, causal=False)     # [B, C, T]
    z = g * np.transpose(v, (0, 2, 1))
    h = gelu_erf(blockdiag_apply(W_up, z))
    return blockdiag_apply(W_down, h), z


# ----------------------------------------------------------------------------
# Learnable (causal) Monarch matrices from polynomial coefficients (App. D.5, block size sqrt N)
# ----------------------------------------------------------------------------


def blocky_monarch(Lt: np.ndarray, Rt: np.ndarray, sign: int = +1):
    """Alg. BlockyMonarch: coefficient matrices -> the block-diagonal factors of M = P L P R P, N = b^2.

    Lt: [N, b], column j holds the N coefficients of l_j(Z) = sum_a Lt[a, j] Z^a.
    Rt: [N, b] = b stacked blocks Rt_c [b, b]; column j of block c holds the coefficients of
        r~_{c,j}(Y) = sum_a Rt_c[a, j] Y^a.
    Returns (L [b, b, b], R [b, b, b]) in this module's weight layout [block][out][in], complex.

    Steps, in the algorithm's order: F_N is taken as the Monarch matrix of the corollary "DFT is M";
    L' = P F_N Lt and block c of L is rows c b .. c b + b - 1 of L'; block c of R is F_b Rt_c.
    Reading (the appendix prints two formulas for the blocks of L that cannot both hold): the one used in the
    proof of the theorem on BlockyMonarch's return value, block i0 of L has entry [i1, j] = l_j(omega_N^{i1 b + i0});
    only this one makes the corollary true (pinned: identity coefficients give monarch_dft_factors).
    With it, M[i1 b + i0, j1 b + j0] = l_{j0}(w) r~_{j0,j1}(w^b), w = omega_N^{i1 b + i0}: column j of M is the basis
    polynomial l_{j0}(Z) r~_{j0,j1}(Z^b) at the N-th roots of unity."""
    N, b = Lt.shape
    assert b * b == N and Rt.shape == (N, b)
    FL, FR = monarch_dft_factors(b, b, sign)
    L2 = monarch_apply(FL, FR, Lt.T.astype(np.complex128)).T      # F_N Lt, column by column, by the factored apply
    L1 = apply_perm(b, N, L2.T).T                                 # P (F_N Lt): the rows permuted
    L = L1.reshape(b, b, b).copy()                                # block c = rows c b .. c b + b - 1
    Fb = dft_matrix(b, sign)
    R = np.stack([Fb @ Rt[c * b:(c + 1) * b, :] for c in range(b)])
    return L, R


def causal_coefficient_masks(b: int):
    """The zero patterns of the lemma on masking and basis degree (App. D.5): returns (mask_L [N, b], mask_R [N, b])
    of zeros and ones, N = b^2.
      Lt': only the top b x b block survives, and there only entries [i0, j] with i0 >= j  (l_j has minimum degree j
           and degree < b);
      Rt'_c[i0, j0] is zeroed where i0 < j0 (minimum degree j0) or where i0 >= floor(b/2) and j0 < floor(b/2)
           (degree < floor(b/2) for the first half of the columns)."""
    N = b * b
    mL = np.zeros((N, b))
    i0 = np.arange(b)[:, None]
    j = np.arange(b)[None, :]
    mL[:b, :] = (i0 >= j)
    h = b // 2
    blockR = ((i0 >= j) & ~((i0 >= h) & (j < h))).astype(np.float64)
    mR = np.tile(blockR, (b, 1))
    return mL, mR


def blocky_monarch_conv(Lt: np.ndarray, Rt: np.ndarray, k: np.ndarray, u: np.ndarray, sign: int = +1,
                        stages: dict | None = None) -> np.ndarray:
    """Alg. BlockMonarchConv with the padding of the theorem on causal block Monarch convolution:
    f = M^-1 ((M k') (.) (M u'))[0:n], k' = (k, 0), u' = (u, 0) of length N = b^2, M = P L P R P from
    blocky_monarch(Lt, Rt).  k: [..., n], u: [..., n] (broadcast against each other), n <= N/2.
    M^-1 is applied through the block inverses of L and R.  With the masked coefficient matrices
    (causal_coefficient_masks, non-zero diagonals) the map u -> f is causal and f is real up to rounding; the complex
    result is returned so that tests can check that."""
    N, b = Lt.shape
    n = u.shape[-1]
    assert k.shape[-1] == n and 2 * n <= N
    L, R = blocky_monarch(Lt, Rt, sign)
    Linv, Rinv = monarch_inverse_factors(L, R)
    kp = np.concatenate([k, np.zeros((*k.shape[:-1], N - n))], axis=-1).astype(np.complex128)
    up = np.concatenate([u, np.zeros((*u.shape[:-1], N - n))], axis=-1).astype(np.complex128)
    k_f = monarch_apply(L, R, kp)
    u_f = monarch_apply(L, R, up)
    f = monarch_inverse_apply(Linv, Rinv, k_f * u_f)
    if stages is not None:
        stages.update(L=L, R=R, Linv=Linv, Rinv=Rinv, k_f=k_f, u_f=u_f, f=f)
    return f[..., :n]
