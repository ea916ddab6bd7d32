"""CPU pins for the oracle: each check ties an oracle function to something other than
itself -- a closed form, a brute-force sum, a library routine computing the same thing by a
different algorithm, an invariant, or a number the paper prints."""
import math
import os

import numpy as np
import pytest

from oracle import monarch_oracle as O

rng = np.random.default_rng(20231012)

RECT = [(2, 2), (2, 3), (3, 2), (4, 4), (8, 8), (32, 16), (16, 32), (3, 5)]


# ---- permutations (App. D notation; Sec. 3.1 "reshape to 2D, transpose, flatten") --------

@pytest.mark.parametrize("N1,N2", RECT)
def test_stride_perm_is_reshape_transpose(N1, N2):
    N = N1 * N2
    x = rng.standard_normal(N)
    # P_(N1,N) x == view x as N1 x N2 row-major, transpose, flatten
    assert np.array_equal(O.apply_perm(N1, N, x), x.reshape(N1, N2).T.reshape(-1))
    # einops "(m n) -> (n m)" with n = N2 is the same thing
    from einops import rearrange
    assert np.array_equal(O.apply_perm(N1, N, x), rearrange(x, "(m n) -> (n m)", n=N2))


@pytest.mark.parametrize("N1,N2", RECT)
def test_perm_inverse_and_transpose(N1, N2):
    N = N1 * N2
    P = O.perm_matrix(N1, N)
    Q = O.perm_matrix(N2, N)
    assert np.array_equal(P.T, Q)                       # P_(b,N)^T = P_(N/b,N)
    assert np.array_equal(P @ Q, np.eye(N))
    assert sorted(O.stride_perm(N1, N).tolist()) == list(range(N))
    if N1 == N2:
        assert np.array_equal(P @ P, np.eye(N))         # square case: an involution
    # composing the index maps gives the identity
    s1, s2 = O.stride_perm(N1, N), O.stride_perm(N2, N)
    assert np.array_equal(s1[s2], np.arange(N))


def test_stride_perm_small_literal():
    # N = 6, b = 2: i = i1*2 + i0 -> i0*3 + i1
    assert O.stride_perm(2, 6).tolist() == [0, 3, 1, 4, 2, 5]
    assert O.stride_perm(3, 6).tolist() == [0, 2, 4, 1, 3, 5]


# ---- block-diagonal multiply and dense Monarch ---------------------------------------------

def test_blockdiag_apply_matches_dense_and_loops():
    W = rng.standard_normal((3, 4, 5))
    x = rng.standard_normal((2, 15))
    D = O.blockdiag_dense(W)
    assert D.shape == (12, 15)
    ref = np.zeros((2, 12))
    for r in range(2):
        for b in range(3):
            for o in range(4):
                for i in range(5):
                    ref[r, b * 4 + o] += W[b, o, i] * x[r, b * 5 + i]
    np.testing.assert_allclose(O.blockdiag_apply(W, x), ref, rtol=0, atol=1e-13)
    np.testing.assert_allclose(x @ D.T, ref, rtol=0, atol=1e-13)


@pytest.mark.parametrize("N1,N2", [(2, 2), (2, 3), (3, 2), (3, 4), (4, 4), (8, 8)])
def test_factored_apply_equals_dense_product(N1, N2):
    N = N1 * N2
    L = rng.standard_normal((N1, N2, N2))
    R = rng.standard_normal((N2, N1, N1))
    x = rng.standard_normal((3, N))
    M = O.monarch_dense(L, R)
    y = O.monarch_apply(L, R, x)
    np.testing.assert_allclose(y, x @ M.T, rtol=0, atol=1e-12)
    # tensor form: y[k2*N1+k1] = sum_{n2} L[k1][k2,n2] sum_{n1} R[n2][k1,n1] x[n1*N2+n2]
    ref = np.zeros((3, N))
    for k1 in range(N1):
        for k2 in range(N2):
            for n2 in range(N2):
                for n1 in range(N1):
                    ref[:, k2 * N1 + k1] += L[k1, k2, n2] * R[n2, k1, n1] * x[:, n1 * N2 + n2]
    np.testing.assert_allclose(y, ref, rtol=0, atol=1e-12)
    # order-p routine, p = 2, is the same map
    y2 = O.monarch_apply_order_p([R, L], (N1, N2), x)
    np.testing.assert_allclose(y2, y, rtol=0, atol=1e-12)


def test_identity_blocks_give_the_permutation():
    N1, N2 = 4, 3
    N = N1 * N2
    L = np.broadcast_to(np.eye(N2), (N1, N2, N2)).copy()
    R = np.broadcast_to(np.eye(N1), (N2, N1, N1)).copy()
    x = rng.standard_normal(N)
    np.testing.assert_array_equal(O.monarch_apply(L, R, x), O.apply_perm(N1, N, x))   # P P^T P = P


def test_listing_semantics_square():
    """The MonarchMatrix listing (App. A) applies its first parameter right after the
    first rearrange; in M = P L P R P that slot is R.  Re-enact the listing with plain
    reshapes and compare with the dense product."""
    s = 4
    N = s * s
    first = rng.standard_normal((s, s, s))
    second = rng.standard_normal((s, s, s))
    x = rng.standard_normal((2, N))

    def rearr(v):
        return v.reshape(-1, s, s).transpose(0, 2, 1).reshape(-1, N)

    def bd(v, w):
        return np.einsum("bnm,rbm->rbn", w, v.reshape(-1, s, s)).reshape(-1, N)

    out = rearr(bd(rearr(bd(rearr(x), first)), second))
    M = O.monarch_dense(second, first)
    np.testing.assert_allclose(out, x @ M.T, rtol=0, atol=1e-12)


def test_inverse_factors_roundtrip():
    N1, N2 = 4, 6
    L = rng.standard_normal((N1, N2, N2)) + np.eye(N2)
    R = rng.standard_normal((N2, N1, N1)) + np.eye(N1)
    x = rng.standard_normal((2, N1 * N2))
    Li, Ri = O.monarch_inverse_factors(L, R)
    np.testing.assert_allclose(O.monarch_inverse_apply(Li, Ri, O.monarch_apply(L, R, x)), x, atol=1e-9)


# ---- the DFT as a Monarch matrix (Corollary "DFT is M") -----------------------------------

def test_dft_matrix_convention():
    F = O.dft_matrix(8, +1)
    w = np.exp(2j * np.pi / 8)
    assert abs(F[1, 1] - w) < 1e-15 and abs(F[3, 5] - w ** 15) < 1e-14
    x = rng.standard_normal(8)
    # sign=+1 is the conjugate of numpy's forward transform, i.e. N * ifft
    np.testing.assert_allclose(F @ x, 8 * np.fft.ifft(x), atol=1e-13)
    np.testing.assert_allclose(O.dft_matrix(8, -1) @ x, np.fft.fft(x), atol=1e-13)
    np.testing.assert_allclose(F @ np.conj(F) / 8, np.eye(8), atol=1e-13)


@pytest.mark.parametrize("N1,N2", RECT)
@pytest.mark.parametrize("sign", [+1, -1])
def test_monarch_dft_is_the_dft_matrix(N1, N2, sign):
    L, R = O.monarch_dft_factors(N1, N2, sign)
    M = O.monarch_dense(L, R)
    np.testing.assert_allclose(M, O.dft_matrix(N1 * N2, sign), rtol=0, atol=2e-12)


def test_twiddle_free_factors_are_not_the_dft_but_the_2d_transform():
    """L = R = I (x) F_sqrtN (Sec. 3.1) without twiddles is the 2-D DFT of the sqrtN x sqrtN
    reshape; its Monarch convolution is the 2-D circular convolution (Thm 2), not the 1-D one."""
    s = 4
    N = s * s
    F = O.dft_matrix(s)
    L = np.broadcast_to(F, (s, s, s)).copy()
    M = O.monarch_dense(L, L)
    assert np.abs(M - O.dft_matrix(N)).max() > 0.5
    x = rng.standard_normal(N)
    k = rng.standard_normal(N)
    Minv = np.linalg.inv(M)
    y = np.real(Minv @ ((M @ k) * (M @ x)))
    X2, K2 = x.reshape(s, s), k.reshape(s, s)
    ref = np.zeros((s, s))
    for a in range(s):
        for b in range(s):
            for c in range(s):
                for d in range(s):
                    ref[a, b] += K2[c, d] * X2[(a - c) % s, (b - d) % s]
    np.testing.assert_allclose(y, ref.reshape(-1), atol=1e-11)
    assert np.abs(y - O.direct_circular_conv(k, x)).max() > 1e-3


@pytest.mark.parametrize("dims", [(2, 3, 4), (4, 4, 4), (8, 4, 2), (3, 3, 3), (2, 2, 2, 2), (32, 16), (16, 32)])
def test_order_p_monarch_dft_full(dims):
    N = int(np.prod(dims))
    X = np.eye(N)
    Y = O.monarch_dft(X, dims, +1)              # rows = F_N e_j = column j of F_N
    np.testing.assert_allclose(Y.T, O.dft_matrix(N, +1), rtol=0, atol=5e-12)


def test_order3_monarch_dft_32768_against_library_fft():
    dims = (32, 32, 32)
    N = 32768
    x = rng.standard_normal((2, N))
    y = O.monarch_dft(x, dims, +1)
    ref = N * np.fft.ifft(x, axis=-1)           # omega = e^{+2 pi i / N}
    assert np.linalg.norm(y - ref) / np.linalg.norm(ref) < 1e-12
    # Parseval: ||F x||^2 = N ||x||^2
    np.testing.assert_allclose(np.sum(np.abs(y) ** 2, -1), N * np.sum(x ** 2, -1), rtol=1e-12)
    # sampled columns of the matrix itself
    for j in (0, 1, 31, 32, 1023, 1024, 16385, 32767):
        e = np.zeros(N)
        e[j] = 1.0
        col = O.monarch_dft(e, dims, +1)
        kk = np.arange(N)
        np.testing.assert_allclose(col, np.exp(2j * np.pi * ((kk * j) % N) / N), atol=1e-11)


def test_plan_order_is_digit_reversal():
    dims = (2, 3, 4)
    pos = O.plan_order_index(dims)
    assert sorted(pos.tolist()) == list(range(24))
    for k1 in range(2):
        for k2 in range(3):
            for k3 in range(4):
                assert pos[(k1 * 3 + k2) * 4 + k3] == k1 + 2 * k2 + 6 * k3
    x = rng.standard_normal(24)
    nat = O.monarch_dft(x, dims)
    np.testing.assert_array_equal(O.monarch_dft(x, dims, plan_order=True), nat[pos])


# ---- convolution ---------------------------------------------------------------------------

def test_direct_convs_against_loops_and_library():
    n = 13
    k = rng.standard_normal(n)
    x = rng.standard_normal(n)
    cau = np.zeros(n)
    cir = np.zeros(n)
    for t in range(n):
        for u in range(n):
            if u <= t:
                cau[t] += k[u] * x[t - u]
            cir[t] += k[u] * x[(t - u) % n]
    np.testing.assert_allclose(O.direct_causal_conv(k, x), cau, atol=1e-13)
    np.testing.assert_allclose(O.direct_circular_conv(k, x), cir, atol=1e-13)
    np.testing.assert_allclose(O.direct_causal_conv(k, x), np.convolve(k, x)[:n], atol=1e-13)
    full = np.convolve(k, x)
    wrap = full[:n].copy()
    wrap[:n - 1] += full[n:]
    np.testing.assert_allclose(O.direct_circular_conv(k, x), wrap, atol=1e-12)


@pytest.mark.parametrize("dims", [(2, 2), (2, 3), (4, 4), (32, 16), (16, 32), (4, 4, 4), (2, 3, 4)])
def test_monarch_conv_equals_direct_circular(dims):
    N = int(np.prod(dims))
    k = rng.standard_normal((3, N))
    x = rng.standard_normal((2, 3, N))
    y = O.monarch_conv(k[None], x, dims, causal=False)
    ref = O.direct_circular_conv(k[None], x)
    assert np.linalg.norm(y - ref) / np.linalg.norm(ref) < 1e-12


@pytest.mark.parametrize("dims,n", [((2, 2), 2), ((4, 4), 8), ((4, 4), 5), ((32, 16), 256), ((4, 4, 4), 32), ((8, 8, 8), 256)])
def test_monarch_conv_equals_direct_causal(dims, n):
    k = rng.standard_normal((3, n))
    x = rng.standard_normal((2, 3, n))
    y = O.monarch_conv(k[None], x, dims, causal=True)
    ref = O.direct_causal_conv(k[None], x)
    assert y.shape == ref.shape
    assert np.linalg.norm(y - ref) / np.linalg.norm(ref) < 1e-12


def test_monarch_conv_sign_independent_and_stages():
    dims = (4, 8)
    k = rng.standard_normal(32)
    x = rng.standard_normal(32)
    st = {}
    yp = O.monarch_conv(k, x, dims, causal=False, sign=+1, stages=st)
    ym = O.monarch_conv(k, x, dims, causal=False, sign=-1)
    np.testing.assert_allclose(yp, ym, atol=1e-12)
    np.testing.assert_allclose(st["u_f"], O.dft_matrix(32) @ x, atol=1e-11)
    assert np.abs(np.imag(st["f"])).max() < 1e-12


def test_monarch_conv_special_kernels_and_invariants():
    dims = (32, 16)
    N = 512
    x = rng.standard_normal((2, N))
    delta = np.zeros(N)
    delta[0] = 1.0
    np.testing.assert_allclose(O.monarch_conv(delta, x, dims, causal=False), x, atol=1e-12)
    d1 = np.zeros(N)
    d1[1] = 1.0
    np.testing.assert_allclose(O.monarch_conv(d1, x, dims, causal=False), np.roll(x, 1, -1), atol=1e-12)
    k = rng.standard_normal(N)
    # shift equivariance (circular) and linearity
    y = O.monarch_conv(k, x, dims, causal=False)
    np.testing.assert_allclose(O.monarch_conv(k, np.roll(x, 7, -1), dims, causal=False), np.roll(y, 7, -1), atol=1e-11)
    x2 = rng.standard_normal((2, N))
    np.testing.assert_allclose(O.monarch_conv(k, 2 * x - 3 * x2, dims, causal=False),
                               2 * y - 3 * O.monarch_conv(k, x2, dims, causal=False), atol=1e-11)
    # causality: changing x[t0:] leaves y[:t0] unchanged
    n = 256
    kc = rng.standard_normal(n)
    xa = rng.standard_normal(n)
    xb = xa.copy()
    xb[100:] += rng.standard_normal(n - 100)
    ya = O.monarch_conv(kc, xa, dims, causal=True)
    yb = O.monarch_conv(kc, xb, dims, causal=True)
    np.testing.assert_allclose(ya[:100], yb[:100], atol=1e-12)
    assert np.abs(ya[100:] - yb[100:]).max() > 1e-3
    # causal delta_1 is a shift with zero fill
    d1c = np.zeros(n)
    d1c[1] = 1.0
    ys = O.monarch_conv(d1c, xa, dims, causal=True)
    np.testing.assert_allclose(ys[1:], xa[:-1], atol=1e-12)
    assert abs(ys[0]) < 1e-12


def test_order3_causal_conv_full_size_sampled():
    """Thm (arbitrary basis, any matrix equal to F_N) => zero padding to N = 2n suffices for
    order 3 as well: check a full-length row against the direct sum at sampled outputs."""
    from paper_2310_12109_b200 import synth
    n = 16384
    x = rng.standard_normal(n)
    k = synth.decay_kernel(4, 1, n, 0.0005, 128.0)[0].astype(np.float64)
    y = O.monarch_conv(k, x, (32, 32, 32), causal=True)
    for t in (0, 1, 2, 31, 32, 1023, 1024, 5000, 16383):
        ref = float(np.dot(k[:t + 1], x[t::-1]))
        assert abs(y[t] - ref) < 1e-10 * max(1.0, abs(ref))


# ---- M2 block pieces ---------------------------------------------------------------------

def test_conv_adjoints_are_transposes_and_match_the_conjugated_spectrum():
    """The adjoint oracles: (i) equal the transposed dense circulant / Toeplitz matrix applied to g, (ii) satisfy
    <conv(k, x), g> = <x, adjoint(k, g)>, (iii) the factored version (conjugated kernel spectrum) equals the direct one."""
    n = 12
    k, x, g = rng.standard_normal(n), rng.standard_normal((3, n)), rng.standard_normal((3, n))
    Cm = np.array([[k[(t - u) % n] for u in range(n)] for t in range(n)])          # y = Cm x (circular)
    Tm = np.array([[k[t - u] if t >= u else 0.0 for u in range(n)] for t in range(n)])  # y = Tm x (causal)
    assert np.allclose(O.direct_circular_conv(k, x), x @ Cm.T)
    assert np.allclose(O.direct_circular_conv_adjoint(k, g), g @ Cm)
    assert np.allclose(O.direct_causal_conv(k, x), x @ Tm.T)
    assert np.allclose(O.direct_causal_conv_adjoint(k, g), g @ Tm)
    assert np.isclose(np.sum(O.direct_causal_conv(k, x) * g), np.sum(x * O.direct_causal_conv_adjoint(k, g)))
    for dims, nn, causal in [((4, 3), 12, False), ((4, 3, 2), 12, True), ((32, 16), 256, True), ((8, 8), 64, False)]:
        kk, gg, xx = rng.standard_normal((2, nn)), rng.standard_normal((3, 2, nn)), rng.standard_normal((3, 2, nn))
        direct = O.direct_causal_conv_adjoint(kk, gg) if causal else O.direct_circular_conv_adjoint(kk, gg)
        assert np.allclose(O.monarch_conv_adjoint(kk, gg, dims, causal), direct, atol=1e-10)
        assert np.allclose(O.monarch_conv_adjoint(kk, gg, dims, causal, sign=-1), direct, atol=1e-10)
        lhs = np.sum(O.monarch_conv(kk, xx, dims, causal) * gg)
        assert np.isclose(lhs, np.sum(xx * O.monarch_conv_adjoint(kk, gg, dims, causal)), rtol=1e-10)


@pytest.mark.parametrize("N1,N2", [(4, 4), (3, 5), (8, 2), (16, 16)])
def test_monarch_transpose_apply(N1, N2):
    """M^T g: against the dense matrix, by <M x, g> = <x, M^T g>, and as the forward apply with the block-wise
    transposed factors in swapped roles (the identity the library's backward-input call rests on)."""
    L, R = rng.standard_normal((N1, N2, N2)), rng.standard_normal((N2, N1, N1))
    Md = O.monarch_dense(L, R)
    x, g = rng.standard_normal((3, N1 * N2)), rng.standard_normal((3, N1 * N2))
    assert np.allclose(O.monarch_apply_transpose(L, R, g), g @ Md)
    assert np.isclose(np.sum(O.monarch_apply(L, R, x) * g), np.sum(x * O.monarch_apply_transpose(L, R, g)))
    Lt, Rt = np.swapaxes(R, 1, 2).copy(), np.swapaxes(L, 1, 2).copy()
    assert np.allclose(O.monarch_apply(Lt, Rt, g), g @ Md)


def test_monarch_mix_operator():
    """M_b sigma(K (.) M_a x): against dense matrices; with identity blocks M = P, so the operator is the closed-form
    permutation y = P (K (.) P x); with M_a = F, M_b = F^-1 (complex factors) it is the circular convolution."""
    N1, N2, T, Hk = 3, 4, 6, 2
    N = N1 * N2
    La, Lb = rng.standard_normal((2, N1, N2, N2))
    Ra, Rb = rng.standard_normal((2, N2, N1, N1))
    K, x = rng.standard_normal((Hk, N)), rng.standard_normal((T, N))
    Ma, Mb = O.monarch_dense(La, Ra), O.monarch_dense(Lb, Rb)
    for act in ("none", "relu"):
        mid = np.tile(K, (T // Hk, 1)) * (x @ Ma.T)
        if act == "relu":
            mid = np.where(mid > 0, mid, 0.0)
        assert np.allclose(O.monarch_mix(La, Ra, Lb, Rb, K, x, act), mid @ Mb.T)
    # identity blocks: M = P with (P v)[n2 N1 + n1] = v[n1 N2 + n2]
    I_L, I_R = np.broadcast_to(np.eye(N2), (N1, N2, N2)), np.broadcast_to(np.eye(N1), (N2, N1, N1))
    y = O.monarch_mix(I_L, I_R, I_L, I_R, K[:1], x)
    Px = x.reshape(T, N1, N2).swapaxes(1, 2).reshape(T, N)
    want = (K[0] * Px).reshape(T, N1, N2).swapaxes(1, 2).reshape(T, N)
    assert np.array_equal(y, want)
    # DFT factors: the operator is the circular convolution with the kernel whose spectrum is K (Eq. 2)
    Lf, Rf = O.monarch_dft_factors(N1, N2)
    k = rng.standard_normal((Hk, N))
    kf = k @ O.dft_matrix(N).T
    y = O.monarch_mix(Lf, Rf, np.conj(Lf), np.conj(Rf) / N, kf, x.astype(complex))
    assert np.allclose(y.imag, 0) and np.allclose(y.real, np.stack([O.direct_circular_conv(k[t % Hk], x[t]) for t in range(T)]))


def test_monarch_cols_oracle():
    """Columns as vectors: the dense matrix times X, and the factor / ReLU applied afterwards."""
    N1, N2, d = 3, 4, 5
    L, R = rng.standard_normal((N1, N2, N2)), rng.standard_normal((N2, N1, N1))
    X, K = rng.standard_normal((2, N1 * N2, d)), rng.standard_normal((N1 * N2, d))
    Md = O.monarch_dense(L, R)
    assert np.allclose(O.monarch_cols(L, R, X), Md @ X)
    assert np.allclose(O.monarch_cols(L, R, X, K, "relu"), np.where(K * (Md @ X) > 0, K * (Md @ X), 0.0))
    assert np.allclose(O.monarch_cols(L, R, X, K), K * (Md @ X))


def test_m2_bert_mixer_oracle():
    """The gated mixer against explicit per-channel loops with the direct O(n^2) circular convolution; with identity
    projections and the pass-through short filter (0, 1, 0) it is x (.) conv(k, x (.) x) + conv(k_res, x); circular-shift
    equivariance along the sequence does not hold with zero-padded short filters unless they are pass-through, where it does."""
    B, dims, d = 2, (4, 4), 5
    n = 16
    p = {k: rng.standard_normal((d, d)) for k in ("W_q", "W_k", "W_v", "W_o")}
    for k in ("w_q", "w_k", "w_v"):
        p[k] = rng.standard_normal((d, 3))
    p["k"], p["k_res"] = rng.standard_normal((d, n)), rng.standard_normal((d, n))
    x = rng.standard_normal((B, n, d))
    y = O.m2_bert_mixer(x, p, dims)
    want = np.zeros_like(y)
    for b in range(B):
        def dw(a, w):   # [n, d], zero padded, centred
            g = np.zeros_like(a)
            for t_ in range(n):
                for c in range(d):
                    g[t_, c] = w[c, 1] * a[t_, c] + (w[c, 0] * a[t_ - 1, c] if t_ > 0 else 0.0) + (w[c, 2] * a[t_ + 1, c] if t_ + 1 < n else 0.0)
            return g
        Q, K, V = dw(x[b] @ p["W_q"], p["w_q"]), dw(x[b] @ p["W_k"], p["w_k"]), dw(x[b] @ p["W_v"], p["w_v"])
        Z = np.zeros((n, d))
        for c in range(d):
            Z[:, c] = V[:, c] * O.direct_circular_conv(p["k"][c], Q[:, c] * K[:, c]) + O.direct_circular_conv(p["k_res"][c], x[b][:, c])
        want[b] = Z @ p["W_o"]
    assert np.allclose(y, want)
    eye = np.eye(d)
    thru = np.tile(np.array([0.0, 1.0, 0.0]), (d, 1))
    p2 = dict(p, W_q=eye, W_k=eye, W_v=eye, W_o=eye, w_q=thru, w_k=thru, w_v=thru)
    xc = np.swapaxes(x, 1, 2)
    want2 = xc * O.direct_circular_conv(p["k"][None], xc * xc) + O.direct_circular_conv(p["k_res"][None], xc)
    assert np.allclose(O.m2_bert_mixer(x, p2, dims), np.swapaxes(want2, 1, 2))
    assert np.allclose(O.m2_bert_mixer(np.roll(x, 3, axis=1), p2, dims), np.roll(O.m2_bert_mixer(x, p2, dims), 3, axis=1))


def test_m2_hyena_heads_oracle():
    """The layer against the same computation spelled out with explicit loops over heads and positions and the direct
    O(n^2) causal convolution; causality of the whole layer; head dimension 1 = a gated double convolution."""
    B, n, d, dh = 2, 8, 6, 2
    dims = (4, 4)
    p = {k: rng.standard_normal((d, d)) for k in ("W_x1", "W_x2", "W_v", "W_o")}
    for k in ("K1", "K2", "K3"):
        p[k] = rng.standard_normal((d, n))
    p["K_long"] = rng.standard_normal((d // dh, n))
    u = rng.standard_normal((B, n, d))
    y = O.m2_hyena_heads(u, p, dims, dh)
    conv = lambda k, x: O.direct_causal_conv(k, x)   # noqa: E731
    want = np.zeros((B, n, d))
    for b in range(B):
        X1, X2, V = u[b] @ p["W_x1"], u[b] @ p["W_x2"], u[b] @ p["W_v"]     # [n, d]
        X1c = np.stack([conv(p["K1"][c], X1[:, c]) for c in range(d)], 1)
        X2c = np.stack([conv(p["K2"][c], X2[:, c]) for c in range(d)], 1)
        Vc = np.stack([conv(p["K3"][c], V[:, c]) for c in range(d)], 1)
        Oc = np.zeros((n, d))
        for h in range(d // dh):
            sl = slice(h * dh, (h + 1) * dh)
            XV = np.einsum("ti,tj->tij", X2c[:, sl], Vc[:, sl])               # [n, dh, dh]
            XVc = np.zeros_like(XV)
            for i in range(dh):
                for j in range(dh):
                    XVc[:, i, j] = conv(p["K_long"][h], XV[:, i, j])
            for t_ in range(n):
                Oc[t_, sl] = X1c[t_, sl] @ XVc[t_]
        want[b] = Oc @ p["W_o"]
    assert np.allclose(y, want)
    u2 = u.copy()
    u2[:, 5:] += rng.standard_normal((B, 3, d))      # perturbing positions >= 5 leaves outputs < 5 unchanged
    assert np.allclose(O.m2_hyena_heads(u2, p, dims, dh)[:, :5], y[:, :5])
    p1 = dict(p, K_long=rng.standard_normal((d, n)))
    y1 = O.m2_hyena_heads(u, p1, dims, 1)           # d_h = 1: y = (X1~ (.) conv(K_long, X2~ (.) V~)) W_o
    st = {}
    O.m2_hyena_heads(u, p1, dims, 1, stages=st)
    inner = O.direct_causal_conv(p1["K_long"][None], st["X2c"] * st["Vc"])
    assert np.allclose(y1, np.swapaxes(st["X1c"] * inner, 1, 2) @ p["W_o"])


def test_m2_layer_oracle():
    """The layer against the same computation with dense matrices and einsum over the un-transposed [B, n, d] tensor;
    LayerNorm against torch's routine and its invariants (zero mean, unit variance, shift/scale invariance)."""
    import torch
    B, sn, sd = 2, 3, 2
    n, d = sn * sn, sd * sd
    p = {}
    for i in (1, 2):
        p[f"L{i}"], p[f"R{i}"] = rng.standard_normal((sn, sn, sn)), rng.standard_normal((sn, sn, sn))
    for i in (3, 4):
        p[f"L{i}"], p[f"R{i}"] = rng.standard_normal((sd, sd, sd)), rng.standard_normal((sd, sd, sd))
    p["n_kernel"], p["d_kernel"] = rng.standard_normal((d, n)), rng.standard_normal((1, d))
    p["gamma"], p["beta"] = rng.standard_normal(d), rng.standard_normal(d)
    x = rng.standard_normal((B, n, d))
    st = {}
    out = O.m2_layer(x, p, stages=st)
    D = {i: O.monarch_dense(p[f"L{i}"], p[f"R{i}"]) for i in (1, 2, 3, 4)}
    a = np.einsum("kn,bnc->bkc", D[1], x) * p["n_kernel"].T[None]                 # [B, n, d], kernel indexed [c, k]
    xt = np.einsum("kn,bnc->bkc", D[2], np.maximum(a, 0))
    y = np.maximum(p["d_kernel"][0] * (xt @ D[3].T), 0) @ D[4].T
    assert np.allclose(st["x_tilde"], xt) and np.allclose(st["y"], y)
    s = y + xt
    want = torch.nn.functional.layer_norm(torch.from_numpy(s), (d,), torch.from_numpy(p["gamma"]), torch.from_numpy(p["beta"]), 1e-5).numpy()
    assert np.allclose(out, want)
    v = rng.standard_normal((5, 64))
    ln = O.layer_norm(v, np.ones(64), np.zeros(64), 0.0)
    assert np.allclose(ln.mean(-1), 0) and np.allclose(ln.var(-1), 1)
    assert np.allclose(O.layer_norm(3.0 * v + 7.0, np.ones(64), np.zeros(64), 0.0), ln)


@pytest.mark.parametrize("N1,N2", [(2, 3), (4, 4), (5, 2)])
def test_monarch_weight_grads(N1, N2):
    """y is linear in L and in R, so perturbing one weight by 1 changes sum <y, g> by exactly that weight's
    gradient: brute force over every entry, with the dense matrix doing the forward."""
    L, R = rng.standard_normal((N1, N2, N2)), rng.standard_normal((N2, N1, N1))
    x, g = rng.standard_normal((5, N1 * N2)), rng.standard_normal((5, N1 * N2))
    dL, dR = O.monarch_weight_grads(L, R, x, g)
    base = np.sum((x @ O.monarch_dense(L, R).T) * g)
    for idx in np.ndindex(*L.shape):
        Lp = L.copy(); Lp[idx] += 1.0
        assert np.isclose(np.sum((x @ O.monarch_dense(Lp, R).T) * g) - base, dL[idx], atol=1e-9), ("dL", idx)
    for idx in np.ndindex(*R.shape):
        Rp = R.copy(); Rp[idx] += 1.0
        assert np.isclose(np.sum((x @ O.monarch_dense(L, Rp).T) * g) - base, dR[idx], atol=1e-9), ("dR", idx)


def test_kernel_gradient_oracles():
    """dk: (i) the convolution is linear in k, so <conv(k, x), g> summed over the batch equals <k, dk> for every k;
    (ii) the factored version equals the direct one; (iii) a brute-force triple loop on a tiny case."""
    B, H, n = 2, 3, 6
    x, g = rng.standard_normal((B, H, n)), rng.standard_normal((B, H, n))
    for causal in (True, False):
        dk = O.direct_conv_kernel_grad(x, g, causal)
        brute = np.zeros((H, n))
        for b in range(B):
            for h in range(H):
                for u in range(n):
                    for t in range(n):
                        if causal and t < u:
                            continue
                        brute[h, u] += g[b, h, t] * x[b, h, (t - u) % n]
        assert np.allclose(dk, brute)
    for dims, nn, causal in [((4, 3), 12, False), ((4, 3, 2), 12, True), ((32, 16), 256, True), ((8, 8), 64, False)]:
        xx, gg, kk = rng.standard_normal((3, 2, nn)), rng.standard_normal((3, 2, nn)), rng.standard_normal((2, nn))
        dk = O.direct_conv_kernel_grad(xx, gg, causal)
        assert np.allclose(O.monarch_conv_kernel_grad(xx, gg, dims, causal), dk, atol=1e-9)
        assert np.allclose(O.monarch_conv_kernel_grad(xx, gg, dims, causal, sign=-1), dk, atol=1e-9)
        assert np.isclose(np.sum(O.monarch_conv(kk, xx, dims, causal) * gg), np.sum(kk * dk), rtol=1e-10)


def test_gelu_values():
    v = np.array([0.0, 1.0, -1.0, 3.0])
    ref = np.array([0.0, 0.8413447460685429, -0.15865525393145707, 2.9959502191322303])
    np.testing.assert_allclose(O.gelu_erf(v), ref, atol=1e-14)
    from scipy.special import erf
    w = rng.standard_normal(100)
    np.testing.assert_allclose(O.gelu_erf(w), 0.5 * w * (1 + erf(w / math.sqrt(2))), atol=1e-15)


def test_depthwise_conv_against_library():
    x = rng.standard_normal((2, 9, 3))
    w = rng.standard_normal((3, 3))
    g = O.depthwise_conv3_same(x, w)
    for b in range(2):
        for c in range(3):
            # np.convolve flips its kernel: g[t] = sum_j w[j] x[t + j - 1]
            ref = np.convolve(x[b, :, c], w[c, ::-1], mode="same")
            np.testing.assert_allclose(g[b, :, c], ref, atol=1e-13)


def test_block_forward_composition_small():
    B, T, C = 2, 16, 8
    x = rng.standard_normal((B, T, C))
    k = rng.standard_normal((C, T))
    w = rng.standard_normal((C, 3))
    Wu = rng.standard_normal((4, 8, 2))
    Wd = rng.standard_normal((4, 2, 8))
    y, z = O.m2_block_forward(x, k, w, Wu, Wd, dims=(4, 4))
    # explicit per-element evaluation
    for b in range(B):
        for c in range(C):
            v = O.direct_circular_conv(k[c], x[b, :, c])
            g = np.convolve(x[b, :, c], w[c, ::-1], mode="same")
            np.testing.assert_allclose(z[b, :, c], g * v, atol=1e-11)
    h = O.gelu_erf(z @ O.blockdiag_dense(Wu).T)
    np.testing.assert_allclose(y, h @ O.blockdiag_dense(Wd).T, atol=1e-11)


# ---- the one set of numbers the paper prints for this path: Table 2 FLOP costs ---------------

def test_table2_flop_convention():
    path = os.path.join(os.path.dirname(__file__), "golden", "table2_flop_cost.txt")
    rows = [ln.split() for ln in open(path) if ln.strip() and not ln.startswith("#")]
    for N, dense, m2 in rows:
        N = int(N)
        dense_model = 2.0 * N * N * 768 / 1e12
        m2_model = 8.0 * N ** 1.5 * 768 / 1e12
        # printed with 3 significant digits (two entries differ in the last printed digit)
        assert abs(dense_model - float(dense)) <= 0.012 * float(dense) + 6e-4
        assert abs(m2_model - float(m2)) <= 0.012 * float(m2) + 6e-4


# ---- learnable / causal Monarch from polynomial coefficients (App. D.5) -----------------------------------

def _basis_coefficients(Lt, Rt):
    """Coefficient vectors (length N, ascending powers) of the basis polynomials b_j(Z) = l_{j0}(Z) r~_{j0,j1}(Z^b) mod (Z^N - 1),
    j = j1 b + j0, by explicit polynomial products -- no DFT, no Monarch factor anywhere."""
    N, b = Lt.shape
    Bc = np.zeros((N, N))
    for j1 in range(b):
        for j0 in range(b):
            l = Lt[:, j0]
            r = np.zeros(b * (b - 1) + 1)
            r[::b] = Rt[j0 * b:(j0 + 1) * b, j1]          # r~(Z^b): coefficient a sits at power a b
            prod = np.convolve(l, r)
            col = np.zeros(N)
            for d, c in enumerate(prod):
                col[d % N] += c                            # reduction mod Z^N - 1
            Bc[:, j1 * b + j0] = col
    return Bc


@pytest.mark.parametrize("b", [2, 3, 4, 6])
def test_blocky_monarch_columns_are_the_basis_polynomials_on_the_roots_of_unity(b):
    """Theorem on BlockyMonarch's return value: M[i, j1 b + j0] = l_{j0}(w_N^i) r~_{j0,j1}(w_N^{i b}), evaluated here by
    Horner's rule on the raw coefficients."""
    N = b * b
    rng = np.random.default_rng(100 + b)
    Lt, Rt = rng.standard_normal((N, b)), rng.standard_normal((N, b))
    for sign in (+1, -1):
        L, R = O.blocky_monarch(Lt, Rt, sign)
        Md = O.monarch_dense(L, R)
        w = np.exp(sign * 2j * np.pi / N)
        for i in range(N):
            z = w ** i
            for j1 in range(b):
                for j0 in range(b):
                    want = np.polyval(Lt[::-1, j0], z) * np.polyval(Rt[j0 * b:(j0 + 1) * b, j1][::-1], z ** b)
                    assert abs(Md[i, j1 * b + j0] - want) < 1e-9 * max(1.0, abs(want))
        # the same statement through the coefficient matrix of the basis: M = F_N B
        assert np.allclose(Md, O.dft_matrix(N, sign) @ _basis_coefficients(Lt, Rt), atol=1e-9)


@pytest.mark.parametrize("b", [2, 4, 8, 16])
def test_blocky_monarch_with_identity_coefficients_is_the_dft(b):
    """Corollary "DFT is M": identity blocks in Rt, identity top block in Lt -> the factors of monarch_dft_factors."""
    N = b * b
    Lt = np.zeros((N, b))
    Lt[:b] = np.eye(b)
    Rt = np.tile(np.eye(b), (b, 1))
    for sign in (+1, -1):
        L, R = O.blocky_monarch(Lt, Rt, sign)
        FL, FR = O.monarch_dft_factors(b, b, sign)
        assert np.allclose(L, FL, atol=1e-12) and np.allclose(R, FR, atol=1e-12)
        assert np.allclose(O.monarch_dense(L, R), O.dft_matrix(N, sign), atol=1e-10)


def test_causal_masks_literal_b4():
    mL, mR = O.causal_coefficient_masks(4)
    assert mL.shape == (16, 4) and mR.shape == (16, 4)
    assert (mL[:4] == np.array([[1, 0, 0, 0], [1, 1, 0, 0], [1, 1, 1, 0], [1, 1, 1, 1]])).all() and (mL[4:] == 0).all()
    blk = np.array([[1, 0, 0, 0], [1, 1, 0, 0], [0, 0, 1, 0], [0, 0, 1, 1]])   # rows >= 2 of columns < 2 are cut (degree < 2)
    for c in range(4):
        assert (mR[4 * c:4 * c + 4] == blk).all()


@pytest.mark.parametrize("b", [4, 5, 6])
def test_masked_basis_has_the_degrees_the_lemma_states(b):
    """Lemma on masking: basis polynomial j = j1 b + j0 of M has minimum degree j; for j < b floor(b/2) its degree is < N/2."""
    N = b * b
    rng = np.random.default_rng(7 + b)
    mL, mR = O.causal_coefficient_masks(b)
    Lt = (np.eye(N, b) + rng.standard_normal((N, b))) * mL
    Rt = (np.tile(np.eye(b), (b, 1)) + rng.standard_normal((N, b))) * mR
    Bc = _basis_coefficients(Lt, Rt)
    for j in range(N):
        nz = np.nonzero(np.abs(Bc[:, j]) > 1e-12)[0]
        assert nz.min() == j
        if j < b * (b // 2):
            assert nz.max() <= N // 2 - 1


@pytest.mark.parametrize("b,n", [(4, 8), (4, 5), (6, 18), (5, 12), (8, 32)])
def test_blocky_monarch_conv_is_the_polynomial_product_in_the_basis(b, n):
    """Alg. BlockMonarchConv against its plain definition (the theorem on the univariate convolution): with k(Z) = sum k_j b_j,
    u(Z) = sum u_j b_j, f holds the coefficients of k(Z) u(Z) mod (Z^N - 1) in the basis (b_i) -- computed here with explicit
    polynomial products and one dense solve."""
    N = b * b
    rng = np.random.default_rng(50 + b + n)
    mL, mR = O.causal_coefficient_masks(b)
    Lt = (np.eye(N, b) + 0.4 * rng.standard_normal((N, b))) * mL
    Rt = (np.tile(np.eye(b), (b, 1)) + 0.4 * rng.standard_normal((N, b))) * mR
    k, u = rng.standard_normal((3, n)), rng.standard_normal((2, 3, n))
    f = O.blocky_monarch_conv(Lt, Rt, k, u)
    assert np.abs(f.imag).max() < 1e-9
    Bc = _basis_coefficients(Lt, Rt)
    for bi in range(2):
        for h in range(3):
            kz, uz = Bc[:, :n] @ k[h], Bc[:, :n] @ u[bi, h]
            prod = np.zeros(N)
            for d, c in enumerate(np.convolve(kz, uz)):
                prod[d % N] += c
            want = np.linalg.solve(Bc, prod)[:n]
            assert np.allclose(f[bi, h].real, want, atol=1e-8 * max(1.0, np.abs(want).max()))


@pytest.mark.parametrize("b", [4, 6, 8])
def test_masked_blocky_monarch_conv_is_causal_and_unmasked_is_not(b):
    """Theorem on causal block Monarch convolution: with the masked coefficients, f[:t0] does not change when u[t0:] does."""
    N = b * b
    n = N // 2
    rng = np.random.default_rng(9 + b)
    mL, mR = O.causal_coefficient_masks(b)
    Lt0, Rt0 = np.eye(N, b) + 0.3 * rng.standard_normal((N, b)), np.tile(np.eye(b), (b, 1)) + 0.3 * rng.standard_normal((N, b))
    k, u = rng.standard_normal(n), rng.standard_normal(n)
    f = O.blocky_monarch_conv(Lt0 * mL, Rt0 * mR, k, u)
    for t0 in (1, 2, n // 2, n - 1):
        u2 = u.copy()
        u2[t0:] += rng.standard_normal(n - t0)
        f2 = O.blocky_monarch_conv(Lt0 * mL, Rt0 * mR, k, u2)
        assert np.abs(f2[:t0] - f[:t0]).max() < 1e-9 * max(1.0, np.abs(f).max())
        assert np.abs(f2[t0:] - f[t0:]).max() > 1e-6
    g = O.blocky_monarch_conv(Lt0, Rt0, k, u)
    u2 = u.copy()
    u2[-1] += 1.0
    assert abs(O.blocky_monarch_conv(Lt0, Rt0, k, u2)[0] - g[0]) > 1e-6     # without the masks the future leaks


def test_blocky_monarch_conv_with_dft_coefficients_is_the_causal_convolution():
    b, n = 8, 32
    N = b * b
    Lt = np.zeros((N, b))
    Lt[:b] = np.eye(b)
    Rt = np.tile(np.eye(b), (b, 1))
    rng = np.random.default_rng(3)
    k, u = rng.standard_normal((2, n)), rng.standard_normal((3, 2, n))
    f = O.blocky_monarch_conv(Lt, Rt, k, u)
    assert np.allclose(f.real, O.direct_causal_conv(k[None], u), atol=1e-10) and np.abs(f.imag).max() < 1e-10
