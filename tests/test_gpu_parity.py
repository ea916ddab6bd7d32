"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded
inputs.  Tolerances (relative L2 over the whole tensor; worst single row at twice that):
fp32 path 1e-5, bf16-in / fp32-accumulate / bf16-out path 2e-2.  Integer tables are bit-exact
(tests/test_abi_host.py)."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import monarch_oracle as O
from paper_2310_12109_b200 import binding as M
from paper_2310_12109_b200 import synth

pytestmark = pytest.mark.gpu

TOL_FP32 = 1e-5
TOL_BF16 = 2e-2


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    return t.to(dtype) if dtype is not None else t


def host(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def check(got, ref, tol, what=""):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, (got.shape, ref.shape)
    assert np.isfinite(got).all(), what + ": non-finite output"
    g = np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-300)
    rows_g = got.reshape(-1, got.shape[-1])
    rows_r = ref.reshape(-1, ref.shape[-1])
    per = np.linalg.norm(rows_g - rows_r, axis=1) / np.maximum(np.linalg.norm(rows_r, axis=1), 1e-300)
    assert g <= tol, f"{what}: global rel-L2 {g:.3e} > {tol}"
    assert per.max() <= 2 * tol, f"{what}: worst row rel-L2 {per.max():.3e} (row {per.argmax()}) > {2 * tol}"
    return g


def run_conv(dims, x_np, k_np, causal, dtype, sign=+1):
    plan = M.Plan(dims, dtype=dtype, sign=sign, device=0)
    tdt = torch.bfloat16 if dtype == M.M2_BF16 else torch.float32
    x = dev(x_np.astype(np.float32), tdt)
    k = dev(k_np.astype(np.float32))
    kf = M.m2_kernel_spectrum(plan, k)
    y = M.m2_monarch_conv_fwd(plan, x, kf, M.M2_CAUSAL if causal else M.M2_CIRCULAR)
    torch.cuda.synchronize()
    assert plan.device_status() == 0
    name = plan.last_kernel()
    plan.close()
    return host(y), name


# ---- config 1: fp32, order 2, causal, checked against the direct sum --------------------------

def test_config1_fp32_causal_vs_direct():
    c = synth.config1()
    y, name = run_conv(c["dims"], c["x"], c["k"], True, M.M2_FP32)
    ref = O.direct_causal_conv(c["k"].astype(np.float64)[None], c["x"].astype(np.float64))
    check(y, ref, TOL_FP32, "config1 " + name)
    ref2 = O.monarch_conv(c["k"].astype(np.float64)[None], c["x"].astype(np.float64), c["dims"], causal=True)
    check(y, ref2, TOL_FP32, "config1 vs factored oracle")


@pytest.mark.parametrize("dims", [(32, 16), (2, 3), (4, 4, 4), (32, 32, 32)])
@pytest.mark.parametrize("sign", [+1, -1])
def test_kernel_spectrum_is_the_dft(dims, sign):
    N = int(np.prod(dims))
    H, n = 3, N // 2
    k = synth.normal(900 + N, (H, n)).astype(np.float32)
    plan = M.Plan(dims, dtype=M.M2_FP32, sign=sign, device=0)
    kf = M.m2_kernel_spectrum(plan, dev(k))
    nat = host(M.m2_spectrum_to_natural(plan, kf, H))
    got = nat[..., 0] + 1j * nat[..., 1]
    kp = np.concatenate([k.astype(np.float64), np.zeros((H, N - n))], -1)
    ref = O.monarch_dft(kp, dims, sign)
    err = np.linalg.norm(got - ref) / np.linalg.norm(ref)
    assert err < TOL_FP32, err
    plan.close()


@pytest.mark.parametrize("dims,n,causal", [
    ((32, 16), 256, True), ((32, 16), 200, True), ((32, 16), 1, True), ((32, 16), 512, False),
    ((16, 32), 512, False), ((2, 3), 6, False), ((3, 5), 7, True), ((4, 4, 4), 32, True),
    ((8, 4, 2), 64, False), ((16, 16, 16), 2048, True), ((64, 64), 4096, False), ((32, 32, 8), 4096, True),
])
def test_fp32_conv_shapes(dims, n, causal):
    B, H = 2, 3
    x = synth.normal(700 + n, (B, H, n)).astype(np.float32)
    k = (synth.normal(701 + n, (H, n)) / np.sqrt(n)).astype(np.float32)
    y, name = run_conv(dims, x, k, causal, M.M2_FP32)
    x64, k64 = x.astype(np.float64), k.astype(np.float64)
    ref = O.direct_causal_conv(k64[None], x64) if causal else O.direct_circular_conv(k64[None], x64)
    check(y, ref, TOL_FP32, f"{dims} n={n} {name}")


def test_fp32_conv_sign_minus_matches():
    c = synth.config1()
    y, _ = run_conv(c["dims"], c["x"], c["k"], True, M.M2_FP32, sign=-1)
    ref = O.direct_causal_conv(c["k"].astype(np.float64)[None], c["x"].astype(np.float64))
    check(y, ref, TOL_FP32, "sign=-1")


# ---- config 2: bf16 circular, N = 512 = 32 x 16 ----------------------------------------------

@pytest.mark.parametrize("B,H", [(4, 24), (3, 5), (1, 1), (32, 9), (9, 5), (16, 3), (19, 6), (40, 150)])
def test_config2_small_full_compare(B, H):   # more than 8 batch rows: the kernel that packs row pairs as complex rows
    c = synth.config2(B=B, H=H)
    y, name = run_conv(c["dims"], c["x"], c["k"], False, M.M2_BF16)
    ref = O.monarch_conv(c["k"].astype(np.float64)[None], c["x"].astype(np.float64), c["dims"], causal=False)
    check(y, ref, TOL_BF16, f"config2 B={B} H={H} {name}")
    # up to 8 batch rows: one row per lane; more: two batch rows packed as one complex row
    assert name == ("conv_umma_o2_512_pairs" if B > 8 else "conv_umma_o2_512_rows")


def test_config2_full_size():
    c = synth.config2()
    y, name = run_conv(c["dims"], c["x"], c["k"], False, M.M2_BF16)
    x64, k64 = c["x"].astype(np.float64), c["k"].astype(np.float64)
    ref = O.monarch_conv(k64[None], x64, c["dims"], causal=False)
    check(y, ref, TOL_BF16, "config2 full " + name)
    assert name == "conv_umma_o2_512_pairs"
    # sampled rows against the direct O(N^2) sum
    for b, h in [(0, 0), (31, 767), (7, 100), (16, 384), (1, 766), (30, 1), (12, 511), (5, 513)]:
        d = O.direct_circular_conv(k64[h], x64[b, h])
        check(y[b, h][None], d[None], TOL_BF16 / 2, f"config2 row ({b},{h}) direct")


@pytest.mark.parametrize("B,dims,n,causal,dtype,group", [(19, (32, 16), 512, False, M.M2_BF16, 4), (5, (32, 16), 256, True, M.M2_BF16, 3),
                                                          (3, (8, 4, 2), 30, True, M.M2_FP32, 2), (2, (32, 16), 100, True, M.M2_BF16, 6)])
def test_conv_with_a_kernel_shared_by_channel_groups(B, dims, n, causal, dtype, group):
    """m2_monarch_conv_fwd_grouped: channel h uses spectrum row h // group (both N = 512 tensor-core kernels and the
    general-shape kernel); same result as the plain call with the kernels repeated."""
    Hk = 5
    H = Hk * group
    rnd = (lambda a: synth.round_bf16(a)) if dtype == M.M2_BF16 else (lambda a: a.astype(np.float32).astype(np.float64))
    x = rnd(synth.normal(synth.stream_id(19, n), (B, H, n)))
    k = synth.decay_kernel(19, Hk, n, 0.01, 8.0)
    plan = M.Plan(dims, dtype=dtype, device=0)
    tdt = torch.bfloat16 if dtype == M.M2_BF16 else torch.float32
    kf = M.m2_kernel_spectrum(plan, dev(k))
    y = M.m2_monarch_conv_fwd_grouped(plan, dev(x.astype(np.float32), tdt), kf, M.M2_CAUSAL if causal else M.M2_CIRCULAR, group)
    torch.cuda.synchronize()
    assert plan.device_status() == 0
    krep = np.repeat(k.astype(np.float64), group, axis=0)
    ref = O.direct_causal_conv(krep[None], x) if causal else O.direct_circular_conv(krep[None], x)
    check(host(y), ref, TOL_BF16 if dtype == M.M2_BF16 else TOL_FP32, "grouped conv " + plan.last_kernel())
    lib, s = M.lib(), torch.cuda.current_stream().cuda_stream
    xd = dev(x.astype(np.float32), tdt)
    assert lib.m2_monarch_conv_fwd_grouped(plan.handle, xd.data_ptr(), kf.data_ptr(), y.data_ptr(), B, H, n, M.M2_CAUSAL if causal else M.M2_CIRCULAR, 0, s) == M.M2_ERR_INVALID_ARG
    assert lib.m2_monarch_conv_fwd_grouped(plan.handle, xd.data_ptr(), kf.data_ptr(), y.data_ptr(), B, H, n, M.M2_CAUSAL if causal else M.M2_CIRCULAR, H + 1, s) == M.M2_ERR_INVALID_ARG
    plan.close()


@pytest.mark.parametrize("B", [5, 19])
def test_bf16_causal_order2_and_ragged(B):
    for n in (256, 100, 48):
        H = 7
        x = synth.round_bf16(synth.normal(800 + n, (B, H, n)))
        k = synth.decay_kernel(2, H, n, 0.005, float(np.sqrt(512.0)))
        y, name = run_conv((32, 16), x, k, True, M.M2_BF16)
        ref = O.direct_causal_conv(k.astype(np.float64)[None], x.astype(np.float64))
        check(y, ref, TOL_BF16, f"bf16 causal n={n} {name}")


# ---- config 3: Monarch matmul ------------------------------------------------------------------

def run_matmul(c, dtype=M.M2_BF16):
    b = c["L"].shape[0]
    plan = M.Plan((b, b), dtype=dtype, device=0)
    tdt = torch.bfloat16 if dtype == M.M2_BF16 else torch.float32
    Y = M.m2_monarch_matmul(plan, dev(c["X"], tdt), dev(c["L"], tdt), dev(c["R"], tdt))
    torch.cuda.synchronize()
    assert plan.device_status() == 0
    name = plan.last_kernel()
    plan.close()
    return host(Y), name


@pytest.mark.parametrize("T,b", [(37, 64), (128, 64), (5, 8), (300, 16), (1, 64), (5001, 64)])   # 5001 tokens: both passes in one launch, ragged last tile
def test_config3_small_full_compare(T, b):
    c = synth.config3(T=T, b=b)
    Y, name = run_matmul(c)
    ref = O.monarch_apply(c["L"].astype(np.float64), c["R"].astype(np.float64), c["X"].astype(np.float64))
    check(Y, ref, TOL_BF16, f"config3 T={T} b={b} {name}")


def test_matmul_token_counts_around_the_tile_boundaries():
    """Token counts on both sides of the 32-token tile and of the 148 x 4 item boundaries, one plan and ONE workspace for
    all calls, no synchronisation between them (a call's pass 1 may only overwrite the workspace after the previous call's
    pass 2 has read it); rows past T of the output buffer must stay untouched."""
    c = synth.config3(T=4800, b=64)
    plan = M.Plan((64, 64), dtype=M.M2_BF16, device=0)
    L, R = dev(c["L"], torch.bfloat16), dev(c["R"], torch.bfloat16)
    Xall = dev(c["X"], torch.bfloat16)
    ws = M.m2_matmul_workspace(plan, 4800)
    counts = (31, 32, 33, 63, 64, 65, 1183, 1184, 1185, 4735, 4737, 4800, 2, 95)
    outs = []
    for T in counts:
        Y = torch.full((T + 3, 4096), 5.0, dtype=torch.bfloat16, device="cuda")
        M.m2_monarch_matmul(plan, Xall[:T], L, R, Y[:T], ws=ws)
        outs.append(Y)
    torch.cuda.synchronize()
    assert plan.device_status() == 0
    L64, R64 = c["L"].astype(np.float64), c["R"].astype(np.float64)
    ref = O.monarch_apply(L64, R64, c["X"].astype(np.float64))
    for T, Y in zip(counts, outs):
        assert bool((Y[T:] == 5.0).all()), f"T={T}: rows past T were written"
        check(host(Y[:T]), ref[:T], TOL_BF16, f"matmul T={T}")
    plan.close()


def test_matmul_input_at_an_odd_16_byte_offset():
    """X that is only 16-byte aligned (a view into a larger buffer) takes the kernels with 16-byte pieces: same result."""
    c = synth.config3(T=200, b=64)
    plan = M.Plan((64, 64), dtype=M.M2_BF16, device=0)
    buf = torch.zeros(200 * 4096 + 8, dtype=torch.bfloat16, device="cuda")
    X = buf[8:].view(200, 4096)
    X.copy_(dev(c["X"], torch.bfloat16))
    assert X.data_ptr() % 32 == 16
    Y = M.m2_monarch_matmul(plan, X, dev(c["L"], torch.bfloat16), dev(c["R"], torch.bfloat16))
    torch.cuda.synchronize()
    assert plan.device_status() == 0 and plan.last_kernel() == "matmul_umma_64x64_g8"
    ref = O.monarch_apply(c["L"].astype(np.float64), c["R"].astype(np.float64), c["X"].astype(np.float64))
    check(host(Y), ref, TOL_BF16, "matmul, 16-byte aligned input")
    plan.close()


@pytest.mark.parametrize("dims,T,dtype", [((4, 3, 5), 7, "fp32"), ((8, 8, 8), 9, "fp32"), ((2, 9, 5), 5, "fp32"), ((7,), 3, "fp32"),
                                          ((16, 16, 16), 33, "bf16"), ((32, 32, 32), 6, "bf16"), ((12, 40), 10, "bf16")])
def test_monarch_apply_order_p(dims, T, dtype):
    """Order-p product with arbitrary blocks (Eq. 1; App. D.6) against the oracle's direct form: orders 1 to 3, mixed digit
    sizes, the tokens-per-block variants of the kernel (4 for N <= 10240, 1 beyond)."""
    N = int(np.prod(dims))
    bf = dtype == "bf16"
    rnd = (lambda a: synth.round_bf16(a)) if bf else (lambda a: a.astype(np.float32))
    X = rnd(synth.normal(900 + N, (T, N)))
    W = [rnd(synth.normal(901 + N + a, (N // Na, Na, Na)) / np.sqrt(Na)) for a, Na in enumerate(dims)]
    plan = M.Plan(dims, dtype=M.M2_BF16 if bf else M.M2_FP32, device=0)
    tdt = torch.bfloat16 if bf else torch.float32
    Y = M.m2_monarch_apply_order_p(plan, dev(X, tdt), [dev(w, tdt) for w in W])
    torch.cuda.synchronize()
    assert plan.device_status() == 0 and plan.last_kernel() == "monarch_order_p_generic"
    ref = O.monarch_apply_order_p([w.astype(np.float64) for w in W], tuple(dims), X.astype(np.float64))
    check(host(Y), ref, TOL_BF16 if bf else TOL_FP32, f"order-p product {dims} {dtype}")
    plan.close()


def test_monarch_apply_order_p_is_the_matmul_for_p_2():
    """For p = 2 the direct form with W = (R, L) is M = P L P^T R P (Sec. 3.1): same result as m2_monarch_matmul."""
    c = synth.config3(T=40, b=16)
    plan = M.Plan((16, 16), dtype=M.M2_FP32, device=0)
    X, L, R = dev(c["X"].astype(np.float32)), dev(c["L"].astype(np.float32)), dev(c["R"].astype(np.float32))
    Y2 = M.m2_monarch_matmul(plan, X, L, R)
    Yp = M.m2_monarch_apply_order_p(plan, X, [R, L])
    torch.cuda.synchronize()
    check(host(Yp), host(Y2).astype(np.float64), 1e-6, "order-p product, p = 2, against the order-2 kernel")
    ref = O.monarch_apply(c["L"].astype(np.float64), c["R"].astype(np.float64), c["X"].astype(np.float64))
    check(host(Yp), ref, TOL_FP32, "order-p product, p = 2, against the oracle")
    # bad arguments: a missing factor, a digit beyond 256
    lib, st = M.lib(), torch.cuda.current_stream().cuda_stream
    import ctypes
    ptrs = (ctypes.c_void_p * 2)(R.data_ptr(), None)
    assert lib.m2_monarch_apply_order_p(plan.handle, X.data_ptr(), ptrs, Yp.data_ptr(), 40, st) == M.M2_ERR_INVALID_ARG
    plan.close()
    big = M.Plan((512, 8), dtype=M.M2_FP32, device=0)
    Xb = torch.zeros(1, 4096, device="cuda")
    Wb = [torch.zeros(8, 512, 512, device="cuda"), torch.zeros(512, 8, 8, device="cuda")]
    ptrs = (ctypes.c_void_p * 2)(Wb[0].data_ptr(), Wb[1].data_ptr())
    assert lib.m2_monarch_apply_order_p(big.handle, Xb.data_ptr(), ptrs, Xb.clone().data_ptr(), 1, st) == M.M2_ERR_UNSUPPORTED
    big.close()


def test_matmul_fp32_rectangular_vs_dense():
    N1, N2, T = 8, 4, 9
    X = synth.normal(31, (T, N1 * N2)).astype(np.float32)
    L = synth.normal(32, (N1, N2, N2)).astype(np.float32)
    R = synth.normal(33, (N2, N1, N1)).astype(np.float32)
    plan = M.Plan((N1, N2), dtype=M.M2_FP32, device=0)
    Y = host(M.m2_monarch_matmul(plan, dev(X), dev(L), dev(R)))
    Md = O.monarch_dense(L.astype(np.float64), R.astype(np.float64))
    check(Y, X.astype(np.float64) @ Md.T, TOL_FP32, "fp32 rectangular matmul vs dense P L P^T R P")
    plan.close()


def test_config3_full_size_every_token():
    """Config 3 at full size, every one of the 16384 tokens against the oracle, row by row (the oracle runs in chunks of
    2048 tokens to bound host memory)."""
    c = synth.config3()
    Y, name = run_matmul(c)
    assert name == "matmul_umma_64x64"
    L64, R64 = c["L"].astype(np.float64), c["R"].astype(np.float64)
    num = den = 0.0
    for t0 in range(0, c["X"].shape[0], 2048):
        ref = O.monarch_apply(L64, R64, c["X"][t0:t0 + 2048].astype(np.float64))
        check(Y[t0:t0 + 2048], ref, TOL_BF16, f"config3 full, tokens {t0}..{t0 + 2047} " + name)
        num += float(np.sum((Y[t0:t0 + 2048] - ref) ** 2))
        den += float(np.sum(ref ** 2))
    assert np.sqrt(num / den) <= TOL_BF16


# ---- config 4: order-3 causal, N = 32768 ------------------------------------------------------------

@pytest.mark.parametrize("B,H", [(1, 3), (2, 2)])
def test_config4_small_full_rows(B, H):
    c = synth.config4(B=B, H=H)
    y, name = run_conv(c["dims"], c["x"], c["k"], True, M.M2_BF16)
    ref = O.monarch_conv(c["k"].astype(np.float64)[None], c["x"].astype(np.float64), c["dims"], causal=True)
    check(y, ref, TOL_BF16, f"config4 B={B} H={H} {name}")


def test_config4_full_size_sampled():
    c = synth.config4()
    y, name = run_conv(c["dims"], c["x"], c["k"], True, M.M2_BF16)
    assert np.isfinite(y).all() and name == "conv_umma_o3_32k"
    # The kernel walks row pairs p = h * 2 + b0 / 2 (rows b0, b0 + 1 of channel h), CTA c of 148 taking p = c, c + 148, ...:
    # one row of every CTA's first pair and of its last pair, plus pairs spread over the whole range; the row within the
    # pair alternates, so every batch index occurs and the channels span 0 .. 1023.
    B4, H4, ctas = 4, 1024, 148
    npairs = H4 * (B4 // 2)
    first = list(range(ctas))
    last = [cta + ctas * ((npairs - 1 - cta) // ctas) for cta in range(ctas)]
    spread = list(range(7, npairs, 41))
    rows = [(3, 1023), (0, 0)]   # rows[0] is also checked against the direct sum below
    for i, p in enumerate(first + last + spread):
        rows.append((2 * (p % 2) + (i % 2), p // 2))
    rows = list(dict.fromkeys(rows))
    assert len(rows) >= 300 and {b for b, _ in rows} == {0, 1, 2, 3}
    xs = np.stack([c["x"][b, h] for b, h in rows]).astype(np.float64)
    ks = np.stack([c["k"][h] for b, h in rows]).astype(np.float64)
    ref = O.monarch_conv(ks, xs, c["dims"], causal=True)
    got = np.stack([y[b, h] for b, h in rows])
    check(got, ref, TOL_BF16, "config4 full sampled " + name)
    # direct sum at sampled outputs of one row
    for t in (0, 1, 1024, 9999, 16383):
        d = float(np.dot(ks[0][: t + 1], xs[0][t::-1]))
        assert abs(got[0][t] - d) <= 4e-2 * max(abs(d), np.abs(ref[0]).mean())
    # every row is sane: output energy within the range of the checked rows
    e = np.linalg.norm(y.reshape(-1, y.shape[-1]), axis=1)
    assert e.min() > 0.2 * np.median(e) and e.max() < 5 * np.median(e)


@pytest.mark.parametrize("B,H,n,causal", [(2, 3, 32768, False), (1, 2, 8192, True)])
def test_bf16_general_shape_kernel_on_long_rows(B, H, n, causal):
    """(32, 32, 32) bf16 requests the order-3 tensor-core kernel does not cover (circular, or causal with n != 16384) run on the
    general-shape kernel, which for rows this long keeps the row between its stages as bf16 pairs."""
    x = synth.round_bf16(synth.normal(synth.stream_id(17, n), (B, H, n)))
    k = synth.decay_kernel(17, H, n, 0.0005, 128.0)
    y, name = run_conv((32, 32, 32), x, k, causal, M.M2_BF16)
    assert name == "conv_generic_bf16io"
    ref = O.monarch_conv(k.astype(np.float64)[None], x.astype(np.float64), (32, 32, 32), causal=causal)
    check(y, ref, TOL_BF16, f"bf16 general-shape kernel n={n} causal={causal}")


# ---- config 5: the M2 block -------------------------------------------------------------------------

def run_block(c, kernel=None):
    plan = M.Plan(c["dims"], dtype=M.M2_BF16, device=0)
    kf = M.m2_kernel_spectrum(plan, dev(c["k"]))
    nblk, hid, cin = c["W_up"].shape
    y, z = M.m2_block_fwd(plan, dev(c["x"], torch.bfloat16), kf, dev(c["w_short"]), dev(c["W_up"], torch.bfloat16),
                          dev(c["W_down"], torch.bfloat16), nblk=nblk, expand=hid // cin)
    torch.cuda.synchronize()
    assert plan.device_status() == 0
    if kernel is not None:
        assert plan.last_kernel() == kernel
    plan.close()
    return host(y), host(z)


def block_ref(c, bsel=None):
    x = c["x"].astype(np.float64)
    if bsel is not None:
        x = x[bsel]
    return O.m2_block_forward(x, c["k"].astype(np.float64), c["w_short"].astype(np.float64),
                              c["W_up"].astype(np.float64), c["W_down"].astype(np.float64), c["dims"])


def test_config5_small():
    c = synth.config5(B=2)
    y, z = run_block(c, "block_conv_umma_mlp_umma")
    yr, zr = block_ref(c)
    check(z.reshape(2 * 512, 768), zr.reshape(2 * 512, 768), TOL_BF16, "config5 z")
    check(y.reshape(2 * 512, 768), yr.reshape(2 * 512, 768), TOL_BF16, "config5 y")


@pytest.mark.parametrize("T,C,nblk,expand,dims,kernel", [
    (64, 32, 4, 2, (8, 8), "block_generic"),                       # neither tensor-core kernel covers it
    (512, 128, 4, 2, (32, 16), "block_conv_umma_mlp_generic"),    # tensor-core mixer, CUDA-core MLP
])
def test_block_other_shapes(T, C, nblk, expand, dims, kernel):
    c = synth.config5(B=3, T=T, C=C, nblk=nblk, expand=expand)
    c["dims"] = dims
    y, z = run_block(c, kernel)
    yr, zr = block_ref(c)
    check(z.reshape(-1, C), zr.reshape(-1, C), TOL_BF16, "block z")
    check(y.reshape(-1, C), yr.reshape(-1, C), TOL_BF16, "block y")


@pytest.mark.parametrize("B", [1, 9, 17])
def test_config5_ragged_batches(B):
    """Batch sizes that leave the last 16-row unit of the gated convolution partly empty (rows past B are never read or written)."""
    c = synth.config5(B=B)
    y, z = run_block(c, "block_conv_umma_mlp_umma")
    sel = sorted({0, B // 2, B - 1})
    yr, zr = block_ref(c, sel)
    check(z[sel].reshape(-1, 768), zr.reshape(-1, 768), TOL_BF16, "config5 ragged z")
    check(y[sel].reshape(-1, 768), yr.reshape(-1, 768), TOL_BF16, "config5 ragged y")


def test_block_z_layout_query_matches_the_buffer():
    """Where the query says so, the z buffer is channel-first [B, C, T]; elsewhere [B, T, C].  Called through the C ABI with the
    caller's own buffers, canaries behind both."""
    lib = M.lib()
    s = torch.cuda.current_stream().cuda_stream
    for (T, C, nblk, expand, dims, want) in ((512, 768, 4, 4, (32, 16), 1), (512, 128, 4, 2, (32, 16), 0), (64, 32, 4, 2, (8, 8), 0)):
        c = synth.config5(B=3, T=T, C=C, nblk=nblk, expand=expand)
        c["dims"] = dims
        plan = M.Plan(dims, dtype=M.M2_BF16, device=0)
        assert lib.m2_block_z_channel_first(plan.handle, T, C, nblk, expand) == want
        assert lib.m2_block_z_channel_first(plan.handle, T, C, 0, expand) == 0 and lib.m2_block_z_channel_first(None, T, C, nblk, expand) == 0
        kf = M.m2_kernel_spectrum(plan, dev(c["k"]))
        x, w, wu, wd = dev(c["x"], torch.bfloat16), dev(c["w_short"]), dev(c["W_up"], torch.bfloat16), dev(c["W_down"], torch.bfloat16)
        n = 3 * T * C
        zbuf = torch.full((n + 64,), 7.0, dtype=torch.bfloat16, device="cuda")
        ybuf = torch.full((n + 64,), 7.0, dtype=torch.bfloat16, device="cuda")
        assert lib.m2_block_fwd(plan.handle, x.data_ptr(), kf.data_ptr(), w.data_ptr(), wu.data_ptr(), wd.data_ptr(), zbuf.data_ptr(),
                                ybuf.data_ptr(), 3, T, C, nblk, expand, s) == M.M2_OK
        torch.cuda.synchronize()
        assert plan.device_status() == 0
        assert (zbuf[n:] == 7).all().item() and (ybuf[n:] == 7).all().item()
        yr, zr = block_ref(c)
        z = zbuf[:n].view(3, C, T).transpose(1, 2) if want else zbuf[:n].view(3, T, C)
        check(host(z).reshape(-1, C), zr.reshape(-1, C), TOL_BF16, f"block z buffer layout T={T} C={C}")
        check(host(ybuf[:n].view(3, T, C)).reshape(-1, C), yr.reshape(-1, C), TOL_BF16, f"block y T={T} C={C}")
        plan.close()


def test_config5_full_size_sampled():
    c = synth.config5()
    y, z = run_block(c)
    assert np.isfinite(y).all()
    sel = [0, 17, 31]
    yr, zr = block_ref(c, sel)
    check(z[sel].reshape(-1, 768), zr.reshape(-1, 768), TOL_BF16, "config5 full z")
    check(y[sel].reshape(-1, 768), yr.reshape(-1, 768), TOL_BF16, "config5 full y")


# ---- gradient with respect to the input: the same kernels with the conjugated spectrum ---------------------

@pytest.mark.parametrize("cfg,kernel", [("c1", None), ("c2", "conv_umma_o2_512_rows"), ("c2causal", "conv_umma_o2_512_rows"), ("c2pairs", "conv_umma_o2_512_pairs"),
                                         ("c4", "conv_umma_o3_32k")])
def test_conv_input_gradient(cfg, kernel):
    if cfg == "c1":
        c, causal, dtype, tol = synth.config1(), True, M.M2_FP32, TOL_FP32
    elif cfg == "c2":
        c, causal, dtype, tol = synth.config2(B=8, H=12), False, M.M2_BF16, TOL_BF16
    elif cfg == "c2pairs":
        c, causal, dtype, tol = synth.config2(B=11, H=12), False, M.M2_BF16, TOL_BF16
    elif cfg == "c2causal":
        c = synth.config2(B=8, H=12)
        c = dict(c, x=c["x"][..., :256].copy(), k=c["k"][..., :256].copy())
        causal, dtype, tol = True, M.M2_BF16, TOL_BF16
    else:
        c, causal, dtype, tol = synth.config4(B=2, H=2), True, M.M2_BF16, TOL_BF16
    plan = M.Plan(c["dims"], dtype=dtype, device=0)
    tdt = torch.bfloat16 if dtype == M.M2_BF16 else torch.float32
    g = dev(c["x"].astype(np.float32), tdt)               # any tensor of the right shape serves as upstream gradient
    H = c["k"].shape[0]
    kf = M.m2_kernel_spectrum(plan, dev(c["k"].astype(np.float32)))
    kfc = M.m2_spectrum_conjugate(plan, kf, H)
    dx = M.m2_monarch_conv_fwd(plan, g, kfc, M.M2_CAUSAL if causal else M.M2_CIRCULAR)
    torch.cuda.synchronize()
    assert plan.device_status() == 0
    if kernel is not None:
        assert plan.last_kernel() == kernel
    ref = O.monarch_conv_adjoint(c["k"].astype(np.float64), c["x"].astype(np.float64), c["dims"], causal)
    check(host(dx), ref, tol, "input gradient " + cfg)
    # conjugating twice gives the spectrum back, bit for bit, in place
    M.m2_spectrum_conjugate(plan, kfc, H, out=kfc)
    torch.cuda.synchronize()
    assert torch.equal(kfc, kf)
    plan.close()


@pytest.mark.parametrize("cfg,use_ws", [("c1", True), ("c2", False), ("c2", True), ("c2big", True), ("c2causal", True),
                                        ("c2causal256", True), ("small3", True), ("c4small", True), ("c4odd", True), ("c4cuda", True)])
def test_conv_kernel_gradient(cfg, use_ws):
    if cfg == "c1":
        c, causal, dtype, tol = synth.config1(), True, M.M2_FP32, 1e-5
    elif cfg == "c2":
        c, causal, dtype, tol = synth.config2(B=8, H=12), False, M.M2_BF16, 1e-5   # bf16 inputs are exact in fp32: fp32 accuracy
    elif cfg == "c2big":     # several units per pipeline, a ragged last batch group
        c, causal, dtype, tol = synth.config2(B=19, H=160), False, M.M2_BF16, 1e-5
    elif cfg == "c2causal":  # n not a multiple of 16: no tensor-core kernel
        c = synth.config2(B=5, H=7)
        c = dict(c, x=c["x"][..., :200].copy(), k=c["k"][..., :200].copy())
        causal, dtype, tol = True, M.M2_BF16, 1e-5
    elif cfg == "c2causal256":
        c = synth.config2(B=5, H=7)
        c = dict(c, x=c["x"][..., :256].copy(), k=c["k"][..., :256].copy())
        causal, dtype, tol = True, M.M2_BF16, 1e-5
    elif cfg == "c4small":   # N = 32768 on the tensor cores: pair spectra, convolution of the g pairs, sum over the pairs
        c, causal, dtype, tol = synth.config4(B=4, H=3), True, M.M2_BF16, 1e-5
    elif cfg == "c4odd":     # an odd batch: the last pair has one row
        c, causal, dtype, tol = synth.config4(B=3, H=2), True, M.M2_BF16, 1e-5
    elif cfg == "c4cuda":    # N = 32768 with a workspace that only the CUDA-core kernel can use (rows too long for shared memory)
        c, causal, dtype, tol = synth.config4(B=8, H=1), True, M.M2_BF16, 1e-5
    else:
        c = dict(x=synth.round_bf16(synth.normal(synth.stream_id(9, 0), (3, 4, 32))), dims=(4, 4, 4))
        causal, dtype, tol = True, M.M2_BF16, 1e-5
    plan = M.Plan(c["dims"], dtype=dtype, device=0)
    tdt = torch.bfloat16 if dtype == M.M2_BF16 else torch.float32
    x = c["x"].astype(np.float64)
    gup = synth.round_bf16(synth.normal(synth.stream_id(9, 1), x.shape)).astype(np.float64)   # upstream gradient
    ws = None
    if cfg == "c4cuda":   # 3 complex rows of one channel: less than the tensor-core path needs for 4 pairs
        ws = torch.empty(3 * 32768 * 8, dtype=torch.uint8, device="cuda")
    dk = M.m2_monarch_conv_bwd_kernel(plan, dev(x.astype(np.float32), tdt), dev(gup.astype(np.float32), tdt),
                                      M.M2_CAUSAL if causal else M.M2_CIRCULAR, ws=ws, use_workspace=use_ws)
    torch.cuda.synchronize()
    umma = use_ws and cfg in ("c2", "c2big", "c2causal256", "c4small", "c4odd")
    want = "conv_wgrad_generic" if not umma else "conv_wgrad_umma_o3_32k" if cfg.startswith("c4") else "conv_wgrad_umma_o2_512"
    assert plan.device_status() == 0 and plan.last_kernel() == want
    ref = O.monarch_conv_kernel_grad(x, gup, c["dims"], causal)
    check(host(dk), ref, TOL_BF16 if umma else tol, "kernel gradient " + cfg)   # tensor-core path: bf16 intermediates
    plan.close()


@pytest.mark.parametrize("T,dims,dtype", [(300, (64, 64), M.M2_BF16), (40, (8, 8), M.M2_BF16), (17, (6, 4), M.M2_FP32)])
def test_matmul_input_gradient(T, dims, dtype):
    N1, N2 = dims
    tdt = torch.bfloat16 if dtype == M.M2_BF16 else torch.float32
    rnd = (lambda a: synth.round_bf16(a)) if dtype == M.M2_BF16 else (lambda a: a.astype(np.float32).astype(np.float64))
    L = rnd(synth.normal(synth.stream_id(8, 0), (N1, N2, N2)) / np.sqrt(N2))
    R = rnd(synth.normal(synth.stream_id(8, 1), (N2, N1, N1)) / np.sqrt(N1))
    G = rnd(synth.normal(synth.stream_id(8, 2), (T, N1 * N2)))
    plan_t = M.Plan((N2, N1), dtype=dtype, device=0)       # factors in the opposite order
    dX = M.m2_monarch_matmul_bwd_input(plan_t, dev(G.astype(np.float32), tdt), dev(L.astype(np.float32), tdt),
                                       dev(R.astype(np.float32), tdt))
    torch.cuda.synchronize()
    assert plan_t.device_status() == 0
    if dims == (64, 64):
        assert plan_t.last_kernel() == "matmul_umma_64x64"
    ref = O.monarch_apply_transpose(L.astype(np.float64), R.astype(np.float64), G.astype(np.float64))
    check(host(dX), ref, TOL_BF16 if dtype == M.M2_BF16 else TOL_FP32, "matmul input gradient")
    plan_t.close()


@pytest.mark.parametrize("T,dims,dtype", [(300, (64, 64), M.M2_BF16), (2500, (64, 64), M.M2_BF16), (64, (64, 64), M.M2_BF16),
                                          (0, (64, 64), M.M2_BF16), (77, (8, 16), M.M2_BF16), (33, (6, 4), M.M2_FP32),
                                          (40, (64, 64), M.M2_FP32), (0, (4, 4), M.M2_FP32)])
def test_matmul_weight_gradients(T, dims, dtype):
    N1, N2 = dims
    tdt = torch.bfloat16 if dtype == M.M2_BF16 else torch.float32
    rnd = (lambda a: synth.round_bf16(a)) if dtype == M.M2_BF16 else (lambda a: a.astype(np.float32).astype(np.float64))
    L = rnd(synth.normal(synth.stream_id(9, 0), (N1, N2, N2)) / np.sqrt(N2))
    R = rnd(synth.normal(synth.stream_id(9, 1), (N2, N1, N1)) / np.sqrt(N1))
    X = rnd(synth.normal(synth.stream_id(9, 2), (T, N1 * N2)))
    G = rnd(synth.normal(synth.stream_id(9, 3), (T, N1 * N2)))
    plan = M.Plan(dims, dtype=dtype, device=0)
    dL, dR = M.m2_monarch_matmul_bwd_weights(plan, dev(X.astype(np.float32), tdt), dev(G.astype(np.float32), tdt),
                                             dev(L.astype(np.float32), tdt), dev(R.astype(np.float32), tdt))
    torch.cuda.synchronize()
    umma = dims == (64, 64) and dtype == M.M2_BF16
    assert plan.device_status() == 0
    if T > 0:
        assert plan.last_kernel() == ("matmul_wgrad_umma_64x64" if umma else "matmul_wgrad_generic")
    rL, rR = O.monarch_weight_grads(L, R, X, G)
    # CUDA-core path: inputs are exactly representable and every product is accumulated in fp32, so the fp32 tolerance holds
    # for both dtypes; tensor-core path: the stage intermediate passes through bf16
    check(host(dL), rL, TOL_BF16 if umma else TOL_FP32, "dL")
    check(host(dR), rR, TOL_BF16 if umma else TOL_FP32, "dR")
    plan.close()


@pytest.mark.parametrize("T,Hk,dims,dtype,act", [(300, 3, (64, 64), M.M2_BF16, "relu"), (257, 257, (64, 64), M.M2_BF16, "none"),
                                                  (50, 1, (8, 4), M.M2_BF16, "relu"), (19, 5, (4, 6), M.M2_FP32, "relu"),
                                                  (19, 19, (4, 6), M.M2_FP32, "none")])
def test_monarch_mix_operator(T, Hk, dims, dtype, act):
    """Y = M_b sigma(K (.) M_a X) with general Monarch factors (Eq. 2; the mixing lines of the M2 layer listing)."""
    N1, N2 = dims
    N = N1 * N2
    tdt = torch.bfloat16 if dtype == M.M2_BF16 else torch.float32
    rnd = (lambda a: synth.round_bf16(a)) if dtype == M.M2_BF16 else (lambda a: a.astype(np.float32).astype(np.float64))
    W = [rnd(synth.normal(synth.stream_id(10, i), shp) / np.sqrt(shp[-1]))
         for i, shp in enumerate([(N1, N2, N2), (N2, N1, N1), (N1, N2, N2), (N2, N1, N1)])]
    K = rnd(synth.normal(synth.stream_id(10, 4), (Hk, N)))
    X = rnd(synth.normal(synth.stream_id(10, 5), (T, N)))
    plan = M.Plan(dims, dtype=dtype, device=0)
    d = lambda a: dev(a.astype(np.float32), tdt)   # noqa: E731
    Xd = d(X)
    Y = M.m2_monarch_mix(plan, Xd, d(K), d(W[0]), d(W[1]), d(W[2]), d(W[3]), act=M.M2_ACT_RELU if act == "relu" else M.M2_ACT_NONE)
    torch.cuda.synchronize()
    assert plan.device_status() == 0
    assert plan.last_kernel() == ("matmul_umma_64x64" if dims == (64, 64) else "matmul_generic")
    ref = O.monarch_mix(W[0], W[1], W[2], W[3], K, X, act)
    tol = TOL_BF16 if dtype == M.M2_BF16 else TOL_FP32
    check(host(Y), ref, tol, "monarch mix")
    # in place (Y = X) gives the same bits
    Y2 = M.m2_monarch_mix(plan, Xd, d(K), d(W[0]), d(W[1]), d(W[2]), d(W[3]), act=M.M2_ACT_RELU if act == "relu" else M.M2_ACT_NONE, Y=Xd)
    torch.cuda.synchronize()
    assert torch.equal(Y2, Y)
    plan.close()


@pytest.mark.parametrize("B,sn,sd,dtype", [(2, 64, 8, M.M2_BF16), (3, 5, 3, M.M2_FP32), (2, 8, 64, M.M2_BF16)])
def test_m2_layer_fwd(B, sn, sd, dtype):
    """The basic M2 layer (the MonarchMixerLayer listing): sequence mix, feature mix, residual LayerNorm."""
    n, d = sn * sn, sd * sd
    tdt = torch.bfloat16 if dtype == M.M2_BF16 else torch.float32
    rnd = (lambda a: synth.round_bf16(a)) if dtype == M.M2_BF16 else (lambda a: a.astype(np.float32).astype(np.float64))
    p = {}
    for i, s in ((1, sn), (2, sn), (3, sd), (4, sd)):
        p[f"L{i}"] = rnd(synth.normal(synth.stream_id(11, 2 * i), (s, s, s)) / np.sqrt(s))
        p[f"R{i}"] = rnd(synth.normal(synth.stream_id(11, 2 * i + 1), (s, s, s)) / np.sqrt(s))
    p["n_kernel"] = rnd(synth.normal(synth.stream_id(11, 20), (d, n)))
    p["d_kernel"] = rnd(synth.normal(synth.stream_id(11, 21), (1, d)))
    p["gamma"] = (1.0 + 0.1 * synth.normal(synth.stream_id(11, 22), (d,))).astype(np.float32).astype(np.float64)
    p["beta"] = (0.1 * synth.normal(synth.stream_id(11, 23), (d,))).astype(np.float32).astype(np.float64)
    x = rnd(synth.normal(synth.stream_id(11, 24), (B, n, d)))
    plan_n, plan_d = M.Plan((sn, sn), dtype=dtype, device=0), M.Plan((sd, sd), dtype=dtype, device=0)
    dv = lambda a: dev(a.astype(np.float32), tdt)   # noqa: E731
    fac = [dv(p[k]) for k in ("L1", "R1", "L2", "R2", "L3", "R3", "L4", "R4")]
    y = M.m2_layer_fwd(plan_n, plan_d, dv(x), fac, dv(p["n_kernel"]), dv(p["d_kernel"]),
                       dev(p["gamma"].astype(np.float32), torch.float32), dev(p["beta"].astype(np.float32), torch.float32))
    torch.cuda.synchronize()
    assert plan_n.device_status() == 0 and plan_d.device_status() == 0 and plan_n.last_kernel() == "layer_fwd"
    ref = O.m2_layer(x, p)
    check(host(y), ref, TOL_BF16 if dtype == M.M2_BF16 else TOL_FP32, "M2 layer")
    plan_n.close()
    plan_d.close()


@pytest.mark.parametrize("b,Bt,d,dtype,withK", [(64, 2, 192, M.M2_BF16, True), (128, 1, 256, M.M2_BF16, True), (256, 1, 64, M.M2_BF16, False),
                                                 (256, 2, 256, M.M2_BF16, True), (64, 1, 768, M.M2_BF16, False), (64, 2, 200, M.M2_BF16, True),
                                                 (128, 1, 328, M.M2_BF16, True), (64, 1, 8, M.M2_BF16, False), (192, 1, 72, M.M2_BF16, True), (8, 3, 40, M.M2_BF16, True), (6, 2, 33, M.M2_FP32, True)])
def test_monarch_cols(b, Bt, d, dtype, withK):
    """Y = sigma(K (.) M X) with the columns of X [Bt, N, d] as the vectors (the layout of the operator benchmark)."""
    run_monarch_cols(b, b, Bt, d, dtype, withK)


@pytest.mark.parametrize("N1,N2,d", [(64, 128, 72), (128, 64, 256), (192, 64, 64)])
def test_monarch_cols_rectangular(N1, N2, d):
    run_monarch_cols(N1, N2, 2, d, M.M2_BF16, True)


@pytest.mark.parametrize("N1,N2,d,dtype", [(64, 64, 72, M.M2_BF16), (64, 128, 64, M.M2_BF16), (5, 3, 7, M.M2_FP32)])
def test_monarch_cols_input_gradient(N1, N2, d, dtype):
    """dX = M^T G in the column layout: the forward kernels with swapped, block-transposed factors on the (N2, N1) plan."""
    tdt = torch.bfloat16 if dtype == M.M2_BF16 else torch.float32
    rnd = (lambda a: synth.round_bf16(a)) if dtype == M.M2_BF16 else (lambda a: a.astype(np.float32).astype(np.float64))
    L = rnd(synth.normal(synth.stream_id(16, 0), (N1, N2, N2)) / np.sqrt(N2))
    R = rnd(synth.normal(synth.stream_id(16, 1), (N2, N1, N1)) / np.sqrt(N1))
    G = rnd(synth.normal(synth.stream_id(16, 2), (2, N1 * N2, d)))
    plan_t = M.Plan((N2, N1), dtype=dtype, device=0)
    dv = lambda a: dev(a.astype(np.float32), tdt)   # noqa: E731
    dX = M.m2_monarch_cols_bwd_input(plan_t, dv(G), dv(L), dv(R))
    torch.cuda.synchronize()
    assert plan_t.device_status() == 0
    ref = np.swapaxes(O.monarch_apply_transpose(L, R, np.swapaxes(G, 1, 2)), 1, 2)   # M^T applied down the columns
    check(host(dX), ref, TOL_BF16 if dtype == M.M2_BF16 else TOL_FP32, "cols input gradient")
    plan_t.close()


def run_monarch_cols(N1, N2, Bt, d, dtype, withK):
    b = N1
    N = N1 * N2
    tdt = torch.bfloat16 if dtype == M.M2_BF16 else torch.float32
    rnd = (lambda a: synth.round_bf16(a)) if dtype == M.M2_BF16 else (lambda a: a.astype(np.float32).astype(np.float64))
    L = rnd(synth.normal(synth.stream_id(13, 0), (N1, N2, N2)) / np.sqrt(N2))
    R = rnd(synth.normal(synth.stream_id(13, 1), (N2, N1, N1)) / np.sqrt(N1))
    X = rnd(synth.normal(synth.stream_id(13, 2), (Bt, N, d)))
    K = rnd(synth.normal(synth.stream_id(13, 3), (N, d))) if withK else None
    plan = M.Plan((N1, N2), dtype=dtype, device=0)
    dv = lambda a: dev(a.astype(np.float32), tdt)   # noqa: E731
    Y = M.m2_monarch_cols(plan, dv(X), dv(L), dv(R), None if K is None else dv(K), act=M.M2_ACT_RELU if withK else M.M2_ACT_NONE)
    torch.cuda.synchronize()
    assert plan.device_status() == 0
    umma = dtype == M.M2_BF16 and N1 % 64 == 0 and N2 % 64 == 0 and d % 8 == 0
    assert plan.last_kernel() == ("monarch_cols_umma" if umma else "monarch_cols_generic")
    ref = O.monarch_cols(L, R, X, K, "relu" if withK else "none")
    check(host(Y), ref, TOL_BF16 if dtype == M.M2_BF16 else TOL_FP32, f"monarch cols {N1}x{N2}")
    plan.close()


@pytest.mark.parametrize("B,n,d,dh,dims,dtype", [(9, 256, 128, 16, (32, 16), M.M2_BF16),   # heads of 16: one fused tensor-core kernel
                                                  (3, 112, 64, 16, (32, 16), M.M2_BF16),    # the same with a ragged sequence length
                                                  (2, 100, 64, 4, (32, 16), M.M2_BF16),     # other head sizes: three kernels
                                                  (2, 24, 12, 3, (8, 8), M.M2_FP32)])
def test_m2_hyena_heads_fwd(B, n, d, dh, dims, dtype):
    """The M2 Hyena layer with heads: projections, short convolutions, head outer products through the long convolution, output
    projection (all channel-first after one transposition)."""
    tdt = torch.bfloat16 if dtype == M.M2_BF16 else torch.float32
    rnd = (lambda a: synth.round_bf16(a)) if dtype == M.M2_BF16 else (lambda a: a.astype(np.float32).astype(np.float64))
    p = {k: rnd(synth.normal(synth.stream_id(14, i), (d, d)) / np.sqrt(d)) for i, k in enumerate(("W_x1", "W_x2", "W_v", "W_o"))}
    dec = np.exp(-0.05 * np.arange(n))[None]
    for i, k in enumerate(("K1", "K2", "K3")):
        p[k] = (synth.normal(synth.stream_id(14, 4 + i), (d, n)) * dec / 4).astype(np.float32).astype(np.float64)
    p["K_long"] = (synth.normal(synth.stream_id(14, 7), (d // dh, n)) * dec / 4).astype(np.float32).astype(np.float64)
    u = rnd(synth.normal(synth.stream_id(14, 8), (B, n, d)))
    plan = M.Plan(dims, dtype=dtype, device=0)
    f32 = lambda a: torch.from_numpy(a.astype(np.float32)).cuda()   # noqa: E731
    kfs = [M.m2_kernel_spectrum(plan, f32(p[k])) for k in ("K1", "K2", "K3")]
    kfl = M.m2_kernel_spectrum(plan, f32(p["K_long"]))       # one row per head; its dh^2 sequences share it
    dv = lambda a: dev(a.astype(np.float32), tdt)   # noqa: E731
    W = [dv(np.ascontiguousarray(p[k].T)) for k in ("W_x1", "W_x2", "W_v", "W_o")]   # stored outputs x inputs
    y = M.m2_hyena_heads_fwd(plan, dv(u), W, kfs[0], kfs[1], kfs[2], kfl, dh)
    torch.cuda.synchronize()
    fused = dtype == M.M2_BF16 and dims == (32, 16) and dh == 16 and n % 16 == 0 and n <= 256
    assert plan.device_status() == 0 and plan.last_kernel() == ("hyena_heads_fwd_fused" if fused else "hyena_heads_fwd")
    ref = O.m2_hyena_heads(u, p, dims, dh)
    # The first positions of a causal layer have tiny outputs (one term of every convolution), so their rows are judged
    # against the typical row norm: an absolute error bound of 2 tol x the RMS row norm, plus the global relative bound.
    tol = TOL_BF16 if dtype == M.M2_BF16 else TOL_FP32
    got = host(y).reshape(B * n, d)
    want = ref.reshape(B * n, d)
    assert np.isfinite(got).all()
    gl = np.linalg.norm(got - want) / np.linalg.norm(want)
    rms_row = np.sqrt(np.mean(np.sum(want ** 2, axis=1)))
    worst = np.max(np.linalg.norm(got - want, axis=1)) / rms_row
    assert gl <= tol, f"global rel-L2 {gl:.3e} > {tol}"
    assert worst <= 2 * tol, f"worst row error {worst:.3e} of the RMS row norm > {2 * tol}"
    plan.close()


def test_m2_hyena_heads_full_size_sampled():
    """The layer at the benchmark shape (B = 32, n = 256, d = 768, heads of 16: 24 576 units of the fused kernel, many rounds per
    pipeline); batch entries are independent, so the first and the last one are compared with the oracle run on them alone."""
    B, n, d, dh, dims = 32, 256, 768, 16, (32, 16)
    rnd = synth.round_bf16
    p = {k: rnd(synth.normal(synth.stream_id(16, i), (d, d)) / np.sqrt(d)) for i, k in enumerate(("W_x1", "W_x2", "W_v", "W_o"))}
    dec = np.exp(-0.05 * np.arange(n))[None]
    for i, k in enumerate(("K1", "K2", "K3")):
        p[k] = (synth.normal(synth.stream_id(16, 4 + i), (d, n)) * dec / 4).astype(np.float32).astype(np.float64)
    p["K_long"] = (synth.normal(synth.stream_id(16, 7), (d // dh, n)) * dec / 4).astype(np.float32).astype(np.float64)
    u = rnd(synth.normal(synth.stream_id(16, 8), (B, n, d)))
    plan = M.Plan(dims, dtype=M.M2_BF16, device=0)
    f32 = lambda a: torch.from_numpy(a.astype(np.float32)).cuda()   # noqa: E731
    kfs = [M.m2_kernel_spectrum(plan, f32(p[k])) for k in ("K1", "K2", "K3")]
    kfl = M.m2_kernel_spectrum(plan, f32(p["K_long"]))
    dv = lambda a: dev(a.astype(np.float32), torch.bfloat16)   # noqa: E731
    W = [dv(np.ascontiguousarray(p[k].T)) for k in ("W_x1", "W_x2", "W_v", "W_o")]
    y = M.m2_hyena_heads_fwd(plan, dv(u), W, kfs[0], kfs[1], kfs[2], kfl, dh)
    torch.cuda.synchronize()
    assert plan.device_status() == 0 and plan.last_kernel() == "hyena_heads_fwd_fused"
    got_all = host(y)
    assert np.isfinite(got_all).all()
    sel = [0, B - 1]
    ref = O.m2_hyena_heads(u[sel], p, dims, dh)
    got, want = got_all[sel].reshape(-1, d), ref.reshape(-1, d)
    gl = np.linalg.norm(got - want) / np.linalg.norm(want)
    rms_row = np.sqrt(np.mean(np.sum(want * want, axis=1)))
    worst = np.max(np.linalg.norm(got - want, axis=1)) / rms_row   # (first causal positions are tiny: judged against the typical row)
    assert gl <= TOL_BF16, f"global rel-L2 {gl:.3e}"
    assert worst <= 2 * TOL_BF16, f"worst row error {worst:.3e} of the RMS row norm"
    plan.close()


@pytest.mark.parametrize("B,d,dims,dtype", [(12, 128, (32, 16), M.M2_BF16), (3, 24, (32, 16), M.M2_BF16), (2, 10, (6, 4), M.M2_FP32)])
def test_m2_bert_mixer_fwd(B, d, dims, dtype):
    """The gated bidirectional M2-BERT sequence mixer: projections, short filters, gated long convolution + residual convolution,
    output projection."""
    n = int(np.prod(dims))
    tdt = torch.bfloat16 if dtype == M.M2_BF16 else torch.float32
    rnd = (lambda a: synth.round_bf16(a)) if dtype == M.M2_BF16 else (lambda a: a.astype(np.float32).astype(np.float64))
    p = {k: rnd(synth.normal(synth.stream_id(15, i), (d, d)) / np.sqrt(d)) for i, k in enumerate(("W_q", "W_k", "W_v", "W_o"))}
    for i, k in enumerate(("w_q", "w_k", "w_v")):
        p[k] = (synth.normal(synth.stream_id(15, 4 + i), (d, 3)) / np.sqrt(3.0)).astype(np.float32).astype(np.float64)
    dec = np.exp(-0.02 * np.arange(n))[None]
    p["k"] = (synth.normal(synth.stream_id(15, 7), (d, n)) * dec / 4).astype(np.float32).astype(np.float64)
    p["k_res"] = (synth.normal(synth.stream_id(15, 8), (d, n)) * dec / 4).astype(np.float32).astype(np.float64)
    x = rnd(synth.normal(synth.stream_id(15, 9), (B, n, d)))
    plan = M.Plan(dims, dtype=dtype, device=0)
    f32 = lambda a: torch.from_numpy(a.astype(np.float32)).cuda()   # noqa: E731
    kf, kfr = M.m2_kernel_spectrum(plan, f32(p["k"])), M.m2_kernel_spectrum(plan, f32(p["k_res"]))
    dv = lambda a: dev(a.astype(np.float32), tdt)   # noqa: E731
    W = [dv(np.ascontiguousarray(p[k].T)) for k in ("W_q", "W_k", "W_v", "W_o")]
    y = M.m2_bert_mixer_fwd(plan, dv(x), W, [f32(p[k]) for k in ("w_q", "w_k", "w_v")], kf, kfr)
    torch.cuda.synchronize()
    fused = dtype == M.M2_BF16 and dims == (32, 16)   # output gate and residual add inside the main convolution
    assert plan.device_status() == 0 and plan.last_kernel() == ("bert_mixer_fwd_fused_gate" if fused else "bert_mixer_fwd")
    ref = O.m2_bert_mixer(x, p, dims)
    check(host(y), ref, TOL_BF16 if dtype == M.M2_BF16 else TOL_FP32, "M2-BERT gated mixer")
    plan.close()


# ---- learnable (causal) Monarch from polynomial coefficients (App. D.5) --------------------------------------------------

def _blocky_coefficients(b, seed, noise):
    """Near-identity coefficient matrices (the DFT's plus noise), rounded to fp32: what a learnable layer starts from."""
    N = b * b
    Lt = np.zeros((N, b))
    Lt[:b] = np.eye(b)
    Rt = np.tile(np.eye(b), (b, 1))
    Lt = Lt + noise * synth.normal(synth.stream_id(18, seed), (N, b)) / np.sqrt(b)
    Rt = Rt + noise * synth.normal(synth.stream_id(18, seed + 1), (N, b)) / np.sqrt(b)
    return Lt.astype(np.float32).astype(np.float64), Rt.astype(np.float32).astype(np.float64)


@pytest.mark.parametrize("b,n,dtype,masked,noise", [(8, 32, M.M2_FP32, True, 0.3), (16, 128, M.M2_FP32, True, 0.3), (16, 100, M.M2_BF16, True, 0.3),
                                                     (32, 512, M.M2_BF16, True, 0.2), (6, 11, M.M2_FP32, True, 0.3), (8, 30, M.M2_FP32, False, 0.3),
                                                     (16, 128, M.M2_FP32, True, 0.0), (64, 2048, M.M2_BF16, True, 0.1)])
def test_blocky_monarch_conv(b, n, dtype, masked, noise):
    """Alg. BlockyMonarch + Alg. BlockMonarchConv on the device against the oracle: factors from coefficient matrices (with the
    causal zero patterns applied on the device), kernel spectrum, convolution; the masked operator is causal on the device too."""
    N = b * b
    Bn, H = 3, 4
    Lt, Rt = _blocky_coefficients(b, 10 * b, noise)
    k = synth.decay_kernel(18, H, n, 2.0 / n, 4.0).astype(np.float64)
    rnd = (lambda a: synth.round_bf16(a)) if dtype == M.M2_BF16 else (lambda a: a.astype(np.float32).astype(np.float64))
    x = rnd(synth.normal(synth.stream_id(18, 3), (Bn, H, n)))
    plan = M.Plan((b, b), dtype=dtype, device=0)
    tdt = torch.bfloat16 if dtype == M.M2_BF16 else torch.float32
    fac = M.m2_blocky_monarch(plan, dev(Lt.astype(np.float32)), dev(Rt.astype(np.float32)), causal_mask=masked)
    kf = M.m2_blocky_kernel_spectrum(plan, fac, dev(k.astype(np.float32)))
    y = M.m2_blocky_monarch_conv_fwd(plan, fac, dev(x.astype(np.float32), tdt), kf)
    torch.cuda.synchronize()
    assert plan.device_status() == 0 and plan.last_kernel() == "blocky_monarch_conv"
    mL, mR = O.causal_coefficient_masks(b) if masked else (1.0, 1.0)
    st = {}
    f = O.blocky_monarch_conv(Lt * mL, Rt * mR, k[None], x, stages=st)
    if masked:
        assert np.abs(f.imag).max() <= 1e-8 * np.abs(f.real).max()
    tol = TOL_BF16 if dtype == M.M2_BF16 else TOL_FP32
    # factors and the kernel spectrum against the oracle's, as complex arrays
    per = N * b
    fv = fac.view(torch.float32).cpu().numpy().astype(np.float64).reshape(4, per, 2)
    got = [(fv[i, :, 0] + 1j * fv[i, :, 1]).reshape(b, b, b) for i in range(4)]
    # (the device inverts its fp32-rounded factors in fp64, the oracle the fp64 factors: the inverses differ by cond x 6e-8)
    for name, g, want, ftol in zip(("L", "R", "Linv", "Rinv"), got, (st["L"], st["R"], st["Linv"], st["Rinv"]), (1e-6, 1e-6, 2e-5, 2e-5)):
        assert np.linalg.norm(g - want) <= ftol * np.linalg.norm(want), name
    kfg = host(kf)
    kfg = kfg[..., 0] + 1j * kfg[..., 1]
    want_kf = st["k_f"][0].reshape(H, b, b).transpose(0, 2, 1).reshape(H, N)      # natural [k2][k1] -> plan order [k1][k2]
    assert np.linalg.norm(kfg - want_kf) <= 1e-5 * np.linalg.norm(want_kf)
    check(host(y), f.real, tol, f"blocky Monarch conv b={b} n={n}")
    if masked:     # causality on the device: changing x[t0:] leaves y[:t0] as it was, up to rounding
        t0 = n // 3 + 1
        x2 = x.copy()
        x2[..., t0:] = rnd(synth.normal(synth.stream_id(18, 4), (Bn, H, n - t0)))
        y2 = M.m2_blocky_monarch_conv_fwd(plan, fac, dev(x2.astype(np.float32), tdt), kf)
        torch.cuda.synchronize()
        d = (host(y2) - host(y))[..., :t0]
        assert np.abs(d).max() <= tol * np.abs(host(y)).max()
    if noise == 0.0:   # the DFT's coefficients: the plain causal convolution
        check(host(y), O.direct_causal_conv(k[None], x), tol, "blocky Monarch with the DFT's coefficients")
    plan.close()


def test_blocky_monarch_singular_block_and_bad_arguments():
    b = 8
    N = b * b
    plan = M.Plan((b, b), dtype=M.M2_FP32, device=0)
    Lt, Rt = _blocky_coefficients(b, 5, 0.2)
    Rt[3 * b:4 * b] = 0.0                                    # block 3 of R becomes the zero matrix
    fac = M.m2_blocky_monarch(plan, dev(Lt.astype(np.float32)), dev(Rt.astype(np.float32)), causal_mask=True)
    torch.cuda.synchronize()
    assert plan.device_status() == M.M2_ERR_SINGULAR and plan.device_status() == 0
    lib, s = M.lib(), torch.cuda.current_stream().cuda_stream
    rect = M.Plan((8, 4), dtype=M.M2_FP32, device=0)
    assert lib.m2_blocky_factors_bytes(rect.handle) == -1
    x = torch.zeros((1, 1, 40), dtype=torch.float32, device="cuda")
    kf = torch.zeros((1, N, 2), dtype=torch.float32, device="cuda")
    assert lib.m2_blocky_monarch(rect.handle, x.data_ptr(), x.data_ptr(), 1, fac.data_ptr(), s) == M.M2_ERR_UNSUPPORTED
    assert lib.m2_blocky_monarch_conv_fwd(plan.handle, fac.data_ptr(), x.data_ptr(), kf.data_ptr(), x.data_ptr(), 1, 1, 40, s) == M.M2_ERR_INVALID_ARG   # 2 n > N
    assert lib.m2_blocky_monarch_conv_fwd(plan.handle, fac.data_ptr(), None, kf.data_ptr(), x.data_ptr(), 1, 1, 32, s) == M.M2_ERR_INVALID_ARG
    assert lib.m2_blocky_monarch_conv_fwd(plan.handle, fac.data_ptr(), None, None, None, 0, 1, 32, s) == M.M2_OK      # empty batch
    torch.cuda.synchronize()
    plan.close()
    rect.close()


# ---- edge cases, error paths, determinism -------------------------------------------------------------

def test_empty_batches_and_error_codes():
    plan = M.Plan((32, 16), dtype=M.M2_BF16, device=0)
    k = dev(synth.decay_kernel(2, 2, 512, 0.005, 22.6))
    kf = M.m2_kernel_spectrum(plan, k)
    x0 = torch.empty((0, 2, 512), dtype=torch.bfloat16, device="cuda")
    assert M.m2_monarch_conv_fwd(plan, x0, kf, M.M2_CIRCULAR).shape == (0, 2, 512)
    lib = M.lib()
    x = torch.zeros((1, 2, 512), dtype=torch.bfloat16, device="cuda")
    y = torch.empty_like(x)
    s = torch.cuda.current_stream().cuda_stream
    # causal needs n <= N/2; circular needs n == N
    assert lib.m2_monarch_conv_fwd(plan.handle, x.data_ptr(), kf.data_ptr(), y.data_ptr(), 1, 2, 512, M.M2_CAUSAL, s) == M.M2_ERR_INVALID_ARG
    assert lib.m2_monarch_conv_fwd(plan.handle, x.data_ptr(), kf.data_ptr(), y.data_ptr(), 1, 2, 256, M.M2_CIRCULAR, s) == M.M2_ERR_INVALID_ARG
    assert lib.m2_monarch_conv_fwd(plan.handle, x.data_ptr() + 2, kf.data_ptr(), y.data_ptr(), 1, 2, 256, M.M2_CAUSAL, s) == M.M2_ERR_ALIGNMENT
    assert lib.m2_monarch_conv_fwd(plan.handle, x.data_ptr(), kf.data_ptr(), y.data_ptr(), 1, 2, 256, 9, s) == M.M2_ERR_INVALID_ARG
    assert lib.m2_monarch_matmul(plan.handle, x.data_ptr(), x.data_ptr(), x.data_ptr(), None, 1, None, 0, s) == M.M2_ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert plan.device_status() == 0
    plan.close()


def test_error_codes_of_the_operator_and_gradient_calls():
    """Bad arguments are refused on the host, before anything is launched."""
    lib = M.lib()
    s = torch.cuda.current_stream().cuda_stream
    plan = M.Plan((64, 64), dtype=M.M2_BF16, device=0)
    plan3 = M.Plan((4, 4, 4), dtype=M.M2_BF16, device=0)
    T, N = 4, 4096
    X = torch.zeros((T, N), dtype=torch.bfloat16, device="cuda")
    W = torch.zeros((64, 64, 64), dtype=torch.bfloat16, device="cuda")
    Y = torch.empty_like(X)
    dW = torch.empty((64, 64, 64), dtype=torch.float32, device="cuda")
    ws = torch.empty(1 << 20, dtype=torch.uint8, device="cuda")
    p, w, y = X.data_ptr(), W.data_ptr(), Y.data_ptr()
    # m2_monarch_mix: unknown activation, missing kernel, Hk < 1, misaligned kernel, order-3 plan
    assert lib.m2_monarch_mix(plan.handle, p, p, 1, 7, w, w, w, w, y, T, ws.data_ptr(), ws.numel(), s) == M.M2_ERR_INVALID_ARG
    assert lib.m2_monarch_mix(plan.handle, p, None, 1, 0, w, w, w, w, y, T, ws.data_ptr(), ws.numel(), s) == M.M2_ERR_INVALID_ARG
    assert lib.m2_monarch_mix(plan.handle, p, p, 0, 0, w, w, w, w, y, T, ws.data_ptr(), ws.numel(), s) == M.M2_ERR_INVALID_ARG
    assert lib.m2_monarch_mix(plan.handle, p, p + 2, 1, 0, w, w, w, w, y, T, ws.data_ptr(), ws.numel(), s) == M.M2_ERR_ALIGNMENT
    assert lib.m2_monarch_mix(plan3.handle, p, p, 1, 0, w, w, w, w, y, T, ws.data_ptr(), ws.numel(), s) == M.M2_ERR_UNSUPPORTED
    # m2_monarch_cols: workspace too small, missing workspace, unknown activation
    assert lib.m2_monarch_cols(plan.handle, p, w, w, None, 0, y, 1, 4, ws.data_ptr(), 16, s) == M.M2_ERR_INVALID_ARG
    assert lib.m2_monarch_cols(plan.handle, p, w, w, None, 0, y, 1, 4, None, 0, s) == M.M2_ERR_INVALID_ARG
    assert lib.m2_monarch_cols(plan.handle, p, w, w, None, 5, y, 1, 4, ws.data_ptr(), ws.numel(), s) == M.M2_ERR_INVALID_ARG
    assert lib.m2_monarch_cols(plan.handle, p, w, w, None, 0, y, 0, 4, None, 0, s) == M.M2_OK          # empty batch
    # m2_monarch_matmul_bwd_weights: workspace too small, missing gradient buffers
    assert lib.m2_monarch_matmul_bwd_weights(plan.handle, p, p, w, w, dW.data_ptr(), dW.data_ptr(), T, ws.data_ptr(), 16, s) == M.M2_ERR_INVALID_ARG
    assert lib.m2_monarch_matmul_bwd_weights(plan.handle, p, p, w, w, None, dW.data_ptr(), T, ws.data_ptr(), ws.numel(), s) == M.M2_ERR_INVALID_ARG
    assert lib.m2_matmul_bwd_workspace_bytes(plan3.handle, T) == -1
    # m2_blocks_transpose: non-positive block shape
    assert lib.m2_blocks_transpose(plan.handle, w, dW.data_ptr(), 64, 0, 64, s) == M.M2_ERR_INVALID_ARG
    # m2_layer_fwd: plans of different dtypes, scratch too small
    pf = M.Plan((8, 8), dtype=M.M2_FP32, device=0)
    pb = M.Plan((8, 8), dtype=M.M2_BF16, device=0)
    fac = (ctypes.c_void_p * 8)(*([w] * 8))
    g = torch.ones(64, dtype=torch.float32, device="cuda")
    assert lib.m2_layer_fwd(pb.handle, pf.handle, p, fac, p, p, g.data_ptr(), g.data_ptr(), 1e-5, y, 1, ws.data_ptr(), ws.numel(), None, 0, s) == M.M2_ERR_INVALID_ARG
    assert lib.m2_layer_fwd(pb.handle, pb.handle, p, fac, p, p, g.data_ptr(), g.data_ptr(), 1e-5, y, 1, ws.data_ptr(), 64, None, 0, s) == M.M2_ERR_INVALID_ARG
    torch.cuda.synchronize()
    for q in (plan, plan3, pf, pb):
        assert q.device_status() == 0
        q.close()


def test_runs_are_bit_identical_and_stay_in_bounds():
    c = synth.config2(B=8, H=16)
    plan = M.Plan(c["dims"], dtype=M.M2_BF16, device=0)
    kf = M.m2_kernel_spectrum(plan, dev(c["k"]))
    x = dev(c["x"], torch.bfloat16)
    # canary-padded output: the kernel must not write outside [B, H, n]
    pad = 4096
    buf = torch.full((x.numel() + 2 * pad,), 7.0, dtype=torch.bfloat16, device="cuda")
    y = buf[pad:pad + x.numel()].view_as(x)
    M.m2_monarch_conv_fwd(plan, x, kf, M.M2_CIRCULAR, y=y)
    y1 = y.clone()
    M.m2_monarch_conv_fwd(plan, x, kf, M.M2_CIRCULAR, y=y)
    torch.cuda.synchronize()
    assert torch.equal(y1, y)
    assert bool((buf[:pad] == 7.0).all()) and bool((buf[pad + x.numel():] == 7.0).all())
    plan.close()


def test_new_kernels_are_bit_identical_and_stay_in_bounds():
    """Column-layout Monarch, weight gradients and kernel gradient: two runs give the same bits; nothing is written outside the outputs."""
    torch.manual_seed(7)
    b, d, Bt = 128, 192, 2
    N = b * b
    plan = M.Plan((b, b), dtype=M.M2_BF16, device=0)
    L = (torch.randn(b, b, b, device="cuda") / b ** 0.5).to(torch.bfloat16)
    R = (torch.randn(b, b, b, device="cuda") / b ** 0.5).to(torch.bfloat16)
    X = torch.randn(Bt, N, d, device="cuda").to(torch.bfloat16)
    K = torch.randn(N, d, device="cuda").to(torch.bfloat16)
    pad = 8192
    buf = torch.full((X.numel() + 2 * pad,), 7.0, dtype=torch.bfloat16, device="cuda")
    Y = buf[pad:pad + X.numel()].view_as(X)
    M.m2_monarch_cols(plan, X, L, R, K, M.M2_ACT_RELU, Y=Y)
    Y1 = Y.clone()
    M.m2_monarch_cols(plan, X, L, R, K, M.M2_ACT_RELU, Y=Y)
    torch.cuda.synchronize()
    assert plan.device_status() == 0 and torch.equal(Y1, Y)
    assert bool((buf[:pad] == 7.0).all()) and bool((buf[pad + X.numel():] == 7.0).all())
    plan.close()
    plan = M.Plan((64, 64), dtype=M.M2_BF16, device=0)
    T = 700
    X = torch.randn(T, 4096, device="cuda").to(torch.bfloat16)
    G = torch.randn(T, 4096, device="cuda").to(torch.bfloat16)
    L = (torch.randn(64, 64, 64, device="cuda") / 8).to(torch.bfloat16)
    R = (torch.randn(64, 64, 64, device="cuda") / 8).to(torch.bfloat16)
    a = M.m2_monarch_matmul_bwd_weights(plan, X, G, L, R)
    b2 = M.m2_monarch_matmul_bwd_weights(plan, X, G, L, R)
    torch.cuda.synchronize()
    assert plan.device_status() == 0 and torch.equal(a[0], b2[0]) and torch.equal(a[1], b2[1])
    plan.close()
    plan = M.Plan((32, 16), dtype=M.M2_BF16, device=0)
    x = torch.randn(24, 40, 512, device="cuda").to(torch.bfloat16)
    g = torch.randn(24, 40, 512, device="cuda").to(torch.bfloat16)
    d1 = M.m2_monarch_conv_bwd_kernel(plan, x, g, M.M2_CIRCULAR)
    d2 = M.m2_monarch_conv_bwd_kernel(plan, x, g, M.M2_CIRCULAR)
    torch.cuda.synchronize()
    assert plan.device_status() == 0 and plan.last_kernel() == "conv_wgrad_umma_o2_512" and torch.equal(d1, d2)
    plan.close()


def test_bounded_wait_runs_out_and_the_plan_recovers():
    """A device-side wait that runs out: the row-pair kernel is launched in its self-test mode (no copy issued, a few polls per
    wait), must come back by itself through its abort path with nothing in flight, report M2_ERR_TIMEOUT in the plan's status
    word and leave y alone; the next ordinary calls on the same plan are correct and clean."""
    c = synth.config2(B=19, H=40)     # more pipelines than one CTA holds, a ragged last batch group
    plan = M.Plan(c["dims"], dtype=M.M2_BF16, device=0)
    kf = M.m2_kernel_spectrum(plan, dev(c["k"]))
    x = dev(c["x"], torch.bfloat16)
    y = torch.full_like(x, 7.0)
    M.m2_selftest_bounded_wait(plan, x, kf, M.M2_CIRCULAR, y)
    torch.cuda.synchronize()
    assert plan.device_status() == M.M2_ERR_TIMEOUT
    assert plan.device_status() == 0                      # reading the word resets it
    assert bool((y == 7.0).all())                         # nothing was written
    ref = O.monarch_conv(c["k"].astype(np.float64)[None], c["x"].astype(np.float64), c["dims"], causal=False)
    for _ in range(2):                                    # the scheduler words were reset: two ordinary calls in a row
        M.m2_monarch_conv_fwd(plan, x, kf, M.M2_CIRCULAR, y=y)
        torch.cuda.synchronize()
        assert plan.device_status() == 0 and plan.last_kernel() == "conv_umma_o2_512_pairs"
        check(host(y), ref, TOL_BF16, "after the timed-out launch")
    # up to 8 batch rows there is no row-pair kernel to test
    lib, s = M.lib(), torch.cuda.current_stream().cuda_stream
    assert lib.m2_selftest_bounded_wait(plan.handle, x.data_ptr(), kf.data_ptr(), y.data_ptr(), 8, 40, 512, M.M2_CIRCULAR, s) == M.M2_ERR_UNSUPPORTED
    plan.close()


def test_bounded_wait_runs_out_in_the_matmul_and_the_plan_recovers():
    """The same for the tensor-core matmul: both passes are launched in the mode where the issuing threads give the tensor
    core nothing and every wait for it runs out after a few polls; the loading, draining and issuing warps of every CTA
    must leave through their abort paths, report M2_ERR_TIMEOUT and write neither Y nor the workspace; ordinary calls on
    the same plan are correct afterwards."""
    c = synth.config3(T=5000, b=64)                       # more items than CTAs: every CTA has a next tile in flight when it gives up
    plan = M.Plan((64, 64), dtype=M.M2_BF16, device=0)
    X, L, R = dev(c["X"], torch.bfloat16), dev(c["L"], torch.bfloat16), dev(c["R"], torch.bfloat16)
    ws = M.m2_matmul_workspace(plan, 5000)
    ws.fill_(3)
    Y = torch.full_like(X, 7.0)
    M.m2_selftest_bounded_wait_matmul(plan, X, L, R, Y, ws)
    torch.cuda.synchronize()
    assert plan.device_status() == M.M2_ERR_TIMEOUT
    assert plan.device_status() == 0                      # reading the word resets it
    assert bool((Y == 7.0).all()) and bool((ws == 3).all())
    ref = O.monarch_apply(c["L"].astype(np.float64), c["R"].astype(np.float64), c["X"].astype(np.float64))
    for _ in range(2):
        M.m2_monarch_matmul(plan, X, L, R, Y, ws=ws)
        torch.cuda.synchronize()
        assert plan.device_status() == 0 and plan.last_kernel() == "matmul_umma_64x64"
        check(host(Y), ref, TOL_BF16, "after the timed-out launches")
    # no workspace, no self-test
    lib, st = M.lib(), torch.cuda.current_stream().cuda_stream
    assert lib.m2_selftest_bounded_wait_matmul(plan.handle, X.data_ptr(), L.data_ptr(), R.data_ptr(), Y.data_ptr(), 5000, None, 0, st) == M.M2_ERR_UNSUPPORTED
    plan.close()


def test_host_buffer_entry_points():
    c = synth.config2(B=2, H=8)
    plan = M.Plan(c["dims"], dtype=M.M2_BF16, device=0)
    kf = M.m2_kernel_spectrum(plan, dev(c["k"]))
    xh = torch.from_numpy(c["x"]).to(torch.bfloat16).pin_memory()
    yh = torch.empty_like(xh).pin_memory()
    xs, ys = torch.empty_like(xh, device="cuda"), torch.empty_like(xh, device="cuda")
    M.m2_monarch_conv_fwd_host(plan, xh, kf, yh, xs, ys, M.M2_CIRCULAR)
    torch.cuda.synchronize()
    yd = M.m2_monarch_conv_fwd(plan, xs, kf, M.M2_CIRCULAR)
    torch.cuda.synchronize()
    assert torch.equal(yh, yd.cpu())
    plan.close()
    c3 = synth.config3(T=9, b=16)
    plan = M.Plan((16, 16), dtype=M.M2_BF16, device=0)
    Xh = torch.from_numpy(c3["X"]).to(torch.bfloat16).pin_memory()
    Yh = torch.empty_like(Xh).pin_memory()
    L, R = dev(c3["L"], torch.bfloat16), dev(c3["R"], torch.bfloat16)
    Xs, Ys = torch.empty_like(Xh, device="cuda"), torch.empty_like(Xh, device="cuda")
    M.m2_monarch_matmul_host(plan, Xh, L, R, Yh, Xs, Ys)
    torch.cuda.synchronize()
    ref = O.monarch_apply(c3["L"].astype(np.float64), c3["R"].astype(np.float64), c3["X"].astype(np.float64))
    check(host(Yh), ref, TOL_BF16, "matmul host entry")
    plan.close()


def test_back_to_back_calls_see_each_other():
    """The tensor-core kernels are launched so that a kernel's CTAs may start while the previous kernel's
    last CTAs still run; a call that consumes the previous call's output (no synchronisation in between,
    output buffers reused in place) must still give what the synchronised sequence gives."""
    c = synth.config2(B=32, H=96)
    plan = M.Plan(c["dims"], dtype=M.M2_BF16, device=0)
    kf = M.m2_kernel_spectrum(plan, dev(c["k"]))
    x = dev(c["x"], torch.bfloat16)
    ref = x
    for _ in range(4):   # synchronised chain
        ref = M.m2_monarch_conv_fwd(plan, ref, kf, M.M2_CIRCULAR)
        torch.cuda.synchronize()
    a, b = torch.empty_like(x), torch.empty_like(x)
    M.m2_monarch_conv_fwd(plan, x, kf, M.M2_CIRCULAR, y=a)       # unsynchronised chain, ping-pong buffers
    M.m2_monarch_conv_fwd(plan, a, kf, M.M2_CIRCULAR, y=b)
    M.m2_monarch_conv_fwd(plan, b, kf, M.M2_CIRCULAR, y=a)
    M.m2_monarch_conv_fwd(plan, a, kf, M.M2_CIRCULAR, y=b)
    torch.cuda.synchronize()
    assert plan.device_status() == 0
    assert torch.equal(b, ref)
    plan.close()

    c3 = synth.config3(T=2048, b=64)
    plan = M.Plan((64, 64), dtype=M.M2_BF16, device=0)
    X, L, R = dev(c3["X"], torch.bfloat16), dev(c3["L"], torch.bfloat16), dev(c3["R"], torch.bfloat16)
    ws = M.m2_matmul_workspace(plan, X.shape[0])
    ref = X
    for _ in range(3):
        ref = M.m2_monarch_matmul(plan, ref, L, R, ws=ws)
        torch.cuda.synchronize()
    A, Bb = torch.empty_like(X), torch.empty_like(X)
    M.m2_monarch_matmul(plan, X, L, R, A, ws=ws)
    M.m2_monarch_matmul(plan, A, L, R, Bb, ws=ws)
    M.m2_monarch_matmul(plan, Bb, L, R, A, ws=ws)
    torch.cuda.synchronize()
    assert plan.device_status() == 0 and plan.last_kernel() == "matmul_umma_64x64"
    assert torch.equal(A, ref)
    plan.close()
