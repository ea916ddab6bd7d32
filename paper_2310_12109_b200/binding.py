"""ctypes binding of libm2.so: argument marshalling only.

Function names mirror the C ABI (include/m2.h).  Tensors are torch CUDA tensors used purely as
device memory; the current torch stream is passed as the cudaStream_t.  There is no fallback: if
the shared library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libm2.so")

M2_FP32, M2_BF16 = 0, 1
M2_CAUSAL, M2_CIRCULAR = 0, 1
M2_STATIC_SCRATCH_BYTES = 8 * 1024 * 1024
M2_TABLE_PERM, M2_TABLE_PERM_INV, M2_TABLE_DIGIT_REV, M2_TABLE_TW_EXP = 0, 1, 2, 16
M2_OK, M2_ERR_INVALID_ARG, M2_ERR_UNSUPPORTED, M2_ERR_ALIGNMENT, M2_ERR_CUDA, M2_ERR_TIMEOUT, M2_ERR_NO_DEVICE, M2_ERR_SINGULAR = range(8)

# every symbol include/m2.h declares: (name, restype, argtypes)
_vp, _i32, _i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
SIGNATURES = {
    "m2_plan_create": (_i32, [ctypes.POINTER(_vp), _i64, _i32, ctypes.POINTER(_i32), _i32, _i32, _i32]),
    "m2_plan_destroy": (_i32, [_vp]),
    "m2_plan_get_table": (_i32, [_vp, _i32, ctypes.POINTER(_i32), _i64]),
    "m2_spectrum_bytes": (_i64, [_vp, _i64]),
    "m2_kernel_spectrum": (_i32, [_vp, _vp, _i64, _i64, _vp, _vp]),
    "m2_spectrum_to_natural": (_i32, [_vp, _vp, _i64, _vp, _vp]),
    "m2_monarch_conv_fwd": (_i32, [_vp, _vp, _vp, _vp, _i64, _i64, _i64, _i32, _vp]),
    "m2_monarch_conv_fwd_grouped": (_i32, [_vp, _vp, _vp, _vp, _i64, _i64, _i64, _i32, _i64, _vp]),
    "m2_monarch_conv_fwd_host": (_i32, [_vp, _vp, _vp, _vp, _vp, _vp, _i64, _i64, _i64, _i32, _vp]),
    "m2_matmul_workspace_bytes": (_i64, [_vp, _i64]),
    "m2_spectrum_conjugate": (_i32, [_vp, _vp, _i64, _vp, _vp]),
    "m2_matmul_bwd_workspace_bytes": (_i64, [_vp, _i64]),
    "m2_monarch_matmul_bwd_weights": (_i32, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _i64, _vp, _i64, _vp]),
    "m2_monarch_mix": (_i32, [_vp, _vp, _vp, _i64, _i32, _vp, _vp, _vp, _vp, _vp, _i64, _vp, _i64, _vp]),
    "m2_layer_scratch_bytes": (_i64, [_vp, _vp, _i64]),
    "m2_layer_fwd": (_i32, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, ctypes.c_float, _vp, _i64, _vp, _i64, _vp, _i64, _vp]),
    "m2_monarch_cols": (_i32, [_vp, _vp, _vp, _vp, _vp, _i32, _vp, _i64, _i64, _vp, _i64, _vp]),
    "m2_bert_mixer_scratch_bytes": (_i64, [_vp, _i64, _i64]),
    "m2_bert_mixer_fwd": (_i32, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _i64, _i64, _vp, _i64, _vp]),
    "m2_hyena_scratch_bytes": (_i64, [_vp, _i64, _i64, _i64, _i64]),
    "m2_hyena_heads_fwd": (_i32, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i64, _i64, _i64, _i64, _vp, _i64, _vp]),
    "m2_blocks_transpose": (_i32, [_vp, _vp, _vp, _i64, _i64, _i64, _vp]),
    "m2_conv_bwd_workspace_bytes": (_i64, [_vp, _i64, _i64]),
    "m2_monarch_conv_bwd_kernel": (_i32, [_vp, _vp, _vp, _vp, _i64, _i64, _i64, _i32, _vp, _i64, _vp]),
    "m2_monarch_matmul": (_i32, [_vp, _vp, _vp, _vp, _vp, _i64, _vp, _i64, _vp]),
    "m2_monarch_matmul_host": (_i32, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _i64, _vp, _i64, _vp]),
    "m2_block_fwd": (_i32, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i64, _i64, _i64, _i32, _i32, _vp]),
    "m2_block_z_channel_first": (_i32, [_vp, _i64, _i64, _i32, _i32]),
    "m2_block_fwd_static": (_i32, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _i64, _i64, _i64, _i32, _i32, _vp]),
    "m2_blocky_factors_bytes": (_i64, [_vp]),
    "m2_blocky_monarch": (_i32, [_vp, _vp, _vp, _i32, _vp, _vp]),
    "m2_blocky_kernel_spectrum": (_i32, [_vp, _vp, _vp, _i64, _i64, _vp, _vp]),
    "m2_blocky_monarch_conv_fwd": (_i32, [_vp, _vp, _vp, _vp, _vp, _i64, _i64, _i64, _vp]),
    "m2_selftest_bounded_wait": (_i32, [_vp, _vp, _vp, _vp, _i64, _i64, _i64, _i32, _vp]),
    "m2_selftest_bounded_wait_matmul": (_i32, [_vp, _vp, _vp, _vp, _vp, _i64, _vp, _i64, _vp]),
    "m2_monarch_apply_order_p": (_i32, [_vp, _vp, ctypes.POINTER(ctypes.c_void_p), _vp, _i64, _vp]),
    "m2_status_string": (ctypes.c_char_p, [_i32]),
    "m2_last_device_status": (_i32, [_vp, ctypes.POINTER(_i32)]),
    "m2_last_kernel_name": (ctypes.c_char_p, [_vp]),
    "m2_launch_count": (_i64, [_vp]),
}

_lib = None


class M2Error(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().m2_status_string(status).decode()
        super().__init__(f"{where}: {msg} (status {status})")


def lib() -> ctypes.CDLL:
    """Loads libm2.so (built by paper_2310_12109_b200.build); raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} not built: run `python -m paper_2310_12109_b200.build`")
        l = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(l, name)
            fn.restype = res
            fn.argtypes = args
        _lib = l
    return _lib


def _check(status: int, where: str) -> None:
    if status != M2_OK:
        raise M2Error(status, where)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t) -> int:
    return 0 if t is None else t.data_ptr()


class Plan:
    """m2_plan_create / m2_plan_destroy."""

    def __init__(self, dims, dtype: int = M2_BF16, sign: int = +1, device: int = 0):
        self.dims = tuple(int(d) for d in dims)
        self.N = 1
        for d in self.dims:
            self.N *= d
        self.dtype, self.sign, self.device = dtype, sign, device
        self.handle = _vp()
        arr = (_i32 * len(self.dims))(*self.dims)
        _check(lib().m2_plan_create(ctypes.byref(self.handle), self.N, len(self.dims), arr, dtype, sign, device),
               "m2_plan_create")

    def close(self):
        if self.handle:
            lib().m2_plan_destroy(self.handle)
            self.handle = _vp()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def torch_dtype(self):
        return torch.bfloat16 if self.dtype == M2_BF16 else torch.float32

    def get_table(self, which: int):
        import numpy as np
        out = (_i32 * self.N)()
        _check(lib().m2_plan_get_table(self.handle, which, out, self.N), "m2_plan_get_table")
        return np.frombuffer(out, dtype=np.int32).copy()

    def last_kernel(self) -> str:
        return lib().m2_last_kernel_name(self.handle).decode()

    def launch_count(self) -> int:
        return int(lib().m2_launch_count(self.handle))

    def device_status(self) -> int:
        out = _i32(0)
        _check(lib().m2_last_device_status(self.handle, ctypes.byref(out)), "m2_last_device_status")
        return out.value


def m2_spectrum_bytes(plan: Plan, H: int) -> int:
    return int(lib().m2_spectrum_bytes(plan.handle, H))


def m2_kernel_spectrum(plan: Plan, k: torch.Tensor, kf: torch.Tensor | None = None) -> torch.Tensor:
    """k: [H, n] float32 CUDA.  Returns the opaque spectrum buffer (uint8)."""
    assert k.is_cuda and k.dtype == torch.float32 and k.is_contiguous() and k.dim() == 2
    H, n = k.shape
    if kf is None:
        kf = torch.empty(max(m2_spectrum_bytes(plan, H), 16), dtype=torch.uint8, device=k.device)
    _check(lib().m2_kernel_spectrum(plan.handle, _ptr(k), H, n, _ptr(kf), _stream()), "m2_kernel_spectrum")
    return kf


def m2_spectrum_conjugate(plan: Plan, kf: torch.Tensor, H: int, out: torch.Tensor | None = None) -> torch.Tensor:
    """conj(k_f) in every layout of the buffer: the spectrum with which m2_monarch_conv_fwd computes the gradient
    with respect to its input."""
    if out is None:
        out = torch.empty_like(kf)
    _check(lib().m2_spectrum_conjugate(plan.handle, _ptr(kf), H, _ptr(out), _stream()), "m2_spectrum_conjugate")
    return out


def m2_monarch_conv_bwd_kernel(plan: Plan, x: torch.Tensor, g: torch.Tensor, mode: int, ws: torch.Tensor | None = None,
                               use_workspace: bool = True) -> torch.Tensor:
    """dk[H, n] (float32): gradient of sum_b <conv(k, x_b), g_b> with respect to the kernel; x, g: [B, H, n].
    use_workspace=False selects the fp32 CUDA-core kernel even where a tensor-core one exists."""
    assert x.is_cuda and g.is_cuda and x.dtype == plan.torch_dtype and g.dtype == plan.torch_dtype
    assert x.is_contiguous() and g.is_contiguous() and x.shape == g.shape and x.dim() == 3
    B, H, n = x.shape
    dk = torch.empty((H, n), dtype=torch.float32, device=x.device)
    if ws is None and use_workspace:
        need = int(lib().m2_conv_bwd_workspace_bytes(plan.handle, B, H))
        ws = torch.empty(need, dtype=torch.uint8, device=x.device) if need > 0 else None
    _check(lib().m2_monarch_conv_bwd_kernel(plan.handle, _ptr(x), _ptr(g), _ptr(dk), B, H, n, mode, _ptr(ws),
                                            0 if ws is None else ws.numel(), _stream()), "m2_monarch_conv_bwd_kernel")
    return dk


def m2_spectrum_to_natural(plan: Plan, kf: torch.Tensor, H: int) -> torch.Tensor:
    out = torch.empty((H, plan.N, 2), dtype=torch.float32, device=kf.device)
    _check(lib().m2_spectrum_to_natural(plan.handle, _ptr(kf), H, _ptr(out), _stream()), "m2_spectrum_to_natural")
    return out


def m2_monarch_conv_fwd(plan: Plan, x: torch.Tensor, kf: torch.Tensor, mode: int, y: torch.Tensor | None = None):
    """x: [B, H, n] CUDA tensor of the plan dtype; returns y of the same shape."""
    assert x.is_cuda and x.dtype == plan.torch_dtype and x.is_contiguous() and x.dim() == 3
    B, H, n = x.shape
    if y is None:
        y = torch.empty_like(x)
    _check(lib().m2_monarch_conv_fwd(plan.handle, _ptr(x), _ptr(kf), _ptr(y), B, H, n, mode, _stream()),
           "m2_monarch_conv_fwd")
    return y


def m2_monarch_conv_fwd_grouped(plan: Plan, x: torch.Tensor, kf: torch.Tensor, mode: int, kf_group: int, y: torch.Tensor | None = None):
    """Like m2_monarch_conv_fwd with channel h using spectrum row h // kf_group (kf computed for H // kf_group kernels)."""
    assert x.is_cuda and x.dtype == plan.torch_dtype and x.is_contiguous() and x.dim() == 3
    B, H, n = x.shape
    if y is None:
        y = torch.empty_like(x)
    _check(lib().m2_monarch_conv_fwd_grouped(plan.handle, _ptr(x), _ptr(kf), _ptr(y), B, H, n, mode, kf_group, _stream()),
           "m2_monarch_conv_fwd_grouped")
    return y


def m2_selftest_bounded_wait(plan: Plan, x: torch.Tensor, kf: torch.Tensor, mode: int, y: torch.Tensor):
    """Launches the row-pair convolution kernel so that its first bounded wait runs out; y is left untouched and the
    plan's device status reads M2_ERR_TIMEOUT afterwards."""
    assert x.is_cuda and x.dtype == plan.torch_dtype and x.is_contiguous() and x.dim() == 3
    B, H, n = x.shape
    _check(lib().m2_selftest_bounded_wait(plan.handle, _ptr(x), _ptr(kf), _ptr(y), B, H, n, mode, _stream()),
           "m2_selftest_bounded_wait")


def m2_monarch_conv_fwd_host(plan: Plan, x_host: torch.Tensor, kf: torch.Tensor, y_host: torch.Tensor,
                             x_scratch: torch.Tensor, y_scratch: torch.Tensor, mode: int):
    """x_host / y_host: pinned CPU tensors [B, H, n]; scratch: CUDA tensors of the same shape."""
    assert not x_host.is_cuda and not y_host.is_cuda and x_scratch.is_cuda and y_scratch.is_cuda
    B, H, n = x_host.shape
    _check(lib().m2_monarch_conv_fwd_host(plan.handle, _ptr(x_host), _ptr(kf), _ptr(y_host), _ptr(x_scratch),
                                          _ptr(y_scratch), B, H, n, mode, _stream()), "m2_monarch_conv_fwd_host")
    return y_host


def m2_matmul_workspace(plan: Plan, T: int, device=None):
    """Device workspace for m2_monarch_matmul (None if the plan's kernels need none)."""
    nbytes = int(lib().m2_matmul_workspace_bytes(plan.handle, T))
    if nbytes <= 0:
        return None
    return torch.empty(nbytes, dtype=torch.uint8, device=device if device is not None else f"cuda:{plan.device}")


def m2_monarch_matmul(plan: Plan, X: torch.Tensor, L: torch.Tensor, R: torch.Tensor, Y: torch.Tensor | None = None,
                      ws: torch.Tensor | None = None):
    """X: [T, N]; L: [N1, N2, N2]; R: [N2, N1, N1]; all CUDA, plan dtype.  ws: m2_matmul_workspace(plan, T)."""
    for t in (X, L, R):
        assert t.is_cuda and t.dtype == plan.torch_dtype and t.is_contiguous()
    N1, N2 = plan.dims
    assert X.dim() == 2 and X.shape[1] == plan.N and tuple(L.shape) == (N1, N2, N2) and tuple(R.shape) == (N2, N1, N1)
    if Y is None:
        Y = torch.empty_like(X)
    if ws is None:
        ws = m2_matmul_workspace(plan, X.shape[0], X.device)
    _check(lib().m2_monarch_matmul(plan.handle, _ptr(X), _ptr(L), _ptr(R), _ptr(Y), X.shape[0], _ptr(ws),
                                   0 if ws is None else ws.numel(), _stream()), "m2_monarch_matmul")
    return Y


def m2_monarch_apply_order_p(plan: Plan, X: torch.Tensor, W, Y: torch.Tensor | None = None) -> torch.Tensor:
    """Order-p product in the direct form; W: list of p tensors, W[a] of shape [N / N_a, N_a, N_a] (plan dtype)."""
    assert len(W) == len(plan.dims)
    for t in [X] + list(W):
        assert t.is_cuda and t.dtype == plan.torch_dtype and t.is_contiguous()
    for a, w in enumerate(W):
        assert tuple(w.shape) == (plan.N // plan.dims[a], plan.dims[a], plan.dims[a])
    assert X.dim() == 2 and X.shape[1] == plan.N
    if Y is None:
        Y = torch.empty_like(X)
    ptrs = (ctypes.c_void_p * len(W))(*[w.data_ptr() for w in W])
    _check(lib().m2_monarch_apply_order_p(plan.handle, _ptr(X), ptrs, _ptr(Y), X.shape[0], _stream()), "m2_monarch_apply_order_p")
    return Y


def m2_selftest_bounded_wait_matmul(plan: Plan, X: torch.Tensor, L: torch.Tensor, R: torch.Tensor, Y: torch.Tensor, ws: torch.Tensor):
    """The two matmul passes in the mode where every wait for the tensor core runs out; Y and ws are not written."""
    for t in (X, L, R, Y):
        assert t.is_cuda and t.dtype == plan.torch_dtype and t.is_contiguous()
    _check(lib().m2_selftest_bounded_wait_matmul(plan.handle, _ptr(X), _ptr(L), _ptr(R), _ptr(Y), X.shape[0], _ptr(ws), ws.numel(),
                                                 _stream()), "m2_selftest_bounded_wait_matmul")


M2_ACT_NONE, M2_ACT_RELU = 0, 1


def m2_monarch_mix(plan: Plan, X: torch.Tensor, K: torch.Tensor, La, Ra, Lb, Rb, act: int = M2_ACT_NONE, Y: torch.Tensor | None = None,
                   ws: torch.Tensor | None = None) -> torch.Tensor:
    """Y = M_b sigma(K (.) M_a X); X: [T, N], K: [Hk, N] (row t uses K[t % Hk]), all of the plan dtype."""
    for a in (X, K, La, Ra, Lb, Rb):
        assert a.is_cuda and a.dtype == plan.torch_dtype and a.is_contiguous()
    T = X.shape[0]
    if Y is None:
        Y = torch.empty_like(X)
    assert X.dim() == 2 and X.shape[1] == plan.N and K.dim() == 2 and K.shape[1] == plan.N
    if ws is None:
        ws = m2_matmul_workspace(plan, T, X.device)
    _check(lib().m2_monarch_mix(plan.handle, _ptr(X), _ptr(K), K.shape[0], act, _ptr(La), _ptr(Ra), _ptr(Lb), _ptr(Rb), _ptr(Y), T,
                                _ptr(ws), 0 if ws is None else ws.numel(), _stream()), "m2_monarch_mix")
    return Y


def m2_layer_fwd(plan_n: Plan, plan_d: Plan, x: torch.Tensor, factors, n_kernel: torch.Tensor, d_kernel: torch.Tensor,
                 gamma: torch.Tensor, beta: torch.Tensor, eps: float = 1e-5, ws: torch.Tensor | None = None) -> torch.Tensor:
    """The basic M2 layer on x [B, n, d]; factors = (L1, R1, L2, R2, L3, R3, L4, R4); gamma, beta fp32 [d]."""
    B, n, d = x.shape
    assert n == plan_n.N and d == plan_d.N and len(factors) == 8
    for a in (x, n_kernel, d_kernel, *factors):
        assert a.is_cuda and a.dtype == plan_n.torch_dtype and a.is_contiguous()
    for a in (gamma, beta):
        assert a.is_cuda and a.dtype == torch.float32 and a.is_contiguous() and a.numel() == d
    assert tuple(n_kernel.shape) == (d, n) and d_kernel.numel() == d
    y = torch.empty_like(x)
    sb = int(lib().m2_layer_scratch_bytes(plan_n.handle, plan_d.handle, B))
    scratch = torch.empty(max(sb, 16), dtype=torch.uint8, device=x.device)
    if ws is None:
        need = max(int(lib().m2_matmul_workspace_bytes(plan_n.handle, B * d)), int(lib().m2_matmul_workspace_bytes(plan_d.handle, B * n)))
        ws = torch.empty(need, dtype=torch.uint8, device=x.device) if need > 0 else None
    fp = (ctypes.c_void_p * 8)(*[f.data_ptr() for f in factors])
    _check(lib().m2_layer_fwd(plan_n.handle, plan_d.handle, _ptr(x), fp, _ptr(n_kernel), _ptr(d_kernel), _ptr(gamma), _ptr(beta), eps,
                              _ptr(y), B, _ptr(scratch), scratch.numel(), _ptr(ws), 0 if ws is None else ws.numel(), _stream()),
           "m2_layer_fwd")
    return y


def m2_monarch_cols(plan: Plan, X: torch.Tensor, L: torch.Tensor, R: torch.Tensor, K: torch.Tensor | None = None, act: int = M2_ACT_NONE,
                    Y: torch.Tensor | None = None, ws: torch.Tensor | None = None) -> torch.Tensor:
    """Y[bt] = sigma(K (.) M X[bt]) for X [Bt, N, d] (the columns are the vectors); K: [N, d] or None."""
    for a in (X, L, R) + ((K,) if K is not None else ()):
        assert a.is_cuda and a.dtype == plan.torch_dtype and a.is_contiguous()
    assert X.dim() == 3 and X.shape[1] == plan.N
    Bt, N, d = X.shape
    assert K is None or tuple(K.shape) == (N, d)
    if Y is None:
        Y = torch.empty_like(X)
    if ws is None:
        ws = torch.empty_like(X)
    _check(lib().m2_monarch_cols(plan.handle, _ptr(X), _ptr(L), _ptr(R), _ptr(K), act, _ptr(Y), Bt, d, _ptr(ws),
                                 ws.numel() * ws.element_size(), _stream()), "m2_monarch_cols")
    return Y


def m2_bert_mixer_fwd(plan: Plan, x: torch.Tensor, W, w_short, kf, kf_res, scratch: torch.Tensor | None = None,
                      y: torch.Tensor | None = None) -> torch.Tensor:
    """The gated bidirectional M2-BERT sequence mixer on x [B, n, d], n = plan.N; W = (W_q, W_k, W_v, W_o), each [d, d] stored
    outputs x inputs; w_short = three fp32 [d, 3] filters; kf, kf_res = m2_kernel_spectrum of the long and residual kernels."""
    B, n, d = x.shape
    assert n == plan.N and len(W) == 4 and len(w_short) == 3
    for a in (x, *W):
        assert a.is_cuda and a.dtype == plan.torch_dtype and a.is_contiguous()
    for a in w_short:
        assert a.is_cuda and a.dtype == torch.float32 and a.is_contiguous() and tuple(a.shape) == (d, 3)
    if y is None:
        y = torch.empty_like(x)
    if scratch is None:
        sb = int(lib().m2_bert_mixer_scratch_bytes(plan.handle, B, d))
        scratch = torch.empty(max(sb, 16), dtype=torch.uint8, device=x.device)
    wp = (ctypes.c_void_p * 4)(*[w.data_ptr() for w in W])
    sp = (ctypes.c_void_p * 3)(*[w.data_ptr() for w in w_short])
    _check(lib().m2_bert_mixer_fwd(plan.handle, _ptr(x), wp, sp, _ptr(kf), _ptr(kf_res), _ptr(y), B, d, _ptr(scratch), scratch.numel(),
                                   _stream()), "m2_bert_mixer_fwd")
    return y


def m2_hyena_scratch(plan: Plan, B: int, n: int, d: int, dh: int, device=None) -> torch.Tensor:
    sb = int(lib().m2_hyena_scratch_bytes(plan.handle, B, n, d, dh))
    return torch.empty(max(sb, 16), dtype=torch.uint8, device=device if device is not None else f"cuda:{plan.device}")


def m2_hyena_heads_fwd(plan: Plan, u: torch.Tensor, W, kf1, kf2, kf3, kf_long, dh: int, scratch: torch.Tensor | None = None,
                       y: torch.Tensor | None = None) -> torch.Tensor:
    """The M2 Hyena layer with heads on u [B, n, d]; W = (W_X1, W_X2, W_V, W_O), each [d, d] stored outputs x inputs;
    kf1..kf3 = m2_kernel_spectrum of the short kernels [d, n]; kf_long = m2_kernel_spectrum of the long kernels
    [d // dh, n], one row per head (its dh^2 outer-product sequences share it)."""
    B, n, d = u.shape
    assert len(W) == 4 and d % dh == 0
    for a in (u, *W):
        assert a.is_cuda and a.dtype == plan.torch_dtype and a.is_contiguous()
    if y is None:
        y = torch.empty_like(u)
    if scratch is None:   # hundreds of MB at model sizes: callers in a loop should pass one buffer (m2_hyena_scratch)
        scratch = m2_hyena_scratch(plan, B, n, d, dh, u.device)
    wp = (ctypes.c_void_p * 4)(*[w.data_ptr() for w in W])
    _check(lib().m2_hyena_heads_fwd(plan.handle, _ptr(u), wp, _ptr(kf1), _ptr(kf2), _ptr(kf3), _ptr(kf_long), _ptr(y), B, n, d, dh,
                                    _ptr(scratch), scratch.numel(), _stream()), "m2_hyena_heads_fwd")
    return y


def m2_monarch_cols_bwd_input(plan_t: Plan, G: torch.Tensor, L: torch.Tensor, R: torch.Tensor, ws: torch.Tensor | None = None):
    """dX = M^T G for Y = M X in the column layout (X, G: [Bt, N, d]): the forward call with the block-wise transposed factors
    in swapped roles.  plan_t: a plan with the factors (N2, N1) (the forward plan itself when N1 == N2)."""
    return m2_monarch_cols(plan_t, G, m2_blocks_transpose(plan_t, R), m2_blocks_transpose(plan_t, L), ws=ws)


def m2_blocks_transpose(plan: Plan, W: torch.Tensor) -> torch.Tensor:
    """W: [nblocks, rows, cols] CUDA tensor of the plan dtype; returns [nblocks, cols, rows]."""
    assert W.is_cuda and W.dtype == plan.torch_dtype and W.is_contiguous() and W.dim() == 3
    nb, r, c = W.shape
    out = torch.empty((nb, c, r), dtype=W.dtype, device=W.device)
    _check(lib().m2_blocks_transpose(plan.handle, _ptr(W), _ptr(out), nb, r, c, _stream()), "m2_blocks_transpose")
    return out


def m2_monarch_matmul_bwd_input(plan_t: Plan, G: torch.Tensor, L: torch.Tensor, R: torch.Tensor, ws: torch.Tensor | None = None):
    """dX = M^T G for M = P L P^T R P: the forward call with the block-wise transposed factors in swapped roles.
    plan_t: a plan with the factors (N2, N1) (the forward plan itself when N1 == N2)."""
    return m2_monarch_matmul(plan_t, G, m2_blocks_transpose(plan_t, R), m2_blocks_transpose(plan_t, L), ws=ws)


def m2_monarch_matmul_bwd_weights(plan: Plan, X: torch.Tensor, G: torch.Tensor, L: torch.Tensor, R: torch.Tensor,
                                  ws: torch.Tensor | None = None):
    """(dL, dR) in fp32 for the upstream gradient G of Y = M X; X, G: [T, N] of the plan dtype."""
    for a in (X, G, L, R):
        assert a.is_cuda and a.dtype == plan.torch_dtype and a.is_contiguous()
    T = X.shape[0]
    assert X.shape == G.shape
    dL = torch.empty(L.shape, dtype=torch.float32, device=X.device)
    dR = torch.empty(R.shape, dtype=torch.float32, device=X.device)
    need = int(lib().m2_matmul_bwd_workspace_bytes(plan.handle, T))
    if ws is None:
        ws = torch.empty(max(need, 16), dtype=torch.uint8, device=X.device)
    _check(lib().m2_monarch_matmul_bwd_weights(plan.handle, _ptr(X), _ptr(G), _ptr(L), _ptr(R), _ptr(dL), _ptr(dR), T,
                                               _ptr(ws), ws.numel() * ws.element_size(), _stream()),
           "m2_monarch_matmul_bwd_weights")
    return dL, dR


def m2_monarch_matmul_host(plan: Plan, X_host, L, R, Y_host, X_scratch, Y_scratch, ws: torch.Tensor | None = None):
    if ws is None:
        ws = m2_matmul_workspace(plan, X_host.shape[0], X_scratch.device)
    _check(lib().m2_monarch_matmul_host(plan.handle, _ptr(X_host), _ptr(L), _ptr(R), _ptr(Y_host), _ptr(X_scratch),
                                        _ptr(Y_scratch), X_host.shape[0], _ptr(ws), 0 if ws is None else ws.numel(),
                                        _stream()), "m2_monarch_matmul_host")
    return Y_host


def m2_block_fwd(plan: Plan, x: torch.Tensor, kf: torch.Tensor, w_short: torch.Tensor, W_up: torch.Tensor,
                 W_down: torch.Tensor, nblk: int = 4, expand: int = 4):
    """x: [B, T, C] bf16.  Returns (y, z), both indexed [b, t, c]; where the library leaves z channel-first
    (m2_block_z_channel_first) the returned z is a transposed view of that buffer."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.is_contiguous() and x.dim() == 3
    assert w_short.dtype == torch.float32 and W_up.dtype == torch.bfloat16 and W_down.dtype == torch.bfloat16
    B, T, C = x.shape
    zcf = int(lib().m2_block_z_channel_first(plan.handle, T, C, nblk, expand)) == 1
    z = torch.empty((B, C, T) if zcf else (B, T, C), dtype=x.dtype, device=x.device)
    y = torch.empty_like(x)
    _check(lib().m2_block_fwd(plan.handle, _ptr(x), _ptr(kf), _ptr(w_short), _ptr(W_up), _ptr(W_down), _ptr(z), _ptr(y),
                              B, T, C, nblk, expand, _stream()), "m2_block_fwd")
    return y, (z.transpose(1, 2) if zcf else z)


def m2_block_fwd_static(plan: Plan, x: torch.Tensor, kf: torch.Tensor, w_short: torch.Tensor, W_up: torch.Tensor,
                        W_down: torch.Tensor, y: torch.Tensor, nblk: int = 4, expand: int = 4):
    """m2_block_fwd without any allocation inside the library and without a caller-provided scratch: the
    intermediate lives in a fixed array inside libm2.so (x.numel() * 2 <= M2_STATIC_SCRATCH_BYTES).  The caller
    passes the output tensor y; calls that overlap on the GPU must be ordered by the caller."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.is_contiguous() and x.dim() == 3
    assert y.is_cuda and y.dtype == torch.bfloat16 and y.is_contiguous() and y.shape == x.shape
    B, T, C = x.shape
    _check(lib().m2_block_fwd_static(plan.handle, _ptr(x), _ptr(kf), _ptr(w_short), _ptr(W_up), _ptr(W_down), _ptr(y),
                                     B, T, C, nblk, expand, _stream()), "m2_block_fwd_static")
    return y


def m2_blocky_monarch(plan: Plan, Lt: torch.Tensor, Rt: torch.Tensor, causal_mask: bool = True):
    """Lt, Rt: float32 CUDA tensors [N, b] of polynomial coefficients.  Returns the opaque factor set (uint8 tensor)."""
    b = plan.dims[0]
    for t in (Lt, Rt):
        assert t.is_cuda and t.dtype == torch.float32 and t.is_contiguous() and tuple(t.shape) == (plan.N, b)
    nbytes = int(lib().m2_blocky_factors_bytes(plan.handle))
    if nbytes < 0:
        raise M2Error(M2_ERR_UNSUPPORTED, "m2_blocky_factors_bytes")
    fac = torch.empty(nbytes, dtype=torch.uint8, device=Lt.device)
    _check(lib().m2_blocky_monarch(plan.handle, _ptr(Lt), _ptr(Rt), 1 if causal_mask else 0, _ptr(fac), _stream()), "m2_blocky_monarch")
    return fac


def m2_blocky_kernel_spectrum(plan: Plan, factors: torch.Tensor, k: torch.Tensor):
    """k: float32 CUDA tensor [H, n].  Returns kf: float32 [H, N, 2] (complex, plan order)."""
    assert k.is_cuda and k.dtype == torch.float32 and k.is_contiguous() and k.dim() == 2
    H, n = k.shape
    kf = torch.empty((H, plan.N, 2), dtype=torch.float32, device=k.device)
    _check(lib().m2_blocky_kernel_spectrum(plan.handle, _ptr(factors), _ptr(k), H, n, _ptr(kf), _stream()), "m2_blocky_kernel_spectrum")
    return kf


def m2_blocky_monarch_conv_fwd(plan: Plan, factors: torch.Tensor, x: torch.Tensor, kf: torch.Tensor, y: torch.Tensor | None = None):
    """x: [B, H, n] CUDA tensor of the plan dtype, 2 n <= N; returns y of the same shape."""
    assert x.is_cuda and x.dtype == plan.torch_dtype and x.is_contiguous() and x.dim() == 3
    B, H, n = x.shape
    if y is None:
        y = torch.empty_like(x)
    _check(lib().m2_blocky_monarch_conv_fwd(plan.handle, _ptr(factors), _ptr(x), _ptr(kf), _ptr(y), B, H, n, _stream()),
           "m2_blocky_monarch_conv_fwd")
    return y
