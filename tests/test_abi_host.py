"""CPU-side checks of the C ABI: the library loads, exports what the header declares, builds
bit-exact integer tables, and rejects bad arguments before touching a device."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import monarch_oracle as O
from paper_2310_12109_b200 import binding as M
from paper_2310_12109_b200 import build as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    B.build()


def header_functions():
    names = []
    for fn in sorted(os.listdir(os.path.join(ROOT, "include"))):
        if not fn.endswith(".h"):
            continue
        src = open(os.path.join(ROOT, "include", fn)).read()
        src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
        names += re.findall(r"\b(m2_[a-z0-9_]+)\s*\(", src)
    return sorted(set(names))


def test_every_declared_symbol_is_exported_and_bound():
    names = header_functions()
    assert len(names) >= 12
    lib = ctypes.CDLL(M.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), n
        assert n in M.SIGNATURES, f"{n} has no binding"
    assert sorted(M.SIGNATURES) == names


def host_plan(dims):
    return M.Plan(dims, dtype=M.M2_FP32, sign=+1, device=-1)


@pytest.mark.parametrize("dims", [(2, 3), (32, 16), (16, 32), (64, 64), (2, 3, 4), (32, 32, 32)])
def test_integer_tables_bit_exact(dims):
    pl = host_plan(dims)
    N = int(np.prod(dims))
    assert np.array_equal(pl.get_table(M.M2_TABLE_PERM), O.stride_perm(dims[0], N).astype(np.int32))
    assert np.array_equal(pl.get_table(M.M2_TABLE_PERM_INV), O.stride_perm(N // dims[0], N).astype(np.int32))
    assert np.array_equal(pl.get_table(M.M2_TABLE_DIGIT_REV), O.plan_order_index(dims).astype(np.int32))
    # twiddle exponents: the oracle's stage-s blocks are F_{Ns} diag(omega_M^e); recover e from them
    blocks = O.monarch_dft_factors_order_p(dims, +1)
    p = len(dims)
    for s in range(1, p):
        e_lib = pl.get_table(M.M2_TABLE_TW_EXP + s).reshape(dims)
        Mcur = int(np.prod(dims[: s + 1]))
        Blk = blocks[s].reshape(*dims[:s], *dims[s + 1:], dims[s], dims[s])
        # row k_s = 0 of a block is exactly the twiddle diagonal
        diag = Blk[..., 0, :]                      # axes: k1..ks, n_{s+2}.., n_{s+1}
        diag = np.moveaxis(diag, -1, s)            # -> k1..ks, n_{s+1}, n_{s+2}..
        e_or = np.rint(np.angle(diag) * Mcur / (2 * np.pi)).astype(np.int64) % Mcur
        assert np.array_equal(e_lib.astype(np.int64), e_or)
    pl.close()


def test_argument_validation_without_device():
    lib = M.lib()
    h = ctypes.c_void_p()
    f = (ctypes.c_int32 * 2)(32, 16)
    assert lib.m2_plan_create(None, 512, 2, f, 0, 1, -1) == M.M2_ERR_INVALID_ARG
    assert lib.m2_plan_create(ctypes.byref(h), 500, 2, f, 0, 1, -1) == M.M2_ERR_INVALID_ARG
    assert lib.m2_plan_create(ctypes.byref(h), 512, 2, f, 7, 1, -1) == M.M2_ERR_INVALID_ARG
    assert lib.m2_plan_create(ctypes.byref(h), 512, 2, f, 0, 0, -1) == M.M2_ERR_INVALID_ARG
    assert lib.m2_plan_create(ctypes.byref(h), 512, 5, f, 0, 1, -1) == M.M2_ERR_INVALID_ARG
    assert lib.m2_plan_create(ctypes.byref(h), 512, 2, f, 0, 1, -1) == M.M2_OK
    buf = (ctypes.c_int32 * 512)()
    assert lib.m2_plan_get_table(h, 0, buf, 100) == M.M2_ERR_INVALID_ARG
    assert lib.m2_plan_get_table(h, 99, buf, 512) == M.M2_ERR_INVALID_ARG
    assert lib.m2_plan_get_table(h, M.M2_TABLE_TW_EXP + 2, buf, 512) == M.M2_ERR_INVALID_ARG
    # a host-only plan refuses device work, null pointers are rejected first
    assert lib.m2_monarch_conv_fwd(h, None, None, None, 1, 1, 256, 0, None) == M.M2_ERR_INVALID_ARG
    assert lib.m2_monarch_conv_fwd(h, 16, 16, 16, 1, 1, 256, 0, None) == M.M2_ERR_NO_DEVICE
    assert lib.m2_monarch_matmul(h, 16, 16, 16, 16, 4, None, 0, None) == M.M2_ERR_NO_DEVICE
    assert lib.m2_kernel_spectrum(h, 16, 1, 256, 16, None) == M.M2_ERR_NO_DEVICE
    assert lib.m2_spectrum_bytes(h, 3) == 3 * 512 * 8
    # a host-only plan has no tensor-core route, so its block forward would leave z channel-last; bad arguments answer 0 too
    assert lib.m2_block_z_channel_first(h, 512, 768, 4, 4) == 0
    assert lib.m2_block_z_channel_first(None, 512, 768, 4, 4) == 0 and lib.m2_block_z_channel_first(h, 512, 768, 5, 4) == 0
    assert lib.m2_plan_destroy(h) == M.M2_OK
    assert lib.m2_plan_destroy(None) == M.M2_ERR_INVALID_ARG
    assert lib.m2_status_string(M.M2_ERR_TIMEOUT) == b"device-side wait timed out"


def test_matmul_workspace_covers_whole_token_tiles():
    """The tensor-core matmul keeps its intermediate in 128-token tiles: the workspace is sized for whole tiles
    (bf16 plan with 64 x 64 blocks); plans it does not cover need none."""
    pl = M.Plan((64, 64), dtype=M.M2_BF16, sign=+1, device=-1)
    lib = M.lib()
    for T, tiles in [(0, 0), (1, 1), (128, 1), (129, 2), (16384, 128)]:
        assert int(lib.m2_matmul_workspace_bytes(pl.handle, T)) == tiles * 128 * 4096 * 2
    assert int(lib.m2_matmul_workspace_bytes(host_plan((8, 8)).handle, 100)) == 0
    assert int(lib.m2_matmul_workspace_bytes(host_plan((64, 64)).handle, 100)) == 0   # fp32 plan: CUDA-core kernels
