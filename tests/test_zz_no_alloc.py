"""m2_block_fwd_static: the block forward for callers that cannot allocate device memory (a serving process
whose framework owns all of it, a loop that cannot take cudaMalloc's synchronisation).  Its intermediate lives in
a fixed array inside the library, so this checks, through the C ABI, that it gives what m2_block_fwd gives with a
caller-provided scratch and what the CPU oracle gives -- twice in a row, because the array keeps the previous call's
contents --, that the call leaves the amount of free device memory unchanged, and that an input too large for the
array is refused.  Collected last so a failure here cannot hide other tests."""
import numpy as np
import pytest
import torch

from oracle import monarch_oracle as O
from paper_2310_12109_b200 import binding as M
from paper_2310_12109_b200 import synth

pytestmark = pytest.mark.gpu

TOL_BF16 = 2e-2


def _dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    return t.to(dtype) if dtype is not None else t


def _rel(a, b):
    return float(np.linalg.norm(a - b) / np.linalg.norm(b))


@pytest.mark.parametrize("dims,T,C,nblk,expand,kernel", [
    ((32, 16), 512, 768, 4, 4, "block_conv_umma_mlp_umma_static"),     # both tensor-core kernels
    ((16, 8), 128, 64, 4, 2, "block_generic_static"),                  # the strided CUDA-core route
])
def test_static_scratch_matches_caller_scratch_and_oracle_twice(dims, T, C, nblk, expand, kernel):
    plan = M.Plan(dims, dtype=M.M2_BF16, device=0)
    outs = []
    for B, shift in ((2, 0), (3, 1)):          # two calls in a row, different sizes and data
        c = synth.config5(B=B, T=T, C=C, nblk=nblk, expand=expand)
        c["dims"] = dims
        c["x"] = np.ascontiguousarray(np.roll(c["x"], shift, axis=1))
        x = _dev(c["x"], torch.bfloat16)
        kf = M.m2_kernel_spectrum(plan, _dev(c["k"]))
        w, Wu, Wd = _dev(c["w_short"]), _dev(c["W_up"], torch.bfloat16), _dev(c["W_down"], torch.bfloat16)
        y_ref, _ = M.m2_block_fwd(plan, x, kf, w, Wu, Wd, nblk=nblk, expand=expand)
        y = torch.full_like(x, 7.0)
        torch.cuda.synchronize()
        free0, _ = torch.cuda.mem_get_info()
        M.m2_block_fwd_static(plan, x, kf, w, Wu, Wd, y, nblk=nblk, expand=expand)
        torch.cuda.synchronize()
        free1, _ = torch.cuda.mem_get_info()
        if outs:                                # (the first call on a device may load the module that holds the array)
            assert free1 == free0, (free0, free1)
        assert plan.device_status() == 0 and plan.last_kernel() == kernel
        a, b = y.float().cpu().numpy().astype(np.float64), y_ref.float().cpu().numpy().astype(np.float64)
        assert np.isfinite(a).all()
        err = _rel(a, b)
        assert err <= TOL_BF16, err
        outs.append(err)
        # ... and against the oracle, row by row
        yr, _ = O.m2_block_forward(c["x"].astype(np.float64), c["k"].astype(np.float64), c["w_short"].astype(np.float64),
                                   c["W_up"].astype(np.float64), c["W_down"].astype(np.float64), dims)
        ar, br = a.reshape(-1, C), yr.reshape(-1, C)
        assert _rel(ar, br) <= TOL_BF16
        per = np.linalg.norm(ar - br, axis=1) / np.linalg.norm(br, axis=1)
        assert per.max() <= 2 * TOL_BF16, per.max()
    # same kernels, same inputs: in fact identical to the caller-scratch entry point
    assert max(outs) == 0.0
    plan.close()


def test_static_scratch_rejects_oversize_and_bad_args():
    plan = M.Plan((32, 16), dtype=M.M2_BF16, device=0)
    lib = M.lib()
    B_big = M.M2_STATIC_SCRATCH_BYTES // (512 * 768 * 2) + 1
    x = torch.zeros((1, 512, 768), dtype=torch.bfloat16, device="cuda")
    p = x.data_ptr()
    s = torch.cuda.current_stream().cuda_stream
    assert lib.m2_block_fwd_static(plan.handle, p, p, p, p, p, p, B_big, 512, 768, 4, 4, s) == M.M2_ERR_UNSUPPORTED
    assert lib.m2_block_fwd_static(plan.handle, p, p, p, p, p, p, 1 << 62, 512, 768, 4, 4, s) == M.M2_ERR_UNSUPPORTED   # no wrap-around
    assert lib.m2_block_fwd_static(plan.handle, p, p, p, p, p, None, 1, 512, 768, 4, 4, s) == M.M2_ERR_INVALID_ARG
    assert lib.m2_block_fwd_static(plan.handle, p, p, p, p, p, p, 1, 256, 768, 4, 4, s) == M.M2_ERR_INVALID_ARG
    torch.cuda.synchronize()
    plan.close()
