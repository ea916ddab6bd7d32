"""m2_block_fwd_static: the block forward for callers that cannot allocate device memory (a serving process
whose framework owns all of it, a loop that cannot take cudaMalloc's synchronisation).  Its intermediate lives in
a fixed array inside the library, so this checks, through the C ABI, that it gives what m2_block_fwd gives with a
caller-provided scratch -- twice in a row, because the array keeps the previous call's contents -- and that an
input too large for the array is refused.  Collected last so a failure here cannot hide other tests."""
import numpy as np
import pytest
import torch

from paper_2310_12109_b200 import binding as M
from paper_2310_12109_b200 import synth

pytestmark = pytest.mark.gpu

TOL_BF16 = 2e-2


def _dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    return t.to(dtype) if dtype is not None else t


def test_static_scratch_matches_caller_scratch_twice():
    plan = M.Plan((32, 16), dtype=M.M2_BF16, device=0)
    outs = []
    for B, stream_shift in ((2, 0), (3, 1)):          # two calls in a row, different sizes and data
        c = synth.config5(B=B)
        x = _dev(np.roll(c["x"], stream_shift, axis=1), torch.bfloat16)
        kf = M.m2_kernel_spectrum(plan, _dev(c["k"]))
        w, Wu, Wd = _dev(c["w_short"]), _dev(c["W_up"], torch.bfloat16), _dev(c["W_down"], torch.bfloat16)
        y_ref, _ = M.m2_block_fwd(plan, x, kf, w, Wu, Wd)
        y = torch.full_like(x, 7.0)
        M.m2_block_fwd_static(plan, x, kf, w, Wu, Wd, y)
        torch.cuda.synchronize()
        assert plan.device_status() == 0
        a, b = y.float().cpu().numpy().astype(np.float64), y_ref.float().cpu().numpy().astype(np.float64)
        assert np.isfinite(a).all()
        err = np.linalg.norm(a - b) / np.linalg.norm(b)
        assert err <= TOL_BF16, err
        outs.append(err)
    # same kernels, same inputs: in fact identical
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
    assert lib.m2_block_fwd_static(plan.handle, p, p, p, p, p, None, 1, 512, 768, 4, 4, s) == M.M2_ERR_INVALID_ARG
    assert lib.m2_block_fwd_static(plan.handle, p, p, p, p, p, p, 1, 256, 768, 4, 4, s) == M.M2_ERR_INVALID_ARG
    torch.cuda.synchronize()
    plan.close()
