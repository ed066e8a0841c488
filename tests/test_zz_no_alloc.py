"""avq_forward_static, the entry point for callers that cannot allocate device scratch.

Collected last on purpose (the file name sorts after every other test file): if it fails, a
run that stops at the first failure has already run everything else.  The GPU test calls the
entry point through the C ABI twice in a row - the second call finds the first call's
leftovers in the shared built-in array - and checks both results against avq_forward with a
caller-supplied workspace."""
import ctypes

import pytest
import torch

from paper_2607_12789_b200 import binding, build, synth
from tests import parity


def test_oversized_problem_is_rejected_before_any_launch():
    build.build()
    lib = binding.lib()
    cap = lib.avq_static_workspace_bytes()
    assert cap == 24 * 1024 * 1024
    big = binding.problem(4, 16, 65536, 65536, 64, 256, 4, binding.AVQ_BF16, 0.125)
    assert binding.workspace_bytes(big, 32, 128) > cap
    fake = ctypes.c_void_p(0x1000)
    st = lib.avq_forward_static(ctypes.byref(big), fake, fake, fake, fake, fake, 32, 128, fake, None, None, None)
    assert st == 5                                               # AVQ_ERR_WORKSPACE
    bad = binding.problem(1, 1, 256, 256, 64, 16, 4, binding.AVQ_F32, 0.125)
    st = lib.avq_forward_static(ctypes.byref(bad), fake, fake, fake, fake, fake, 99, 64, fake, None, None, None)
    assert st == 2                                               # P > M: AVQ_ERR_SHAPE, as avq_forward says


@pytest.mark.gpu
@pytest.mark.parametrize("wl", [synth.C0, synth.C1.with_(B=2, H=3)], ids=["f32_cuda_cores", "bf16_tensor_cores"])
def test_static_workspace_matches_caller_workspace_twice_in_a_row(wl):
    tol = parity.TOL[wl.dtype]["max_abs"]
    first = synth.generate(wl)
    second = synth.generate(wl.with_(seed=wl.seed + 100))        # different data: stale scratch would show
    for x in (first, second):
        dv = parity.to_device(x, wl.dtype)
        args = (dv["Q"], dv["K"], dv["V"], dv["Cp"], dv["Cc"], wl.P, wl.block_q)
        Y_ref, topp_ref, imp_ref, _ = binding.forward(*args, scale=wl.scale, aux=True)
        Y, topp, imp = binding.forward_static(*args, scale=wl.scale, aux=True)
        torch.cuda.synchronize()
        assert torch.isfinite(Y.float()).all()
        assert (Y.float() - Y_ref.float()).abs().max().item() <= tol
        assert torch.equal(topp, topp_ref)
        assert torch.allclose(imp, imp_ref, rtol=1e-4, atol=1e-5)
    # the entry point itself allocates nothing: free device memory is the same before and after a call
    # whose outputs already exist (the caching allocator is not involved: raw ctypes call, own buffers)
    prob = binding._problem_from(dv["Q"], dv["K"], dv["Cp"], dv["Cc"], wl.scale, 0)
    Y2 = torch.empty_like(dv["Q"])
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    st = binding.lib().avq_forward_static(ctypes.byref(prob), binding._ptr(dv["Q"]), binding._ptr(dv["K"]),
                                          binding._ptr(dv["V"]), binding._ptr(dv["Cp"]), binding._ptr(dv["Cc"]),
                                          wl.P, wl.block_q, binding._ptr(Y2), None, None, binding._stream())
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert st == 0 and free_after == free_before
    assert (Y2.float() - Y_ref.float()).abs().max().item() <= tol
