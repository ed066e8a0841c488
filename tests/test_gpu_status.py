"""The device status word: how a kernel that gives up on a wait, or meets a bad index, reports it.

Nothing here faults or hangs the GPU: the expired wait is a wait with a one-millisecond limit on a barrier
that nothing arrives on (the kernel then returns normally), and the "earlier failure" is a status word
written by the test itself."""
import ctypes

import numpy as np
import pytest
import torch

from paper_2607_12789_b200 import binding, synth
from tests import parity

pytestmark = pytest.mark.gpu


def _forward_object(wl, dv):
    f = binding.Forward(wl.B, wl.H, wl.N, wl.N, wl.d, wl.M, wl.C, wl.P, wl.block_q, dtype=torch.bfloat16,
                        scale=wl.scale, aux=True)
    Y = f(dv["Q"], dv["K"], dv["V"], dv["Cp"], dv["Cc"])
    f.check()
    return f, Y


def test_recorded_failure_stops_later_kernels_and_check_reports_then_clears_it():
    wl = synth.C1.with_(B=1, H=2, N=512)
    dv = parity.to_device(synth.generate(wl), "bf16")
    f, Y = _forward_object(wl, dv)
    word = f.workspace[:4].view(torch.int32)
    word.fill_(102)                                       # as if the attention kernel of an earlier call gave up
    sentinel = torch.full_like(Y, 7.0)
    f.attend(dv["Q"], dv["Cp"], dv["Cc"], sentinel)
    torch.cuda.synchronize()
    assert torch.equal(sentinel, torch.full_like(Y, 7.0))  # the kernel left at once: nothing written
    st = binding.lib().avq_check(binding._ptr(f.workspace), binding._stream())
    assert st == 7                                        # AVQ_ERR_DEVICE_TIMEOUT
    assert binding.lib().avq_check(binding._ptr(f.workspace), binding._stream()) == 0   # cleared by the first check
    Y2 = f.attend(dv["Q"], dv["Cp"], dv["Cc"])            # and the workspace is usable again
    f.check()
    assert torch.equal(Y2, Y)


def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    wl = synth.C1.with_(B=1, H=2, N=512)
    dv = parity.to_device(synth.generate(wl), "bf16")
    f, Y = _forward_object(wl, dv)
    lib = binding.lib()
    lib.avq_selftest_wait_expiry.restype = ctypes.c_int32
    lib.avq_selftest_wait_expiry.argtypes = [ctypes.c_void_p, ctypes.c_uint32, ctypes.c_void_p, ctypes.c_void_p]
    gave_up = torch.zeros(1, dtype=torch.int32, device="cuda")
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    assert lib.avq_selftest_wait_expiry(binding._ptr(f.workspace), 1000, binding._ptr(gave_up), binding._stream()) == 0
    t1.record()
    torch.cuda.synchronize()
    assert 0.9 <= t0.elapsed_time(t1) < 100.0             # it waited about the 1 ms it was given, then returned
    assert int(gave_up.item()) == 32
    assert lib.avq_check(binding._ptr(f.workspace), binding._stream()) == 7
    assert lib.avq_check(binding._ptr(f.workspace), binding._stream()) == 0
    Y2 = f(dv["Q"], dv["K"], dv["V"], dv["Cp"], dv["Cc"])  # a following forward on the same workspace is correct
    f.check()
    assert torch.equal(Y2, Y)


def test_aggregate_with_caller_indices_stay_keys_and_out_of_range_keys():
    """avq_aggregate on the bf16 path with indices the caller supplies: child index -1 (the key stays with
    its parent, Algorithm 1's masked scatter) enters the parent sums only; an index outside the codebook is
    left out of every sum instead of being used as an address.  Both aggregate variants (per-key scatter
    for a short head, leaf-ordered chunks for a long one)."""
    from oracle import avq_oracle as orc
    for N, M, C, d in ((1500, 64, 4, 64), (40000, 32, 8, 128)):
        g = np.random.default_rng(N)
        V = synth.round_to_bf16(g.standard_normal((1, 2, N, d)).astype(np.float32))
        pidx = g.integers(0, M, size=(1, 2, N)).astype(np.int32)
        cidx = g.integers(-1, C, size=(1, 2, N)).astype(np.int32)          # about 1 / (C + 1) of the keys stay
        bad = g.choice(N, size=40, replace=False)
        pb, cb = pidx.copy(), cidx.copy()
        pb[0, 0, bad[:10]] = M
        pb[0, 1, bad[10:20]] = -3
        cb[0, 0, bad[20:30]] = C
        cb[0, 1, bad[30:]] = -2
        dev = lambda a: torch.from_numpy(a).cuda()
        Vp, n_p, Vc, n_c = binding.aggregate(dev(V).to(torch.bfloat16), dev(pb), dev(cb), M, C)
        torch.cuda.synchronize()
        for h in range(2):
            ok = (pb[0, h] >= 0) & (pb[0, h] < M) & (cb[0, h] >= -1) & (cb[0, h] < C)
            rVp, rnp, rVc, rnc = orc.aggregate_head(V[0, h][ok], pb[0, h][ok], cb[0, h][ok], M, C)
            assert (cb[0, h][ok] < 0).sum() > 50
            assert np.array_equal(n_p[0, h].cpu().numpy(), rnp)
            assert np.array_equal(n_c[0, h].cpu().numpy(), rnc)
            assert np.allclose(Vc[0, h].cpu().numpy(), rVc, rtol=2e-5, atol=2e-3)
            assert np.allclose(Vp[0, h].cpu().numpy(), rVp, rtol=2e-5, atol=2e-3)


@pytest.mark.parametrize("stays", [False, True])
def test_back_to_back_forwards_are_repeatable(stays):
    """The kernels of one call overlap their set-up with the kernel before them (programmatic dependent
    launch); a load that slipped ahead of the dependency wait would read counts or sums that are not final
    and show up as a run that differs from the others.  Forty calls back to back (no host synchronisation in
    between), two shapes: indices, counts and selections identical every time, sums and outputs within the
    rounding of a different atomic order."""
    flags = binding.FLAG_PARENT_STAYS if stays else 0
    for wl in (synth.C1.with_(B=2, H=3, N=1024, seed=61, keys_around_parents=stays),
               synth.sweep_point(16384, 256, 64).with_(H=1, N=32768, seed=62, keys_around_parents=stays)):   # chained tiles
        dv = parity.to_device(synth.generate(wl), "bf16")
        f = binding.Forward(wl.B, wl.H, wl.N, wl.N, wl.d, wl.M, wl.C, wl.P, wl.block_q, dtype=torch.bfloat16,
                            scale=wl.scale, flags=flags, aux=True)
        runs = []
        for _ in range(40):
            Y = f(dv["Q"], dv["K"], dv["V"], dv["Cp"], dv["Cc"])
            im = f.intermediates()
            runs.append((Y.clone(), f.topp.clone(), im["np"].clone(), im["nc"].clone(), im["parent_idx"].clone(),
                         im["child_idx"].clone(), im["Vp"].clone()))
        f.check()
        Y0, t0, np0, nc0, p0, c0, Vp0 = runs[0]
        assert float(np0.sum()) == wl.B * wl.H * wl.N
        for Y, t, np_, nc, p, c, Vp in runs[1:]:
            assert torch.equal(p, p0) and torch.equal(c, c0)
            assert torch.equal(np_, np0) and torch.equal(nc, nc0)
            assert torch.equal(t, t0)
            assert (Vp - Vp0).abs().max().item() <= 1e-3
            assert (Y.float() - Y0.float()).abs().max().item() <= 2e-2
