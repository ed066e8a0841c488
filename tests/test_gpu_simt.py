"""GPU parity of the CUDA-core kernels (float32 path and AVQ_FLAG_SIMT) against the oracle."""
import numpy as np
import pytest
import torch

from oracle import avq_oracle as orc
from paper_2607_12789_b200 import binding, synth
from tests import parity

pytestmark = pytest.mark.gpu
SIMT, STAYS = binding.FLAG_SIMT, binding.FLAG_PARENT_STAYS


def test_c0_tiny_f32_full_parity():
    rep = parity.full_parity(synth.C0)
    assert rep["max_abs"] <= 1e-4
    assert rep["stay_count"] == 0


@pytest.mark.parametrize("P", [0, 1, 5, 16])
def test_c0_endpoints_and_other_P(P):
    parity.full_parity(synth.C0, P=P)


def test_ragged_shapes_f32():
    wl = synth.Workload("ragged", B=2, H=3, N=333, d=36, M=11, C=3, P=4, block_q=50, dtype="f32", seed=21,
                        alpha=0.5)
    x = synth.generate(wl)
    x["Q"] = np.ascontiguousarray(x["Q"][:, :, :171])          # Nq != Nk, both ragged
    parity.full_parity(wl, x=x)


def test_parent_stays_f32():
    wl = synth.C0.with_(seed=5, H=2)
    x = synth.generate(wl)
    g = np.random.default_rng(0)
    for h in range(2):                                           # every other key hugs a parent: it stays
        near = x["Cp"][h][g.integers(0, 16, 128)] + 0.05 * g.standard_normal((128, 64)).astype(np.float32)
        x["K"][0, h, ::2] = near
    rep = parity.full_parity(wl, flags=STAYS, parent_stays=True, x=x)
    assert 200 <= rep["stay_count"] < 2 * 256                   # a real mixture of stayed and moved keys


def test_bf16_inputs_through_cuda_cores():
    wl = synth.C1.with_(B=1, H=3, N=512)
    rep = parity.full_parity(wl, flags=SIMT)
    assert rep["empty_parents"] > 0
    wl = synth.C2.with_(B=1, H=2, N=640)
    parity.full_parity(wl, flags=SIMT)


def test_exact_ties_resolve_to_lowest_index():
    g = np.random.default_rng(0)
    d, M, C = 16, 8, 4
    base = (np.clip(np.round(g.normal(size=(4, d)) * 4), -8, 8) / 4).astype(np.float32)   # exact in bf16
    Cp = np.stack([base[0], base[1], base[1], base[2], base[0], base[3], base[3], base[3]])[None]
    Cc = np.repeat(Cp[:, :, None, :], C, axis=2).copy()
    Cc[0, :, 2:] += 0.25                                          # children 0,1 equal; 2,3 equal
    K = np.concatenate([Cp[0], Cp[0] + 0.125, 0.5 * (Cp[0, [0]] + Cp[0, [1]])])[None, None]
    ref = orc.assign_head(K[0, 0], Cp[0], Cc[0])
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    for dt, fl in ((torch.float32, 0), (torch.bfloat16, SIMT)):
        pi, ci = binding.assign(t(K).to(dt), t(Cp).to(dt), t(Cc).to(dt), flags=fl)
        assert np.array_equal(pi.cpu().numpy()[0, 0], ref["parent_idx"])
        assert np.array_equal(ci.cpu().numpy()[0, 0], ref["child_idx"])
    assert ref["parent_idx"][:8].tolist() == [0, 1, 1, 3, 0, 5, 5, 5]
    assert (ref["parent_margin"][:8] == 0).sum() >= 6


def test_standalone_stages_match_forward_intermediates():
    wl = synth.C0.with_(H=2, seed=3)
    x = synth.generate(wl)
    dv = parity.to_device(x, "f32")
    pi, ci = binding.assign(dv["K"], dv["Cp"], dv["Cc"])
    Vp, n_p, Vc, n_c = binding.aggregate(dv["V"], pi, ci, wl.M, wl.C)
    _, _, _, inter = binding.forward(dv["Q"], dv["K"], dv["V"], dv["Cp"], dv["Cc"], wl.P, wl.block_q, aux=True)
    assert torch.equal(pi, inter["parent_idx"]) and torch.equal(ci, inter["child_idx"])
    assert torch.equal(n_p, inter["np"]) and torch.equal(n_c, inter["nc"])
    assert torch.allclose(Vp, inter["Vp"], atol=1e-4) and torch.allclose(Vc, inter["Vc"], atol=1e-4)
    assert float(n_p.sum()) == wl.B * wl.H * wl.N


def test_forward_host_matches_device_call():
    wl = synth.C0
    x = synth.generate(wl)
    dv = parity.to_device(x, "f32")
    f = binding.Forward(1, 1, 256, 256, 64, 16, 4, 2, 64, dtype=torch.float32)
    Y = f(dv["Q"], dv["K"], dv["V"], dv["Cp"], dv["Cc"])
    hq, hk, hv = (torch.from_numpy(x[k]).pin_memory() for k in "QKV")
    hy = torch.empty_like(hq).pin_memory()
    dq, dk, dv_, dy = (torch.empty_like(dv["Q"]) for _ in range(4))
    f.host(hq, hk, hv, dv["Cp"], dv["Cc"], hy, dq, dk, dv_, dy)
    torch.cuda.synchronize()
    f.check()
    assert torch.allclose(hy, Y.cpu(), atol=1e-6)


def test_correcting_form_matches_the_oracle_and_the_masked_form_on_recentred_codebooks():
    """AVQ_FLAG_CORRECTING (Algorithm 2's child pass as printed) on the CUDA-core kernels.  float32, re-centred
    children: equal to the oracle's correcting form and (the constraint holds to fp32 rounding) to the default
    masked form.  bfloat16 codebooks: rounding breaks parent = mean(children) by an ulp, so the kernel is
    compared with the oracle's correcting form on the same rounded codebooks, and its distance from the masked
    form is what the variant costs in accuracy."""
    wl = synth.C0.with_(H=2, seed=33, recenter_children=True)
    x = synth.generate(wl)
    dv = parity.to_device(x, "f32")
    args = (dv["Q"], dv["K"], dv["V"], dv["Cp"], dv["Cc"], wl.P, wl.block_q)
    Yc = binding.forward(*args, scale=wl.scale, flags=binding.FLAG_CORRECTING)
    Ym = binding.forward(*args, scale=wl.scale)
    ref = orc.forward(x["Q"], x["K"], x["V"], x["Cp"], x["Cc"], wl.P, wl.block_q, wl.scale, form="correcting")
    assert np.abs(Yc.cpu().numpy() - ref["Y"]).max() <= 1e-4
    assert (Yc - Ym).abs().max().item() <= 1e-4
    wl = synth.C1.with_(B=1, H=2, N=512, seed=34, recenter_children=True)
    x = synth.generate(wl)
    dv = parity.to_device(x, "bf16")
    args = (dv["Q"], dv["K"], dv["V"], dv["Cp"], dv["Cc"], wl.P, wl.block_q)
    Yc = binding.forward(*args, scale=wl.scale, flags=binding.FLAG_CORRECTING | SIMT)
    Ym = binding.forward(*args, scale=wl.scale, flags=SIMT)
    ref = orc.forward(x["Q"], x["K"], x["V"], x["Cp"], x["Cc"], wl.P, wl.block_q, wl.scale, form="correcting")
    assert np.abs(Yc.float().cpu().numpy() - ref["Y"]).max() <= 2e-2
    dev = (Yc.float() - Ym.float()).abs().max().item()
    print(f"correcting vs masked form, bf16-rounded re-centred codebooks: max-abs {dev:.3e}")
    assert dev <= 0.25
