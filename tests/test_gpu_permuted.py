"""avq_forward_permuted: query tiles that follow a caller-supplied token order.

The oracle has no notion of a permutation: it is given the queries already in tile order and its output
rows are put back by hand, which is what the entry point must reproduce."""
import numpy as np
import pytest
import torch

from oracle import avq_oracle as orc
from paper_2607_12789_b200 import binding, synth
from tests import parity

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("wl", [synth.C0.with_(H=2, N=250, seed=9),
                                synth.C1.with_(B=2, H=2, N=777, seed=12),
                                synth.C3.with_(H=2, N=1000, seed=13)],
                         ids=["f32", "bf16_d64", "bf16_d128_M256"])
def test_permuted_tiles_match_the_oracle_on_reordered_queries(wl):
    x = synth.generate(wl)
    g = np.random.default_rng(wl.seed)
    perm = g.permutation(wl.N).astype(np.int32)
    dv = parity.to_device(x, wl.dtype)
    Y, topp, imp, status = binding.forward_permuted(dv["Q"], dv["K"], dv["V"], dv["Cp"], dv["Cc"], wl.P, wl.block_q,
                                                    torch.from_numpy(perm).cuda(), scale=wl.scale)
    torch.cuda.synchronize()
    assert status == 0
    ref = orc.forward(np.ascontiguousarray(x["Q"][:, :, perm]), x["K"], x["V"], x["Cp"], x["Cc"], wl.P, wl.block_q,
                      wl.scale)
    Y_ref = np.empty_like(ref["Y"])
    Y_ref[:, :, perm] = ref["Y"]                                 # back to the caller's order
    same, excused = parity.compare_selection(dict(selected=topp.cpu().numpy(), importance=imp.cpu().numpy()), ref)
    assert excused == 0
    rows = np.empty((wl.B, wl.H, wl.N), dtype=bool)
    rows[:, :, perm] = np.repeat(same, wl.block_q, axis=-1)[..., :wl.N]
    parity.compare_output(Y.float().cpu().numpy().astype(np.float64), Y_ref, wl.dtype, rows)
    # the identity order is the plain forward
    ident = torch.arange(wl.N, dtype=torch.int32, device="cuda")
    Yi, _, _, st = binding.forward_permuted(dv["Q"], dv["K"], dv["V"], dv["Cp"], dv["Cc"], wl.P, wl.block_q, ident,
                                            scale=wl.scale)
    Y0 = binding.forward(dv["Q"], dv["K"], dv["V"], dv["Cp"], dv["Cc"], wl.P, wl.block_q, scale=wl.scale)
    # (equal up to the summation order of the aggregation's atomic adds, which differs from run to run)
    assert st == 0 and (Yi.float() - Y0.float()).abs().max().item() <= (1e-5 if wl.dtype == "f32" else 1.6e-2)
    assert (Yi.float() - Y0.float()).abs().mean().item() <= 1e-4
    # and a different grouping of the queries really gives a different result
    assert (Y.float() - Y0.float()).abs().max().item() > 5e-2


def test_out_of_range_entries_are_skipped_and_reported():
    wl = synth.C1.with_(B=1, H=2, N=512, seed=14)
    dv = parity.to_device(synth.generate(wl), "bf16")
    perm = torch.arange(wl.N, dtype=torch.int32, device="cuda")
    perm[7] = wl.N + 5
    perm[300] = -1
    Y, _, _, status = binding.forward_permuted(dv["Q"], dv["K"], dv["V"], dv["Cp"], dv["Cc"], wl.P, wl.block_q, perm,
                                               scale=wl.scale)
    torch.cuda.synchronize()
    assert status == 8                                           # AVQ_ERR_INDEX
    assert torch.isfinite(Y.float()).all()
    assert (Y[:, :, 7] == 0).all() and (Y[:, :, 300] == 0).all()  # the rows nothing was scattered to stay as they were
