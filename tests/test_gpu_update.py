"""avq_codebook_update against the oracle's codebook_update (appendix "Codeword Clustering During Training")."""
import numpy as np
import pytest
import torch

from oracle import avq_oracle as orc
from paper_2607_12789_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _state(wl, seed):
    g = np.random.default_rng(seed)
    H, M, C, d = wl.H, wl.M, wl.C, wl.d
    Np = g.uniform(0.0, 40.0, size=(H, M)).astype(np.float32)
    Nc = g.uniform(0.0, 10.0, size=(H, M, C)).astype(np.float32)
    Np[:, ::7] = 0.0                                             # codes that have never seen a key
    Nc[:, ::5, 1] = 0.0
    Sp = (g.normal(size=(H, M, d)) * 3 * Np[..., None]).astype(np.float32)
    Sc = (g.normal(size=(H, M, C, d)) * 3 * Nc[..., None]).astype(np.float32)
    return Sp, Np, Sc, Nc


@pytest.mark.parametrize("wl,flags", [(synth.C0.with_(B=2, H=2, seed=21), 0),
                                      (synth.C0.with_(B=2, H=2, seed=22, keys_around_parents=True, sigma_k=0.4),
                                       binding.FLAG_PARENT_STAYS),
                                      (synth.C1.with_(B=2, H=3, N=2000, seed=23), 0),
                                      (synth.C3.with_(B=1, H=2, N=3000, seed=24), 0),
                                      (synth.C1.with_(B=2, H=2, N=1500, seed=25, keys_around_parents=True,
                                                      sigma_k=0.45), binding.FLAG_PARENT_STAYS)],
                         ids=["f32", "f32_parent_stays", "bf16_d64", "bf16_d128_M256", "bf16_parent_stays"])
def test_update_matches_the_oracle(wl, flags):
    x = synth.generate(wl)
    Sp, Np, Sc, Nc = _state(wl, wl.seed)
    td = torch.float32 if wl.dtype == "f32" else torch.bfloat16
    dev = lambda a, t=torch.float32: torch.from_numpy(np.ascontiguousarray(a)).cuda().to(t)
    dS = [dev(a) for a in (Sp, Np, Sc, Nc)]
    Cp2, Cc2 = binding.codebook_update(dev(x["K"], td), dev(x["Cp"], td), dev(x["Cc"], td), *dS, 0.9, flags=flags)
    torch.cuda.synchronize()
    ref = orc.codebook_update(x["K"], x["Cp"], x["Cc"], Sp, Np, Sc, Nc, 0.9,
                              parent_stays=bool(flags & binding.FLAG_PARENT_STAYS))
    for got, key in zip(dS, ("Sp", "Np", "Sc", "Nc")):
        np.testing.assert_allclose(got.cpu().numpy(), ref[key], rtol=2e-5, atol=2e-3, err_msg=key)
    assert np.array_equal(dS[1].cpu().numpy() > 0, ref["Np"] > 0)
    # codebooks: fp32 arithmetic on the fp32 path; one bf16 rounding on top of it on the bf16 path.  A child
    # with (almost) no mass divides a residual by a tiny number on both sides, so compare relative to the
    # displacement it can take.
    tol = 2e-3 if wl.dtype == "f32" else 6e-2
    scale_c = 1.0 + np.abs(ref["Cc"])
    assert np.abs(Cp2.float().cpu().numpy() - ref["Cp"]).max() <= tol
    assert (np.abs(Cc2.float().cpu().numpy() - ref["Cc"]) / scale_c).max() <= tol
    if wl.dtype == "f32":
        np.testing.assert_allclose(Cc2.cpu().numpy().mean(axis=2), Cp2.cpu().numpy(), atol=2e-3)
