"""avq_forward_tiled (importance from tiled parents, Eq. "aproxdenom") against the oracle, for codebooks
beyond one tile (M = 512, 1024) and for the degenerate tilings."""
import numpy as np
import pytest
import torch

from oracle import avq_oracle as orc
from paper_2607_12789_b200 import binding, synth
from tests import parity

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("wl,tile_m", [
    (synth.Workload("t512", B=1, H=2, N=1536, d=64, M=512, C=4, P=32, block_q=128, seed=61, alpha=0.3,
                    hot_queries=True), 128),
    (synth.Workload("t1024", B=1, H=1, N=2048, d=64, M=1024, C=4, P=64, block_q=128, seed=62, alpha=0.3,
                    hot_queries=True), 256),
    (synth.Workload("t96", B=2, H=2, N=300, d=32, M=96, C=2, P=9, block_q=50, dtype="f32", seed=63, alpha=0.5), 32),
], ids=["bf16_M512_tile128", "bf16_M1024_tile256", "f32_M96_tile32"])
def test_tiled_selection_importance_and_output_match_the_oracle(wl, tile_m):
    x = synth.generate(wl)
    dv = parity.to_device(x, wl.dtype)
    Y, topp, imp = binding.forward_tiled(dv["Q"], dv["K"], dv["V"], dv["Cp"], dv["Cc"], wl.P, wl.block_q, tile_m,
                                         scale=wl.scale)
    torch.cuda.synchronize()
    ref = orc.forward(x["Q"], x["K"], x["V"], x["Cp"], x["Cc"], wl.P, wl.block_q, wl.scale, form="factorised",
                      tile_m=tile_m)
    same, excused = parity.compare_selection(dict(selected=topp.cpu().numpy(), importance=imp.cpu().numpy()), ref)
    assert excused == 0
    rows = np.repeat(same, wl.block_q, axis=-1)[..., :wl.N]
    parity.compare_output(Y.float().cpu().numpy().astype(np.float64), ref["Y"], wl.dtype, rows)
    # the tiling really changed some selections with respect to the exact importance
    exact = orc.forward(x["Q"], x["K"], x["V"], x["Cp"], x["Cc"], wl.P, wl.block_q, wl.scale, form="factorised")
    assert (exact["selected"] != ref["selected"]).any()


def test_one_tile_reproduces_the_plain_forward():
    wl = synth.C0.with_(H=2, seed=64)
    x = synth.generate(wl)
    dv = parity.to_device(x, "f32")
    Y, topp, imp = binding.forward_tiled(dv["Q"], dv["K"], dv["V"], dv["Cp"], dv["Cc"], wl.P, wl.block_q, 32)
    Y0, topp0, imp0, _ = binding.forward(dv["Q"], dv["K"], dv["V"], dv["Cp"], dv["Cc"], wl.P, wl.block_q, aux=True)
    assert torch.equal(topp, topp0) and torch.allclose(imp, imp0, rtol=1e-5, atol=1e-6)
    assert (Y - Y0).abs().max().item() <= 1e-5
