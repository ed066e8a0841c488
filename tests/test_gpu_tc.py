"""GPU parity of the tcgen05 tensor-core path (bf16) against the fp64 oracle.

Small and mid-size configurations are compared whole; the long ones on whole sampled heads
(assignments, aggregates) and sampled query blocks (importance, top-P, output)."""
import numpy as np
import pytest
import torch

from paper_2607_12789_b200 import binding, synth
from tests import parity

pytestmark = pytest.mark.gpu


def test_small_bf16_single_child_tile():
    rep = parity.full_parity(synth.C1.with_(B=1, H=2, N=512))
    assert rep["empty_parents"] > 0


def test_c1_vitb_full():
    rep = parity.full_parity(synth.C1)
    print("c1", rep)


def test_c2_mid_full():
    rep = parity.full_parity(synth.C2)
    print("c2", rep)


def test_c3_long_sampled():
    rep, gpu, x = parity.sampled_parity(synth.C3, heads=[(0, 3), (0, 12)], blocks_per_head=8)
    print("c3", rep)
    # properties that hold at any size, over the whole tensor
    assert np.isfinite(gpu["Y"]).all()
    assert np.array_equal(gpu["np"].sum(axis=-1), np.full((1, 16), 16384.0))
    assert np.array_equal(gpu["nc"].sum(axis=-1), gpu["np"])
    np.testing.assert_allclose(gpu["importance"].sum(axis=-1), 128.0, rtol=1e-4)
    np.testing.assert_allclose(gpu["Vp"].sum(axis=2), x["V"].astype(np.float64).sum(axis=2), atol=5e-3)
    # every query tile of six heads against the factorised oracle (768 of the 2048 tiles)
    rep2, _ = parity.heads_parity_factorised(synth.C3, [(0, h) for h in (0, 3, 6, 9, 12, 15)], x=x, gpu=gpu)
    print("c3 whole heads", rep2)
    assert rep2["blocks"] >= 6 * 128 - rep2["topp_flips_excused"]


# Sweep configuration: every (N, M, P) point has a parity test.  All P of one (N, M) share their data, so
# the oracle's assignment of a head is computed once per (N, M).  N <= 16384: every query tile of the
# listed heads (factorised oracle); N = 65536: one head, every tile.
@pytest.mark.parametrize("M", [32, 64, 128, 256])
def test_sweep_N1024_all_P(M):
    for P in synth.sweep_P(M):
        parity.full_parity(synth.sweep_point(1024, M, P).with_(H=4))


@pytest.mark.parametrize("M", [32, 64, 128, 256])
@pytest.mark.parametrize("N,H", [(4096, 2), (16384, 1), (65536, 1)])
def test_sweep_all_P_whole_heads(N, H, M):
    wl0 = synth.sweep_point(N, M, 0).with_(H=H)
    x = synth.generate(wl0)
    heads = [(0, h) for h in range(H)]
    cache = {}
    for P in synth.sweep_P(M):
        rep, cache = parity.heads_parity_factorised(wl0.with_(P=P), heads, x=x, assignments=cache, P=P)
        print(f"sweep N={N} M={M} P={P}", rep)


def test_sweep_dense_definition_on_sampled_tiles():
    """The O(N^2) definition itself on sampled tiles of long sweep points."""
    parity.sampled_parity(synth.sweep_point(16384, 256, 32), heads=[(0, 5)], blocks_per_head=6)
    parity.sampled_parity(synth.sweep_point(65536, 64, 16), heads=[(0, 9)], blocks_per_head=4)


def _exact_grid(g, shape, step=0.25, lim=4.0):
    """Random values on a coarse grid: exactly representable in bf16, sums of squares exact in fp32."""
    return (np.clip(np.round(g.normal(size=shape) / step), -lim / step, lim / step) * step).astype(np.float32)


@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("C", [4, 8])
def test_exact_ties_on_the_tensor_core_path(d, C):
    """Duplicated parent codewords, duplicated children, keys at exact midpoints and keys equal to
    codewords, inside the tcgen05 envelope (M = 32): best and runner-up distances coincide, so the
    float64 recheck of avq_assign decides, and the lowest index must win (Algorithm 1's strict '<')."""
    from oracle import avq_oracle as orc
    g = np.random.default_rng(7 + d + C)
    M = 32
    base = _exact_grid(g, (12, d))
    Cp = base[g.integers(0, 12, size=M)]                      # 32 parents drawn from 12 distinct rows
    Cp[5] = Cp[2]; Cp[9] = Cp[2]; Cp[31] = Cp[30]
    Cc = np.repeat(Cp[:, None, :], C, axis=1).copy()
    Cc[:, C // 2:] += 0.5                                     # children 0..C/2-1 equal, C/2..C-1 equal
    Cc[3] = _exact_grid(g, (C, d))
    Cc[3, 2] = Cc[3, 1]                                       # a duplicated pair in the middle
    keys = [Cp,                                               # keys on parent codewords
            Cc.reshape(-1, d),                                # keys on child codewords
            0.5 * (Cp[:16] + Cp[16:]),                        # exact midpoints of two parents
            0.5 * (Cc[:, 0] + Cc[:, C - 1]),                  # exact midpoints of two children
            _exact_grid(g, (200, d))]
    K = np.concatenate(keys).astype(np.float32)
    assert np.array_equal(synth.round_to_bf16(K), K) and np.array_equal(synth.round_to_bf16(Cc), Cc)
    ref = orc.assign_head(K, Cp, Cc)
    assert (ref["parent_margin"] == 0).sum() >= M and (ref["child_margin"] == 0).sum() >= M
    # a key that sits on parent i must be given the FIRST parent with that codeword (written out by hand)
    first_equal = [min(j for j in range(M) if np.array_equal(Cp[j], Cp[i])) for i in range(M)]
    assert ref["parent_idx"][:M].tolist() == first_equal and first_equal[5] == first_equal[9] == first_equal[2]
    assert len(set(first_equal)) <= 12
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda().to(torch.bfloat16)
    pi, ci = binding.assign(t(K[None, None]), t(Cp[None]), t(Cc[None]))
    torch.cuda.synchronize()
    assert np.array_equal(pi.cpu().numpy()[0, 0], ref["parent_idx"])
    assert np.array_equal(ci.cpu().numpy()[0, 0], ref["child_idx"])


def test_ragged_tail_and_nq_not_nk():
    wl = synth.C1.with_(B=1, H=3, N=1000, seed=31)
    x = synth.generate(wl)
    x["Q"] = np.ascontiguousarray(x["Q"][:, :, :700])
    parity.full_parity(wl, x=x)


def test_other_shapes_d128_C8_M96():
    parity.full_parity(synth.Workload("odd", B=1, H=2, N=768, d=128, M=96, C=8, P=12, block_q=128, seed=77,
                                      alpha=0.5, hot_queries=True))


@pytest.mark.parametrize("wl", [synth.C1.with_(B=2, H=2, N=1500, seed=51), synth.C3.with_(H=2, N=2000, seed=52),
                                synth.C2.with_(B=1, H=2, N=1100, seed=53),
                                synth.sweep_point(4096, 32, 8).with_(H=2, seed=54),      # long head: leaf-ordered aggregate
                                synth.sweep_point(4096, 128, 128).with_(H=2, seed=55)],  # every parent refined, 4 child chunks
                         ids=["d64_M64_C4", "d128_M256_C4", "d64_M128_C8", "long_head_M32", "all_refined_M128"])
def test_parent_stays_on_the_tensor_core_path(wl):
    """Algorithm 1's masked scatter on the tcgen05 path: half of the keys hug their parent and stay with it
    (child index -1), the others move to a child; a refined parent keeps the stay residual."""
    x = synth.generate(wl)
    g = np.random.default_rng(wl.seed)
    for b in range(wl.B):
        for h in range(wl.H):
            near = x["Cp"][h][g.integers(0, wl.M, wl.N // 2)] + 0.05 * g.standard_normal((wl.N // 2, wl.d))
            x["K"][b, h, ::2] = synth.round_to_bf16(near.astype(np.float32))[: len(x["K"][b, h, ::2])]
    rep = parity.full_parity(wl, flags=binding.FLAG_PARENT_STAYS, parent_stays=True, x=x)
    print("stays", rep)
    total = wl.B * wl.H * wl.N
    assert 0.3 * total <= rep["stay_count"] <= 0.7 * total        # a real mixture of stayed and moved keys
    # and the two rules really differ on this input
    gpu_rep = parity.gpu_forward(wl, x, flags=0)
    gpu_st = parity.gpu_forward(wl, x, flags=binding.FLAG_PARENT_STAYS)
    assert (gpu_rep["child_idx"] >= 0).all() and (gpu_st["child_idx"] < 0).any()
    assert np.abs(gpu_rep["Y"] - gpu_st["Y"]).max() > 1e-3


def test_tensor_core_and_cuda_core_paths_agree_at_full_size():
    wl = synth.C3.with_(H=4)
    dv = parity.to_device(synth.generate(wl), "bf16")
    args = (dv["Q"], dv["K"], dv["V"], dv["Cp"], dv["Cc"], wl.P, wl.block_q)
    Yt, St, Wt, It = binding.forward(*args, scale=wl.scale, aux=True)
    Ys, Ss, Ws, Is = binding.forward(*args, scale=wl.scale, flags=binding.FLAG_SIMT, aux=True)
    assert torch.equal(It["parent_idx"], Is["parent_idx"]) and torch.equal(It["child_idx"], Is["child_idx"])
    assert torch.equal(It["np"], Is["np"]) and torch.equal(It["nc"], Is["nc"])
    same = (St == Ss).all(dim=-1)
    assert same.float().mean() > 0.99                      # selections may differ only at near-ties
    rows = same.repeat_interleave(wl.block_q, dim=-1)
    diff = (Yt.float() - Ys.float()).abs()[rows]
    assert diff.max() <= 2e-2


@pytest.mark.parametrize("H,N,d,M,C", [(2, 40001, 64, 32, 4), (2, 80003, 128, 32, 8), (16, 16384, 64, 64, 4),
                                       (1, 1300000, 64, 256, 8)])
def test_aggregate_long_heads_few_leaves(H, N, d, M, C):
    """avq_aggregate where every leaf collects many keys (the chunked, leaf-ordered variant), ragged
    lengths, skewed and empty leaves: counts exact, sums within fp32 accumulation error of the oracle."""
    from oracle import avq_oracle as orc
    g = np.random.default_rng(100 + N)
    V = synth.round_to_bf16(g.standard_normal((1, H, N, d)).astype(np.float32))
    # skewed leaves: a few popular ones, some never used
    pm = g.dirichlet(np.full(M, 0.3))
    pidx = g.choice(M, size=(1, H, N), p=pm).astype(np.int32)
    cidx = np.minimum(g.geometric(0.5, size=(1, H, N)) - 1, C - 1).astype(np.int32)
    dev = dict(V=torch.from_numpy(V).cuda().to(torch.bfloat16), p=torch.from_numpy(pidx).cuda(),
               c=torch.from_numpy(cidx).cuda())
    Vp, n_p, Vc, n_c = binding.aggregate(dev["V"], dev["p"], dev["c"], M, C)
    torch.cuda.synchronize()
    for h in range(H):
        rVp, rnp, rVc, rnc = orc.aggregate_head(V[0, h], pidx[0, h], cidx[0, h], M, C)
        assert np.array_equal(n_p[0, h].cpu().numpy(), rnp)
        assert np.array_equal(n_c[0, h].cpu().numpy(), rnc)
        scale = 1e-6 * np.sqrt(np.maximum(rnc, 1.0))[..., None] * 50 + 1e-5 * np.abs(rVc)
        assert (np.abs(Vc[0, h].cpu().numpy() - rVc) <= scale + 1e-4).all()
        assert np.allclose(Vp[0, h].cpu().numpy(), rVp, rtol=2e-5, atol=2e-3)


def _random_shapes(n, seed):
    g = np.random.default_rng(seed)
    out = []
    for i in range(n):
        d = int(g.choice([64, 128]))
        C = int(g.choice([4, 8]))
        M = int(g.choice([32, 64, 96, 128, 160, 256]))
        P = int(g.choice([0, 1, M // 8, M // 4, M]))
        H = int(g.integers(1, 4))
        B = int(g.integers(1, 3))
        N = int(g.integers(129, 1400))
        out.append(synth.Workload(f"rnd{i}", B=B, H=H, N=N, d=d, M=M, C=C, P=P, block_q=128, seed=500 + i,
                                  alpha=float(g.choice([0.3, 0.8])), hot_queries=bool(g.integers(0, 2))))
    return out


@pytest.mark.parametrize("wl", _random_shapes(12, seed=20261), ids=lambda w: f"{w.name}-B{w.B}H{w.H}N{w.N}d{w.d}M{w.M}C{w.C}P{w.P}")
def test_random_shapes_full_parity(wl):
    """Seeded random shapes inside the tensor-core envelope (ragged lengths, every d, C, several M and P,
    endpoints included): every stage against the oracle, whole tensors."""
    parity.full_parity(wl)


def test_long_ragged_head_uses_chunked_aggregate_end_to_end():
    """A ragged long head over few leaves (the chunked aggregate inside avq_forward), sampled against the oracle."""
    wl = synth.sweep_point(16384, 32, 4).with_(H=2, N=16384 + 77, name="ragged_long")
    parity.sampled_parity(wl, heads=[(0, 1)], blocks_per_head=4)


def test_degenerate_all_keys_on_one_codeword():
    """Every key equals one parent codeword: that parent holds all keys, every other parent is empty, the
    importances are zero but one, and the top-P set is that parent plus the lowest-index empty ones (the
    tie rule across a whole group of equal importances); empty children must not disturb the maxima."""
    wl = synth.C1.with_(B=1, H=2, N=512, seed=41)
    x = synth.generate(wl)
    for h in range(wl.H):
        x["K"][0, h, :, :] = x["Cp"][h, 5]
    rep = parity.full_parity(wl, x=x)
    assert rep["empty_parents"] == wl.H * (wl.M - 1)
    assert rep["topp_flips_excused"] == 0


def test_single_query_block_shorter_than_a_tile_and_tiny_key_set():
    """Nq = 1 and Nk = 5: one ragged query tile, one ragged key tile, almost every codeword empty."""
    wl = synth.C1.with_(B=1, H=1, N=5, seed=43)
    x = synth.generate(wl)
    x["Q"] = np.ascontiguousarray(x["Q"][:, :, :1])
    parity.full_parity(wl, x=x)


def test_chained_tiles_with_several_child_chunks():
    """More tiles than one wave of CTAs (every CTA takes several tiles in a row) with every parent refined, so
    that each tile runs through several child chunks before the next tile's loads are issued."""
    parity.sampled_parity(synth.sweep_point(16384, 64, 64), heads=[(0, 7)], blocks_per_head=4)
    parity.sampled_parity(synth.sweep_point(16384, 256, 64).with_(H=4), heads=[(0, 2)], blocks_per_head=3)
