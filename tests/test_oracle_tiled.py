"""Pins for the oracle's tiled importance (appendix "Computing Importance with Tiled Codewords") and for the
capture measure (Table "tiled_capture"), CPU only."""
import math

import numpy as np
import pytest

from oracle import avq_oracle as orc


def _block(seed, rows=7, M=12, d=3):
    g = np.random.default_rng(seed)
    Qb = g.normal(size=(rows, d))
    Cp = g.normal(size=(M, d)) * 2
    n_p = g.integers(0, 6, size=M).astype(float)
    n_p[3] = 0
    n_p[0] = 4
    return Qb, Cp, n_p


def test_one_tile_is_the_exact_importance_and_the_last_tile_is_always_exact():
    Qb, Cp, n_p = _block(0)
    w_exact, _, _, _ = orc.importance_block(Qb, Cp, n_p, 0.7)
    np.testing.assert_allclose(orc.importance_block_tiled(Qb, Cp, n_p, 0.7, tile_m=12), w_exact, atol=1e-14)
    np.testing.assert_allclose(orc.importance_block_tiled(Qb, Cp, n_p, 0.7, tile_m=64), w_exact, atol=1e-14)
    w4 = orc.importance_block_tiled(Qb, Cp, n_p, 0.7, tile_m=4)
    np.testing.assert_allclose(w4[8:], w_exact[8:], atol=1e-14)      # N_seen = N for the last tile
    assert np.abs(w4[:8] - w_exact[:8]).max() > 1e-3                  # earlier tiles really are approximations
    assert w4[3] == 0.0


def test_tiled_importance_against_scalar_loops():
    Qb, Cp, n_p = _block(1, rows=5, M=10)
    scale, tile = 0.5, 4
    N = n_p.sum()
    want = np.zeros(10)
    for j in range(10):
        J = j // tile
        upto = min(10, (J + 1) * tile)
        n_seen = sum(n_p[:upto])
        for i in range(5):
            s = [scale * sum(Qb[i, k] * Cp[jj, k] for k in range(3)) for jj in range(10)]
            zpart = sum(math.exp(s[jj]) * n_p[jj] for jj in range(upto))
            if n_p[j] > 0:
                want[j] += math.exp(s[j]) * n_p[j] / (N / n_seen * zpart)
    np.testing.assert_allclose(orc.importance_block_tiled(Qb, Cp, n_p, scale, tile), want, rtol=1e-12)


def test_flat_attention_makes_the_extrapolation_exact():
    # all logits equal: every key gets the same weight, the part of the denominator seen so far is exactly
    # N_seen / N of the whole, and the tiled importance equals the exact one, |I| n_j / N
    g = np.random.default_rng(2)
    n_p = g.integers(1, 9, size=16).astype(float)
    Qb = np.zeros((6, 4))
    Cp = g.normal(size=(16, 4))
    w = orc.importance_block_tiled(Qb, Cp, n_p, 1.0, tile_m=4)
    np.testing.assert_allclose(w, 6 * n_p / n_p.sum(), rtol=1e-13)


def test_leading_tiles_of_empty_parents_get_zero_importance():
    Qb, Cp, n_p = _block(3, M=12)
    n_p[:4] = 0
    w = orc.importance_block_tiled(Qb, Cp, n_p, 0.7, tile_m=4)
    assert np.all(w[:4] == 0) and np.isfinite(w).all() and w[4:].sum() > 0


def test_capture_and_exact_selection_by_brute_force():
    g = np.random.default_rng(4)
    Qb, K = g.normal(size=(3, 2)), g.normal(size=(9, 2))
    pidx = np.array([0, 1, 2, 0, 1, 2, 3, 3, 3])
    mass = np.zeros(4)
    total = 0.0
    for i in range(3):
        e = [math.exp(0.9 * sum(Qb[i, k] * K[j, k] for k in range(2))) for j in range(9)]
        z = sum(e)
        for j in range(9):
            mass[pidx[j]] += e[j] / z
    assert orc.capture(Qb, K, pidx, [1, 3], 0.9) == pytest.approx((mass[1] + mass[3]) / 3, rel=1e-12)
    assert orc.capture(Qb, K, pidx, [0, 1, 2, 3], 0.9) == pytest.approx(1.0, rel=1e-12)
    assert orc.capture(Qb, K, pidx, [], 0.9) == 0.0
    best2 = sorted(np.argsort(-mass, kind="stable")[:2].tolist())
    assert orc.exact_selection(Qb, K, pidx, 4, 2, 0.9).tolist() == best2


def test_forward_with_tiles_changes_only_the_selection():
    g = np.random.default_rng(5)
    M, C, d, N = 24, 2, 4, 96
    Cp = g.normal(size=(M, d)) * 2
    Cc = Cp[:, None, :] + 0.4 * g.normal(size=(M, C, d))
    K = Cc[g.integers(0, M, N), g.integers(0, C, N)] + 0.2 * g.normal(size=(N, d))
    Q, V = g.normal(size=(N, d)), g.normal(size=(N, d))
    a = orc.forward_head(Q, K, V, Cp, Cc, 6, 32, 0.5, tile_m=8)
    b = orc.forward_head(Q, K, V, Cp, Cc, 6, 32, 0.5)
    c = orc.forward_head(Q, K, V, Cp, Cc, 6, 32, 0.5, tile_m=M)
    assert np.array_equal(b["selected"], c["selected"]) and np.allclose(b["Y"], c["Y"], atol=1e-14)
    for t in range(3):
        w = orc.importance_block_tiled(Q[32 * t:32 * t + 32], Cp, a["np"], 0.5, 8, n_keys=N)
        assert np.array_equal(a["selected"][t], orc.top_p(w, 6)[0])
        Yt = orc.forward_block_dense(Q[32 * t:32 * t + 32], V, Cp, Cc, a["assignment"]["parent_idx"],
                                     a["assignment"]["child_idx"], a["selected"][t], 0.5)
        np.testing.assert_allclose(a["Y"][32 * t:32 * t + 32], Yt, atol=1e-14)
