"""Pins for the oracle's assignment, aggregation, importance and top-P steps (CPU only).

Each test fixes the oracle to something that is not the oracle: scalar brute-force
loops on tiny inputs, constructed cases with a known answer, and conservation laws
that follow from Eq. "aggregates" and Eq. "importance".
"""
import math

import numpy as np
import pytest

from oracle import avq_oracle as orc
from paper_2607_12789_b200 import synth


def _tiny(seed, N=37, M=5, C=3, d=4):
    g = np.random.default_rng(seed)
    Cp = g.normal(size=(M, d)) * 2
    Cc = Cp[:, None, :] + 0.7 * g.normal(size=(M, C, d))
    K = g.normal(size=(N, d)) * 2
    V = g.normal(size=(N, d))
    Q = g.normal(size=(N, d))
    return Q, K, V, Cp, Cc


def _brute_assign(K, Cp, Cc, parent_stays):
    """Scalar loops: scan parents upward keeping the first strict minimum, then the children."""
    N, d = K.shape
    M, C, _ = Cc.shape
    pidx, cidx = [], []
    for j in range(N):
        best, a = math.inf, -1
        for m in range(M):
            dist = 0.0
            for k in range(d):
                dist += (K[j, k] - Cp[m, k]) ** 2
            if dist < best:
                best, a = dist, m
        bc, c_star = math.inf, -1
        for c in range(C):
            dist = 0.0
            for k in range(d):
                dist += (K[j, k] - Cc[a, c, k]) ** 2
            if dist < bc:
                bc, c_star = dist, c
        if parent_stays and not (bc < best):
            c_star = -1
        pidx.append(a)
        cidx.append(c_star)
    return np.array(pidx), np.array(cidx)


@pytest.mark.parametrize("seed", [0, 1, 2])
@pytest.mark.parametrize("parent_stays", [False, True])
def test_assign_matches_scalar_bruteforce(seed, parent_stays):
    _, K, _, Cp, Cc = _tiny(seed)
    got = orc.assign_head(K, Cp, Cc, parent_stays=parent_stays, chunk=8)
    pidx, cidx = _brute_assign(K, Cp, Cc, parent_stays)
    assert np.array_equal(got["parent_idx"], pidx)
    assert np.array_equal(got["child_idx"], cidx)


def test_keys_on_codewords_have_zero_distance_and_known_index():
    g = np.random.default_rng(5)
    M, C, d = 7, 4, 6
    Cp = g.normal(size=(M, d)) * 5
    Cc = Cp[:, None, :] + 0.2 * g.normal(size=(M, C, d))
    want_p = g.integers(0, M, size=50)
    want_c = g.integers(0, C, size=50)
    K = Cc[want_p, want_c]
    got = orc.assign_head(K, Cp, Cc)
    assert np.array_equal(got["parent_idx"], want_p)
    assert np.array_equal(got["child_idx"], want_c)
    assert np.all(got["d_child"] == 0.0)
    K = Cp[want_p]
    got = orc.assign_head(K, Cp, Cc, parent_stays=True)
    assert np.array_equal(got["parent_idx"], want_p)
    assert np.all(got["d_parent"] == 0.0)
    assert np.all(got["child_idx"] == -1)          # nothing is strictly closer than distance 0


def test_duplicate_codewords_pick_lowest_index_and_report_zero_margin():
    g = np.random.default_rng(6)
    d = 5
    base = g.normal(size=(3, d))
    Cp = np.stack([base[0], base[1], base[1], base[2], base[0]])        # 1==2, 0==4
    Cc = np.repeat(Cp[:, None, :], 3, axis=1) + 0.0                     # all children equal
    K = np.stack([base[1] + 0.01, base[0] - 0.01, base[2]])
    got = orc.assign_head(K, Cp, Cc)
    assert got["parent_idx"].tolist() == [1, 0, 3]
    assert got["child_idx"].tolist() == [0, 0, 0]
    assert got["parent_margin"][0] == 0.0 and got["parent_margin"][1] == 0.0
    assert got["parent_margin"][2] > 0.5
    assert np.all(got["child_margin"] == 0.0)


def test_midpoint_key_is_a_tie_resolved_to_lower_index():
    Cp = np.array([[1.0, 0.0], [-1.0, 0.0], [0.0, 50.0]])
    Cc = Cp[:, None, :] + np.array([[0.0, 0.5], [0.0, -0.5]])[None]
    K = np.array([[0.0, 0.0]])
    got = orc.assign_head(K, Cp, Cc)
    assert got["parent_idx"][0] == 0 and got["parent_margin"][0] == 0.0
    assert got["child_idx"][0] == 0 and got["child_margin"][0] == 0.0


def test_stay_margin_is_the_relative_gap_between_child_and_parent_distance():
    """One parent at the origin with children at x = 3 and x = -5 (1-d keys written out by hand):
    key 1.0 -> parent distance 1, nearest child distance 4, margin (4 - 1) / 4 = 0.75, the key stays;
    key 2.0 -> 4 vs 1, margin 0.75, the key moves; key 1.5 -> 2.25 vs 2.25: margin 0, strict '<' keeps
    it with the parent; key 0 on the parent -> 0 vs 9, margin 1."""
    Cp = np.array([[0.0]])
    Cc = np.array([[[3.0], [-5.0]]])
    K = np.array([[1.0], [2.0], [1.5], [0.0]])
    got = orc.assign_head(K, Cp, Cc, parent_stays=True)
    np.testing.assert_allclose(got["d_parent"], [1.0, 4.0, 2.25, 0.0], rtol=0, atol=0)
    np.testing.assert_allclose(got["d_child"], [4.0, 1.0, 2.25, 9.0], rtol=0, atol=0)
    np.testing.assert_allclose(got["stay_margin"], [0.75, 0.75, 0.0, 1.0], rtol=0, atol=1e-15)
    assert got["child_idx"].tolist() == [-1, 0, -1, -1]
    rep = orc.assign_head(K, Cp, Cc, parent_stays=False)
    assert rep["child_idx"].tolist() == [0, 0, 0, 0]
    np.testing.assert_allclose(rep["stay_margin"], got["stay_margin"])


def test_replace_and_parent_stays_differ_only_where_the_parent_is_closer():
    w = synth.C0.with_(keys_around_parents=True, sigma_k=0.05)
    x = synth.generate(w)
    K, Cp, Cc = x["K"][0, 0], x["Cp"][0], x["Cc"][0]
    rep = orc.assign_head(K, Cp, Cc, parent_stays=False)
    stay = orc.assign_head(K, Cp, Cc, parent_stays=True)
    assert np.array_equal(rep["parent_idx"], stay["parent_idx"])
    assert np.all(rep["child_idx"] >= 0)
    assert np.all(stay["child_idx"] == -1)            # keys hug the parents: every key stays
    # on the benchmark generator (keys around children) nobody stays, the two rules coincide
    x = synth.generate(synth.C0)
    K, Cp, Cc = x["K"][0, 0], x["Cp"][0], x["Cc"][0]
    rep = orc.assign_head(K, Cp, Cc, parent_stays=False)
    stay = orc.assign_head(K, Cp, Cc, parent_stays=True)
    assert np.array_equal(rep["child_idx"], stay["child_idx"])


@pytest.mark.parametrize("parent_stays", [False, True])
def test_aggregate_conservation(parent_stays):
    _, K, V, Cp, Cc = _tiny(11, N=200, M=6, C=3, d=5)
    K[:60] = Cp[np.arange(60) % 6] + 0.01 * K[:60]      # some keys that stay
    a = orc.assign_head(K, Cp, Cc, parent_stays=parent_stays)
    Vp, n_p, Vc, n_c = orc.aggregate_head(V, a["parent_idx"], a["child_idx"], 6, 3)
    assert n_p.sum() == 200
    np.testing.assert_allclose(Vp.sum(axis=0), V.sum(axis=0), rtol=0, atol=1e-12)
    if parent_stays:
        assert np.all(n_p - n_c.sum(axis=1) >= 0)
        assert (n_p - n_c.sum(axis=1)).sum() == np.count_nonzero(a["child_idx"] < 0) > 0
    else:
        assert np.array_equal(n_c.sum(axis=1), n_p)
        np.testing.assert_allclose(Vc.sum(axis=1), Vp, rtol=0, atol=1e-12)
    # per-bin check against an explicit python accumulation
    for m in range(6):
        rows = [j for j in range(200) if a["parent_idx"][j] == m]
        assert n_p[m] == len(rows)
        np.testing.assert_allclose(Vp[m], sum((V[j] for j in rows), np.zeros(5)), atol=1e-12)
        for c in range(3):
            rows_c = [j for j in rows if a["child_idx"][j] == c]
            assert n_c[m, c] == len(rows_c)
            np.testing.assert_allclose(Vc[m, c], sum((V[j] for j in rows_c), np.zeros(5)), atol=1e-12)


def test_importance_sums_to_block_size_and_vanishes_only_for_empty_parents():
    x = synth.generate(synth.C1.with_(B=1, H=2, N=512))
    for h in range(2):
        a = orc.assign_head(x["K"][0, h], x["Cp"][h], x["Cc"][h])
        n_p = np.bincount(a["parent_idx"], minlength=64).astype(float)
        assert (n_p == 0).any()                      # Dirichlet(0.5) leaves some parents empty
        for t in range(4):
            Qb = x["Q"][0, h, t * 128:(t + 1) * 128]
            w, s, m, z = orc.importance_block(Qb, x["Cp"][h], n_p, 0.125)
            assert abs(w.sum() - 128.0) < 1e-9       # each query's softmax mass over parents is 1
            assert np.array_equal(w == 0, n_p == 0)
            assert np.all(w >= 0)


def test_importance_against_scalar_loops():
    g = np.random.default_rng(3)
    bq, M, d = 6, 4, 3
    Qb, Cp = g.normal(size=(bq, d)), g.normal(size=(M, d))
    n_p = np.array([3.0, 0.0, 1.0, 5.0])
    w, _, _, _ = orc.importance_block(Qb, Cp, n_p, 0.7)
    want = [0.0] * M
    for i in range(bq):
        e = [math.exp(0.7 * sum(Qb[i, k] * Cp[j, k] for k in range(d))) * n_p[j] for j in range(M)]
        for j in range(M):
            want[j] += e[j] / sum(e)
    np.testing.assert_allclose(w, want, rtol=1e-12)


def test_top_p_bruteforce_and_ties():
    g = np.random.default_rng(9)
    for _ in range(20):
        w = g.random(11)
        w[g.integers(0, 11, size=3)] = 0.0
        for P in range(0, 12):
            sel, _ = orc.top_p(w, P)
            ranked = sorted(range(11), key=lambda j: (-w[j], j))[:P]
            assert sel.tolist() == sorted(ranked)
    sel, margin = orc.top_p(np.array([0.5, 0.9, 0.5, 0.5, 0.1]), 2)
    assert sel.tolist() == [0, 1] and margin == 0.0
    sel, margin = orc.top_p(np.array([0.0, 0.0, 1.0, 0.0]), 3)
    assert sel.tolist() == [0, 1, 2] and margin == 0.0
    assert orc.top_p(np.array([3.0, 1.0]), 0)[0].size == 0
    assert orc.top_p(np.array([3.0, 1.0]), 2)[0].tolist() == [0, 1]
    sel, margin = orc.top_p(np.array([4.0, 1.0, 2.0]), 1)
    assert sel.tolist() == [0] and margin == pytest.approx(0.5)
