"""Pins for the oracle's codebook update (appendix "Codeword Clustering During Training"), CPU only.

The projection is pinned by what defines it - feasibility, the Lagrange condition of the mass-weighted
least-squares problem, an independent numerical solver, closed-form special cases - and the EMA step by
scalar loops."""
import numpy as np
import pytest
from scipy import optimize

from oracle import avq_oracle as orc


def _case(seed, B=2, H=2, N=60, d=3, M=4, C=3):
    g = np.random.default_rng(seed)
    Cp = g.normal(size=(H, M, d)) * 2
    Cc = Cp[:, :, None, :] + 0.6 * g.normal(size=(H, M, C, d))
    K = Cc[np.arange(H)[None, :, None], g.integers(0, M, (B, H, N)), g.integers(0, C, (B, H, N))] \
        + 0.3 * g.normal(size=(B, H, N, d))
    Sp = g.normal(size=(H, M, d))
    Np = g.uniform(0.5, 3.0, size=(H, M))
    Sc = g.normal(size=(H, M, C, d))
    Nc = g.uniform(0.2, 2.0, size=(H, M, C))
    return K, Cp, Cc, Sp, Np, Sc, Nc


@pytest.mark.parametrize("parent_stays", [False, True])
def test_children_average_to_their_parent_and_satisfy_the_lagrange_condition(parent_stays):
    K, Cp, Cc, Sp, Np, Sc, Nc = _case(0)
    out = orc.codebook_update(K, Cp, Cc, Sp, Np, Sc, Nc, decay=0.9, parent_stays=parent_stays)
    np.testing.assert_allclose(out["Cc"].mean(axis=2), out["Cp"], atol=1e-12)
    # stationarity of sum_c N_c |M_c - C_c|^2 + mu . (sum_c C_c - C * C_p): N_c (C_c - M_c) is the same for every c
    Mc = out["Sc"] / out["Nc"][..., None]
    g = out["Nc"][..., None] * (out["Cc"] - Mc)
    np.testing.assert_allclose(g, np.broadcast_to(g[:, :, :1], g.shape), atol=1e-12)
    np.testing.assert_allclose(out["Cp"], out["Sp"] / out["Np"][..., None], atol=0)


def test_projection_agrees_with_a_numerical_constrained_solver():
    K, Cp, Cc, Sp, Np, Sc, Nc = _case(1, B=1, H=1, N=40, d=2, M=2, C=3)
    out = orc.codebook_update(K, Cp, Cc, Sp, Np, Sc, Nc, decay=0.5)
    for m in range(2):
        Mc = out["Sc"][0, m] / out["Nc"][0, m][:, None]
        w = out["Nc"][0, m]
        target = out["Cp"][0, m]
        obj = lambda x: float((w[:, None] * (x.reshape(3, 2) - Mc) ** 2).sum())
        con = dict(type="eq", fun=lambda x: x.reshape(3, 2).mean(axis=0) - target)
        res = optimize.minimize(obj, Mc.ravel(), constraints=[con], method="SLSQP",
                                options=dict(ftol=1e-14, maxiter=500))
        assert res.success
        np.testing.assert_allclose(res.x.reshape(3, 2), out["Cc"][0, m], atol=1e-6)


def test_ema_statistics_against_scalar_loops_and_kmeans_limit():
    K, Cp, Cc, Sp, Np, Sc, Nc = _case(2, B=2, H=1, N=30, d=2, M=3, C=2)
    lam = 0.75
    out = orc.codebook_update(K, Cp, Cc, Sp, Np, Sc, Nc, decay=lam)
    sums = np.zeros((3, 2)); cnts = np.zeros(3); csums = np.zeros((3, 2, 2)); ccnts = np.zeros((3, 2))
    for b in range(2):
        for j in range(30):
            k = K[b, 0, j]
            a = min(range(3), key=lambda m: (sum((k - Cp[0, m]) ** 2), m))
            c = min(range(2), key=lambda c_: (sum((k - Cc[0, a, c_]) ** 2), c_))
            sums[a] += k; cnts[a] += 1; csums[a, c] += k; ccnts[a, c] += 1
    np.testing.assert_allclose(out["Sp"][0], lam * Sp[0] + (1 - lam) * sums, atol=1e-12)
    np.testing.assert_allclose(out["Np"][0], lam * Np[0] + (1 - lam) * cnts, atol=1e-12)
    np.testing.assert_allclose(out["Sc"][0], lam * Sc[0] + (1 - lam) * csums, atol=1e-12)
    np.testing.assert_allclose(out["Nc"][0], lam * Nc[0] + (1 - lam) * ccnts, atol=1e-12)
    # decay 0 forgets the history: a parent that received keys moves to their centroid (one k-means step)
    out0 = orc.codebook_update(K, Cp, Cc, Sp, Np, Sc, Nc, decay=0.0)
    live = cnts > 0
    np.testing.assert_allclose(out0["Cp"][0][live], sums[live] / cnts[live][:, None], atol=1e-12)


def test_closed_form_special_cases():
    # equal child masses: every child is shifted by the same delta / C; means that already average to the
    # parent are left alone; a child without mass keeps its position as its mean and takes the whole residual
    H, M, C, d = 1, 1, 4, 2
    Cp = np.zeros((H, M, d)); Cc = np.arange(8.0).reshape(H, M, C, d)
    K = np.zeros((1, H, 0, d))                                   # no new keys: statistics only decay
    Sp = np.array([[[2.0, 4.0]]]); Np = np.array([[2.0]])
    Mc = np.array([[0.0, 0.0], [2.0, 0.0], [0.0, 2.0], [6.0, 2.0]])
    Nc = np.full((H, M, C), 2.0); Sc = (Mc * 2.0)[None, None]
    out = orc.codebook_update(K, Cp, Cc, Sp, Np, Sc, Nc, decay=0.5)
    np.testing.assert_allclose(out["Cp"][0, 0], [1.0, 2.0])
    delta = Mc.sum(axis=0) - 4 * np.array([1.0, 2.0])            # (4, -4)
    np.testing.assert_allclose(out["Cc"][0, 0], Mc - delta / 4, atol=1e-12)
    Sp2 = np.array([[[4.0, 2.0]]])                               # parent mean (2, 1) = mean of the child means
    out = orc.codebook_update(K, Cp, Cc, Sp2, Np, Sc, Nc, decay=0.5)
    np.testing.assert_allclose(out["Cc"][0, 0], Mc, atol=1e-12)
    Nc0 = Nc.copy(); Nc0[0, 0, 3] = 0.0; Sc0 = Sc.copy(); Sc0[0, 0, 3] = 0.0
    out = orc.codebook_update(K, Cp, Cc, Sp, Np, Sc0, Nc0, decay=0.5)
    np.testing.assert_allclose(out["Cc"][0, 0][:3], Mc[:3], atol=1e-4)          # the massive children barely move
    np.testing.assert_allclose(out["Cc"][0, 0].mean(axis=0), [1.0, 2.0], atol=1e-9)
