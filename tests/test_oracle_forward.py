"""Pins for the oracle's forward pass (CPU only).

The paper prints no worked numeric example, so the forward is pinned by
(1) a hand-built case whose answer is written out with ``math.exp``,
(2) scalar brute force on tiny random inputs,
(3) special cases that collapse to ordinary attention, checked against torch's
    ``scaled_dot_product_attention`` (a routine the oracle does not use),
(4) Algorithm 2 executed literally (online-softmax merge, parent logits recovered
    as the mean of the child logits, correcting attention) on codebooks that obey
    the parent = mean(children) constraint,
(5) symmetries: key permutation, codeword relabelling.
"""
import math

import numpy as np
import pytest
import torch

from oracle import avq_oracle as orc
from paper_2607_12789_b200 import synth


def _sdpa(Q, K, V, scale):
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.float64))[None, None]
    return torch.nn.functional.scaled_dot_product_attention(t(Q), t(K), t(V), scale=scale)[0, 0].numpy()


# ---------------------------------------------------------------- (1) closed form
def test_hand_built_case_all_P():
    Cp = np.array([[2.0, 0.5], [-2.0, 0.25]])
    Cc = np.array([[[2.5, 0.5], [1.5, 0.75]], [[-1.5, 0.25], [-2.5, 0.0]]])
    K = np.array([[2.6, 0.5], [1.4, 0.8], [-2.2, 0.1]])       # -> (p0,c0) (p0,c1) (p1,c1)
    V = np.array([[1.0, -1.0], [10.0, 0.5], [100.0, 2.0]])
    Q = np.array([[1.0, 2.0], [-0.5, 1.0]])
    sc = 0.5
    a = orc.assign_head(K, Cp, Cc)
    assert a["parent_idx"].tolist() == [0, 0, 1] and a["child_idx"].tolist() == [0, 1, 1]

    def logit(q, c):
        return sc * (q[0] * c[0] + q[1] * c[1])

    def expect(reps):     # reps[j] = codeword standing in for key j
        out = []
        for q in Q:
            e = [math.exp(logit(q, r)) for r in reps]
            out.append([sum(e[j] * V[j][k] for j in range(3)) / sum(e) for k in range(2)])
        return np.array(out)

    # importance of parent 0 for the single block of two queries
    w0 = sum(2 * math.exp(logit(q, Cp[0])) / (2 * math.exp(logit(q, Cp[0])) + math.exp(logit(q, Cp[1])))
             for q in Q)
    res = {P: orc.forward_head(Q, K, V, Cp, Cc, P, 2, sc) for P in (0, 1, 2)}
    assert res[1]["importance"][0, 0] == pytest.approx(w0, rel=1e-13)
    assert w0 > 1.0                                      # parent 0 is the more important one
    assert res[1]["selected"][0].tolist() == [0]
    np.testing.assert_allclose(res[0]["Y"], expect([Cp[0], Cp[0], Cp[1]]), rtol=1e-13)
    np.testing.assert_allclose(res[1]["Y"], expect([Cc[0, 0], Cc[0, 1], Cp[1]]), rtol=1e-13)
    np.testing.assert_allclose(res[2]["Y"], expect([Cc[0, 0], Cc[0, 1], Cc[1, 1]]), rtol=1e-13)
    for P in (0, 1, 2):
        f = orc.forward_head(Q, K, V, Cp, Cc, P, 2, sc, form="factorised")
        np.testing.assert_allclose(f["Y"], res[P]["Y"], rtol=1e-13)


# ---------------------------------------------------------------- (2) scalar brute force
def _brute_forward(Q, K, V, Cp, Cc, P, bq, sc, parent_stays):
    N, d = K.shape
    M, C, _ = Cc.shape
    dist = lambda x, y: sum((x[k] - y[k]) ** 2 for k in range(d))
    dot = lambda x, y: sum(x[k] * y[k] for k in range(d))
    par, chi = [], []
    for j in range(N):
        dp = [dist(K[j], Cp[m]) for m in range(M)]
        a = dp.index(min(dp))
        dc = [dist(K[j], Cc[a, c]) for c in range(C)]
        c = dc.index(min(dc))
        if parent_stays and not (dc[c] < dp[a]):
            c = -1
        par.append(a)
        chi.append(c)
    Y = np.zeros((Q.shape[0], d))
    sels = []
    for i0 in range(0, Q.shape[0], bq):
        rows = range(i0, min(Q.shape[0], i0 + bq))
        w = [0.0] * M
        for i in rows:                                  # mass each parent receives = sum over its keys
            e = [math.exp(sc * dot(Q[i], Cp[par[j]])) for j in range(N)]
            for j in range(N):
                w[par[j]] += e[j] / sum(e)
        sel = sorted(sorted(range(M), key=lambda m: (-w[m], m))[:P])
        sels.append(sel)
        for i in rows:
            e = []
            for j in range(N):
                rep = Cc[par[j], chi[j]] if (par[j] in sel and chi[j] >= 0) else Cp[par[j]]
                e.append(math.exp(sc * dot(Q[i], rep)))
            for k in range(d):
                Y[i, k] = sum(e[j] * V[j, k] for j in range(N)) / sum(e)
    return Y, sels


@pytest.mark.parametrize("seed,P,parent_stays", [(0, 0, False), (1, 1, False), (2, 2, False), (3, 4, False),
                                                 (4, 2, True), (5, 1, True)])
def test_forward_matches_scalar_bruteforce(seed, P, parent_stays):
    g = np.random.default_rng(seed)
    N, M, C, d, bq = 14, 4, 2, 3, 5
    Cp = g.normal(size=(M, d)) * 1.5
    Cc = Cp[:, None, :] + 0.8 * g.normal(size=(M, C, d))
    K = Cp[g.integers(0, M, N)] + 0.6 * g.normal(size=(N, d))
    V, Q = g.normal(size=(N, d)), g.normal(size=(N, d))
    want, sels = _brute_forward(Q, K, V, Cp, Cc, P, bq, 0.9, parent_stays)
    for form in ("dense", "factorised"):
        got = orc.forward_head(Q, K, V, Cp, Cc, P, bq, 0.9, parent_stays=parent_stays, form=form)
        np.testing.assert_allclose(got["Y"], want, rtol=1e-11, atol=1e-13)
        assert [s.tolist() for s in got["selected"]] == sels


# ---------------------------------------------------------------- (3) collapse to ordinary attention
def test_keys_equal_to_codewords_give_exact_attention():
    x = synth.generate(synth.C0)
    Q, V, Cp, Cc = x["Q"][0, 0], x["V"][0, 0], x["Cp"][0], x["Cc"][0]
    g = np.random.default_rng(0)
    pj, cj = g.integers(0, 16, 256), g.integers(0, 4, 256)
    K = Cp[pj]                                            # keys sit on parents: P=0 is exact
    got = orc.forward_head(Q, K, V, Cp, Cc, 0, 64, 0.125)
    np.testing.assert_allclose(got["Y"], _sdpa(Q, K, V, 0.125), rtol=1e-10, atol=1e-12)
    K = Cc[pj, cj]                                        # keys sit on children: P=M is exact
    got = orc.forward_head(Q, K, V, Cp, Cc, 16, 64, 0.125)
    np.testing.assert_allclose(got["Y"], _sdpa(Q, K, V, 0.125), rtol=1e-10, atol=1e-12)
    part = orc.forward_head(Q, K, V, Cp, Cc, 2, 64, 0.125)   # P=2 is then NOT exact
    assert np.abs(part["Y"] - got["Y"]).max() > 1e-3


@pytest.mark.parametrize("form", ["dense", "factorised"])
def test_endpoints_are_flat_vq_attention(form):
    """P=0: attention over keys quantised to parents.  P=M: over keys quantised to the tree's leaf."""
    x = synth.generate(synth.C0)
    Q, K, V, Cp, Cc = x["Q"][0, 0], x["K"][0, 0], x["V"][0, 0], x["Cp"][0], x["Cc"][0]
    a = orc.assign_head(K, Cp, Cc)
    y0 = orc.forward_head(Q, K, V, Cp, Cc, 0, 64, 0.125, form=form)["Y"]
    np.testing.assert_allclose(y0, _sdpa(Q, Cp[a["parent_idx"]], V, 0.125), rtol=1e-10, atol=1e-12)
    yM = orc.forward_head(Q, K, V, Cp, Cc, 16, 64, 0.125, form=form)["Y"]
    np.testing.assert_allclose(yM, _sdpa(Q, Cc[a["parent_idx"], a["child_idx"]], V, 0.125), rtol=1e-10,
                               atol=1e-12)


def test_all_keys_identical_returns_mean_value():
    g = np.random.default_rng(2)
    Cp = g.normal(size=(3, 4)) * 3
    Cc = Cp[:, None, :] + 0.3 * g.normal(size=(3, 2, 4))
    K = np.repeat(Cp[1:2] + 0.01, 9, axis=0)
    V, Q = g.normal(size=(9, 4)), g.normal(size=(5, 4))
    for P in (0, 1, 3):
        y = orc.forward_head(Q, K, V, Cp, Cc, P, 4, 1.0)["Y"]
        np.testing.assert_allclose(y, np.repeat(V.mean(axis=0)[None], 5, axis=0), rtol=1e-12)


# ---------------------------------------------------------------- (4) Algorithm 2, literally
def _algorithm2(Qb, Cp, Cc, Vp, n_p, Vc, n_c, P, sc):
    """Parent pass, importance, top-P, then one online-softmax merge per selected parent in
    which the parent's logit is the mean of its children's logits and the accumulators
    are updated with exp(s_c - m) - exp(s_p - m)."""
    s = sc * Qb @ Cp.T
    live = n_p > 0
    m = np.where(live[None], s, -np.inf).max(axis=1)
    A = np.where(live[None], np.exp(s - m[:, None]), 0.0)
    xbar = A @ Vp
    zbar = A @ n_p
    w = (A * n_p[None] / zbar[:, None]).sum(axis=0)
    S = np.argsort(-w, kind="stable")[:P]
    for p in S:
        s_c = sc * Qb @ Cc[p].T
        live_c = n_c[p] > 0
        m_new = np.maximum(m, np.where(live_c[None], s_c, -np.inf).max(axis=1))
        xbar *= np.exp(m - m_new)[:, None]
        zbar *= np.exp(m - m_new)
        m = m_new
        s_p = s_c.mean(axis=1)
        dA = np.exp(s_c - m[:, None]) - np.exp(s_p - m)[:, None]
        dA[:, ~live_c] = 0.0
        xbar += dA @ Vc[p]
        zbar += dA @ n_c[p]
    return xbar / zbar[:, None], np.sort(S)


@pytest.mark.parametrize("parent_stays", [False, True])
@pytest.mark.parametrize("P", [0, 2, 5, 16])
def test_algorithm2_literal_on_constrained_codebook(P, parent_stays):
    w = synth.C0.with_(recenter_children=True, seed=4)
    x = {k: v.astype(np.float64) for k, v in synth.generate(w).items()}
    Cc = x["Cc"][0] - x["Cc"][0].mean(axis=1, keepdims=True) + x["Cp"][0][:, None]   # exact in fp64
    Q, K, V, Cp = x["Q"][0, 0], x["K"][0, 0], x["V"][0, 0], x["Cp"][0]
    if parent_stays:
        K = K.copy()
        K[::3] = Cp[np.arange(0, 256, 3) % 16] + 0.05 * K[::3]
    res = orc.forward_head(Q, K, V, Cp, Cc, P, 64, 0.125, parent_stays=parent_stays)
    if parent_stays:
        assert (res["assignment"]["child_idx"] < 0).sum() > 50
    for t in range(4):
        y, S = _algorithm2(Q[t * 64:(t + 1) * 64], Cp, Cc, res["Vp"], res["np"], res["Vc"], res["nc"], P, 0.125)
        assert S.tolist() == res["selected"][t].tolist()
        np.testing.assert_allclose(y, res["Y"][t * 64:(t + 1) * 64], rtol=1e-9, atol=1e-11)


def test_mean_recovery_needs_the_constraint():
    """Without re-centred children the literal algorithm is visibly off; the definition is not."""
    x = {k: v.astype(np.float64) for k, v in synth.generate(synth.C0).items()}
    Q, K, V, Cp, Cc = x["Q"][0, 0], x["K"][0, 0], x["V"][0, 0], x["Cp"][0], x["Cc"][0]
    res = orc.forward_head(Q, K, V, Cp, Cc, 2, 64, 0.125)
    y, _ = _algorithm2(Q[:64], Cp, Cc, res["Vp"], res["np"], res["Vc"], res["nc"], 2, 0.125)
    assert np.abs(y - res["Y"][:64]).max() > 1e-3


# ---------------------------------------------------------------- (5) symmetries, forms, ragged tail
@pytest.mark.parametrize("wl", [synth.C0, synth.C1.with_(B=1, H=1, N=640), synth.C2.with_(B=1, H=1, N=512)])
def test_dense_equals_factorised_on_benchmark_like_data(wl):
    x = synth.generate(wl)
    a = orc.forward_head(x["Q"][0, 0], x["K"][0, 0], x["V"][0, 0], x["Cp"][0], x["Cc"][0], wl.P, wl.block_q,
                         wl.scale, form="dense")
    b = orc.forward_head(x["Q"][0, 0], x["K"][0, 0], x["V"][0, 0], x["Cp"][0], x["Cc"][0], wl.P, wl.block_q,
                         wl.scale, form="factorised", assignment=a["assignment"])
    np.testing.assert_allclose(a["Y"], b["Y"], rtol=1e-9, atol=1e-12)
    assert np.array_equal(a["selected"], b["selected"])


def test_key_permutation_and_codeword_relabelling_leave_output_unchanged():
    x = synth.generate(synth.C0)
    Q, K, V, Cp, Cc = x["Q"][0, 0], x["K"][0, 0], x["V"][0, 0], x["Cp"][0], x["Cc"][0]
    ref = orc.forward_head(Q, K, V, Cp, Cc, 3, 64, 0.125)
    g = np.random.default_rng(1)
    perm = g.permutation(256)
    got = orc.forward_head(Q, K[perm], V[perm], Cp, Cc, 3, 64, 0.125)
    np.testing.assert_allclose(got["Y"], ref["Y"], rtol=1e-11, atol=1e-13)
    assert np.array_equal(got["selected"], ref["selected"])
    rel = g.permutation(16)                               # new parent m is old parent rel[m]
    got = orc.forward_head(Q, K, V, Cp[rel], Cc[rel][:, ::-1], 3, 64, 0.125)
    np.testing.assert_allclose(got["Y"], ref["Y"], rtol=1e-11, atol=1e-13)
    for t in range(4):
        assert sorted(rel[got["selected"][t]].tolist()) == ref["selected"][t].tolist()
    assert np.array_equal(rel[got["assignment"]["parent_idx"]], ref["assignment"]["parent_idx"])
    assert np.array_equal(3 - got["assignment"]["child_idx"], ref["assignment"]["child_idx"])


def test_ragged_last_block_and_nq_differs_from_nk():
    x = synth.generate(synth.C0)
    Q, K, V, Cp, Cc = x["Q"][0, 0][:150], x["K"][0, 0], x["V"][0, 0], x["Cp"][0], x["Cc"][0]
    res = orc.forward_head(Q, K, V, Cp, Cc, 2, 64, 0.125)
    assert res["Y"].shape == (150, 64) and res["selected"].shape == (3, 2)
    assert abs(res["importance"][2].sum() - 22.0) < 1e-9           # 150 = 64 + 64 + 22
    tail = orc.forward_head(Q[128:], K, V, Cp, Cc, 2, 64, 0.125)
    np.testing.assert_allclose(res["Y"][128:], tail["Y"], rtol=1e-12)
    only = orc.forward_head(Q, K, V, Cp, Cc, 2, 64, 0.125, blocks=[1])
    np.testing.assert_allclose(only["Y"][64:128], res["Y"][64:128], rtol=0, atol=0)
    assert np.isnan(only["Y"][:64]).all()


def test_batched_forward_uses_one_codebook_per_head():
    wl = synth.C0.with_(B=2, H=2, N=128, seed=8)
    x = synth.generate(wl)
    out = orc.forward(x["Q"], x["K"], x["V"], x["Cp"], x["Cc"], 2, 64, 0.125)
    assert out["Y"].shape == (2, 2, 128, 64)
    one = orc.forward_head(x["Q"][1, 0], x["K"][1, 0], x["V"][1, 0], x["Cp"][0], x["Cc"][0], 2, 64, 0.125)
    np.testing.assert_array_equal(out["Y"][1, 0], one["Y"])
    assert np.array_equal(out["parent_idx"][1, 0], one["assignment"]["parent_idx"])


def test_benchmark_generator_structure():
    """The structure the input recipe promises: nobody stays, no assignment near-ties, empties exist."""
    x = synth.generate(synth.C1.with_(B=1, H=2))
    for h in range(2):
        rep = orc.assign_head(x["K"][0, h], x["Cp"][h], x["Cc"][h])
        stay = orc.assign_head(x["K"][0, h], x["Cp"][h], x["Cc"][h], parent_stays=True)
        assert (stay["child_idx"] < 0).sum() == 0
        assert rep["parent_margin"].min() > 0.3
    for k, v in x.items():
        assert np.array_equal(synth.round_to_bf16(v), v), k          # already bf16-representable
    y = synth.generate(synth.C1.with_(B=1, H=2))
    assert all(np.array_equal(x[k], y[k]) for k in x)                 # seeded, reproducible


@pytest.mark.parametrize("parent_stays", [False, True])
def test_correcting_form_equals_the_definition_exactly_when_parents_are_child_means(parent_stays):
    """Algorithm 2 as printed (mean-recovered logit, Delta A) against the dense definition: equal on codebooks
    that satisfy parent = mean(children) in float64, visibly different on codebooks that do not."""
    g = np.random.default_rng(17)
    M, C, d, N = 10, 3, 5, 150
    Cp = g.normal(size=(M, d)) * 2
    Cc = Cp[:, None, :] + 0.5 * g.normal(size=(M, C, d))
    Cc_ok = Cc - Cc.mean(axis=1, keepdims=True) + Cp[:, None, :]
    K = np.concatenate([Cc_ok[g.integers(0, M, N // 2), g.integers(0, C, N // 2)] + 0.2 * g.normal(size=(N // 2, d)),
                        Cp[g.integers(0, M, N - N // 2)] + 0.05 * g.normal(size=(N - N // 2, d))])
    Q, V = g.normal(size=(N, d)), g.normal(size=(N, d))
    dense = orc.forward_head(Q, K, V, Cp, Cc_ok, 4, 50, 0.6, parent_stays=parent_stays, form="dense")
    corr = orc.forward_head(Q, K, V, Cp, Cc_ok, 4, 50, 0.6, parent_stays=parent_stays, form="correcting")
    np.testing.assert_allclose(corr["Y"], dense["Y"], atol=1e-12)
    if parent_stays:
        assert (dense["assignment"]["child_idx"] < 0).any()
    bad = orc.forward_head(Q, K, V, Cp, Cc, 4, 50, 0.6, parent_stays=parent_stays, form="correcting")
    good = orc.forward_head(Q, K, V, Cp, Cc, 4, 50, 0.6, parent_stays=parent_stays, form="dense")
    assert np.abs(bad["Y"] - good["Y"]).max() > 1e-3
