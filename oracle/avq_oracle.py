"""fp64 CPU oracle for the AVQ-attention forward pass.  TEST INFRASTRUCTURE ONLY.

This file is the yardstick the CUDA library is checked against.  It is plain,
slow numpy in float64, written from the paper's definitions; it shares no code
with the CUDA path and must never be imported by the product package.  Only the
test-suite, the smoke check and the benchmark's CPU-baseline leg may call it.

What each function follows in the paper:

* ``assign_head``      - Sec. 3.2 (VQ assignment, ``a(K_j) = argmin_a ||C_a - K_j||^2``)
                         and Algorithm 1 (parent argmin, then the children of the
                         chosen parent scanned upward with a strict ``<``).
* ``aggregate_head``   - Eq. "aggregates" (``n_a`` counts, ``Vbar_a`` value SUMS) and
                         the two scatter steps of Algorithm 1.
* ``importance_block`` - Eq. "vqflashattention" + Eq. "importance" and Algorithm 2's
                         parent pass, with the non-empty-only maximum of the appendix on
                         numerical stability.
* ``top_p``            - "Child spawning": the P most important parents of a query tile.
* ``forward_block_dense``      - the definition: ordinary softmax attention
                         (Eq. "standardattention") over the block's effective key set, where
                         a key is represented by its child codeword if its parent was
                         selected for that block (and the key moved to a child), else by
                         its parent codeword ("quantised-key attention", Sec. 3.2).
* ``forward_block_correcting`` - Algorithm 2's child pass as printed (mean-recovered parent logit,
                         Eq. "parent_recovery"; Delta A updates, Eq. "correcting_attention").
* ``forward_block_factorised`` - the O(M N) regrouped form of the same quantity
                         (Sec. 3.2 regrouping + the post-refinement sum of the appendix
                         "Correcting Attention Derivation": ``A_p Vbar_stay + sum_c A_c Vbar_c``).

* ``importance_block_tiled`` - appendix "Computing Importance with Tiled Codewords": the parents are
                         visited in tiles; a tile's importances use the denominator seen so far,
                         extrapolated by key counts (Eq. "aproxdenom", Eq. "codewordimportance").
* ``capture``          - the fraction of a block's TRUE attention mass (exact softmax over the
                         original keys) that falls on keys of the selected parents (the measure of
                         Table "tiled_capture").
* ``codebook_update``  - appendix "Codeword Clustering During Training": EMA statistics of the
                         keys assigned to every parent and child, parents moved to their EMA mean,
                         children to the mass-weighted projection of their EMA means onto the
                         parent = mean(children) constraint (Eq. "child_constraint_solve").

Two child-assignment rules are implemented.  REPLACE (default): every key goes
to the nearest child of its parent.  PARENT_STAYS (Algorithm 1's masked scatter):
a key moves to that child only if it is strictly closer than the parent.

Readings taken where the paper is silent: ties go to the lowest index
everywhere; the logit scale is an explicit argument; the importance denominator
is the exact parent-pass one; query blocks are contiguous ranges of ``block_q``
queries inside one (batch, head), the last one may be short.

``codebook_update`` reading where the paper is silent: a code whose EMA mass is (still) zero keeps
its previous position as its "unconstrained mean" and enters the projection with a mass floor of
``mass_floor`` (it has no data to resist the displacement, so it absorbs the residual).

Pins (tests/test_oracle_*.py): brute-force loops on tiny inputs, closed forms,
conservation laws, the exact-attention special case checked against
``torch.nn.functional.scaled_dot_product_attention``, and Algorithm 2 re-derived
literally (mean-recovered parent logits + correcting attention) on codebooks
that satisfy the parent = mean(children) constraint.
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


# --------------------------------------------------------------------------- assignment
def _two_smallest(D: np.ndarray):
    """Smallest and second smallest entry of every row (second = +inf for one column)."""
    if D.shape[1] == 1:
        return D[:, 0].copy(), np.full(D.shape[0], np.inf)
    part = np.partition(D, 1, axis=1)
    return part[:, 0], part[:, 1]


def _rel_margin(d1: np.ndarray, d2: np.ndarray) -> np.ndarray:
    """(d2 - d1) / d2 with 0/0 counted as a tie (margin 0) and d2 = inf as margin 1."""
    out = np.ones_like(d1)
    fin = np.isfinite(d2)
    pos = fin & (d2 > 0)
    out[pos] = (d2[pos] - d1[pos]) / d2[pos]
    out[fin & ~(d2 > 0)] = 0.0
    return out


def assign_head(K, Cp, Cc, parent_stays: bool = False, chunk: int = 1024):
    """Nearest parent, then nearest child of that parent, for the keys of one head.

    K [N,d], Cp [M,d], Cc [M,C,d].  Distances are the direct form
    ``sum_k (K_jk - C_ak)^2`` in float64 (Sec. 3.2; Algorithm 1 parent and child steps).

    Returns a dict:
      parent_idx [N] int64           - argmin over parents, lowest index on ties
      child_idx  [N] int64           - argmin over the C children of that parent, lowest
                                       index on ties; -1 where the key stays with the parent
                                       (only possible with ``parent_stays``)
      d_parent, d_child [N]          - the winning squared distances
      parent_margin, child_margin    - relative gap best vs runner-up, (d2-d1)/d2
      stay_margin                    - relative gap between child and parent distance
                                       (only meaningful with ``parent_stays``)
    """
    K = np.asarray(K, dtype=F64)
    Cp = np.asarray(Cp, dtype=F64)
    Cc = np.asarray(Cc, dtype=F64)
    N, d = K.shape
    M, C, _ = Cc.shape
    parent_idx = np.empty(N, dtype=np.int64)
    child_idx = np.empty(N, dtype=np.int64)
    d_parent = np.empty(N)
    d_child = np.empty(N)
    parent_margin = np.empty(N)
    child_margin = np.empty(N)
    for j0 in range(0, N, chunk):
        j1 = min(N, j0 + chunk)
        k = K[j0:j1]
        diff = k[:, None, :] - Cp[None, :, :]
        Dp = (diff * diff).sum(axis=2)                       # [n, M]
        a = np.argmin(Dp, axis=1)                            # first minimum = lowest index
        d1, d2 = _two_smallest(Dp)
        parent_idx[j0:j1] = a
        d_parent[j0:j1] = d1
        parent_margin[j0:j1] = _rel_margin(d1, d2)
        diffc = k[:, None, :] - Cc[a]                        # [n, C, d]
        Dc = (diffc * diffc).sum(axis=2)                     # [n, C]
        c = np.argmin(Dc, axis=1)
        e1, e2 = _two_smallest(Dc)
        child_idx[j0:j1] = c
        d_child[j0:j1] = e1
        child_margin[j0:j1] = _rel_margin(e1, e2)
    hi = np.maximum(d_child, d_parent)
    stay_margin = np.where(hi > 0, np.abs(d_child - d_parent) / np.where(hi > 0, hi, 1.0), 0.0)
    if parent_stays:
        moved = d_child < d_parent                           # strict, Algorithm 1's masked scatter
        child_idx = np.where(moved, child_idx, -1)
    return dict(parent_idx=parent_idx, child_idx=child_idx, d_parent=d_parent, d_child=d_child,
                parent_margin=parent_margin, child_margin=child_margin, stay_margin=stay_margin)


# --------------------------------------------------------------------------- aggregation
def aggregate_head(V, parent_idx, child_idx, M: int, C: int):
    """Per-codeword value sums and key counts for one head (Eq. "aggregates", Algorithm 1).

    Parents collect every key assigned to them; child (m, c) collects the keys
    with ``parent_idx == m`` and ``child_idx == c`` (keys with child_idx -1 stay).
    Returns Vp [M,d], np [M], Vc [M,C,d], nc [M,C] in float64.
    """
    V = np.asarray(V, dtype=F64)
    N, d = V.shape
    Vp = np.zeros((M, d))
    n_p = np.zeros(M)
    Vc = np.zeros((M, C, d))
    n_c = np.zeros((M, C))
    np.add.at(Vp, parent_idx, V)
    np.add.at(n_p, parent_idx, 1.0)
    moved = child_idx >= 0
    np.add.at(Vc, (parent_idx[moved], child_idx[moved]), V[moved])
    np.add.at(n_c, (parent_idx[moved], child_idx[moved]), 1.0)
    return Vp, n_p, Vc, n_c


# --------------------------------------------------------------------------- importance, top-P
def importance_block(Qb, Cp, n_p, scale: float):
    """Per-parent importance of one query block (Eq. "importance"; Algorithm 2 parent pass).

    ``s = scale * Qb Cp^T``; the row maximum runs over non-empty parents only;
    ``A = exp(s - m)`` with empty parents zeroed; ``z_i = sum_j A_ij n_j``;
    ``w_j = sum_i A_ij n_j / z_i``.  Returns (w [M], s [bq,M], m [bq], z [bq]).
    """
    Qb = np.asarray(Qb, dtype=F64)
    Cp = np.asarray(Cp, dtype=F64)
    n_p = np.asarray(n_p, dtype=F64)
    s = scale * (Qb @ Cp.T)
    live = n_p > 0
    m = np.max(np.where(live[None, :], s, -np.inf), axis=1)
    A = np.where(live[None, :], np.exp(s - m[:, None]), 0.0)
    z = A @ n_p
    w = ((A * n_p[None, :]) / z[:, None]).sum(axis=0)
    return w, s, m, z


def importance_block_tiled(Qb, Cp, n_p, scale: float, tile_m: int, n_keys: float | None = None):
    """Importance when the parents are visited in tiles of ``tile_m`` codewords, in index order
    (appendix "Computing Importance with Tiled Codewords").

    After tiles ``t <= J`` the denominator of row i is known only over the visited codewords,
    ``Zpart_i(J) = sum_{t<=J} sum_{j in t} A_ij n_j``; it is extrapolated by key counts,
    ``Ztilde_i(J) = N / N_seen(J) * Zpart_i(J)`` (Eq. "aproxdenom"), and the codewords of tile J get
    ``w_j = sum_i A_ij n_j / Ztilde_i(J)`` (Eq. "codewordimportance").  The ratio does not depend on the
    stabiliser, so the plain row maximum over non-empty parents is used.  A tile reached before any key has
    been seen holds only empty parents: their importance is 0.  ``n_keys`` defaults to ``sum(n_p)``.
    """
    Qb = np.asarray(Qb, dtype=F64)
    Cp = np.asarray(Cp, dtype=F64)
    n_p = np.asarray(n_p, dtype=F64)
    M = n_p.shape[0]
    N = float(n_p.sum()) if n_keys is None else float(n_keys)
    s = scale * (Qb @ Cp.T)
    live = n_p > 0
    m = np.max(np.where(live[None, :], s, -np.inf), axis=1)
    An = np.where(live[None, :], np.exp(s - m[:, None]), 0.0) * n_p[None, :]     # A_ij n_j
    w = np.zeros(M)
    zpart = np.zeros(Qb.shape[0])
    n_seen = 0.0
    for j0 in range(0, M, tile_m):
        j1 = min(M, j0 + tile_m)
        zpart = zpart + An[:, j0:j1].sum(axis=1)
        n_seen += float(n_p[j0:j1].sum())
        if n_seen > 0:
            ztilde = (N / n_seen) * zpart
            w[j0:j1] = (An[:, j0:j1] / ztilde[:, None]).sum(axis=0)
    return w


def capture(Qb, K, parent_idx, selected, scale: float) -> float:
    """Share of the block's true attention mass on the keys whose parent is in ``selected``: exact softmax of
    the block's queries over the ORIGINAL keys, summed over those keys and averaged over the queries."""
    Qb = np.asarray(Qb, dtype=F64)
    K = np.asarray(K, dtype=F64)
    s = scale * (Qb @ K.T)
    s -= s.max(axis=1, keepdims=True)
    E = np.exp(s)
    E /= E.sum(axis=1, keepdims=True)
    hit = np.isin(parent_idx, np.asarray(selected, dtype=np.int64))
    return float(E[:, hit].sum(axis=1).mean())


def exact_selection(Qb, K, parent_idx, M: int, P: int, scale: float):
    """The P parents whose keys receive the most true attention mass from the block (the "exact" column of
    Table "tiled_capture"), ascending."""
    Qb = np.asarray(Qb, dtype=F64)
    K = np.asarray(K, dtype=F64)
    s = scale * (Qb @ K.T)
    s -= s.max(axis=1, keepdims=True)
    E = np.exp(s)
    E /= E.sum(axis=1, keepdims=True)
    mass = np.zeros(M)
    np.add.at(mass, parent_idx, E.sum(axis=0))
    return top_p(mass, P)[0]


def top_p(w, P: int):
    """Indices of the P largest importances, lowest index first among equals.

    Returns (selected indices ascending [P], relative margin between the P-th and
    (P+1)-th importance; 1.0 when P is 0 or M, 0.0 for 0/0).
    """
    w = np.asarray(w, dtype=F64)
    M = w.shape[0]
    order = np.argsort(-w, kind="stable")
    sel = np.sort(order[:P])
    if P <= 0 or P >= M:
        return sel, 1.0
    a, b = w[order[P - 1]], w[order[P]]
    margin = (a - b) / a if a > 0 else 0.0
    return sel, float(margin)


# --------------------------------------------------------------------------- forward, one block
def effective_keys(Cp, Cc, parent_idx, child_idx, selected):
    """Codeword that represents each key for a block whose refined parents are ``selected``."""
    Cp = np.asarray(Cp, dtype=F64)
    Cc = np.asarray(Cc, dtype=F64)
    is_sel = np.zeros(Cp.shape[0], dtype=bool)
    is_sel[np.asarray(selected, dtype=np.int64)] = True
    use_child = is_sel[parent_idx] & (child_idx >= 0)
    Khat = Cp[parent_idx].copy()
    Khat[use_child] = Cc[parent_idx[use_child], child_idx[use_child]]
    return Khat


def forward_block_dense(Qb, V, Cp, Cc, parent_idx, child_idx, selected, scale: float):
    """Softmax attention of a query block over its effective key set, O(bq * N * d).

    Eq. "standardattention" with K_j replaced by the block's effective codeword of key j.
    """
    Qb = np.asarray(Qb, dtype=F64)
    V = np.asarray(V, dtype=F64)
    Khat = effective_keys(Cp, Cc, parent_idx, child_idx, selected)
    s = scale * (Qb @ Khat.T)
    s -= s.max(axis=1, keepdims=True)
    E = np.exp(s)
    return (E @ V) / E.sum(axis=1, keepdims=True)


def forward_block_factorised(Qb, Cp, Cc, Vp, n_p, Vc, n_c, selected, scale: float):
    """The same output through per-codeword aggregates, O(bq * (M + P C) * d).

    Unselected parent p contributes ``e^{s_p} (Vp_p, n_p)``.  A selected parent
    contributes its stay residual ``e^{s_p} (Vp_p - sum_c Vc_pc, n_p - sum_c n_pc)``
    plus ``e^{s_pc} (Vc_pc, n_pc)`` for each child.  Empty codewords are skipped.
    """
    Qb = np.asarray(Qb, dtype=F64)
    Cp = np.asarray(Cp, dtype=F64)
    Cc = np.asarray(Cc, dtype=F64)
    M, C, d = Cc.shape
    selected = np.asarray(selected, dtype=np.int64)
    is_sel = np.zeros(M, dtype=bool)
    is_sel[selected] = True
    V_stay = Vp - Vc.sum(axis=1)
    n_stay = n_p - n_c.sum(axis=1)
    codes = [Cp[~is_sel], Cp[is_sel], Cc[is_sel].reshape(-1, d)]
    vals = [Vp[~is_sel], V_stay[is_sel], Vc[is_sel].reshape(-1, d)]
    cnts = [n_p[~is_sel], n_stay[is_sel], n_c[is_sel].reshape(-1)]
    codes, vals, cnts = np.concatenate(codes), np.concatenate(vals), np.concatenate(cnts)
    live = cnts > 0
    codes, vals, cnts = codes[live], vals[live], cnts[live]
    s = scale * (Qb @ codes.T)
    s -= s.max(axis=1, keepdims=True)
    A = np.exp(s)
    return (A @ vals) / (A @ cnts)[:, None]


def forward_block_correcting(Qb, Cp, Cc, Vp, n_p, Vc, n_c, selected, scale: float):
    """Algorithm 2's child pass as printed: every parent keeps its full term ``e^{s_p} (Vp_p, n_p)``; for a
    selected parent the logit is RECOVERED as the mean of its children's logits (Eq. "parent_recovery") and
    each non-empty child adds ``(e^{s_pc} - e^{s_p,rec}) (Vc_pc, n_pc)`` (Eq. "correcting_attention").
    Equals ``forward_block_factorised`` when every parent is the mean of its children."""
    Qb = np.asarray(Qb, dtype=F64)
    Cp = np.asarray(Cp, dtype=F64)
    Cc = np.asarray(Cc, dtype=F64)
    selected = np.asarray(selected, dtype=np.int64)
    s_p = scale * (Qb @ Cp.T)                                     # [bq, M]
    s_c = scale * np.einsum("id,pcd->ipc", Qb, Cc[selected])      # [bq, P, C]
    s_rec = s_c.mean(axis=2)                                      # recovered parent logits
    live_p = n_p > 0
    live_c = n_c[selected] > 0
    m = np.max(np.where(live_p[None, :], s_p, -np.inf), axis=1)
    if selected.size:
        m = np.maximum(m, np.max(np.where(live_c[None], s_c, -np.inf), axis=(1, 2)))
    A_p = np.where(live_p[None, :], np.exp(s_p - m[:, None]), 0.0)
    X = A_p @ Vp
    Z = A_p @ n_p
    dA = np.where(live_c[None], np.exp(s_c - m[:, None, None]) - np.exp(s_rec - m[:, None])[:, :, None], 0.0)
    X = X + np.einsum("ipc,pcd->id", dA, Vc[selected])
    Z = Z + np.einsum("ipc,pc->i", dA, n_c[selected])
    return X / Z[:, None]


# --------------------------------------------------------------------------- forward, one head / all heads
def forward_head(Q, K, V, Cp, Cc, P: int, block_q: int, scale: float, parent_stays: bool = False,
                 form: str = "dense", blocks=None, assignment=None, tile_m: int | None = None):
    """AVQ-attention forward for one (batch, head).

    Q [Nq,d], K,V [Nk,d], Cp [M,d], Cc [M,C,d].  ``form`` is "dense" (definition) or
    "factorised".  ``blocks`` optionally restricts the evaluation to some query-block
    indices (rows of other blocks are left NaN).  ``assignment`` may carry a
    previously computed ``assign_head`` result for these keys.  ``tile_m`` switches the selection to the
    tiled importance (the output is still exact for the parents that selection refines).

    Returns a dict: Y [Nq,d]; selected [nblk,P] (ascending, -1 rows for skipped
    blocks); importance [nblk,M]; topp_margin [nblk]; plus the assignment dict and
    the aggregates (Vp, np, Vc, nc).
    """
    Q = np.asarray(Q, dtype=F64)
    V = np.asarray(V, dtype=F64)
    Cp64 = np.asarray(Cp, dtype=F64)
    Cc64 = np.asarray(Cc, dtype=F64)
    Nq, d = Q.shape
    M, C, _ = Cc64.shape
    asg = assignment if assignment is not None else assign_head(K, Cp64, Cc64, parent_stays)
    pidx, cidx = asg["parent_idx"], asg["child_idx"]
    Vp, n_p, Vc, n_c = aggregate_head(V, pidx, cidx, M, C)
    nblk = (Nq + block_q - 1) // block_q
    Y = np.full((Nq, d), np.nan)
    selected = np.full((nblk, P), -1, dtype=np.int64)
    importance = np.full((nblk, M), np.nan)
    margins = np.ones(nblk)
    todo = range(nblk) if blocks is None else blocks
    for t in todo:
        i0, i1 = t * block_q, min(Nq, (t + 1) * block_q)
        Qb = Q[i0:i1]
        if tile_m is None:
            w, _, _, _ = importance_block(Qb, Cp64, n_p, scale)
        else:
            w = importance_block_tiled(Qb, Cp64, n_p, scale, tile_m, n_keys=float(np.asarray(K).shape[0]))
        sel, mg = top_p(w, P)
        importance[t] = w
        selected[t] = sel
        margins[t] = mg
        if form == "dense":
            Y[i0:i1] = forward_block_dense(Qb, V, Cp64, Cc64, pidx, cidx, sel, scale)
        elif form == "factorised":
            Y[i0:i1] = forward_block_factorised(Qb, Cp64, Cc64, Vp, n_p, Vc, n_c, sel, scale)
        elif form == "correcting":
            Y[i0:i1] = forward_block_correcting(Qb, Cp64, Cc64, Vp, n_p, Vc, n_c, sel, scale)
        else:
            raise ValueError(form)
    return dict(Y=Y, selected=selected, importance=importance, topp_margin=margins, assignment=asg,
                Vp=Vp, np=n_p, Vc=Vc, nc=n_c)


def forward(Q, K, V, Cp, Cc, P: int, block_q: int, scale: float, parent_stays: bool = False,
            form: str = "dense", tile_m: int | None = None):
    """All (batch, head) pairs.  Q,K,V [B,H,N,d]; Cp [H,M,d]; Cc [H,M,C,d] (one codebook per head)."""
    B, H = Q.shape[:2]
    res = [[forward_head(Q[b, h], K[b, h], V[b, h], Cp[h], Cc[h], P, block_q, scale, parent_stays, form,
                         tile_m=tile_m)
            for h in range(H)] for b in range(B)]

    def stack(key):
        return np.stack([np.stack([res[b][h][key] for h in range(H)]) for b in range(B)])

    out = {k: stack(k) for k in ("Y", "selected", "importance", "topp_margin", "Vp", "np", "Vc", "nc")}
    for k in ("parent_idx", "child_idx", "parent_margin", "child_margin", "stay_margin"):
        out[k] = np.stack([np.stack([res[b][h]["assignment"][k] for h in range(H)]) for b in range(B)])
    return out


# --------------------------------------------------------------------------- codebook update (training)
def codebook_update(K, Cp, Cc, Sp, Np, Sc, Nc, decay: float, parent_stays: bool = False,
                    mass_floor: float = 1e-6):
    """One codebook update from a batch of keys (appendix "Codeword Clustering During Training").

    K [B,H,N,d]; Cp [H,M,d], Cc [H,M,C,d] the current codebooks (one per head, shared over the batch);
    Sp [H,M,d], Np [H,M], Sc [H,M,C,d], Nc [H,M,C] the EMA statistics before the update.

    1. keys are assigned with the current codebooks (``assign_head``); a parent collects every key assigned
       to it, a child the keys that moved to it;
    2. ``S <- decay * S + (1 - decay) * sum of the code's keys``, ``N <- decay * N + (1 - decay) * count``;
    3. parents: ``Cp' = Sp / Np``; children: unconstrained means ``Mc = Sc / Nc``, then
       ``Cc' = Mc - delta / (Nc * sigma)`` with ``delta = sum_c Mc - C * Cp'`` and ``sigma = sum_c 1 / Nc``
       (Eq. "child_constraint_solve"), which restores ``mean_c Cc' = Cp'``.

    Returns a dict with the new Sp, Np, Sc, Nc, Cp, Cc (float64).
    """
    K = np.asarray(K, dtype=F64)
    Cp = np.asarray(Cp, dtype=F64)
    Cc = np.asarray(Cc, dtype=F64)
    B, H, N, d = K.shape
    M, C = Cc.shape[1], Cc.shape[2]
    sum_p = np.zeros((H, M, d))
    cnt_p = np.zeros((H, M))
    sum_c = np.zeros((H, M, C, d))
    cnt_c = np.zeros((H, M, C))
    for b in range(B):
        for h in range(H):
            a = assign_head(K[b, h], Cp[h], Cc[h], parent_stays)
            kp, n_p, kc, n_c = aggregate_head(K[b, h], a["parent_idx"], a["child_idx"], M, C)
            sum_p[h] += kp
            cnt_p[h] += n_p
            sum_c[h] += kc
            cnt_c[h] += n_c
    Sp2 = decay * np.asarray(Sp, dtype=F64) + (1.0 - decay) * sum_p
    Np2 = decay * np.asarray(Np, dtype=F64) + (1.0 - decay) * cnt_p
    Sc2 = decay * np.asarray(Sc, dtype=F64) + (1.0 - decay) * sum_c
    Nc2 = decay * np.asarray(Nc, dtype=F64) + (1.0 - decay) * cnt_c
    has_p = Np2 > mass_floor
    Cp2 = np.where(has_p[..., None], Sp2 / np.where(has_p, Np2, 1.0)[..., None], Cp)
    has_c = Nc2 > mass_floor
    Mc = np.where(has_c[..., None], Sc2 / np.where(has_c, Nc2, 1.0)[..., None], Cc)
    mass = np.maximum(Nc2, mass_floor)
    delta = Mc.sum(axis=2) - C * Cp2                                  # [H,M,d]
    sigma = (1.0 / mass).sum(axis=2)                                  # [H,M]
    Cc2 = Mc - delta[:, :, None, :] / (mass * sigma[:, :, None])[..., None]
    return dict(Sp=Sp2, Np=Np2, Sc=Sc2, Nc=Nc2, Cp=Cp2, Cc=Cc2)
