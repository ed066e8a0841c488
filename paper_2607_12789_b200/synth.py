"""Seeded synthetic inputs for AVQ-attention (queries, keys, values, hierarchical codebook).

This module draws random arrays and nothing else: it contains none of the
method's arithmetic (no distances, assignments, softmax or aggregation), so
both the CUDA tests and the CPU oracle tests can consume its output.

Recipe (one numpy ``Generator(PCG64(seed))``, arrays drawn in this order):

1. parents   ``Cp[H, M, d]      = parent_scale * N(0, 1)``
2. children  ``Cc[H, M, C, d]   = Cp[:, :, None] + sigma_c * N(0, 1)``
   (optionally re-centred so each parent is the mean of its children, the
   constraint of Eq. "parent_constraint")
3. cluster weights ``pi[B, H, M]``: uniform, or ``Dirichlet(alpha)`` per (b, h)
4. keys: parent ``~ Categorical(pi)``, child uniform in ``0..C-1``,
   ``K = Cc[h, parent, child] + sigma_k * N(0, 1)``
5. queries: ``N(0, 1)``, or "hot": each (b, h) picks ``ceil(0.1 M)`` parents,
   every query sits at one of them plus ``sigma_q * N(0, 1)``
6. values ``V = N(0, 1)``

Everything is returned as float32; for a bf16 workload every array has already
been rounded to the nearest bf16 value (ties to even), so widening it to fp64
for a CPU check or narrowing it to bf16 for the GPU loses nothing.
"""
from __future__ import annotations

import dataclasses
import math

import numpy as np


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    B: int
    H: int
    N: int
    d: int
    M: int
    C: int
    P: int
    block_q: int
    dtype: str = "bf16"            # "f32" or "bf16"
    seed: int = 0
    alpha: float | None = None     # Dirichlet concentration of the parent weights; None = uniform
    hot_queries: bool = False      # queries drawn near a random 10 % of the parents
    parent_scale: float = 3.0
    sigma_c: float = 0.5           # child spread around the parent
    sigma_k: float = 0.3           # key spread around its child
    sigma_q: float = 1.0           # query spread around a hot parent
    recenter_children: bool = False
    keys_around_parents: bool = False   # adversarial: keys sit at parents, not children

    @property
    def scale(self) -> float:
        return 1.0 / math.sqrt(self.d)

    def with_(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


# The five benchmark configurations (tiny fp32; ViT-B-like; mid-length; long; sweep).
C0 = Workload("c0_tiny_f32", B=1, H=1, N=256, d=64, M=16, C=4, P=2, block_q=64, dtype="f32", seed=0)
C1 = Workload("c1_vitb", B=8, H=12, N=1024, d=64, M=64, C=4, P=8, block_q=128, seed=1, alpha=0.5)
C2 = Workload("c2_mid", B=2, H=16, N=4096, d=64, M=128, C=8, P=16, block_q=128, seed=2, alpha=0.3,
              hot_queries=True)
C3 = Workload("c3_long", B=1, H=16, N=16384, d=128, M=256, C=4, P=32, block_q=128, seed=3, alpha=0.3,
              hot_queries=True, sigma_c=0.4 * 3.0)

SWEEP_N = (1024, 4096, 16384, 65536)
SWEEP_M = (32, 64, 128, 256)


def sweep_point(N: int, M: int, P: int) -> Workload:
    """One point of the sweep: B=1, H=16, d=64, C=4, query block 128, bf16.

    All P values of one (N, M) share a seed, hence the same data, so P=0 and P=M
    are the two endpoints of one instance.
    """
    seed = 1000 + 4 * SWEEP_N.index(N) + SWEEP_M.index(M)
    return Workload(f"c4_N{N}_M{M}_P{P}", B=1, H=16, N=N, d=64, M=M, C=4, P=P, block_q=128, seed=seed,
                    alpha=0.3, hot_queries=True)


def sweep_P(M: int) -> tuple[int, ...]:
    return (0, M // 8, M // 4, M)


NAMED = {"c0": C0, "c1": C1, "c2": C2, "c3": C3}


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 (ties to even); result stays float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = (u + np.uint32(0x7FFF) + lsb) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def generate(w: Workload) -> dict[str, np.ndarray]:
    """Draw Q, K, V [B,H,N,d], Cp [H,M,d], Cc [H,M,C,d] for a workload (float32 arrays)."""
    g = np.random.Generator(np.random.PCG64(w.seed))
    B, H, N, d, M, C = w.B, w.H, w.N, w.d, w.M, w.C
    f32 = np.float32

    Cp = (w.parent_scale * g.standard_normal((H, M, d))).astype(f32)
    Cc = (Cp[:, :, None, :] + w.sigma_c * g.standard_normal((H, M, C, d))).astype(f32)
    if w.recenter_children:
        Cc = (Cc - Cc.mean(axis=2, keepdims=True) + Cp[:, :, None, :]).astype(f32)

    if w.alpha is None:
        pi = np.full((B, H, M), 1.0 / M)
    else:
        pi = g.dirichlet(np.full(M, w.alpha), size=(B, H))
    cdf = np.cumsum(pi, axis=-1)
    cdf[..., -1] = 1.0
    u = g.random((B, H, N))
    pj = np.empty((B, H, N), dtype=np.int64)
    for b in range(B):
        for h in range(H):
            pj[b, h] = np.minimum(np.searchsorted(cdf[b, h], u[b, h], side="right"), M - 1)
    cj = g.integers(0, C, size=(B, H, N))

    K = np.empty((B, H, N, d), dtype=f32)
    for b in range(B):
        for h in range(H):
            centre = Cp[h, pj[b, h]] if w.keys_around_parents else Cc[h, pj[b, h], cj[b, h]]
            K[b, h] = centre + (w.sigma_k * g.standard_normal((N, d))).astype(f32)

    if w.hot_queries:
        n_hot = max(1, math.ceil(0.1 * M))
        Q = np.empty((B, H, N, d), dtype=f32)
        for b in range(B):
            for h in range(H):
                hot = g.choice(M, size=n_hot, replace=False)
                pick = hot[g.integers(0, n_hot, size=N)]
                Q[b, h] = Cp[h, pick] + (w.sigma_q * g.standard_normal((N, d))).astype(f32)
    else:
        Q = g.standard_normal((B, H, N, d)).astype(f32)

    V = g.standard_normal((B, H, N, d)).astype(f32)

    out = {"Q": Q, "K": K, "V": V, "Cp": Cp, "Cc": Cc}
    if w.dtype == "bf16":
        out = {k: round_to_bf16(v) for k, v in out.items()}
    return {k: np.ascontiguousarray(v) for k, v in out.items()}
