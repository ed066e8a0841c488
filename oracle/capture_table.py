"""Top-P capture on synthetic data: tiled importance vs exact importance vs exact selection.

Reproduces the COMPARISON of Table "tiled_capture" (appendix "Computing Importance with Tiled Codewords") on the
seeded synthetic generator (the paper's datasets and trained models are not available): for every query
block, the share of the true attention mass (exact softmax over the original keys) that falls on the keys
of the P parents chosen by (a) the tiled importance with the count-extrapolated denominator, (b) the
importance with the exact denominator, (c) the parents that truly receive the most mass.
CPU only; calls nothing but the oracle and the input generator.

    python -m oracle.capture_table
"""
from __future__ import annotations

import numpy as np

from oracle import avq_oracle as orc
from paper_2607_12789_b200 import synth


def capture_rows(M: int, C: int, P: int, tile_m: int, N: int = 4096, H: int = 2, seed: int = 700):
    wl = synth.Workload(f"cap_M{M}", B=1, H=H, N=N, d=64, M=M, C=C, P=P, block_q=128, seed=seed + M, alpha=0.3,
                        hot_queries=True)
    x = synth.generate(wl)
    caps = dict(tiled=[], nontiled=[], exact=[])
    for h in range(H):
        asg = orc.assign_head(x["K"][0, h], x["Cp"][h], x["Cc"][h])
        _, n_p, _, _ = orc.aggregate_head(x["V"][0, h], asg["parent_idx"], asg["child_idx"], M, C)
        for t in range(N // wl.block_q):
            Qb = x["Q"][0, h][t * 128:(t + 1) * 128]
            w_t = orc.importance_block_tiled(Qb, x["Cp"][h], n_p, wl.scale, tile_m, n_keys=N)
            w_e, _, _, _ = orc.importance_block(Qb, x["Cp"][h], n_p, wl.scale)
            sels = dict(tiled=orc.top_p(w_t, P)[0], nontiled=orc.top_p(w_e, P)[0],
                        exact=orc.exact_selection(Qb, x["K"][0, h], asg["parent_idx"], M, P, wl.scale))
            for k, sel in sels.items():
                caps[k].append(orc.capture(Qb, x["K"][0, h], asg["parent_idx"], sel, wl.scale))
    return {k: float(np.mean(v)) for k, v in caps.items()}


def main():
    print("| M | C | P | tile | tiled | non-tiled | exact |")
    print("|---|---|---|---|---|---|---|")
    for M, C, P, tile in ((256, 8, 24, 128), (256, 8, 32, 128), (512, 4, 32, 128), (512, 4, 64, 128),
                          (1024, 4, 64, 256), (1024, 4, 128, 256)):
        r = capture_rows(M, C, P, tile)
        print(f"| {M} | {C} | {P} | {tile} | {100 * r['tiled']:.1f} % | {100 * r['nontiled']:.1f} % | "
              f"{100 * r['exact']:.1f} % |", flush=True)


if __name__ == "__main__":
    main()
