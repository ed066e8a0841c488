"""Writes tests/golden/c0_oracle.json from the CPU oracle alone (never from the CUDA path).

The paper prints no worked numeric example, so this fixture pins nothing to the paper: it is a
regression guard that makes an unintended change of the oracle's arithmetic visible.  Run
``python tests/golden/make_golden.py`` after an intended change and say why in the commit."""
import hashlib
import json
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

from oracle import avq_oracle as orc  # noqa: E402
from paper_2607_12789_b200 import synth  # noqa: E402


def summary():
    wl = synth.C0
    x = synth.generate(wl)
    out = orc.forward(x["Q"], x["K"], x["V"], x["Cp"], x["Cc"], wl.P, wl.block_q, wl.scale)
    h = lambda a: hashlib.sha256(np.ascontiguousarray(a).tobytes()).hexdigest()[:16]
    return {
        "workload": wl.name,
        "parent_idx_sha": h(out["parent_idx"].astype(np.int32)),
        "child_idx_sha": h(out["child_idx"].astype(np.int32)),
        "np": out["np"][0, 0].astype(int).tolist(),
        "selected": out["selected"][0, 0].tolist(),
        "importance_block0": [round(float(v), 9) for v in out["importance"][0, 0, 0]],
        "Y_row0_first8": [round(float(v), 12) for v in out["Y"][0, 0, 0, :8]],
        "Y_abs_sum": round(float(np.abs(out["Y"]).sum()), 8),
    }


if __name__ == "__main__":
    with open(os.path.join(HERE, "c0_oracle.json"), "w") as f:
        json.dump(summary(), f, indent=1)
    print("written")
