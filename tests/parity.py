"""Shared helpers for the GPU parity tests: run the CUDA library on a seeded workload and
compare every stage boundary with the fp64 oracle, element by element."""
from __future__ import annotations

import numpy as np
import torch

from oracle import avq_oracle as orc
from paper_2607_12789_b200 import binding, synth

NEAR_TIE = 1e-6          # relative margin below which an index / selection flip is excused (and counted)
TOL = {"f32": dict(max_abs=1e-4, rel_l2=None), "bf16": dict(max_abs=2e-2, rel_l2=5e-3)}


def to_device(x: dict, dtype: str) -> dict:
    td = torch.float32 if dtype == "f32" else torch.bfloat16
    return {k: torch.from_numpy(v).to("cuda").to(td).contiguous() for k, v in x.items()}


def gpu_forward(wl: synth.Workload, x: dict, flags: int = 0, P: int | None = None):
    dv = to_device(x, wl.dtype)
    P = wl.P if P is None else P
    Y, topp, imp, inter = binding.forward(dv["Q"], dv["K"], dv["V"], dv["Cp"], dv["Cc"], P, wl.block_q,
                                          scale=wl.scale, flags=flags, aux=True)
    torch.cuda.synchronize()
    out = dict(Y=Y.float().cpu().numpy().astype(np.float64), selected=topp.cpu().numpy(),
               importance=imp.cpu().numpy())
    out.update({k: v.cpu().numpy() for k, v in inter.items()})
    return out


def compare_indices(gpu, ref, parent_stays: bool = False):
    """Bit-exact indices except where the oracle's own margin is a near-tie.  Returns counters.
    The child-versus-parent margin can excuse a flip only under the PARENT_STAYS rule: with the default
    rule the parent distance plays no part in the child index."""
    pm = gpu["parent_idx"] != ref["parent_idx"]
    p_excused = pm & (ref["parent_margin"] < NEAR_TIE)
    assert not (pm & ~p_excused).any(), f"{(pm & ~p_excused).sum()} parent mismatches outside near-ties"
    cm = (gpu["child_idx"] != ref["child_idx"]) & ~pm
    near = ref["child_margin"] < NEAR_TIE
    if parent_stays:
        near = near | (ref["stay_margin"] < NEAR_TIE)
    c_excused = cm & near
    assert not (cm & ~c_excused).any(), f"{(cm & ~c_excused).sum()} child mismatches outside near-ties"
    return dict(parent_flips_excused=int(p_excused.sum()), child_flips_excused=int(c_excused.sum()),
                parent_near_ties=int((ref["parent_margin"] < NEAR_TIE).sum()),
                child_near_ties=int((ref["child_margin"] < NEAR_TIE).sum()))


def compare_aggregates(gpu, ref, atol=2e-3):
    for k in ("np", "nc"):
        assert np.array_equal(gpu[k], ref[k]), k
    for k in ("Vp", "Vc"):
        err = np.abs(gpu[k] - ref[k]).max()
        assert err <= atol, (k, err)


def compare_selection(gpu, ref):
    """Top-P sets equal per block except where the P-th / (P+1)-th margin is a near-tie."""
    sel_g, sel_r = gpu["selected"], ref["selected"]
    assert sel_g.shape == sel_r.shape
    same = (sel_g == sel_r).all(axis=-1) if sel_g.shape[-1] else np.ones(sel_g.shape[:-1], bool)
    excused = ~same & (ref["topp_margin"] < NEAR_TIE)
    assert not (~same & ~excused).any(), f"{(~same & ~excused).sum()} blocks with a wrong top-P set"
    if sel_g.shape[-1] > 1:
        assert (np.diff(sel_g, axis=-1) > 0).all(), "top-P indices must be ascending"
    imp_ok = np.isclose(gpu["importance"], ref["importance"], rtol=2e-3, atol=2e-4)
    assert imp_ok.all(), np.abs(gpu["importance"] - ref["importance"]).max()
    return same, int(excused.sum())


def compare_output(Yg, Yr, dtype, row_mask=None):
    tol = TOL[dtype]
    if row_mask is not None:
        Yg, Yr = Yg[row_mask], Yr[row_mask]
    assert np.isfinite(Yg).all()
    max_abs = float(np.abs(Yg - Yr).max())
    rel_l2 = float(np.linalg.norm(Yg - Yr) / np.linalg.norm(Yr))
    assert max_abs <= tol["max_abs"], f"max-abs {max_abs:.3e} > {tol['max_abs']}"
    if tol["rel_l2"] is not None:
        assert rel_l2 <= tol["rel_l2"], f"rel-L2 {rel_l2:.3e} > {tol['rel_l2']}"
    return max_abs, rel_l2


def full_parity(wl: synth.Workload, flags: int = 0, P: int | None = None, parent_stays: bool = False, x=None):
    """Whole-tensor comparison of every stage; for sizes the oracle finishes in seconds."""
    x = synth.generate(wl) if x is None else x
    P = wl.P if P is None else P
    gpu = gpu_forward(wl, x, flags=flags, P=P)
    ref = orc.forward(x["Q"], x["K"], x["V"], x["Cp"], x["Cc"], P, wl.block_q, wl.scale,
                      parent_stays=parent_stays, form="dense")
    rep = compare_indices(gpu, ref, parent_stays=parent_stays)
    if rep["parent_flips_excused"] == 0 and rep["child_flips_excused"] == 0:
        compare_aggregates(gpu, ref)
    same, excused = compare_selection(gpu, ref)
    rep["topp_flips_excused"] = excused
    nq = x["Q"].shape[2]
    rows_ok = np.repeat(same, wl.block_q, axis=-1)[..., :nq]
    rep["max_abs"], rep["rel_l2"] = compare_output(gpu["Y"], ref["Y"], wl.dtype, rows_ok)
    rep["stay_count"] = int((ref["child_idx"] < 0).sum())
    rep["empty_parents"] = int((ref["np"] == 0).sum())
    return rep


def sampled_parity(wl: synth.Workload, heads, blocks_per_head: int = 8, flags: int = 0, seed: int = 0):
    """Full-size run on the GPU, oracle on a sample: whole heads for assignment and aggregates,
    a few query blocks per sampled head for importance, selection and output."""
    x = synth.generate(wl)
    gpu = gpu_forward(wl, x, flags=flags)
    g = np.random.default_rng(seed)
    nblk = (wl.N + wl.block_q - 1) // wl.block_q
    rep = dict(parent_flips_excused=0, child_flips_excused=0, topp_flips_excused=0, max_abs=0.0, rel_l2=0.0)
    num = den = 0.0
    for (b, h) in heads:
        blocks = sorted(g.choice(nblk, size=min(blocks_per_head, nblk), replace=False).tolist())
        ref = orc.forward_head(x["Q"][b, h], x["K"][b, h], x["V"][b, h], x["Cp"][h], x["Cc"][h], wl.P, wl.block_q,
                               wl.scale, form="dense", blocks=blocks)
        gh = {k: v[b, h] for k, v in gpu.items()}
        asg = ref["assignment"]
        r = compare_indices(gh, dict(parent_idx=asg["parent_idx"], child_idx=asg["child_idx"],
                                     parent_margin=asg["parent_margin"], child_margin=asg["child_margin"],
                                     stay_margin=asg["stay_margin"]))
        rep["parent_flips_excused"] += r["parent_flips_excused"]
        rep["child_flips_excused"] += r["child_flips_excused"]
        if r["parent_flips_excused"] == 0 and r["child_flips_excused"] == 0:
            compare_aggregates(gh, ref)
        # importance and selection of EVERY block of the head (cheap for the oracle: no O(N^2) part)
        n_all = 0
        for t in range(nblk):
            Qb = x["Q"][b, h][t * wl.block_q:(t + 1) * wl.block_q]
            w_or, _, _, _ = orc.importance_block(Qb, x["Cp"][h], ref["np"], wl.scale)
            sel_or, margin = orc.top_p(w_or, wl.P)
            if not np.array_equal(gh["selected"][t], sel_or):
                assert margin < NEAR_TIE, f"head {(b, h)} block {t}: wrong top-P set at margin {margin:.2e}"
                rep["topp_flips_excused"] += 1
            assert np.allclose(gh["importance"][t], w_or, rtol=2e-3, atol=2e-4)
            n_all += 1
        rep["blocks_selection_checked"] = rep.get("blocks_selection_checked", 0) + n_all
        sub = dict(selected=gh["selected"][blocks], importance=gh["importance"][blocks])
        same, excused = compare_selection(sub, dict(selected=ref["selected"][blocks],
                                                    importance=ref["importance"][blocks],
                                                    topp_margin=ref["topp_margin"][blocks]))
        for t, ok in zip(blocks, same):     # `excused` is already counted by the all-block loop above
            if not ok:
                continue
            rows = slice(t * wl.block_q, min(wl.N, (t + 1) * wl.block_q))
            yg, yr = gh["Y"][rows], ref["Y"][rows]
            assert np.isfinite(yg).all()
            rep["max_abs"] = max(rep["max_abs"], float(np.abs(yg - yr).max()))
            num += float(((yg - yr) ** 2).sum())
            den += float((yr ** 2).sum())
    rep["rel_l2"] = float(np.sqrt(num / den))
    tol = TOL[wl.dtype]
    assert rep["max_abs"] <= tol["max_abs"], rep
    assert tol["rel_l2"] is None or rep["rel_l2"] <= tol["rel_l2"], rep
    return rep, gpu, x


def heads_parity_factorised(wl: synth.Workload, heads, x=None, gpu=None, assignments=None, P=None):
    """Full-size run on the GPU; for every listed (b, h) the oracle evaluates EVERY query block in its
    O(M N) factorised form (pinned equal to the dense definition by the CPU tests): indices, aggregates,
    importance, top-P set and output of the whole head.  Returns the report and the oracle's assignments
    (so that several P values of one data set share them)."""
    x = synth.generate(wl) if x is None else x
    P = wl.P if P is None else P
    gpu = gpu_forward(wl, x, P=P) if gpu is None else gpu
    assignments = {} if assignments is None else assignments
    rep = dict(parent_flips_excused=0, child_flips_excused=0, topp_flips_excused=0, max_abs=0.0, blocks=0)
    num = den = 0.0
    nq = x["Q"].shape[2]
    for (b, h) in heads:
        if (b, h) not in assignments:
            assignments[(b, h)] = orc.assign_head(x["K"][b, h], x["Cp"][h], x["Cc"][h])
        ref = orc.forward_head(x["Q"][b, h], x["K"][b, h], x["V"][b, h], x["Cp"][h], x["Cc"][h], P, wl.block_q,
                               wl.scale, form="factorised", assignment=assignments[(b, h)])
        gh = {k: v[b, h] for k, v in gpu.items()}
        asg = ref["assignment"]
        r = compare_indices(gh, asg)
        rep["parent_flips_excused"] += r["parent_flips_excused"]
        rep["child_flips_excused"] += r["child_flips_excused"]
        if r["parent_flips_excused"] == 0 and r["child_flips_excused"] == 0:
            compare_aggregates(gh, ref)
        same, excused = compare_selection(gh, ref)
        rep["topp_flips_excused"] += excused
        rows = np.repeat(same, wl.block_q)[:nq]
        yg, yr = gh["Y"][rows], ref["Y"][rows]
        assert np.isfinite(gh["Y"]).all()
        rep["max_abs"] = max(rep["max_abs"], float(np.abs(yg - yr).max()))
        num += float(((yg - yr) ** 2).sum())
        den += float((yr ** 2).sum())
        rep["blocks"] += int(same.sum())
    rep["rel_l2"] = float(np.sqrt(num / den))
    tol = TOL[wl.dtype]
    assert rep["max_abs"] <= tol["max_abs"], rep
    assert tol["rel_l2"] is None or rep["rel_l2"] <= tol["rel_l2"], rep
    return rep, assignments
