"""Comparison of the CUDA path with the float64 oracle, stage by stage, on one image.

Rules (written out here so the tolerances are visible in the tests):
  * S, C, E, sigma_i (i <= r): relative error <= 1e-3; sigma beyond r: within 1e-3 * sigma_1.
  * Index results are compared exactly, except for tokens inside a band the floating-point
    scores cannot resolve: a token may sit on either side of a cut (Stage-I cut, A/B cut) only
    if its oracle score is within 1e-3 relative of the score at that cut; a Set-B token may be
    in or out of the merge set only if its best similarity is within 1e-4 of the similarity at
    the merge cut; its destination may differ only among Set-A tokens whose similarity is
    within 1e-4 of the best.  Every later stage is then checked against the oracle run on the
    CUDA path's own earlier decision, so one allowed flip cannot hide a later error.
  * X', K', V': absolute error <= 2e-2 in the storage type, and exact where nothing merges.
"""
from __future__ import annotations

from typing import Dict, Optional

import numpy as np

from oracle import ipgs_oracle as orc

REL_SCORE = 1e-3
SIM_BAND = 1e-4
ABS_OUT = 2e-2


def rel_err(got: np.ndarray, ref: np.ndarray) -> float:
    ref = np.asarray(ref, np.float64)
    got = np.asarray(got, np.float64)
    den = np.maximum(np.abs(ref), 1e-300)
    return float(np.max(np.abs(got - ref) / den)) if ref.size else 0.0


def check_scores(g: Dict[str, np.ndarray], o: Dict[str, np.ndarray], rank_tol: float) -> None:
    """g: CUDA outputs of one image (E, C, S, sigma, rank); o: oracle.score() result."""
    assert rel_err(g["S"], o["S"]) <= REL_SCORE, ("S", rel_err(g["S"], o["S"]))
    r = int(o["rank"])
    assert int(g["rank"]) == r, ("rank", int(g["rank"]), r)
    sig_o = o["sigma"]
    assert rel_err(g["sigma"][:r], sig_o[:r]) <= REL_SCORE, ("sigma", rel_err(g["sigma"][:r], sig_o[:r]))
    if len(sig_o) > r:
        assert np.max(np.abs(g["sigma"][r:len(sig_o)] - sig_o[r:])) <= REL_SCORE * sig_o[0], "sigma tail"
    assert rel_err(g["C"], o["C"]) <= REL_SCORE, ("C", rel_err(g["C"], o["C"]))
    assert rel_err(g["E"], o["E"]) <= REL_SCORE, ("E", rel_err(g["E"], o["E"]))


def band_population(E_or: np.ndarray, P: int, nA: int) -> int:
    """How many tokens sit inside the 1e-3 band around the two cuts (Stage-I cut and A/B cut):
    the tokens for which "exact outside the band" says nothing."""
    N = len(E_or)
    E32 = np.asarray(E_or, np.float64).astype(np.float32).astype(np.float64)
    order = orc.descending_order(E_or)
    inside = np.zeros(N, bool)
    for c in (nA, P):
        if 0 < c < N:
            v = 0.5 * (E32[order[c - 1]] + E32[order[c]])
            inside |= np.abs(E32 - v) <= REL_SCORE * abs(v)
    return int(inside.sum())


def cut_gaps(E_or: np.ndarray, P: int, nA: int):
    """Relative gap of the float32-rounded oracle scores across the A/B cut and the Stage-I cut."""
    N = len(E_or)
    E32 = np.asarray(E_or, np.float64).astype(np.float32).astype(np.float64)
    order = orc.descending_order(E_or)
    gaps = []
    for c in (nA, P):
        if 0 < c < N:
            hi, lo = E32[order[c - 1]], E32[order[c]]
            gaps.append((hi - lo) / max(abs(hi), 1e-300))
    return gaps


def open_score_gaps(O: np.ndarray, A: np.ndarray, cfgp: dict, min_gap: float = 3e-3,
                    near: float = 2.5e-3, step: float = 4e-3, max_pass: int = 6) -> np.ndarray:
    """Test-side conditioning of one image's O (storage dtype in, storage dtype out): rows whose
    oracle score lies within `near` (relative) of the Stage-I cut or of the A/B cut (Sec. 3.3.1
    last paragraph, Eq. 3-9) are scaled by (1 + step) when they are above the cut and by
    (1 - step) when below, bit-identical rows together so that twins stay twins, then rounded
    to the storage type again; repeated until both gaps exceed `min_gap`.  Scaling a row of O
    scales its information contribution (Eq. 3-6) by nearly the same factor.  Returns the new O;
    raises if the gaps cannot be opened."""
    O = np.array(O, copy=True)
    N = O.shape[0]
    M, P, nA, nB = orc.resolve_counts(N, cfgp["keep"], cfgp["rho"], cfgp.get("n_merge", -1))
    # groups of bit-identical rows
    keys = {}
    for x in range(N):
        keys.setdefault(O[x].tobytes(), []).append(x)
    group_of = {x: g for g in keys.values() for x in g}
    for _ in range(max_pass):
        o = oracle_scores(cfgp, O, A)
        if min(cut_gaps(o["E"], P, nA), default=1.0) >= min_gap:
            return O
        E32 = np.asarray(o["E"], np.float64).astype(np.float32).astype(np.float64)
        order = orc.descending_order(o["E"])
        pos = np.empty(N, int)
        pos[order] = np.arange(N)
        done = set()
        for c in (nA, P):
            if not 0 < c < N:
                continue
            v = 0.5 * (E32[order[c - 1]] + E32[order[c]])
            for x in np.nonzero(np.abs(E32 - v) <= near * abs(v))[0]:
                if int(x) in done:
                    continue
                up = pos[x] < c
                f = (1.0 + step) if up else (1.0 - step)
                for y in group_of[int(x)]:
                    O[y] = (O[y].astype(np.float64) * f).astype(O.dtype)
                    done.add(y)
    raise AssertionError("score gaps could not be opened")


def check_sets(E_or: np.ndarray, setA_g, setB_g, P: int, nA: int) -> int:
    """Exact agreement outside the unresolvable band; returns the number of in-band flips."""
    N = len(E_or)
    E32 = np.asarray(E_or, np.float64).astype(np.float32).astype(np.float64)
    order = orc.descending_order(E_or)
    cls_o = np.zeros(N, np.int8)
    cls_o[order[:nA]] = 1
    cls_o[order[nA:P]] = 2
    cls_g = np.zeros(N, np.int8)
    setA_g = np.asarray(setA_g)
    setB_g = np.asarray(setB_g)
    assert len(setA_g) == nA and len(setB_g) == P - nA
    assert np.all(np.diff(setA_g) > 0) and np.all(np.diff(setB_g) > 0), "lists must ascend"
    assert len(set(setA_g.tolist()) & set(setB_g.tolist())) == 0
    cls_g[setA_g] = 1
    cls_g[setB_g] = 2
    cuts = []
    for c in (nA, P):
        if 0 < c < N:
            cuts.append(0.5 * (E32[order[c - 1]] + E32[order[c]]))
    flips = 0
    for x in np.nonzero(cls_o != cls_g)[0]:
        ok = any(abs(E32[x] - v) <= REL_SCORE * abs(v) for v in cuts)
        assert ok, f"token {x}: oracle class {cls_o[x]}, CUDA class {cls_g[x]}, E={E32[x]}, cuts={cuts}"
        flips += 1
    return flips


def check_merge(O: np.ndarray, setA, setB, M: int, src_g, dst_g, kept_g, keep: int) -> int:
    """Oracle matching on the given sets against the CUDA lists; returns in-band flips."""
    setA = [int(a) for a in setA]
    setB = [int(b) for b in setB]
    src_g = np.asarray(src_g)
    dst_g = np.asarray(dst_g)
    kept_g = np.asarray(kept_g)
    assert len(src_g) == M and len(dst_g) == M and len(kept_g) == keep
    flips = 0
    if M > 0:
        assert np.all(np.diff(src_g) > 0), "merge_src must ascend"
        sim = orc.similarity(O, setA, setB)
        best = sim.max(axis=1)
        src_o, dst_o = orc.match_and_select(sim, setA, setB, M)
        order = sorted(range(len(setB)), key=lambda j: (-float(np.float32(best[j])), setB[j]))
        cut = 0.5 * (best[order[M - 1]] + best[order[M]]) if M < len(setB) else -np.inf
        pos = {b: j for j, b in enumerate(setB)}
        for b in set(src_o.tolist()) ^ set(src_g.tolist()):
            assert b in pos and abs(best[pos[b]] - cut) <= SIM_BAND, f"merge set differs at token {b}"
            flips += 1
        dmap_o = dict(zip(src_o.tolist(), dst_o.tolist()))
        colA = {a: i for i, a in enumerate(setA)}
        for b, a in zip(src_g.tolist(), dst_g.tolist()):
            assert b in pos and a in colA, "merge pair outside the sets"
            row = sim[pos[b]]
            if dmap_o.get(b, None) != a:
                assert row.max() - row[colA[a]] <= SIM_BAND, f"destination of {b}: {a} is not a best match"
                # a bit-identical alternative must respect the lower-index rule
                exact = [x for x in setA if row[colA[x]] == row[colA[a]] and np.array_equal(O[x], O[a])]
                assert a == min(exact), f"tie among identical rows must go to the lower index ({b}->{a})"
                flips += 1
    expect_kept = sorted(set(setA) | (set(setB) - set(src_g.tolist())))
    assert kept_g.tolist() == expect_kept, "kept_idx != Set A + unmerged Set B, ascending"
    return flips


def check_compact(X, K, V, kept, src, dst, Xo_g, Ko_g, Vo_g, weights=None, storage=None) -> None:
    """weights: the IPGS scores when the merge is the score-weighted variant.  storage: "bf16"
    when the float32 arrays hold bfloat16 values (numpy has no such type)."""
    out_dtype = "bf16" if storage == "bf16" else X.dtype
    ref = orc.compact(X, K, V, kept, src, dst, out_dtype, weights)
    dests = set(int(t) for t in dst)
    plain = np.array([int(a) not in dests for a in kept])
    for name, got, want in (("X", Xo_g, ref["X"]), ("K", Ko_g, ref["K"]), ("V", Vo_g, ref["V"])):
        if want is None:
            assert got is None
            continue
        got = np.asarray(got)
        assert got.shape == want.shape and got.dtype == want.dtype, name
        err = np.max(np.abs(got.astype(np.float64) - want.astype(np.float64))) if got.size else 0.0
        assert err <= (ABS_OUT if storage != "bf16" else 4 * ABS_OUT), (name, err)
        # rows nothing merges into are copies
        if name == "X":
            assert np.array_equal(got[plain], want[plain]), "unmerged rows must be bit-exact copies"
        else:
            assert np.array_equal(got[:, plain], want[:, plain]), "unmerged rows must be bit-exact copies"
        # a merged 16-bit row is at most one unit in the last place away (float32 sum, one
        # division, one rounding); a float32 row carries the rounding of its float32 sum
        diff = np.abs(got.astype(np.float64) - want.astype(np.float64))
        if storage == "bf16":
            mag = np.maximum(np.abs(want.astype(np.float64)), 2.0 ** -126)
            ulp = 2.0 ** (np.floor(np.log2(mag)) - 7)
            assert np.all(diff <= ulp), name
        elif want.dtype == np.float16:
            ulp = np.spacing(np.abs(want).astype(want.dtype)).astype(np.float64)
            assert np.all(diff <= ulp + 1e-30), name
        else:
            assert np.all(diff <= 4e-6 * (1.0 + np.abs(want.astype(np.float64)))), name


def oracle_scores(cfgp, O, A) -> Dict[str, np.ndarray]:
    return orc.score(O.astype(np.float64), A.astype(np.float64), cfgp["lam"], cfgp["rank_tol"],
                     cfgp["score_norm"])


def check_image(cfgp: dict, im: Dict[str, np.ndarray], g: Dict[str, np.ndarray],
                with_scores: bool = True) -> Dict[str, int]:
    """Full staged comparison of one image.  cfgp: keep, rho, n_merge, lam, rank_tol, score_norm.
    im: O, A, X, K, V (storage dtype).  g: CUDA results of that image: E, C, S, sigma, rank, setA,
    setB, src, dst, kept, Xo, Ko, Vo."""
    N = im["O"].shape[0]
    M, P, nA, nB = orc.resolve_counts(N, cfgp["keep"], cfgp["rho"], cfgp.get("n_merge", -1))
    o = oracle_scores(cfgp, im["O"], im["A"])
    if with_scores:
        check_scores(g, o, cfgp["rank_tol"])
    flips_sets = check_sets(o["E"], g["setA"], g["setB"], P, nA)
    # Eq. 3-10 features: the attention output (the paper), or the variants' hidden states /
    # head-mean keys
    src_name = cfgp.get("sim_source", "O")
    feats = {"O": im["O"], "X": im["X"],
             "meanK": None if im.get("K") is None else orc.mean_heads(im["K"])}[src_name]
    flips_merge = check_merge(np.asarray(feats, np.float64), g["setA"], g["setB"], M, g["src"],
                              g["dst"], g["kept"], cfgp["keep"])
    check_compact(im["X"], im.get("K"), im.get("V"), g["kept"], g["src"], g["dst"], g["Xo"],
                  g.get("Ko"), g.get("Vo"), weights=g["E"] if cfgp.get("weighted") else None,
                  storage=cfgp.get("dtype"))
    # (the weights of the score-weighted variant are the CUDA path's own scores, which
    # check_scores has just compared with the oracle's: like every later stage, the merge is
    # checked against the oracle run on the earlier stage's CUDA result, and can then be held
    # to one unit in the last place)
    return {"flips_sets": flips_sets, "flips_merge": flips_merge,
            "in_band": band_population(o["E"], P, nA)}
