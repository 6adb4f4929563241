"""Pins for the float64 oracle: closed forms, invariants, brute force, independent routines.

Each test is chosen so that a plausible slip in the oracle (dropped term, wrong sign or
index, transposed operand, wrong tie rule) fails at least one of them.  No GPU needed.
"""
import itertools
import os

import numpy as np
import pytest

from oracle import ipgs_oracle as orc

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _gold(name):
    vals = {}
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            k, v = line.split()
            vals[k] = float(v)
    return vals


def _rand_orth(n, rng):
    q, r = np.linalg.qr(rng.standard_normal((n, n)))
    return q * np.sign(np.diag(r))


# ------------------------------------------------------------------ counts
def test_counts_paper_operating_points():
    # 576 -> 128 with rho = 0.5: Stage I keeps 192, Stage II merges 64 (Sec. 3.3.1 / 3.3.2)
    assert orc.resolve_counts(576, 128, 0.5) == (64, 192, 96, 96)
    assert orc.resolve_counts(576, 192, 0.5) == (96, 288, 144, 144)
    assert orc.resolve_counts(576, 64, 0.5) == (32, 96, 48, 48)
    # odd P: B gets the odd one;   keep = N: nothing to prune or merge
    assert orc.resolve_counts(576, 333, 0.5) == (166, 499, 249, 250)
    assert orc.resolve_counts(576, 576, 0.5) == (0, 576, 288, 288)
    # clamp to N - keep
    assert orc.resolve_counts(100, 90, 0.5) == (10, 100, 50, 50)
    assert orc.resolve_counts(50, 10, 0.0) == (0, 10, 5, 5)
    assert orc.resolve_counts(50, 10, 0.5, n_merge=3) == (3, 13, 6, 7)
    with pytest.raises(ValueError):
        orc.resolve_counts(10, 0)
    with pytest.raises(ValueError):
        orc.resolve_counts(10, 11)


# ------------------------------------------------------------------ SVD
@pytest.mark.parametrize("shape", [(5, 9), (9, 5), (12, 12), (16, 7)])
def test_svd_two_routes_agree_and_reconstruct(shape):
    rng = np.random.default_rng(1)
    O = rng.standard_normal(shape)
    Uj, sj = orc.svd_jacobi(O)
    Ul, sl = orc.svd_lapack(O)
    q = min(shape)
    assert sj.shape == (q,) and sl.shape == (q,)
    np.testing.assert_allclose(sj, sl, rtol=1e-12, atol=1e-12)
    assert np.all(np.diff(sj) <= 1e-15)
    for U, s in ((Uj, sj), (Ul, sl)):
        # left singular vectors: orthonormal, and U^T O has orthogonal rows of norm sigma (Eq. 3-5)
        np.testing.assert_allclose(U.T @ U, np.eye(q), atol=1e-12)
        B = U.T @ O
        np.testing.assert_allclose(B @ B.T, np.diag(s ** 2), atol=1e-10)
        np.testing.assert_allclose(U @ B, O, atol=1e-11)       # sum_i u_xi sigma_i v_i^T = row x
    # |u_xi| agree between routes (sign is free)
    np.testing.assert_allclose(np.abs(Uj), np.abs(Ul), atol=1e-9)


def test_svd_frobenius_scaling_rotation_rank1():
    rng = np.random.default_rng(2)
    O = rng.standard_normal((10, 14))
    for fn in (orc.svd_jacobi, orc.svd_lapack):
        _, s = fn(O)
        assert abs(np.sum(s ** 2) - np.sum(O * O)) < 1e-10
        _, s3 = fn(-3.0 * O)
        np.testing.assert_allclose(s3, 3.0 * s, rtol=1e-12)
        Q = _rand_orth(14, rng)
        _, sq = fn(O @ Q)
        np.testing.assert_allclose(sq, s, rtol=1e-11)
        _, sp = fn(O[:, rng.permutation(14)])
        np.testing.assert_allclose(sp, s, rtol=1e-11)
        a = rng.standard_normal(10)
        b = rng.standard_normal(14)
        _, s1 = fn(np.outer(a, b))
        assert abs(s1[0] - np.linalg.norm(a) * np.linalg.norm(b)) < 1e-10
        assert np.all(s1[1:] < 1e-10)


# ------------------------------------------------------------------ ICS, Eq. 3-6
@pytest.mark.parametrize("method", ["lapack", "jacobi"])
def test_ics_hand_example(method):
    g = _gold("ics_2x2.txt")
    O = np.array([[3.0, 0.0], [4.0, 5.0]])
    C, s, r = orc.information_contribution(O, 0.0, method)
    assert r == 2
    np.testing.assert_allclose(s, [g["sigma_1"], g["sigma_2"]], rtol=1e-13)
    np.testing.assert_allclose(C, [g["C0_full"], g["C1_full"]], rtol=1e-13)
    C, s, r = orc.information_contribution(O, 0.5, method)
    assert r == 1
    np.testing.assert_allclose(C, [g["C0_rank1"], g["C1_rank1"]], rtol=1e-13)


@pytest.mark.parametrize("method", ["lapack", "jacobi"])
def test_ics_rank1_closed_form(method):
    rng = np.random.default_rng(3)
    a = rng.standard_normal(9)
    b = rng.standard_normal(13)
    C, s, r = orc.information_contribution(np.outer(a, b), 1e-9, method)
    assert r == 1
    np.testing.assert_allclose(C, np.abs(a) * np.linalg.norm(b), rtol=1e-10)


@pytest.mark.parametrize("method", ["lapack", "jacobi"])
def test_ics_orthogonal_rows_distinct_norms(method):
    rng = np.random.default_rng(4)
    Q = _rand_orth(16, rng)[:7]                      # 7 orthonormal rows in R^16
    norms = np.array([5.0, 0.5, 3.0, 7.0, 1.0, 2.0, 4.0])
    O = Q * norms[:, None]
    C, s, r = orc.information_contribution(O, 0.0, method)
    np.testing.assert_allclose(C, norms, rtol=1e-10)   # each token is its own singular direction
    np.testing.assert_allclose(s, np.sort(norms)[::-1], rtol=1e-12)
    # numerical rank: tokens below rank_tol * sigma_1 drop out of the sum entirely
    C2, _, r2 = orc.information_contribution(O, 0.2, method)       # threshold 1.4
    assert r2 == 5
    np.testing.assert_allclose(C2, np.where(norms > 1.4, norms, 0.0), atol=1e-10)


def test_ics_orthogonal_rows_equal_norms_give_equal_contributions():
    rng = np.random.default_rng(5)
    O = 2.5 * _rand_orth(12, rng)[:6]
    C, s, r = orc.information_contribution(O, 0.0, "jacobi")     # Jacobi starts from a diagonal Gram
    np.testing.assert_allclose(C, 2.5, rtol=1e-12)
    np.testing.assert_allclose(s, 2.5, rtol=1e-12)


@pytest.mark.parametrize("method", ["lapack", "jacobi"])
def test_ics_identity_bounds_blocks_duplicates(method):
    rng = np.random.default_rng(6)
    O = rng.standard_normal((11, 15)) * rng.uniform(0.2, 3.0, size=(11, 1))
    C, s, r = orc.information_contribution(O, 0.0, method)
    rn = np.linalg.norm(O, axis=1)
    assert np.all(C >= rn * (1 - 1e-12)) and np.all(C <= np.sqrt(11) * rn * (1 + 1e-12))
    # scaling the matrix scales C; rotating the feature space leaves C alone
    C3, _, _ = orc.information_contribution(3.0 * O, 0.0, method)
    np.testing.assert_allclose(C3, 3.0 * C, rtol=1e-11)
    Cq, _, _ = orc.information_contribution(O @ _rand_orth(15, rng), 0.0, method)
    np.testing.assert_allclose(Cq, C, rtol=1e-9)
    # permuting tokens permutes C
    p = rng.permutation(11)
    Cp, _, _ = orc.information_contribution(O[p], 0.0, method)
    np.testing.assert_allclose(Cp, C[p], rtol=1e-9)
    # block-diagonal O: C is computed per block
    O1 = rng.standard_normal((4, 5))
    O2 = 0.37 * rng.standard_normal((3, 6))
    Ob = np.zeros((7, 11))
    Ob[:4, :5] = O1
    Ob[4:, 5:] = O2
    Cb, _, _ = orc.information_contribution(Ob, 0.0, method)
    C1, _, _ = orc.information_contribution(O1, 0.0, method)
    C2, _, _ = orc.information_contribution(O2, 0.0, method)
    np.testing.assert_allclose(Cb, np.concatenate([C1, C2]), rtol=1e-9)
    # exact duplicate rows get equal C and add no rank
    Od = np.vstack([O, O[3:4], O[7:8]])
    Cd, sd, rd = orc.information_contribution(Od, 1e-10, method)
    assert rd == 11
    assert abs(Cd[11] - Cd[3]) < 1e-10 and abs(Cd[12] - Cd[7]) < 1e-10


def test_ics_leave_one_out_brute_force():
    """Recompute the spectrum without token x: pins the rank statements, and equals C(x)
    where the drop of sum(sigma) has a closed form (orthogonal rows)."""
    rng = np.random.default_rng(7)
    base = rng.standard_normal((6, 10))
    O = np.vstack([base, base[2:3]])                  # token 6 duplicates token 2
    _, s_all, r_all = orc.information_contribution(O, 1e-10)
    assert r_all == 6
    for x in range(7):
        rest = np.delete(O, x, axis=0)
        _, s, r = orc.information_contribution(rest, 1e-10)
        if x in (2, 6):
            assert r == r_all                        # a duplicated token carries no rank of its own
        else:
            assert r == r_all - 1
    Q = _rand_orth(9, rng)[:5]
    norms = np.array([4.0, 1.0, 2.5, 0.7, 3.0])
    Oo = Q * norms[:, None]
    C, s_all, _ = orc.information_contribution(Oo, 0.0)
    for x in range(5):
        _, s, _ = orc.information_contribution(np.delete(Oo, x, axis=0), 0.0)
        assert abs((s_all.sum() - s.sum()) - C[x]) < 1e-10
    # generic matrix: leave-one-out drop and C are strongly rank-correlated (sanity, not identity)
    Og = rng.standard_normal((12, 20)) * rng.uniform(0.1, 4.0, size=(12, 1))
    C, s_all, _ = orc.information_contribution(Og, 0.0)
    drop = np.array([s_all.sum() - orc.information_contribution(np.delete(Og, x, 0), 0.0)[1].sum()
                     for x in range(12)])
    ra, rb = np.argsort(np.argsort(C)), np.argsort(np.argsort(drop))
    assert np.corrcoef(ra, rb)[0, 1] > 0.5


# ------------------------------------------------------------------ AS, Eq. 3-7
def test_attention_score_closed_forms():
    H, T, N = 3, 4, 7
    np.testing.assert_allclose(orc.attention_score(np.full((H, T, N), 1.0 / N)), 1.0 / N, rtol=1e-14)
    A = np.zeros((H, T, N))
    hits = np.zeros(N)
    rng = np.random.default_rng(8)
    for h in range(H):
        for t in range(T):
            x = rng.integers(N)
            A[h, t, x] = 1.0
            hits[x] += 1
    np.testing.assert_allclose(orc.attention_score(A), hits / (H * T), rtol=1e-14)
    z = rng.standard_normal((H, T, N))
    P = np.exp(z) / np.exp(z).sum(-1, keepdims=True)
    S = orc.attention_score(P)
    assert abs(S.sum() - 1.0) < 1e-13
    np.testing.assert_allclose(S, P.mean(axis=(0, 1)), rtol=1e-13)     # library mean, other order
    # the mean is over heads and queries, not over tokens: a transposed slice must differ
    assert S.shape == (N,)


# ------------------------------------------------------------------ E, Eq. 3-8
def test_combined_score_extremes_and_midpoint():
    rng = np.random.default_rng(9)
    C = rng.uniform(1, 5, 9)
    S = rng.uniform(0, 1, 9)
    np.testing.assert_array_equal(orc.combined_score(C, S, 0.0), C)
    np.testing.assert_array_equal(orc.combined_score(C, S, 1.0), S)
    np.testing.assert_allclose(orc.combined_score(C, S, 0.25), 0.75 * C + 0.25 * S, rtol=1e-15)
    E = orc.combined_score(C, S, 0.25, "sum1")
    assert abs(E.sum() - 1.0) < 1e-13
    np.testing.assert_allclose(E, 0.75 * C / C.sum() + 0.25 * S / S.sum(), rtol=1e-14)
    with pytest.raises(ValueError):
        orc.combined_score(C, S, 1.5)


# ------------------------------------------------------------------ prune / split, Eq. 3-9
def test_prune_split_vs_rank_counting_and_ties():
    rng = np.random.default_rng(10)
    for trial in range(20):
        N = int(rng.integers(4, 17))
        E = rng.integers(0, 6, N).astype(float)          # many exact ties
        P = int(rng.integers(1, N + 1))
        nA = P // 2
        setA, setB = orc.prune_split(E, P, nA)
        # brute force: position of x = #{y: E_y > E_x} + #{y < x: E_y == E_x}
        pos = [sum(1 for y in range(N) if E[y] > E[x] or (E[y] == E[x] and y < x)) for x in range(N)]
        expA = sorted(range(N), key=lambda x: pos[x])[:nA]
        expB = sorted(range(N), key=lambda x: pos[x])[nA:P]
        assert list(setA) == expA and list(setB) == expB
    E = np.array([1.0, 7.0, 7.0, 3.0, 7.0])
    a, b = orc.prune_split(E, 4, 2)
    assert list(a) == [1, 2] and list(b) == [4, 3]
    a, b = orc.prune_split(E, 5, 2)                       # keep everything: only an ordering
    assert sorted(list(a) + list(b)) == [0, 1, 2, 3, 4]


def test_prune_lambda_extremes_are_plain_topk():
    rng = np.random.default_rng(11)
    O = rng.standard_normal((14, 20)) * rng.uniform(0.2, 3, (14, 1))
    z = rng.standard_normal((2, 5, 14))
    A = np.exp(z) / np.exp(z).sum(-1, keepdims=True)
    sc1 = orc.score(O, A, lam=1.0)
    a, b = orc.prune_split(sc1["E"], 6, 3)
    top = np.argsort(-A.mean(axis=(0, 1)), kind="stable")[:6]
    assert list(a) + list(b) == list(top)
    sc0 = orc.score(O, A, lam=0.0)
    a, b = orc.prune_split(sc0["E"], 6, 3)
    assert list(a) + list(b) == list(np.argsort(-sc0["C"], kind="stable")[:6])


# ------------------------------------------------------------------ similarity / match, Eq. 3-10
def test_similarity_known_angles_and_zero_row():
    ang = np.deg2rad([0.0, 30.0, 90.0, 135.0])
    O = np.stack([np.cos(ang), np.sin(ang)], 1) * np.array([[1.0], [4.0], [0.5], [2.0]])
    O = np.vstack([O, [0.0, 0.0]])
    sim = orc.similarity(O, [0, 1], [2, 3, 4])             # rows = B, columns = A
    exp = np.array([[np.cos(ang[2] - ang[0]), np.cos(ang[2] - ang[1])],
                    [np.cos(ang[3] - ang[0]), np.cos(ang[3] - ang[1])],
                    [0.0, 0.0]])
    np.testing.assert_allclose(sim, exp, atol=1e-14)
    assert sim.shape == (3, 2)


def test_match_and_select_brute_force_and_ties():
    rng = np.random.default_rng(12)
    for trial in range(20):
        nA, nB = int(rng.integers(1, 7)), int(rng.integers(1, 7))
        ids = rng.permutation(20)[:nA + nB]
        setA, setB = ids[:nA], ids[nA:]
        sim = rng.integers(0, 4, (nB, nA)) / 4.0           # ties on purpose
        M = int(rng.integers(0, nB + 1))
        src, dst = orc.match_and_select(sim, setA, setB, M)
        best = {}
        for j, b in enumerate(setB):
            mx = sim[j].max()
            best[int(b)] = (mx, min(int(setA[i]) for i in range(nA) if sim[j, i] == mx))
        order = sorted(best, key=lambda b: (-best[b][0], b))[:M]
        assert list(src) == order
        assert list(dst) == [best[b][1] for b in order]
    # two identical Set-A rows: the lower original index wins, whatever its position in Set A
    src, dst = orc.match_and_select(np.array([[0.9, 0.9]]), [7, 3], [5], 1)
    assert list(dst) == [3]


def test_twin_is_merged_into_its_twin():
    """An exact duplicate adds no rank (above) and, once the attention term separates the
    twins into Set A and Set B, the Set-B twin has similarity 1 and merges into its twin."""
    rng = np.random.default_rng(13)
    N, d = 10, 24
    O = rng.standard_normal((N, d))
    O[7] = O[2]
    # attention that ranks token 2 first and token 7 fourth of P = 6 (lambda = 1: AS only)
    S_target = np.array([0.05, 0.06, 0.30, 0.20, 0.15, 0.01, 0.02, 0.12, 0.07, 0.02])
    A = np.tile(S_target, (2, 3, 1))
    X = rng.standard_normal((N, d))
    X[7] = X[2]
    res = orc.carve(O, A, X, None, None, keep=4, rho=0.5, lam=1.0)
    assert res["P"] == 6 and res["M"] == 2
    assert list(res["setA"]) == [2, 3, 4] and list(res["setB"]) == [7, 8, 1]
    assert res["merge_src"][0] == 7 and res["merge_dst"][0] == 2
    j = list(res["kept_idx"]).index(2)
    others = [s for s, t in zip(res["merge_src"], res["merge_dst"]) if t == 2 and s != 7]
    if not others:
        np.testing.assert_allclose(res["Xo"][j], X[2], rtol=1e-15)     # mean of two equal rows


# ------------------------------------------------------------------ merge / compact
def test_compact_rho0_is_a_pure_gather():
    rng = np.random.default_rng(14)
    N, d, H, dh = 12, 16, 2, 8
    O = rng.standard_normal((N, d))
    z = rng.standard_normal((H, 3, N))
    A = np.exp(z) / np.exp(z).sum(-1, keepdims=True)
    X = rng.standard_normal((N, d)).astype(np.float16)
    K = rng.standard_normal((H, N, dh)).astype(np.float16)
    V = rng.standard_normal((H, N, dh)).astype(np.float16)
    res = orc.carve(O, A, X, K, V, keep=5, rho=0.0)
    kept = res["kept_idx"]
    assert len(kept) == 5 and np.all(np.diff(kept) > 0) and len(res["merge_src"]) == 0
    assert res["Xo"].dtype == np.float16
    np.testing.assert_array_equal(res["Xo"], X[kept])
    np.testing.assert_array_equal(res["Ko"], K[:, kept])
    np.testing.assert_array_equal(res["Vo"], V[:, kept])
    order = orc.descending_order(res["E"])
    assert sorted(order[:5]) == list(kept)


@pytest.mark.parametrize("keep,rho", [(4, 0.5), (5, 1.0), (6, 0.34), (3, 0.7)])
def test_merge_invariants(keep, rho):
    rng = np.random.default_rng(15)
    N, d, H, dh = 14, 10, 2, 4
    O = rng.standard_normal((N, d))
    z = rng.standard_normal((H, 3, N))
    A = np.exp(z) / np.exp(z).sum(-1, keepdims=True)
    X = rng.standard_normal((N, d))
    K = rng.standard_normal((H, N, dh))
    V = rng.standard_normal((H, N, dh))
    res = orc.carve(O, A, X, K, V, keep=keep, rho=rho)
    M, P = res["M"], res["P"]
    kept, src, dst = res["kept_idx"], res["merge_src"], res["merge_dst"]
    assert len(kept) == keep and np.all(np.diff(kept) > 0)
    assert len(src) == M == len(set(src.tolist()))               # each source merged exactly once
    assert set(src.tolist()) <= set(res["setB"].tolist())
    assert set(dst.tolist()) <= set(res["setA"].tolist())
    assert set(kept.tolist()) == (set(res["setA"].tolist()) | set(res["setB"].tolist())) - set(src.tolist())
    surv = sorted(res["setA"].tolist() + res["setB"].tolist())
    cnt = np.array([1 + sum(1 for t in dst if t == a) for a in kept])
    # the merge keeps the size-weighted sum of the survivors
    np.testing.assert_allclose((cnt[:, None] * res["Xo"]).sum(0), X[surv].sum(0), atol=1e-12)
    for h in range(H):
        np.testing.assert_allclose((cnt[:, None] * res["Ko"][h]).sum(0), K[h, surv].sum(0), atol=1e-12)
        np.testing.assert_allclose((cnt[:, None] * res["Vo"][h]).sum(0), V[h, surv].sum(0), atol=1e-12)
    # a destination row is the plain mean of its group
    for j, a in enumerate(kept):
        grp = [a] + [s for s, t in zip(src, dst) if t == a]
        np.testing.assert_allclose(res["Xo"][j], X[grp].mean(0), atol=1e-13)


def test_carve_tiny_against_independent_brute_force():
    """Whole path re-derived with different code (eigen-decomposition of the Gram, counting
    ranks, dense loops) on small inputs."""
    rng = np.random.default_rng(16)
    for trial in range(6):
        N, d = int(rng.integers(6, 15)), int(rng.integers(6, 20))
        keep = int(rng.integers(2, N))
        lam = [0.0, 0.3, 1.0][trial % 3]
        O = rng.standard_normal((N, d)) * rng.uniform(0.3, 3, (N, 1))
        z = rng.standard_normal((2, 4, N))
        A = np.exp(z) / np.exp(z).sum(-1, keepdims=True)
        X = rng.standard_normal((N, d))
        res = orc.carve(O, A, X, None, None, keep=keep, rho=0.5, lam=lam, score_norm="sum1")
        # independent: U, sigma from the symmetric eigenproblem of O O^T
        w, Q = np.linalg.eigh(O @ O.T)
        w = np.clip(w[::-1], 0, None)
        Q = Q[:, ::-1]
        q = min(N, d)
        C = (np.abs(Q[:, :q]) * np.sqrt(w[:q])).sum(1)
        S = A.reshape(-1, N).sum(0) / 8
        E = (1 - lam) * C / C.sum() + lam * S / S.sum()
        np.testing.assert_allclose(res["E"], E, rtol=1e-6)  # Gram route: sqrt of ~1e-16 eigenvalues when N > d
        M = min(int(np.floor(keep * 0.5)), N - keep)
        P = keep + M
        E32 = E.astype(np.float32)
        pos = [sum(1 for y in range(N) if E32[y] > E32[x] or (E32[y] == E32[x] and y < x)) for x in range(N)]
        byrank = sorted(range(N), key=lambda x: pos[x])
        SA, SB = byrank[:P // 2], byrank[P // 2:P]
        assert list(res["setA"]) == SA and list(res["setB"]) == SB
        Gm = O @ O.T
        best = {}
        for b in SB:
            vals = [(np.float32(Gm[b, a] / np.sqrt(Gm[b, b] * Gm[a, a])), a) for a in SA]
            mx = max(v for v, _ in vals)
            best[b] = (mx, min(a for v, a in vals if v == mx))
        chosen = sorted(SB, key=lambda b: (-best[b][0], b))[:M]
        assert list(res["merge_src"]) == chosen
        assert list(res["merge_dst"]) == [best[b][1] for b in chosen]
        kept = sorted(set(SA) | (set(SB) - set(chosen)))
        assert list(res["kept_idx"]) == kept
        for j, a in enumerate(kept):
            grp = [a] + [b for b in chosen if best[b][1] == a]
            np.testing.assert_allclose(res["Xo"][j], X[grp].sum(0) / len(grp), atol=1e-13)


# ------------------------------------------------------------------ Sec. 3.2: rank of a token set
def test_token_information_closed_forms():
    rng = np.random.default_rng(5)
    # mutually orthogonal rows: every subset of n rows has rank n and its sigma are the row norms
    Q, _ = np.linalg.qr(rng.standard_normal((12, 12)))
    norms = np.arange(1.0, 13.0)
    O = Q * norms[:, None]
    for idx in ([0, 3, 7], [11, 2], list(range(12))):
        sig, r = orc.token_information(O, idx, 1e-6)
        assert r == len(idx)
        assert np.allclose(sig[:len(idx)], sorted(norms[idx], reverse=True), rtol=1e-12)
    # both SVD routes
    assert np.allclose(orc.token_information(O, [1, 4, 9], 0.0, "jacobi")[0],
                       orc.token_information(O, [1, 4, 9], 0.0, "lapack")[0], rtol=1e-10)
    # a copy of a row adds no rank; a row outside the span adds one
    L = rng.standard_normal((9, 4)) @ rng.standard_normal((4, 30))      # rank 4
    assert orc.token_information(L, None, 1e-9)[1] == 4
    assert orc.token_information(np.vstack([L, L[2:3]]), None, 1e-9)[1] == 4
    assert orc.token_information(np.vstack([L, rng.standard_normal((1, 30))]), None, 1e-9)[1] == 5
    # fewer rows than the rank: the rank is the row count; removing rows never raises it
    assert orc.token_information(L, [0, 5, 8], 1e-9)[1] == 3
    ranks = [orc.token_information(L, list(range(n)), 1e-9)[1] for n in range(9, 0, -1)]
    assert all(a >= b for a, b in zip(ranks, ranks[1:])) and ranks[-1] == 1
    # order of the token list and scaling of O do not matter; rank_tol cuts relative to sigma_1
    s1, r1 = orc.token_information(L, [1, 6, 3, 8], 1e-9)
    s2, r2 = orc.token_information(7.0 * L, [8, 3, 6, 1], 1e-9)
    assert r1 == r2 and np.allclose(7.0 * s1, s2, rtol=1e-12)
    D = np.diag([10.0, 1.0, 0.1, 0.01])
    assert [orc.token_information(D, None, t)[1] for t in (0.5, 0.05, 0.005, 0.0)] == [1, 2, 3, 4]
    # sum of squares of sigma = squared Frobenius norm of the chosen rows
    sig, _ = orc.token_information(L, [0, 2, 4, 6], 0.0)
    assert np.isclose(np.sum(sig ** 2), np.sum(L[[0, 2, 4, 6]] ** 2), rtol=1e-12)


# ------------------------------------------------------------------ sequence after the compression
def test_reassemble_closed_forms():
    rng = np.random.default_rng(9)
    n_sys, n_vis, n_text, d = 3, 7, 4, 5
    Hs = rng.standard_normal((n_sys + n_vis + n_text, d)).astype(np.float32)
    vis = Hs[n_sys:n_sys + n_vis]
    # nothing removed: the sequence and its positions come back unchanged
    rows, pos = orc.reassemble(Hs, n_sys, n_vis, vis, range(n_vis))
    assert np.array_equal(rows, Hs) and pos.tolist() == list(range(len(Hs)))
    # three visual tokens kept: system rows, those three, then the prompt rows, positions original
    kept = [1, 4, 6]
    Xo = 2.0 * vis[kept]
    rows, pos = orc.reassemble(Hs, n_sys, n_vis, Xo, kept)
    assert rows.shape == (n_sys + 3 + n_text, d) and rows.dtype == Hs.dtype
    assert np.array_equal(rows[:3], Hs[:3]) and np.array_equal(rows[3:6], Xo)
    assert np.array_equal(rows[6:], Hs[10:])
    assert pos.tolist() == [0, 1, 2, 4, 7, 9, 10, 11, 12, 13]
    assert np.all(np.diff(pos) > 0)
    # no system or prompt tokens at all
    rows, pos = orc.reassemble(vis, 0, n_vis, Xo, kept)
    assert np.array_equal(rows, Xo) and pos.tolist() == kept



def test_rope_tables_closed_forms():
    # Conclusion: rotary encodings of the layers after the compression use the original
    # positions.  Pins: position 0 is the identity rotation; the first pair turns by exactly
    # `pos` radians (theta_0 = 1); the last pair by pos * base^-(dh-2)/dh; every pair is a
    # rotation (cos^2 + sin^2 = 1); rotating by a then by b is rotating by a + b.
    dh, base = 16, 10000.0
    pos = [0, 1, 7, 35, 611, 4095]
    cos, sin = orc.rope_tables(pos, dh, base)
    assert cos.shape == (6, 8) and sin.shape == (6, 8)
    assert np.array_equal(cos[0], np.ones(8)) and np.array_equal(sin[0], np.zeros(8))
    np.testing.assert_allclose(cos[:, 0], np.cos(np.array(pos, float)), rtol=0, atol=1e-12)
    np.testing.assert_allclose(sin[:, 0], np.sin(np.array(pos, float)), rtol=0, atol=1e-12)
    np.testing.assert_allclose(cos[3, 7], np.cos(35.0 / 10000.0 ** (14.0 / 16.0)), atol=1e-15)
    np.testing.assert_allclose(cos ** 2 + sin ** 2, 1.0, atol=1e-14)
    ca, sa = orc.rope_tables([13], dh, base)
    cb, sb = orc.rope_tables([598], dh, base)
    cc, sc = orc.rope_tables([611], dh, base)
    np.testing.assert_allclose(ca * cb - sa * sb, cc, atol=1e-12)
    np.testing.assert_allclose(sa * cb + ca * sb, sc, atol=1e-12)
    # a different base changes every pair but the first
    c2, _ = orc.rope_tables([35], dh, 500000.0)
    assert c2[0, 0] == cos[3, 0] and np.all(c2[0, 1:] != cos[3, 1:])


def test_variant_weighted_merge_and_mean_key_similarity():
    # Variants beside Sec. 3.3.2's choices.  Weighted merge: equal weights give the plain mean;
    # a source of weight zero leaves its destination untouched; the weighted sum is preserved
    # (sum_j W_j X'_j = sum over the survivors of w_x X_x); weights that add up to nothing fall
    # back to the plain mean.  Mean-key features: with one head they are the keys themselves; the
    # similarity on them is the brute-force cosine.
    rng = np.random.default_rng(12)
    N, w = 10, 6
    R = rng.standard_normal((N, w))
    kept, src, dst = [0, 2, 5, 7], [3, 4, 9], [2, 2, 7]
    plain = orc.compact_rows(R, kept, src, dst, np.float64)
    same = orc.compact_rows(R, kept, src, dst, np.float64, weights=np.full(N, 0.25))
    np.testing.assert_allclose(same, plain, rtol=1e-15)
    wts = rng.uniform(0.5, 2.0, N)
    wts32 = wts.astype(np.float32).astype(np.float64)
    out = orc.compact_rows(R, kept, src, dst, np.float64, weights=wts)
    np.testing.assert_allclose(out[1], (wts32[2] * R[2] + wts32[3] * R[3] + wts32[4] * R[4])
                               / (wts32[2] + wts32[3] + wts32[4]), rtol=1e-14)
    assert np.array_equal(out[0], R[0]) and np.array_equal(out[2], R[5])
    W = np.array([wts32[0], wts32[2] + wts32[3] + wts32[4], wts32[5], wts32[7] + wts32[9]])
    surv = [0, 2, 3, 4, 5, 7, 9]
    np.testing.assert_allclose((W[:, None] * out).sum(0), sum(wts32[x] * R[x] for x in surv), rtol=1e-13)
    w0 = wts.copy()
    w0[9] = 0.0
    np.testing.assert_allclose(orc.compact_rows(R, kept, src, dst, np.float64, weights=w0)[3], R[7], rtol=1e-15)
    np.testing.assert_allclose(orc.compact_rows(R, kept, src, dst, np.float64, weights=np.zeros(N)), plain)
    K = rng.standard_normal((3, N, 4))
    np.testing.assert_allclose(orc.mean_heads(K), K.mean(axis=0), rtol=1e-15)
    assert np.array_equal(orc.mean_heads(K[:1]), K[0])
    F = orc.mean_heads(K)
    sim = orc.similarity(F, [1, 4], [0, 6, 8])
    for j, b in enumerate([0, 6, 8]):
        for i, a in enumerate([1, 4]):
            want = F[b] @ F[a] / (np.linalg.norm(F[b]) * np.linalg.norm(F[a]))
            assert abs(sim[j, i] - want) < 1e-14


def test_round_to_storage_bf16_is_round_to_nearest_even():
    # bfloat16 keeps the top 16 bits of a float32: 1 + 2^-8 is half-way between 1 and 1 + 2^-7
    # (goes to the even one, 1), 1 + 3 * 2^-8 half-way between 1 + 2^-7 and 1 + 2^-6 (goes up)
    x = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -30, -2.5, 3.0e38, 1e-40])
    got = orc.round_to_storage(x, "bf16")
    assert got.dtype == np.float32
    assert got[0] == 1.0 and got[1] == 1.0 and got[2] == 1.0 + 2.0 ** -6 and got[3] == 1.0 + 2.0 ** -7
    assert got[4] == -2.5
    assert np.all((got.view(np.uint32) & 0xFFFF) == 0)
    rng = np.random.default_rng(2)
    y = rng.standard_normal(2000) * 10.0
    r = orc.round_to_storage(y, "bf16").astype(np.float64)
    assert np.all(np.abs(r - y) <= np.abs(y) * 2.0 ** -8)


def test_layer2_probe_closed_forms():
    # Eq. 3-1 / 3-2 on [system, visual, prompt].  Pins: every probability row sums to one over
    # the keys it may see, so its visual part sums to at most one; all keys equal => uniform
    # probabilities and Z = the running mean of V (causal) or the mean of V (not causal); one key
    # that dominates a row => that row of Z is that key's V; causal rows do not change when later
    # keys and values change; the loop route and the matrix route agree.
    rng = np.random.default_rng(21)
    H, dh, n_sys, n_vis, n_text = 2, 8, 3, 6, 4
    L = n_sys + n_vis + n_text
    Q = rng.standard_normal((H, L, dh))
    K = rng.standard_normal((H, L, dh))
    V = rng.standard_normal((H, L, dh))
    probe = list(range(n_sys + n_vis, L))
    O, A = orc.layer2_probe(Q, K, V, n_sys, n_vis, probe)
    O2, A2 = orc.layer2_probe_matrix(Q, K, V, n_sys, n_vis, probe)
    np.testing.assert_allclose(O, O2, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(A, A2, rtol=1e-12, atol=1e-14)
    assert O.shape == (n_vis, H * dh) and A.shape == (H, n_text, n_vis)
    assert np.all(A >= 0) and np.all(A.sum(axis=2) <= 1.0 + 1e-12)
    # equal keys: uniform attention
    Ke = np.broadcast_to(K[:, :1], K.shape).copy()
    Oe, Ae = orc.layer2_probe(Q, Ke, V, n_sys, n_vis, probe)
    for x in range(n_vis):
        i = n_sys + x
        np.testing.assert_allclose(Oe[x, :dh], V[0, :i + 1].mean(axis=0), rtol=1e-12)
    for t, i in enumerate(probe):
        np.testing.assert_allclose(Ae[:, t, :], 1.0 / (i + 1), rtol=1e-12)
    On, An = orc.layer2_probe(Q, Ke, V, n_sys, n_vis, probe, causal=False)
    np.testing.assert_allclose(On[:, dh:], np.broadcast_to(V[1].mean(axis=0), (n_vis, dh)), rtol=1e-12)
    np.testing.assert_allclose(An, 1.0 / L, rtol=1e-12)
    # a dominating key
    Kd = K.copy()
    Kd[0, 2] = 80.0 * Q[0, n_sys + 4] / np.linalg.norm(Q[0, n_sys + 4])
    Od, _ = orc.layer2_probe(Q, Kd, V, n_sys, n_vis, probe)
    np.testing.assert_allclose(Od[4, :dh], V[0, 2], atol=1e-6)
    # causality: later keys / values do not reach earlier rows
    K2, V2 = K.copy(), V.copy()
    K2[:, n_sys + 3:] += 1.0
    V2[:, n_sys + 3:] -= 2.0
    O3, _ = orc.layer2_probe(Q, K2, V2, n_sys, n_vis, probe)
    assert np.array_equal(O3[:3], O[:3]) and not np.allclose(O3[3:], O[3:])
    # a probe row in front of some visual tokens sees nothing of them
    _, Ap = orc.layer2_probe(Q, K, V, n_sys, n_vis, [n_sys + 1])
    assert np.all(Ap[:, 0, 2:] == 0.0) and np.all(Ap[:, 0, :2] > 0.0)
