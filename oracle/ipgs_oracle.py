"""Float64 CPU oracle for the two-stage IPGS visual-token compression of TokenCarve.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
path computes, written from the paper's equations.  It is imported by the tests,
by the smoke check and by the benchmark's CPU-baseline leg, and by nothing else:
the CUDA library never calls it and shares no code, table or constant with it.

Everything is float64 numpy.  Library primitives are used only as single steps
the paper itself names (an SVD, a matrix product, a sort); there is no blocking,
fusion or reordering.  A LAPACK-free one-sided Jacobi SVD (`svd_jacobi`) is kept
beside the LAPACK call so each can check the other.

Paper passages followed (TokenCarve, Sec. 3.3; Sec. 3.2 for `token_information`; Sec. 3.1
Eq. 3-1 / 3-2 for `layer2_probe`, the producer of the matrices the compression reads):
  Sec. 3.2    the information quantity of the visual tokens is measured by the
              matrix rank of their rows of the attention-output matrix, followed
              as tokens are removed (Visual Token Information curve; appendix
              "Attention Output Matrix Rank").
  Sec. 3.3.1  Z = U Sigma V^T; row expansion Eq. 3-5; information contribution
              score Eq. 3-6; attention score Eq. 3-7; combined score Eq. 3-8;
              Stage I keeps L_vc (1 + rho) tokens.
  Sec. 3.3.2  Set A / Set B split of the survivors by descending score Eq. 3-9;
              cosine similarity of normalised attention-output rows Eq. 3-10;
              the L_vc * rho Set-B tokens with the highest similarity are merged
              into their Set-A match with ToMe's average; the rest stay intact;
              L_vc tokens result.
  Conclusion  surviving tokens keep their original positional relationships
              (`reassemble`, `rope_tables`).

Readings taken where the paper is silent (each is a parameter or a stated rule):
  * r in Eq. 3-5/3-6 is the numerical rank  #{sigma_i > rank_tol * sigma_1};
    rank_tol = 0 sums every min(N, d) term.
  * Eq. 3-8 is applied to the raw C and S ("none"), or to C / sum(C) and
    S / sum(S) ("sum1") as an opt-in variant.
  * M = floor(L_vc * rho) clamped to [0, N - L_vc];  P = L_vc + M survivors;
    Set A gets floor(P / 2), Set B the rest.
  * All ties are broken towards the lower original token index.
  * Decisions (orderings, arg-max) are taken on float32-rounded scores /
    similarities, the precision in which the library stores them.
  * "Norm" in Eq. 3-10 is the L2 row normalisation  x / max(|x|_2, 1e-12).
  * The merged token is the unweighted mean of the destination and every source
    that chose it; K and V get the same map per head (an extension: the paper
    merges tokens, it does not say K/V).  Variants kept beside the paper's choices:
    matching on the hidden states or on the head-mean keys (ToMe's features), and a
    mean weighted by the IPGS scores.
  * Output rows are in ascending original index; that index list is returned.
  * `layer2_probe`: the attention is causal (a decoder-only LLM), Q and K arrive with
    their rotary encodings applied, Z is taken before the output projection with the
    heads side by side, and the rows whose attention Eq. 3-7 averages are a parameter.

Parity status: every function below is pinned by tests against closed forms,
invariants, brute force or an independent routine, except `carve` as a whole
against the paper's own end-task numbers: the paper prints no intermediate
values, so end-to-end agreement with the authors' run is "parity unpinned".
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

F64 = np.float64


# --------------------------------------------------------------------------
# counts
# --------------------------------------------------------------------------
def resolve_counts(n_tokens: int, keep: int, rho: float = 0.5,
                   n_merge: int = -1) -> Tuple[int, int, int, int]:
    """(M, P, nA, nB): merged count, Stage-I survivors, |Set A|, |Set B|.

    Stage I keeps L_vc (1 + rho) tokens (Sec. 3.3.1, last paragraph); Stage II
    merges L_vc * rho of them (Sec. 3.3.2, last paragraph); Eq. 3-9 cuts the
    sorted survivors at half.
    """
    if not (1 <= keep <= n_tokens):
        raise ValueError("keep out of range")
    if n_merge < 0:
        if not (0.0 <= rho <= 1.0):
            raise ValueError("rho out of range")
        M = int(np.floor(F64(keep) * F64(np.float32(rho))))
    else:
        M = int(n_merge)
    M = max(0, min(M, n_tokens - keep))
    P = keep + M
    nA = P // 2
    nB = P - nA
    if M > nB:
        raise ValueError("n_merge exceeds |Set B|")
    return M, P, nA, nB


# --------------------------------------------------------------------------
# SVD (Sec. 3.3.1) -- two independent routes
# --------------------------------------------------------------------------
def svd_lapack(O: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """U [N, q], sigma [q] (descending), q = min(N, d): the thin SVD as a library step."""
    U, s, _ = np.linalg.svd(np.asarray(O, F64), full_matrices=False)
    return U, s


def svd_jacobi(O: np.ndarray, max_sweeps: int = 60, tol: float = 1e-15
               ) -> Tuple[np.ndarray, np.ndarray]:
    """One-sided (Hestenes) Jacobi SVD written out with plain loops.

    Works on M = O^T when N <= d (so the N columns of M are the tokens) and
    orthogonalises the columns of M J; the accumulated J is then U and the
    column norms are sigma.  For N > d it works on O's columns and recovers U
    from the rotated matrix.  Small inputs only (O(N^2 d) per sweep in Python).
    """
    O = np.asarray(O, F64)
    N, d = O.shape
    if N <= d:
        M = O.T.copy()                 # d x N, columns = tokens
        J = np.eye(N)
        n = N
    else:
        M = O.copy()                   # N x d, columns = features
        J = None
        n = d
    for _ in range(max_sweeps):
        rotated = False
        for p in range(n - 1):
            for q in range(p + 1, n):
                a = M[:, p] @ M[:, p]
                b = M[:, q] @ M[:, q]
                g = M[:, p] @ M[:, q]
                if abs(g) <= tol * np.sqrt(a * b) or g == 0.0:
                    continue
                rotated = True
                zeta = (b - a) / (2.0 * g)
                t = np.sign(zeta) / (abs(zeta) + np.sqrt(1.0 + zeta * zeta)) if zeta != 0 else 1.0
                c = 1.0 / np.sqrt(1.0 + t * t)
                s = c * t
                mp = M[:, p].copy()
                M[:, p] = c * mp - s * M[:, q]
                M[:, q] = s * mp + c * M[:, q]
                if J is not None:
                    jp = J[:, p].copy()
                    J[:, p] = c * jp - s * J[:, q]
                    J[:, q] = s * jp + c * J[:, q]
        if not rotated:
            break
    sig = np.sqrt(np.sum(M * M, axis=0))
    order = np.argsort(-sig, kind="stable")
    sig = sig[order]
    if J is not None:
        U = J[:, order]
    else:
        U = np.zeros((N, n))
        for k, j in enumerate(order):
            U[:, k] = M[:, j] / sig[k] if sig[k] > 0 else 0.0
    return U, sig


def numerical_rank(sigma: np.ndarray, rank_tol: float) -> int:
    """r = #{ sigma_i > rank_tol * sigma_1 } (upper limit of the sums in Eq. 3-5 / 3-6)."""
    if sigma.size == 0 or sigma[0] <= 0.0:
        return 0
    return int(np.sum(sigma > F64(np.float32(rank_tol)) * sigma[0]))


def token_information(O: np.ndarray, idx: Optional[Sequence[int]], rank_tol: float,
                      method: str = "lapack") -> Tuple[np.ndarray, int]:
    """Information quantity of a set of visual tokens (Sec. 3.2, "Visual Token Information";
    appendix "Attention Output Matrix Rank"): the matrix rank of the rows of the attention
    output that belong to the tokens `idx` (all rows when idx is None), taken as the numerical
    rank #{sigma_i > rank_tol * sigma_1}.  Returns (sigma descending [min(n, d)], rank)."""
    rows = np.asarray(O, F64) if idx is None else np.asarray(O, F64)[np.asarray(list(idx), int)]
    _, sigma = svd_lapack(rows) if method == "lapack" else svd_jacobi(rows)
    return sigma, numerical_rank(sigma, rank_tol)


def reassemble(Hs: np.ndarray, n_sys: int, n_vis: int, Xo: np.ndarray, kept_idx: Sequence[int]
               ) -> Tuple[np.ndarray, np.ndarray]:
    """Sequence after the compression (Sec. 3.1: the input is [system, visual, prompt] tokens;
    Sec. 3.2: the visual part is rows L_s .. L_s + L_v; Conclusion: the surviving tokens keep
    their original position IDs).  Hs [L, d] holds all L = n_sys + n_vis + n_text hidden states
    before it, Xo [keep, d] the compacted visual tokens in ascending original order, kept_idx
    their original visual-token numbers.  Returns (rows [n_sys + keep + n_text, d] in Hs's dtype,
    original position of every row)."""
    kept = np.asarray(list(kept_idx), np.int64)
    L = Hs.shape[0]
    rows = np.concatenate([Hs[:n_sys], np.asarray(Xo, Hs.dtype), Hs[n_sys + n_vis:]], axis=0)
    pos = np.concatenate([np.arange(n_sys), n_sys + kept, np.arange(n_sys + n_vis, L)])
    return rows, pos.astype(np.int64)


def rope_tables(pos: Sequence[int], head_dim: int, base: float = 10000.0
                ) -> Tuple[np.ndarray, np.ndarray]:
    """Rotary-encoding tables for the rows of the re-assembled sequence (Conclusion: the
    surviving tokens keep their original position IDs, so the layers after the compression
    rotate queries and keys by those positions, not by the new row numbers).  Rotary position
    embedding as published (RoFormer): pair i of a head's dimensions is rotated by the angle
    pos * theta_i with theta_i = base^(-2 i / head_dim).  Returns (cos, sin), each
    [len(pos), head_dim / 2], float64."""
    assert head_dim % 2 == 0
    half = head_dim // 2
    cos = np.zeros((len(pos), half), F64)
    sin = np.zeros((len(pos), half), F64)
    for j, p in enumerate(pos):
        for i in range(half):
            theta = F64(base) ** (-2.0 * i / head_dim)
            cos[j, i] = np.cos(F64(int(p)) * theta)
            sin[j, i] = np.sin(F64(int(p)) * theta)
    return cos, sin


# --------------------------------------------------------------------------
# the layer-2 probe: what IPGS reads from the second LLM layer (Sec. 3.1, Sec. 3.2)
# --------------------------------------------------------------------------
def layer2_probe(Q: np.ndarray, K: np.ndarray, V: np.ndarray, n_sys: int, n_vis: int,
                 probe_rows: Sequence[int], causal: bool = True
                 ) -> Tuple[np.ndarray, np.ndarray]:
    """Attention of one layer on the sequence [system, visual, prompt] (Sec. 3.1):
    A = Softmax(Q K^T / sqrt(d_k)) per head (Eq. 3-1), Z = A V (Eq. 3-2), and from them the two
    things the compression reads (Sec. 3.2, Sec. 3.3.1): the visual rows of Z with the heads
    side by side, O [n_vis, H * dh], and the attention the rows `probe_rows` pay to the visual
    tokens, A_slice [H, len(probe_rows), n_vis] (the slice Eq. 3-7 averages).
    Q, K, V: [H, L, dh], L = n_sys + n_vis + n_text, taken as given (rotary encodings, if any,
    already applied).  causal: row i attends to the keys j <= i, as in a decoder-only LLM (the
    paper's LLaVA models); False lets every row see every key.
    Plain loops over heads and rows; nothing is blocked or fused."""
    Q = np.asarray(Q, F64)
    K = np.asarray(K, F64)
    V = np.asarray(V, F64)
    H, L, dh = Q.shape
    scale = 1.0 / np.sqrt(F64(dh))
    O = np.zeros((n_vis, H * dh), F64)
    A_slice = np.zeros((H, len(probe_rows), n_vis), F64)
    for h in range(H):
        for i in list(range(n_sys, n_sys + n_vis)) + [int(r) for r in probe_rows]:
            last = i + 1 if causal else L
            logits = np.array([np.dot(Q[h, i], K[h, j]) * scale for j in range(last)])
            logits -= logits.max()
            w = np.exp(logits)
            w /= w.sum()
            if n_sys <= i < n_sys + n_vis:
                z = np.zeros(dh, F64)
                for j in range(last):
                    z += w[j] * V[h, j]
                O[i - n_sys, h * dh:(h + 1) * dh] = z
        for t, i in enumerate(probe_rows):
            last = int(i) + 1 if causal else L
            logits = np.array([np.dot(Q[h, int(i)], K[h, j]) * scale for j in range(last)])
            logits -= logits.max()
            w = np.exp(logits)
            w /= w.sum()
            for x in range(n_vis):
                j = n_sys + x
                A_slice[h, t, x] = w[j] if j < last else 0.0
    return O, A_slice


def layer2_probe_matrix(Q: np.ndarray, K: np.ndarray, V: np.ndarray, n_sys: int, n_vis: int,
                        probe_rows: Sequence[int], causal: bool = True
                        ) -> Tuple[np.ndarray, np.ndarray]:
    """The same quantities by the textbook route (one matrix product per head, a masked
    softmax over whole rows): fast enough for the benchmark-sized checks, and a second route
    the loop version is pinned against."""
    Q = np.asarray(Q, F64)
    K = np.asarray(K, F64)
    V = np.asarray(V, F64)
    H, L, dh = Q.shape
    O = np.zeros((n_vis, H * dh), F64)
    A_slice = np.zeros((H, len(probe_rows), n_vis), F64)
    rows = np.array(list(range(n_sys, n_sys + n_vis)) + [int(r) for r in probe_rows])
    for h in range(H):
        S = (Q[h, rows] @ K[h].T) / np.sqrt(F64(dh))
        if causal:
            S = np.where(np.arange(L)[None, :] <= rows[:, None], S, -np.inf)
        S = S - S.max(axis=1, keepdims=True)
        W = np.exp(S)
        W /= W.sum(axis=1, keepdims=True)
        O[:, h * dh:(h + 1) * dh] = W[:n_vis] @ V[h]
        A_slice[h] = W[n_vis:, n_sys:n_sys + n_vis]
    return O, A_slice


# --------------------------------------------------------------------------
# scores (Sec. 3.3.1)
# --------------------------------------------------------------------------
def information_contribution(O: np.ndarray, rank_tol: float = 0.0, method: str = "lapack"
                             ) -> Tuple[np.ndarray, np.ndarray, int]:
    """C(x) = sum_{i<=r} |u_xi sigma_i|  (Eq. 3-6).  Returns (C [N], sigma [q], r)."""
    U, sigma = svd_lapack(O) if method == "lapack" else svd_jacobi(O)
    r = numerical_rank(sigma, rank_tol)
    C = np.zeros(U.shape[0])
    for i in range(r):
        C += np.abs(U[:, i] * sigma[i])
    return C, sigma, r


def attention_score(A: np.ndarray) -> np.ndarray:
    """S(x) = mean over heads and query rows of A[:, :, x]  (Eq. 3-7).  A is [H, T, N]."""
    A = np.asarray(A, F64)
    H, T, N = A.shape
    S = np.zeros(N)
    for h in range(H):
        for t in range(T):
            S += A[h, t]
    return S / (H * T)


def combined_score(C: np.ndarray, S: np.ndarray, lam: float, score_norm: str = "none"
                   ) -> np.ndarray:
    """E(x) = (1 - lambda) C(x) + lambda S(x)  (Eq. 3-8), on raw or sum-normalised terms."""
    lam = F64(np.float32(lam))
    if not (0.0 <= lam <= 1.0):
        raise ValueError("lambda out of range")
    C = np.asarray(C, F64)
    S = np.asarray(S, F64)
    if score_norm == "sum1":
        cs, ss = C.sum(), S.sum()
        C = C / cs if cs > 0 else C
        S = S / ss if ss > 0 else S
    elif score_norm != "none":
        raise ValueError("score_norm")
    return (1.0 - lam) * C + lam * S


def score(O: np.ndarray, A: np.ndarray, lam: float = 0.5, rank_tol: float = 0.0,
          score_norm: str = "none", method: str = "lapack") -> Dict[str, np.ndarray]:
    C, sigma, r = information_contribution(O, rank_tol, method)
    S = attention_score(A)
    E = combined_score(C, S, lam, score_norm)
    return {"E": E, "C": C, "S": S, "sigma": sigma, "rank": r}


# --------------------------------------------------------------------------
# Stage I prune + Set A / Set B (Sec. 3.3.1 end, Eq. 3-9)
# --------------------------------------------------------------------------
def descending_order(values: np.ndarray) -> List[int]:
    """Indices by (value descending, index ascending); value compared in float32."""
    v = np.asarray(values, F64).astype(np.float32)
    idx = list(range(len(v)))
    idx.sort(key=lambda i: (-float(v[i]), i))
    return idx


def prune_split(E: np.ndarray, P: int, nA: int) -> Tuple[np.ndarray, np.ndarray]:
    """Survivors = the P best tokens; Set A = the first nA of them, Set B = the rest
    (Eq. 3-9: IndexSort is the descending-score order of the IPGS scores)."""
    order = descending_order(E)
    setA = np.array(order[:nA], dtype=np.int32)
    setB = np.array(order[nA:P], dtype=np.int32)
    return setA, setB


# --------------------------------------------------------------------------
# Stage II similarity, matching, merge selection (Eq. 3-10 and the paragraph after it)
# --------------------------------------------------------------------------
def normalise_rows(O: np.ndarray) -> np.ndarray:
    O = np.asarray(O, F64)
    out = np.empty_like(O)
    for x in range(O.shape[0]):
        nrm = np.sqrt(np.sum(O[x] * O[x]))
        out[x] = O[x] / max(nrm, 1e-12)
    return out


def mean_heads(K: np.ndarray) -> np.ndarray:
    """Mean over the heads of K [H, N, dh] -> [N, dh]: the token features ToMe matches on (the
    paper's Sec. 3.3.2 takes its merging from ToMe but matches on the attention output; this is
    the variant with ToMe's own choice of features)."""
    K = np.asarray(K, F64)
    out = np.zeros(K.shape[1:], F64)
    for h in range(K.shape[0]):
        out += K[h]
    return out / K.shape[0]


def similarity(O: np.ndarray, setA: Sequence[int], setB: Sequence[int]) -> np.ndarray:
    """Simi_AB [nB, nA] = Norm(Z)[Set B] x Norm(Z)[Set A]^T  (Eq. 3-10).  Z is the matrix whose
    rows describe the tokens: the attention output in the paper; the variants pass the hidden
    states or the head-mean keys instead."""
    Zn = normalise_rows(O)
    return Zn[np.asarray(setB, int)] @ Zn[np.asarray(setA, int)].T


def match_and_select(sim: np.ndarray, setA: Sequence[int], setB: Sequence[int], M: int
                     ) -> Tuple[np.ndarray, np.ndarray]:
    """Each Set-B token's best Set-A partner, then the M Set-B tokens with the highest
    best-similarity.  Returns (merge_src [M], merge_dst [M]) as original token indices,
    in selection order (best first).  Ties: lower original index."""
    setA = [int(a) for a in setA]
    setB = [int(b) for b in setB]
    sim32 = np.asarray(sim, F64).astype(np.float32)
    best_val = []
    best_dst = []
    for j, b in enumerate(setB):
        bv, ba = None, None
        for i, a in enumerate(setA):
            v = float(sim32[j, i])
            if bv is None or v > bv or (v == bv and a < ba):
                bv, ba = v, a
        best_val.append(bv)
        best_dst.append(ba)
    cand = list(range(len(setB)))
    cand.sort(key=lambda j: (-best_val[j], setB[j]))
    chosen = cand[:M]
    src = np.array([setB[j] for j in chosen], dtype=np.int32)
    dst = np.array([best_dst[j] for j in chosen], dtype=np.int32)
    return src, dst


def merge(O: np.ndarray, setA: Sequence[int], setB: Sequence[int], M: int
          ) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """(merge_src, merge_dst, kept_idx) for given sets; kept = Set A ∪ unmerged Set B, ascending."""
    if M > 0 and len(setA) > 0:
        sim = similarity(O, setA, setB)
        src, dst = match_and_select(sim, setA, setB, M)
    else:
        src = np.zeros(0, np.int32)
        dst = np.zeros(0, np.int32)
    merged = set(int(s) for s in src)
    kept = sorted([int(a) for a in setA] + [int(b) for b in setB if int(b) not in merged])
    return src, dst, np.array(kept, dtype=np.int32)


# --------------------------------------------------------------------------
# merge + compaction of X, K, V
# --------------------------------------------------------------------------
def round_to_storage(x: np.ndarray, out_dtype) -> np.ndarray:
    """Round float64 values once, to nearest even, to the storage type.  "bf16" (which numpy
    does not have) gives float32 values that are exactly representable in bfloat16."""
    if isinstance(out_dtype, str) and out_dtype == "bf16":
        f = np.asarray(x, F64).astype(np.float32)
        u = f.view(np.uint32).astype(np.uint64)
        # float64 -> float32 -> bfloat16 is a double rounding only when the float32 lands
        # exactly half-way between two bfloat16 values; redo those few from the float64
        u16 = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint32) << 16
        out = u16.astype(np.uint32).view(np.float32).reshape(f.shape)
        tie = (u & 0xFFFF) == 0x8000
        if np.any(tie):
            x64 = np.asarray(x, F64)
            lo = ((u >> 16) << 16).astype(np.uint32).view(np.float32).reshape(f.shape)
            hi = (((u >> 16) + 1) << 16).astype(np.uint32).view(np.float32).reshape(f.shape)
            mid = 0.5 * (lo.astype(F64) + hi.astype(F64))
            fix = np.where(np.abs(x64) > np.abs(mid), hi, np.where(np.abs(x64) < np.abs(mid), lo, out))
            out = np.where(tie.reshape(f.shape), fix, out).astype(np.float32)
        return out
    return np.asarray(x, F64).astype(out_dtype)


def compact_rows(R: np.ndarray, kept_idx: Sequence[int], merge_src: Sequence[int],
                 merge_dst: Sequence[int], out_dtype, weights: Optional[np.ndarray] = None
                 ) -> np.ndarray:
    """Rows `kept_idx` of R [N, w]; a kept row that is a merge destination becomes the
    plain mean of itself and all its sources (ToMe average with unit sizes), computed
    in float64 and rounded once (to nearest even) to the storage dtype.  With `weights`
    [N] (the variant: IPGS scores, float32-rounded like every decision input) the mean is
    weighted, sum(w_i R_i) / sum(w_i) over the group; a group whose weights do not add up to a
    positive number falls back to the plain mean."""
    R = np.asarray(R, F64)
    w = None if weights is None else np.asarray(weights, F64).astype(np.float32).astype(F64)
    out = np.empty((len(kept_idx), R.shape[1]), F64)
    for j, a in enumerate(kept_idx):
        group = [int(a)] + [int(s) for s, t in zip(merge_src, merge_dst) if int(t) == int(a)]
        tot = sum(w[g] for g in group) if w is not None else 0.0
        if w is not None and tot > 0.0 and len(group) > 1:
            acc = np.zeros(R.shape[1], F64)
            for g in group:
                acc += w[g] * R[g]
            out[j] = acc / tot
        else:
            acc = np.zeros(R.shape[1], F64)
            for g in group:
                acc += R[g]
            out[j] = acc / len(group)
    return round_to_storage(out, out_dtype)


def compact(X: np.ndarray, K: Optional[np.ndarray], V: Optional[np.ndarray],
            kept_idx: Sequence[int], merge_src: Sequence[int], merge_dst: Sequence[int],
            out_dtype, weights: Optional[np.ndarray] = None) -> Dict[str, Optional[np.ndarray]]:
    """X' [keep, d], K' / V' [H, keep, dh] under one merge map."""
    res: Dict[str, Optional[np.ndarray]] = {
        "X": compact_rows(X, kept_idx, merge_src, merge_dst, out_dtype, weights), "K": None, "V": None}
    for name, T in (("K", K), ("V", V)):
        if T is not None:
            res[name] = np.stack([compact_rows(T[h], kept_idx, merge_src, merge_dst, out_dtype, weights)
                                  for h in range(T.shape[0])], axis=0)
    return res


# --------------------------------------------------------------------------
# the whole path for one image
# --------------------------------------------------------------------------
def carve(O: np.ndarray, A: np.ndarray, X: np.ndarray, K: Optional[np.ndarray],
          V: Optional[np.ndarray], keep: int, rho: float = 0.5, lam: float = 0.5,
          rank_tol: float = 0.0, score_norm: str = "none", n_merge: int = -1,
          method: str = "lapack", sim_source: str = "O", weighted: bool = False,
          out_dtype=None) -> Dict[str, object]:
    """score -> prune -> split -> similarity -> match/select -> merge -> compact, one image.

    Inputs are taken as given (already rounded to their storage dtype); outputs X', K', V'
    are rounded to X's dtype (or `out_dtype`).  Variants beside the paper's choices:
    sim_source "X" / "meanK" matches on the hidden states / the head-mean keys instead of the
    attention output; weighted = True merges with the IPGS scores as weights."""
    N = O.shape[0]
    M, P, nA, nB = resolve_counts(N, keep, rho, n_merge)
    sc = score(O, A, lam, rank_tol, score_norm, method)
    setA, setB = prune_split(sc["E"], P, nA)
    feats = {"O": O, "X": X, "meanK": None if K is None else mean_heads(K)}[sim_source]
    src, dst, kept = merge(np.asarray(feats, F64), setA, setB, M)
    out = compact(X, K, V, kept, src, dst, X.dtype if out_dtype is None else out_dtype,
                  sc["E"] if weighted else None)
    return {**sc, "M": M, "P": P, "setA": setA, "setB": setB, "merge_src": src,
            "merge_dst": dst, "kept_idx": kept, "Xo": out["X"], "Ko": out["K"], "Vo": out["V"]}
