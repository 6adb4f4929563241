"""CUDA path against the float64 oracle, through the C ABI, on the same seeded inputs."""
import numpy as np
import pytest
import torch

from oracle import ipgs_oracle as orc
from paper_2503_10501_b200 import binding as tcb
from paper_2503_10501_b200 import inputs
import parity_util as pu

pytestmark = pytest.mark.gpu


def dev(a, bf16=False):
    """Device tensor of a numpy array; bf16: the float32 array holds bfloat16 values."""
    if a is None:
        return None
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    return t.to(torch.bfloat16) if bf16 else t


def host(t):
    if t is None:
        return None
    return (t.float() if t.dtype == torch.bfloat16 else t).cpu().numpy()


def params_of(cfg, **over):
    kw = dict(batch=cfg.batch, n_tokens=cfg.n_tokens, d_model=cfg.d_model, n_heads=cfg.n_heads,
              head_dim=cfg.head_dim, n_query=cfg.n_query, keep=cfg.keep, rho=cfg.rho, lam=cfg.lam,
              rank_tol=cfg.rank_tol, dtype=cfg.dtype, rank_cap=cfg.rank_cap)
    kw.update(over)
    return tcb.Params(**kw)


def run_staged(p, batch, with_kv=True):
    """Every stage through its own entry point, each fed with the previous stage's CUDA output."""
    bf = p.dtype == "bf16"
    O, A, X = dev(batch["O"], bf), dev(batch["A"], bf), dev(batch["X"], bf)
    K = dev(batch["K"], bf) if with_kv else None
    V = dev(batch["V"], bf) if with_kv else None
    ws = tcb.workspace(p)
    sc = tcb.tc_score(p, O, A, ws)
    setA, setB = tcb.tc_prune(p, sc["E"], ws)
    feats = {"O": O, "X": X, "meanK": K}[p.sim_source]     # what Eq. 3-10 is taken on
    src, dst, kept = tcb.tc_merge(p, feats, setA, setB, ws)
    if p.weighted_merge:
        Xo, Ko, Vo = tcb.tc_compact_weighted(p, X, K, V, kept, src, dst, sc["E"], ws)
    else:
        Xo, Ko, Vo = tcb.tc_compact(p, X, K, V, kept, src, dst, ws)
    cX, cK, cV, ckept, cstatus = tcb.tc_carve(p, O, A, X, K, V, ws)
    torch.cuda.synchronize()
    res = {k: host(v) for k, v in sc.items()}
    res.update(setA=host(setA), setB=host(setB), src=host(src), dst=host(dst), kept=host(kept),
               Xo=host(Xo), Ko=host(Ko), Vo=host(Vo), cX=host(cX), cK=host(cK), cV=host(cV),
               ckept=host(ckept), cstatus=host(cstatus))
    return res


def image_slice(res, b, with_kv=True):
    g = {k: res[k][b] for k in ("E", "C", "S", "sigma", "rank", "setA", "setB", "src", "dst",
                                "kept", "Xo")}
    g["Ko"] = res["Ko"][b] if with_kv else None
    g["Vo"] = res["Vo"][b] if with_kv else None
    return g


def cfgp_of(p):
    return dict(keep=p.keep, rho=p.rho, n_merge=p.n_merge, lam=p.lam, rank_tol=p.rank_tol,
                score_norm=p.score_norm, sim_source=p.sim_source, weighted=p.weighted_merge,
                dtype=p.dtype)


def check_config(cfg, images, with_kv=True, max_flips=0, **over):
    """Staged and fused calls on the configuration, sampled images against the oracle.
    max_flips: how many tokens in all may sit on the other side of a cut than in the oracle
    (always inside the band the float32 scores cannot resolve, see parity_util); the count of
    tokens inside the band is printed so that the weight of "exact outside the band" shows."""
    p = params_of(cfg, **over)
    batch = inputs.make_batch(cfg)
    res = run_staged(p, batch, with_kv)
    assert np.all(res["img_status"] == 0), res["img_status"]
    assert np.all(res["cstatus"] == 0), res["cstatus"]
    # the fused call must reproduce the staged calls
    assert np.array_equal(res["ckept"], res["kept"])
    assert np.array_equal(res["cX"], res["Xo"])
    if with_kv:
        assert np.array_equal(res["cK"], res["Ko"]) and np.array_equal(res["cV"], res["Vo"])
    flips = {"flips_sets": 0, "flips_merge": 0, "in_band": 0}
    for b in images:
        im = {k: batch[k][b] for k in batch}
        if not with_kv:
            im.pop("K"), im.pop("V")
        f = pu.check_image(cfgp_of(p), im, image_slice(res, b, with_kv))
        print(f"{cfg.name} image {b}: tokens inside the score band {f['in_band']}, "
              f"flips at the score cuts {f['flips_sets']}, in the matching {f['flips_merge']}")
        for k in f:
            flips[k] += f[k]
    assert flips["flips_sets"] + flips["flips_merge"] <= max_flips, flips
    return flips


# ------------------------------------------------------------------ tiny shapes, full solve
@pytest.mark.parametrize("N,d,keep,rho,lam,norm,dtype", [
    (12, 16, 4, 0.5, 0.5, "none", "f32"),
    (16, 32, 7, 0.5, 0.0, "none", "f32"),
    (24, 16, 9, 0.3, 1.0, "none", "f32"),      # N > d: rank <= d
    (33, 64, 11, 1.0, 0.5, "sum1", "f32"),     # odd N (bye column in the tournament)
    (64, 128, 20, 0.5, 0.5, "sum1", "f16"),
    (40, 64, 40, 0.5, 0.5, "none", "f16"),     # keep = N: nothing pruned or merged
    (40, 64, 1, 0.0, 0.5, "none", "f16"),      # keep = 1, rho = 0: Set A empty
    (40, 64, 1, 1.0, 0.5, "none", "f16"),
    (50, 64, 10, 0.0, 0.5, "none", "f16"),     # rho = 0: pure gather
])
def test_tiny_full_solve(N, d, keep, rho, lam, norm, dtype):
    cfg = inputs.tiny_config(n_tokens=N, d_model=d, n_heads=2, head_dim=8, n_query=5, keep=keep,
                             rank=min(N, d) // 2, dtype=dtype, batch=3, seed=17 + N, noise=0.3,
                             rho=rho, lam=lam, rank_tol=0.0)
    check_config(cfg, range(3), score_norm=norm)


def test_without_kv_and_with_n_merge_override():
    cfg = inputs.tiny_config(n_tokens=48, d_model=64, n_heads=2, head_dim=8, n_query=4, keep=13,
                             rank=20, dtype="f16", batch=2, seed=5, noise=0.3, rank_tol=0.0)
    check_config(cfg, range(2), with_kv=False)
    check_config(cfg, range(2), n_merge=3)


# ------------------------------------------------------------------ medium, ragged against every tile
@pytest.mark.parametrize("rank_cap", [0, 96])
def test_medium_ragged(rank_cap):
    cfg = inputs.tiny_config(n_tokens=200, d_model=264, n_heads=3, head_dim=24, n_query=37, keep=61,
                             rank=40, dtype="f16", batch=5, seed=23, noise=0.01, tau=2.0,
                             rank_tol=2e-3, dup_frac=0.05)
    check_config(cfg, range(5), rank_cap=rank_cap, max_flips=2)


def test_maximum_token_count():
    # N = 4096 is the most the selection kernels take (16 tokens per thread); a subspace size
    # that none of the kernels is specialised for, and fewer attention rows than one chunk
    cfg = inputs.tiny_config(n_tokens=4096, d_model=256, n_heads=2, head_dim=64, n_query=8,
                             keep=512, rank=48, dtype="f16", batch=1, seed=31, noise=0.01, tau=2.0,
                             rank_tol=2e-3)
    check_config(cfg, [0], rank_cap=64, max_flips=4)


# ------------------------------------------------------------------ selection kernels alone
def test_prune_exact_with_ties():
    rng = np.random.default_rng(3)
    N, B = 576, 4
    p = tcb.Params(batch=B, n_tokens=N, d_model=64, n_heads=1, head_dim=8, n_query=1, keep=128)
    M, P, nA, nB = tcb.tc_counts(p)
    E = rng.integers(0, 40, size=(B, N)).astype(np.float32) / 8.0      # many exact ties
    E[1] = 1.0                                                          # all equal
    E[2, ::3] *= -1.0                                                   # negative scores
    setA, setB = tcb.tc_prune(p, dev(E))
    torch.cuda.synchronize()
    for b in range(B):
        a_o, b_o = orc.prune_split(E[b].astype(np.float64), P, nA)
        assert host(setA)[b].tolist() == sorted(a_o.tolist())
        assert host(setB)[b].tolist() == sorted(b_o.tolist())


def test_merge_duplicate_rows_tie_to_lower_index():
    # Set A holds two bit-identical rows; the Set-B twin of both must pick the lower index.
    N, d = 32, 64
    rng = np.random.default_rng(9)
    O = rng.standard_normal((1, N, d)).astype(np.float16)
    O[0, 20] = O[0, 5]
    O[0, 11] = O[0, 5]
    p = tcb.Params(batch=1, n_tokens=N, d_model=d, n_heads=1, head_dim=8, n_query=1, keep=6,
                   n_merge=2)
    M, P, nA, nB = tcb.tc_counts(p)            # P = 8, nA = 4, nB = 4
    setA = np.array([[3, 5, 20, 30]], np.int32)
    setB = np.array([[7, 11, 12, 25]], np.int32)
    src, dst, kept = tcb.tc_merge(p, dev(O), dev(setA), dev(setB))
    torch.cuda.synchronize()
    src, dst, kept = host(src)[0], host(dst)[0], host(kept)[0]
    assert 11 in src.tolist() and dst[src.tolist().index(11)] == 5
    pu.check_merge(O[0].astype(np.float64), setA[0], setB[0], M, src, dst, kept, 6)


# ------------------------------------------------------------------ the named workloads
@pytest.mark.parametrize("lam,norm", [(0.5, "none"), (0.5, "sum1"), (0.0, "none"), (1.0, "none")])
def test_cfg1_single_f32(lam, norm):
    cfg = inputs.CONFIGS["cfg1_single_f32"]
    check_config(cfg, [0], lam=lam, score_norm=norm, max_flips=1)


@pytest.mark.parametrize("lam,norm", [(0.5, "none"), (0.5, "sum1"), (0.0, "none"), (1.0, "none")])
def test_cfg2_llava7b(lam, norm):
    cfg = inputs.CONFIGS["cfg2_llava7b_f16"]
    check_config(cfg, [0, 7, 15], lam=lam, score_norm=norm, max_flips=2)


@pytest.mark.parametrize("norm", ["none", "sum1"])
def test_cfg3_llava13b(norm):
    cfg = inputs.CONFIGS["cfg3_llava13b_f16"]
    check_config(cfg, [1, 14], score_norm=norm, max_flips=2)


def test_cfg2_full_solve_agrees():
    cfg = inputs.CONFIGS["cfg2_llava7b_f16"].with_(batch=2)
    check_config(cfg, [0, 1], rank_cap=0, max_flips=2)


def test_rank_cap_too_small_is_reported():
    cfg = inputs.CONFIGS["cfg2_llava7b_f16"].with_(batch=1)
    p = params_of(cfg, rank_cap=96)          # the numerical rank is 128
    batch = inputs.make_batch(cfg, "OA")
    sc = tcb.tc_score(p, dev(batch["O"]), dev(batch["A"]))
    torch.cuda.synchronize()
    assert host(sc["img_status"])[0] == 6


# ------------------------------------------------------------------ the Gram matrix alone
@pytest.mark.parametrize("B,N,d", [(2, 576, 4096), (3, 200, 264), (2, 64, 128), (1, 130, 72)])
def test_gram_f16_against_float64(B, N, d):
    rng = np.random.default_rng(N + d)
    O = (rng.standard_normal((B, N, 24)) @ rng.standard_normal((24, d)) * 3.0
         + 0.01 * rng.standard_normal((B, N, d))).astype(np.float16)
    O[:, 7] = O[:, 3]                       # identical rows must give identical entries
    p = tcb.Params(batch=B, n_tokens=N, d_model=d, n_heads=1, head_dim=8, n_query=1, keep=1,
                   dtype="f16")
    G = host(tcb.tc_gram(p, dev(O)))
    torch.cuda.synchronize()
    O64 = O.astype(np.float64)
    G64 = O64 @ O64.transpose(0, 2, 1)
    scale = np.sqrt(np.einsum("bii->bi", G64))
    err = np.abs(G - G64) / (scale[:, :, None] * scale[:, None, :])
    # float32 accumulation of d products of float16 values: a few 1e-7 relative to |O_i||O_j|
    assert err.max() <= 2e-6, err.max()
    assert np.array_equal(G, G.transpose(0, 2, 1)), "G must be symmetric bit for bit"
    assert np.array_equal(G[:, 7], G[:, 3]) and np.array_equal(G[:, :, 7], G[:, :, 3])


# ------------------------------------------------------------------ large shapes
def test_cfg5_bench_point_sampled_images():
    # the launch configuration bench.py times: 64 images, T = 128, keep = 128
    cfg = inputs.CONFIGS["cfg5_sweep_f16"]
    check_config(cfg, [0, 31, 63], max_flips=2)
    check_config(cfg, [17, 50], score_norm="sum1", max_flips=2)


def test_cfg5_bench_point_in_the_bench_launch_mode():
    # bench.py times the replay of a CUDA graph of one tc_carve with eight image groups: the
    # replay must give, bit for bit, what the plain call gives (which the test above compares
    # with the oracle), and sampled images are compared with the oracle once more from it
    cfg = inputs.CONFIGS["cfg5_sweep_f16"]
    p = params_of(cfg)
    batch = inputs.make_batch(cfg)
    d = {k: dev(v) for k, v in batch.items()}
    ws = tcb.workspace(p)
    tcb.tc_set_groups(4)
    plain = [host(t) for t in tcb.tc_carve(p, d["O"], d["A"], d["X"], d["K"], d["V"], ws)]
    tcb.tc_set_groups(8)
    try:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            tcb.tc_carve(p, d["O"], d["A"], d["X"], d["K"], d["V"], ws)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        held = tcb._outputs(p, d["O"].device, True) + (
            torch.zeros(p.batch, p.keep, dtype=torch.int32, device="cuda"),
            torch.zeros(p.batch, dtype=torch.int32, device="cuda"))
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            tcb.tc_carve(p, d["O"], d["A"], d["X"], d["K"], d["V"], ws, held)
        for t in held:
            t.zero_()
        g.replay()
        g.replay()
        torch.cuda.synchronize()
    finally:
        tcb.tc_set_groups(4)
    replay = [host(t) for t in held]
    for a, b in zip(plain, replay):
        assert np.array_equal(a, b)
    assert not replay[4].any()
    # sampled images of the replay against the oracle, stage by stage: the lists the staged
    # entry points give on the same inputs (bit-identical kept_idx was asserted above) and the
    # replay's own X', K', V'
    sc = tcb.tc_score(p, d["O"], d["A"], ws)
    setA, setB = tcb.tc_prune(p, sc["E"], ws)
    src, dst, kept = tcb.tc_merge(p, d["O"], setA, setB, ws)
    torch.cuda.synchronize()
    assert np.array_equal(host(kept), replay[3])
    for b in (5, 40):
        g = {k: host(sc[k])[b] for k in ("E", "C", "S", "sigma", "rank")}
        g.update(setA=host(setA)[b], setB=host(setB)[b], src=host(src)[b], dst=host(dst)[b],
                 kept=replay[3][b], Xo=replay[0][b], Ko=replay[1][b], Vo=replay[2][b])
        f = pu.check_image(cfgp_of(p), {k: batch[k][b] for k in batch}, g)
        assert f["flips_sets"] + f["flips_merge"] <= 2, f


def test_cfg5_bench_point_properties_of_every_image():
    # what must hold for each of the 64 images at the bench point whatever the scores are, checked
    # on the staged outputs without the oracle: exact selection on the library's own scores,
    # consistent lists, untouched rows copied bit for bit, merged rows the float32 mean
    cfg = inputs.CONFIGS["cfg5_sweep_f16"]
    p = params_of(cfg)
    batch = inputs.make_batch(cfg)
    res = run_staged(p, batch)
    M, P, nA, nB = tcb.tc_counts(p)
    assert not res["img_status"].any() and not res["cstatus"].any()
    assert np.array_equal(res["ckept"], res["kept"]) and np.array_equal(res["cX"], res["Xo"])
    O64 = batch["O"].astype(np.float64)
    fro = np.sum(O64 * O64, axis=(1, 2))
    assert np.all(np.abs(np.sum(res["sigma"].astype(np.float64) ** 2, axis=1) - fro) <= 1e-3 * fro)
    assert np.all(res["rank"] == cfg.rank)
    for b in range(cfg.batch):
        E, A_, B_ = res["E"][b], res["setA"][b], res["setB"][b]
        surv = np.concatenate([A_, B_])
        assert len(set(surv.tolist())) == P and np.all(np.diff(A_) > 0) and np.all(np.diff(B_) > 0)
        out = np.setdiff1d(np.arange(cfg.n_tokens), surv)
        # selection is exact on the library's own float32 scores, ties to the lower index
        key = lambda t: (-float(E[t]), int(t))
        assert max(map(key, A_)) < min(map(key, B_)) and max(map(key, B_)) < min(map(key, out))
        src, dst, kept = res["src"][b], res["dst"][b], res["kept"][b]
        assert set(src.tolist()) <= set(B_.tolist()) and set(dst.tolist()) <= set(A_.tolist())
        assert len(set(src.tolist())) == M and np.all(np.diff(src) > 0)
        assert kept.tolist() == sorted(set(A_.tolist()) | (set(B_.tolist()) - set(src.tolist())))
        X, Xo = batch["X"][b], res["Xo"][b]
        for j, a in enumerate(kept):
            group = src[dst == a]
            if len(group) == 0:
                assert np.array_equal(Xo[j], X[a])
            else:
                acc = X[a].astype(np.float32)
                for t in group:
                    acc = acc + X[t].astype(np.float32)
                want = (acc / np.float32(len(group) + 1)).astype(np.float16)
                assert np.array_equal(Xo[j], want), (b, j)
        if b in (0, 63):  # the same map on every head of K and V
            for name in ("K", "V"):
                T_, To = batch[name][b], res[name + "o"][b]        # [H, N, dh], [H, keep, dh]
                for j, a in enumerate(kept):
                    group = src[dst == a]
                    acc = T_[:, a].astype(np.float32)
                    for t in group:
                        acc = acc + T_[:, t].astype(np.float32)
                    want = T_[:, a] if len(group) == 0 else \
                        (acc / np.float32(len(group) + 1)).astype(np.float16)
                    assert np.array_equal(To[:, j], want), (name, b, j)


@pytest.mark.parametrize("T,keep", [(32, 64), (512, 288)])
def test_cfg5_sweep_corners(T, keep):
    cfg = inputs.CONFIGS["cfg5_sweep_f16"].with_(batch=8, n_query=T, keep=keep)
    check_config(cfg, [0, 7], max_flips=2)


@pytest.mark.parametrize("norm,image", [("none", 2), ("sum1", 1)])
def test_cfg4_anyres(norm, image):
    cfg = inputs.CONFIGS["cfg4_anyres_f16"]
    check_config(cfg, [image], score_norm=norm, max_flips=4)


# ------------------------------------------------------------------ inputs with a gap at the cuts
@pytest.mark.parametrize("name,nb", [("cfg2_llava7b_f16", 4), ("cfg5_sweep_f16", 6)])
def test_gapped_scores_give_the_oracle_lists_bit_for_bit(name, nb):
    # The scores of the synthetic images are dense around the cuts (several tokens within 1e-3 of
    # the Stage-I cut and of the A/B cut of Eq. 3-9), where float32 cannot be asked to agree with
    # float64.  Here the rows next to a cut are rescaled by the test (oracle side only, see
    # parity_util.open_score_gaps) until both cuts have a gap of 3e-3: then Set A, Set B must be
    # the oracle's exactly, and so must merge_src, merge_dst and kept_idx unless two
    # similarities of Eq. 3-10 that decide a choice are closer than 1e-4 and not identical.
    cfg = inputs.CONFIGS[name].with_(batch=nb)
    p = params_of(cfg)
    cfgp = cfgp_of(p)
    batch = inputs.make_batch(cfg)
    for b in range(nb):
        batch["O"][b] = pu.open_score_gaps(batch["O"][b], batch["A"][b], cfgp)
    res = run_staged(p, batch)
    assert not res["img_status"].any() and not res["cstatus"].any()
    assert np.array_equal(res["ckept"], res["kept"])
    M, P, nA, nB = tcb.tc_counts(p)
    exact_images = 0
    for b in range(nb):
        im = {k: batch[k][b] for k in batch}
        f = pu.check_image(cfgp, im, image_slice(res, b))
        assert f["in_band"] == 0 and f["flips_sets"] == 0, f
        o = orc.carve(im["O"].astype(np.float64), im["A"].astype(np.float64), im["X"], im["K"],
                      im["V"], cfg.keep, cfg.rho, cfg.lam, cfg.rank_tol, "none")
        assert res["setA"][b].tolist() == sorted(o["setA"].tolist())
        assert res["setB"][b].tolist() == sorted(o["setB"].tolist())
        # similarities that decide something: the merge cut and each merged token's best two
        sim = orc.similarity(im["O"].astype(np.float64), sorted(o["setA"].tolist()), sorted(o["setB"].tolist()))
        best = np.sort(sim.max(axis=1))[::-1]
        tight = M < nB and best[M - 1] - best[M] <= pu.SIM_BAND
        top2 = np.sort(sim, axis=1)[:, -2:]
        rows_tight = (top2[:, 1] - top2[:, 0] <= pu.SIM_BAND) & (top2[:, 1] != top2[:, 0])
        if not tight and not rows_tight.any():
            order = np.argsort(o["merge_src"])
            assert res["src"][b].tolist() == o["merge_src"][order].tolist()
            assert res["dst"][b].tolist() == o["merge_dst"][order].tolist()
            assert res["kept"][b].tolist() == o["kept_idx"].tolist()
            assert f["flips_merge"] == 0
            exact_images += 1
    print(f"{name}: {exact_images} of {nb} images compared bit for bit with the unconditioned oracle")
    assert exact_images >= 1


# ------------------------------------------------------------------ Sec. 3.2: rank of a token set
def test_token_information_against_oracle():
    # the rank curve of Sec. 3.2 on one workload: all tokens, the tokens a carve keeps, a random
    # half, a handful (fewer rows than the rank), in shuffled order
    cfg = inputs.CONFIGS["cfg2_llava7b_f16"].with_(batch=3)
    p = params_of(cfg)
    batch = inputs.make_batch(cfg)
    O = dev(batch["O"])
    kept = host(tcb.tc_carve(p, O, dev(batch["A"]), dev(batch["X"]), dev(batch["K"]), dev(batch["V"]))[3])
    rng = np.random.default_rng(3)
    sets = {"all": None, "kept": kept,
            "half": np.stack([rng.permutation(cfg.n_tokens)[:288] for _ in range(3)]).astype(np.int32),
            "few": np.stack([rng.permutation(cfg.n_tokens)[:40] for _ in range(3)]).astype(np.int32)}
    # A token set's spectrum has no gap where rank_tol cuts, unlike the carve workloads', so the
    # comparison is the one float32 eigenvalues of a Gram matrix allow: sigma^2 within 4e-6 of
    # sigma_1^2 (the Gram entries carry ~2e-6 relative error), and the rank anywhere between the
    # counts that this band leaves open at the cut.
    pr = params_of(cfg, rank_tol=1e-2)
    for name, idx in sets.items():
        g = tcb.tc_rank(pr, O, None if idx is None else dev(idx))
        torch.cuda.synchronize()
        assert not host(g["img_status"]).any(), (name, host(g["img_status"]))
        for b in range(3):
            sig, r = orc.token_information(batch["O"][b].astype(np.float64),
                                           None if idx is None else idx[b], pr.rank_tol)
            gs = host(g["sigma"])[b].astype(np.float64)
            band = 4e-6 * sig[0] ** 2
            assert np.max(np.abs(gs[:len(sig)] ** 2 - sig ** 2)) <= band, (name, b)
            cut2 = (float(np.float32(pr.rank_tol)) * sig[0]) ** 2
            r_lo, r_hi = int(np.sum(sig ** 2 > cut2 + band)), int(np.sum(sig ** 2 > cut2 - band))
            assert r_lo <= int(host(g["rank"])[b]) <= r_hi, (name, b, int(host(g["rank"])[b]), r)
            # well above the cut the singular values themselves agree to the usual 1e-3
            big = sig > 0.05 * sig[0]
            assert pu.rel_err(gs[:len(sig)][big], sig[big]) <= pu.REL_SCORE, (name, b)
    # the order of the token list does not matter; a bad token number is reported, not a fault
    idx = sets["half"].copy()
    a = tcb.tc_rank(pr, O, dev(idx))
    b2 = tcb.tc_rank(pr, O, dev(np.ascontiguousarray(idx[:, ::-1])))
    torch.cuda.synchronize()
    assert np.array_equal(host(a["rank"]), host(b2["rank"]))
    assert pu.rel_err(host(b2["sigma"])[:, :100], host(a["sigma"])[:, :100]) <= 1e-4
    idx[1, 5] = cfg.n_tokens
    bad = tcb.tc_rank(pr, O, dev(idx))
    torch.cuda.synchronize()
    assert host(bad["img_status"]).tolist() == [0, 1, 0]


def test_reassembled_sequence_and_positions():
    cfg = inputs.CONFIGS["cfg2_llava7b_f16"].with_(batch=3)
    p = params_of(cfg)
    batch = inputs.make_batch(cfg)
    out = tcb.tc_carve(p, dev(batch["O"]), dev(batch["A"]), dev(batch["X"]), dev(batch["K"]), dev(batch["V"]))
    Xo, kept = out[0], out[3]
    rng = np.random.default_rng(8)
    for n_sys, n_text in ((35, 64), (0, 7), (5, 0), (0, 0)):
        L = n_sys + cfg.n_tokens + n_text
        Hs = rng.standard_normal((3, L, cfg.d_model)).astype(np.float16)
        Hs[:, n_sys:n_sys + cfg.n_tokens] = batch["X"]
        Ho, pos = tcb.tc_reassemble(p, n_sys, n_text, dev(Hs) if n_sys + n_text else None, Xo, kept)
        torch.cuda.synchronize()
        for b in range(3):
            rows, want = orc.reassemble(Hs[b], n_sys, cfg.n_tokens, host(Xo)[b], host(kept)[b])
            assert np.array_equal(host(Ho)[b], rows) and host(pos)[b].tolist() == want.tolist()
        # rotary tables of the re-assembled rows, from their original positions
        if n_sys == 35:
            cos, sin = tcb.tc_rope_tables(pos, cfg.head_dim, 10000.0)
            torch.cuda.synchronize()
            for b in (0, 2):
                co, so = orc.rope_tables(host(pos)[b].tolist(), cfg.head_dim, 10000.0)
                assert np.max(np.abs(host(cos)[b] - co)) <= 1.5e-7
                assert np.max(np.abs(host(sin)[b] - so)) <= 1.5e-7


# ------------------------------------------------------------------ launch modes
def test_image_groups_and_graph_replay_do_not_change_results():
    cfg = inputs.CONFIGS["cfg2_llava7b_f16"].with_(batch=6)
    p = params_of(cfg)
    batch = inputs.make_batch(cfg)
    d = {k: dev(v) for k, v in batch.items()}
    ws = tcb.workspace(p)
    outs = []
    for groups in (1, 2, 4, 8):
        tcb.tc_set_groups(groups)
        o = tcb.tc_carve(p, d["O"], d["A"], d["X"], d["K"], d["V"], ws)
        torch.cuda.synchronize()
        outs.append([host(t) for t in o])
    # the same call captured into a CUDA graph (its internal fork/join becomes graph edges)
    tcb.tc_set_groups(4)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        tcb.tc_carve(p, d["O"], d["A"], d["X"], d["K"], d["V"], ws)          # warm-up on the side stream
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    held = tcb._outputs(p, d["O"].device, True) + (
        torch.zeros(p.batch, p.keep, dtype=torch.int32, device="cuda"),
        torch.zeros(p.batch, dtype=torch.int32, device="cuda"))
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        tcb.tc_carve(p, d["O"], d["A"], d["X"], d["K"], d["V"], ws, held)
    for t in held:
        t.zero_()
    g.replay()
    torch.cuda.synchronize()
    outs.append([host(t) for t in held])
    for o in outs[1:]:
        for a, b in zip(outs[0], o):
            assert np.array_equal(a, b)
    assert not outs[0][4].any()


def test_start_waves_and_group_tails_do_not_change_results():
    # 32 images or more with eight or more groups: the groups start in four waves and every
    # group runs its own selection and gather; ragged group sizes (34 = 3,3,2,2,...)
    cfg = inputs.CONFIGS["cfg5_sweep_f16"].with_(batch=34, n_heads=4, n_query=16)
    p = params_of(cfg)
    batch = inputs.make_batch(cfg)
    d = {k: dev(v) for k, v in batch.items()}
    ws = tcb.workspace(p)
    outs = []
    try:
        for groups in (1, 4, 16):
            tcb.tc_set_groups(groups)
            o = tcb.tc_carve(p, d["O"], d["A"], d["X"], d["K"], d["V"], ws)
            torch.cuda.synchronize()
            outs.append([host(t) for t in o])
    finally:
        tcb.tc_set_groups(4)
    for o in outs[1:]:
        for a, b in zip(outs[0], o):
            assert np.array_equal(a, b)
    assert not outs[0][4].any()
    # ... and the staged calls (whole batch, no groups in their selection and gather) agree with
    # the fused ones bit for bit and with the oracle
    res = run_staged(p, batch, True)
    assert np.array_equal(res["kept"], outs[2][3]) and np.array_equal(res["Xo"], outs[2][0])
    assert np.array_equal(res["Ko"], outs[2][1]) and np.array_equal(res["Vo"], outs[2][2])
    for bi in (0, 17, 33):
        f = pu.check_image(cfgp_of(p), {k: batch[k][bi] for k in batch}, image_slice(res, bi))
        assert f["flips_sets"] + f["flips_merge"] <= 2, f


def test_refused_launcher_returns_a_status_and_leaves_the_library_usable():
    # a launcher that cannot get its tensor map (host-side refusal, injected through the test
    # hook: nothing faults on the device) must surface as a status from the call, with the
    # internal streams joined, and the next call must work and give the usual results
    cfg = inputs.CONFIGS["cfg2_llava7b_f16"].with_(batch=6)
    p = params_of(cfg)
    batch = inputs.make_batch(cfg)
    d = {k: dev(v) for k, v in batch.items()}
    ws = tcb.workspace(p)
    ref = [host(t) for t in tcb.tc_carve(p, d["O"], d["A"], d["X"], d["K"], d["V"], ws)]
    try:
        for groups in (1, 4):
            tcb.tc_set_groups(groups)
            tcb.tc_test_fail_tensor_maps(True)
            with pytest.raises(tcb.TokenCarveError) as e:
                tcb.tc_carve(p, d["O"], d["A"], d["X"], d["K"], d["V"], ws)
            assert e.value.status == 5                  # TC_ERR_CUDA
            with pytest.raises(tcb.TokenCarveError):
                tcb.tc_score(p, d["O"], d["A"], ws)
            torch.cuda.synchronize()                    # nothing is left running or waiting
            tcb.tc_test_fail_tensor_maps(False)
            out = [host(t) for t in tcb.tc_carve(p, d["O"], d["A"], d["X"], d["K"], d["V"], ws)]
            for a, b in zip(ref, out):
                assert np.array_equal(a, b)
    finally:
        tcb.tc_test_fail_tensor_maps(False)
        tcb.tc_set_groups(4)


def test_host_entry_point_matches_the_device_one():
    cfg = inputs.CONFIGS["cfg2_llava7b_f16"].with_(batch=6)       # chunks of 2, 2, 1, 1 images
    p = params_of(cfg)
    batch = inputs.make_batch(cfg)
    d = {k: dev(v) for k, v in batch.items()}
    ref = [host(t) for t in tcb.tc_carve(p, d["O"], d["A"], d["X"], d["K"], d["V"])]
    hin = {k: torch.from_numpy(v).pin_memory() for k, v in batch.items()}
    hout = tuple(torch.empty(r.shape, dtype=torch.from_numpy(r).dtype).pin_memory() for r in ref)
    ws = tcb.workspace(p, host=True)
    for _ in range(2):                                             # the second call reuses the streams
        for t in hout:
            t.zero_()
        tcb.tc_carve_host(p, hin["O"], hin["A"], hin["X"], hin["K"], hin["V"], hout, ws)
        torch.cuda.synchronize()
        for a, b in zip(ref, hout):
            assert np.array_equal(a, b.numpy())


# ------------------------------------------------------------------ caller-supplied lists
def test_staged_calls_skip_and_report_bad_list_entries():
    # Sec. 3.3.2 as staged calls: Set A / Set B, the merge lists and kept_idx come from the caller.
    # A token number outside [0, N) is skipped on the device (never an address) and reported per
    # image through tc_stage_status; the other images are untouched.
    cfg = inputs.tiny_config(n_tokens=72, d_model=64, n_heads=2, head_dim=8, n_query=5, keep=20,
                             rank=16, dtype="f16", batch=3, seed=41, noise=0.3, rank_tol=0.0)
    p = params_of(cfg)
    batch = inputs.make_batch(cfg)
    O, A, X, K, V = (dev(batch[k]) for k in "OAXKV")
    ws = tcb.workspace(p)
    sc = tcb.tc_score(p, O, A, ws)
    setA, setB = tcb.tc_prune(p, sc["E"], ws)
    src, dst, kept = tcb.tc_merge(p, O, setA, setB, ws)
    good = [host(t) for t in tcb.tc_compact(p, X, K, V, kept, src, dst, ws)]
    st = host(tcb.tc_stage_status(p, ws))
    torch.cuda.synchronize()
    assert st.tolist() == [0, 0, 0]
    N = cfg.n_tokens
    # a bad Set-A entry in image 1, a bad Set-B entry in image 2
    a2, b2 = host(setA).copy(), host(setB).copy()
    a2[1, 3] = N + 5
    b2[2, 0] = -7
    s2, d2, k2 = tcb.tc_merge(p, O, dev(a2), dev(b2), ws)
    st = host(tcb.tc_stage_status(p, ws))
    torch.cuda.synchronize()
    assert st.tolist() == [0, 1, 1]
    assert np.array_equal(host(k2)[0], host(kept)[0]) and np.array_equal(host(s2)[0], host(src)[0])
    k2h = host(k2)
    assert np.all((k2h >= -1) & (k2h < N))
    # a bad kept entry in image 0 (row of zeros), a bad merge source in image 2 (left out)
    k3, s3 = host(kept).copy(), host(src).copy()
    k3[0, 4] = N
    s3[2, 1] = 1 << 20
    out = [host(t) for t in tcb.tc_compact(p, X, K, V, dev(k3), dev(s3), dst, ws)]
    st = host(tcb.tc_stage_status(p, ws))
    torch.cuda.synchronize()
    assert st.tolist() == [1, 0, 1]
    assert not out[0][0, 4].any() and not out[1][0, :, 4].any() and not out[2][0, :, 4].any()
    assert np.array_equal(np.delete(out[0][0], 4, axis=0), np.delete(good[0][0], 4, axis=0))
    for o, g in zip(out, good):
        assert np.array_equal(o[1], g[1])
        assert np.all(np.isfinite(o.astype(np.float32)))
    # the call after a bad one starts from a clean record
    tcb.tc_compact(p, X, K, V, kept, src, dst, ws)
    st = host(tcb.tc_stage_status(p, ws))
    torch.cuda.synchronize()
    assert st.tolist() == [0, 0, 0]


# ------------------------------------------------------------------ variants beside the paper's choices
@pytest.mark.parametrize("sim_source,weighted", [("X", False), ("meanK", False), ("O", True),
                                                 ("meanK", True)])
def test_variants_similarity_source_and_weighted_merge(sim_source, weighted):
    # Eq. 3-10 on the hidden states or on the head-mean keys (ToMe's features) instead of the
    # attention output, and the merge of Sec. 3.3.2 weighted by the IPGS scores of Eq. 3-8:
    # staged and fused calls against the oracle's same variant, ragged shapes and twins
    cfg = inputs.tiny_config(n_tokens=200, d_model=264, n_heads=3, head_dim=24, n_query=37, keep=61,
                             rank=40, dtype="f16", batch=3, seed=29, noise=0.01, tau=2.0,
                             rank_tol=2e-3, dup_frac=0.05)
    check_config(cfg, range(3), rank_cap=96, max_flips=2, sim_source=sim_source,
                 weighted_merge=weighted)


def test_variants_at_a_named_workload():
    cfg = inputs.CONFIGS["cfg2_llava7b_f16"].with_(batch=4)
    check_config(cfg, [0, 3], max_flips=2, sim_source="meanK", weighted_merge=True, score_norm="sum1")


@pytest.mark.parametrize("rank_cap", [0, 96])
def test_bfloat16_storage(rank_cap):
    # bfloat16 in and out (the storage type of most LLaVA checkpoints): the Gram matrix comes from
    # the same tensor-core kernel with bfloat16 operands, the scores obey the same float32
    # tolerances (the inputs are taken as given), the merged rows are one bfloat16 rounding of the
    # float32 mean
    cfg = inputs.tiny_config(n_tokens=200, d_model=264, n_heads=3, head_dim=24, n_query=37, keep=61,
                             rank=40, dtype="bf16", batch=3, seed=37, noise=0.01, tau=2.0,
                             rank_tol=2e-3, dup_frac=0.05)
    check_config(cfg, range(3), rank_cap=rank_cap, max_flips=2)


def test_bfloat16_at_a_named_workload():
    cfg = inputs.CONFIGS["cfg2_llava7b_f16"].with_(batch=4, dtype="bf16")
    check_config(cfg, [1, 2], max_flips=2)
