"""tc_attn_score_noalloc against tc_score's S and against the oracle's Eq. 3-7.

The entry point exists for callers that cannot allocate device memory where they need the
attention scores (a plug-in inside someone else's forward pass, a latency-bound serving loop, a
process whose GPU memory is already owned by a pool).  It keeps its partial sums in an array
built into the library, shared by all calls, so the interesting cases are: a second call right
after a first one that used more of the array, and a request that does not fit.  This file is
named to be collected last.
"""
import numpy as np
import pytest
import torch

from oracle import ipgs_oracle as orc
from paper_2503_10501_b200 import binding as tcb
from paper_2503_10501_b200 import inputs

pytestmark = pytest.mark.gpu


def _params(cfg):
    return tcb.Params(batch=cfg.batch, n_tokens=cfg.n_tokens, d_model=cfg.d_model,
                      n_heads=cfg.n_heads, head_dim=cfg.head_dim, n_query=cfg.n_query,
                      keep=cfg.keep, rank_tol=cfg.rank_tol, dtype=cfg.dtype, rank_cap=cfg.rank_cap)


def _reference_S(p, batch):
    sc = tcb.tc_score(p, torch.from_numpy(batch["O"]).cuda(), torch.from_numpy(batch["A"]).cuda())
    torch.cuda.synchronize()
    assert int(sc["img_status"].abs().sum()) == 0
    return sc["S"].cpu().numpy()


def test_two_calls_in_a_row_match_the_workspace_entry_point():
    big = inputs.tiny_config(n_tokens=200, d_model=264, n_heads=3, head_dim=24, n_query=37, keep=61,
                             rank=40, dtype="f16", batch=5, seed=31, noise=0.01, tau=2.0,
                             rank_tol=2e-3, rank_cap=96)
    small = inputs.tiny_config(n_tokens=72, d_model=64, n_heads=2, head_dim=8, n_query=19, keep=20,
                               rank=16, dtype="f32", batch=2, seed=32, noise=0.05, tau=1.0,
                               rank_tol=0.0)
    runs = []
    for cfg in (big, small):                      # the second call uses less of the shared array
        p = _params(cfg)
        batch = inputs.make_batch(cfg, "OA")
        A = torch.from_numpy(batch["A"]).cuda()
        S = torch.full((cfg.batch, cfg.n_tokens), float("nan"), device="cuda")
        runs.append((p, batch, A, S))
    for p, batch, A, S in runs:                   # back to back on one stream, no sync between
        tcb.tc_attn_score_noalloc(p, A, S)
    torch.cuda.synchronize()
    for p, batch, A, S in runs:
        want = _reference_S(p, batch)
        got = S.cpu().numpy()
        assert np.all(np.isfinite(got))
        np.testing.assert_allclose(got, want, rtol=1e-3, atol=0)
        for b in range(p.batch):                  # and Eq. 3-7 itself, in float64
            ref = orc.attention_score(batch["A"][b].astype(np.float64))
            np.testing.assert_allclose(got[b], ref, rtol=1e-3, atol=0)
    # and once more for the first problem, after the array has held the second one's sums
    p, batch, A, S = runs[0]
    S.fill_(float("nan"))
    tcb.tc_attn_score_noalloc(p, A, S)
    torch.cuda.synchronize()
    np.testing.assert_allclose(S.cpu().numpy(), _reference_S(p, batch), rtol=1e-3, atol=0)


def test_request_beyond_the_built_in_scratch_is_refused():
    # B * chunks * N floats: 64 images x 10 chunks x 4096 tokens = 10.5 MB > 4 MiB
    p = tcb.Params(batch=64, n_tokens=4096, d_model=64, n_heads=32, head_dim=8, n_query=128,
                   keep=16, rank_cap=64)
    A = torch.zeros(16, dtype=torch.float16, device="cuda")      # never read: refused first
    S = torch.zeros(64, 4096, dtype=torch.float32, device="cuda")
    with pytest.raises(tcb.TokenCarveError) as e:
        tcb.tc_attn_score_noalloc(p, A, S)
    assert e.value.status == 8
    assert "scratch" in tcb.tc_status_string(8)
