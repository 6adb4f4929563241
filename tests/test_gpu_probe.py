"""The layer-2 probe (Sec. 3.1, Eq. 3-1 / 3-2; Sec. 3.2's visual slice) against the float64 oracle,
through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import ipgs_oracle as orc
from paper_2503_10501_b200 import binding as tcb
from paper_2503_10501_b200 import inputs

pytestmark = pytest.mark.gpu


def _qkv(B, H, L, dh, dtype, seed, hot=True):
    """Seeded queries, keys, values in the storage type (numpy float32 holding the rounded
    values for bfloat16); a few keys are made to stand out so that the softmax is peaked."""
    rng = np.random.default_rng(seed)
    Q = rng.standard_normal((B, H, L, dh)).astype(np.float32)
    K = rng.standard_normal((B, H, L, dh)).astype(np.float32)
    V = rng.standard_normal((B, H, L, dh)).astype(np.float32)
    if hot:
        for b in range(B):
            for h in range(H):
                j = int(rng.integers(0, L // 2))
                K[b, h, j] *= 3.0
    return tuple(inputs.to_storage(t, dtype) for t in (Q, K, V))


def _dev(a, dtype):
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    return t.to(torch.bfloat16) if dtype == "bf16" else t


def _host(t):
    return (t.float() if t.dtype == torch.bfloat16 else t).cpu().numpy().astype(np.float64)


def _check(B, H, n_sys, N, n_text, probe_start, T, dtype, seed):
    dh = 128
    L = n_sys + N + n_text
    Q, K, V = _qkv(B, H, L, dh, dtype, seed)
    p = tcb.Params(batch=B, n_tokens=N, d_model=H * dh, n_heads=H, head_dim=dh, n_query=T, keep=1,
                   dtype=dtype)
    O, A, st = tcb.tc_probe(p, n_sys, n_text, probe_start, _dev(Q, dtype), _dev(K, dtype), _dev(V, dtype))
    torch.cuda.synchronize()
    assert int(st.abs().sum()) == 0
    O, A = _host(O), _host(A)
    eps = 2.0 ** -11 if dtype == "f16" else 2.0 ** -8     # half an ulp of the storage type
    for b in range(B):
        Or, Ar = orc.layer2_probe_matrix(Q[b], K[b], V[b], n_sys, N, range(probe_start, probe_start + T))
        # Z: the probabilities are rounded to the storage type before they multiply V (a relative
        # error eps per term, random in sign), then the row is rounded once more
        tol = 4 * eps * np.abs(Or).max() + 1e-4
        assert np.max(np.abs(O[b] - Or)) <= tol, (b, np.max(np.abs(O[b] - Or)), tol)
        # probabilities: float32 arithmetic, one rounding to the storage type
        assert np.max(np.abs(A[b] - Ar) - 2 * eps * Ar) <= 2e-6, (b, np.max(np.abs(A[b] - Ar)))
        assert np.all(A[b][Ar == 0.0] == 0.0)
    return O, A


def test_probe_small_ragged_f16():
    # one ragged key block and a half: 5 system, 200 visual, 9 prompt tokens; the prompt rows probe
    _check(B=2, H=2, n_sys=5, N=200, n_text=9, probe_start=205, T=9, dtype="f16", seed=1)


def test_probe_llava_shaped_f16():
    # the LLaVA-1.5 layout: 35 system, 576 visual, 64 prompt tokens (six key blocks, the last
    # ragged), the 64 prompt rows probe
    _check(B=1, H=3, n_sys=35, N=576, n_text=64, probe_start=611, T=64, dtype="f16", seed=2)


def test_probe_bf16_and_more_probe_rows_than_a_tile():
    _check(B=1, H=2, n_sys=16, N=320, n_text=150, probe_start=336, T=150, dtype="bf16", seed=3)


def test_probe_rows_inside_the_visual_range_see_only_what_precedes_them():
    # probe rows in the middle of the image: the visual tokens after a row get probability zero
    O, A = _check(B=1, H=2, n_sys=3, N=260, n_text=4, probe_start=100, T=40, dtype="f16", seed=4)
    assert np.all(A[0][:, 0, 98:] == 0.0) and np.all(A[0][:, 0, :98] > 0.0)


def test_probe_feeds_the_score_stage():
    # O and A of the probe are what tc_score takes: the attention score of Eq. 3-7 from the
    # probe's A equals the oracle's on the oracle's A
    B, H, n_sys, N, n_text, dh = 1, 2, 8, 192, 32, 128
    L = n_sys + N + n_text
    Q, K, V = _qkv(B, H, L, dh, "f16", 5)
    p = tcb.Params(batch=B, n_tokens=N, d_model=H * dh, n_heads=H, head_dim=dh, n_query=n_text,
                   keep=48, dtype="f16", rank_tol=0.0)
    O, A, st = tcb.tc_probe(p, n_sys, n_text, n_sys + N, _dev(Q, "f16"), _dev(K, "f16"), _dev(V, "f16"))
    sc = tcb.tc_score(p, O, A)
    torch.cuda.synchronize()
    assert int(st.abs().sum()) == 0 and int(sc["img_status"].abs().sum()) == 0
    _, Ar = orc.layer2_probe_matrix(Q[0], K[0], V[0], n_sys, N, range(n_sys + N, L))
    S = orc.attention_score(Ar)
    np.testing.assert_allclose(sc["S"].cpu().numpy()[0], S, rtol=2e-3, atol=1e-7)


def test_probe_rejects_unsupported_shapes():
    p = tcb.Params(batch=1, n_tokens=64, d_model=128, n_heads=2, head_dim=64, n_query=4, keep=1)
    z = torch.zeros(1, 2, 80, 64, dtype=torch.float16, device="cuda")
    with pytest.raises(tcb.TokenCarveError) as e:
        tcb.tc_probe(p, 8, 8, 72, z, z, z)
    assert e.value.status == 2
