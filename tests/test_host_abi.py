"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, derives the same counts as the oracle, and rejects bad arguments."""
import ctypes as C
import os
import re

import pytest

from oracle import ipgs_oracle as orc
from paper_2503_10501_b200 import binding as tcb

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _params(**kw):
    base = dict(batch=2, n_tokens=576, d_model=4096, n_heads=32, head_dim=128, n_query=64, keep=128)
    base.update(kw)
    return tcb.Params(**base)


def test_library_exports_every_declared_symbol():
    lib = tcb.lib()
    header = open(os.path.join(ROOT, "include", "tokencarve.h")).read()
    declared = set(re.findall(r"\b(tc_[a-z0-9_]+)\s*\(", header))
    assert declared == set(tcb.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None
    assert tcb.tc_version() >= 100
    assert tcb.tc_status_string(0) == "ok"
    assert "rank" in tcb.tc_status_string(6)


@pytest.mark.parametrize("N,keep,rho,n_merge", [
    (576, 128, 0.5, -1), (576, 192, 0.5, -1), (576, 64, 0.5, -1), (576, 333, 0.5, -1),
    (576, 576, 0.5, -1), (100, 90, 0.5, -1), (50, 10, 0.0, -1), (50, 10, 0.5, 3),
    (2880, 640, 0.5, -1), (576, 155, 0.3, -1), (576, 1, 1.0, -1), (576, 40, 0.7, -1)])
def test_counts_match_oracle(N, keep, rho, n_merge):
    got = tcb.tc_counts(_params(n_tokens=N, keep=keep, rho=rho, n_merge=n_merge,
                                 rank_cap=448 if N > 1024 else 0))
    assert got == orc.resolve_counts(N, keep, rho, n_merge)


def test_bad_arguments_are_rejected_on_the_host():
    for kw, code in [(dict(keep=0), 1), (dict(keep=577), 1), (dict(lam=1.5), 1), (dict(rho=-0.1), 1),
                     (dict(n_tokens=5000, keep=10), 2), (dict(d_model=4100, dtype="f16"), 2),
                     (dict(rank_cap=-1), 1), (dict(rank_cap=4), 1), (dict(n_tokens=2880, keep=640), 2),
                     (dict(batch=0), 1),
                     # one past the largest token count and the largest subspace
                     (dict(n_tokens=4097, keep=10, rank_cap=64), 2),
                     (dict(n_tokens=4096, keep=10, rank_cap=1025), 2)]:
        with pytest.raises(tcb.TokenCarveError) as e:
            tcb.tc_workspace_bytes(_params(**kw))
        assert e.value.status == code, kw


def test_largest_supported_shape_is_accepted():
    assert tcb.tc_workspace_bytes(_params(n_tokens=4096, keep=10, rank_cap=1024)) > 0


def test_workspace_grows_with_batch_and_host_variant_adds_staging():
    p1, p2 = _params(batch=1, rank_cap=160), _params(batch=4, rank_cap=160)
    w1, w2 = tcb.tc_workspace_bytes(p1), tcb.tc_workspace_bytes(p2)
    assert 0 < w1 < w2 <= 4 * w1 + 4096
    assert w1 >= 576 * 576 * 4
    staged = (2 * 576 * 4096 + 32 * 64 * 576 + 2 * 32 * 576 * 128) * 2
    assert tcb.tc_workspace_bytes_host(p1) >= w1 + staged
    # the full solve needs no subspace buffers but two N x N work matrices
    assert tcb.tc_workspace_bytes(_params(batch=1)) >= 3 * 576 * 576 * 4


def test_null_pointers_and_short_workspace_return_status_without_a_gpu():
    lib = tcb.lib()
    cp = _params(batch=1, rank_cap=160).c()
    dummy = C.c_void_p(256)          # never dereferenced: the checks below fail first
    assert lib.tc_carve(C.byref(cp), None, dummy, dummy, None, None, dummy, None, None, dummy,
                        dummy, dummy, 1 << 40, None) == 1
    assert lib.tc_carve(C.byref(cp), dummy, dummy, dummy, None, None, dummy, None, None, dummy,
                        dummy, dummy, 16, None) == 3
    assert lib.tc_prune(C.byref(cp), None, dummy, dummy, dummy, 1 << 40, None) == 1
    assert lib.tc_compact(C.byref(cp), dummy, dummy, None, dummy, dummy, dummy, dummy, None, None,
                          dummy, 1 << 40, None) == 1


def test_tc_rank_arguments_are_checked_on_the_host():
    lib = tcb.lib()
    p = _params(batch=2, rank_cap=160)
    full, half, few = (tcb.tc_rank_workspace_bytes(p, n) for n in (576, 288, 40))
    assert full > half > few > 0
    assert half >= 2 * 288 * 4096 * 2 + 2 * 288 * 288 * 4           # gathered rows + Gram
    assert few >= 2 * 40 * 4096 * 2 + 4 * 2 * 40 * 40 * 4            # ... + tridiagonal scratch
    for n_sub in (0, 577, -3):
        with pytest.raises(tcb.TokenCarveError) as e:
            tcb.tc_rank_workspace_bytes(p, n_sub)
        assert e.value.status == 1
    cp = p.c()
    dummy = C.c_void_p(256)          # never dereferenced: the checks below fail first
    # no token list means all rows
    assert lib.tc_rank(C.byref(cp), dummy, None, 288, dummy, dummy, dummy, dummy, 1 << 40, None) == 1
    # rank and status outputs are required, sigma is optional; a short workspace is refused
    assert lib.tc_rank(C.byref(cp), dummy, dummy, 288, dummy, None, dummy, dummy, 1 << 40, None) == 1
    assert lib.tc_rank(C.byref(cp), dummy, dummy, 288, None, dummy, dummy, dummy, 16, None) == 3


def test_tc_reassemble_arguments_are_checked_on_the_host():
    lib = tcb.lib()
    cp = _params(batch=2, rank_cap=160).c()
    dummy = C.c_void_p(256)          # never dereferenced: the checks below fail first
    assert lib.tc_reassemble(C.byref(cp), -1, 4, dummy, dummy, dummy, dummy, dummy, None) == 1
    assert lib.tc_reassemble(C.byref(cp), 3, 4, None, dummy, dummy, dummy, dummy, None) == 1
    assert lib.tc_reassemble(C.byref(cp), 3, 4, dummy, None, dummy, dummy, dummy, None) == 1
    assert lib.tc_reassemble(C.byref(cp), 0, 0, None, dummy, dummy, dummy, None, None) == 1
    assert lib.tc_reassemble(C.byref(cp), 3, 4, C.c_void_p(8), dummy, dummy, dummy, dummy, None) == 1
