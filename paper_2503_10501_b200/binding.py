"""ctypes binding of ``libtokencarve.so``: argument marshalling only.

Every function takes torch CUDA tensors (used purely as device memory) and enqueues the
library call of the same name on the current CUDA stream.  There is no fallback: if the
shared library cannot be built or loaded, importing the entry points raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Dict, Optional, Tuple

import torch

from . import build as _build

TC_OK = 0
TC_F16, TC_F32, TC_BF16 = 0, 1, 2
TC_FLAG_SIM_X, TC_FLAG_SIM_MEAN_K, TC_FLAG_WEIGHTED_MERGE = 1, 2, 16
TC_NORM_NONE, TC_NORM_SUM1 = 0, 1
STATUS_NAMES = {0: "TC_OK", 1: "TC_ERR_INVALID_ARG", 2: "TC_ERR_UNSUPPORTED", 3: "TC_ERR_WORKSPACE",
                4: "TC_ERR_NOT_CONVERGED", 5: "TC_ERR_CUDA", 6: "TC_ERR_RANK_CAP",
                7: "TC_ERR_BREAKDOWN", 8: "TC_ERR_SCRATCH_LIMIT"}

# every symbol include/tokencarve.h declares
EXPORTS = ("tc_counts", "tc_workspace_bytes", "tc_score", "tc_prune", "tc_merge", "tc_compact",
           "tc_carve", "tc_workspace_bytes_host", "tc_carve_host", "tc_gram", "tc_status_string",
           "tc_version", "tc_launch_count", "tc_profile_begin", "tc_profile_end",
           "tc_kernel_class_name", "tc_attn_score_noalloc", "tc_set_groups", "tc_test_fail_tensor_maps", "tc_rank",
           "tc_rank_workspace_bytes", "tc_reassemble", "tc_matmul_f32x3", "tc_stage_status", "tc_rope_tables",
           "tc_compact_weighted", "tc_probe", "tc_probe_workspace_bytes")


class TcParams(C.Structure):
    _fields_ = [("batch", C.c_int32), ("n_tokens", C.c_int32), ("d_model", C.c_int32),
                ("n_heads", C.c_int32), ("head_dim", C.c_int32), ("n_query", C.c_int32),
                ("keep", C.c_int32), ("n_merge", C.c_int32), ("rho", C.c_float),
                ("lambda_", C.c_float), ("rank_tol", C.c_float), ("dtype", C.c_int32),
                ("score_norm", C.c_int32), ("max_sweeps", C.c_int32), ("rank_cap", C.c_int32),
                ("flags", C.c_uint32)]


class TokenCarveError(RuntimeError):
    def __init__(self, fn: str, status: int):
        super().__init__(f"{fn} returned {STATUS_NAMES.get(status, status)}")
        self.status = status


_lib = None


def lib() -> C.CDLL:
    """Load (building first if needed) the shared library; raises if that is impossible."""
    global _lib
    if _lib is None:
        path = _build.LIB
        if not _build.up_to_date():
            try:
                path = _build.build()
            except Exception:
                if not os.path.exists(path):
                    raise
        L = C.CDLL(path)
        vp, sz = C.c_void_p, C.c_size_t
        pp = C.POINTER(TcParams)
        L.tc_counts.argtypes = [pp] + [C.POINTER(C.c_int32)] * 4
        L.tc_workspace_bytes.argtypes = [pp, C.POINTER(sz)]
        L.tc_workspace_bytes_host.argtypes = [pp, C.POINTER(sz)]
        L.tc_score.argtypes = [pp] + [vp] * 8 + [vp, sz, vp]
        L.tc_prune.argtypes = [pp, vp, vp, vp, vp, sz, vp]
        L.tc_merge.argtypes = [pp] + [vp] * 6 + [vp, sz, vp]
        L.tc_compact.argtypes = [pp] + [vp] * 9 + [vp, sz, vp]
        L.tc_compact_weighted.argtypes = [pp] + [vp] * 10 + [vp, sz, vp]
        L.tc_carve.argtypes = [pp] + [vp] * 10 + [vp, sz, vp]
        L.tc_carve_host.argtypes = [pp] + [vp] * 10 + [vp, sz, vp]
        L.tc_rank_workspace_bytes.argtypes = [pp, C.c_int32, C.POINTER(sz)]
        L.tc_rank.argtypes = [pp, vp, vp, C.c_int32, vp, vp, vp, vp, sz, vp]
        L.tc_reassemble.argtypes = [pp, C.c_int32, C.c_int32, vp, vp, vp, vp, vp, vp]
        L.tc_gram.argtypes = [pp, vp, vp, vp]
        L.tc_stage_status.argtypes = [pp, vp, sz, vp, vp]
        L.tc_rope_tables.argtypes = [vp, C.c_int64, C.c_int32, C.c_float, vp, vp, vp]
        L.tc_probe_workspace_bytes.argtypes = [pp, C.c_int32, C.c_int32, C.POINTER(sz)]
        L.tc_probe.argtypes = [pp, C.c_int32, C.c_int32, C.c_int32] + [vp] * 7 + [sz, vp]
        L.tc_matmul_f32x3.argtypes = [vp, vp, vp, vp] + [C.c_int32] * 4 + [vp, vp]
        L.tc_set_groups.argtypes = [C.c_int32]
        L.tc_test_fail_tensor_maps.argtypes = [C.c_int32]
        L.tc_attn_score_noalloc.argtypes = [pp, vp, vp, vp]
        L.tc_status_string.argtypes = [C.c_int32]
        L.tc_status_string.restype = C.c_char_p
        L.tc_kernel_class_name.argtypes = [C.c_int32]
        L.tc_kernel_class_name.restype = C.c_char_p
        L.tc_profile_end.argtypes = [C.POINTER(C.c_double), C.POINTER(C.c_int64), C.c_int32]
        for name in EXPORTS:
            if name not in ("tc_status_string", "tc_kernel_class_name", "tc_attn_score_noalloc", "tc_set_groups"):
                getattr(L, name).restype = C.c_int32
        L.tc_launch_count.restype = C.c_int64
        _lib = L
    return _lib


@dataclass
class Params:
    """Python mirror of ``tc_params`` (see include/tokencarve.h for the meaning of each field)."""
    batch: int
    n_tokens: int
    d_model: int
    n_heads: int
    head_dim: int
    n_query: int
    keep: int
    n_merge: int = -1
    rho: float = 0.5
    lam: float = 0.5
    rank_tol: float = 0.0
    dtype: str = "f16"
    score_norm: str = "none"
    max_sweeps: int = 30
    rank_cap: int = 0
    sim_source: str = "O"      # "O" (Eq. 3-10 as printed), "X", "meanK"
    weighted_merge: bool = False

    def c(self) -> TcParams:
        return TcParams(self.batch, self.n_tokens, self.d_model, self.n_heads, self.head_dim,
                        self.n_query, self.keep, self.n_merge, self.rho, self.lam, self.rank_tol,
                        {"f16": TC_F16, "f32": TC_F32, "bf16": TC_BF16}[self.dtype],
                        TC_NORM_SUM1 if self.score_norm == "sum1" else TC_NORM_NONE,
                        self.max_sweeps, self.rank_cap,
                        {"O": 0, "X": TC_FLAG_SIM_X, "meanK": TC_FLAG_SIM_MEAN_K}[self.sim_source]
                        | (TC_FLAG_WEIGHTED_MERGE if self.weighted_merge else 0))

    @property
    def torch_dtype(self):
        return {"f16": torch.float16, "bf16": torch.bfloat16, "f32": torch.float32}[self.dtype]


def _check(fn: str, status: int) -> None:
    if status != TC_OK:
        raise TokenCarveError(fn, status)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device, contiguous tensors only"
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def tc_counts(p: Params) -> Tuple[int, int, int, int]:
    v = [C.c_int32() for _ in range(4)]
    cp = p.c()
    _check("tc_counts", lib().tc_counts(C.byref(cp), *[C.byref(x) for x in v]))
    return tuple(x.value for x in v)


def tc_workspace_bytes(p: Params) -> int:
    n = C.c_size_t()
    cp = p.c()
    _check("tc_workspace_bytes", lib().tc_workspace_bytes(C.byref(cp), C.byref(n)))
    return n.value


def tc_workspace_bytes_host(p: Params) -> int:
    n = C.c_size_t()
    cp = p.c()
    _check("tc_workspace_bytes_host", lib().tc_workspace_bytes_host(C.byref(cp), C.byref(n)))
    return n.value


def workspace(p: Params, device="cuda", host: bool = False) -> torch.Tensor:
    n = tc_workspace_bytes_host(p) if host else tc_workspace_bytes(p)
    return torch.empty(n, dtype=torch.uint8, device=device)


def tc_gram(p: Params, O: torch.Tensor) -> torch.Tensor:
    G = torch.empty(p.batch, p.n_tokens, p.n_tokens, dtype=torch.float32, device=O.device)
    cp = p.c()
    _check("tc_gram", lib().tc_gram(C.byref(cp), _ptr(O), _ptr(G), _stream()))
    return G


def tc_probe(p: Params, n_sys: int, n_text: int, probe_start: int, Q, K, V, want_o=True, want_a=True,
             ws=None, out=None):
    """Layer-2 probe: returns (O [B, N, H*dh] or None, A [B, H, T, N] or None, img_status)."""
    dev = Q.device
    cp = p.c()
    if ws is None and want_o:
        n = C.c_size_t(0)
        _check("tc_probe_workspace_bytes",
               lib().tc_probe_workspace_bytes(C.byref(cp), n_sys, n_text, C.byref(n)))
        ws = torch.empty(max(int(n.value), 256), dtype=torch.uint8, device=dev)
    if out is None:
        O = torch.empty(p.batch, p.n_tokens, p.n_heads * p.head_dim, dtype=p.torch_dtype, device=dev) if want_o else None
        A = torch.empty(p.batch, p.n_heads, p.n_query, p.n_tokens, dtype=p.torch_dtype, device=dev) if want_a else None
        st = torch.empty(p.batch, dtype=torch.int32, device=dev)
    else:
        O, A, st = out
    _check("tc_probe", lib().tc_probe(C.byref(cp), n_sys, n_text, probe_start, _ptr(Q), _ptr(K), _ptr(V),
                                      _ptr(O), _ptr(A), _ptr(st), _ptr(ws), ws.numel() if ws is not None else 0,
                                      _stream()))
    return O, A, st


def tc_rope_tables(pos: torch.Tensor, head_dim: int, base: float = 10000.0):
    """cos / sin tables [..., head_dim / 2] (float32) for int32 position IDs of any shape."""
    assert pos.dtype == torch.int32
    shape = tuple(pos.shape) + (head_dim // 2,)
    cos = torch.empty(shape, dtype=torch.float32, device=pos.device)
    sin = torch.empty(shape, dtype=torch.float32, device=pos.device)
    _check("tc_rope_tables", lib().tc_rope_tables(_ptr(pos), pos.numel(), head_dim, base, _ptr(cos),
                                                  _ptr(sin), _stream()))
    return cos, sin


def tc_stage_status(p: Params, ws: torch.Tensor) -> torch.Tensor:
    """Per-image findings of the last tc_merge / tc_compact that used `ws`."""
    st = torch.empty(p.batch, dtype=torch.int32, device=ws.device)
    cp = p.c()
    _check("tc_stage_status", lib().tc_stage_status(C.byref(cp), _ptr(ws), ws.numel(), _ptr(st), _stream()))
    return st


def tc_matmul_f32x3(A: torch.Tensor, B: torch.Tensor, transposed: bool = False):
    """C = A B^T per image for float32 A [batch, M, K], B [batch, NN, K] through the three-product
    TF32 tensor-core kernel; returns (C, CT or None, img_status)."""
    assert A.dtype == torch.float32 and B.dtype == torch.float32 and A.is_contiguous() and B.is_contiguous()
    batch, M, K = A.shape
    NN = B.shape[1]
    assert B.shape[0] == batch and B.shape[2] == K
    L = lib()
    Cm = torch.empty(batch, M, NN, dtype=torch.float32, device=A.device)
    CT = torch.empty(batch, NN, M, dtype=torch.float32, device=A.device) if transposed else None
    st = torch.empty(batch, dtype=torch.int32, device=A.device)
    _check("tc_matmul_f32x3",
           L.tc_matmul_f32x3(_ptr(A), _ptr(B), _ptr(Cm), _ptr(CT) if CT is not None else None,
                             batch, M, NN, K, _ptr(st), _stream()))
    return Cm, CT, st


def tc_attn_score_noalloc(p: Params, A: torch.Tensor, S: torch.Tensor) -> torch.Tensor:
    """Eq. 3-7 into the caller's S [B, N] float32 tensor, using the library's built-in scratch
    array instead of a workspace: this call creates no tensor and allocates nothing."""
    assert S.dtype == torch.float32 and tuple(S.shape) == (p.batch, p.n_tokens)
    cp = p.c()
    _check("tc_attn_score_noalloc",
           lib().tc_attn_score_noalloc(C.byref(cp), _ptr(A), _ptr(S), _stream()))
    return S


def tc_score(p: Params, O, A, ws=None) -> Dict[str, torch.Tensor]:
    dev = O.device
    ws = ws if ws is not None else workspace(p, dev)
    B, N = p.batch, p.n_tokens
    q = min(N, p.d_model)
    out = {"E": torch.empty(B, N, dtype=torch.float32, device=dev),
           "C": torch.empty(B, N, dtype=torch.float32, device=dev),
           "S": torch.empty(B, N, dtype=torch.float32, device=dev),
           "sigma": torch.empty(B, q, dtype=torch.float32, device=dev),
           "rank": torch.empty(B, dtype=torch.int32, device=dev),
           "img_status": torch.empty(B, dtype=torch.int32, device=dev)}
    cp = p.c()
    _check("tc_score", lib().tc_score(C.byref(cp), _ptr(O), _ptr(A), _ptr(out["E"]), _ptr(out["C"]),
                                      _ptr(out["S"]), _ptr(out["sigma"]), _ptr(out["rank"]),
                                      _ptr(out["img_status"]), _ptr(ws), ws.numel(), _stream()))
    return out


def tc_rank_workspace_bytes(p: Params, n_sub: int) -> int:
    n = C.c_size_t()
    cp = p.c()
    _check("tc_rank_workspace_bytes", lib().tc_rank_workspace_bytes(C.byref(cp), n_sub, C.byref(n)))
    return n.value


def tc_rank(p: Params, O, idx=None, ws=None) -> Dict[str, torch.Tensor]:
    """sigma [B, min(n_sub, d)], rank [B], img_status [B] of the rows idx [B, n_sub] of O."""
    dev = O.device
    n_sub = p.n_tokens if idx is None else int(idx.shape[1])
    if ws is None:
        ws = torch.empty(tc_rank_workspace_bytes(p, n_sub), dtype=torch.uint8, device=dev)
    out = {"sigma": torch.empty(p.batch, min(n_sub, p.d_model), dtype=torch.float32, device=dev),
           "rank": torch.empty(p.batch, dtype=torch.int32, device=dev),
           "img_status": torch.empty(p.batch, dtype=torch.int32, device=dev)}
    cp = p.c()
    _check("tc_rank", lib().tc_rank(C.byref(cp), _ptr(O), _ptr(idx), n_sub, _ptr(out["sigma"]),
                                    _ptr(out["rank"]), _ptr(out["img_status"]), _ptr(ws), ws.numel(),
                                    _stream()))
    return out


def tc_reassemble(p: Params, n_sys: int, n_text: int, Hs, Xo, kept_idx):
    """(Ho [B, n_sys + keep + n_text, d], pos [B, n_sys + keep + n_text] int32)."""
    dev = Xo.device
    Lo = n_sys + p.keep + n_text
    Ho = torch.empty(p.batch, Lo, p.d_model, dtype=Xo.dtype, device=dev)
    pos = torch.empty(p.batch, Lo, dtype=torch.int32, device=dev)
    cp = p.c()
    _check("tc_reassemble", lib().tc_reassemble(C.byref(cp), n_sys, n_text, _ptr(Hs), _ptr(Xo),
                                                _ptr(kept_idx), _ptr(Ho), _ptr(pos), _stream()))
    return Ho, pos


def tc_prune(p: Params, E, ws=None) -> Tuple[torch.Tensor, torch.Tensor]:
    dev = E.device
    ws = ws if ws is not None else workspace(p, dev)
    M, P, nA, nB = tc_counts(p)
    setA = torch.empty(p.batch, nA, dtype=torch.int32, device=dev)
    setB = torch.empty(p.batch, nB, dtype=torch.int32, device=dev)
    cp = p.c()
    _check("tc_prune", lib().tc_prune(C.byref(cp), _ptr(E), _ptr(setA) if nA else None, _ptr(setB),
                                      _ptr(ws), ws.numel(), _stream()))
    return setA, setB


def tc_merge(p: Params, O, setA, setB, ws=None):
    dev = O.device
    ws = ws if ws is not None else workspace(p, dev)
    M, P, nA, nB = tc_counts(p)
    src = torch.empty(p.batch, M, dtype=torch.int32, device=dev)
    dst = torch.empty(p.batch, M, dtype=torch.int32, device=dev)
    kept = torch.empty(p.batch, p.keep, dtype=torch.int32, device=dev)
    cp = p.c()
    _check("tc_merge", lib().tc_merge(C.byref(cp), _ptr(O), _ptr(setA) if nA else None, _ptr(setB),
                                      _ptr(src) if M else None, _ptr(dst) if M else None,
                                      _ptr(kept), _ptr(ws), ws.numel(), _stream()))
    return src, dst, kept


def _outputs(p: Params, dev, with_kv: bool):
    dt = p.torch_dtype
    Xo = torch.empty(p.batch, p.keep, p.d_model, dtype=dt, device=dev)
    Ko = Vo = None
    if with_kv:
        Ko = torch.empty(p.batch, p.n_heads, p.keep, p.head_dim, dtype=dt, device=dev)
        Vo = torch.empty_like(Ko)
    return Xo, Ko, Vo


def tc_compact(p: Params, X, K, V, kept, src, dst, ws=None):
    dev = X.device
    ws = ws if ws is not None else workspace(p, dev)
    M = tc_counts(p)[0]
    Xo, Ko, Vo = _outputs(p, dev, K is not None)
    cp = p.c()
    _check("tc_compact", lib().tc_compact(C.byref(cp), _ptr(X), _ptr(K), _ptr(V), _ptr(kept),
                                          _ptr(src) if M else None, _ptr(dst) if M else None,
                                          _ptr(Xo), _ptr(Ko), _ptr(Vo), _ptr(ws), ws.numel(),
                                          _stream()))
    return Xo, Ko, Vo


def tc_compact_weighted(p: Params, X, K, V, kept, src, dst, E, ws=None):
    """tc_compact with the IPGS scores E [B, N] as merge weights."""
    dev = X.device
    ws = ws if ws is not None else workspace(p, dev)
    M = tc_counts(p)[0]
    Xo, Ko, Vo = _outputs(p, dev, K is not None)
    cp = p.c()
    _check("tc_compact_weighted",
           lib().tc_compact_weighted(C.byref(cp), _ptr(X), _ptr(K), _ptr(V), _ptr(kept),
                                     _ptr(src) if M else None, _ptr(dst) if M else None, _ptr(E),
                                     _ptr(Xo), _ptr(Ko), _ptr(Vo), _ptr(ws), ws.numel(), _stream()))
    return Xo, Ko, Vo


def tc_carve(p: Params, O, A, X, K=None, V=None, ws=None, out=None):
    """Returns (Xo, Ko, Vo, kept_idx, img_status); `out` may supply those five tensors."""
    dev = O.device
    ws = ws if ws is not None else workspace(p, dev)
    if out is None:
        Xo, Ko, Vo = _outputs(p, dev, K is not None)
        kept = torch.empty(p.batch, p.keep, dtype=torch.int32, device=dev)
        status = torch.empty(p.batch, dtype=torch.int32, device=dev)
    else:
        Xo, Ko, Vo, kept, status = out
    cp = p.c()
    _check("tc_carve", lib().tc_carve(C.byref(cp), _ptr(O), _ptr(A), _ptr(X), _ptr(K), _ptr(V),
                                      _ptr(Xo), _ptr(Ko), _ptr(Vo), _ptr(kept), _ptr(status),
                                      _ptr(ws), ws.numel(), _stream()))
    return Xo, Ko, Vo, kept, status


def tc_carve_host(p: Params, O, A, X, K, V, out, ws):
    """Host-memory variant: inputs and `out` = (Xo, Ko, Vo, kept_idx, img_status) are (pinned)
    CPU tensors, `ws` a device workspace of tc_workspace_bytes_host() bytes."""
    for t in (O, A, X, K, V) + tuple(out):
        assert t is None or (not t.is_cuda and t.is_contiguous())
    hp = lambda t: None if t is None else t.data_ptr()
    Xo, Ko, Vo, kept, status = out
    cp = p.c()
    _check("tc_carve_host", lib().tc_carve_host(C.byref(cp), hp(O), hp(A), hp(X), hp(K), hp(V),
                                                hp(Xo), hp(Ko), hp(Vo), hp(kept), hp(status),
                                                _ptr(ws), ws.numel(), _stream()))
    return out


def tc_status_string(status: int) -> str:
    return lib().tc_status_string(status).decode()


def tc_set_groups(groups: int) -> None:
    _check("tc_set_groups", lib().tc_set_groups(C.c_int32(groups)))


def tc_test_fail_tensor_maps(on: bool) -> None:
    """Test hook: refuse every tensor-map encode on the host while set."""
    _check("tc_test_fail_tensor_maps", lib().tc_test_fail_tensor_maps(C.c_int32(1 if on else 0)))


def tc_version() -> int:
    return lib().tc_version()


def tc_launch_count() -> int:
    return lib().tc_launch_count()


N_KERNEL_CLASSES = 15


def tc_profile_begin() -> None:
    _check("tc_profile_begin", lib().tc_profile_begin())


def tc_profile_end() -> Dict[str, Tuple[float, int]]:
    """{kernel class name: (device milliseconds, launches)} since tc_profile_begin()."""
    ms = (C.c_double * N_KERNEL_CLASSES)()
    n = (C.c_int64 * N_KERNEL_CLASSES)()
    _check("tc_profile_end", lib().tc_profile_end(ms, n, N_KERNEL_CLASSES))
    return {lib().tc_kernel_class_name(i).decode(): (ms[i], n[i]) for i in range(N_KERNEL_CLASSES)}
