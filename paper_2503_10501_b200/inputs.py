"""Seeded synthetic inputs for the IPGS carve path.

This module only *produces* inputs (random tensors with the shapes and value
structure of LLaVA-1.5 / AnyRes prefill at LLM layer 2).  It holds none of the
method's arithmetic: no scores, no selection, no similarity, no merging.  Both
the CUDA path and the float64 oracle are fed from here, so neither needs the
other to obtain test data.

Shapes follow the paper's set-up (Fig. 3-2: 576 visual tokens per image for
LLaVA-1.5; Sec. 4.2: 7B and 13B widths):

  O  [B, N, d]      visual rows of the layer-2 attention output  Z = A V   (Eq. 3-2)
  A  [B, H, T, N]   attention probabilities of T query rows over the N visual
                    tokens, per head (the slice Eq. 3-7 averages)
  X  [B, N, d]      hidden states entering layer 3 (what Stage II merges)
  K,V[B, H, N, dh]  per-head keys / values of the visual tokens

Recipe per image b (rng = numpy default_rng(seed + 1000*b)):
  O = Uf diag(s) Wf + sigma_n * N(0,1),  Uf[N,r], Wf[r,d] ~ N(0,1),
      s geometric from 1 down to 0.01                     (low rank + noise)
  A = softmax over N of  tau * N(0,1)  (+ hot_bias on `hot` random columns)
  X, K, V ~ N(0,1)
  dup_frac  of the tokens are overwritten by an exact copy (O, X, K, V rows) of a
            random other token;
  near_frac of the tokens are overwritten by a copy plus small noise, halved
            until the cosine between the O rows is >= near_cos.
Everything is generated in float64/float32, then rounded once to the storage
dtype of the configuration ("f16" or "f32"); both consumers see the rounded
values.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, Optional

import numpy as np


@dataclass(frozen=True)
class CarveConfig:
    """One workload: tensor shapes, generator knobs and the carve parameters."""
    name: str
    batch: int
    n_tokens: int          # N = L_v
    d_model: int           # d
    n_heads: int           # H
    head_dim: int          # dh
    n_query: int           # T
    dtype: str             # "f16" | "f32" | "bf16"
    rank: int              # r of the low-rank part of O
    noise: float           # sigma_n
    tau: float             # std of the attention logits
    keep: int              # L_vc
    rho: float = 0.5
    lam: float = 0.5
    rank_tol: float = 2e-3
    rank_cap: int = 0      # bound on the numerical rank handed to the solver (0 = full solve)
    dup_frac: float = 0.0
    near_frac: float = 0.0
    near_cos: float = 0.98
    hot: int = 0
    hot_bias: float = 0.0
    seed: int = 0

    def with_(self, **kw) -> "CarveConfig":
        return replace(self, **kw)


# The five workloads the benchmark description names (index 0 is the small one).
CONFIGS: Dict[str, CarveConfig] = {
    "cfg1_single_f32": CarveConfig("cfg1_single_f32", 1, 576, 4096, 32, 128, 32, "f32",
                                   rank=96, noise=0.01, tau=1.5, keep=192, rank_cap=128, seed=0),
    "cfg2_llava7b_f16": CarveConfig("cfg2_llava7b_f16", 16, 576, 4096, 32, 128, 64, "f16",
                                    rank=128, noise=0.01, tau=2.0, keep=128,
                                    rank_cap=160, dup_frac=0.05, seed=2),
    "cfg3_llava13b_f16": CarveConfig("cfg3_llava13b_f16", 16, 576, 5120, 40, 128, 64, "f16",
                                     rank=160, noise=0.02, tau=2.0, keep=64,
                                     rank_cap=192, hot=8, hot_bias=4.0, seed=3),
    "cfg4_anyres_f16": CarveConfig("cfg4_anyres_f16", 4, 2880, 4096, 32, 128, 128, "f16",
                                   rank=384, noise=0.01, tau=2.0, keep=640,
                                   rank_cap=736, near_frac=0.10, seed=4),
    "cfg5_sweep_f16": CarveConfig("cfg5_sweep_f16", 64, 576, 4096, 32, 128, 128, "f16",
                                  rank=128, noise=0.01, tau=2.0, keep=128, rank_cap=144,
                                  seed=5),
}


def np_dtype(dtype: str):
    if dtype == "f16":
        return np.float16
    if dtype in ("f32", "bf16"):
        return np.float32   # numpy has no bfloat16: its values are held in float32 (see to_storage)
    raise ValueError(f"unknown dtype {dtype!r}")


def to_storage(a: np.ndarray, dtype: str) -> np.ndarray:
    """One rounding (to nearest even) to the storage type.  "bf16" returns float32 values that
    are exactly representable in bfloat16 (the top 16 bits of a float32), so that a torch
    tensor made from them converts to torch.bfloat16 without a second rounding."""
    if dtype != "bf16":
        return a.astype(np_dtype(dtype))
    f = np.ascontiguousarray(a, dtype=np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    u = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16) << 16
    return u.astype(np.uint32).view(np.float32).reshape(f.shape)


def _softmax_last(z: np.ndarray) -> np.ndarray:
    z = z - z.max(axis=-1, keepdims=True)
    np.exp(z, out=z)
    z /= z.sum(axis=-1, keepdims=True)
    return z


def make_image(cfg: CarveConfig, b: int, want: str = "OAXKV") -> Dict[str, np.ndarray]:
    """Tensors of image `b` of the configuration, already rounded to cfg.dtype.

    `want` selects which of O, A, X, K, V to produce.  The random stream is
    consumed in a fixed order whatever `want` says, so a tensor's values do not
    depend on which others were requested.
    """
    N, d, H, dh, T, r = cfg.n_tokens, cfg.d_model, cfg.n_heads, cfg.head_dim, cfg.n_query, cfg.rank
    dt = cfg.dtype
    root = np.random.SeedSequence(cfg.seed + 1000 * b)
    s_o, s_a, s_x, s_k, s_v, s_d = [np.random.default_rng(s) for s in root.spawn(6)]
    out: Dict[str, np.ndarray] = {}

    # duplicate / near-duplicate plan (drawn first from its own stream)
    n_dup = int(round(cfg.dup_frac * N))
    n_near = int(round(cfg.near_frac * N))
    perm = s_d.permutation(N)
    dup_dst = perm[:n_dup]
    near_dst = perm[n_dup:n_dup + n_near]
    free = perm[n_dup + n_near:]            # tokens that stay original: copy sources
    dup_src = free[s_d.integers(0, len(free), size=n_dup)] if n_dup else np.zeros(0, np.int64)
    near_src = free[s_d.integers(0, len(free), size=n_near)] if n_near else np.zeros(0, np.int64)
    near_noise_seed = s_d.integers(0, 2**31 - 1)

    def apply_copies(M: np.ndarray, axis_tokens: int, scale: float) -> None:
        """Overwrite duplicate rows in place; M indexed [..., token, feature]."""
        if n_dup:
            if axis_tokens == 0:
                M[dup_dst] = M[dup_src]
            else:
                M[:, dup_dst] = M[:, dup_src]
        if n_near:
            g = np.random.default_rng(near_noise_seed + axis_tokens + int(scale * 7))
            for t, s in zip(near_dst, near_src):
                src = M[s] if axis_tokens == 0 else M[:, s]
                eps = scale
                while True:
                    cand = src + eps * g.standard_normal(src.shape)
                    a = src.reshape(-1).astype(np.float64)
                    c = cand.reshape(-1).astype(np.float64)
                    cosv = a @ c / max(np.sqrt((a @ a) * (c @ c)), 1e-300)
                    if cosv >= cfg.near_cos + 0.005:
                        break
                    eps *= 0.5
                if axis_tokens == 0:
                    M[t] = cand
                else:
                    M[:, t] = cand

    if "O" in want:
        Uf = s_o.standard_normal((N, r))
        Wf = s_o.standard_normal((r, d))
        s = np.geomspace(1.0, 0.01, r)
        Om = (Uf * s) @ Wf
        Om += cfg.noise * s_o.standard_normal((N, d))
        row_rms = float(np.sqrt(np.mean(Om * Om)))
        apply_copies(Om, 0, 0.1 * row_rms)
        out["O"] = to_storage(Om, dt)
    if "A" in want:
        z = s_a.standard_normal((H, T, N), dtype=np.float32)
        z *= np.float32(cfg.tau)
        if cfg.hot:
            hot_idx = s_a.choice(N, size=cfg.hot, replace=False)
            z[:, :, hot_idx] += np.float32(cfg.hot_bias)
        out["A"] = to_storage(_softmax_last(z), dt)
    if "X" in want:
        Xm = s_x.standard_normal((N, d), dtype=np.float32)
        apply_copies(Xm, 0, 0.1)
        out["X"] = to_storage(Xm, dt)
    if "K" in want:
        Km = s_k.standard_normal((H, N, dh), dtype=np.float32)
        apply_copies(Km, 1, 0.1)
        out["K"] = to_storage(Km, dt)
    if "V" in want:
        Vm = s_v.standard_normal((H, N, dh), dtype=np.float32)
        apply_copies(Vm, 1, 0.1)
        out["V"] = to_storage(Vm, dt)
    return out


def make_batch(cfg: CarveConfig, want: str = "OAXKV",
               images: Optional[range] = None) -> Dict[str, np.ndarray]:
    """Stack `make_image` over the batch (or over the given image numbers)."""
    ids = list(images) if images is not None else list(range(cfg.batch))
    per = [make_image(cfg, b, want) for b in ids]
    return {k: np.stack([p[k] for p in per], axis=0) for k in per[0]}


def tiny_config(n_tokens: int = 12, d_model: int = 16, n_heads: int = 2, head_dim: int = 8,
                n_query: int = 3, keep: int = 4, rank: int = 5, dtype: str = "f32",
                batch: int = 1, seed: int = 11, **kw) -> CarveConfig:
    """Small shapes for brute-force checks (d_model need not equal H*dh here)."""
    return CarveConfig("tiny", batch, n_tokens, d_model, n_heads, head_dim, n_query, dtype,
                       rank=rank, noise=kw.pop("noise", 0.05), tau=kw.pop("tau", 1.0),
                       keep=keep, seed=seed, **kw)
