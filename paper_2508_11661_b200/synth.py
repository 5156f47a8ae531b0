"""Seeded synthetic workloads shaped like multi-document RAG KV caches.

This module only MAKES INPUTS (random tensors, rotary position encoding, planted
outlier channels / attention-sink keys, recompute-token lists).  It holds none of the
method's arithmetic and is used by the tests (for both the CPU oracle and the CUDA
library) and by the benchmark.  Tensors are torch tensors because torch owns the
device memory; generation on "cpu" is bit-reproducible everywhere, generation on
"cuda" is reproducible for a given seed on the same GPU model, and in both cases the
oracle and the CUDA path read the very same stored values.

Layouts (innermost dimension contiguous):
  K, V   [L, Bt, Hkv, L_tot, d]   per-document caches concatenated on the token axis
  Q      [L, Bt, T_q, Hq, d]      the user query's per-layer Q rows (scoring input)
  Qloc   [L, Bt, D, T_loc, Hq, d] each document's local-position Q cache
  Qa     [L, Bt, T_q, Hq, d]      fresh Q rows of the final re-prefill (attention input)
  Kq, Vq [L, Bt, T_q, Hkv, d]     the query chunk's own keys/values (appended, causal)
"""
from __future__ import annotations

import dataclasses
import math
from typing import Optional, Sequence

import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    n_layers: int
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    dtype: str                      # "bf16" | "f32"
    ctx_lens: tuple                 # tokens per context (shared across the batch)
    q_tokens: int                   # T_q
    budget_bp: int = 1500           # sequence budget in basis points (1500 = 15 %)
    block_size: int = 1             # selection unit B in tokens (1 = token mode; paper: 64)
    n_init: int = 16                # protected initial tokens per context
    n_local: int = 32               # protected local tokens per context
    t_loc: int = 1                  # rows of each document's local Q cache (1 = pre-pooled)
    rope_base: float = 500000.0
    outlier_channels: int = 0       # K channels per (layer, kv head) scaled x10
    sink_scale: float = 0.0         # >0: each context's token-0 key scaled by this factor
    recompute_share_bp: int = 0     # recomputed rows as a share of the kept tokens
    decode_steps: int = 0
    seed: int = 1000

    @property
    def n_ctx(self) -> int:
        return len(self.ctx_lens)

    @property
    def l_tot(self) -> int:
        return int(sum(self.ctx_lens))

    @property
    def ctx_offsets(self) -> list:
        off = [0]
        for n in self.ctx_lens:
            off.append(off[-1] + int(n))
        return off

    @property
    def torch_dtype(self):
        return {"bf16": torch.bfloat16, "f32": torch.float32}[self.dtype]

    @property
    def elem_bytes(self) -> int:
        return {"bf16": 2, "f32": 4}[self.dtype]

    def replace(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


# The five configurations the benchmark description names.
CONFIGS = {
    "cfg0": Workload("cfg0", 1, 1, 4, 2, 64, "f32", (256,) * 4, 16, n_init=4, n_local=8,
                     rope_base=10000.0, t_loc=8, seed=1000),
    "cfg1": Workload("cfg1", 1, 1, 32, 8, 128, "bf16", (1024,) * 10, 32, seed=1001),
    "cfg2": Workload("cfg2", 32, 4, 32, 8, 128, "bf16", (1536,) * 20, 64, outlier_channels=4,
                     sink_scale=8.0, recompute_share_bp=1500, seed=1002),
    "cfg3": Workload("cfg3", 1, 32, 32, 8, 128, "bf16", (2048,) * 10, 32, decode_steps=128, seed=1003),
    "cfg4": Workload("cfg4", 1, 1, 64, 8, 128, "bf16", (2048,) * 50, 128, seed=1004),
}


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _randn(shape, g, device) -> torch.Tensor:
    return torch.randn(shape, generator=g, device=device, dtype=torch.float32)


def rope_(x: torch.Tensor, positions: torch.Tensor, base: float) -> torch.Tensor:
    """Rotary position encoding, half-rotation pairing (i, i + d/2), applied in fp32.
    x: [..., T, d] with `positions` [T] indexing the second-to-last axis."""
    d = x.shape[-1]
    half = d // 2
    inv_freq = base ** (-torch.arange(0, half, device=x.device, dtype=torch.float32) / half)
    ang = positions.to(torch.float32)[:, None] * inv_freq[None, :]
    cos, sin = ang.cos(), ang.sin()
    x1, x2 = x[..., :half], x[..., half:]
    return torch.cat([x1 * cos - x2 * sin, x2 * cos + x1 * sin], dim=-1)


def context_positions(w: Workload, device) -> torch.Tensor:
    """Every context restarts at position 0: the caches were prefilled independently."""
    return torch.cat([torch.arange(n, device=device) for n in w.ctx_lens])


def make_kv_layer(w: Workload, layer: int, device) -> tuple:
    """K, V of one layer: [Bt, Hkv, L_tot, d] in the workload dtype."""
    g = _gen(device, w.seed * 1_000_003 + 17 * layer + 1)
    shape = (w.batch, w.n_kv_heads, w.l_tot, w.head_dim)
    K = rope_(_randn(shape, g, device), context_positions(w, device), w.rope_base)
    V = _randn(shape, g, device)
    if w.outlier_channels > 0:
        gc = _gen("cpu", w.seed * 7919 + layer)
        for h in range(w.n_kv_heads):
            ch = torch.randperm(w.head_dim, generator=gc)[: w.outlier_channels].to(device)
            K[:, h, :, ch] *= 10.0
    if w.sink_scale > 0:
        starts = torch.tensor(w.ctx_offsets[:-1], device=device)
        K[:, :, starts, :] *= w.sink_scale
    return K.to(w.torch_dtype), V.to(w.torch_dtype)


def make_query_layer(w: Workload, layer: int, device) -> dict:
    """Q (scoring), Qloc, Qa/Kq/Vq (attention chunk) of one layer."""
    g = _gen(device, w.seed * 1_000_003 + 17 * layer + 2)
    Bt, Tq, Hq, Hkv, d, D = w.batch, w.q_tokens, w.n_q_heads, w.n_kv_heads, w.head_dim, w.n_ctx
    qpos = torch.arange(w.l_tot, w.l_tot + Tq, device=device)

    def roped(shape_bhtd):
        x = rope_(_randn(shape_bhtd, g, device), qpos, w.rope_base)     # [Bt, H, T, d]
        return x.permute(0, 2, 1, 3).contiguous()                        # [Bt, T, H, d]

    Q = roped((Bt, Hq, Tq, d)).to(w.torch_dtype)
    Qa = roped((Bt, Hq, Tq, d)).to(w.torch_dtype)
    Kq = roped((Bt, Hkv, Tq, d)).to(w.torch_dtype)
    Vq = _randn((Bt, Tq, Hkv, d), g, device).to(w.torch_dtype)
    # local Q cache: noise plus a small component along the pooled query direction so that
    # the per-head cosine with the pooled query lands in about +-0.3 (the range the paper reports)
    qbar = Q.to(torch.float64).mean(dim=1)                               # [Bt, Hq, d]
    qbar = qbar / qbar.norm(dim=-1, keepdim=True).clamp_min(1e-30)
    beta = (torch.rand((Bt, D, 1, Hq, 1), generator=g, device=device) * 0.6 - 0.3)
    Qloc = _randn((Bt, D, w.t_loc, Hq, d), g, device)
    Qloc = Qloc + beta * math.sqrt(d / w.t_loc) * qbar[:, None, None, :, :].to(torch.float32)
    return dict(Q=Q, Qloc=Qloc.to(w.torch_dtype), Qa=Qa, Kq=Kq, Vq=Vq)


def make_inputs(w: Workload, device="cpu") -> dict:
    """All layers stacked.  K/V: [L, Bt, Hkv, L_tot, d] etc."""
    dev = torch.device(device)
    Ks, Vs, qs = [], [], []
    K = torch.empty((w.n_layers, w.batch, w.n_kv_heads, w.l_tot, w.head_dim), dtype=w.torch_dtype, device=dev)
    V = torch.empty_like(K)
    out = {}
    for l in range(w.n_layers):
        k, v = make_kv_layer(w, l, dev)
        K[l].copy_(k)
        V[l].copy_(v)
        del k, v
        qs.append(make_query_layer(w, l, dev))
    out["K"], out["V"] = K, V
    for name in ("Q", "Qloc", "Qa", "Kq", "Vq"):
        out[name] = torch.stack([q[name] for q in qs], dim=0).contiguous()
    return out


def make_recompute(w: Workload, K: torch.Tensor, V: torch.Tensor, sel_tokens_head0: torch.Tensor, n_rows: int):
    """Recomputed rows for the update step.

    sel_tokens_head0: [L, Bt, S] token ids kept by KV head 0 (batch element 0's list is used
    for every batch element: the token list is per layer).  Picks `n_rows` of those tokens at
    random per layer (seeded); other heads that did not keep a token skip it.  New rows are
    old + 0.484 * N(0,1), which puts cos(new, old) near 0.9 (the value the paper reports).
    Returns tok_ids int32 [L, R], Knew, Vnew [L, Bt, R, Hkv, d]."""
    L, Bt, Hkv, L_tot, d = K.shape
    dev = K.device
    g = _gen("cpu", w.seed * 104729 + 5)
    gd = _gen(dev, w.seed * 104729 + 6)
    tok_ids = torch.empty((L, n_rows), dtype=torch.int32)
    S = sel_tokens_head0.shape[-1]
    for l in range(L):
        perm = torch.randperm(S, generator=g)[:n_rows]
        tok_ids[l] = sel_tokens_head0[l, 0].cpu()[perm].to(torch.int32)
    tok_ids = tok_ids.to(dev)
    Knew = torch.empty((L, Bt, n_rows, Hkv, d), dtype=K.dtype, device=dev)
    Vnew = torch.empty_like(Knew)
    for l in range(L):
        idx = tok_ids[l].long()
        oldk = K[l][:, :, idx, :].permute(0, 2, 1, 3).float()            # [Bt, R, Hkv, d]
        oldv = V[l][:, :, idx, :].permute(0, 2, 1, 3).float()
        Knew[l] = (oldk + 0.484 * _randn(oldk.shape, gd, dev)).to(K.dtype)
        Vnew[l] = (oldv + 0.484 * _randn(oldv.shape, gd, dev)).to(K.dtype)
    return tok_ids, Knew, Vnew


def ragged_workload(name="ragged", ctx_lens=(100, 257, 64, 1000), dtype="f32", head_dim=64,
                    n_q_heads=4, n_kv_heads=2, q_tokens=5, block_size=1, n_init=4, n_local=8,
                    budget_bp=1500, seed=77, **kw) -> Workload:
    return Workload(name, 1, 1, n_q_heads, n_kv_heads, head_dim, dtype, tuple(ctx_lens), q_tokens,
                    budget_bp=budget_bp, block_size=block_size, n_init=n_init, n_local=n_local,
                    rope_base=10000.0, t_loc=3, seed=seed, **kw)
