"""Seeded synthetic inputs for the LCA hot path.

This module only draws random tensors of the shapes and value distributions of the five
benchmark configurations and applies RoPE to the positional parts.  It holds none of the
method's arithmetic (no scores, pooling, anchors or attention) and is the one module that the
CUDA tests, the benchmark and the CPU oracle's tests all share: the oracle is always fed the
bit patterns produced here (copied back from the device when they were drawn there).

Recipe (all values bf16):
  * latents / keys / values / queries: i.i.d. N(0,1), drawn in fp32 in chunks of 4096 tokens
    from one torch.Generator(seed) per tensor, then rounded to bf16;
  * "needles": a few seeded token positions whose key-side rows (C^KV and K^R, or K and V)
    are multiplied by 4;
  * optional slowly varying mean: C^KV gets a per-segment, per-coordinate offset N(0, 0.3^2)
    (segment = 8192 tokens), which gives groups something poolable;
  * RoPE (half-split pairing (x_i, x_{i+d/2}), angle pos * theta^(-2i/d), positions 0..L-1)
    on q_rope and K^R (MLA) or on Q and K (GQA), computed in fp32 before the bf16 rounding.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Optional

import torch

CHUNK_TOKENS = 4096


@dataclass(frozen=True)
class LcaConfig:
    name: str
    variant: str            # "mla" or "gqa"
    batch: int
    seq_len: int
    n_q_heads: int
    n_kv_heads: int
    d_sem: int              # MLA: d_c = 512 ; GQA: head_dim
    d_pos: int              # MLA: d_R = 64  ; GQA: 0
    group_size: int
    window: int
    softmax_scale: float
    rope_theta: float
    needle_every: int = 0   # 0: `n_needles` seeded positions; >0: one per block of that many tokens
    n_needles: int = 8
    segment: int = 0        # >0: slowly varying mean on the pooled stream
    seed: int = 20260412


CONFIGS = {
    # cfg1: single MLA layer, L=1024, 4 heads
    "mla_1k": LcaConfig("mla_1k", "mla", 1, 1024, 4, 1, 512, 64, 64, 128, 1.0 / math.sqrt(192.0), 10000.0,
                        needle_every=0, n_needles=8, seed=20260412 + 1),
    # cfg2: DeepSeek-V2-Lite-shaped layer
    "mla_32k": LcaConfig("mla_32k", "mla", 1, 32768, 16, 1, 512, 64, 64, 2048, 1.0 / math.sqrt(192.0), 10000.0,
                         needle_every=4096, seed=20260412 + 2),
    # cfg3: DeepSeek-V3-shaped layer at 128K
    "mla_128k": LcaConfig("mla_128k", "mla", 1, 131072, 128, 1, 512, 64, 64, 4096, 1.0 / math.sqrt(192.0), 10000.0,
                          needle_every=0, n_needles=0, segment=8192, seed=20260412 + 3),
    # cfg4: decode against the condensed cache (per-sequence context 65536, batch 64)
    "mla_decode": LcaConfig("mla_decode", "mla", 64, 65536, 128, 1, 512, 64, 64, 4096, 1.0 / math.sqrt(192.0), 10000.0,
                            needle_every=0, n_needles=0, seed=20260412 + 4),
    # cfg5: Llama-3-8B-shaped GQA layer
    "gqa_64k": LcaConfig("gqa_64k", "gqa", 1, 65536, 32, 8, 128, 0, 64, 4096, 1.0 / math.sqrt(128.0), 500000.0,
                         needle_every=0, n_needles=0, seed=20260412 + 5),
}


def scaled(cfg: LcaConfig, **kw) -> LcaConfig:
    """A copy of a configuration with some fields replaced (used for scaled-down parity cases)."""
    d = dict(cfg.__dict__)
    d.update(kw)
    return LcaConfig(**d)


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _randn_chunks(shape, seed, device, post=None, dtype=torch.bfloat16):
    """N(0,1) tensor of `shape` = [L, ...] drawn chunk by chunk along dim 0 (fp32 -> post -> bf16)."""
    L = shape[0]
    out = torch.empty(shape, dtype=dtype, device=device)
    g = _gen(seed, device)
    for s in range(0, L, CHUNK_TOKENS):
        e = min(L, s + CHUNK_TOKENS)
        x = torch.randn((e - s,) + tuple(shape[1:]), generator=g, device=device, dtype=torch.float32)
        if post is not None:
            x = post(x, s, e)
        out[s:e] = x.to(dtype)
    return out


def rope_half_split(x: torch.Tensor, pos0: int, theta: float) -> torch.Tensor:
    """RoPE on the last dim of x [T, ..., d]; token t of the chunk has position pos0 + t."""
    d = x.shape[-1]
    half = d // 2
    T = x.shape[0]
    pos = torch.arange(pos0, pos0 + T, device=x.device, dtype=torch.float32)
    inv = theta ** (-torch.arange(0, half, device=x.device, dtype=torch.float32) * 2.0 / d)
    ang = pos[:, None] * inv[None, :]
    shape = [T] + [1] * (x.dim() - 2) + [half]
    cos = torch.cos(ang).reshape(shape)
    sin = torch.sin(ang).reshape(shape)
    x1, x2 = x[..., :half], x[..., half:]
    return torch.cat([x1 * cos - x2 * sin, x2 * cos + x1 * sin], dim=-1)


def needle_positions(cfg: LcaConfig, L: Optional[int] = None) -> torch.Tensor:
    L = cfg.seq_len if L is None else L
    g = _gen(cfg.seed + 7919, "cpu")
    if cfg.needle_every > 0:
        nblk = max(1, L // cfg.needle_every)
        off = int(torch.randint(0, min(cfg.needle_every, L), (1,), generator=g))
        return torch.tensor([min(L - 1, i * cfg.needle_every + off) for i in range(nblk)], dtype=torch.long)
    if cfg.n_needles > 0:
        return torch.randperm(L, generator=g)[: cfg.n_needles].sort().values
    return torch.zeros(0, dtype=torch.long)


def make_mla_inputs(cfg: LcaConfig, device="cpu", batch_index: int = 0, q_positions: Optional[slice] = None):
    """One sequence of an MLA configuration.

    Returns dict(q_sem [Lq,H,d_c], q_pos [Lq,H,d_R], ckv [L,d_c], kr [L,d_R]) in bf16 on `device`.
    `q_positions` (a slice of token positions) restricts the queries that are materialised
    (decode contexts only need the last `group_size` queries for the summary query).
    """
    assert cfg.variant == "mla"
    L, H = cfg.seq_len, cfg.n_q_heads
    seed = cfg.seed * 1000 + batch_index * 10

    seg_mu = None
    if cfg.segment > 0:
        nseg = (L + cfg.segment - 1) // cfg.segment
        seg_mu = (torch.randn((nseg, cfg.d_sem), generator=_gen(seed + 5, "cpu"), dtype=torch.float32) * 0.3).to(device)
    needles = needle_positions(cfg).to(device)

    def post_ckv(x, s, e):
        if seg_mu is not None:
            idx = torch.arange(s, e, device=x.device) // cfg.segment
            x = x + seg_mu[idx]
        return _scale_needles(x, s, e, needles)

    def post_kr(x, s, e):
        return _scale_needles(rope_half_split(x, s, cfg.rope_theta), s, e, needles)

    ckv = _randn_chunks((L, cfg.d_sem), seed + 1, device, post_ckv)
    kr = _randn_chunks((L, cfg.d_pos), seed + 2, device, post_kr)

    q0, q1 = 0, L
    if q_positions is not None:
        q0, q1, _ = q_positions.indices(L)
    Lq = q1 - q0
    q_sem = _randn_chunks((Lq, H, cfg.d_sem), seed + 3, device)
    q_pos = _randn_chunks((Lq, H, cfg.d_pos), seed + 4, device,
                          lambda x, s, e: rope_half_split(x, q0 + s, cfg.rope_theta))
    return dict(q_sem=q_sem, q_pos=q_pos, ckv=ckv, kr=kr)


def make_gqa_inputs(cfg: LcaConfig, device="cpu", batch_index: int = 0):
    """One sequence of a GQA configuration: dict(q [L,Hq,d], k [L,Hkv,d], v [L,Hkv,d]) in bf16."""
    assert cfg.variant == "gqa"
    L = cfg.seq_len
    seed = cfg.seed * 1000 + batch_index * 10
    needles = needle_positions(cfg).to(device)
    k = _randn_chunks((L, cfg.n_kv_heads, cfg.d_sem), seed + 1, device,
                      lambda x, s, e: _scale_needles(rope_half_split(x, s, cfg.rope_theta), s, e, needles))
    v = _randn_chunks((L, cfg.n_kv_heads, cfg.d_sem), seed + 2, device,
                      lambda x, s, e: _scale_needles(x, s, e, needles))
    q = _randn_chunks((L, cfg.n_q_heads, cfg.d_sem), seed + 3, device,
                      lambda x, s, e: rope_half_split(x, s, cfg.rope_theta))
    return dict(q=q, k=k, v=v)


def _scale_needles(x, s, e, needles):
    if needles.numel() == 0:
        return x
    sel = needles[(needles >= s) & (needles < e)] - s
    if sel.numel():
        x = x.clone()
        x[sel] = x[sel] * 4.0
    return x


# ------------------------------------------------------------------ parity-only stress inputs
def stress_peaky_queries(inp: dict, cfg: LcaConfig, strength: float = 3.0) -> dict:
    """Give the last `group_size` queries a common direction so that the group softmax is far
    from uniform (i.i.d. queries average out to a tiny summary query)."""
    out = dict(inp)
    g = _gen(cfg.seed + 31, "cpu")
    n = cfg.group_size
    if cfg.variant == "mla":
        for name, d in (("q_sem", cfg.d_sem), ("q_pos", cfg.d_pos)):
            direction = torch.randn((d,), generator=g, dtype=torch.float32).to(inp[name].device)
            t = inp[name].clone()
            t[-n:] = (t[-n:].float() * 0.2 + strength * direction).to(t.dtype)
            out[name] = t
    else:
        direction = torch.randn((cfg.d_sem,), generator=g, dtype=torch.float32).to(inp["q"].device)
        t = inp["q"].clone()
        t[-n:] = (t[-n:].float() * 0.2 + strength * direction).to(t.dtype)
        out["q"] = t
    return out


def stress_duplicate_tokens(inp: dict, cfg: LcaConfig, every: int = 3) -> dict:
    """Copy token 1 of every `every`-th group over token 5 of the same group: exact score ties."""
    out = dict(inp)
    g = cfg.group_size
    names = ("ckv", "kr") if cfg.variant == "mla" else ("k", "v")
    for name in names:
        t = inp[name].clone()
        L = t.shape[0]
        for j in range(0, L // g, every):
            if g > 5:
                t[j * g + 5] = t[j * g + 1]
        out[name] = t
    return out
