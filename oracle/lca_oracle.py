"""ctypes front end of the fp64 CPU oracle (oracle/lca_oracle.cpp).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the benchmark's
cpu_baseline / reference leg.  Nothing here touches CUDA or the CUDA package.

The functions keep the paper's notation: L tokens, window w, group size g, m groups,
k local tokens, q_bar, s_i, alpha_i, c_rep_j, anchor I_j (Alg. 1, Eq. 6-10).
Arrays are numpy float64 unless a name ends in ``_bits`` (uint16 bfloat16 bit patterns).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lca_oracle.cpp")
_SO = os.path.join(_HERE, "_lca_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (OpenMP).  Returns the path of the shared object."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        cmd = ["g++", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c++17",
               "-ffp-contract=off", "-o", _SO, _SRC]
        subprocess.check_call(cmd)
    return _SO


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = C.CDLL(_SO)
        _lib.lca_oracle_num_threads.restype = C.c_int
        _lib.lca_oracle_round_bf16_scalar.restype = C.c_uint16
        _lib.lca_oracle_round_bf16_scalar.argtypes = [C.c_double]
    return _lib


def _dp(a):
    return a.ctypes.data_as(C.POINTER(C.c_double))


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float64)


def num_threads() -> int:
    return int(_load().lca_oracle_num_threads())


# ----------------------------------------------------------------------------- bf16 helpers
def bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Widen bfloat16 bit patterns (uint16) to float64, exactly."""
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def round_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float64 -> nearest bfloat16 (ties to even), returned as uint16 bit patterns."""
    x = _f64(x)
    out = np.empty(x.shape, dtype=np.uint16)
    _load().lca_oracle_round_bf16(_dp(x), C.c_int64(x.size),
                                  out.ctypes.data_as(C.POINTER(C.c_uint16)))
    return out


def torch_bf16_to_bits(t) -> np.ndarray:
    """A (CPU) torch.bfloat16 tensor -> uint16 bit patterns."""
    import torch
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def torch_bf16_to_f64(t) -> np.ndarray:
    return bits_to_f64(torch_bf16_to_bits(t))


# ------------------------------------------------------------------------------- partition
def partition(L: int, w: int, g: int):
    """(m, k) of Sec. 4.2: m = floor((L-w)/g) groups, k = w + (L-w) mod g local tokens;
    m = 0, k = L when L < w + g (fallback to plain attention)."""
    m = C.c_int64()
    k = C.c_int64()
    _load().lca_oracle_partition(C.c_int64(L), C.c_int64(w), C.c_int64(g), C.byref(m), C.byref(k))
    return int(m.value), int(k.value)


# ------------------------------------------------------------------------- generic streams
def summary_query(q_tail: np.ndarray) -> np.ndarray:
    """Summary query of Alg. 1 (Sec. 4.2).  q_tail [n, heads, d] (the last n query positions) -> q_bar [d]."""
    q = _f64(q_tail)
    n, heads, d = q.shape
    out = np.empty(d, dtype=np.float64)
    _load().lca_oracle_summary_query(_dp(q), C.c_int64(n), C.c_int64(heads), C.c_int64(d), _dp(out))
    return out


def condense_stream(key: np.ndarray, pool: np.ndarray, qbar: np.ndarray, g: int, w: int,
                    scale: float):
    """The condensation steps of Alg. 1 (scores, Eq. 6, Eq. 7, Eq. 8) on one key/value stream.  Returns dict(scores, alpha, pooled, anchor, m, k)."""
    key = _f64(key)
    pool = _f64(pool)
    qbar = _f64(qbar)
    L, dk = key.shape
    dp_ = pool.shape[1]
    m, k = partition(L, w, g)
    scores = np.zeros(max(m * g, 1), dtype=np.float64)
    alpha = np.zeros(max(m * g, 1), dtype=np.float64)
    pooled = np.zeros((max(m, 1), dp_), dtype=np.float64)
    anchor = np.zeros(max(m, 1), dtype=np.int32)
    _load().lca_oracle_condense_stream(
        _dp(key), C.c_int64(dk), _dp(pool), C.c_int64(dp_), _dp(qbar), C.c_int64(L),
        C.c_int64(g), C.c_int64(w), C.c_double(scale), _dp(scores), _dp(alpha), _dp(pooled),
        anchor.ctypes.data_as(C.POINTER(C.c_int32)))
    return dict(scores=scores[:m * g], alpha=alpha[:m * g], pooled=pooled[:m], anchor=anchor[:m],
                m=m, k=k)


def attend_rows(q_rows: np.ndarray, pos: np.ndarray, key: np.ndarray, val: np.ndarray,
                rkey: np.ndarray, rval: np.ndarray, g: int, w: int, scale: float,
                rep_logit_bias: float = 0.0):
    """Eq. 10 at prefix length pos+1 for each listed query position.
    q_rows [n, heads, dk]; returns (out [n, heads, dv], lse [n, heads])."""
    q = _f64(q_rows)
    pos = np.ascontiguousarray(pos, dtype=np.int64)
    key = _f64(key)
    val = _f64(val)
    n, heads, dk = q.shape
    L = key.shape[0]
    dv = val.shape[1]
    m = int(rkey.shape[0]) if rkey is not None else 0
    rkey = _f64(rkey) if m else np.zeros((1, dk))
    rval = _f64(rval) if m else np.zeros((1, dv))
    out = np.empty((n, heads, dv), dtype=np.float64)
    lse = np.empty((n, heads), dtype=np.float64)
    _load().lca_oracle_attend_rows(
        _dp(q), pos.ctypes.data_as(C.POINTER(C.c_int64)), C.c_int64(n), C.c_int64(heads),
        _dp(key), _dp(val), C.c_int64(L), _dp(rkey), _dp(rval), C.c_int64(m), C.c_int64(dk),
        C.c_int64(dv), C.c_int64(g), C.c_int64(w), C.c_double(scale), C.c_double(rep_logit_bias),
        _dp(out), _dp(lse))
    return out, lse


def decode_rows(q: np.ndarray, ckey: np.ndarray, cval: np.ndarray, n_rep: int, scale: float,
                rep_logit_bias: float = 0.0):
    """Sec. 4.3 decode: q [heads, dk] over every cache row.  Returns (out [heads, dv], lse)."""
    q = _f64(q)
    ckey = _f64(ckey)
    cval = _f64(cval)
    heads, dk = q.shape
    rows, dv = cval.shape
    out = np.empty((heads, dv), dtype=np.float64)
    lse = np.empty(heads, dtype=np.float64)
    _load().lca_oracle_decode(_dp(q), C.c_int64(heads), _dp(ckey), _dp(cval), C.c_int64(rows),
                              C.c_int64(n_rep), C.c_int64(dk), C.c_int64(dv), C.c_double(scale),
                              C.c_double(rep_logit_bias), _dp(out), _dp(lse))
    return out, lse


# --------------------------------------------------------------------- ablation reducers
def reduce_groups(x: np.ndarray, alpha: np.ndarray, anchor: np.ndarray, g: int, m: int, mode: str) -> np.ndarray:
    """One vector per group from the g vectors x[j*g:(j+1)*g] (Table 5 operators):
    "weighted" = sum_i alpha_i x_i (Eq. 7), "maxsel" = x of the arg-max token (Eq. 8),
    "meanpool" = plain mean, "maxpool" = element-wise maximum."""
    x = _f64(x)
    out = np.zeros((m, x.shape[1]))
    for j in range(m):
        grp = x[j * g:(j + 1) * g]
        if mode == "weighted":
            out[j] = (alpha[j * g:(j + 1) * g, None] * grp).sum(axis=0)
        elif mode == "maxsel":
            out[j] = x[anchor[j]]
        elif mode == "meanpool":
            out[j] = grp.sum(axis=0) / g
        elif mode == "maxpool":
            out[j] = grp.max(axis=0)
        else:
            raise ValueError(mode)
    return out


# ------------------------------------------------------------------------------ MLA flavour
def mla_summary_query(q_sem_tail: np.ndarray, q_pos_tail: np.ndarray) -> np.ndarray:
    """q_bar over [q_latent | q_rope] of the last n positions and all heads -> [d_c + d_R]."""
    return summary_query(np.concatenate([_f64(q_sem_tail), _f64(q_pos_tail)], axis=-1))


def mla_condense(qbar: np.ndarray, ckv: np.ndarray, kr: np.ndarray, g: int, w: int, scale: float,
                 sem_reducer: str = "weighted", pos_reducer: str = "maxsel"):
    """Condensed MLA cache of one sequence (the condensation and local-window steps of Alg. 1).

    Returns dict with
      scores, alpha [m*g]; c_rep [m, d_c] (unrounded); anchor [m] int32 (absolute 0-based);
      cache_sem_bits [m+k, d_c], cache_pos_bits [m+k, d_R] (uint16 bf16: rows 0..m-1 = the
      representatives, c_rep rounded to nearest-even bf16 and k^R of the anchor copied; rows
      m.. = the last k tokens copied), m, k.
    ckv / kr must hold bf16-representable values (they are copied into the cache bit-exactly).
    """
    ckv = _f64(ckv)
    kr = _f64(kr)
    key = np.concatenate([ckv, kr], axis=1)
    r = condense_stream(key, ckv, qbar, g, w, scale)
    m, k = r["m"], r["k"]
    L = ckv.shape[0]
    c_rep = r["pooled"] if sem_reducer == "weighted" else reduce_groups(ckv, r["alpha"], r["anchor"], g, m, sem_reducer)
    k_rep = reduce_groups(kr, r["alpha"], r["anchor"], g, m, pos_reducer)
    cache_sem = np.concatenate([c_rep, ckv[L - k:]], axis=0)
    cache_pos = np.concatenate([k_rep, kr[L - k:]], axis=0)
    return dict(scores=r["scores"], alpha=r["alpha"], c_rep=c_rep, anchor=r["anchor"],
                cache_sem_bits=round_bf16_bits(cache_sem), cache_pos_bits=round_bf16_bits(cache_pos),
                m=m, k=k)


def mla_prefill_rows(q_sem_rows, q_pos_rows, pos, ckv, kr, rep_sem, rep_pos, g, w, scale,
                     rep_logit_bias=0.0):
    """Absorbed-form LCA prefill rows: logits q.[c|k^R], values c (latent space)."""
    q = np.concatenate([_f64(q_sem_rows), _f64(q_pos_rows)], axis=-1)
    ckv = _f64(ckv)
    key = np.concatenate([ckv, _f64(kr)], axis=1)
    m = 0 if rep_sem is None else rep_sem.shape[0]
    rkey = np.concatenate([_f64(rep_sem), _f64(rep_pos)], axis=1) if m else None
    rval = _f64(rep_sem) if m else None
    return attend_rows(q, pos, key, ckv, rkey, rval, g, w, scale, rep_logit_bias)


def mla_decode(q_sem, q_pos, cache_sem, cache_pos, n_rep, scale, rep_logit_bias=0.0):
    q = np.concatenate([_f64(q_sem), _f64(q_pos)], axis=-1)
    cs = _f64(cache_sem)
    ckey = np.concatenate([cs, _f64(cache_pos)], axis=1)
    return decode_rows(q, ckey, cs, n_rep, scale, rep_logit_bias)


def latent_to_value(attn_latent: np.ndarray, w_uv: np.ndarray) -> np.ndarray:
    """Value up-projection of the latent attention output (Alg. 1: v = c W^UV, applied after the
    attention in the absorbed form of Sec. 4.3): attn_latent [..., H, d_c], w_uv [H, d_c, d_v] ->
    [..., H, d_v], one matrix product per head."""
    return np.einsum("...hc,hcv->...hv", _f64(attn_latent), _f64(w_uv))


# ------------------------------------------------------------------------------ GQA flavour
def gqa_summary_query(q_tail: np.ndarray, n_kv_heads: int) -> np.ndarray:
    """q_tail [n, Hq, d] -> q_bar [Hkv, d]: mean over positions and the Hq/Hkv heads of each KV head."""
    q = _f64(q_tail)
    n, hq, d = q.shape
    rep = hq // n_kv_heads
    return np.stack([summary_query(q[:, h * rep:(h + 1) * rep, :]) for h in range(n_kv_heads)])


def gqa_condense(qbar: np.ndarray, k: np.ndarray, v: np.ndarray, g: int, w: int, scale: float):
    """Per KV head: anchor selection on keys, weighted pooling on values (Sec. 5.4).
    k, v [L, Hkv, d].  Returns dict(anchor [m, Hkv], v_rep [m, Hkv, d], scores [m*g, Hkv],
    cache_k_bits / cache_v_bits [m+k, Hkv, d], m, k)."""
    k = _f64(k)
    v = _f64(v)
    L, hkv, d = k.shape
    outs = [condense_stream(k[:, h, :], v[:, h, :], qbar[h], g, w, scale) for h in range(hkv)]
    m, kk = outs[0]["m"], outs[0]["k"]
    anchor = np.stack([o["anchor"] for o in outs], axis=1) if m else np.zeros((0, hkv), np.int32)
    v_rep = np.stack([o["pooled"] for o in outs], axis=1) if m else np.zeros((0, hkv, d))
    scores = np.stack([o["scores"] for o in outs], axis=1) if m else np.zeros((0, hkv))
    k_rep = np.stack([k[outs[h]["anchor"], h, :] for h in range(hkv)], axis=1) if m else np.zeros((0, hkv, d))
    cache_k = np.concatenate([k_rep, k[L - kk:]], axis=0)
    cache_v = np.concatenate([v_rep, v[L - kk:]], axis=0)
    return dict(anchor=anchor.astype(np.int32), v_rep=v_rep, scores=scores,
                cache_k_bits=round_bf16_bits(cache_k), cache_v_bits=round_bf16_bits(cache_v),
                m=m, k=kk)


def gqa_prefill_rows(q_rows, pos, k, v, k_rep, v_rep, g, w, scale, rep_logit_bias=0.0):
    """q_rows [n, Hq, d]; k, v [L, Hkv, d]; k_rep, v_rep [m, Hkv, d] -> out [n, Hq, d], lse [n, Hq]."""
    q = _f64(q_rows)
    k = _f64(k)
    v = _f64(v)
    n, hq, d = q.shape
    hkv = k.shape[1]
    rep = hq // hkv
    out = np.empty((n, hq, d))
    lse = np.empty((n, hq))
    for h in range(hkv):
        rk = None if k_rep is None or k_rep.shape[0] == 0 else _f64(k_rep)[:, h, :]
        rv = None if rk is None else _f64(v_rep)[:, h, :]
        o, l = attend_rows(q[:, h * rep:(h + 1) * rep, :], pos, k[:, h, :], v[:, h, :], rk, rv,
                           g, w, scale, rep_logit_bias)
        out[:, h * rep:(h + 1) * rep, :] = o
        lse[:, h * rep:(h + 1) * rep] = l
    return out, lse


def gqa_decode(q, cache_k, cache_v, n_rep, scale, rep_logit_bias=0.0):
    """q [Hq, d]; cache_k, cache_v [rows, Hkv, d] -> out [Hq, d], lse [Hq]."""
    q = _f64(q)
    ck = _f64(cache_k)
    cv = _f64(cache_v)
    hq, d = q.shape
    hkv = ck.shape[1]
    rep = hq // hkv
    out = np.empty((hq, d))
    lse = np.empty(hq)
    for h in range(hkv):
        o, l = decode_rows(q[h * rep:(h + 1) * rep], ck[:, h, :], cv[:, h, :], n_rep, scale,
                           rep_logit_bias)
        out[h * rep:(h + 1) * rep] = o
        lse[h * rep:(h + 1) * rep] = l
    return out, lse


# ------------------------------------------------------------------- online cache update
def mla_decode_update(cache_sem_bits: np.ndarray, cache_pos_bits: np.ndarray, n_rep: int, n_rows: int,
                      qbar: np.ndarray, g: int, w: int, scale: float):
    """Sec. 4.3 "Decoding and Online Cache Update" for one sequence.

    cache_*_bits [rows, d] are bf16 bit patterns: rows 0..n_rep-1 the representatives, rows
    n_rep..n_rows-1 the buffered tokens in order.  When the buffer holds w + g tokens, its earliest g
    tokens are condensed with the summary query q_bar (scores of Sec. 4.2, Eq. 6 softmax, Eq. 7
    pooling, Eq. 8 anchor) into one representative that is appended to the representatives; the
    other tokens keep their order.  Returns (cache_sem_bits, cache_pos_bits, n_rep, n_rows, anchor)
    with anchor = offset of the anchor token in the condensed group, or -1 when nothing happened.
    """
    if n_rows - n_rep < w + g:
        return cache_sem_bits, cache_pos_bits, n_rep, n_rows, -1
    grp_sem = bits_to_f64(cache_sem_bits[n_rep:n_rep + g])
    grp_pos = bits_to_f64(cache_pos_bits[n_rep:n_rep + g])
    r = condense_stream(np.concatenate([grp_sem, grp_pos], axis=1), grp_sem, qbar, g, 0, scale)   # one group
    assert r["m"] == 1
    ia = int(r["anchor"][0])
    new_sem = np.concatenate([cache_sem_bits[:n_rep], round_bf16_bits(r["pooled"]), cache_sem_bits[n_rep + g:n_rows]], axis=0)
    new_pos = np.concatenate([cache_pos_bits[:n_rep], cache_pos_bits[n_rep + ia:n_rep + ia + 1],
                              cache_pos_bits[n_rep + g:n_rows]], axis=0)
    return new_sem, new_pos, n_rep + 1, n_rows - (g - 1), ia


# ------------------------------------------------------- ring layout of the decode cache
# Sec. 4.3 states what the cache holds while decoding (the m representatives and the most recent tokens) and says
# nothing about where they live.  The packed layout above moves every buffered token when a group is
# condensed; the ring layout moves none:
#   rows [0, R), R = w + g : token number n of the sequence (0-based from its start) at row n % R;
#   rows [R, R + n_rep)    : the representatives in group order.
# With n_rep representatives and n_tok tokens so far, the uncondensed tokens are n_rep*g .. n_tok-1.
def ring_from_packed(cache_sem_bits: np.ndarray, cache_pos_bits: np.ndarray, n_rep: int, n_rows: int,
                     g: int, w: int, capacity: int):
    """Packed [representatives ; tokens in order] -> ring layout.  Returns (ring_sem_bits
    [capacity, d], ring_pos_bits, n_tok); rows that hold nothing are zero."""
    R = w + g
    assert w % g == 0 and n_rows - n_rep <= R and R + n_rep <= capacity
    ring_sem = np.zeros((capacity,) + cache_sem_bits.shape[1:], dtype=cache_sem_bits.dtype)
    ring_pos = np.zeros((capacity,) + cache_pos_bits.shape[1:], dtype=cache_pos_bits.dtype)
    first = n_rep * g
    for i in range(n_rows - n_rep):
        ring_sem[(first + i) % R] = cache_sem_bits[n_rep + i]
        ring_pos[(first + i) % R] = cache_pos_bits[n_rep + i]
    ring_sem[R:R + n_rep] = cache_sem_bits[:n_rep]
    ring_pos[R:R + n_rep] = cache_pos_bits[:n_rep]
    return ring_sem, ring_pos, first + (n_rows - n_rep)


def ring_to_packed(ring_sem_bits: np.ndarray, ring_pos_bits: np.ndarray, n_rep: int, n_tok: int, g: int, w: int):
    """The rows of a ring cache that take part, in the order [representatives ; tokens in order]
    (what decode attends to).  Returns (cache_sem_bits, cache_pos_bits, n_rows)."""
    R = w + g
    first = n_rep * g
    assert 0 <= n_tok - first <= R
    rows = [R + j for j in range(n_rep)] + [n % R for n in range(first, n_tok)]
    return ring_sem_bits[rows], ring_pos_bits[rows], len(rows)


def mla_decode_update_ring(ring_sem_bits: np.ndarray, ring_pos_bits: np.ndarray, n_rep: int, n_tok: int,
                           qbar: np.ndarray, g: int, w: int, scale: float):
    """Sec. 4.3 online update on the ring layout, one sequence: when w + g tokens are uncondensed,
    the earliest g of them (tokens n_rep*g .. n_rep*g + g - 1) become representative number n_rep
    (scores of Sec. 4.2 with q_bar, Eq. 6, Eq. 7, Eq. 8), written to row R + n_rep; no other row
    changes.  Returns (ring_sem_bits, ring_pos_bits, n_rep, anchor offset or -1)."""
    R = w + g
    first = n_rep * g
    if n_tok - first < R or R + n_rep >= ring_sem_bits.shape[0]:
        return ring_sem_bits, ring_pos_bits, n_rep, -1
    rows = [(first + i) % R for i in range(g)]
    grp_sem = bits_to_f64(ring_sem_bits[rows])
    grp_pos = bits_to_f64(ring_pos_bits[rows])
    r = condense_stream(np.concatenate([grp_sem, grp_pos], axis=1), grp_sem, qbar, g, 0, scale)   # one group
    ia = int(r["anchor"][0])
    ring_sem = ring_sem_bits.copy()
    ring_pos = ring_pos_bits.copy()
    ring_sem[R + n_rep] = round_bf16_bits(r["pooled"])[0]
    ring_pos[R + n_rep] = ring_pos_bits[rows[ia]]
    return ring_sem, ring_pos, n_rep + 1, ia


def gqa_decode_update_ring(ring_k_bits: np.ndarray, ring_v_bits: np.ndarray, n_rep: int, n_tok: int,
                           qbar: np.ndarray, g: int, w: int, scale: float):
    """The online update of Sec. 4.3 for the GQA variant (Sec. 5.4: select K, pool V, per KV head) on the
    ring layout.  ring_*_bits [capacity, Hkv, d] bf16 bit patterns, qbar [Hkv, d].  Returns
    (ring_k_bits, ring_v_bits, n_rep, anchors [Hkv] or None when nothing was condensed)."""
    R = w + g
    first = n_rep * g
    if n_tok - first < R or R + n_rep >= ring_k_bits.shape[0]:
        return ring_k_bits, ring_v_bits, n_rep, None
    rows = [(first + i) % R for i in range(g)]
    ring_k = ring_k_bits.copy()
    ring_v = ring_v_bits.copy()
    anchors = []
    for h in range(ring_k_bits.shape[1]):
        grp_k = bits_to_f64(ring_k_bits[rows, h])
        grp_v = bits_to_f64(ring_v_bits[rows, h])
        r = condense_stream(grp_k, grp_v, qbar[h], g, 0, scale)       # one group: scores on K, pooling of V
        ia = int(r["anchor"][0])
        ring_v[R + n_rep, h] = round_bf16_bits(r["pooled"])[0]
        ring_k[R + n_rep, h] = ring_k_bits[rows[ia], h]
        anchors.append(ia)
    return ring_k, ring_v, n_rep + 1, np.array(anchors, dtype=np.int32)
