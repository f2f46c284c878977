"""Shared helpers of the parity tests: run the CPU oracle on the bit patterns the GPU consumed."""
from __future__ import annotations

import math

import numpy as np
import torch

from oracle import lca_oracle as O

ATOL = 2e-2          # max-abs bound on outputs of unit scale (bf16 inputs, fp32 accumulation)
RTOL = 2.0 ** -7     # one bf16 ulp of the reference, for outputs larger than unit scale
MEAN_ATOL = 2e-3     # mean-abs bound on outputs of unit scale
MEAN_RTOL = 2.0 ** -9  # half a bf16 ulp of the mean output magnitude (the output format's own rounding)


def f32(x: float) -> float:
    """The value the library sees for a float parameter."""
    return float(np.float32(x))


def sample_positions(L: int, g: int, w: int, extra=(), n_uniform: int = 16, seed: int = 0):
    """Stratified query positions: window/group boundaries, both ends, a few uniform ones."""
    cand = [0, 1, g - 1, g, w - 2, w - 1, w, w + 1, w + g - 2, w + g - 1, w + g, w + g + 1,
            w + 2 * g - 1, w + 2 * g, L // 2, L - g - 1, L - 2, L - 1]
    cand += list(extra)
    rng = np.random.default_rng(seed)
    cand += list(rng.integers(0, L, size=n_uniform))
    return np.array(sorted({int(c) for c in cand if 0 <= c < L}), dtype=np.int64)


def oracle_mla(inp: dict, g: int, w: int, scale: float, rows=None, n_summary: int = 0,
               rep_logit_bias: float = 0.0, qbar=None, heads=None):
    """Oracle pipeline for one MLA sequence given torch bf16 CPU tensors.
    Returns dict(cond=..., rows, out [n,H,d_c], lse [n,H])."""
    ckv = O.torch_bf16_to_f64(inp["ckv"])
    kr = O.torch_bf16_to_f64(inp["kr"])
    L = ckv.shape[0]
    n = g if n_summary <= 0 else n_summary
    n = min(n, L)
    if qbar is None:
        Lq = inp["q_sem"].shape[0]
        qbar = O.mla_summary_query(O.torch_bf16_to_f64(inp["q_sem"][Lq - n:]),
                                   O.torch_bf16_to_f64(inp["q_pos"][Lq - n:]))
    cond = O.mla_condense(qbar, ckv, kr, g, w, f32(scale))
    res = dict(cond=cond, qbar=qbar)
    if rows is not None:
        rows = np.asarray(rows, dtype=np.int64)
        m = cond["m"]
        rep_sem = O.bits_to_f64(cond["cache_sem_bits"][:m])
        rep_pos = O.bits_to_f64(cond["cache_pos_bits"][:m])
        qs = inp["q_sem"][torch.from_numpy(rows)]
        qp = inp["q_pos"][torch.from_numpy(rows)]
        if heads is not None:
            qs, qp = qs[:, heads], qp[:, heads]
        out, lse = O.mla_prefill_rows(O.torch_bf16_to_f64(qs), O.torch_bf16_to_f64(qp), rows, ckv, kr,
                                      rep_sem if m else None, rep_pos if m else None, g, w, f32(scale),
                                      f32(rep_logit_bias))
        res.update(rows=rows, out=out, lse=lse)
    return res


def oracle_gqa(inp: dict, g: int, w: int, scale: float, rows=None, n_summary: int = 0,
               rep_logit_bias: float = 0.0):
    k = O.torch_bf16_to_f64(inp["k"])
    v = O.torch_bf16_to_f64(inp["v"])
    L, hkv, d = k.shape
    n = min(g if n_summary <= 0 else n_summary, L)
    qbar = O.gqa_summary_query(O.torch_bf16_to_f64(inp["q"][L - n:]), hkv)
    cond = O.gqa_condense(qbar, k, v, g, w, f32(scale))
    res = dict(cond=cond, qbar=qbar)
    if rows is not None:
        rows = np.asarray(rows, dtype=np.int64)
        m = cond["m"]
        k_rep = O.bits_to_f64(cond["cache_k_bits"][:m])
        v_rep = O.bits_to_f64(cond["cache_v_bits"][:m])
        q = O.torch_bf16_to_f64(inp["q"][torch.from_numpy(rows)])
        out, lse = O.gqa_prefill_rows(q, rows, k, v, k_rep if m else None, v_rep if m else None, g, w,
                                      f32(scale), f32(rep_logit_bias))
        res.update(rows=rows, out=out, lse=lse)
    return res


def bits(t: torch.Tensor) -> np.ndarray:
    return O.torch_bf16_to_bits(t)


def bf16_ulp_distance(a_bits: np.ndarray, b_bits: np.ndarray) -> np.ndarray:
    """Distance in units of bf16 codes (monotone integer mapping of the sign-magnitude bits)."""
    def key(x):
        x = x.astype(np.int32)
        return np.where(x & 0x8000, 0x8000 - x, x)
    return np.abs(key(a_bits) - key(b_bits))


def bits_t(t: torch.Tensor) -> torch.Tensor:
    """bf16 tensor -> its bit patterns as int16 (for exact comparisons on the device)."""
    return t.contiguous().view(torch.int16)


def check_outputs(got: torch.Tensor, ref: np.ndarray, what: str = ""):
    """max-abs <= ATOL + RTOL*|ref| element-wise and mean-abs <= MEAN_ATOL + MEAN_RTOL*mean|ref|;
    returns the stats.  The relative terms only matter where outputs exceed unit scale (rows that
    lock onto a x4 "needle" token reach |out| ~ 16, where one bf16 ulp is already 0.06)."""
    g = got.detach().float().cpu().numpy().astype(np.float64)
    err = np.abs(g - ref)
    bound = ATOL + RTOL * np.abs(ref)
    worst = float((err / bound).max()) if err.size else 0.0
    stats = dict(max_abs=float(err.max()) if err.size else 0.0, mean_abs=float(err.mean()) if err.size else 0.0,
                 worst_ratio=worst, max_ref=float(np.abs(ref).max()) if err.size else 0.0)
    assert np.isfinite(g).all(), f"{what}: non-finite output"
    assert worst <= 1.0, f"{what}: {stats}"
    assert stats["mean_abs"] <= MEAN_ATOL + MEAN_RTOL * float(np.abs(ref).mean()), f"{what}: {stats}"
    return stats


def check_condense(res: dict, cond: dict, kind: str = "mla"):
    """Compare the device cache with the oracle's: anchors, copied rows and layout bit-exact;
    c_rep within one bf16 ulp (fp32 pooling against fp64), differences counted.  `res` holds one sequence (batch index
    already taken)."""
    m, k = cond["m"], cond["k"]
    assert res["m"] == m and res["k"] == k
    sem_key, pos_key = ("cache_sem_bits", "cache_pos_bits") if kind == "mla" else ("cache_v_bits", "cache_k_bits")
    ref_sem = cond[sem_key].reshape(m + k, -1)
    ref_pos = cond[pos_key].reshape(m + k, -1)
    got_sem = bits(res["cache_sem"]).reshape(m + k, -1)
    got_pos = bits(res["cache_pos"]).reshape(m + k, -1)
    if m:
        anchor = res["anchor_idx"].cpu().numpy().reshape(m, -1)
        ref_anchor = cond["anchor"].reshape(m, -1)
        assert np.array_equal(anchor, ref_anchor), f"anchor mismatches: {(anchor != ref_anchor).sum()}"
    assert np.array_equal(got_pos, ref_pos), "positional rows (anchors / local window) differ"
    assert np.array_equal(got_sem[m:], ref_sem[m:]), "local-window rows differ"
    ulp = bf16_ulp_distance(got_sem[:m], ref_sem[:m])
    n_off = int((ulp > 0).sum())
    # The kernel pools in fp32 and the oracle in fp64.  A sum of g terms carries an absolute error
    # of at most g * 2^-24 * sum_i alpha_i |c_i| <= g * 2^-24 * max|c|; where the pooled value is
    # not tiny that is far below one bf16 ulp, so c_rep is within one ulp; where the terms cancel
    # (|c_rep| << |c_i|) an ulp is smaller than that error and the absolute bound applies.
    g_max = 64
    abs_err = np.abs(O.bits_to_f64(got_sem[:m]) - O.bits_to_f64(ref_sem[:m]))
    abs_bound = g_max * 2.0 ** -24 * float(np.abs(O.bits_to_f64(ref_sem)).max()) if ref_sem.size else 0.0
    bad = (ulp > 1) & (abs_err > abs_bound)
    assert not bad.any(), f"c_rep off by more than one bf16 ulp and more than {abs_bound:.2e}: max ulp {ulp.max()}"
    # a bf16 rounding boundary (spacing 2^-8 relative) is crossed by about one element in 2500
    assert n_off <= max(2, ulp.size // 250), f"too many c_rep differences: {n_off}/{ulp.size}"
    return dict(crep_one_ulp=n_off, crep_elems=int(ulp.size))


def oracle_mla_sampled(ckv, kr, q_tail_sem, q_tail_pos, q_rows_sem, q_rows_pos, rows, g, w, scale, heads=None):
    """Oracle for one full-size MLA sequence when only some query rows are on the host: the
    condensation of the whole sequence plus the listed prefill rows (torch bf16 CPU tensors in)."""
    ckv64, kr64 = O.torch_bf16_to_f64(ckv), O.torch_bf16_to_f64(kr)
    qbar = O.mla_summary_query(O.torch_bf16_to_f64(q_tail_sem), O.torch_bf16_to_f64(q_tail_pos))
    cond = O.mla_condense(qbar, ckv64, kr64, g, w, f32(scale))
    m = cond["m"]
    rep_sem = O.bits_to_f64(cond["cache_sem_bits"][:m]) if m else None
    rep_pos = O.bits_to_f64(cond["cache_pos_bits"][:m]) if m else None
    qs, qp = q_rows_sem, q_rows_pos
    if heads is not None:
        qs, qp = qs[:, heads], qp[:, heads]
    out, lse = O.mla_prefill_rows(O.torch_bf16_to_f64(qs), O.torch_bf16_to_f64(qp), np.asarray(rows, dtype=np.int64),
                                  ckv64, kr64, rep_sem, rep_pos, g, w, f32(scale))
    return dict(cond=cond, out=out, lse=lse)
