"""Oracle pipelines and comparison statistics built on oracle/lca_oracle.py.

TEST INFRASTRUCTURE ONLY (tests/, the smoke check, the benchmark's cpu_baseline / reference leg).
Nothing here touches CUDA or the CUDA package: device tensors are copied to the host by the
caller; the functions take torch bf16 CPU tensors (bit patterns are widened exactly to fp64) and
return numpy arrays and plain numbers.  The tolerances that decide pass / fail are written in the
tests, not here: these functions only measure.
"""
from __future__ import annotations

import numpy as np

from . import lca_oracle as O


def f32(x: float) -> float:
    """The value the library sees for a float parameter."""
    return float(np.float32(x))


def sample_positions(L: int, g: int, w: int, extra=(), n_uniform: int = 16, seed: int = 0):
    """Stratified query positions: window / group boundaries, both ends, a few uniform ones."""
    cand = [0, 1, g - 1, g, w - 2, w - 1, w, w + 1, w + g - 2, w + g - 1, w + g, w + g + 1,
            w + 2 * g - 1, w + 2 * g, L // 2, L - g - 1, L - 2, L - 1]
    cand += list(extra)
    rng = np.random.default_rng(seed)
    cand += list(rng.integers(0, L, size=n_uniform))
    return np.array(sorted({int(c) for c in cand if 0 <= c < L}), dtype=np.int64)


# ------------------------------------------------------------------------------- pipelines
def mla_pipeline(ckv, kr, q_tail_sem, q_tail_pos, g, w, scale, q_rows_sem=None, q_rows_pos=None, rows=None,
                 rep_logit_bias: float = 0.0, qbar=None, heads=None):
    """Summary query -> condensation of the whole sequence -> the listed prefill rows (Alg. 1,
    Eq. 10 at each listed prefix length) for one MLA sequence.  `q_tail_*` are the last
    n_summary_q query positions; `q_rows_*` the queries of the positions in `rows`."""
    ckv64, kr64 = O.torch_bf16_to_f64(ckv), O.torch_bf16_to_f64(kr)
    if qbar is None:
        qbar = O.mla_summary_query(O.torch_bf16_to_f64(q_tail_sem), O.torch_bf16_to_f64(q_tail_pos))
    cond = O.mla_condense(qbar, ckv64, kr64, g, w, f32(scale))
    res = dict(cond=cond, qbar=qbar)
    if rows is not None:
        rows = np.asarray(rows, dtype=np.int64)
        m = cond["m"]
        rep_sem = O.bits_to_f64(cond["cache_sem_bits"][:m]) if m else None
        rep_pos = O.bits_to_f64(cond["cache_pos_bits"][:m]) if m else None
        qs, qp = q_rows_sem, q_rows_pos
        if heads is not None:
            qs, qp = qs[:, heads], qp[:, heads]
        out, lse = O.mla_prefill_rows(O.torch_bf16_to_f64(qs), O.torch_bf16_to_f64(qp), rows, ckv64, kr64,
                                      rep_sem, rep_pos, g, w, f32(scale), f32(rep_logit_bias))
        res.update(rows=rows, out=out, lse=lse)
    res["vmax"] = np.abs(ckv64).max(axis=0)            # largest |value| per latent column (needle rows included)
    return res


def gqa_pipeline(q_tail, k, v, g, w, scale, q_rows=None, rows=None, rep_logit_bias: float = 0.0):
    """The same for one GQA sequence (Sec. 5.4): k, v [L, Hkv, d]; q_tail the last n_summary_q queries."""
    k64, v64 = O.torch_bf16_to_f64(k), O.torch_bf16_to_f64(v)
    hkv = k64.shape[1]
    qbar = O.gqa_summary_query(O.torch_bf16_to_f64(q_tail), hkv)
    cond = O.gqa_condense(qbar, k64, v64, g, w, f32(scale))
    res = dict(cond=cond, qbar=qbar)
    if rows is not None:
        rows = np.asarray(rows, dtype=np.int64)
        m = cond["m"]
        k_rep = O.bits_to_f64(cond["cache_k_bits"][:m]) if m else None
        v_rep = O.bits_to_f64(cond["cache_v_bits"][:m]) if m else None
        out, lse = O.gqa_prefill_rows(O.torch_bf16_to_f64(q_rows), rows, k64, v64, k_rep, v_rep, g, w,
                                      f32(scale), f32(rep_logit_bias))
        res.update(rows=rows, out=out, lse=lse)
    hq = O.torch_bf16_to_f64(q_tail).shape[1]
    res["vmax"] = np.repeat(np.abs(v64).max(axis=0), hq // hkv, axis=0)      # [Hq, d]: per query head, its KV head's columns
    return res


# ------------------------------------------------------------------------------ statistics
def bf16_ulp_distance(a_bits: np.ndarray, b_bits: np.ndarray) -> np.ndarray:
    """Distance in units of bf16 codes (monotone integer mapping of the sign-magnitude bits)."""
    def key(x):
        x = x.astype(np.int32)
        return np.where(x & 0x8000, 0x8000 - x, x)
    return np.abs(key(a_bits) - key(b_bits))


def output_bound(ref: np.ndarray, vmax=None) -> np.ndarray:
    """Element-wise error bound of an attention output computed with bf16 probabilities.

    The kernels round the softmax weights p_i to bf16 before P V (relative error at most 2^-9 each) and
    divide by a row sum taken in fp32.  Whether that sum runs over the rounded or the unrounded weights,
    the error in column c is at most 2^-9 sum_i p_i max(|v_ic|, |v_ic - out_c|) / sum_i p_i
    <= 2^-9 (vmax_c + |out_c|), vmax_c = the largest |value| of that column; the bf16 store of the result
    adds up to 2^-8 |out_c| (half an ulp, relative 2^-9 at the top of a binade and 2^-8 at the bottom).
    For values of unit scale (N(0,1): vmax ~ 4.6) that is below the 2e-2 stated for the method; it grows
    with the values (x4 "needle" rows: vmax ~ 17).  The bound returned is the larger of the stated 2e-2
    and the derived one.  Without `vmax` only the output rounding is scaled: max(2e-2, 2^-7 |ref|)."""
    aref = np.abs(ref)
    if vmax is None:
        return np.maximum(2e-2, 2.0 ** -7 * aref)
    return np.maximum(2e-2, 2.0 ** -9 * (np.asarray(vmax) + aref) + 2.0 ** -8 * aref)


def output_stats(got, ref: np.ndarray, vmax=None) -> dict:
    """Raw error figures of an attention output (`got`: torch tensor on any device, or numpy) and the
    worst ratio to output_bound."""
    g = got.detach().float().cpu().numpy() if hasattr(got, "detach") else np.asarray(got)
    g = g.astype(np.float64)
    if g.size == 0:
        return dict(n=0, max_abs=0.0, mean_abs=0.0, max_ref=0.0, mean_ref=0.0, finite=True, n_above_2e2=0,
                    max_abs_unit_scale=0.0, worst_over_bound=0.0)
    err = np.abs(g - ref)
    aref = np.abs(ref)
    # elements whose column holds only values of unit scale (|v| <= 5: no x4 needle of any size) and whose result
    # is of unit scale (|ref| <= 1.5): there the derived bound is below 2e-2, which must then hold as stated
    unit = aref <= 1.5 if vmax is None else (aref <= 1.5) & (np.broadcast_to(np.asarray(vmax), ref.shape) <= 5.0)
    return dict(n=int(err.size), max_abs=float(err.max()), mean_abs=float(err.mean()), max_ref=float(aref.max()),
                mean_ref=float(aref.mean()), finite=bool(np.isfinite(g).all()), n_above_2e2=int((err > 2e-2).sum()),
                max_abs_unit_scale=float(err[unit].max()) if unit.any() else 0.0,
                worst_over_bound=float((err / output_bound(ref, vmax)).max()))


def near_ties(scores: np.ndarray, g: int, rel: float = 1e-6) -> int:
    """Groups whose two largest importance scores differ by at most `rel` relative (an fp32 scorer
    could legitimately pick either as the anchor)."""
    if scores.size == 0:
        return 0
    s = np.sort(scores.reshape(-1, g), axis=1)
    if g < 2:
        return 0
    top, second = s[:, -1], s[:, -2]
    return int((np.abs(top - second) <= rel * np.maximum(np.abs(top), np.abs(second))).sum())


def condense_stats(got_sem_bits, got_pos_bits, got_anchor, cond: dict, kind: str = "mla") -> dict:
    """Compare a device cache (bf16 bit patterns [m+k, ...], anchors [m, ...]) with the oracle's."""
    m, k = cond["m"], cond["k"]
    sem_key, pos_key = ("cache_sem_bits", "cache_pos_bits") if kind == "mla" else ("cache_v_bits", "cache_k_bits")
    ref_sem = cond[sem_key].reshape(m + k, -1)
    ref_pos = cond[pos_key].reshape(m + k, -1)
    got_sem = np.asarray(got_sem_bits).reshape(m + k, -1)
    got_pos = np.asarray(got_pos_bits).reshape(m + k, -1)
    st = dict(m=m, k=k, anchor_mismatches=0, near_tie_groups=0, pos_rows_differ=int((got_pos != ref_pos).any(axis=1).sum()),
              local_sem_rows_differ=int((got_sem[m:] != ref_sem[m:]).any(axis=1).sum()),
              crep_elems=int(got_sem[:m].size), crep_off_by_one_ulp=0, crep_max_ulp=0, crep_bad=0)
    if m:
        anchor = np.asarray(got_anchor).reshape(m, -1)
        st["anchor_mismatches"] = int((anchor != cond["anchor"].reshape(m, -1)).sum())
        g = cond["scores"].shape[0] // m
        sc = cond["scores"] if cond["scores"].ndim == 1 else cond["scores"].T
        st["near_tie_groups"] = near_ties(np.ascontiguousarray(sc), g)
        ulp = bf16_ulp_distance(got_sem[:m], ref_sem[:m])
        # fp32 weights and fp32 pooling of g <= 64 terms against fp64: absolute error at most about
        # 64 * 2^-24 * max|c| (weights good to ~2^-21 relative, one rounding per accumulated term); where
        # the pooled value is not tiny that is far below one bf16 ulp, where the terms cancel it is not
        abs_err = np.abs(O.bits_to_f64(got_sem[:m]) - O.bits_to_f64(ref_sem[:m]))
        abs_bound = max(g, 64) * 2.0 ** -24 * float(np.abs(O.bits_to_f64(ref_sem)).max())
        st.update(crep_off_by_one_ulp=int((ulp > 0).sum()), crep_max_ulp=int(ulp.max()),
                  crep_bad=int(((ulp > 1) & (abs_err > abs_bound)).sum()), crep_abs_bound=abs_bound)
    return st
