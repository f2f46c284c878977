"""Shared helpers of the parity tests: run the CPU oracle on the bit patterns the GPU consumed and
apply the tolerances (written here, measured by oracle/parity.py)."""
from __future__ import annotations

import json
import os

import numpy as np
import torch

from oracle import lca_oracle as O
from oracle import parity as P

# Outputs (bf16 inputs, bf16 tensor-core products, fp32 accumulation and softmax, bf16 result):
#   every element   |err| <= max(ATOL, derived bound)      (oracle/parity.py: output_bound)
#   the mean        mean|err| <= max(MEAN_ATOL, MEAN_RTOL * mean|ref|)
# ATOL / MEAN_ATOL are the bounds stated for the method (values of unit scale); elements of unit scale
# (|ref| <= 1.5 and every value of their column within 5) must meet ATOL as it stands.  The derived bound follows
# the arithmetic -- bf16 weights, fp32 row sum, bf16 store:
# 2^-9 (vmax_c + |ref|) + 2^-8 |ref| -- and only exceeds ATOL where the values or the result are large
# (rows that attend to a x4 needle token reach |out| ~ 16, one bf16 ulp = 0.125).  The rounding of the
# stored output alone has a mean of about 0.7 * 2^-9 of the mean magnitude.
ATOL = 2e-2
MEAN_ATOL = 2e-3
MEAN_RTOL = 2.0 ** -9

f32 = P.f32
sample_positions = P.sample_positions
bf16_ulp_distance = P.bf16_ulp_distance


def oracle_mla(inp: dict, g: int, w: int, scale: float, rows=None, n_summary: int = 0,
               rep_logit_bias: float = 0.0, qbar=None, heads=None):
    """Oracle pipeline for one MLA sequence given torch bf16 CPU tensors (all query rows present).
    Returns dict(cond=..., rows, out [n,H,d_c], lse [n,H])."""
    L = inp["ckv"].shape[0]
    n = min(g if n_summary <= 0 else n_summary, L)
    Lq = inp["q_sem"].shape[0]
    qrs = qrp = None
    if rows is not None:
        idx = torch.from_numpy(np.asarray(rows, dtype=np.int64))
        qrs, qrp = inp["q_sem"][idx], inp["q_pos"][idx]
    return P.mla_pipeline(inp["ckv"], inp["kr"], inp["q_sem"][Lq - n:], inp["q_pos"][Lq - n:], g, w, scale,
                          qrs, qrp, rows, rep_logit_bias, qbar, heads)


def oracle_gqa(inp: dict, g: int, w: int, scale: float, rows=None, n_summary: int = 0,
               rep_logit_bias: float = 0.0):
    L = inp["k"].shape[0]
    n = min(g if n_summary <= 0 else n_summary, L)
    qr = None if rows is None else inp["q"][torch.from_numpy(np.asarray(rows, dtype=np.int64))]
    return P.gqa_pipeline(inp["q"][L - n:], inp["k"], inp["v"], g, w, scale, qr, rows, rep_logit_bias)


def oracle_mla_sampled(ckv, kr, q_tail_sem, q_tail_pos, q_rows_sem, q_rows_pos, rows, g, w, scale, heads=None):
    """Oracle for one full-size MLA sequence when only some query rows are on the host."""
    return P.mla_pipeline(ckv, kr, q_tail_sem, q_tail_pos, g, w, scale, q_rows_sem, q_rows_pos, rows, heads=heads)


def bits(t: torch.Tensor) -> np.ndarray:
    return O.torch_bf16_to_bits(t)


def bits_t(t: torch.Tensor) -> torch.Tensor:
    """bf16 tensor -> its bit patterns as int16 (for exact comparisons on the device)."""
    return t.contiguous().view(torch.int16)


def check_outputs(got: torch.Tensor, ref, what: str = "", vmax=None):
    """Apply the output gate stated at the top of this file; returns the raw statistics (and appends
    them to the file named by LCA_PARITY_LOG, if set, before any assertion).  `ref` is the oracle's
    output array, or the dict of an oracle pipeline (its "out" and "vmax" are used)."""
    if isinstance(ref, dict):
        ref, vmax = ref["out"], ref["vmax"][None] if vmax is None else vmax
    st = P.output_stats(got, ref, vmax)
    if os.environ.get("LCA_PARITY_LOG"):
        with open(os.environ["LCA_PARITY_LOG"], "a") as f:
            f.write(json.dumps(dict(what=what, **st)) + "\n")
    assert st["finite"], f"{what}: non-finite output"
    assert st["max_abs_unit_scale"] <= ATOL, f"{what}: {st}"
    assert st["worst_over_bound"] <= 1.0, f"{what}: {st}"
    assert st["mean_abs"] <= max(MEAN_ATOL, MEAN_RTOL * st["mean_ref"]), f"{what}: {st}"
    return st


def check_condense(res: dict, cond: dict, kind: str = "mla"):
    """Compare the device cache with the oracle's: anchors, copied rows and layout bit-exact
    (both sides score in fp64, so there is no tie allowance to apply; groups whose two best scores
    lie within 1e-6 relative are counted and returned); c_rep within one bf16 ulp (fp32 pooling
    against fp64) or within the absolute bound of the fp32 sum, and at most one element in 250
    different at all.  `res` holds one sequence (batch index already taken)."""
    m, k = cond["m"], cond["k"]
    assert res["m"] == m and res["k"] == k
    st = P.condense_stats(bits(res["cache_sem"]), bits(res["cache_pos"]),
                          res["anchor_idx"].cpu().numpy() if m else None, cond, kind)
    assert st["anchor_mismatches"] == 0, f"anchor mismatches: {st}"
    assert st["pos_rows_differ"] == 0, "positional rows (anchors / local window) differ"
    assert st["local_sem_rows_differ"] == 0, "local-window rows differ"
    assert st["crep_bad"] == 0, f"c_rep off by more than one bf16 ulp and more than the fp32 bound: {st}"
    # a bf16 rounding boundary (spacing 2^-8 relative) is crossed by about one element in 2500
    assert st["crep_off_by_one_ulp"] <= max(2, st["crep_elems"] // 250), f"too many c_rep differences: {st}"
    return st
