"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU needed).

Each test compares the oracle with something that is not the oracle: a numpy restatement of a
textbook definition, a closed form, an invariant of the paper's propositions, or a number the
paper prints (tests/golden/).  A plausible slip in the oracle (dropped term, wrong index or
sign, transposed operand, off-by-one in the window) fails at least one of them.
"""
import math
import os

import numpy as np
import pytest

from oracle import lca_oracle as O

HERE = os.path.dirname(os.path.abspath(__file__))
RNG = np.random.default_rng


# ------------------------------------------------------------------ independent numpy pieces
def np_softmax(x):
    x = x - x.max()
    e = np.exp(x)
    return e / e.sum()


def np_dense_causal(q, key, val, scale):
    """Textbook causal attention (Eq. 5): q [L,H,dk], key [L,dk], val [L,dv] -> [L,H,dv]."""
    L, H, _ = q.shape
    out = np.zeros((L, H, val.shape[1]))
    for t in range(L):
        for h in range(H):
            p = np_softmax(key[: t + 1] @ q[t, h] * scale)
            out[t, h] = p @ val[: t + 1]
    return out


def np_fused_context_attention(qbar, q_last, C, KR, w, g, scale, bias=0.0):
    """LCA for ONE sequence prefix and its LAST query (all heads), written from the definitions of
    Sec. 4.2 / Eq. 6-10 with whole-array numpy operations (the oracle loops over tokens): the distant
    history is folded into an [m, g, .] block, the group softmax, the pooled latents and the anchors
    come out of that block at once, and the fused key / value matrices of Eq. 9-10 are materialised
    before a single softmax.  q_last [H, dc+dr]; C [t, dc]; KR [t, dr]."""
    t, dc = C.shape
    m = (t - w) // g if t >= w + g else 0
    K = np.concatenate([C, KR], axis=1)
    hist = K[: m * g].reshape(m, g, K.shape[1])                              # G_1 .. G_m
    s = hist @ qbar * scale                                           # importance scores, [m, g]
    e = np.exp(s - s.max(axis=1, keepdims=True, initial=-np.inf))
    alpha = e / e.sum(axis=1, keepdims=True)                          # Eq. 6
    c_rep = np.einsum("mg,mgc->mc", alpha, C[: m * g].reshape(m, g, dc))      # Eq. 7
    anchor = (s.argmax(axis=1) if m else np.zeros(0, int)) + g * np.arange(m)     # Eq. 8 (first maximum)
    k_rep = np.concatenate([c_rep, KR[anchor.astype(int)]], axis=1)
    K_f = np.concatenate([k_rep, K[m * g:]], axis=0)                  # Eq. 9: every token after the groups
    V_f = np.concatenate([c_rep, C[m * g:]], axis=0)
    logits = q_last @ K_f.T * scale                                   # Eq. 10
    logits[:, :m] += bias
    p = np.exp(logits - logits.max(axis=1, keepdims=True))
    return (p / p.sum(axis=1, keepdims=True)) @ V_f


def np_summary_query(qs, qp, n):
    """Mean over the last n positions and all heads of [q_latent | q_rope] (Alg. 1, first step)."""
    q = np.concatenate([qs, qp], axis=-1)
    return q[q.shape[0] - n:].reshape(-1, q.shape[-1]).mean(axis=0)


def rand_mla(rng, L, H, dc, dr):
    return (rng.standard_normal((L, H, dc)), rng.standard_normal((L, H, dr)),
            rng.standard_normal((L, dc)), rng.standard_normal((L, dr)))


def oracle_full_prefill(qs, qp, C, KR, g, w, scale, bias=0.0, n_summary=None):
    """Run the whole oracle pipeline (summary query -> condense -> every prefill row), keeping
    the representatives UNROUNDED so that fp64 identities can be checked to round-off."""
    L = C.shape[0]
    n = min(L, g if n_summary is None else n_summary)
    qbar = O.mla_summary_query(qs[L - n:], qp[L - n:])
    key = np.concatenate([C, KR], axis=1)
    cs = O.condense_stream(key, C, qbar, g, w, scale)
    rep_sem = cs["pooled"]
    rep_pos = KR[cs["anchor"]] if cs["m"] else np.zeros((0, KR.shape[1]))
    out, lse = O.mla_prefill_rows(qs, qp, np.arange(L), C, KR, rep_sem, rep_pos, g, w, scale, bias)
    return qbar, cs, out, lse


# ------------------------------------------------------------------------------------ pins
def test_partition_accounts_for_every_token():
    # Sec. 4.2: m = floor((L-w)/g), k = w + (L-w) mod g, "every token is accounted for".
    for L in range(1, 200):
        for g in (1, 2, 3, 4, 7, 16):
            for w in (0, 1, 5, 16, 64, 300):
                m, k = O.partition(L, w, g)
                assert m * g + k == L
                if L < w + g:
                    assert m == 0 and k == L
                else:
                    assert m == (L - w) // g and w <= k < w + g


def test_cache_reduction_matches_printed_sizes():
    # One representative per group shared by all heads + w local tokens reproduces the sizes
    # the paper prints at 128K with g=16, w=1024 (golden file cites where each is printed).
    L, g, w = 131072, 16, 1024
    m, k = O.partition(L, w, g)
    assert (m, k) == (8128, 1024)
    ratio = (m + k) / L
    assert abs((1 - ratio) - 0.9302) < 1e-4
    with open(os.path.join(HERE, "golden", "kv_cache_sizes.txt")) as f:
        rows = [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 3
    for name, full, small in rows:
        pred = float(full) * ratio
        assert abs(pred - float(small)) <= 0.0051 + 0.005 * ratio, (name, pred, small)


def test_bf16_rounding_matches_ieee_rne():
    torch = pytest.importorskip("torch")
    rng = RNG(0)
    x32 = (rng.standard_normal(20000) * np.exp(rng.uniform(-30, 30, 20000))).astype(np.float32)
    ref = torch.from_numpy(x32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = O.round_bf16_bits(x32.astype(np.float64))
    assert np.array_equal(ref, got)
    # exact ties go to even: 1 + 2^-8 is halfway between 1 and 1 + 2^-7
    assert O.round_bf16_bits(np.array([1.0 + 2.0 ** -8]))[0] == 0x3F80
    assert O.round_bf16_bits(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 0x3F82
    # a double just above the tie must round up although its float32 image is the tie itself
    assert O.round_bf16_bits(np.array([1.0 + 2.0 ** -8 + 2.0 ** -40]))[0] == 0x3F81
    b = np.arange(0, 0x7F80, 7, dtype=np.uint16)
    assert np.array_equal(O.round_bf16_bits(O.bits_to_f64(b)), b)


@pytest.mark.parametrize("w", [0, 1, 3, 8])
def test_group_size_one_is_dense_attention(w):
    # g = 1: alpha = 1, c_rep = c_i, I_j = i, so LCA is exactly dense causal MLA (Eq. 5).
    rng = RNG(1)
    L, H, dc, dr = 23, 2, 6, 4
    qs, qp, C, KR = rand_mla(rng, L, H, dc, dr)
    scale = 0.3
    _, cs, out, _ = oracle_full_prefill(qs, qp, C, KR, 1, w, scale)
    assert cs["m"] == L - w and np.array_equal(cs["anchor"], np.arange(L - w))
    ref = np_dense_causal(np.concatenate([qs, qp], -1), np.concatenate([C, KR], 1), C, scale)
    np.testing.assert_allclose(out, ref, rtol=0, atol=1e-12)


def test_window_covering_sequence_is_dense_attention():
    # L < w + g: no complete group, the method reverts to standard MLA (Sec. 4.3).
    rng = RNG(2)
    L, H, dc, dr = 19, 3, 5, 2
    qs, qp, C, KR = rand_mla(rng, L, H, dc, dr)
    ref = np_dense_causal(np.concatenate([qs, qp], -1), np.concatenate([C, KR], 1), C, 0.25)
    for g, w in ((4, 16), (4, 19), (8, 100), (20, 0)):
        _, cs, out, _ = oracle_full_prefill(qs, qp, C, KR, g, w, 0.25)
        assert cs["m"] == 0
        np.testing.assert_allclose(out, ref, rtol=0, atol=1e-12)


@pytest.mark.parametrize("g,w", [(2, 0), (2, 1), (3, 5), (4, 1), (4, 5), (3, 0)])
def test_every_row_is_alg1_on_its_prefix(g, w):
    # Row t of the prefill equals Alg. 1 run literally on the length-t prefix (same q_bar):
    # pins the per-query window, the group staircase and the K_loc row count (Eq. 9).
    rng = RNG(3)
    L, H, dc, dr = 41, 2, 5, 3
    qs, qp, C, KR = rand_mla(rng, L, H, dc, dr)
    scale = 0.4
    for bias in (0.0, math.log(g)):
        _, _, out, _ = oracle_full_prefill(qs, qp, C, KR, g, w, scale, bias)
        qbar = np_summary_query(qs, qp, min(L, g))          # not the oracle's: [latent | rope] order is part of the pin
        q = np.concatenate([qs, qp], -1)
        for t in range(1, L + 1):
            ref = np_fused_context_attention(qbar, q[t - 1], C[:t], KR[:t], w, g, scale, bias)
            np.testing.assert_allclose(out[t - 1], ref, rtol=0, atol=1e-12, err_msg=f"t={t}")


def test_summary_query_is_mean_of_last_rows_and_heads():
    rng = RNG(4)
    q = rng.standard_normal((9, 3, 7))
    np.testing.assert_allclose(O.summary_query(q[-4:]), q[-4:].reshape(-1, 7).mean(0), atol=1e-15)
    # a single head with a single row is returned untouched
    np.testing.assert_array_equal(O.summary_query(q[-1:, :1]), q[-1, 0])


def test_mla_summary_query_is_latent_part_then_rope_part():
    # Alg. 1 first step on the absorbed query [q_latent | q_rope]: d_c != d_R, so a swapped concatenation,
    # a mean over the wrong axis or a dropped head cannot pass.
    rng = RNG(41)
    n, H, dc, dr = 5, 3, 7, 2
    qs, qp = rng.standard_normal((n, H, dc)), rng.standard_normal((n, H, dr)) + 10.0
    got = O.mla_summary_query(qs, qp)
    assert got.shape == (dc + dr,)
    np.testing.assert_allclose(got, np.concatenate([qs, qp], -1).mean((0, 1)), atol=1e-14)
    np.testing.assert_allclose(got[:dc], qs.reshape(-1, dc).mean(0), atol=1e-14)
    assert (got[dc:] > 5.0).all()                       # the rope part (shifted by 10) sits at the end


def test_alpha_is_a_distribution_and_pooling_is_convex():
    rng = RNG(5)
    L, g, w, dc, dr = 70, 8, 6, 9, 4
    C, KR = rng.standard_normal((L, dc)), rng.standard_normal((L, dr))
    qbar = rng.standard_normal(dc + dr)
    cs = O.condense_stream(np.concatenate([C, KR], 1), C, qbar, g, w, 0.5)
    m = cs["m"]
    a = cs["alpha"].reshape(m, g)
    assert (a >= 0).all()
    np.testing.assert_allclose(a.sum(1), 1.0, atol=1e-14)
    grp = C[: m * g].reshape(m, g, dc)
    assert (cs["pooled"] <= grp.max(1) + 1e-14).all() and (cs["pooled"] >= grp.min(1) - 1e-14).all()
    # scores are the scaled dot products against the FULL key [c | k^R]
    np.testing.assert_allclose(cs["scores"], (np.concatenate([C, KR], 1)[: m * g] @ qbar) * 0.5, atol=1e-13)
    # anchors: arg-max inside the group, absolute index
    for j in range(m):
        assert cs["anchor"][j] == j * g + int(np.argmax(cs["scores"][j * g:(j + 1) * g]))


def test_proposition_1_weighted_mean_minimises_expected_error():
    # Prop. 1: c_rep = sum_i alpha_i c_i is the unique minimiser of sum_i alpha_i ||c_i - c||^2.
    rng = RNG(6)
    L, g, w, dc, dr = 48, 6, 0, 7, 3
    C, KR = rng.standard_normal((L, dc)), rng.standard_normal((L, dr))
    qbar = rng.standard_normal(dc + dr) * 2
    cs = O.condense_stream(np.concatenate([C, KR], 1), C, qbar, g, w, 0.7)
    for j in range(cs["m"]):
        a = cs["alpha"][j * g:(j + 1) * g]
        ci = C[j * g:(j + 1) * g]
        loss = lambda c: float((a * ((ci - c) ** 2).sum(1)).sum())
        base = loss(cs["pooled"][j])
        grad = 2 * (cs["pooled"][j] - a @ ci)
        np.testing.assert_allclose(grad, 0, atol=1e-14)
        for _ in range(5):
            assert loss(cs["pooled"][j] + 1e-3 * rng.standard_normal(dc)) > base


def test_zero_summary_query_gives_mean_pooling_and_first_token_anchor():
    # alpha_i = 1/g is the mean-pooling special case (App. A.1); ties -> lowest index.
    rng = RNG(7)
    L, g, w, dc, dr = 40, 5, 3, 6, 2
    C, KR = rng.standard_normal((L, dc)), rng.standard_normal((L, dr))
    cs = O.condense_stream(np.concatenate([C, KR], 1), C, np.zeros(dc + dr), g, w, 1.0)
    m = cs["m"]
    np.testing.assert_allclose(cs["pooled"], C[: m * g].reshape(m, g, dc).mean(1), atol=1e-15)
    assert np.array_equal(cs["anchor"], np.arange(m) * g)


def test_dominant_token_gives_one_hot_and_constant_group_is_preserved():
    rng = RNG(8)
    L, g, w, dc, dr = 32, 8, 0, 4, 2
    C, KR = rng.standard_normal((L, dc)), rng.standard_normal((L, dr))
    qbar = rng.standard_normal(dc + dr)
    key = np.concatenate([C, KR], 1)
    hot = 8 + 5                                       # token 5 of group 1
    key[hot] = qbar * 1000.0                          # s = 1000 |q|^2: softmax must not overflow
    cs = O.condense_stream(key, C, qbar, g, w, 1.0)
    assert np.isfinite(cs["pooled"]).all()
    np.testing.assert_allclose(cs["pooled"][1], C[hot], atol=1e-12)
    assert cs["anchor"][1] == hot
    C2 = C.copy()
    C2[16:24] = C2[16]                                # constant group 2
    cs2 = O.condense_stream(np.concatenate([C2, KR], 1), C2, qbar, g, w, 1.0)
    np.testing.assert_allclose(cs2["pooled"][2], C2[16], atol=1e-15)


def test_absorbed_form_equals_unabsorbed_form():
    # Alg. 1 builds k_rep = [c_rep W^UK, k^R_I], v_rep = c_rep W^UV.  With
    # q_latent = q_nope W^UK^T the latent-space result times W^UV must equal it exactly.
    rng = RNG(9)
    L, H, dc, dr, dn, dv = 37, 2, 6, 4, 5, 3
    g, w, scale = 4, 6, 0.35
    C, KR = rng.standard_normal((L, dc)), rng.standard_normal((L, dr))
    WUK = rng.standard_normal((H, dc, dn))
    WUV = rng.standard_normal((H, dc, dv))
    q_nope, q_rope = rng.standard_normal((L, H, dn)), rng.standard_normal((L, H, dr))
    q_lat = np.einsum("lhn,hcn->lhc", q_nope, WUK)
    qbar, cs, out_lat, _ = oracle_full_prefill(q_lat, q_rope, C, KR, g, w, scale)
    m = cs["m"]
    for t in (1, 7, 10, 11, 25, L):
        p = t - 1
        mt = 0 if t < w + g else (t - w) // g
        for h in range(H):
            ks = [np.concatenate([cs["pooled"][j] @ WUK[h], KR[cs["anchor"][j]]]) for j in range(mt)]
            vs = [cs["pooled"][j] @ WUV[h] for j in range(mt)]
            for i in range(mt * g, t):
                ks.append(np.concatenate([C[i] @ WUK[h], KR[i]]))
                vs.append(C[i] @ WUV[h])
            qh = np.concatenate([q_nope[p, h], q_rope[p, h]])
            ref = np_softmax(np.array(ks) @ qh * scale) @ np.array(vs)
            np.testing.assert_allclose(O.latent_to_value(out_lat[p], WUV)[h], ref, atol=1e-11)
    assert m == (L - w) // g


def test_latent_to_value_is_one_matrix_product_per_head():
    # explicit loops, non-square shapes and heads that differ: a transposed W^UV, a shared head or a wrong
    # contraction axis cannot pass
    rng = RNG(44)
    T, H, dc, dv = 3, 2, 5, 4
    x = rng.standard_normal((T, H, dc))
    W = rng.standard_normal((H, dc, dv)) * np.array([1.0, -3.0])[:, None, None]
    got = O.latent_to_value(x, W)
    assert got.shape == (T, H, dv)
    for t in range(T):
        for h in range(H):
            for v in range(dv):
                assert abs(got[t, h, v] - sum(x[t, h, c] * W[h, c, v] for c in range(dc))) < 1e-13


def test_decode_equals_prefill_row_of_longer_sequence():
    # Decoding token L+1 against the cache of L tokens with its own latent appended equals the
    # prefill row L+1 of the longer sequence as long as no new group completes (Sec. 4.3).
    rng = RNG(10)
    H, dc, dr, g, w, scale = 2, 5, 3, 4, 6, 0.45
    L = 30                                   # (L - w) = 24 = 6 groups exactly; L+1 adds a residual token
    qs, qp, C, KR = rand_mla(rng, L + 1, H, dc, dr)
    qbar = O.mla_summary_query(qs[L - g:L], qp[L - g:L])
    key = np.concatenate([C[:L], KR[:L]], 1)
    cs = O.condense_stream(key, C[:L], qbar, g, w, scale)
    m, k = cs["m"], cs["k"]
    cache_sem = np.concatenate([cs["pooled"], C[L - k:L], C[L:L + 1]], 0)
    cache_pos = np.concatenate([KR[cs["anchor"]], KR[L - k:L], KR[L:L + 1]], 0)
    out_d, lse_d = O.mla_decode(qs[L], qp[L], cache_sem, cache_pos, m, scale)
    out_p, lse_p = O.mla_prefill_rows(qs[L:L + 1], qp[L:L + 1], np.array([L]), C, KR, cs["pooled"],
                                      KR[cs["anchor"]], g, w, scale)
    np.testing.assert_allclose(out_d, out_p[0], atol=1e-12)
    np.testing.assert_allclose(lse_d, lse_p[0], atol=1e-12)
    # and the last prefill row is Alg. 1 on the whole sequence (summary query restated in numpy)
    np.testing.assert_allclose(qbar, np_summary_query(qs[:L], qp[:L], g), atol=1e-15)
    ref = np_fused_context_attention(np_summary_query(qs[:L], qp[:L], g), np.concatenate([qs[L - 1], qp[L - 1]], -1),
                                     C[:L], KR[:L], w, g, scale)
    out_last, _ = O.mla_prefill_rows(qs[L - 1:L], qp[L - 1:L], np.array([L - 1]), C[:L], KR[:L],
                                     cs["pooled"], KR[cs["anchor"]], g, w, scale)
    np.testing.assert_allclose(out_last[0], ref, atol=1e-12)


def test_lse_is_log_sum_exp_of_logits():
    rng = RNG(11)
    L, H, dc, dr = 12, 1, 4, 2
    qs, qp, C, KR = rand_mla(rng, L, H, dc, dr)
    _, _, out, lse = oracle_full_prefill(qs, qp, C, KR, 3, 100, 0.5)
    q = np.concatenate([qs, qp], -1)
    K = np.concatenate([C, KR], 1)
    for t in range(L):
        lg = K[: t + 1] @ q[t, 0] * 0.5
        assert abs(lse[t, 0] - np.log(np.exp(lg).sum())) < 1e-12


def test_attention_invariances():
    rng = RNG(12)
    L, H, dc, dr, g, w, scale = 33, 2, 5, 3, 4, 5, 0.4
    qs, qp, C, KR = rand_mla(rng, L, H, dc, dr)
    qbar, cs, out, _ = oracle_full_prefill(qs, qp, C, KR, g, w, scale)
    rs, rp = cs["pooled"], KR[cs["anchor"]]
    rows = np.array([L - 1])
    # permuting the representatives leaves the last row unchanged
    perm = rng.permutation(cs["m"])
    o2, _ = O.mla_prefill_rows(qs[-1:], qp[-1:], rows, C, KR, rs[perm], rp[perm], g, w, scale)
    np.testing.assert_allclose(o2[0], out[-1], atol=1e-13)
    # a huge constant added to every logit (through the bias on reps only it is NOT invariant,
    # so shift all keys along q instead): softmax shift invariance via lse
    # scaling all values scales the output: values are the latents themselves, so use decode
    ckey = np.concatenate([np.concatenate([rs, C[L - cs["k"]:]], 0), np.concatenate([rp, KR[L - cs["k"]:]], 0)], 1)
    cval = np.concatenate([rs, C[L - cs["k"]:]], 0)
    qv = np.concatenate([qs[-1], qp[-1]], -1)
    o3, l3 = O.decode_rows(qv, ckey, cval, cs["m"], scale)
    np.testing.assert_allclose(o3, out[-1], atol=1e-13)
    o4, l4 = O.decode_rows(qv, ckey, 3.0 * cval, cs["m"], scale)
    np.testing.assert_allclose(o4, 3.0 * o3, atol=1e-13)
    np.testing.assert_allclose(l4, l3, atol=1e-13)
    # rep_logit_bias multiplies each representative's weight by e^bias
    b = 0.7
    o5, _ = O.decode_rows(qv, ckey, cval, cs["m"], scale, b)
    for h in range(H):
        lg = ckey @ qv[h] * scale
        lg[: cs["m"]] += b
        np.testing.assert_allclose(o5[h], np_softmax(lg) @ cval, atol=1e-13)


def _theorem_terms(q_t, K, V, rep_k, rep_v, mt, g, scale):
    dk = max((np.linalg.norm(K[i] - rep_k[i // g]) for i in range(mt * g)), default=0.0)
    dv = max((np.linalg.norm(V[i] - rep_v[i // g]) for i in range(mt * g)), default=0.0)
    Q = np.linalg.norm(q_t)
    Vn = max(np.linalg.norm(V[i]) for i in range(len(V)))
    return Vn * (math.exp(2 * Q * dk * scale) - 1) + dv


@pytest.mark.parametrize("L", [64, 256])
def test_theorem_1_bound_holds_for_multiplicity_weighted_form(L):
    # Theorem 1 (uniform, L-independent bound).  Its proof weights every representative by the
    # size of its group, i.e. rep_logit_bias = ln g; that form must satisfy the bound for all t.
    rng = RNG(13)
    H, dc, dr, g, w = 1, 6, 2, 4, 8
    scale = 1 / math.sqrt(dc + dr)
    base = rng.standard_normal((L // g + 1, dc + dr))
    tok = np.repeat(base, g, axis=0)[:L] + 0.02 * rng.standard_normal((L, dc + dr))   # clustered groups
    C, KR = tok[:, :dc], tok[:, dc:]
    qs, qp = rng.standard_normal((L, H, dc)), rng.standard_normal((L, H, dr))
    qbar, cs, out, _ = oracle_full_prefill(qs, qp, C, KR, g, w, scale, bias=math.log(g))
    K = np.concatenate([C, KR], 1)
    rep_k = np.concatenate([cs["pooled"], KR[cs["anchor"]]], 1)
    q = np.concatenate([qs, qp], -1)
    dense = np_dense_causal(q, K, C, scale)
    worst = 0.0
    for t in range(1, L + 1):
        mt = 0 if t < w + g else (t - w) // g
        bound = _theorem_terms(q[t - 1, 0], K[:t], C[:t], rep_k, cs["pooled"], mt, g, scale)
        err = np.linalg.norm(dense[t - 1, 0] - out[t - 1, 0])
        assert err <= bound + 1e-12, (t, err, bound)
        worst = max(worst, err / max(bound, 1e-300)) if bound > 0 else worst
    assert worst <= 1.0


def test_theorem_1_counter_example_for_unweighted_form():
    # Identical keys (delta_k = 0), history values a, recent values b (delta_v = 0): the bound is
    # 0.  The ln g form reproduces dense attention exactly; Alg. 1 as printed (bias 0) gives
    # (m a + k b)/(m + k) instead of ((t-k) a + k b)/t.
    g, w, L, dc, dr = 4, 4, 20, 3, 2
    a, b = np.array([1.0, 0.0, 2.0]), np.array([-1.0, 3.0, 0.5])
    m, k = O.partition(L, w, g)
    C = np.concatenate([np.tile(a, (m * g, 1)), np.tile(b, (k, 1))], 0)
    KR = np.ones((L, dr))
    # keys must be identical although values differ: make the query blind to the latent part
    qs, qp = np.zeros((L, 1, dc)), np.ones((L, 1, dr))
    _, cs, out_ln, _ = oracle_full_prefill(qs, qp, C, KR, g, w, 0.5, bias=math.log(g))
    _, _, out_0, _ = oracle_full_prefill(qs, qp, C, KR, g, w, 0.5, bias=0.0)
    dense_last = ((L - k) * a + k * b) / L
    np.testing.assert_allclose(out_ln[-1, 0], dense_last, atol=1e-13)
    np.testing.assert_allclose(out_0[-1, 0], (m * a + k * b) / (m + k), atol=1e-13)
    assert np.linalg.norm(out_0[-1, 0] - dense_last) > 0.1


def test_gqa_with_group_one_is_textbook_mha():
    # Sec. 5.4 adaptation: max-selection on keys, weighted pooling on values, per KV head.
    rng = RNG(14)
    L, Hq, Hkv, d, scale = 17, 4, 2, 6, 0.4
    q = rng.standard_normal((L, Hq, d))
    k = rng.standard_normal((L, Hkv, d))
    v = rng.standard_normal((L, Hkv, d))
    qbar = O.gqa_summary_query(q[-1:], Hkv)
    cs = O.gqa_condense(qbar, k, v, 1, 3, scale)
    k_rep = np.stack([k[cs["anchor"][:, h], h] for h in range(Hkv)], axis=1)
    out, _ = O.gqa_prefill_rows(q, np.arange(L), k, v, k_rep, cs["v_rep"], 1, 3, scale)
    for h in range(Hq):
        ref = np_dense_causal(q[:, h:h + 1], k[:, h // 2], v[:, h // 2], scale)
        np.testing.assert_allclose(out[:, h], ref[:, 0], atol=1e-12)


def test_gqa_decode_maps_each_query_head_to_its_kv_head():
    # Sec. 5.4 decode: query head h reads KV head h // (Hq / Hkv).  Three query heads per KV head and
    # keys / values that differ strongly per KV head, so a wrong mapping (h % Hkv, transposed cache,
    # shared head) fails; the bias applies to the leading n_rep rows only.
    rng = RNG(42)
    rows, Hq, Hkv, d, n_rep, scale, bias = 23, 6, 2, 5, 4, 0.37, 0.6
    q = rng.standard_normal((Hq, d))
    ck = rng.standard_normal((rows, Hkv, d)) + np.array([0.0, 3.0])[None, :, None]
    cv = rng.standard_normal((rows, Hkv, d)) * np.array([1.0, -2.0])[None, :, None]
    out, lse = O.gqa_decode(q, ck, cv, n_rep, scale, bias)
    assert out.shape == (Hq, d) and lse.shape == (Hq,)
    for h in range(Hq):
        kv = h // (Hq // Hkv)
        lg = ck[:, kv] @ q[h] * scale
        lg[:n_rep] += bias
        np.testing.assert_allclose(out[h], np_softmax(lg) @ cv[:, kv], atol=1e-13)
        assert abs(lse[h] - np.log(np.exp(lg).sum())) < 1e-12


def test_gqa_decode_equals_last_prefill_row():
    # Decoding the last token against the cache [representatives ; last k tokens] of the same sequence
    # is the last row of the prefill (Sec. 4.3 / 5.4), for every query head.
    rng = RNG(43)
    L, Hq, Hkv, d, g, w, scale = 31, 6, 2, 4, 4, 5, 0.5
    q = rng.standard_normal((L, Hq, d))
    k = rng.standard_normal((L, Hkv, d)) + np.array([0.0, 1.5])[None, :, None]
    v = rng.standard_normal((L, Hkv, d))
    qbar = O.gqa_summary_query(q[-g:], Hkv)
    cs = O.gqa_condense(qbar, k, v, g, w, scale)
    m, kk = cs["m"], cs["k"]
    assert m > 0
    k_rep = np.stack([k[cs["anchor"][:, h], h] for h in range(Hkv)], axis=1)
    cache_k = np.concatenate([k_rep, k[L - kk:]], axis=0)
    cache_v = np.concatenate([cs["v_rep"], v[L - kk:]], axis=0)
    out_d, lse_d = O.gqa_decode(q[-1], cache_k, cache_v, m, scale, 0.3)
    out_p, lse_p = O.gqa_prefill_rows(q[-1:], np.array([L - 1]), k, v, k_rep, cs["v_rep"], g, w, scale, 0.3)
    np.testing.assert_allclose(out_d, out_p[0], atol=1e-12)
    np.testing.assert_allclose(lse_d, lse_p[0], atol=1e-12)


def test_gqa_condense_selects_keys_and_pools_values():
    rng = RNG(15)
    L, Hq, Hkv, d, g, w, scale = 29, 4, 2, 5, 4, 3, 0.6
    q = rng.standard_normal((L, Hq, d))
    k = rng.standard_normal((L, Hkv, d))
    v = rng.standard_normal((L, Hkv, d))
    qbar = O.gqa_summary_query(q[-g:], Hkv)
    np.testing.assert_allclose(qbar[1], q[-g:, 2:4].reshape(-1, d).mean(0), atol=1e-15)
    cs = O.gqa_condense(qbar, k, v, g, w, scale)
    m = cs["m"]
    assert m == (L - w) // g
    for h in range(Hkv):
        for j in range(m):
            s = k[j * g:(j + 1) * g, h] @ qbar[h] * scale
            assert cs["anchor"][j, h] == j * g + int(np.argmax(s))
            np.testing.assert_allclose(cs["v_rep"][j, h], np_softmax(s) @ v[j * g:(j + 1) * g, h], atol=1e-13)
    # cache layout: representatives first (selected key, pooled value), then the last k tokens
    kk = cs["k"]
    ck = O.bits_to_f64(cs["cache_k_bits"])
    assert ck.shape == (m + kk, Hkv, d)


def test_mla_cache_layout_and_bit_exact_copies():
    torch = pytest.importorskip("torch")
    rng = RNG(16)
    L, dc, dr, g, w = 50, 8, 4, 4, 6
    C = torch.from_numpy(rng.standard_normal((L, dc))).to(torch.bfloat16)
    KR = torch.from_numpy(rng.standard_normal((L, dr))).to(torch.bfloat16)
    Cb, KRb = O.torch_bf16_to_bits(C), O.torch_bf16_to_bits(KR)
    qbar = rng.standard_normal(dc + dr)
    r = O.mla_condense(qbar, O.bits_to_f64(Cb), O.bits_to_f64(KRb), g, w, 0.5)
    m, k = r["m"], r["k"]
    assert r["cache_sem_bits"].shape == (m + k, dc) and r["cache_pos_bits"].shape == (m + k, dr)
    assert np.array_equal(r["cache_sem_bits"][m:], Cb[L - k:])          # local tail copied bit-exactly
    assert np.array_equal(r["cache_pos_bits"][m:], KRb[L - k:])
    assert np.array_equal(r["cache_pos_bits"][:m], KRb[r["anchor"]])    # anchors copied bit-exactly
    assert np.array_equal(r["cache_sem_bits"][:m], O.round_bf16_bits(r["c_rep"]))


def test_online_cache_update_reproduces_alg1_on_the_longer_sequence():
    """Streaming (Sec. 4.3) against Alg. 1: feed tokens one at a time and condense whenever the buffer
    reaches w + g tokens.  With one fixed summary query for every update the cache after T more tokens
    must equal the cache Alg. 1 builds from scratch on the longer sequence with that summary query:
    same representatives, same anchors, same tokens in the window, nothing lost or duplicated."""
    rng = RNG(21)
    g, w, dc, dr = 4, 6, 8, 4
    L0, T = w + 2 * g + 3, 3 * g + 2
    import torch
    C = torch.from_numpy(rng.standard_normal((L0 + T, dc))).bfloat16()
    KR = torch.from_numpy(rng.standard_normal((L0 + T, dr))).bfloat16()
    Cb, KRb = O.torch_bf16_to_bits(C), O.torch_bf16_to_bits(KR)
    qbar = rng.standard_normal(dc + dr)
    scale = 0.3
    start = O.mla_condense(qbar, O.bits_to_f64(Cb[:L0]), O.bits_to_f64(KRb[:L0]), g, w, scale)
    sem, pos = start["cache_sem_bits"], start["cache_pos_bits"]
    n_rep, n_rows = start["m"], start["m"] + start["k"]
    sizes = []
    for t in range(L0, L0 + T):
        sem = np.concatenate([sem[:n_rows], Cb[t:t + 1]], axis=0)          # the new token's row
        pos = np.concatenate([pos[:n_rows], KRb[t:t + 1]], axis=0)
        n_rows += 1
        sem, pos, n_rep, n_rows, _ = O.mla_decode_update(sem, pos, n_rep, n_rows, qbar, g, w, scale)
        sizes.append(n_rows - n_rep)
        whole = O.mla_condense(qbar, O.bits_to_f64(Cb[:t + 1]), O.bits_to_f64(KRb[:t + 1]), g, w, scale)
        assert n_rep == whole["m"] and n_rows == whole["m"] + whole["k"]
        assert np.array_equal(sem[:n_rows], whole["cache_sem_bits"])
        assert np.array_equal(pos[:n_rows], whole["cache_pos_bits"])
    assert min(sizes) == w and max(sizes) == w + g - 1                       # the buffer breathes between w and w+g-1


def test_online_cache_update_waits_for_a_full_group_and_zero_query_gives_the_mean():
    rng = RNG(22)
    g, w, dc, dr = 4, 3, 6, 2
    import torch
    rows = w + g
    sem = O.torch_bf16_to_bits(torch.from_numpy(rng.standard_normal((rows, dc))).bfloat16())
    pos = O.torch_bf16_to_bits(torch.from_numpy(rng.standard_normal((rows, dr))).bfloat16())
    # one token short: untouched
    s2, p2, nr, nrows, ia = O.mla_decode_update(sem[:-1], pos[:-1], 0, rows - 1, np.zeros(dc + dr), g, w, 1.0)
    assert ia == -1 and nr == 0 and nrows == rows - 1 and s2 is sem[:-1].base or np.array_equal(s2, sem[:-1])
    # threshold reached, q_bar = 0: uniform weights -> mean of the earliest g tokens, anchor = first of them
    s3, p3, nr, nrows, ia = O.mla_decode_update(sem, pos, 0, rows, np.zeros(dc + dr), g, w, 1.0)
    assert (nr, nrows, ia) == (1, w + 1, 0)
    mean = O.bits_to_f64(sem[:g]).mean(axis=0)
    assert np.array_equal(s3[0], O.round_bf16_bits(mean))
    assert np.array_equal(p3[0], pos[0]) and np.array_equal(s3[1:], sem[g:]) and np.array_equal(p3[1:], pos[g:])


def test_ring_layout_streaming_reproduces_alg1_on_the_longer_sequence():
    """The ring layout of the decode cache (token n at row n % (w + g), representatives behind the ring) against
    Alg. 1: start from the packed cache of a prefix, append tokens at their ring rows, update whenever w + g tokens
    are uncondensed.  After every token the rows that take part, read in the order [representatives ; tokens], must
    be the cache Alg. 1 builds from scratch on the longer sequence; the ring wraps several times on the way, and no
    row other than the new representative's changes in an update."""
    rng = RNG(23)
    g, w, dc, dr = 4, 8, 8, 4
    R = w + g
    L0, T = w + 2 * g + 3, 4 * R + 5
    import torch
    C = torch.from_numpy(rng.standard_normal((L0 + T, dc))).bfloat16()
    KR = torch.from_numpy(rng.standard_normal((L0 + T, dr))).bfloat16()
    Cb, KRb = O.torch_bf16_to_bits(C), O.torch_bf16_to_bits(KR)
    qbar = rng.standard_normal(dc + dr)
    scale = 0.3
    start = O.mla_condense(qbar, O.bits_to_f64(Cb[:L0]), O.bits_to_f64(KRb[:L0]), g, w, scale)
    cap = R + (L0 + T) // g + 1
    sem, pos, n_tok = O.ring_from_packed(start["cache_sem_bits"], start["cache_pos_bits"], start["m"],
                                         start["m"] + start["k"], g, w, cap)
    n_rep = start["m"]
    assert n_tok == L0
    back = O.ring_to_packed(sem, pos, n_rep, n_tok, g, w)
    assert back[2] == start["m"] + start["k"]
    assert np.array_equal(back[0], start["cache_sem_bits"]) and np.array_equal(back[1], start["cache_pos_bits"])
    n_updates = 0
    for t in range(L0, L0 + T):
        sem[t % R], pos[t % R] = Cb[t], KRb[t]                             # the new token's row
        n_tok += 1
        before = (sem.copy(), pos.copy())
        sem, pos, n_rep2, ia = O.mla_decode_update_ring(sem, pos, n_rep, n_tok, qbar, g, w, scale)
        if ia >= 0:
            n_updates += 1
            changed = np.flatnonzero((sem != before[0]).any(axis=1) | (pos != before[1]).any(axis=1))
            assert set(changed) <= {R + n_rep} and n_rep2 == n_rep + 1
        else:
            assert n_rep2 == n_rep and np.array_equal(sem, before[0]) and np.array_equal(pos, before[1])
        n_rep = n_rep2
        whole = O.mla_condense(qbar, O.bits_to_f64(Cb[:t + 1]), O.bits_to_f64(KRb[:t + 1]), g, w, scale)
        psem, ppos, n_rows = O.ring_to_packed(sem, pos, n_rep, n_tok, g, w)
        assert n_rep == whole["m"] and n_rows == whole["m"] + whole["k"]
        assert np.array_equal(psem, whole["cache_sem_bits"]) and np.array_equal(ppos, whole["cache_pos_bits"])
    assert n_updates == (L0 + T - w) // g - start["m"] and n_updates >= 4 * R // g


def test_gqa_ring_streaming_reproduces_the_condensation_of_the_longer_sequence():
    """GQA variant of the online update (Sec. 5.4 with Sec. 4.3) on the ring layout: per KV head the anchor key is selected
    and the values are pooled.  Streaming token by token from the packed cache of a prefix must give, after every token, the
    cache gqa_condense builds from scratch on the longer sequence (per head: its own scores, its own anchors)."""
    rng = RNG(24)
    g, w, d, hkv = 4, 8, 6, 3
    R = w + g
    L0, T = w + g + 2, 2 * R + 3
    import torch
    K = torch.from_numpy(rng.standard_normal((L0 + T, hkv, d))).bfloat16()
    V = torch.from_numpy(rng.standard_normal((L0 + T, hkv, d))).bfloat16()
    Kb, Vb = O.torch_bf16_to_bits(K), O.torch_bf16_to_bits(V)
    qbar = rng.standard_normal((hkv, d))
    scale = 0.4
    start = O.gqa_condense(qbar, O.bits_to_f64(Kb[:L0]), O.bits_to_f64(Vb[:L0]), g, w, scale)
    cap = R + (L0 + T) // g + 1
    # ring_from_packed treats the trailing dimensions as one row: the same for [rows, Hkv, d]
    rk, rv, n_tok = O.ring_from_packed(start["cache_k_bits"], start["cache_v_bits"], start["m"], start["m"] + start["k"], g, w, cap)
    n_rep = start["m"]
    n_updates = 0
    for t in range(L0, L0 + T):
        rk[t % R], rv[t % R] = Kb[t], Vb[t]
        n_tok += 1
        rk, rv, n_rep, anchors = O.gqa_decode_update_ring(rk, rv, n_rep, n_tok, qbar, g, w, scale)
        whole = O.gqa_condense(qbar, O.bits_to_f64(Kb[:t + 1]), O.bits_to_f64(Vb[:t + 1]), g, w, scale)
        pk, pv, n_rows = O.ring_to_packed(rk, rv, n_rep, n_tok, g, w)
        assert n_rep == whole["m"] and n_rows == whole["m"] + whole["k"]
        assert np.array_equal(pk, whole["cache_k_bits"]) and np.array_equal(pv, whole["cache_v_bits"])
        if anchors is not None:
            n_updates += 1
            assert np.array_equal(anchors, whole["anchor"][-1] - (n_rep - 1) * g)     # offsets inside the newest group, per head
    assert n_updates == (L0 + T - w) // g - start["m"] and n_updates >= 5


def test_ablation_reducers_have_their_defining_properties():
    """Table 5 operators: the method's pair is the default; mean pooling is weighted pooling at a zero
    summary query; max selection returns a member of the group bit for bit; max pooling dominates every
    member coordinate-wise and is attained; weighted pooling of the rope keys stays in their hull."""
    rng = RNG(31)
    L, g, w, dc, dr = 70, 8, 6, 5, 4
    C, KR = rng.standard_normal((L, dc)), rng.standard_normal((L, dr))
    qbar = rng.standard_normal(dc + dr)
    base = O.mla_condense(qbar, C, KR, g, w, 0.4)
    m = base["m"]
    same = O.mla_condense(qbar, C, KR, g, w, 0.4, "weighted", "maxsel")
    assert np.array_equal(base["cache_sem_bits"], same["cache_sem_bits"]) and np.array_equal(base["cache_pos_bits"], same["cache_pos_bits"])
    mean = O.mla_condense(qbar, C, KR, g, w, 0.4, "meanpool", "meanpool")
    zero = O.mla_condense(np.zeros(dc + dr), C, KR, g, w, 0.4, "weighted", "weighted")
    np.testing.assert_allclose(mean["c_rep"], zero["c_rep"], rtol=1e-13, atol=1e-15)
    sel = O.mla_condense(qbar, C, KR, g, w, 0.4, "maxsel", "maxsel")
    mx = O.mla_condense(qbar, C, KR, g, w, 0.4, "maxpool", "maxpool")
    wk = O.mla_condense(qbar, C, KR, g, w, 0.4, "weighted", "weighted")
    for j in range(m):
        grp, grk = C[j * g:(j + 1) * g], KR[j * g:(j + 1) * g]
        assert np.array_equal(sel["c_rep"][j], C[base["anchor"][j]])
        assert (mx["c_rep"][j] >= grp).all() and all(mx["c_rep"][j][c] in grp[:, c] for c in range(dc))
        kw = O.bits_to_f64(wk["cache_pos_bits"][j])
        assert (kw >= grk.min(axis=0) - 0.02).all() and (kw <= grk.max(axis=0) + 0.02).all()
    # anchors do not depend on the reducers
    assert np.array_equal(mx["anchor"], base["anchor"]) and np.array_equal(mean["anchor"], base["anchor"])
