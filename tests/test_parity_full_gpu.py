"""GPU parity at the full benchmark sizes, in the launch configuration bench.py times.

The oracle cannot compute 131072 x 128 output rows, so the condensed cache is compared in full
(anchors, copied rows, representatives) and the attention output on a stratified sample of query
positions (window / group boundaries, both ends, seeded uniform positions) with all heads.
"""
import numpy as np
import pytest
import torch

from oracle import lca_oracle as O
from paper_2604_12452_b200 import inputs as I
from tests import helpers as Hh

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def B():
    from paper_2604_12452_b200 import build
    build.build()
    from paper_2604_12452_b200 import binding
    return binding


def one_seq(cond, b=0):
    r = dict(cond)
    for key in ("cache_sem", "cache_pos", "anchor_idx"):
        r[key] = cond[key][b]
    return r


def check_mla_full(B, name, n_uniform):
    cfg = I.CONFIGS[name]
    L, g, w = cfg.seq_len, cfg.group_size, cfg.window
    inp = I.make_mla_inputs(cfg, DEV)
    p = B.params_from_config(cfg, batch=1)
    cond = B.condense(p, inp["q_sem"][L - g:], inp["q_pos"][L - g:], inp["ckv"], inp["kr"])
    out, lse = B.prefill_attention(p, inp["q_sem"], inp["q_pos"], inp["ckv"], inp["kr"], cond["cache_sem"],
                                   cond["cache_pos"], want_lse=True)
    torch.cuda.synchronize()
    assert B.lca_last_device_status() == 0
    needles = [int(x) for x in I.needle_positions(cfg)]
    extra = [n + d for n in needles[:4] for d in (-1, 0, 1)] + [8191, 8192, 8193]
    rows = Hh.sample_positions(L, g, w, extra=extra, n_uniform=n_uniform, seed=3)
    idx = torch.from_numpy(rows).to(DEV)
    ref = Hh.oracle_mla_sampled(inp["ckv"].cpu(), inp["kr"].cpu(), inp["q_sem"][L - g:].cpu(), inp["q_pos"][L - g:].cpu(),
                                inp["q_sem"][idx].cpu(), inp["q_pos"][idx].cpu(), rows, g, w, cfg.softmax_scale)
    Hh.check_condense(one_seq(cond), ref["cond"])
    st = Hh.check_outputs(out[0][idx], ref, f"{name} sampled rows")
    np.testing.assert_allclose(lse[0][idx].cpu().numpy(), ref["lse"], atol=2e-3, rtol=1e-4)
    return st


def test_config2_mla_32k_full_size(B):
    check_mla_full(B, "mla_32k", n_uniform=40)


def test_config3_mla_128k_full_size(B):
    check_mla_full(B, "mla_128k", n_uniform=24)


def test_long_context_256k_with_the_paper_default_group_and_window(B):
    # The scaling run's shape (V2-Lite-like layer, g = 16, w = 1024) at 262144 tokens: 16320 representatives, query
    # rows far beyond 2^17, the cache compared in full, sampled rows (the last one included) on every head.
    cfg = I.scaled(I.CONFIGS["mla_32k"], name="v2lite_256k", seq_len=262144, group_size=16, window=1024, needle_every=4096)
    L, g, w = cfg.seq_len, cfg.group_size, cfg.window
    inp = I.make_mla_inputs(cfg, DEV)
    p = B.params_from_config(cfg, batch=1)
    cond = B.condense(p, inp["q_sem"][L - g:], inp["q_pos"][L - g:], inp["ckv"], inp["kr"])
    assert cond["m"] == (L - w) // g == 16320
    out, lse = B.prefill_attention(p, inp["q_sem"], inp["q_pos"], inp["ckv"], inp["kr"], cond["cache_sem"],
                                   cond["cache_pos"], want_lse=True)
    torch.cuda.synchronize()
    assert B.lca_last_device_status() == 0
    rows = Hh.sample_positions(L, g, w, extra=[131071, 131072, 131073, 200000, L - 17, L - 16], n_uniform=24, seed=9)
    assert rows[-1] == L - 1
    idx = torch.from_numpy(rows).to(DEV)
    ref = Hh.oracle_mla_sampled(inp["ckv"].cpu(), inp["kr"].cpu(), inp["q_sem"][L - g:].cpu(), inp["q_pos"][L - g:].cpu(),
                                inp["q_sem"][idx].cpu(), inp["q_pos"][idx].cpu(), rows, g, w, cfg.softmax_scale)
    Hh.check_condense(one_seq(cond), ref["cond"])
    Hh.check_outputs(out[0][idx], ref, "256k sampled rows")
    np.testing.assert_allclose(lse[0][idx].cpu().numpy(), ref["lse"], atol=2e-3, rtol=1e-4)


def test_config5_gqa_64k_full_size(B):
    cfg = I.CONFIGS["gqa_64k"]
    L, g, w = cfg.seq_len, cfg.group_size, cfg.window
    inp = I.make_gqa_inputs(cfg, DEV)
    p = B.params_from_config(cfg, batch=1)
    cond = B.condense(p, None, inp["q"][L - g:], inp["v"], inp["k"])
    out, _ = B.prefill_attention(p, None, inp["q"], inp["v"], inp["k"], cond["cache_sem"], cond["cache_pos"])
    torch.cuda.synchronize()
    assert B.lca_last_device_status() == 0
    rows = Hh.sample_positions(L, g, w, n_uniform=24, seed=5)
    idx = torch.from_numpy(rows).to(DEV)
    k64, v64 = O.torch_bf16_to_f64(inp["k"].cpu()), O.torch_bf16_to_f64(inp["v"].cpu())
    qbar = O.gqa_summary_query(O.torch_bf16_to_f64(inp["q"][L - g:].cpu()), cfg.n_kv_heads)
    rc = O.gqa_condense(qbar, k64, v64, g, w, Hh.f32(cfg.softmax_scale))
    Hh.check_condense(one_seq(cond), rc, kind="gqa")
    m = rc["m"]
    ro, _ = O.gqa_prefill_rows(O.torch_bf16_to_f64(inp["q"][idx].cpu()), rows, k64, v64, O.bits_to_f64(rc["cache_k_bits"][:m]),
                               O.bits_to_f64(rc["cache_v_bits"][:m]), g, w, Hh.f32(cfg.softmax_scale))
    Hh.check_outputs(out[0][idx], ro, "gqa_64k sampled rows")


def test_config4_batched_condense_and_decode_full_size(B):
    cfg = I.CONFIGS["mla_decode"]
    Bsz, L, g, w, H = cfg.batch, cfg.seq_len, cfg.group_size, cfg.window, cfg.n_q_heads
    ckv = torch.empty((Bsz, L, 512), dtype=torch.bfloat16, device=DEV)
    kr = torch.empty((Bsz, L, 64), dtype=torch.bfloat16, device=DEV)
    qts = torch.empty((Bsz, g, H, 512), dtype=torch.bfloat16, device=DEV)
    qtp = torch.empty((Bsz, g, H, 64), dtype=torch.bfloat16, device=DEV)
    for b in range(Bsz):
        one = I.make_mla_inputs(cfg, DEV, batch_index=b, q_positions=slice(L - g, L))
        ckv[b], kr[b], qts[b], qtp[b] = one["ckv"], one["kr"], one["q_sem"], one["q_pos"]
    p = B.params_from_config(cfg, batch=Bsz)
    m, k = B.lca_partition(p)
    cond = B.condense(p, qts, qtp, ckv, kr)
    cap = m + k + 1
    dsem = torch.zeros((Bsz, cap, 1, 512), dtype=torch.bfloat16, device=DEV)
    dpos = torch.zeros((Bsz, cap, 1, 64), dtype=torch.bfloat16, device=DEV)
    dsem[:, :m + k] = cond["cache_sem"]
    dpos[:, :m + k] = cond["cache_pos"]
    gen = torch.Generator(device=DEV)
    gen.manual_seed(77)
    dsem[:, m + k] = torch.randn((Bsz, 1, 512), generator=gen, device=DEV).bfloat16()
    dpos[:, m + k] = torch.randn((Bsz, 1, 64), generator=gen, device=DEV).bfloat16()
    qs = torch.randn((Bsz, H, 512), generator=gen, device=DEV).bfloat16()
    qp = torch.randn((Bsz, H, 64), generator=gen, device=DEV).bfloat16()
    rows = torch.full((Bsz,), cap, dtype=torch.int32, device=DEV)
    out, lse = B.decode_attention(p, qs, qp, dsem, dpos, rows, m, want_lse=True)
    torch.cuda.synchronize()
    assert B.lca_last_device_status() == 0
    for b in (0, 1, 31, 63):
        qbar = O.mla_summary_query(O.torch_bf16_to_f64(qts[b].cpu()), O.torch_bf16_to_f64(qtp[b].cpu()))
        rc = O.mla_condense(qbar, O.torch_bf16_to_f64(ckv[b].cpu()), O.torch_bf16_to_f64(kr[b].cpu()), g, w, Hh.f32(cfg.softmax_scale))
        Hh.check_condense(one_seq(cond, b), rc)
        ro, rl = O.mla_decode(O.torch_bf16_to_f64(qs[b].cpu()), O.torch_bf16_to_f64(qp[b].cpu()), O.bits_to_f64(Hh.bits(dsem[b, :, 0])),
                              O.bits_to_f64(Hh.bits(dpos[b, :, 0])), m, Hh.f32(cfg.softmax_scale))
        Hh.check_outputs(out[b], ro, f"decode seq {b}")
        np.testing.assert_allclose(lse[b].cpu().numpy(), rl, atol=2e-3, rtol=1e-4)


def test_attention_is_bit_reproducible_at_full_size(B):
    # The kernels are deterministic (fixed tile order, no atomics in the data path), so two launches on the same
    # inputs must agree in every bit of the 16.8 M x 512 outputs of config 3: a missed ordering between the
    # softmax threads, the relay signal and the tensor core would show up here as a difference.
    cfg = I.CONFIGS["mla_128k"]
    L, g = cfg.seq_len, cfg.group_size
    inp = I.make_mla_inputs(cfg, DEV)
    p = B.params_from_config(cfg, batch=1)
    cond = B.condense(p, inp["q_sem"][L - g:], inp["q_pos"][L - g:], inp["ckv"], inp["kr"])
    args = (p, inp["q_sem"], inp["q_pos"], inp["ckv"], inp["kr"], cond["cache_sem"], cond["cache_pos"])
    out1, lse1 = B.prefill_attention(*args, want_lse=True)
    out2, lse2 = B.prefill_attention(*args, want_lse=True)
    torch.cuda.synchronize()
    assert B.lca_last_device_status() == 0
    step = 8192                                     # compare in slices: no second full-size temporary
    for t in range(0, L, step):
        assert torch.equal(Hh.bits_t(out1[0, t:t + step]), Hh.bits_t(out2[0, t:t + step])), f"tokens {t}..{t + step}"
    assert torch.equal(lse1, lse2)


def test_config4_ring_cache_update_and_decode_full_size(B):
    # The decode cache of config 4 in the ring layout (64 sequences, ring of w + g = 4160 rows, ~960 representatives):
    # sequences in four phases (ring full and due for an update, one token after an update, one token short of an update,
    # a few representatives fewer).  One update call with the query tails, then one decode call; four sequences against
    # the oracle (every row of the ring buffers, every head of the decode output).
    cfg = I.CONFIGS["mla_decode"]
    Bsz, g, w, H = cfg.batch, cfg.group_size, cfg.window, cfg.n_q_heads
    R = w + g
    m0 = 960
    cap = R + m0 + 8
    gen = torch.Generator(device=DEV)
    gen.manual_seed(91)
    specs = [[(m0, R), (m0, w + 1), (m0, R - 1), (m0 - 3, w + 17)][b % 4] for b in range(Bsz)]
    cap_packed = m0 + R
    psem = torch.randn((Bsz, cap_packed, 1, 512), generator=gen, device=DEV).bfloat16()
    ppos = torch.randn((Bsz, cap_packed, 1, 64), generator=gen, device=DEV).bfloat16()
    p = B.params_from_config(cfg, batch=Bsz)
    d_rep = torch.tensor([r for r, _ in specs], dtype=torch.int32, device=DEV)
    prow = torch.tensor([r + c for r, c in specs], dtype=torch.int32, device=DEV)
    rsem, rpos, d_tok = B.ring_from_packed(p, psem, ppos, prow, d_rep, cap)
    qts = torch.randn((Bsz, g, H, 512), generator=gen, device=DEV).bfloat16()
    qtp = torch.randn((Bsz, g, H, 64), generator=gen, device=DEV).bfloat16()
    before = {b: (Hh.bits(rsem[b, :, 0]), Hh.bits(rpos[b, :, 0])) for b in (0, 1, 2, 63)}
    anchor = B.decode_update_ring(p, qts, qtp, rsem, rpos, d_rep, d_tok)
    qs = torch.randn((Bsz, H, 512), generator=gen, device=DEV).bfloat16()
    qp = torch.randn((Bsz, H, 64), generator=gen, device=DEV).bfloat16()
    out, lse = B.decode_attention_ring(p, qs, qp, rsem, rpos, d_rep, d_tok, want_lse=True)
    torch.cuda.synchronize()
    assert B.lca_last_device_status() == 0
    n_rep_after, tok = d_rep.cpu().tolist(), d_tok.cpu().tolist()
    scale = Hh.f32(cfg.softmax_scale)
    for b in (0, 1, 2, 63):
        r, c = specs[b]
        assert tok[b] == r * g + c
        o_sem, o_pos, n = O.ring_from_packed(Hh.bits(psem[b, :r + c, 0]), Hh.bits(ppos[b, :r + c, 0]), r, r + c, g, w, cap)
        assert n == tok[b] and np.array_equal(before[b][0], o_sem) and np.array_equal(before[b][1], o_pos)
        qbar = O.mla_summary_query(O.torch_bf16_to_f64(qts[b].cpu()), O.torch_bf16_to_f64(qtp[b].cpu()))
        s2, p2, nr, ia = O.mla_decode_update_ring(o_sem, o_pos, r, tok[b], qbar, g, w, scale)
        assert int(anchor[b, 0]) == ia and n_rep_after[b] == nr and (ia >= 0) == (c == R)
        got_sem, got_pos = Hh.bits(rsem[b, :, 0]), Hh.bits(rpos[b, :, 0])
        assert np.array_equal(got_pos, p2)
        if ia >= 0:
            assert (Hh.bf16_ulp_distance(got_sem[R + r], s2[R + r]) <= 1).all()
            s2[R + r] = got_sem[R + r]
        assert np.array_equal(got_sem, s2)
        cs, cp, _ = O.ring_to_packed(s2, p2, nr, tok[b], g, w)
        ro, rl = O.mla_decode(O.torch_bf16_to_f64(qs[b].cpu()), O.torch_bf16_to_f64(qp[b].cpu()), O.bits_to_f64(cs), O.bits_to_f64(cp),
                              nr, scale)
        Hh.check_outputs(out[b], ro, f"ring decode seq {b}")
        np.testing.assert_allclose(lse[b].cpu().numpy(), rl, atol=2e-3, rtol=1e-4)
